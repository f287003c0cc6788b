// Plain-ALU tree-masked attention: one block per (node, head). Used by the fp32 configuration and
// as a debugging stand-in for the tensor-core kernel. Keys are the prefix slots 0..P-1 (all
// visible) followed by the tree nodes at slots P..P+n-1, of which node i sees only those whose
// bit is set in its ancestor-or-self row (Sec. 3.2 "Tree decoder": ones only at the earlier
// positions of the same branch). Masked keys get weight exactly zero. When a tree is extended the
// queries are only its new nodes q_first .. q_first + n - 1, the keys all n_tree nodes.
#include "common.cuh"

namespace llmcad {

constexpr int kAttnThreads = 128;

template <typename T>
__global__ void __launch_bounds__(kAttnThreads)
attention_simt_kernel(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v, int n_heads, int hd,
                      int kv_stride, int P, int n, int n_tree, int q_first, const uint32_t *__restrict__ anc, T *o,
                      const int32_t *status)
{
    pdl_launch_dependents();
    pdl_wait();
    if (*status) return;
    extern __shared__ float smem[];
    float *s_q = smem;              // [hd]
    float *s_p = smem + hd;         // [P + n] scores, then weights
    __shared__ float s_red[kAttnThreads / 32];
    __shared__ float s_acc[kAttnThreads];

    const int i = blockIdx.x, h = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_keys = P + n_tree;
    const float scale = rsqrtf((float)hd);
    const T *kh = k + (size_t)h * kv_stride * hd;
    const T *vh = v + (size_t)h * kv_stride * hd;

    for (int e = tid; e < hd; e += kAttnThreads) s_q[e] = to_f32<T>(q[((size_t)i * n_heads + h) * hd + e]);
    uint32_t my_anc[4];
    for (int w = 0; w < 4; ++w) my_anc[w] = anc[(q_first + i) * 4 + w];
    __syncthreads();

    // scores: one warp per key, lanes split the head dimension
    float mx = -INFINITY;
    for (int s = warp; s < n_keys; s += kAttnThreads / 32) {
        bool visible = true;
        if (s >= P) { const int j = s - P; visible = (my_anc[j >> 5] >> (j & 31)) & 1u; }
        float sc = -INFINITY;
        if (visible) {
            float acc = 0.f;
            for (int e = lane; e < hd; e += 32) acc = fmaf(s_q[e], to_f32<T>(kh[(size_t)s * hd + e]), acc);
            for (int o2 = 16; o2; o2 >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o2);
            sc = acc * scale;
        }
        if (lane == 0) s_p[s] = sc;
        mx = fmaxf(mx, sc);
    }
    if (lane == 0) s_red[warp] = mx;
    __syncthreads();
    mx = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
    __syncthreads();

    float sum = 0.f;
    for (int s = tid; s < n_keys; s += kAttnThreads) {
        const float sc = s_p[s];
        const float p = (sc == -INFINITY) ? 0.f : expf(sc - mx);
        s_p[s] = p;
        sum += p;
    }
    for (int o2 = 16; o2; o2 >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o2);
    if (lane == 0) s_red[warp] = sum;
    __syncthreads();
    const float inv = 1.0f / (s_red[0] + s_red[1] + s_red[2] + s_red[3]);

    // output: thread (part, e) sums keys s = part (mod parts)
    const int parts = kAttnThreads / hd;  // hd is 64 or 128
    const int e = tid % hd, part = tid / hd;
    float acc = 0.f;
    for (int s = part; s < n_keys; s += parts) {
        const float p = s_p[s];
        if (p != 0.f) acc = fmaf(p, to_f32<T>(vh[(size_t)s * hd + e]), acc);
    }
    s_acc[tid] = acc;
    __syncthreads();
    if (part == 0) {
        for (int pp = 1; pp < parts; ++pp) acc += s_acc[pp * hd + e];
        o[((size_t)i * n_heads + h) * hd + e] = from_f32<T>(acc * inv);
    }
}

cudaError_t launch_attention_simt(const void *q, const void *k, const void *v, int dtype, int n_heads, int hd,
                                  int kv_stride, int P, int n, const uint32_t *anc, void *o, const int32_t *status,
                                  cudaStream_t st, int n_tree, int q_first)
{
    if (n_tree <= 0) n_tree = n;
    const size_t smem = sizeof(float) * (size_t)(hd + P + n_tree);
    dim3 grid(n, n_heads);
    if (dtype == LLMCAD_F32) {
        if (smem > 48 * 1024)
            cudaFuncSetAttribute(attention_simt_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        LaunchCfg lc(grid, kAttnThreads, smem, st);
        return cudaLaunchKernelEx(&lc.cfg, attention_simt_kernel<float>, (const float *)q, (const float *)k,
                                  (const float *)v, n_heads, hd, kv_stride, P, n, n_tree, q_first, anc, (float *)o, status);
    } else {
        if (smem > 48 * 1024)
            cudaFuncSetAttribute(attention_simt_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        LaunchCfg lc(grid, kAttnThreads, smem, st);
        return cudaLaunchKernelEx(&lc.cfg, attention_simt_kernel<__nv_bfloat16>, (const __nv_bfloat16 *)q,
                                  (const __nv_bfloat16 *)k, (const __nv_bfloat16 *)v, n_heads, hd, kv_stride, P, n, n_tree, q_first,
                                  anc, (__nv_bfloat16 *)o, status);
    }
}

}  // namespace llmcad
