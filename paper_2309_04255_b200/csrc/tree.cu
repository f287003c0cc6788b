// Integer side of the pass: mask table, embedding gather, argmax, verified-path search,
// cache rollback. Everything here is bit-exact by construction.
#include "common.cuh"

namespace llmcad {

// ------------------------------------------------------------------------------------------
// Mask table (Sec. 3.2 "Tree decoder"): block i handles node i. Thread 0 walks from the node to
// the root, checking every link it uses (0 <= parent < child, root has -1), which yields the
// node's depth and its ancestor-or-self bit row. All threads then fill the node's rotary table
// row at position prefix_len + depth in fp64.
__global__ void tree_prep_kernel(const int32_t *__restrict__ parent, const int32_t *__restrict__ tokens, int n, int P,
                                 int vocab, int hd, double rope_base, int32_t *depth, int32_t *pos, uint32_t *anc,
                                 float2 *rope_cs, int32_t *status)
{
    __shared__ int s_depth;
    const int i = blockIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x == 0) {
        uint32_t bits[4] = {0, 0, 0, 0};
        int d = 0, cur = i, err = 0;
        if (tokens != nullptr && (tokens[i] < 0 || tokens[i] >= vocab)) err = LLMCAD_ERR_BAD_TOKEN;
        // cur strictly decreases, so the walk ends within n steps whatever the array holds
        while (true) {
            bits[cur >> 5] |= 1u << (cur & 31);
            const int p = parent[cur];
            if (cur == 0) {
                if (p != -1) err = LLMCAD_ERR_BAD_TREE;
                break;
            }
            if (p < 0 || p >= cur) { err = LLMCAD_ERR_BAD_TREE; break; }
            cur = p;
            ++d;
        }
        if (err) atomicCAS(status, 0, err);
        depth[i] = d;
        pos[i] = P + d;
        for (int w = 0; w < 4; ++w) anc[i * 4 + w] = bits[w];
        s_depth = d;
    }
    __syncthreads();
    if (rope_cs != nullptr) {
        const double p = (double)(P + s_depth);
        for (int t = threadIdx.x; t < hd / 2; t += blockDim.x) {
            const double ang = p * pow(rope_base, -2.0 * t / hd);
            double sn, cs;
            sincos(ang, &sn, &cs);
            rope_cs[(size_t)i * (hd / 2) + t] = make_float2((float)cs, (float)sn);
        }
    }
}

cudaError_t launch_tree_prep(const int32_t *parent, const int32_t *tokens, int n, int P, int vocab, int hd,
                             float rope_base, TreeBuffers tb, int32_t *status, cudaStream_t st)
{
    LaunchCfg lc(n, 64, 0, st);
    return cudaLaunchKernelEx(&lc.cfg, tree_prep_kernel, parent, tokens, n, P, vocab, hd, (double)rope_base, tb.depth,
                              tb.pos, tb.anc, tb.rope_cs, status);
}

// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void embed_kernel(const T *__restrict__ E, const int32_t *__restrict__ tokens, int d, float *x,
                             const int32_t *status)
{
    pdl_launch_dependents();
    pdl_wait();
    if (*status) return;
    const int i = blockIdx.x;
    const T *row = E + (size_t)tokens[i] * d;
    for (int k = threadIdx.x; k < d; k += blockDim.x) x[(size_t)i * d + k] = to_f32<T>(row[k]);
}

cudaError_t launch_embed(const void *E, int dtype, const int32_t *tokens, int n, int d, float *x, const int32_t *status,
                         cudaStream_t st)
{
    LaunchCfg lc(n, 256, 0, st);
    if (dtype == LLMCAD_F32) return cudaLaunchKernelEx(&lc.cfg, embed_kernel<float>, (const float *)E, tokens, d, x, status);
    return cudaLaunchKernelEx(&lc.cfg, embed_kernel<__nv_bfloat16>, (const __nv_bfloat16 *)E, tokens, d, x, status);
}

// Embedding gather for the tensor-core path, where the first RMSNorm is folded into the QKV GEMM:
// besides x it writes gain * x in the GEMM input dtype (hi and, if comp, lo plane) and the row's
// sum of squares.
template <typename T>
__global__ void __launch_bounds__(256)
embed_norm_kernel(const T *__restrict__ E, const int32_t *__restrict__ tokens, int d, const T *__restrict__ gain, float *x,
                  T *xg, float *ssq, int comp, const int32_t *status)
{
    pdl_launch_dependents();
    pdl_wait();
    if (*status) return;
    __shared__ float red[8];
    const int i = blockIdx.x;
    const T *row = E + (size_t)tokens[i] * d;
    float ss = 0.f;
    for (int k = threadIdx.x; k < d; k += 256) {
        const float v = to_f32<T>(row[k]);
        x[(size_t)i * d + k] = v;
        store_split<T>(xg + (size_t)i * d + k, (size_t)kLoRows * d, v * to_f32<T>(gain[k]), comp != 0);
        ss += v * v;
    }
    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += red[w];
        ssq[i] = t;
    }
}

cudaError_t launch_embed_norm(const void *E, const int32_t *tokens, int n, int d, const void *gain, float *x, void *xg,
                              float *ssq, int comp, const int32_t *status, cudaStream_t st)
{
    LaunchCfg lc(n, 256, 0, st);
    return cudaLaunchKernelEx(&lc.cfg, embed_norm_kernel<__nv_bfloat16>, (const __nv_bfloat16 *)E, tokens, d,
                              (const __nv_bfloat16 *)gain, x, (__nv_bfloat16 *)xg, ssq, comp, status);
}

// ------------------------------------------------------------------------------------------
// RMSNorm of the fp32 residual stream into the GEMM input dtype. One block per node; the row is
// read once with 16-byte loads and kept in registers between the reduction and the scaling
// (rows longer than 4 * kNormVec * blockDim fall back to re-reading).
constexpr int kNormThreads = 512;
constexpr int kNormVec = 4;   // float4 per thread held in registers -> d <= 8192

template <typename T> __device__ __forceinline__ void store4(T *p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float *p, float a, float b, float c, float d)
{
    *reinterpret_cast<float4 *>(p) = make_float4(a, b, c, d);
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16 *p, float a, float b, float c, float d)
{
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t *>(&lo);
    u.y = *reinterpret_cast<uint32_t *>(&hi);
    *reinterpret_cast<uint2 *>(p) = u;
}

template <typename T>
__global__ void __launch_bounds__(kNormThreads)
rmsnorm_kernel(const float *__restrict__ x, const T *__restrict__ g, int d, float eps, T *__restrict__ out,
               const int32_t *status)
{
    pdl_launch_dependents();
    pdl_wait();
    if (*status) return;
    __shared__ float red[kNormThreads / 32];
    const int i = blockIdx.x, tid = threadIdx.x;
    const float4 *xi = reinterpret_cast<const float4 *>(x + (size_t)i * d);
    const int nv = d >> 2;                      // d is a multiple of 8
    float4 r[kNormVec];
    float ss = 0.f;
#pragma unroll
    for (int u = 0; u < kNormVec; ++u) {
        const int k = tid + u * kNormThreads;
        r[u] = k < nv ? __ldcg(xi + k) : make_float4(0.f, 0.f, 0.f, 0.f);
        ss += r[u].x * r[u].x + r[u].y * r[u].y + r[u].z * r[u].z + r[u].w * r[u].w;
    }
    for (int k = tid + kNormVec * kNormThreads; k < nv; k += kNormThreads) {
        const float4 t = __ldcg(xi + k);
        ss += t.x * t.x + t.y * t.y + t.z * t.z + t.w * t.w;
    }
    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((tid & 31) == 0) red[tid >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kNormThreads / 32; ++w) tot += red[w];
    const float rs = rsqrtf(tot / d + eps);
    T *oi = out + (size_t)i * d;
#pragma unroll
    for (int u = 0; u < kNormVec; ++u) {
        const int k = tid + u * kNormThreads;
        if (k < nv) {
            const T *gk = g + 4 * k;
            store4<T>(oi + 4 * k, r[u].x * rs * to_f32<T>(gk[0]), r[u].y * rs * to_f32<T>(gk[1]),
                      r[u].z * rs * to_f32<T>(gk[2]), r[u].w * rs * to_f32<T>(gk[3]));
        }
    }
    for (int k = tid + kNormVec * kNormThreads; k < nv; k += kNormThreads) {
        const float4 t = __ldcg(xi + k);
        const T *gk = g + 4 * k;
        store4<T>(oi + 4 * k, t.x * rs * to_f32<T>(gk[0]), t.y * rs * to_f32<T>(gk[1]), t.z * rs * to_f32<T>(gk[2]),
                  t.w * rs * to_f32<T>(gk[3]));
    }
}

cudaError_t launch_rmsnorm(const float *x, const void *g, int dtype, int n, int d, float eps, void *out,
                           const int32_t *status, cudaStream_t st)
{
    LaunchCfg lc(n, kNormThreads, 0, st);
    if (dtype == LLMCAD_F32)
        return cudaLaunchKernelEx(&lc.cfg, rmsnorm_kernel<float>, x, (const float *)g, d, eps, (float *)out, status);
    return cudaLaunchKernelEx(&lc.cfg, rmsnorm_kernel<__nv_bfloat16>, x, (const __nv_bfloat16 *)g, d, eps,
                              (__nv_bfloat16 *)out, status);
}

// ------------------------------------------------------------------------------------------
// Greedy choice of the target at every node: lowest index of the maximum; a NaN sets status.
constexpr int kArgmaxThreads = 1024;

__device__ __forceinline__ void argmax_take(float v, int t, float &best, int &bi, bool &nan)
{
    nan |= (v != v);
    if (v > best || (v == best && t < bi)) { best = v; bi = t; }
}

__global__ void __launch_bounds__(kArgmaxThreads)
argmax_kernel(const float *__restrict__ logits, int vocab, int32_t *argmax, int32_t *status)
{
    pdl_launch_dependents();
    pdl_wait();
    if (*status) return;
    __shared__ float s_v[32];
    __shared__ int s_i[32];
    const int i = blockIdx.x;
    const float *row = logits + (size_t)i * vocab;
    float best = -INFINITY;
    int bi = 0x7fffffff;
    bool nan = false;
    if ((vocab & 3) == 0) {
        const float4 *r4 = reinterpret_cast<const float4 *>(row);
        for (int t = threadIdx.x; t < (vocab >> 2); t += kArgmaxThreads) {
            const float4 q = __ldcg(r4 + t);
            argmax_take(q.x, 4 * t, best, bi, nan);
            argmax_take(q.y, 4 * t + 1, best, bi, nan);
            argmax_take(q.z, 4 * t + 2, best, bi, nan);
            argmax_take(q.w, 4 * t + 3, best, bi, nan);
        }
    } else {
        for (int t = threadIdx.x; t < vocab; t += kArgmaxThreads) argmax_take(row[t], t, best, bi, nan);
    }
    if (nan) atomicCAS(status, 0, LLMCAD_ERR_NAN);
    for (int o = 16; o; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
    }
    if ((threadIdx.x & 31) == 0) { s_v[threadIdx.x >> 5] = best; s_i[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x < 32) {
        best = s_v[threadIdx.x];
        bi = s_i[threadIdx.x];
        for (int o = 16; o; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
        }
        if (threadIdx.x == 0) argmax[i] = (bi == 0x7fffffff) ? 0 : bi;
    }
}

cudaError_t launch_argmax(const float *logits, int n, int vocab, int32_t *argmax, int32_t *status, cudaStream_t st)
{
    LaunchCfg lc(n, kArgmaxThreads, 0, st);
    return cudaLaunchKernelEx(&lc.cfg, argmax_kernel, logits, vocab, argmax, status);
}

// ------------------------------------------------------------------------------------------
// Confidences of the generating side (Sec. 3.2: a candidate above a confidence threshold opens a
// branch): per node the k most probable next tokens and their softmax probabilities. One block
// per node: the row maximum and the sum of exponentials first, then k rounds of "largest logit
// not yet taken" (ties to the lower id). The row (vocab x 4 bytes) stays in L2 between the rounds.
constexpr int kTopkThreads = 1024;

__global__ void __launch_bounds__(kTopkThreads)
topk_softmax_kernel(const float *__restrict__ logits, int vocab, int k, int32_t *ids, float *probs, int32_t *status)
{
    pdl_launch_dependents();
    pdl_wait();
    if (*status) return;
    __shared__ float s_v[32];
    __shared__ int s_i[32];
    __shared__ float s_max, s_sum;
    __shared__ int s_taken[LLMCAD_MAX_TOPK];
    const int node = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float *row = logits + (size_t)node * vocab;

    auto block_max = [&](float v, int i, float &out_v, int &out_i) {     // argmax over the block, ties to the lower id
        for (int o = 16; o; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, v, o);
            const int oi = __shfl_xor_sync(0xffffffffu, i, o);
            if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
        }
        if (lane == 0) { s_v[warp] = v; s_i[warp] = i; }
        __syncthreads();
        if (warp == 0) {
            v = s_v[lane]; i = s_i[lane];
            for (int o = 16; o; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, v, o);
                const int oi = __shfl_xor_sync(0xffffffffu, i, o);
                if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
            }
            if (lane == 0) { s_v[0] = v; s_i[0] = i; }
        }
        __syncthreads();
        out_v = s_v[0]; out_i = s_i[0];
        __syncthreads();
    };

    // maximum (and NaN check), then the sum of exp(x - max)
    float best = -INFINITY;
    int bi = 0x7fffffff;
    bool nan = false;
    for (int t = tid; t < vocab; t += kTopkThreads) argmax_take(__ldcg(row + t), t, best, bi, nan);
    if (nan) atomicCAS(status, 0, LLMCAD_ERR_NAN);
    float mx; int mi;
    block_max(best, bi, mx, mi);
    float sum = 0.f;
    for (int t = tid; t < vocab; t += kTopkThreads) sum += expf(__ldcg(row + t) - mx);
    for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) s_v[warp] = sum;
    __syncthreads();
    if (tid == 0) {
        float t = 0.f;
        for (int w = 0; w < kTopkThreads / 32; ++w) t += s_v[w];
        s_sum = t; s_max = mx;
    }
    __syncthreads();
    const float inv = 1.0f / s_sum;

    for (int r = 0; r < k; ++r) {
        float v = -INFINITY;
        int vi = 0x7fffffff;
        for (int t = tid; t < vocab; t += kTopkThreads) {
            bool taken = false;
            for (int q = 0; q < r; ++q) taken |= (s_taken[q] == t);
            const float x = __ldcg(row + t);
            if (!taken && (x > v || (x == v && t < vi))) { v = x; vi = t; }
        }
        float bv; int bidx;
        block_max(v, vi, bv, bidx);
        if (tid == 0) {
            s_taken[r] = bidx;
            ids[(size_t)node * k + r] = bidx == 0x7fffffff ? 0 : bidx;
            probs[(size_t)node * k + r] = expf(bv - s_max) * inv;
        }
        __syncthreads();
    }
}

cudaError_t launch_topk_softmax(const float *logits, int n, int vocab, int k, int32_t *ids, float *probs, int32_t *status,
                                cudaStream_t st)
{
    LaunchCfg lc(n, kTopkThreads, 0, st);
    return cudaLaunchKernelEx(&lc.cfg, topk_softmax_kernel, logits, vocab, k, ids, probs, status);
}

// ------------------------------------------------------------------------------------------
// Verified-sequence search (Sec. 3.2 "Depth-first verified sequence searching"), data-parallel
// form: node c is verified iff every link on its root path is correct (the child's draft token
// equals the target's output at the parent). The verified sequence ends at the deepest verified
// node, ties to the lowest index. One block of 128 threads, thread c = node c.
__global__ void accept_kernel(const int32_t *__restrict__ parent, const int32_t *__restrict__ tokens,
                              const int32_t *__restrict__ argmax, int n, int P, int32_t *path, int32_t *scalars)
{
    __shared__ int s_par[LLMCAD_MAX_TREE];
    __shared__ unsigned char s_link[LLMCAD_MAX_TREE];
    __shared__ int s_key[4];
    __shared__ int s_best, s_haschild;
    const int c = threadIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    const int status = scalars[LLMCAD_S_STATUS];
    if (status) {  // an earlier phase failed: report an empty result, leave the cache as it was
        if (c == 0) {
            scalars[LLMCAD_S_ACCEPTED_LEN] = 0;
            scalars[LLMCAD_S_NEXT_TOKEN] = -1;
            scalars[LLMCAD_S_NEW_PREFIX_LEN] = P;
            scalars[LLMCAD_S_N_CORRECT] = 0;
            scalars[LLMCAD_S_N_ALL] = 0;
            scalars[LLMCAD_S_RECTIFIED] = 0;
            scalars[LLMCAD_S_RESERVED] = 0;
        }
        return;
    }
    if (c < n) {
        int p = parent[c];
        if (!LLMCAD_CHECK(c == 0 ? p == -1 : (p >= 0 && p < c), scalars + LLMCAD_S_STATUS)) p = c == 0 ? -1 : 0;
        s_par[c] = p;
        s_link[c] = (c == 0) ? 1 : (tokens[c] == argmax[p]);
    }
    if (c == 0) s_haschild = 0;
    __syncthreads();
    int key = -1, d = 0;
    if (c < n) {
        bool ok = true;
        for (int cur = c; cur > 0; cur = s_par[cur]) { ok &= (s_link[cur] != 0); ++d; }
        if (ok) key = (d << 8) | (LLMCAD_MAX_TREE - 1 - c);
    }
    int m = key;
    for (int o = 16; o; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    if ((c & 31) == 0) s_key[c >> 5] = m;
    __syncthreads();
    if (c == 0) {
        const int mm = max(max(s_key[0], s_key[1]), max(s_key[2], s_key[3]));
        s_best = LLMCAD_MAX_TREE - 1 - (mm & 0xff);
    }
    __syncthreads();
    const int best = s_best;
    // longest draft branch through the verified end node: deepest node that has it on its root path
    int below = -1;
    if (c < n) {
        for (int cur = c;; cur = s_par[cur]) {
            if (cur == best) { below = d; break; }
            if (cur <= 0 || cur < best) break;
        }
        if (c > 0 && s_par[c] == best) s_haschild = 1;
    }
    for (int o = 16; o; o >>= 1) below = max(below, __shfl_xor_sync(0xffffffffu, below, o));
    __syncthreads();
    if ((c & 31) == 0) s_key[c >> 5] = below;
    __syncthreads();
    if (c == 0) {
        int len = 1;
        for (int cur = best; cur > 0; cur = s_par[cur]) ++len;
        int j = len - 1;
        for (int cur = best; j >= 0; cur = s_par[cur], --j) path[j] = cur;
        scalars[LLMCAD_S_ACCEPTED_LEN] = len;
        scalars[LLMCAD_S_NEXT_TOKEN] = argmax[best];
        scalars[LLMCAD_S_NEW_PREFIX_LEN] = P + len;
        scalars[LLMCAD_S_N_CORRECT] = len - 1;
        scalars[LLMCAD_S_N_ALL] = max(max(s_key[0], s_key[1]), max(s_key[2], s_key[3]));
        scalars[LLMCAD_S_RECTIFIED] = s_haschild;
        scalars[LLMCAD_S_RESERVED] = 0;
    }
}

cudaError_t launch_accept(const int32_t *parent, const int32_t *tokens, const int32_t *argmax, int n, int P,
                          int32_t *path, int32_t *scalars, cudaStream_t st)
{
    LaunchCfg lc(1, LLMCAD_MAX_TREE, 0, st);
    return cudaLaunchKernelEx(&lc.cfg, accept_kernel, parent, tokens, argmax, n, P, path, scalars);
}

// ------------------------------------------------------------------------------------------
// Rollback (Sec. 3.2): for every layer, K and V, head: move the row at slot P+path[j] to slot P+j.
// path is strictly increasing with path[j] >= j, so for one fixed 16-byte column of one head an
// ascending copy never reads a slot it has already overwritten; each thread owns one such column
// and walks j upwards (eight rows are read before they are written to keep loads in flight).
__global__ void compact_kernel(uint4 *kv, int n_lkh, int S, int chunks, int P, const int32_t *__restrict__ path,
                               const int32_t *__restrict__ scalars)
{
    pdl_launch_dependents();
    pdl_wait();
    if (scalars[LLMCAD_S_STATUS]) return;
    int len = scalars[LLMCAD_S_ACCEPTED_LEN];
    if (!LLMCAD_CHECK(len >= 0 && P + len <= S && len <= LLMCAD_MAX_TREE, scalars + LLMCAD_S_STATUS)) len = 0;
    const long long w = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (w >= (long long)n_lkh * chunks) return;
    const int lkh = (int)(w / chunks), ch = (int)(w % chunks);
    uint4 *base = kv + ((size_t)lkh * S + P) * chunks + ch;
    int j0 = 0;
    while (j0 < len && path[j0] == j0) ++j0;  // rows already in place
    for (int j = j0; j < len; j += 8) {
        uint4 tmp[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (j + u < len && LLMCAD_CHECK(path[j + u] >= j + u && P + path[j + u] < S, scalars + LLMCAD_S_STATUS))
                tmp[u] = base[(size_t)path[j + u] * chunks];
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (j + u < len) base[(size_t)(j + u) * chunks] = tmp[u];
    }
}

cudaError_t launch_compact(void *kv, int dtype, int n_layers, int n_heads, int S, int hd, int P, const int32_t *path,
                           const int32_t *scalars, cudaStream_t st)
{
    const int elem = dtype == LLMCAD_F32 ? 4 : 2;
    const int chunks = hd * elem / 16;
    const int n_lkh = n_layers * 2 * n_heads;
    const long long total = (long long)n_lkh * chunks;
    const int block = 128;
    LaunchCfg lc((unsigned)((total + block - 1) / block), block, 0, st);
    return cudaLaunchKernelEx(&lc.cfg, compact_kernel, (uint4 *)kv, n_lkh, S, chunks, P, path, scalars);
}

}  // namespace llmcad
