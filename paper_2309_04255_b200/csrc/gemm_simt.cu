// Plain-ALU skinny GEMM: y[i][r] = sum_k W[r][k] x[i][k] for all tree nodes i, with the fused
// epilogues of common.cuh. It serves the fp32 configuration (whose 1e-4 tolerance rules out
// reduced-precision tensor-core inputs) and is a debugging stand-in for the tensor-core kernel on
// bf16. One warp owns a pair of output rows (the two rows of a rotary pair, or the gate and up
// rows of one FFN feature) and streams them once; lanes split the reduction dimension.
#include "common.cuh"

namespace llmcad {

template <typename T> struct Vec4;
template <> struct Vec4<float> {
    float4 v;
    __device__ __forceinline__ void load(const float *p) { v = *reinterpret_cast<const float4 *>(p); }
    __device__ __forceinline__ float get(int j) const { return j == 0 ? v.x : j == 1 ? v.y : j == 2 ? v.z : v.w; }
};
template <> struct Vec4<__nv_bfloat16> {
    uint2 v;
    __device__ __forceinline__ void load(const __nv_bfloat16 *p) { v = *reinterpret_cast<const uint2 *>(p); }
    __device__ __forceinline__ float get(int j) const
    {
        const uint32_t w = j < 2 ? v.x : v.y;
        return __uint_as_float((j & 1) ? (w & 0xffff0000u) : (w << 16));
    }
};

constexpr int kNodeChunk = 8;
constexpr int kWarpsPerBlock = 8;

template <typename T>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
gemm_simt_kernel(const T *__restrict__ W, const T *__restrict__ x, int n_in, EpiParams ep, const int32_t *status)
{
    pdl_launch_dependents();
    pdl_wait();
    if (*status) return;
    const int lane = threadIdx.x & 31;
    const int pair = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const bool swiglu = ep.mode == EPI_SWIGLU;
    const int n_pairs = swiglu ? ep.n_out : (ep.n_out + 1) / 2;
    if (pair >= n_pairs) return;
    const int r0 = swiglu ? pair : 2 * pair;
    const bool has1 = swiglu || (r0 + 1 < ep.n_out);
    const T *wa = W + (size_t)r0 * n_in;
    const T *wb = swiglu ? W + (size_t)(ep.n_out + pair) * n_in : (has1 ? wa + n_in : wa);

    for (int i0 = 0; i0 < ep.n; i0 += kNodeChunk) {
        float a0[kNodeChunk], a1[kNodeChunk];
#pragma unroll
        for (int u = 0; u < kNodeChunk; ++u) a0[u] = a1[u] = 0.f;
        for (int k = lane * 4; k < n_in; k += 128) {
            Vec4<T> va, vb;
            va.load(wa + k);
            vb.load(wb + k);
#pragma unroll
            for (int u = 0; u < kNodeChunk; ++u) {
                if (i0 + u < ep.n) {
                    Vec4<T> vx;
                    vx.load(x + (size_t)(i0 + u) * n_in + k);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float xv = vx.get(j);
                        a0[u] = fmaf(va.get(j), xv, a0[u]);
                        a1[u] = fmaf(vb.get(j), xv, a1[u]);
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kNodeChunk; ++u) {
            for (int o = 16; o; o >>= 1) {
                a0[u] += __shfl_xor_sync(0xffffffffu, a0[u], o);
                a1[u] += __shfl_xor_sync(0xffffffffu, a1[u], o);
            }
        }
#pragma unroll
        for (int u = 0; u < kNodeChunk; ++u)
            if (lane == u && i0 + u < ep.n) epilogue_pair<T>(ep, r0, i0 + u, a0[u], a1[u], has1);
    }
}

cudaError_t launch_gemm_simt(const void *W, const void *x, int dtype, int n_in, const EpiParams &ep,
                             const int32_t *status, cudaStream_t st)
{
    const int n_pairs = ep.mode == EPI_SWIGLU ? ep.n_out : (ep.n_out + 1) / 2;
    const int blocks = (n_pairs + kWarpsPerBlock - 1) / kWarpsPerBlock;
    LaunchCfg lc(blocks, kWarpsPerBlock * 32, 0, st);
    if (dtype == LLMCAD_F32)
        return cudaLaunchKernelEx(&lc.cfg, gemm_simt_kernel<float>, (const float *)W, (const float *)x, n_in, ep, status);
    return cudaLaunchKernelEx(&lc.cfg, gemm_simt_kernel<__nv_bfloat16>, (const __nv_bfloat16 *)W, (const __nv_bfloat16 *)x,
                              n_in, ep, status);
}

}  // namespace llmcad
