// Shared declarations of the token-tree verification library (device + host side).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>

#include "../../include/llmcad.h"

namespace llmcad {

// ---------------------------------------------------------------- element access
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ---------------------------------------------------------------- compensated bf16 activations
// A bf16 keeps 8 significant bits; rounding every activation to it at every GEMM and attention
// input adds up, over tens of layers, to logit errors beyond 2e-2 of the largest logit. The
// tensor-core path therefore carries each activation as hi + lo, hi = bf16(v), lo = bf16(v - hi)
// (16 significant bits together), in two planes of the same buffer: the lo plane of a [128][len]
// activation buffer starts kLoRows rows after the hi plane. The weights stream once either way;
// the MMAs see the nodes twice (N = 2 * n_pad) and the epilogue adds the two accumulator columns.
constexpr int kLoRows = LLMCAD_MAX_TREE;

__device__ __forceinline__ void split_bf16(float v, __nv_bfloat16 &hi, __nv_bfloat16 &lo)
{
    hi = __float2bfloat16_rn(v);
    lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}
// Stores v at *p and its remainder at *p_lo.
template <typename T> __device__ __forceinline__ void store_split(T *p, T *p_lo, float v);
template <> __device__ __forceinline__ void store_split<float>(float *p, float *, float v) { *p = v; }
template <> __device__ __forceinline__ void store_split<__nv_bfloat16>(__nv_bfloat16 *p, __nv_bfloat16 *p_lo, float v)
{
    split_bf16(v, *p, *p_lo);
}
// Stores v at p[0] and, if comp, its remainder at p[lo_off]. For fp32 buffers there is no remainder.
template <typename T> __device__ __forceinline__ void store_split(T *p, size_t lo_off, float v, bool comp);
template <> __device__ __forceinline__ void store_split<float>(float *p, size_t, float v, bool) { *p = v; }
template <> __device__ __forceinline__ void store_split<__nv_bfloat16>(__nv_bfloat16 *p, size_t lo_off, float v, bool comp)
{
    __nv_bfloat16 hi, lo;
    split_bf16(v, hi, lo);
    p[0] = hi;
    if (comp) p[lo_off] = lo;
}

// ---------------------------------------------------------------- GEMM epilogues
// What a GEMM does with a finished pair of output values of one tree node.
enum EpiMode : int {
    EPI_PLAIN = 0,   // y[i][r] = acc                                   (fp32)
    EPI_QKV = 1,     // rotate q,k pairs at pos[i]; q -> q buffer, k,v -> cache slot P+i
    EPI_RESID = 2,   // x[i][r] += acc                                   (fp32 residual stream)
    EPI_SWIGLU = 3,  // h[i][r] = silu(gate) * up                        (pair = gate row r, up row r)
};

struct EpiParams {
    int mode;
    int n;         // tree nodes
    int n_out;     // output features (rows of W); for EPI_SWIGLU the FFN width f
    // EPI_PLAIN
    float *y;
    int ldy;
    // EPI_RESID
    float *x;      // [n][n_out]
    // EPI_SWIGLU
    void *h;       // [n][f] activation dtype
    // EPI_QKV
    void *q_out;   // [n][d] activation dtype
    void *k_cache; // this layer's K: [H][S][hd]
    void *v_cache;
    const float2 *rope_cs;  // [n][hd/2] (cos, sin) of pos[i] * base^(-2t/hd)
    int d, hd, S, P;
    // RMSNorm folded into the tensor-core GEMM. Input side (any mode): the accumulator of node i
    // is multiplied by rsqrt(sum_t ssq_in[t][i] / norm_d + eps); the GEMM input then is gain * x.
    const float *ssq_in;    // [ssq_in_parts][128] partial sums of squares per node, or nullptr
    int ssq_in_parts, norm_d;
    float eps;
    // Output side (EPI_RESID): besides x += acc, emit gain_next * x in the activation dtype and
    // this tile's partial sums of squares (4 per tile, one per 32 rows) for the next norm.
    void *xg_out;           // [n][n_out] or nullptr
    const void *gain_next;  // [n_out]
    float *ssq_out;         // [4 * n_tiles][128]
    // Tensor-core path: q_out, h and xg_out also get their lo plane (see kLoRows), and the bf16
    // remainders of the keys and values go to kv_lo, [2][H][kLoRows][hd] (K then V, row = node).
    int comp;
    void *kv_lo;
};

// (v0, v1) are the accumulators of output rows (r0, r0+1), r0 even, of node i; for
// EPI_SWIGLU they are (gate, up) of output feature r0. has1 says whether row r0+1 exists.
template <typename T>
__device__ __forceinline__ void epilogue_pair(const EpiParams &ep, int r0, int i, float v0, float v1, bool has1)
{
    switch (ep.mode) {
    case EPI_PLAIN:
        ep.y[(size_t)i * ep.ldy + r0] = v0;
        if (has1) ep.y[(size_t)i * ep.ldy + r0 + 1] = v1;
        break;
    case EPI_RESID:
        ep.x[(size_t)i * ep.n_out + r0] += v0;
        if (has1) ep.x[(size_t)i * ep.n_out + r0 + 1] += v1;
        break;
    case EPI_SWIGLU: {
        float s = v0 / (1.0f + expf(-v0));
        reinterpret_cast<T *>(ep.h)[(size_t)i * ep.n_out + r0] = from_f32<T>(s * v1);
        break;
    }
    case EPI_QKV: {
        const int sec = r0 / ep.d, c = r0 - sec * ep.d;
        const int head = c / ep.hd, e = c - head * ep.hd;
        float o0 = v0, o1 = v1;
        if (sec < 2) {
            const float2 cs = ep.rope_cs[(size_t)i * (ep.hd >> 1) + (e >> 1)];
            o0 = v0 * cs.x - v1 * cs.y;
            o1 = v0 * cs.y + v1 * cs.x;
        }
        T *dst;
        if (sec == 0) dst = reinterpret_cast<T *>(ep.q_out) + (size_t)i * ep.d + c;
        else dst = reinterpret_cast<T *>(sec == 1 ? ep.k_cache : ep.v_cache) + ((size_t)head * ep.S + ep.P + i) * ep.hd + e;
        dst[0] = from_f32<T>(o0);
        dst[1] = from_f32<T>(o1);
        break;
    }
    }
}

// ---------------------------------------------------------------- debug checks
// compute-sanitizer is not available where this library is developed. A build with -DLLMCAD_CHECKS
// (build.py: libllmcad_checks.so) verifies, on the device, the indices that are derived from data or
// from the launch arithmetic (workspace slots, cache slots, node and row numbers, path entries) right
// before they are used: a failed check writes LLMCAD_ERR_CHECK into the pass's status word and the
// access is skipped, so that nothing faults. In the normal build the macro is the constant `true`.
#ifdef LLMCAD_CHECKS
#define LLMCAD_CHECK(cond, status_ptr) ((cond) ? true : (atomicCAS(reinterpret_cast<int *>(const_cast<int32_t *>(status_ptr)), 0, (int)LLMCAD_ERR_CHECK), false))
#else
#define LLMCAD_CHECK(cond, status_ptr) (true)
#endif

// ---------------------------------------------------------------- bounded waits
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t) :: "memory");   // the clobber keeps the read where it is written
    return t;
}
constexpr uint64_t kDefaultWaitLimitNs = 2000000000ull;  // every device-side wait gives up after 2 s unless the context says otherwise

// ---------------------------------------------------------------- programmatic dependent launch
// Every kernel of the pass is launched with programmatic stream serialization: it lets its
// successor start (launch latency, prologue, weight prefetch) while it is still running, and it
// calls pdl_wait() before it touches anything an earlier kernel wrote or still reads.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------- completion counters
// Programmatic dependent launch orders two kernels through griddepcontrol.wait, which returns only when
// the earlier grid has exited and its memory is flushed: ~1.3 us after the last CTA's exit on B200. As an
// alternative (an option of the context, off by default: it measured slower) the kernels of the
// tensor-core pass can hand over through counters in global memory: every CTA (or
// warp) of a kernel adds one to the kernel's counter, with release semantics, when its results are
// written, and the consumer polls, with acquire semantics, until the counter reaches the number of
// arrivals it was told to expect. All CTAs of the producer are resident (or done) before any CTA of the
// consumer starts, because a kernel lets its dependents launch only from inside its CTAs, so a poll
// cannot starve the kernel it waits for. A null counter means "use the grid dependency".
struct DepWait {
    const uint32_t *ctr;     // nullptr: griddepcontrol.wait
    uint32_t target;
    uint64_t limit_ns;       // the wait gives up after this long
};

__device__ __forceinline__ uint32_t ld_acquire_gpu_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// One thread waits; false when the limit ran out.
__device__ __forceinline__ bool dep_wait_thread(const DepWait &d)
{
    if (d.ctr == nullptr) { pdl_wait(); return true; }
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (ld_acquire_gpu_u32(d.ctr) >= d.target) return true;
        __nanosleep(32);
        if ((it & 63u) == 63u) {
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > d.limit_ns) return false;
        }
    }
}

// A whole warp waits: lane 0 polls, the barrier orders the other lanes' later reads after its acquire.
__device__ __forceinline__ bool dep_wait_warp(const DepWait &d, int lane)
{
    int ok = 1;
    if (d.ctr == nullptr) { pdl_wait(); return true; }
    if (lane == 0) ok = dep_wait_thread(d) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    return ok != 0;
}

// One arrival: everything this thread wrote, and everything it has observed through a CTA or warp barrier,
// is visible to whoever sees the count.
__device__ __forceinline__ void dep_arrive(uint32_t *ctr)
{
    if (ctr == nullptr) return;
    asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(ctr) : "memory");   // release is cumulative: no separate fence
}

// Data that arrived through ordinary stores of other SMs is about to be read by the copy engine (TMA).
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

struct LaunchCfg {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attrs[2];
    LaunchCfg(dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster_x = 0)
    {
        cfg = {};
        cfg.gridDim = grid;
        cfg.blockDim = block;
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        static const int pdl = [] { const char *e = getenv("LLMCAD_PDL"); return e ? atoi(e) : 1; }();   // tuning aid
        attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attrs[0].val.programmaticStreamSerializationAllowed = pdl;
        cfg.numAttrs = 1;
        if (cluster_x > 0) {
            attrs[1].id = cudaLaunchAttributeClusterDimension;
            attrs[1].val.clusterDim.x = cluster_x;
            attrs[1].val.clusterDim.y = 1;
            attrs[1].val.clusterDim.z = 1;
            cfg.numAttrs = 2;
        }
        cfg.attrs = attrs;
    }
};

// A function attribute (cudaFuncSetAttribute) belongs to the device it was set on: remember per device
// whether a launcher has done its one-time set-up there.
struct PerDeviceOnce {
    bool done[64] = {};
    int dev = -1;
    bool needed()
    {
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { dev = -1; return true; }
        return !done[dev];
    }
    void mark() { if (dev >= 0) done[dev] = true; }
};

// ---------------------------------------------------------------- launchers (host)
struct TreeBuffers {
    int32_t *depth, *pos;
    uint32_t *anc;      // [n][4]
    float2 *rope_cs;    // [n][hd/2]
};

cudaError_t launch_tree_prep(const int32_t *parent, const int32_t *tokens, int n, int P, int vocab, int hd,
                             float rope_base, TreeBuffers tb, int32_t *status, cudaStream_t st);
cudaError_t launch_embed(const void *E, int dtype, const int32_t *tokens, int n, int d, float *x, const int32_t *status,
                         cudaStream_t st);
cudaError_t launch_embed_norm(const void *E, const int32_t *tokens, int n, int d, const void *gain, float *x, void *xg,
                              float *ssq, int comp, const int32_t *status, cudaStream_t st);
cudaError_t launch_rmsnorm(const float *x, const void *g, int dtype, int n, int d, float eps, void *out,
                           const int32_t *status, cudaStream_t st);
cudaError_t launch_argmax(const float *logits, int n, int vocab, int32_t *argmax, int32_t *status, cudaStream_t st);
cudaError_t launch_accept(const int32_t *parent, const int32_t *tokens, const int32_t *argmax, int n, int P,
                          int32_t *path, int32_t *scalars, cudaStream_t st);
cudaError_t launch_compact(void *kv, int dtype, int n_layers, int n_heads, int S, int hd, int P, const int32_t *path,
                           const int32_t *scalars, cudaStream_t st);
size_t tiled_weight_bytes(int n_out, int n_in);
cudaError_t launch_tile_weight(const void *w, int n_out, int n_in, void *dst, cudaStream_t st);
// INT4 weights (pack.cu): bytes of one (128 rows x 64 columns) tile: 4 KB of codes + 128 exponents
constexpr int kW4TileBytes = 4096 + 128;
size_t tiled_weight_int4_bytes(int n_out, int n_in);       // n_in a multiple of 64
cudaError_t launch_tile_weight_int4(const void *w, int n_out, int n_in, void *dst, cudaStream_t st);
cudaError_t launch_quantize_int4_plain(const void *w, int n_out, int n_in, int8_t *q, int8_t *e, cudaStream_t st);
cudaError_t launch_gemm_simt(const void *W, const void *x, int dtype, int n_in, const EpiParams &ep,
                             const int32_t *status, cudaStream_t st);
cudaError_t launch_attention_simt(const void *q, const void *k, const void *v, int dtype, int n_heads, int hd,
                                  int kv_stride, int P, int n, const uint32_t *anc, void *o, const int32_t *status,
                                  cudaStream_t st, int n_tree = 0, int q_first = 0);
// softmax probabilities and ids of the k largest logits of every node (ties: lowest id; NaN -> status)
cudaError_t launch_topk_softmax(const float *logits, int n, int vocab, int k, int32_t *ids, float *probs, int32_t *status,
                                cudaStream_t st);

}  // namespace llmcad
