// Weight-streaming skinny GEMM on the sm_100a tensor cores.
//
// The one-shot verification of Sec. 3.2 visits every parameter once for all N <= 128 tree nodes,
// so each GEMM is D[n_out][N] = W[n_out][K] * X[N][K]^T with a tiny N: it is bound by the bytes
// of W coming from HBM. The kernel therefore puts W on the M side of tcgen05.mma (128 weight
// rows per tile = the 128 TMEM lanes) and the tree nodes on the N side (padded to a multiple of
// 16), streams W exactly once through a deep TMA -> shared-memory ring, and keeps all SMs pulling
// by splitting the (tile, k-block) work evenly over a persistent grid (stream-K): a CTA's range
// may start and end inside a tile; the sharers of a tile leave their partial accumulators in an
// fp32 workspace and whichever warp arrives last at the tile's ticket counter adds them in a
// fixed (CTA) order and runs the fused epilogue, so the result does not depend on timing and
// no CTA ever waits for another.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = TMEM allocator + MMA issuer,
// warps 2..5 = epilogue (tcgen05.ld of their 32 lanes each). Accumulators are double-buffered in
// TMEM so that the epilogue of one tile overlaps the MMAs of the next.
//
// The kernel is launched with programmatic stream serialization: its producer fills the whole
// ring with weight tiles (which no kernel ever writes) while the previous kernel of the pass is
// still running, and only the activation tiles, the workspace and the outputs wait for the grid
// dependency. A status word left by an earlier phase is not looked at here: the GEMM then
// works on stale but finite activations and writes only scratch (slots >= prefix_len, the
// context's buffers), and the search/rollback kernels at the end of the pass report the error.
//
// Every wait (mbarrier, workspace flag) is bounded; on expiry the kernel sets the status word to
// LLMCAD_ERR_TIMEOUT, lets every role fall out of its loop, frees TMEM and returns.
#include <cuda.h>

#include "common.cuh"
#include "gemm_tc.cuh"

namespace llmcad {

namespace {

constexpr int kTileM = 128;     // weight rows per tile
constexpr int kBlockK = 64;     // bf16 elements per k-block = one 128-byte swizzle row
constexpr int kThreads = 192;
constexpr int kATileBytes = kTileM * kBlockK * 2;  // 16 KB

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kWaitLimitNs or as soon as another role has raised `abort`.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 255u) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) return false;
        }
    }
}

// ---------------------------------------------------------------- TMA
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar,
                                            uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar), "l"(policy)
        : "memory");
}

// ---------------------------------------------------------------- tcgen05
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, issued by one thread.
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float *v)
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = __uint_as_float(r[j]);
}

// Shared-memory matrix descriptor: K-major tile of 128-byte rows, 128-byte swizzle, 8-row groups
// 1024 bytes apart (the layout a TMA box of 64 bf16 x rows with CU_TENSOR_MAP_SWIZZLE_128B
// produces). Fields: start address >> 4 [0,14), leading byte offset >> 4 [16,30) (unused for
// swizzled K-major, set to 1), stride byte offset >> 4 [32,46), version 1 [46,48), layout type
// [61,64) = 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor of kind::f16: fp32 accumulator (bits 4-5 = 1), A and B bf16 (bits 7-9,
// 10-12 = 1), both K-major (bits 15, 16 = 0), N >> 3 at bits 17-22, M >> 4 at bits 24-28.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

struct SharedCtl {
    uint64_t full[16];
    uint64_t empty[16];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
    float rs[LLMCAD_MAX_TREE]; // per-node rsqrt(mean(x^2) + eps) of the folded input RMSNorm
};

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t *p, uint32_t v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Walks the (tile, k-block) units of one CTA's range [u0, u1) segment by segment, last segment
// first (see the kernel comment for why), k-blocks ascending inside a segment.
struct UnitWalk {
    long long u0, hi;
    int kb_per_tile;
    int tile, kb, kb1;
    __device__ UnitWalk(long long u0_, long long u1_, int kbpt) : u0(u0_), hi(u1_), kb_per_tile(kbpt), tile(0), kb(0), kb1(0) {}
    // advance to the next unit; false when the range is exhausted
    __device__ bool next()
    {
        if (kb + 1 < kb1) { ++kb; return true; }
        if (hi <= u0) return false;
        tile = (int)((hi - 1) / kb_per_tile);
        const long long t0 = (long long)tile * kb_per_tile;
        const long long lo = u0 > t0 ? u0 : t0;
        kb = (int)(lo - t0);
        kb1 = (int)(hi - t0);
        hi = lo;
        return true;
    }
};

}  // namespace

template <typename T>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x, TcGemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ SharedCtl ctl;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_acc = p.dual ? 2 : 1;
    const uint32_t b_tile_bytes = (uint32_t)p.n_pad * kBlockK * 2;
    const uint32_t stage_bytes = n_acc * kATileBytes + b_tile_bytes;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;

    // Let the next kernel of the stream start its own prologue and weight prefetch early. This
    // kernel in turn must not read activations, the status word or the workspace, nor write
    // anything, before pdl_wait(): until then it only prefetches weights, which no kernel writes.
    pdl_launch_dependents();
#define LLMCAD_TRACE(slot) do { if (p.trace) p.trace[(size_t)blockIdx.x * 16 + (slot)] = global_timer_ns(); } while (0)
    if (threadIdx.x == 0) LLMCAD_TRACE(0);

    // ---- work range of this CTA
    const long long total_units = (long long)p.n_tiles * p.kb_per_tile;
    const long long u0 = min(total_units, (long long)blockIdx.x * p.units_per_cta);
    const long long u1 = min(total_units, u0 + p.units_per_cta);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(smem_u32(&ctl.full[s]), 1);
            mbar_init(smem_u32(&ctl.empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.tmem_full[b]), 1);
            mbar_init(smem_u32(&ctl.tmem_empty[b]), 4);
        }
        ctl.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)),
                     "r"((uint32_t)p.tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl.tmem_base;
    volatile int *abort_flag = &ctl.abort_flag;
    bool timed_out = false;
    if (threadIdx.x == 0) LLMCAD_TRACE(1);

    if (warp == 0) {
        // ================================================= TMA producer
        if (lane == 0) {
            uint64_t pol_stream, pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            // Phase 1, before the grid dependency resolves: fill the ring with weight tiles only.
            int pre = 0;
            {
                UnitWalk w(u0, u1, p.kb_per_tile);
                for (; pre < p.stages && w.next(); ++pre) {
                    const uint32_t full = smem_u32(&ctl.full[pre]);
                    const uint32_t dst = smem_base + pre * stage_bytes;
                    mbar_expect_tx(full, stage_bytes);
                    tma_load_2d(dst, &tm_w, w.kb * kBlockK, w.tile * kTileM, full, pol_stream);
                    if (p.dual) tma_load_2d(dst + kATileBytes, &tm_w, w.kb * kBlockK, p.up_row_offset + w.tile * kTileM, full, pol_stream);
                }
            }
            LLMCAD_TRACE(2);
            pdl_wait();
            LLMCAD_TRACE(3);
            // Phase 2: the activation tiles of the prefetched stages, then the steady state.
            UnitWalk w(u0, u1, p.kb_per_tile);
            for (uint32_t it = 0; w.next(); ++it) {
                const int s = it % p.stages;
                const uint32_t full = smem_u32(&ctl.full[s]);
                const uint32_t dst = smem_base + s * stage_bytes;
                if ((int)it >= pre) {
                    const uint32_t par = ((it / p.stages) & 1u) ^ 1u;
                    if (!mbar_wait(smem_u32(&ctl.empty[s]), par, abort_flag)) { timed_out = true; break; }
                    mbar_expect_tx(full, stage_bytes);
                    tma_load_2d(dst, &tm_w, w.kb * kBlockK, w.tile * kTileM, full, pol_stream);
                    if (p.dual) tma_load_2d(dst + kATileBytes, &tm_w, w.kb * kBlockK, p.up_row_offset + w.tile * kTileM, full, pol_stream);
                }
                tma_load_2d(dst + n_acc * kATileBytes, &tm_x, w.kb * kBlockK, 0, full, pol_keep);
            }
            LLMCAD_TRACE(4);
        }
    } else if (warp == 1) {
        // ================================================= MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc(kTileM, p.n_pad);
            uint32_t it = 0, seg = 0;
            for (long long hi = u1; hi > u0 && !timed_out; ++seg) {
                const int tile = (int)((hi - 1) / p.kb_per_tile);
                const long long lo = max(u0, (long long)tile * p.kb_per_tile);
                const int kb0 = (int)(lo - (long long)tile * p.kb_per_tile), kb1 = (int)(hi - (long long)tile * p.kb_per_tile);
                const int buf = seg & 1;
                if (!mbar_wait(smem_u32(&ctl.tmem_empty[buf]), ((seg >> 1) & 1u) ^ 1u, abort_flag)) { timed_out = true; break; }
                tc_fence_after();
                const uint32_t d0 = tmem_base + (uint32_t)(buf * n_acc * p.n_pad);
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int s = it % p.stages;
                    if (!mbar_wait(smem_u32(&ctl.full[s]), (it / p.stages) & 1u, abort_flag)) { timed_out = true; break; }
                    if (it == 0) LLMCAD_TRACE(5);
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + s * stage_bytes;
                    const uint64_t a_desc = make_smem_desc(a_addr);
                    const uint64_t b_desc = make_smem_desc(a_addr + n_acc * kATileBytes);
#pragma unroll
                    for (int k4 = 0; k4 < kBlockK / 16; ++k4) {
                        const uint32_t acc = (kb > kb0 || k4 > 0) ? 1u : 0u;
                        // advancing 16 bf16 = 32 bytes inside the swizzle row: +2 in the >>4 address field
                        tc_mma_bf16(d0, a_desc + 2 * k4, b_desc + 2 * k4, idesc, acc);
                        if (p.dual) {
                            const uint64_t a2_desc = make_smem_desc(a_addr + kATileBytes);
                            tc_mma_bf16(d0 + p.n_pad, a2_desc + 2 * k4, b_desc + 2 * k4, idesc, acc);
                        }
                    }
                    tc_commit(smem_u32(&ctl.empty[s]));  // frees the stage when these MMAs have read it
                }
                if (timed_out) break;
                tc_commit(smem_u32(&ctl.tmem_full[buf]));
                hi = lo;
            }
            LLMCAD_TRACE(6);
        }
    } else {
        // ================================================= epilogue (warps 2..5)
        const int lane_grp = warp & 3;                 // TMEM lanes 32*lane_grp .. +31 belong to this warp
        const int row_in_tile = lane_grp * 32 + lane;
        const int et = (warp - 2) * 32 + lane;         // 0..127 among the epilogue threads
        const EpiParams &ep = p.ep;
        pdl_wait();
        // RMSNorm of the GEMM input folded into the epilogue: the producer of the residual stream
        // left partial sums of squares per node; acc * rsqrt(mean(x^2) + eps) is applied to the
        // complete sums below. Done once per CTA while the main loop is still filling the pipe.
        if (ep.ssq_in != nullptr) {
            float ss = 0.f;
            for (int t = 0; t < ep.ssq_in_parts; ++t) ss += __ldcg(ep.ssq_in + (size_t)t * LLMCAD_MAX_TREE + et);
            ctl.rs[et] = rsqrtf(ss / (float)ep.norm_d + ep.eps);
            asm volatile("bar.sync 1, 128;" ::: "memory");   // all four epilogue warps get here unconditionally
        }
        uint32_t seg = 0;
        for (long long hi = u1; hi > u0 && !timed_out; ++seg) {
            const int tile = (int)((hi - 1) / p.kb_per_tile);
            const long long tile_u0 = (long long)tile * p.kb_per_tile;
            const long long lo = max(u0, tile_u0);
            const int kb0 = (int)(lo - tile_u0), kb1 = (int)(hi - tile_u0);
            const int buf = seg & 1;
            const bool sole = (kb0 == 0 && kb1 == p.kb_per_tile);      // this CTA holds the whole tile
            const int first_cta = (int)(tile_u0 / p.units_per_cta);
            const int last_cta = (int)((tile_u0 + p.kb_per_tile - 1) / p.units_per_cta);
            const int n_parts = last_cta - first_cta + 1;
            const size_t part_stride = (size_t)n_acc * p.n_pad * kTileM;  // floats per partial slot

            if (!mbar_wait(smem_u32(&ctl.tmem_full[buf]), (seg >> 1) & 1u, abort_flag)) { timed_out = true; break; }
            tc_fence_after();
            if (threadIdx.x == 64) LLMCAD_TRACE(lo == u0 ? 8 : 7);   // 7: first segments, 8: the last one

            const uint32_t t_lane = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(buf * n_acc * p.n_pad);
            const int row = tile * kTileM + row_in_tile;           // output feature (weight row)
            const bool row_ok = row < ep.n_out;
            bool finish = sole;

            if (!sole) {
                // A tile shared by several CTAs: every sharer leaves its partial accumulator in the
                // workspace; the rows of a tile are independent per warp (32 rows each), so each
                // warp takes a ticket for its own row group and the last warp to arrive adds all
                // partials in CTA order and finishes those rows. Nobody waits for anybody.
                // Slot 0 of a CTA holds the segment that contains its range start, slot 1 the other.
                float *dst = p.partials + ((size_t)blockIdx.x * 2 + (lo == u0 ? 0 : 1)) * part_stride + row_in_tile;
                for (int c0 = 0; c0 < n_acc * p.n_pad; c0 += 16) {
                    float v[16];
                    tc_ld16(t_lane + c0, v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) dst[(size_t)(c0 + j) * kTileM] = v[j];
                }
                __threadfence();
                __syncwarp();
                int last = 0;
                if (lane == 0) {
                    uint32_t *ctr = p.tickets + (size_t)tile * 4 + lane_grp;
                    last = (atomicAdd(ctr, 1u) == (uint32_t)n_parts - 1u);
                    if (last) { *ctr = 0; __threadfence(); }
                }
                finish = __shfl_sync(0xffffffffu, last, 0) != 0;
                // the accumulator is in the workspace now: hand the TMEM buffer back early
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl.tmem_empty[buf]));
                if (threadIdx.x == 64) LLMCAD_TRACE(9);
            }

            if (finish) {
                float gain = 0.f;
                if (ep.mode == EPI_RESID && ep.xg_out != nullptr && row_ok)
                    gain = to_f32<T>(reinterpret_cast<const T *>(ep.gain_next)[row]);
                for (int c0 = 0; c0 < p.n_pad; c0 += 16) {
                    float v[16], w[16];
                    if (sole) {
                        tc_ld16(t_lane + c0, v);
                        if (p.dual) tc_ld16(t_lane + p.n_pad + c0, w);
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] = w[j] = 0.f;
                        // partial tiles in CTA order, two CTAs' loads in flight at a time
                        for (int c = first_cta; c <= last_cta; c += 2) {
                            const bool two = c + 1 <= last_cta;
                            const int slot0 = ((long long)c * p.units_per_cta >= tile_u0) ? 0 : 1;
                            const int slot1 = ((long long)(c + 1) * p.units_per_cta >= tile_u0) ? 0 : 1;
                            const float *s0 = p.partials + ((size_t)c * 2 + slot0) * part_stride + (size_t)c0 * kTileM + row_in_tile;
                            const float *s1 = two ? p.partials + ((size_t)(c + 1) * 2 + slot1) * part_stride + (size_t)c0 * kTileM + row_in_tile : s0;
                            float a0[16], a1[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) { a0[j] = __ldcg(s0 + (size_t)j * kTileM); a1[j] = __ldcg(s1 + (size_t)j * kTileM); }
#pragma unroll
                            for (int j = 0; j < 16; ++j) { v[j] += a0[j]; if (two) v[j] += a1[j]; }
                            if (p.dual) {
                                s0 += (size_t)p.n_pad * kTileM;
                                s1 += (size_t)p.n_pad * kTileM;
#pragma unroll
                                for (int j = 0; j < 16; ++j) { a0[j] = __ldcg(s0 + (size_t)j * kTileM); a1[j] = __ldcg(s1 + (size_t)j * kTileM); }
#pragma unroll
                                for (int j = 0; j < 16; ++j) { w[j] += a0[j]; if (two) w[j] += a1[j]; }
                            }
                        }
                    }
                    if (ep.ssq_in != nullptr) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) { const float r = ctl.rs[c0 + j]; v[j] *= r; w[j] *= r; }
                    }
                    // fused epilogue on complete sums; all loads of a 16-column chunk are issued before
                    // any dependent store so that they overlap instead of queueing behind each other
                    if (ep.mode == EPI_SWIGLU) {
                        T *hrow = reinterpret_cast<T *>(ep.h) + row;
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            if (row_ok && c0 + j < ep.n) {
                                const float sg = v[j] / (1.0f + __expf(-v[j]));
                                hrow[(size_t)(c0 + j) * ep.n_out] = from_f32<T>(sg * w[j]);
                            }
                        }
                    } else if (ep.mode == EPI_QKV) {
                        const int sec = row / ep.d, cidx = row - sec * ep.d;
                        const int head = cidx / ep.hd, e = cidx - head * ep.hd;
                        float2 cs[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            cs[j] = (sec < 2 && row_ok && c0 + j < ep.n) ? __ldg(ep.rope_cs + (size_t)(c0 + j) * (ep.hd >> 1) + (e >> 1))
                                                                          : make_float2(1.f, 0.f);
                        T *dst;
                        size_t node_stride;
                        if (sec == 0) { dst = reinterpret_cast<T *>(ep.q_out) + cidx; node_stride = ep.d; }
                        else { dst = reinterpret_cast<T *>(sec == 1 ? ep.k_cache : ep.v_cache) + ((size_t)head * ep.S + ep.P) * ep.hd + e; node_stride = ep.hd; }
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            // the rotary partner (2t <-> 2t+1) lives in the neighbouring lane
                            const float other = __shfl_xor_sync(0xffffffffu, v[j], 1);
                            const float rot = (lane & 1) ? (other * cs[j].y + v[j] * cs[j].x) : (v[j] * cs[j].x - other * cs[j].y);
                            if (row_ok && c0 + j < ep.n) dst[(size_t)(c0 + j) * node_stride] = from_f32<T>(rot);
                        }
                    } else if (ep.mode == EPI_RESID) {
                        float *xr = ep.x + row;
                        float xo[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) xo[j] = (row_ok && c0 + j < ep.n) ? __ldcg(xr + (size_t)(c0 + j) * ep.n_out) : 0.f;
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            xo[j] = (row_ok && c0 + j < ep.n) ? xo[j] + v[j] : 0.f;
                            if (row_ok && c0 + j < ep.n) xr[(size_t)(c0 + j) * ep.n_out] = xo[j];
                        }
                        if (ep.xg_out != nullptr) {
                            // what the next RMSNorm needs: gain * x in the GEMM input dtype, and this
                            // warp's share (32 rows) of every node's sum of squares
                            T *gr = reinterpret_cast<T *>(ep.xg_out) + row;
#pragma unroll
                            for (int j = 0; j < 16; ++j)
                                if (row_ok && c0 + j < ep.n) gr[(size_t)(c0 + j) * ep.n_out] = from_f32<T>(xo[j] * gain);
                            float mine = 0.f;
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                float sq = xo[j] * xo[j];
#pragma unroll
                                for (int o = 16; o; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
                                if (lane == j) mine = sq;
                            }
                            if (lane < 16)
                                ep.ssq_out[(size_t)(tile * 4 + lane_grp) * LLMCAD_MAX_TREE + c0 + lane] = mine;
                        }
                    } else {
                        float *yr = ep.y + row;
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (row_ok && c0 + j < ep.n) yr[(size_t)(c0 + j) * ep.ldy] = v[j];
                    }
                }
            }
            if (sole) {
                // accumulator buffer drained: hand it back to the MMA warp
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl.tmem_empty[buf]));
            }
            hi = lo;
        }
        if (threadIdx.x == 64) LLMCAD_TRACE(10);
    }
    __syncwarp();   // lanes that skipped their role's single-thread section rejoin their warp here

    if (timed_out) {
        *abort_flag = 1;
        atomicCAS(p.status, 0, LLMCAD_ERR_TIMEOUT);
        // give copies that may still be in flight time to land before the shared memory goes away
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) LLMCAD_TRACE(11);
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------------------------------ host

// The driver entry point is fetched through the runtime, so the library does not link libcuda.
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

bool make_tensor_map_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows)
{
    auto fn = get_encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBlockK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

size_t gemm_tc_partial_floats(int n_sms, int max_n_pad) { return (size_t)n_sms * 2 /*slots*/ * 2 /*gate+up*/ * max_n_pad * kTileM; }

cudaError_t launch_gemm_tc(const CUtensorMap &tm_w, const CUtensorMap &tm_x, int n_in, int n_pad, int n_sms,
                           float *partials, uint32_t *flags, uint32_t epoch, int32_t *status, const EpiParams &ep,
                           cudaStream_t st, unsigned long long *trace)
{
    TcGemmParams p;
    p.dual = ep.mode == EPI_SWIGLU;
    p.n_tiles = (ep.n_out + kTileM - 1) / kTileM;
    if (p.n_tiles > 4096) return cudaErrorInvalidValue;   // size of the ticket array
    p.kb_per_tile = (n_in + kBlockK - 1) / kBlockK;
    p.n_pad = n_pad;
    p.up_row_offset = ep.n_out;
    const long long total = (long long)p.n_tiles * p.kb_per_tile;
    int grid = (int)(total < n_sms ? total : n_sms);
    p.units_per_cta = (int)((total + grid - 1) / grid);
    grid = (int)((total + p.units_per_cta - 1) / p.units_per_cta);
    const int n_acc = p.dual ? 2 : 1;
    const size_t stage_bytes = (size_t)n_acc * kATileBytes + (size_t)n_pad * kBlockK * 2;
    const size_t smem_limit = 227 * 1024 - 1024 /*alignment slack*/ - 2048 /*static*/;
    int stages = (int)(smem_limit / stage_bytes);
    if (stages > 16) stages = 16;
    if (stages < 2) return cudaErrorInvalidConfiguration;
    p.stages = stages;
    int cols = 2 * n_acc * n_pad, pow2 = 32;
    while (pow2 < cols) pow2 <<= 1;
    p.tmem_cols = pow2;
    p.partials = partials;
    p.tickets = flags;
    (void)epoch;
    p.status = status;
    p.trace = trace;
    p.ep = ep;
    const size_t smem = (size_t)stages * stage_bytes + 1024;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             227 * 1024 - 2048);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    LaunchCfg lc(grid, kThreads, smem, st);
    return cudaLaunchKernelEx(&lc.cfg, gemm_tc_kernel<__nv_bfloat16>, tm_w, tm_x, p);
}

}  // namespace llmcad
