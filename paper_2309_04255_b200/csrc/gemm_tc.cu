// Weight-streaming skinny GEMMs on the sm_100a tensor cores.
//
// The one-shot verification of Sec. 3.2 visits every parameter once for all N <= 128 tree nodes,
// so each GEMM is D[n_out][N] = W[n_out][K] * X[N][K]^T with a tiny N: it is bound by the bytes
// of W coming from HBM. The streaming kernel therefore puts W on the M side of tcgen05.mma (128
// weight rows per tile = the 128 TMEM lanes) and the tree nodes on the N side (padded to a multiple
// of 16; with hi + lo activation planes the MMA sees every node twice), and streams W exactly once
// through a ring in shared memory: the weights are stored as pre-swizzled 16 KB tiles (pack.cu), so
// a ring item (one tile, two k-blocks) is one contiguous 32 KB bulk copy.
//
// A GEMM is two kernels, chained by programmatic dependent launch.
//
// gemm_stream_kernel: persistent grid, one CTA per SM. The (tile, k-block pair, half) items of the
// GEMM are split evenly over the CTAs (stream-K): a CTA's range may start and end inside a tile.
// For every tile that a CTA holds items of (a "segment") it leaves its accumulators, hi and lo
// columns added, in a workspace slot (slot = tile + CTA, unique because the CTAs' ranges are
// ordered), and exits. Nothing in it waits for another CTA.
//
// gemm_finish_kernel: all warps of the GPU add the segments of every tile in CTA order (so the
// result does not depend on timing) and apply the fused epilogue (rotary + K/V cache write,
// residual + the next norm's gain * x and sums of squares, SwiGLU, or plain fp32 rows). It needs
// next to no shared memory, so the NEXT GEMM's streaming CTAs become resident as soon as this
// GEMM's streaming CTAs leave, and fill their weight rings while the finishing runs: the HBM
// stream pauses only for as long as a ring lasts, not for the whole tail of a GEMM.
//
// Warp roles of the streaming kernel (224 threads): warp 0 = weight producer, warp 1 = TMEM
// allocator + MMA issuer, warps 2..5 = accumulator dump (tcgen05.ld of their 32 lanes each),
// warp 6 = activation loader (TMA). Accumulators are double-buffered in TMEM when two buffers fit,
// so that the dump of one segment overlaps the MMAs of the next.
//
// Programmatic stream serialization: the ring is filled with weight tiles while the previous
// kernels of the pass are still running; activations and the workspace wait for the grid
// dependency. The streaming kernel lets its dependents go only after its own dependency has
// resolved, so the finishing kernel may read what earlier GEMMs produced (norm sums, gains) before
// its own dependency, the streaming kernel, completes. A status word left by an earlier phase is
// not looked at here: the GEMMs then work on stale but finite activations and write only scratch
// and tree slots, and the search/rollback kernels at the end of the pass report the error.
//
// Every wait of the streaming kernel (mbarriers only) is bounded by a deadline; on expiry the
// kernel sets the status word to LLMCAD_ERR_TIMEOUT, lets every role fall out of its loop, frees
// TMEM and returns.
#include <cuda.h>

#include <cstdlib>

#include "common.cuh"
#include "gemm_tc.cuh"

namespace llmcad {

namespace {

constexpr int kTileM = 128;     // weight rows per tile
constexpr int kBlockK = 64;     // bf16 elements per k-block = one 128-byte swizzle row
constexpr int kThreads = 224;   // producer, MMA issuer, 4 epilogue warps, activation loader
constexpr int kFinThreads = 384;  // finishing kernel: 12 warps, up to 112 registers each beside a resident streaming CTA
// An SM's registers come in four banks of 16K, one per warp scheduler: beside the streaming CTA's two warps per
// scheduler (96 registers a thread) three finishing warps fit with up to 106 each.
constexpr int kFinMaxRegs = 96;
constexpr size_t kFinSmem = 24 * 1024;   // dynamic shared memory the finishing kernel asks for (and does not use):
                                         // it keeps two of its CTAs from settling on one SM, which would leave no room
                                         // there for the next GEMM's streaming CTA
constexpr int kATileBytes = kTileM * kBlockK * 2;  // 16 KB
constexpr int kMaxStages = 16;
constexpr int kMaxPStages = 24;   // INT4 weights: ring of packed tiles
constexpr int kMaxAStages = 8;    // INT4 weights: ring of activation k-block sets, apart from the expanded weight tiles
constexpr int kMaxPairK = 2;     // k-blocks per ring item (GemmDesc::pair_k): 2 = one 32 KB weight copy feeds 8 MMAs;
                                 // 1 for wide activation tiles, which would leave too few ring stages otherwise

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
// Bounded wait: gives up after wait_limit ns or as soon as another role has raised `abort`.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint64_t wait_limit)
{
    if (mbar_try(bar, parity)) return true;
    uint64_t t0 = 0;
    for (uint32_t it = 1;; ++it) {
        // (try_wait itself suspends the thread for a while when the phase is not complete; a __nanosleep between the
        // tries, meant to leave issue slots to the warp that shares the scheduler, measured 0.6 % slower per pass)
        if (mbar_try(bar, parity)) return true;
        if ((it & 255u) == 0) {
            if (*abort_flag) return false;
            if (t0 == 0) t0 = global_timer_ns();
            else if (global_timer_ns() - t0 > wait_limit) return false;
        }
    }
}

// Whole-warp wait for roles that are not on the critical path of the weight stream: one lane
// polls and the warp follows. A warp of 32 pollers per barrier would saturate the shared-memory
// pipeline that the producer's copies and barrier operations also go through.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, int lane, uint64_t wait_limit)
{
    int ok = 1;
    if (lane == 0 && !mbar_try(bar, parity)) {
        const uint64_t t0 = global_timer_ns();
        for (uint32_t it = 1;; ++it) {
            if (mbar_try(bar, parity)) break;
            if ((it & 63u) == 0 && (*abort_flag || global_timer_ns() - t0 > wait_limit)) { ok = 0; break; }
        }
    }
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
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

// Activation box (64 columns x rows x planes) at column c0, row 0, plane 0.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(0), "r"(bar), "l"(policy)
        : "memory");
}

// One contiguous run of global memory into shared memory (both 16-byte aligned, size a multiple of 16).
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
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

// 32 consecutive fp32 columns of this thread's TMEM lane at each of two addresses, summed. A load plus
// its wait costs ~0.15 us whatever the width, so the two loads share one wait; everything sits in one
// statement so that no register of the result can be touched before the wait.
__device__ __forceinline__ void tc_ld32_sum2(uint32_t taddr_a, uint32_t taddr_b, float *v)
{
    uint32_t a[32], b[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%64];\n\t"
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%65];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]), "=r"(a[4]), "=r"(a[5]), "=r"(a[6]), "=r"(a[7]), "=r"(a[8]), "=r"(a[9]), "=r"(a[10]), "=r"(a[11]), "=r"(a[12]), "=r"(a[13]), "=r"(a[14]), "=r"(a[15]), "=r"(a[16]), "=r"(a[17]), "=r"(a[18]), "=r"(a[19]), "=r"(a[20]), "=r"(a[21]), "=r"(a[22]), "=r"(a[23]), "=r"(a[24]), "=r"(a[25]), "=r"(a[26]), "=r"(a[27]), "=r"(a[28]), "=r"(a[29]), "=r"(a[30]), "=r"(a[31]), "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3]), "=r"(b[4]), "=r"(b[5]), "=r"(b[6]), "=r"(b[7]), "=r"(b[8]), "=r"(b[9]), "=r"(b[10]), "=r"(b[11]), "=r"(b[12]), "=r"(b[13]), "=r"(b[14]), "=r"(b[15]), "=r"(b[16]), "=r"(b[17]), "=r"(b[18]), "=r"(b[19]), "=r"(b[20]), "=r"(b[21]), "=r"(b[22]), "=r"(b[23]), "=r"(b[24]), "=r"(b[25]), "=r"(b[26]), "=r"(b[27]), "=r"(b[28]), "=r"(b[29]), "=r"(b[30]), "=r"(b[31])
        : "r"(taddr_a), "r"(taddr_b)
        : "memory");
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(a[j]) + __uint_as_float(b[j]);
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
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
    volatile uint32_t a_issued;     // ring items whose weight copy (and expect_tx) has been issued
    uint64_t pfull[kMaxPStages];    // INT4 weights: packed tile landed / packed stage free again
    uint64_t pempty[kMaxPStages];
    uint64_t afull[kMaxAStages];    // INT4 weights: activation tiles of an item landed / their slot free again
    uint64_t aempty[kMaxAStages];
};

// A ring item is (tile, k-block pair, half): up to two consecutive 64-wide k-blocks of one
// 128-row weight tile (32 KB, contiguous in the tiled layout) and the matching activation tiles.
__host__ __device__ __forceinline__ int pairs_per_tile(const GemmDesc &g) { return (g.kb_per_tile + g.pair_k - 1) / g.pair_k; }
// the same with the k-blocks per item as a compile-time constant (the kernel is instantiated for 1 and 2)
template <int PK> __device__ __forceinline__ int pairs_per_tile_c(const GemmDesc &g) { return (g.kb_per_tile + PK - 1) / PK; }

// CTA cta's share of the GEMM: items [begin, end) of its item list.
struct Range {
    int begin, end;
};
template <int PK>
__device__ __forceinline__ Range cta_range(const GemmDesc &g, int cta)
{
    const int total = g.n_tiles * pairs_per_tile_c<PK>(g) * g.halves;
    Range r;
    r.begin = min(total, cta * g.items_per_cta);
    r.end = min(total, r.begin + g.items_per_cta);
    return r;
}

// Cursor over this CTA's items, in order. Coordinates are kept incrementally: the single-thread
// roles have well under a microsecond per item.
template <int PK>
struct Cursor {
    int tile, kp, half;    // coordinates of the current item (kp: k-block pair)
    int left;              // items left in this CTA's range, the current one included
    int ppt, halves, kbpt;
    __device__ void init(const GemmDesc &d)
    {
        const Range r = cta_range<PK>(d, (int)blockIdx.x);
        left = r.end - r.begin;
        kbpt = d.kb_per_tile;
        ppt = pairs_per_tile_c<PK>(d);
        halves = d.halves;
        const int ipt = ppt * halves;
        tile = r.begin / ipt;
        const int q = r.begin - tile * ipt;
        kp = q / halves;
        half = q - kp * halves;
    }
    __device__ bool done() const { return left <= 0; }
    __device__ int kb0() const { return kp * PK; }
    __device__ int nk() const { return min(PK, kbpt - kp * PK); }   // k-blocks in this item
    __device__ void advance()
    {
        --left;
        if (++half == halves) {
            half = 0;
            if (++kp == ppt) { kp = 0; ++tile; }
        }
    }
};

// Floats of one segment slot of the workspace: [4 row groups][halves][n_pad nodes][32 rows].
__host__ __device__ __forceinline__ size_t slot_floats(int halves, int n_pad) { return (size_t)halves * n_pad * kTileM; }

// ------------------------------------------------------------------------------------------------
// Finishing (the work of gemm_finish_kernel). Every streaming CTA that holds items of a tile has left
// its accumulators in the workspace as [row group][gate|up][node][32 rows] fp32 (a "segment").
__device__ __forceinline__ uint2 pack4_bf16(const __nv_bfloat16 (&h)[4])
{
    uint2 r;
    r.x = (uint32_t)__bfloat16_as_ushort(h[0]) | ((uint32_t)__bfloat16_as_ushort(h[1]) << 16);
    r.y = (uint32_t)__bfloat16_as_ushort(h[2]) | ((uint32_t)__bfloat16_as_ushort(h[3]) << 16);
    return r;
}

// Where CTA cc left its segment of tile `tile`, rows of row group lane_grp: slot tile + cc.
__device__ __forceinline__ const float *share_ptr(const GemmParams &p, const GemmDesc &d, int cc, int tile, int lane_grp)
{
    return p.partials + (size_t)(tile + cc) * slot_floats(d.halves, p.n_pad) + (size_t)lane_grp * d.halves * p.n_pad * 32;
}

// What a warp of the finishing kernel works on.
struct FinishArgs {
    const GemmParams *p;
    const GemmDesc *d;              // in shared memory
    const float *rs;                // per-node factors of the folded input norm (shared memory)
    int tile, first_cta, last_cta, lane_grp;
    int it_first, it_step;          // this warp finishes node groups it_first, it_first + it_step, ...
};

// Finishing a 32-row group of an output tile: add the segments of all CTAs that hold part of the
// tile, in CTA order (so the result does not depend on timing), and apply the fused epilogue. What
// this costs is the length of its dependent chain, round trips to L2 and plain instruction latency,
// not bytes. Hence: lane = (node sub-index ns = lane / 8, row quad r4 = lane % 8), iteration `it`
// handles the four output rows 4 * r4 .. + 3 of node 4 * it + ns, everything moves as 16- or 8-byte
// vectors, a rotary pair sits in one thread; the iterations of a group are dealt out to several
// warps of the grid (it_first, it_step); G node groups travel together and kB segments of each are
// loaded at a time, all loads issued before the first use. With `dry` nothing is stored: the
// finishing kernel walks through its code once that way before its input exists (see there).
// One instantiation per epilogue mode: the code is cold whenever it runs, and what that costs is
// the code walked through, not the code that exists.
template <int G, int kB, int MODE>
__device__ __forceinline__ void finish_rows_t(const FinishArgs &fa, int lane, const bool dry)
{
    typedef __nv_bfloat16 T;
    const GemmParams &p = *fa.p;
    const GemmDesc &d = *fa.d;
    const EpiParams &ep = d.ep;
    constexpr int mode = MODE;
    const int n_nodes = ep.n, n_out = ep.n_out, n_pad = p.n_pad;
    constexpr bool dual = MODE == EPI_SWIGLU;      // the one mode with two accumulators per tile (gate, up)
    const bool comp = ep.comp != 0, has_rs = ep.ssq_in != nullptr, has_xg = ep.xg_out != nullptr;
    constexpr bool resid = mode == EPI_RESID;
    const int tile = fa.tile, lane_grp = fa.lane_grp;
    const int ns = lane >> 3, r4 = lane & 7;
    const int row0 = tile * kTileM + lane_grp * 32 + 4 * r4;   // first of this lane's four output rows
    const int n_valid = min(4, n_out - row0);                  // how many of them exist
    const bool rows_ok = n_valid == 4;                         // all modes but EPI_PLAIN have n_out % 4 == 0
    const int n_parts = fa.last_cta - fa.first_cta + 1;
    if (!LLMCAD_CHECK(fa.first_cta >= 0 && fa.last_cta < d.grid && tile < d.n_tiles && row0 >= 0, p.status)) return;
    if (mode == EPI_QKV && !LLMCAD_CHECK(ep.P + n_nodes <= ep.S && row0 < 3 * ep.d, p.status)) return;

    // per-lane constants of the mode
    float gain[4] = {0.f, 0.f, 0.f, 0.f};
    int sec = 0, head = 0, e = 0, cidx = 0;
    if (resid && has_xg && rows_ok) {
        const uint2 g4 = __ldg(reinterpret_cast<const uint2 *>(reinterpret_cast<const T *>(ep.gain_next) + row0));
        gain[0] = __uint_as_float(g4.x << 16); gain[1] = __uint_as_float(g4.x & 0xffff0000u);
        gain[2] = __uint_as_float(g4.y << 16); gain[3] = __uint_as_float(g4.y & 0xffff0000u);
    } else if (mode == EPI_QKV) {
        sec = row0 / ep.d; cidx = row0 - sec * ep.d;
        head = cidx / ep.hd; e = cidx - head * ep.hd;
    }
    // what a node's epilogue reads besides the shares: the residual (EPI_RESID) or the rotary
    // (cos, sin) of the lane's two pairs (EPI_QKV, q and k sections)
    const float *aux = nullptr;
    size_t aux_stride = 0;
    if (rows_ok && resid) { aux = ep.x + row0; aux_stride = (size_t)n_out; }
    if (rows_ok && mode == EPI_QKV && sec < 2) { aux = reinterpret_cast<const float *>(ep.rope_cs) + 2 * (e >> 1); aux_stride = (size_t)ep.hd; }
    const float4 aux_none = resid ? make_float4(0.f, 0.f, 0.f, 0.f) : make_float4(1.f, 0.f, 1.f, 0.f);

    const int iters = n_pad >> 2;
    for (int itg = fa.it_first; itg < iters; itg += G * fa.it_step) {
        // every load of the G iterations is issued before the first use
        float4 axs[G], as[G], bs[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const int node = min(itg + g * fa.it_step, iters - 1) * 4 + ns;
            axs[g] = aux_none;
            if (aux != nullptr && node < n_nodes) axs[g] = __ldcg(reinterpret_cast<const float4 *>(aux + (size_t)node * aux_stride));
            as[g] = bs[g] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int k0 = 0; k0 < n_parts; k0 += kB) {
            float4 t[G][kB], u[G][kB];
#pragma unroll
            for (int k = 0; k < kB; ++k) {
                const float *sk = share_ptr(p, d, fa.first_cta + min(k0 + k, n_parts - 1), tile, lane_grp) + 4 * r4;
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const int node = min(itg + g * fa.it_step, iters - 1) * 4 + ns;
                    t[g][k] = __ldcg(reinterpret_cast<const float4 *>(sk + (size_t)node * 32));
                    if (dual) u[g][k] = __ldcg(reinterpret_cast<const float4 *>(sk + (size_t)(n_pad + node) * 32));
                }
            }
#pragma unroll
            for (int k = 0; k < kB; ++k) {
                if (k0 + k < n_parts) {          // CTA order
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        as[g].x += t[g][k].x; as[g].y += t[g][k].y; as[g].z += t[g][k].z; as[g].w += t[g][k].w;
                        if (dual) { bs[g].x += u[g][k].x; bs[g].y += u[g][k].y; bs[g].z += u[g][k].z; bs[g].w += u[g][k].w; }
                    }
                }
            }
        }
        // two at a time, unrolled, so that the two dependent chains overlap
        for (int g2 = 0; g2 < G; g2 += 2) {
#pragma unroll
        for (int gq = 0; gq < (G < 2 ? G : 2); ++gq) {
        const int g = g2 + gq;
        const int it = itg + g * fa.it_step;
        if (it >= iters) continue;
        const int node = it * 4 + ns;
        const bool ok = rows_ok && node < n_nodes;
        float4 ax = axs[0], a = as[0], b = bs[0];
#pragma unroll
        for (int q = 1; q < G; ++q) if (q == g) { ax = axs[q]; a = as[q]; b = bs[q]; }
        const float r = has_rs ? fa.rs[node] : 1.f;
        float v[4] = {a.x * r, a.y * r, a.z * r, a.w * r};
        float out[4];                 // what goes out in the activation format (hi and lo plane)
        T *dst = nullptr, *dst_lo = nullptr;
        if (resid) {
            const float xo[4] = {ok ? ax.x + v[0] : 0.f, ok ? ax.y + v[1] : 0.f, ok ? ax.z + v[2] : 0.f, ok ? ax.w + v[3] : 0.f};
            if (ok && !dry) *reinterpret_cast<float4 *>(ep.x + (size_t)node * n_out + row0) = make_float4(xo[0], xo[1], xo[2], xo[3]);
#pragma unroll
            for (int k = 0; k < 4; ++k) out[k] = xo[k] * gain[k];
            if (has_xg) {
                // what the next RMSNorm needs: gain * x in the GEMM input format, and this row
                // group's share of every node's sum of squares
                dst = reinterpret_cast<T *>(ep.xg_out) + (size_t)node * n_out + row0;
                dst_lo = dst + (size_t)kLoRows * n_out;
                float ss = xo[0] * xo[0] + xo[1] * xo[1] + xo[2] * xo[2] + xo[3] * xo[3];
                ss += __shfl_xor_sync(0xffffffffu, ss, 1);
                ss += __shfl_xor_sync(0xffffffffu, ss, 2);
                ss += __shfl_xor_sync(0xffffffffu, ss, 4);
                if (r4 == 0 && !dry) ep.ssq_out[(size_t)(tile * 4 + lane_grp) * LLMCAD_MAX_TREE + node] = ss;
            }
        } else if (mode == EPI_SWIGLU) {
#pragma unroll
            for (int k = 0; k < 4; ++k) out[k] = v[k] / (1.0f + __expf(-v[k]));
            out[0] *= b.x * r; out[1] *= b.y * r; out[2] *= b.z * r; out[3] *= b.w * r;
            dst = reinterpret_cast<T *>(ep.h) + (size_t)node * n_out + row0;
            dst_lo = dst + (size_t)kLoRows * n_out;
        } else if (mode == EPI_QKV) {
            // rotary pairs (2t, 2t+1) = (v0, v1), (v2, v3); values pass through with (cos, sin) = (1, 0)
            out[0] = v[0] * ax.x - v[1] * ax.y; out[1] = v[0] * ax.y + v[1] * ax.x;
            out[2] = v[2] * ax.z - v[3] * ax.w; out[3] = v[2] * ax.w + v[3] * ax.z;
            // queries get a lo plane; keys and values go to the cache rounded, their remainders to kv_lo
            if (sec == 0) {
                dst = reinterpret_cast<T *>(ep.q_out) + (size_t)node * ep.d + cidx;
                dst_lo = dst + (size_t)kLoRows * ep.d;
            } else {
                dst = reinterpret_cast<T *>(sec == 1 ? ep.k_cache : ep.v_cache) + ((size_t)head * ep.S + ep.P + node) * ep.hd + e;
                dst_lo = reinterpret_cast<T *>(ep.kv_lo) + ((size_t)((sec - 1) * (ep.d / ep.hd) + head) * kLoRows + node) * ep.hd + e;
            }
        } else if (node < n_nodes && !dry) {
            float *yr = ep.y + (size_t)node * ep.ldy + row0;
            if (rows_ok && (ep.ldy & 3) == 0 && (reinterpret_cast<uintptr_t>(ep.y) & 15) == 0)
                *reinterpret_cast<float4 *>(yr) = make_float4(v[0], v[1], v[2], v[3]);
            else {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (k < n_valid) yr[k] = v[k];
            }
        }
        if (dst != nullptr && ok && !dry) {
            T hi[4], lo[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) split_bf16(out[k], hi[k], lo[k]);
            *reinterpret_cast<uint2 *>(dst) = pack4_bf16(hi);
            if (comp) *reinterpret_cast<uint2 *>(dst_lo) = pack4_bf16(lo);
        }
        }
        }
    }
}

}  // namespace

#define LLMCAD_TRACE(slot) do { if (p.trace && blockIdx.x < 256) p.trace[(size_t)blockIdx.x * 16 + (slot)] = global_timer_ns(); } while (0)

template <int PK, bool W4>
__global__ void __launch_bounds__(kThreads, 1)
gemm_stream_kernel(const __grid_constant__ GemmMaps maps, const __grid_constant__ GemmParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ SharedCtl ctl;
    const GemmDesc &d = p.g;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t nb = (uint32_t)p.n_pad * (p.comp ? 2u : 1u);   // activation rows per k-block = the MMA N: nodes (hi | lo)
    const uint32_t b_tile_bytes = nb * kBlockK * 2;
    // stage: [weights k-block 0 | weights k-block 1 | activations k-block 0 | activations k-block 1]
    const uint32_t stage_bytes = PK * (kATileBytes + b_tile_bytes);
    const uint32_t b_off = PK * kATileBytes;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // INT4 weights: three rings of their own. [p.stages expanded weight items of PK bf16 tiles, written by the dump
    // warps and read by the MMA][p.astages activation items, PK k-blocks each, filled by the activation loader as far
    // ahead as slots are free][p.pstages packed items of PK tiles of 4224 bytes each, filled by the weight producer].
    // Every item needs its activation tiles from L2 (~1.5 us under load) and they are larger than its packed weights:
    // kept in the stage of the expanded weights, as in the bf16 path, too few of them would be in flight.
    constexpr uint32_t pstage_bytes = PK * kW4TileBytes;
    constexpr uint32_t wstage_bytes = PK * kATileBytes;
    const uint32_t astage_bytes = PK * b_tile_bytes;
    const uint32_t act_base = smem_base + (uint32_t)p.stages * wstage_bytes;
    const uint32_t packed_base = W4 ? act_base + (uint32_t)p.astages * astage_bytes : smem_base + (uint32_t)p.stages * stage_bytes;
    const uint32_t acc_cols = 2u * nb;                    // TMEM columns of one accumulator buffer (gate | up)
    const bool two_bufs = p.acc_bufs == 2;
    const uint64_t wait_limit = p.wait_limit_ns;          // every wait below gives up after this many ns
    const DepWait dep{p.dep_ctr, p.dep_target, wait_limit};

    if (threadIdx.x == 0) LLMCAD_TRACE(0);

    // State of the weight producer (thread 0). It lives across the start-up barrier: the first
    // ring-full of copies goes out right after the barriers are initialised, before TMEM allocation
    // and before the other warps are even needed. Until pdl_wait() this kernel only prefetches
    // weights, which no kernel writes.
    Cursor<PK> pc;
    int ps = 0;
    uint32_t ppar = 1, pissued = 0;    // a fresh barrier passes a wait on parity 1: no special first lap
    uint64_t pol_stream = 0;
    auto issue_item = [&]() {          // the next item of the stream into ring stage ps (which must be free)
        const int nk = pc.nk();
        if (W4) {
            // packed tiles go to the packed ring; the dump warps turn them into MMA stages
            const uint32_t pf = smem_u32(&ctl.pfull[ps]);
            mbar_expect_tx(pf, (uint32_t)nk * kW4TileBytes);
            const size_t t = (size_t)(pc.tile + (pc.half ? d.up_tile_offset : 0)) * d.kb_per_tile + pc.kb0();
            bulk_load_1d(packed_base + ps * pstage_bytes, d.w_tiled + t * kW4TileBytes, (uint32_t)nk * kW4TileBytes, pf, pol_stream);
            if (pissued == 0) LLMCAD_TRACE(2);
            ++pissued;
            pc.advance();
            if (++ps == p.pstages) { ps = 0; ppar ^= 1u; }
            return;
        }
        const uint32_t full = smem_u32(&ctl.full[ps]);
        const uint32_t dst = smem_base + ps * stage_bytes;
        mbar_expect_tx(full, (uint32_t)nk * (kATileBytes + b_tile_bytes));
        if (d.w_tiled != nullptr) {
            // consecutive k-blocks of a tile are contiguous in the tiled layout: one copy
            const size_t t = (size_t)(pc.tile + (pc.half ? d.up_tile_offset : 0)) * d.kb_per_tile + pc.kb0();
            bulk_load_1d(dst, d.w_tiled + t * kATileBytes, (uint32_t)nk * kATileBytes, full, pol_stream);
        } else {
            for (int k = 0; k < nk; ++k)
                tma_load_2d(dst + k * kATileBytes, &maps.w, (pc.kb0() + k) * kBlockK,
                            (pc.half ? d.up_row_offset : 0) + pc.tile * kTileM, full, pol_stream);
        }
        __threadfence_block();
        if (pissued == 0) LLMCAD_TRACE(2);
        ctl.a_issued = ++pissued;      // the activation loader may now add its bytes to this stage
        pc.advance();
        if (++ps == p.stages) { ps = 0; ppar ^= 1u; }
    };
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            // INT4: an expanded weight item is full when the four dump warps have written their quarters of it
            mbar_init(smem_u32(&ctl.full[s]), W4 ? 4 : 1);
            mbar_init(smem_u32(&ctl.empty[s]), 1);
        }
        if (W4) {
            for (int s = 0; s < p.pstages; ++s) {
                mbar_init(smem_u32(&ctl.pfull[s]), 1);
                mbar_init(smem_u32(&ctl.pempty[s]), 4);
            }
            for (int s = 0; s < p.astages; ++s) {
                mbar_init(smem_u32(&ctl.afull[s]), 1);
                mbar_init(smem_u32(&ctl.aempty[s]), 1);
            }
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.tmem_full[b]), 1);
            mbar_init(smem_u32(&ctl.tmem_empty[b]), 4);
        }
        ctl.abort_flag = 0;
        ctl.a_issued = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
        pc.init(d);
        while (!pc.done() && pissued < (uint32_t)(W4 ? p.pstages : p.stages)) issue_item();
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
        // ================================================= weight producer
        // Streams this CTA's weight tiles, in order, as fast as ring slots free up.
        if (lane == 0) {
            // (Asking L2 for weights ahead of the ring while it is blocked, or for the first items of the next GEMM
            // once this CTA's are all requested, or from the finishing kernel while HBM idles, was measured on B200
            // and costs more than it brings in every combination: 3.12 ms per pass of the 7B shape without against
            // 3.14-3.34 ms with 2-8 items ahead and 3-24 items of the next GEMM. The stream runs from HBM straight
            // into the ring.)
            uint64_t t_idle = 0;
            while (!pc.done()) {
                if (mbar_try(smem_u32(W4 ? &ctl.pempty[ps] : &ctl.empty[ps]), ppar)) {
                    issue_item();
                    t_idle = 0;
                    continue;
                }
                __nanosleep(32);
                if (t_idle == 0) t_idle = global_timer_ns();
                else if (*abort_flag || global_timer_ns() - t_idle > wait_limit) { timed_out = true; break; }
            }
            LLMCAD_TRACE(6);
        }
    } else if (warp == 6) {
        // ================================================= activation loader
        // Follows the weight producer item by item and adds the (small, L2-resident) activation
        // tiles of each item, once the grid dependency says that the GEMM's input is final.
        if (lane == 0) {
            uint64_t pol_keep;
            asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_keep));
            Cursor<PK> c;
            c.init(d);
            int s = 0;
            uint32_t i = 0;
            if (!dep_wait_thread(dep)) timed_out = true;
            fence_proxy_async();          // the activations were written by ordinary stores; the copies below read them
            pdl_launch_dependents();
            if (W4) {
                // a ring of its own: item i goes to slot i % astages as soon as the MMAs of item i - astages have read it
                uint32_t apar = 1;         // a fresh barrier passes a wait on parity 1
                while (!c.done() && !timed_out && !p.withhold_act) {
                    if (!mbar_wait(smem_u32(&ctl.aempty[s]), apar, abort_flag, wait_limit)) { timed_out = true; break; }
                    const uint32_t full = smem_u32(&ctl.afull[s]);
                    const uint32_t dst = act_base + s * astage_bytes;
                    const int nk = c.nk();
                    mbar_expect_tx(full, (uint32_t)nk * b_tile_bytes);
                    for (int k = 0; k < nk; ++k)
                        tma_load_3d(dst + k * b_tile_bytes, &maps.x, (c.kb0() + k) * kBlockK, full, pol_keep);
                    c.advance();
                    if (++s == p.astages) { s = 0; apar ^= 1u; }
                }
            }
            while (!W4 && !c.done() && !timed_out && !p.withhold_act) {
                uint64_t t0 = 0;
                // the stage is ours: the producer has passed its "empty" wait and armed the barrier
                for (uint32_t spin = 0; (int32_t)(ctl.a_issued - (i + 1)) < 0; ++spin) {
                    __nanosleep(32);
                    if ((spin & 255u) == 255u) {
                        if (t0 == 0) t0 = global_timer_ns();
                        if (*abort_flag || global_timer_ns() - t0 > wait_limit) { timed_out = true; break; }
                    }
                }
                if (timed_out) break;
                const uint32_t full = smem_u32(&ctl.full[s]);
                const uint32_t dst = smem_base + s * stage_bytes + b_off;
                const int nk = c.nk();
                for (int k = 0; k < nk; ++k)
                    tma_load_3d(dst + k * b_tile_bytes, &maps.x, (c.kb0() + k) * kBlockK, full, pol_keep);
                c.advance();
                ++i;
                if (++s == p.stages) s = 0;
            }
        }
    } else if (warp == 1) {
        // ================================================= MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_idesc(kTileM, (int)nb);
            Cursor<PK> c;
            c.init(d);
            uint32_t seg = 0, ph = 0;   // ph: parity the MMA warp waits for on its stage's "full" barrier
            int s = 0;
            int as = 0;                 // INT4: slot of the activation ring, and the parity waited for on its "full" barrier
            uint32_t aph = 0;
            while (!c.done() && !timed_out) {
                // one segment: the items of one tile that belong to this CTA
                const int tile = c.tile, halves = c.halves;
                const int buf = two_bufs ? (seg & 1) : 0;
                const uint32_t use = two_bufs ? (seg >> 1) : seg;     // how often this buffer has been used before
                if (!mbar_wait(smem_u32(&ctl.tmem_empty[buf]), (use & 1u) ^ 1u, abort_flag, wait_limit)) { timed_out = true; break; }
                tc_fence_after();
                const uint32_t d0 = tmem_base + buf * acc_cols;
                for (int q = 0; !c.done() && c.tile == tile; ++q) {
                    if (!mbar_wait(smem_u32(&ctl.full[s]), ph, abort_flag, wait_limit)) { timed_out = true; break; }
                    if (W4 && !mbar_wait(smem_u32(&ctl.afull[as]), aph, abort_flag, wait_limit)) { timed_out = true; break; }
                    tc_fence_after();
                    const uint32_t a_addr = W4 ? smem_base + s * wstage_bytes : smem_base + s * stage_bytes;
                    const uint32_t b_addr = W4 ? act_base + as * astage_bytes : a_addr + b_off;
                    // segments of a two-half GEMM start on a gate item, so the first `halves` items
                    // of a segment are the ones that must overwrite their accumulator
                    const uint32_t dcol = d0 + c.half * nb;
                    const int nk = c.nk();
                    for (int k = 0; k < nk; ++k) {
                        const uint64_t a_desc = make_smem_desc(a_addr + k * kATileBytes);
                        const uint64_t b_desc = make_smem_desc(b_addr + k * b_tile_bytes);
#pragma unroll
                        for (int k4 = 0; k4 < kBlockK / 16; ++k4) {
                            // advancing 16 bf16 = 32 bytes inside the swizzle row: +2 in the >>4 address field
                            tc_mma_bf16(dcol, a_desc + 2 * k4, b_desc + 2 * k4, idesc, (q >= halves || k > 0 || k4 > 0) ? 1u : 0u);
                        }
                    }
                    tc_commit(smem_u32(&ctl.empty[s]));  // frees the stage when these MMAs have read it
                    if (W4) {
                        tc_commit(smem_u32(&ctl.aempty[as]));
                        if (++as == p.astages) { as = 0; aph ^= 1u; }
                    }
                    c.advance();
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
                if (timed_out) break;
                tc_commit(smem_u32(&ctl.tmem_full[buf]));
                ++seg;
            }
            LLMCAD_TRACE(7);
        }
    } else {
        // ================================================= accumulator dump (warps 2..5)
        const int lane_grp = warp & 3;                 // TMEM lanes 32*lane_grp .. +31 belong to this warp
        // the workspace may still be read by the finishing kernel of the previous GEMM
        bool dep_ok = false;
        if (!W4) {
            if (!dep_wait_warp(dep, lane)) timed_out = true;
            pdl_launch_dependents();
            dep_ok = true;
            if (threadIdx.x == 64) LLMCAD_TRACE(3);
        }
        const Range r = cta_range<PK>(d, (int)blockIdx.x);
        const int ipt = pairs_per_tile_c<PK>(d) * d.halves;
        const size_t slot_stride = slot_floats(d.halves, p.n_pad);
        // ---- INT4 weights: these warps also turn every packed item into the bf16 tiles the MMA reads, a quarter
        // of the rows each, in the next free slot of the ring of expanded items. Element j of a word sits where
        // (word >> 4k) & 0x000f000f picks elements 2k, 2k+1; OR-ing 0x4300 into each half makes the bf16 values
        // 128 + u (u = q + 8), and one fused multiply-add per pair, (128 + u) * 2^e - 136 * 2^e, gives q * 2^e exactly.
        Cursor<PK> dc;
        dc.init(d);
        int ds = 0, dps = 0;
        uint32_t dpar = 1, dppar = 0;                  // a fresh "empty" barrier passes a wait on parity 1
        uint8_t *const smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
        auto dequant_item = [&]() -> bool {
            const int nk = dc.nk();
            if (!mbar_wait_warp(smem_u32(&ctl.empty[ds]), dpar, abort_flag, lane, wait_limit)) return false;
            if (!mbar_wait_warp(smem_u32(&ctl.pfull[dps]), dppar, abort_flag, lane, wait_limit)) return false;
            const uint8_t *pk = smem_gen + (packed_base - smem_base) + (size_t)dps * pstage_bytes;
            uint8_t *wt = smem_gen + (size_t)ds * wstage_bytes;
            // lane = (row within a group of four, chunk): iteration `it` handles row 32 * lane_grp + 4 * it + lane / 8,
            // words and stores of a warp instruction are contiguous (no bank conflicts). All loads of a k-block go
            // out before the first conversion: a warp is alone on its scheduler here, so latency is what counts.
            const int r_in = lane >> 3, c = lane & 7;
            for (int k = 0; k < nk; ++k) {
                const uint32_t *words = reinterpret_cast<const uint32_t *>(pk + (size_t)k * kW4TileBytes) + (lane_grp * 32 + r_in) * 8 + c;
                const int8_t *exps = reinterpret_cast<const int8_t *>(pk + (size_t)k * kW4TileBytes + 4096) + lane_grp * 32 + r_in;
                uint8_t *dst = wt + (size_t)k * kATileBytes + (size_t)(lane_grp * 32 + r_in) * 128;
                uint32_t x[8];
                int e[8];
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    x[it] = words[it * 32];
                    e[it] = exps[it * 4];
                }
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const uint32_t s16 = (uint32_t)(e[it] + 127) << 7;                       // bf16 bits of 2^e
                    const uint32_t b16 = 0x8000u | ((uint32_t)(e[it] + 134) << 7) | 8u;      // bf16 bits of -136 * 2^e
                    const uint32_t s2 = s16 | (s16 << 16), b2 = b16 | (b16 << 16);
                    uint32_t o[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t t2 = ((x[it] >> (4 * j)) & 0x000f000fu) | 0x43004300u;
                        const __nv_bfloat162 rr = __hfma2(*reinterpret_cast<const __nv_bfloat162 *>(&t2),
                                                          *reinterpret_cast<const __nv_bfloat162 *>(&s2),
                                                          *reinterpret_cast<const __nv_bfloat162 *>(&b2));
                        o[j] = *reinterpret_cast<const uint32_t *>(&rr);
                    }
                    // row & 7 = (4 * it + r_in) & 7: the 128-byte swizzle of the MMA tile
                    *reinterpret_cast<uint4 *>(dst + (size_t)it * 512 + ((c ^ ((4 * it + r_in) & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the tensor core reads what these threads wrote
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&ctl.full[ds]));
                mbar_arrive(smem_u32(&ctl.pempty[dps]));
            }
            dc.advance();
            if (++ds == p.stages) { ds = 0; dpar ^= 1u; }
            if (++dps == p.pstages) { dps = 0; dppar ^= 1u; }
            return true;
        };
        uint32_t seg = 0;
        for (int seg_begin = r.begin; seg_begin < r.end && !timed_out; ++seg) {
            const int tile = seg_begin / ipt;
            const int seg_end = min(r.end, (tile + 1) * ipt);
            const int buf = two_bufs ? (seg & 1) : 0;
            const uint32_t use = two_bufs ? (seg >> 1) : seg;
            if (W4) {
                for (int i = seg_begin; i < seg_end && !timed_out; ++i)
                    if (!dequant_item()) timed_out = true;
                if (timed_out) break;
                if (!dep_ok) {          // the workspace may still be read by the previous GEMM's finishing kernel
                    if (!dep_wait_warp(dep, lane)) { timed_out = true; break; }
                    pdl_launch_dependents();
                    dep_ok = true;
                    if (threadIdx.x == 64) LLMCAD_TRACE(3);
                }
            }
            if (!mbar_wait_warp(smem_u32(&ctl.tmem_full[buf]), use & 1u, abort_flag, lane, wait_limit)) { timed_out = true; break; }
            tc_fence_after();
            if (threadIdx.x == 64 && seg == 0) LLMCAD_TRACE(4);
            // this CTA's segment of the tile goes to slot tile + CTA, lane = row of the 32-row group;
            // with hi + lo activations a node's two accumulator columns are added first
            const uint32_t t_lane = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + buf * acc_cols;
            if (!LLMCAD_CHECK(tile >= 0 && tile < d.n_tiles && tile + (int)blockIdx.x < d.n_tiles + d.grid, p.status)) { timed_out = true; break; }
            float *dst = p.partials + (size_t)(tile + (int)blockIdx.x) * slot_stride + (size_t)lane_grp * d.halves * p.n_pad * 32 + lane;
            for (int hf = 0; hf < d.halves; ++hf) {
                int c0 = 0;
                if (p.comp) {
                    // 32 nodes at a time, hi and lo columns in one round trip
                    for (; c0 + 32 <= p.n_pad; c0 += 32) {
                        float v[32];
                        tc_ld32_sum2(t_lane + hf * nb + c0, t_lane + hf * nb + p.n_pad + c0, v);
#pragma unroll
                        for (int j = 0; j < 32; ++j) dst[(size_t)(hf * p.n_pad + c0 + j) * 32] = v[j];
                    }
                }
                for (; c0 < p.n_pad; c0 += 16) {
                    float v[16];
                    tc_ld16(t_lane + hf * nb + c0, v);
                    if (p.comp) {
                        float t[16];
                        tc_ld16(t_lane + hf * nb + p.n_pad + c0, t);
#pragma unroll
                        for (int j = 0; j < 16; ++j) v[j] += t[j];
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) dst[(size_t)(hf * p.n_pad + c0 + j) * 32] = v[j];
                }
            }
            // the accumulator has left TMEM: hand the buffer back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl.tmem_empty[buf]));
            seg_begin = seg_end;
        }
        if (threadIdx.x == 64) LLMCAD_TRACE(8);
    }
    __syncwarp();   // lanes that skipped their role's single-thread section rejoin their warp here
    timed_out = __any_sync(0xffffffffu, timed_out);   // keep the warp together on the way out
    // this dump warp's segments are in the workspace (also said after a wait ran out, so that nobody waits for this CTA)
    if (warp >= 2 && warp <= 5 && lane == 0) dep_arrive(p.s_done);

    if (timed_out) {
        *abort_flag = 1;
        atomicCAS(p.status, 0, LLMCAD_ERR_TIMEOUT);
        // give copies that may still be in flight time to land before the shared memory goes away
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)p.tmem_cols) : "memory");
        if (lane == 0) LLMCAD_TRACE(13);
    }
}

// Adds the segments of every tile and applies the fused epilogue; see the head of the file. The
// work is cut into (tile, 32-row group) pairs; k warps share a pair's node groups, k chosen so that
// all warps of the grid have work. G node groups and KB segments of each are loaded in one go
// (the launcher picks them so that a warp normally needs a single round trip to L2).
//
// Until the grid dependency (the streaming kernel) resolves, the CTA has nothing to do but sits on
// its SM already. It uses the time (a) to read what earlier GEMMs left: the description, the norm
// sums, the gains; (b) for a dry run of its own work with the stores switched off, on whatever the
// workspace holds: the code of this kernel runs once per launch and would be fetched from L2 line
// by line otherwise, which costs more than the work itself.
template <int MODE, int G, int KB>
__global__ void __maxnreg__(kFinMaxRegs)
gemm_finish_kernel(const __grid_constant__ GemmParams p)
{
    // The finishing code reads the GEMM's description (pointers, sizes, mode) all over. From the kernel
    // parameters every first touch of a constant-cache line is a miss; a copy in shared memory costs
    // nothing to read.
    __shared__ __align__(16) GemmDesc s_desc;
    __shared__ float s_part[kFinThreads / LLMCAD_MAX_TREE][LLMCAD_MAX_TREE];
    __shared__ float s_rs[LLMCAD_MAX_TREE];
    {
        static_assert(sizeof(GemmDesc) % 4 == 0, "GemmDesc is copied word by word");
        const uint32_t *src = reinterpret_cast<const uint32_t *>(&p.g);
        uint32_t *dst = reinterpret_cast<uint32_t *>(&s_desc);
        for (int i = threadIdx.x; i < (int)(sizeof(GemmDesc) / 4); i += kFinThreads) dst[i] = src[i];
    }
    pdl_launch_dependents();     // the next GEMM's streaming kernel may take the SMs as they free up
    if (threadIdx.x == 0) LLMCAD_TRACE(9);
    // what earlier GEMMs left (norm sums, residual, gains) is final: the streaming kernel of this GEMM
    // waited for the same counter before it let this kernel launch, so this returns at once
    bool late = false;
    if (threadIdx.x == 0 && p.dep_ctr != nullptr) late = !dep_wait_thread(DepWait{p.dep_ctr, p.dep_target, p.wait_limit_ns});
    __syncthreads();
    const GemmDesc &d = s_desc;
    const EpiParams &ep = d.ep;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- RMSNorm of the GEMM input folded into the epilogue: the producer of the residual stream
    // left partial sums of squares per node ([parts][128]); the accumulators of node i are multiplied
    // by rsqrt(mean(x^2) + eps). Three threads per node add every third partial row, in a fixed order.
    if (ep.ssq_in != nullptr) {
        constexpr int kSlices = kFinThreads / LLMCAD_MAX_TREE;
        const int node = threadIdx.x & (LLMCAD_MAX_TREE - 1), slice = threadIdx.x / LLMCAD_MAX_TREE;
        float acc = 0.f;
        if (node < p.n_pad) {
            const float *col = ep.ssq_in + node;
            int t = slice;
            for (; t + 7 * kSlices < ep.ssq_in_parts; t += 8 * kSlices) {
                float v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = __ldcg(col + (size_t)(t + kSlices * u) * LLMCAD_MAX_TREE);
#pragma unroll
                for (int u = 0; u < 8; ++u) acc += v[u];
            }
            for (; t < ep.ssq_in_parts; t += kSlices) acc += __ldcg(col + (size_t)t * LLMCAD_MAX_TREE);
        }
        s_part[slice][node] = acc;
        __syncthreads();
        if (threadIdx.x < LLMCAD_MAX_TREE) {
            float sum = 0.f;
#pragma unroll
            for (int q = 0; q < kSlices; ++q) sum += s_part[q][threadIdx.x];
            s_rs[threadIdx.x] = rsqrtf(sum / (float)ep.norm_d + ep.eps);
        }
        __syncthreads();
    }

    const int ipt = pairs_per_tile(d) * d.halves;
    const int pairs = d.n_tiles * 4, iters = p.n_pad >> 2;
    const int W = (int)gridDim.x * (kFinThreads / 32);
    int k = W / pairs;
    k = k < 1 ? 1 : (k > iters ? iters : k);
    const int groups = W / k;
    const int wg = warp * (int)gridDim.x + (int)blockIdx.x;      // consecutive pairs on different SMs

    for (int round = 0; round < 2; ++round) {
        const bool dry = round == 0;
        if (!dry) {
            // every segment is in the workspace
            if (p.s_done == nullptr) pdl_wait();
            else {
                if (threadIdx.x == 0) late |= !dep_wait_thread(DepWait{p.s_done, 4u * (uint32_t)d.grid, p.wait_limit_ns});
                __syncthreads();
            }
            if (threadIdx.x == 0) LLMCAD_TRACE(10);
        }
        if (wg < groups * k) {
            for (int pair = wg / k; pair < pairs; pair += groups) {
                FinishArgs fa;
                fa.p = &p; fa.d = &d; fa.rs = s_rs;
                fa.tile = pair >> 2; fa.lane_grp = pair & 3;
                const int tile_i0 = fa.tile * ipt;
                fa.first_cta = tile_i0 / d.items_per_cta;
                fa.last_cta = (tile_i0 + ipt - 1) / d.items_per_cta;
                fa.it_first = wg % k; fa.it_step = k;
                finish_rows_t<G, KB, MODE>(fa, lane, dry);
                if (dry) break;          // one pair is enough to have walked through the code
            }
        }
    }
    if (p.f_done != nullptr) {
        __syncthreads();             // all of this CTA's results are written
        if (threadIdx.x == 0) {
            if (late) atomicCAS(p.status, 0, LLMCAD_ERR_TIMEOUT);
            dep_arrive(p.f_done);
        }
    }
    if (threadIdx.x == 0) LLMCAD_TRACE(12);
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

bool make_act_map_bf16(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t planes,
                       uint64_t plane_rows)
{
    auto fn = get_encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t dims[3] = {cols, rows, planes};
    cuuint64_t strides[2] = {cols * 2, plane_rows * cols * 2};
    cuuint32_t box[3] = {(cuuint32_t)kBlockK, box_rows, planes};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_tensor_map_bf16_3d(CUtensorMap *map, const void *base, const uint64_t dims[3], const uint64_t strides_bytes[2],
                             const uint32_t box[3])
{
    auto fn = get_encode_fn();
    if (fn == nullptr) return false;
    cuuint64_t d[3] = {dims[0], dims[1], dims[2]};
    cuuint64_t s[2] = {strides_bytes[0], strides_bytes[1]};
    cuuint32_t b[3] = {box[0], box[1], box[2]};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), d, s, b, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

size_t gemm_tc_partial_floats(int n_sms, int max_tiles, int max_n_pad) { return (size_t)(max_tiles + n_sms) * slot_floats(2, max_n_pad); }

GemmDesc make_gemm_desc(int n_in, const EpiParams &ep, const void *w_tiled, bool w4)
{
    GemmDesc d{};
    d.halves = ep.mode == EPI_SWIGLU ? 2 : 1;
    d.n_tiles = (ep.n_out + kTileM - 1) / kTileM;
    d.kb_per_tile = (n_in + kBlockK - 1) / kBlockK;
    d.pair_k = kMaxPairK;
    d.up_row_offset = ep.n_out;
    d.items_per_cta = 0;
    d.grid = 0;
    d.w_tiled = static_cast<const uint8_t *>(w_tiled);
    d.up_tile_offset = d.n_tiles;
    d.w4 = w4 ? 1 : 0;
    d.ep = ep;
    return d;
}

namespace {
// tuning aids from the environment, read once per process
struct Tuning {
    int pair_k = 0, stages_cap = 0, w4_wstages = 3, w4_pstages = 4;
    Tuning()
    {
        if (const char *e = getenv("LLMCAD_GEMM_PAIR_K")) { const int v = atoi(e); if (v == 1 || v == 2) pair_k = v; }
        if (const char *e = getenv("LLMCAD_GEMM_STAGES")) { const int v = atoi(e); if (v >= 2) stages_cap = v; }
        if (const char *e = getenv("LLMCAD_W4_WSTAGES")) { const int v = atoi(e); if (v >= 2 && v <= kMaxStages) w4_wstages = v; }
        if (const char *e = getenv("LLMCAD_W4_PSTAGES")) { const int v = atoi(e); if (v >= 2 && v <= kMaxPStages) w4_pstages = v; }
    }
};
const Tuning &tuning()
{
    static const Tuning t;
    return t;
}
}  // namespace

cudaError_t plan_gemm_tc(GemmParams &p, int n_sms)
{
    const Tuning &tune = tuning();
    // Ring items of two k-blocks (one 32 KB weight copy each) unless the activation tiles are so wide
    // (hi | lo planes of more than 64 nodes) that only two stages would fit; measured on B200:
    // single k-blocks cost 10-17 % up to 64 nodes and gain 6 % at 128.
    const int nb = p.n_pad * (p.comp ? 2 : 1);       // MMA N
    if (nb > 256 || p.n_pad < 16 || p.n_pad % 16) return cudaErrorInvalidValue;
    int pair_k = nb > 128 ? 1 : kMaxPairK;
    if (tune.pair_k) pair_k = tune.pair_k;
    GemmDesc &d = p.g;
    d.pair_k = pair_k;
    // the items are split evenly over one CTA per SM (fewer CTAs when there are fewer items)
    const long long total = (long long)d.n_tiles * pairs_per_tile(d) * d.halves;
    if (total < 1) return cudaErrorInvalidValue;
    int grid = total < n_sms ? (int)total : n_sms;
    long long ipc = (total + grid - 1) / grid;
    if (d.halves == 2) ipc += ipc & 1;   // ranges of a two-half GEMM start on a gate item
    d.items_per_cta = (int)ipc;
    grid = (int)((total + ipc - 1) / ipc);
    d.grid = grid;
    return cudaSuccess;
}

cudaError_t launch_gemm_tc(const GemmMaps &maps, GemmParams &p, int n_sms, size_t partial_floats, cudaStream_t st, int *launched)
{
    if (launched) *launched = 0;
    const Tuning &tune = tuning();
    {
        const cudaError_t e = plan_gemm_tc(p, n_sms);
        if (e != cudaSuccess) return e;
    }
    GemmDesc &d = p.g;
    const int nb = p.n_pad * (p.comp ? 2 : 1);
    const int pair_k = d.pair_k, grid = d.grid;
    const long long ipc = d.items_per_cta;
    if ((size_t)(d.n_tiles + grid) * slot_floats(d.halves, p.n_pad) > partial_floats) return cudaErrorInvalidValue;
    const size_t stage_bytes = (size_t)pair_k * ((size_t)kATileBytes + (size_t)nb * kBlockK * 2);
    // One CTA per SM with the whole shared memory as the ring.
    // accumulators: (gate | up) x MMA N columns each, double-buffered when two of them fit
    p.acc_bufs = 4 * nb <= 512 ? 2 : 1;
    int cols = p.acc_bufs * 2 * nb, pow2 = 32;
    while (pow2 < cols) pow2 <<= 1;
    p.tmem_cols = pow2;
    // the ring takes what the SM has, less the room that the finishing CTA of the previous GEMM needs beside it
    const size_t full_limit = 227 * 1024 - 1024 /*alignment slack*/ - 2048 /*static*/ - (kFinSmem + 4096);
    int stages = (int)(full_limit / stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (tune.stages_cap && tune.stages_cap < stages) stages = tune.stages_cap;   // tuning aid: cap the ring depth
    if (stages < 2) return cudaErrorInvalidConfiguration;
    size_t smem = (size_t)stages * stage_bytes + 1024;
    p.pstages = 0;
    p.astages = 0;
    if (d.w4) {
        // INT4 weights: three rings (see the kernel). Three expanded items (8-layer pass of the 7B shape at 32 nodes:
        // 1.08 ms with two, 0.97 ms with three or four), a few packed items (they are small, 8.4 KB per 32 KB of
        // bf16; 3 to 12 of them measure the same), and the rest of the shared memory for activation items.
        if (d.w_tiled == nullptr) return cudaErrorInvalidValue;
        const size_t pstage = (size_t)pair_k * kW4TileBytes, wstage = (size_t)pair_k * kATileBytes;
        const size_t astage = (size_t)pair_k * nb * kBlockK * 2;
        stages = tune.w4_wstages;
        int pst = tune.w4_pstages;
        if ((size_t)stages * wstage + (size_t)pst * pstage + 2 * astage > full_limit) return cudaErrorInvalidConfiguration;
        int ast = (int)((full_limit - (size_t)stages * wstage - (size_t)pst * pstage) / astage);
        if (ast > kMaxAStages) ast = kMaxAStages;
        // what the activation ring does not use goes to the packed ring
        pst = (int)((full_limit - (size_t)stages * wstage - (size_t)ast * astage) / pstage);
        if (pst > kMaxPStages) pst = kMaxPStages;
        p.pstages = pst;
        p.astages = ast;
        smem = (size_t)stages * wstage + (size_t)ast * astage + (size_t)pst * pstage + 1024;
    }
    p.stages = stages;
    static PerDeviceOnce attr_set;
    if (attr_set.needed()) {
        cudaError_t e = cudaSuccess;
        typedef void (*SKernel)(GemmMaps, GemmParams);
        const SKernel all[4] = {gemm_stream_kernel<1, false>, gemm_stream_kernel<2, false>, gemm_stream_kernel<1, true>, gemm_stream_kernel<2, true>};
        // An SM splits its on-chip memory between shared memory and L1 when it is empty, to fit the kernel that
        // arrives; a streaming CTA of 195 KB would get a 196 KB split, and the finishing CTA of the same GEMM
        // could not settle beside it. Every kernel of the GEMM asks for the largest shared-memory split.
        for (int i = 0; i < 4 && e == cudaSuccess; ++i) {
            e = cudaFuncSetAttribute(all[i], cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(all[i], cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        }
        if (e != cudaSuccess) return e;
        attr_set.mark();
    }
    if (p.wait_limit_ns == 0) p.wait_limit_ns = kDefaultWaitLimitNs;
    {
        LaunchCfg lc(grid, kThreads, smem, st);
        cudaError_t e;
        if (d.w4) e = pair_k == 1 ? cudaLaunchKernelEx(&lc.cfg, gemm_stream_kernel<1, true>, maps, p)
                                  : cudaLaunchKernelEx(&lc.cfg, gemm_stream_kernel<2, true>, maps, p);
        else e = pair_k == 1 ? cudaLaunchKernelEx(&lc.cfg, gemm_stream_kernel<1, false>, maps, p)
                             : cudaLaunchKernelEx(&lc.cfg, gemm_stream_kernel<2, false>, maps, p);
        if (e != cudaSuccess) return e;
        if (launched) ++*launched;
    }
    // finishing: (tile, row group) pairs x node groups of four, one warp-iteration each; G node groups and
    // KB segments per round trip so that the warps get through in one round where registers allow
    const long long units = (long long)d.n_tiles * 4 * (p.n_pad / 4);
    const int warps_per_cta = kFinThreads / 32;
    int fgrid = (int)((units + warps_per_cta - 1) / warps_per_cta);
    if (fgrid > n_sms) fgrid = n_sms;
    const long long per_warp = (units + (long long)fgrid * warps_per_cta - 1) / ((long long)fgrid * warps_per_cta);
    const int max_parts = (int)(((long long)pairs_per_tile(d) * d.halves + ipc - 1) / ipc) + 1;
    const bool wide = max_parts > 4;           // many segments per tile (tiles split over many CTAs)
    const bool two = per_warp >= 2;            // several node groups per warp
    typedef void (*FinKernel)(GemmParams);
    FinKernel fk = nullptr;
#define LLMCAD_PICK(MODE)                                                                                            \
    fk = wide ? (FinKernel)gemm_finish_kernel<MODE, 1, 8>                                                            \
              : (two ? (FinKernel)gemm_finish_kernel<MODE, 2, 4> : (FinKernel)gemm_finish_kernel<MODE, 1, 4>)
    switch (d.ep.mode) {
    case EPI_QKV: LLMCAD_PICK(EPI_QKV); break;
    case EPI_RESID: LLMCAD_PICK(EPI_RESID); break;
    case EPI_SWIGLU:
        fk = wide ? (FinKernel)gemm_finish_kernel<EPI_SWIGLU, 1, 4> : (two ? (FinKernel)gemm_finish_kernel<EPI_SWIGLU, 2, 2> : (FinKernel)gemm_finish_kernel<EPI_SWIGLU, 1, 4>);
        break;
    default: LLMCAD_PICK(EPI_PLAIN); break;
    }
#undef LLMCAD_PICK
    {
        // once per finishing kernel and device (see above)
        static PerDeviceOnce fin_set[4][3];
        PerDeviceOnce &once = fin_set[d.ep.mode & 3][wide ? 0 : (two ? 1 : 2)];
        if (once.needed()) {
            const cudaError_t e = cudaFuncSetAttribute(fk, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
            if (e != cudaSuccess) return e;
            once.mark();
        }
    }
    p.f_grid = fgrid;
    LaunchCfg lf(fgrid, kFinThreads, kFinSmem, st);
    const cudaError_t e = cudaLaunchKernelEx(&lf.cfg, fk, p);
    if (e == cudaSuccess && launched) ++*launched;
    return e;
}

}  // namespace llmcad
