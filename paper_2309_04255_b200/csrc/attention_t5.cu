// Tree-masked attention on the sm_100a tensor cores (tcgen05 + TMEM), bf16, head_dim 128.
//
// Same operation and interface as attention_tc.cu (Sec. 3.2 "Tree decoder": every tree node sees the
// prefix and its own ancestors), for trees large enough that the legacy mma.sync pipe of that
// kernel sets the pace. Per head the key range is split over the CTAs of a cluster (grid = splits x
// heads); a CTA walks its 64-key tiles with
//   warp 0    producer: TMA boxes of K and V (and, for the tiles that hold tree nodes, of the bf16
//             remainders of their K and V) into a ring of shared-memory stages;
//   warp 1    MMA issuer of S = Q K^T into one of two TMEM score buffers (queries on the 128 TMEM
//             lanes, 64 keys on the columns), two tiles ahead of the softmax;
//   warp 6    MMA issuer of O += P V into another TMEM region; the A operands (Q, P) are read from
//             tensor memory, only K and V come from shared memory;
//   warps 2-5 softmax: thread = query row. Puts its row of Q into TMEM once; per tile reads its row of
//             S from TMEM, masks, keeps a running reference and sum, and writes P (hi + lo bf16
//             pairs) back to TMEM for the second MMA, which accumulates the outputs in TMEM over all
//             tiles; the rare move of a row's reference value rescales that row in TMEM.
// Compensated operands (the verification pass): Q and P are hi + lo pairs, so each product takes two
// MMAs per k-step; tiles with tree keys add Q K_lo^T and P V_lo. V is consumed as it lies in the
// cache ([key][dim], dim contiguous) as an MN-major B operand.
// The partial (max, sum, 128 outputs) of every row goes to shared memory; the splits of a head are
// merged through distributed shared memory exactly as in attention_tc.cu.
//
// Every mbarrier wait is bounded; when one runs out the CTA raises its abort flag, sets the status
// word, lets all roles fall through to the common exit (cluster barriers included) and frees TMEM.
#include <cooperative_groups.h>
#include <cuda.h>

#include "attention_tc.cuh"
#include "gemm_tc.cuh"

namespace cg = cooperative_groups;

namespace llmcad {

namespace {

constexpr int kHd = 128;
constexpr int kKeyTile = 64;
constexpr int kT5Threads = 224;                   // producer, score MMAs, four softmax warps, P V MMAs
constexpr int kStages = 6;                       // three tiles in flight, each possibly with a remainder stage
constexpr int kSubTile = 64 * 64 * 2;            // [64 rows][64 columns] bf16, 128-byte rows
constexpr int kStageBytes = 4 * kSubTile;        // K dims 0-63, K dims 64-127, V dims 0-63, V dims 64-127
constexpr int kWsRow = kHd + 4;                  // partial row: 128 outputs, reference, sum, padding to 16 bytes
constexpr int kMaxSplits = 8;
// Tensor memory, all 512 columns of the SM (one CTA per SM): scores of two tiles in flight (fp32, 64
// keys each), the outputs (fp32, 128 dims), and the A operands of both products as packed bf16 pairs
// (one 32-bit column = two consecutive K elements of a row): the softmax weights of two tiles in
// flight (hi and lo, 32 columns each) and the queries (hi and lo, 64 columns each). Operands that sit
// in tensor memory cost no shared-memory bandwidth, which is what bounds small-N MMAs otherwise.
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColO = 128;
constexpr uint32_t kColP = 256;                  // + 64 * buffer, + 32 for the lo half
constexpr uint32_t kColQ = 384;                  // + 64 for the lo half

struct Ctl {
    uint64_t full[kStages];
    uint64_t empty[kStages];
    uint64_t q_full;
    uint64_t s_full[2];
    uint64_t p_full[2];
    uint64_t o_full[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};

constexpr int kQStage = 32 * 256;                   // per softmax warp: 32 query rows of one plane on their way to TMEM
constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + 4 * kQStage + sizeof(Ctl);

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

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
// Bounded wait of one thread: gives up after wait_limit ns or when another role has raised `abort`.
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint64_t wait_limit)
{
    if (mbar_try(bar, parity)) return true;
    uint64_t t0 = 0;
    for (uint32_t it = 1;; ++it) {
        __nanosleep(20);
        if (mbar_try(bar, parity)) return true;
        if ((it & 255u) == 0) {
            if (*abort_flag) return false;
            if (t0 == 0) t0 = global_timer_ns();
            else if (global_timer_ns() - t0 > wait_limit) return false;
        }
    }
}
// The same for a whole warp: lane 0 polls, the warp follows.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int *abort_flag, int lane, uint64_t wait_limit)
{
    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity, abort_flag, wait_limit) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]^T, bf16 inputs, fp32 accumulate, issued by one thread; A sits in tensor
// memory (lanes = rows, one 32-bit column = two bf16 along K).
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 consecutive 32-bit columns of this thread's TMEM lane
__device__ __forceinline__ void tc_st32(uint32_t taddr, const uint32_t *r)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 64 consecutive fp32 columns of this thread's TMEM lane in one instruction (a load and its wait cost
// ~0.2 us however many columns they move, so the score row is fetched whole).
__device__ __forceinline__ void tc_ld64(uint32_t taddr, float *v)
{
    uint32_t r[64];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31]), "=r"(r[32]), "=r"(r[33]), "=r"(r[34]), "=r"(r[35]), "=r"(r[36]), "=r"(r[37]), "=r"(r[38]), "=r"(r[39]), "=r"(r[40]), "=r"(r[41]), "=r"(r[42]), "=r"(r[43]), "=r"(r[44]), "=r"(r[45]), "=r"(r[46]), "=r"(r[47]), "=r"(r[48]), "=r"(r[49]), "=r"(r[50]), "=r"(r[51]), "=r"(r[52]), "=r"(r[53]), "=r"(r[54]), "=r"(r[55]), "=r"(r[56]), "=r"(r[57]), "=r"(r[58]), "=r"(r[59]), "=r"(r[60]), "=r"(r[61]), "=r"(r[62]), "=r"(r[63])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 64; ++j) v[j] = __uint_as_float(r[j]);
}
__device__ __forceinline__ void tc_st64(uint32_t taddr, const float *v)
{
    uint32_t r[64];
#pragma unroll
    for (int j = 0; j < 64; ++j) r[j] = __float_as_uint(v[j]);
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x64.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63, %64};"
        :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31]), "r"(r[32]), "r"(r[33]), "r"(r[34]), "r"(r[35]), "r"(r[36]), "r"(r[37]), "r"(r[38]), "r"(r[39]), "r"(r[40]), "r"(r[41]), "r"(r[42]), "r"(r[43]), "r"(r[44]), "r"(r[45]), "r"(r[46]), "r"(r[47]), "r"(r[48]), "r"(r[49]), "r"(r[50]), "r"(r[51]), "r"(r[52]), "r"(r[53]), "r"(r[54]), "r"(r[55]), "r"(r[56]), "r"(r[57]), "r"(r[58]), "r"(r[59]), "r"(r[60]), "r"(r[61]), "r"(r[62]), "r"(r[63])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptors, 128-byte swizzle (layout type 2 at bits 61-63, version 1 at bit
// 46), start address >> 4 at bits 0-13.
// K-major operand (rows of 64 bf16 = 128 bytes, as a TMA box of 64 columns leaves them): groups of
// 8 rows are 1024 bytes apart (stride byte offset, bits 32-45); the leading byte offset is unused.
__device__ __forceinline__ uint64_t desc_k_major(uint32_t smem_addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// MN-major operand: the same rows, but a row is 64 consecutive values of the N dimension at one k
// (V as it lies in the cache: row = key, 64 head dims). Groups of 8 k are 1024 bytes apart (stride
// byte offset), the next 64 N values `n_chunk_bytes` further (leading byte offset, bits 16-29).
__device__ __forceinline__ uint64_t desc_mn_major(uint32_t smem_addr, uint32_t n_chunk_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
    d |= (uint64_t)((n_chunk_bytes >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor of kind::f16: fp32 accumulator, bf16 A and B, A K-major, B K-major or
// MN-major (bit 16), N >> 3 at bits 17-22, M >> 4 at bits 24-28.
__host__ __device__ constexpr uint32_t make_idesc(int m, int n, bool b_mn_major)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(m >> 4) << 24);
}

// (a, b) as two bf16 pairs: hi = bf16(value), lo = bf16(value - hi).
__device__ __forceinline__ void pack_split(float a, float b, uint32_t &hi, uint32_t &lo)
{
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    const float2 hf = __bfloat1622float2(h);
    __nv_bfloat162 l = __floats2bfloat162_rn(a - hf.x, b - hf.y);
    hi = *reinterpret_cast<uint32_t *>(&h);
    lo = *reinterpret_cast<uint32_t *>(&l);
}

// 2^x, one instruction; 2^(-inf) = +0
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Merge of the splits of a head for the rows split, split + splits, ... of this CTA: out = sum_s O_s
// 2^(m_s - M) / sum_s l_s 2^(m_s - M), from the partials ([128 outputs][reference][sum] per row) in the
// shared memory of the NS (or fewer) CTAs of the cluster. Remote shared memory answers slowly and the
// compiler will not move loads across the stores of an earlier item, so every thread first collects
// the operands of B items (four outputs of one row each) and only then computes and stores.
template <int NS, int B>
__device__ __forceinline__ void merge_splits(const float *part, cg::cluster_group &cluster, int splits, int split, int n,
                                             int n_heads, int head, __nv_bfloat16 *o, size_t lo_off, int comp, int tid)
{
    const float *peer[NS];
#pragma unroll
    for (int sp = 0; sp < NS; ++sp) peer[sp] = sp < splits ? cluster.map_shared_rank(part, sp) : part;
    const int my_rows = (n - split + splits - 1) / splits;
    const int items = my_rows * (kHd / 4);
    for (int base = tid; base < items; base += B * kT5Threads) {
        float2 ml[B][NS];
        float4 ov[B][NS];
#pragma unroll
        for (int b = 0; b < B; ++b) {
            const int idx = min(base + b * kT5Threads, items - 1);      // a clamped item is loaded twice and stored once
            const int row = split + (idx / (kHd / 4)) * splits, dim = (idx % (kHd / 4)) * 4;
#pragma unroll
            for (int sp = 0; sp < NS; ++sp) {
                if (sp < splits) {
                    ml[b][sp] = *reinterpret_cast<const float2 *>(peer[sp] + (size_t)row * kWsRow + kHd);
                    ov[b][sp] = *reinterpret_cast<const float4 *>(peer[sp] + (size_t)row * kWsRow + dim);
                } else {
                    ml[b][sp] = make_float2(-INFINITY, 0.f);
                    ov[b][sp] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
#pragma unroll
        for (int b = 0; b < B; ++b) {
            const int idx = base + b * kT5Threads;
            if (idx >= items) break;
            const int row = split + (idx / (kHd / 4)) * splits, dim = (idx % (kHd / 4)) * 4;
            float M = -INFINITY;
#pragma unroll
            for (int sp = 0; sp < NS; ++sp) M = fmaxf(M, ml[b][sp].x);
            float L = 0.f;
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int sp = 0; sp < NS; ++sp) {
                const float wgt = (ml[b][sp].x == -INFINITY) ? 0.f : ex2(ml[b][sp].x - M);
                L += ml[b][sp].y * wgt;
                a.x += ov[b][sp].x * wgt; a.y += ov[b][sp].y * wgt; a.z += ov[b][sp].z * wgt; a.w += ov[b][sp].w * wgt;
            }
            const float inv = L > 0.f ? 1.f / L : 0.f;
            uint32_t h0, l0, h1, l1;
            pack_split(a.x * inv, a.y * inv, h0, l0);
            pack_split(a.z * inv, a.w * inv, h1, l1);
            __nv_bfloat16 *dst = o + ((size_t)row * n_heads + head) * kHd + dim;
            *reinterpret_cast<uint2 *>(dst) = make_uint2(h0, h1);
            if (comp) *reinterpret_cast<uint2 *>(dst + lo_off) = make_uint2(l0, l1);
        }
    }
}

}  // namespace

// q: [planes][rows][H*128] (the lo plane kLoRows rows after the hi plane);
// map_k, map_v: [H][P + n_tree keys][128], box 64 columns x 64 keys (keys beyond the end read as zero);
// map_lo: [2H][n rows][128] (K remainders of head h at index h, V remainders at H + h; row = query
// index), box 64 columns x 64 rows; the row coordinate of a tile may be negative or run past n.
__global__ void __launch_bounds__(kT5Threads, 1)
attention_t5_kernel(const __nv_bfloat16 *__restrict__ q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_lo, int n_heads, int P,
                    int n, const uint32_t *__restrict__ anc, __nv_bfloat16 *o, int splits, int tiles_per_split,
                    int32_t *status, unsigned long long *trace, int comp, int n_tree, int q_first, uint64_t wait_limit,
                    DepWait dep, uint32_t *done_ctr)
{
    const int cta = blockIdx.y * gridDim.x + blockIdx.x;
    if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 0] = global_timer_ns();
    pdl_launch_dependents();
    extern __shared__ uint8_t sm_raw[];
    const uint32_t raw = smem_u32(sm_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;          // swizzled tiles want 1024-byte alignment
    uint8_t *smp = sm_raw + (base - raw);
    const uint32_t s_ring = base;
    uint8_t *q_stage = smp + (size_t)kStages * kStageBytes;
    Ctl &ctl = *reinterpret_cast<Ctl *>(q_stage + 4 * kQStage);
    float *part = reinterpret_cast<float *>(smp);   // the ring's space, once the loop is over

    const int split = blockIdx.x, head = blockIdx.y;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_keys = P + n_tree;
    const int n_tiles = (n_keys + kKeyTile - 1) / kKeyTile;
    const int t_begin = min(n_tiles, split * tiles_per_split);
    const int t_end = min(n_tiles, t_begin + tiles_per_split);
    const int T = t_end - t_begin;
    const size_t lo_off = (size_t)kLoRows * n_heads * kHd;   // elements from the hi plane of o to its lo plane
    // a tile that reaches into the tree nodes: their K/V come from this layer's QKV GEMM (wait for
    // it), and with compensation their remainders ride along in a second ring stage
    auto reaches_tree = [&](int t) { return (t + 1) * kKeyTile > P; };

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&ctl.full[s]), 1);
            mbar_init(smem_u32(&ctl.empty[s]), 1);
        }
        mbar_init(smem_u32(&ctl.q_full), 4);
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ctl.s_full[b]), 1);
            mbar_init(smem_u32(&ctl.p_full[b]), 4);
            mbar_init(smem_u32(&ctl.o_full[b]), 1);
        }
        ctl.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl.tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl.tmem_base;
    volatile int *abort_flag = &ctl.abort_flag;
    bool failed = false;
    // A pass whose tree or tokens an earlier phase refused (status word set) does no work here: every
    // role looks at the word once the grid dependency has resolved, and all see the same value.
    // (the dependency is the grid dependency or the producer's completion counter; the one thread that feeds the
    // copy engine with data written by ordinary stores puts a proxy fence behind its wait)
    auto refused = [&]() {
        dep_wait_thread(dep);
        fence_proxy_async();
        return *reinterpret_cast<const volatile int32_t *>(status) != 0;
    };
    auto refused_warp = [&]() {
        dep_wait_warp(dep, lane);
        return *reinterpret_cast<const volatile int32_t *>(status) != 0;
    };

    if (warp == 0) {
        // ================================================= producer
        if (lane == 0) {
            int s = 0;
            uint32_t par = 1;          // a fresh barrier passes a wait on parity 1
            auto issue_kv = [&](int t) {
                const uint32_t full = smem_u32(&ctl.full[s]);
                const uint32_t dst = s_ring + s * kStageBytes;
                mbar_expect_tx(full, kStageBytes);
                for (int j = 0; j < 2; ++j) {
                    tma_load_3d(dst + j * kSubTile, &map_k, j * 64, t * kKeyTile, head, full);
                    tma_load_3d(dst + (2 + j) * kSubTile, &map_v, j * 64, t * kKeyTile, head, full);
                }
                if (++s == kStages) { s = 0; par ^= 1u; }
            };
            auto issue_lo = [&](int t) {
                const uint32_t full = smem_u32(&ctl.full[s]);
                const uint32_t dst = s_ring + s * kStageBytes;
                const int row0 = t * kKeyTile - P - q_first;      // query index of the tile's first key
                mbar_expect_tx(full, kStageBytes);
                for (int j = 0; j < 2; ++j) {
                    tma_load_3d(dst + j * kSubTile, &map_lo, j * 64, row0, head, full);
                    tma_load_3d(dst + (2 + j) * kSubTile, &map_lo, j * 64, row0, n_heads + head, full);
                }
                if (++s == kStages) { s = 0; par ^= 1u; }
            };
            // prefix tiles that fit in the ring go out before the grid dependency: earlier passes wrote them
            int t = t_begin, issued = 0;
            while (t < t_end && !reaches_tree(t) && issued < kStages) {
                issue_kv(t++);
                ++issued;
            }
            if (refused()) {
                // nothing will consume the tiles already requested: let them land before the ring goes away
                for (int i = 0; i < issued; ++i) mbar_wait(smem_u32(&ctl.full[i]), 0, abort_flag, wait_limit);
                t = t_end;
            }
            for (; t < t_end && !failed; ++t) {
                if (issued >= kStages && !mbar_wait(smem_u32(&ctl.empty[s]), par, abort_flag, wait_limit)) { failed = true; break; }
                issue_kv(t);
                ++issued;
                if (comp && reaches_tree(t)) {
                    if (issued >= kStages && !mbar_wait(smem_u32(&ctl.empty[s]), par, abort_flag, wait_limit)) { failed = true; break; }
                    issue_lo(t);
                    ++issued;
                }
            }
        }
    } else if (warp == 1) {
        // ================================================= MMA issuer of S = Q K^T
        if (lane == 0 && T > 0 && !refused()) {
            constexpr uint32_t idesc_s = make_idesc(128, kKeyTile, false);
            int s = 0;
            uint32_t ph = 0;
            int st_kv[4] = {0, 0, 0, 0}, st_lo[4] = {-1, -1, -1, -1};   // ring stages of the (up to three) tiles in flight, by tile & 3
            auto issue_s = [&](int i) -> bool {             // S of tile t_begin + i into score buffer i & 1
                const int t = t_begin + i, b = i & 1;
                const bool lo = comp && reaches_tree(t);
                st_kv[i & 3] = s;
                if (!mbar_wait(smem_u32(&ctl.full[s]), ph, abort_flag, wait_limit)) return false;
                if (++s == kStages) { s = 0; ph ^= 1u; }
                st_lo[i & 3] = -1;
                if (lo) {
                    st_lo[i & 3] = s;
                    if (!mbar_wait(smem_u32(&ctl.full[s]), ph, abort_flag, wait_limit)) return false;
                    if (++s == kStages) { s = 0; ph ^= 1u; }
                }
                // (the softmax warps have read tile i - 2 out of this score buffer: their P of that tile, which
                // the caller has waited for, came after it)
                tc_fence_after();
                // One thread issues every MMA, so the code between two of them is what limits the rate:
                // descriptors are a base plus compile-time offsets (address field in units of 16 bytes).
                const uint32_t d = tmem_base + (uint32_t)b * kKeyTile;
                const uint64_t dk = desc_k_major(s_ring + st_kv[i & 3] * kStageBytes);
                // k-step ks = 16 head dims: 8 columns of the queries in tensor memory, 32 bytes in a row of
                // the K sub-tile that holds dims 64 * (ks / 4) ..
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    tc_mma_ts(d, tmem_base + kColQ + 8 * ks, dk + (uint64_t)(((ks >> 2) * kSubTile >> 4) + 2 * (ks & 3)), idesc_s, ks != 0 ? 1u : 0u);
                if (comp) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        tc_mma_ts(d, tmem_base + kColQ + 64 + 8 * ks, dk + (uint64_t)(((ks >> 2) * kSubTile >> 4) + 2 * (ks & 3)), idesc_s, 1u);
                }
                if (lo) {
                    const uint64_t dl = desc_k_major(s_ring + st_lo[i & 3] * kStageBytes);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        tc_mma_ts(d, tmem_base + kColQ + 8 * ks, dl + (uint64_t)(((ks >> 2) * kSubTile >> 4) + 2 * (ks & 3)), idesc_s, 1u);
                }
                tc_commit(smem_u32(&ctl.s_full[b]));
                return true;
            };
            if (!mbar_wait(smem_u32(&ctl.q_full), 0, abort_flag, wait_limit)) failed = true;
            // Scores run two tiles ahead of the softmax: tile i goes into the buffer that the weights of
            // tile i - 2 have been computed from.
            for (int i = 0; i < T && !failed; ++i) {
                if (i >= 2 && !mbar_wait(smem_u32(&ctl.p_full[i & 1]), (uint32_t)((i - 2) >> 1) & 1u, abort_flag, wait_limit)) { failed = true; break; }
                if (!issue_s(i)) failed = true;
            }
        }
    } else if (warp == 6) {
        // ================================================= MMA issuer of O += P V
        // A second issuing thread: a run of MMAs into one accumulator holds its thread for the ~420 cycles
        // of pipeline latency on top of the MMAs themselves, and two threads keep two runs (scores of a
        // later tile, P V of this one) in flight at once (measured: 1460 cycles for both against 1870 in turn).
        if (lane == 0 && T > 0 && !refused()) {
            constexpr uint32_t idesc_o = make_idesc(128, kHd, true);
            int s = 0;                                    // walks the ring like the score issuer (it has waited for the copies)
            for (int i = 0; i < T && !failed; ++i) {
                const bool lo = comp && reaches_tree(t_begin + i);
                const int s_kv = s;
                if (++s == kStages) s = 0;
                int s_lo = -1;
                if (lo) {
                    s_lo = s;
                    if (++s == kStages) s = 0;
                }
                if (!mbar_wait(smem_u32(&ctl.p_full[i & 1]), (uint32_t)(i >> 1) & 1u, abort_flag, wait_limit)) { failed = true; break; }
                tc_fence_after();
                const int b = i & 1;
                const uint32_t d = tmem_base + kColO;
                // 16 keys further: 8 columns of P in tensor memory, 16 rows (2048 bytes) in V
                const uint32_t tp = tmem_base + kColP + 64 * (uint32_t)b;
                const uint64_t dv = desc_mn_major(s_ring + s_kv * kStageBytes + 2 * kSubTile, kSubTile);
                if (i > 0) {                              // the outputs accumulate in TMEM over the tiles
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) tc_mma_ts(d, tp + 8 * ks, dv + (uint64_t)(ks * 2048 >> 4), idesc_o, 1u);
                } else {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) tc_mma_ts(d, tp + 8 * ks, dv + (uint64_t)(ks * 2048 >> 4), idesc_o, ks != 0 ? 1u : 0u);
                }
                if (comp) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) tc_mma_ts(d, tp + 32 + 8 * ks, dv + (uint64_t)(ks * 2048 >> 4), idesc_o, 1u);
                }
                if (s_lo >= 0) {
                    const uint64_t dvl = desc_mn_major(s_ring + s_lo * kStageBytes + 2 * kSubTile, kSubTile);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) tc_mma_ts(d, tp + 8 * ks, dvl + (uint64_t)(ks * 2048 >> 4), idesc_o, 1u);
                }
                tc_commit(smem_u32(&ctl.o_full[b]));
                tc_commit(smem_u32(&ctl.empty[s_kv]));
                if (s_lo >= 0) tc_commit(smem_u32(&ctl.empty[s_lo]));
            }
        }
    } else if (warp < 6) {
        // ================================================= softmax (warps 2..5): thread = query row
        const int lg = warp & 3;                          // TMEM lanes 32*lg .. 32*lg + 31 belong to this warp
        const int row = lg * 32 + lane;
        const bool warp_active = lg * 32 < n;             // a warp whose rows are all padding only keeps the barriers going
        const uint32_t tlane = tmem_base + ((uint32_t)(lg * 32) << 16);
        dep_wait_warp(dep, lane);
        if (trace && tid == 64 && cta < 256) trace[(size_t)cta * 16 + 1] = global_timer_ns();
        // The loads below go out before the status word is looked at (they read buffers that exist whatever an
        // earlier phase found), so that its round trip overlaps theirs.
        uint32_t a4[4] = {0, 0, 0, 0};
        if (row < n) {
#pragma unroll
            for (int w = 0; w < 4; ++w) a4[w] = __ldcg(anc + (q_first + row) * 4 + w);   // L2: written earlier in this pass
        }
        uint4 g[2][16];
        if (warp_active) {
#pragma unroll
            for (int pl = 0; pl < 2; ++pl) {
                if (pl < (comp ? 2 : 1)) {
#pragma unroll
                    for (int it = 0; it < 16; ++it) {
                        const int rr = it * 2 + (lane >> 4);
                        const int qrow = min(lg * 32 + rr, n - 1);
                        g[pl][it] = __ldcg(reinterpret_cast<const uint4 *>(q + (size_t)pl * lo_off + ((size_t)qrow * n_heads + head) * kHd) + (lane & 15));
                    }
                }
            }
        }
        const bool skip = *reinterpret_cast<const volatile int32_t *>(status) != 0;
        if (!skip) {
        // The queries become the A operand of Q K^T in tensor memory: 64 packed columns per plane, thread =
        // row. A warp fetches its 32 rows with coalesced loads (two rows of 256 bytes per instruction, both
        // planes in flight together), turns them through a small shared-memory buffer (16-byte chunks
        // XOR-swizzled by row) and every thread stores its own row. Rows beyond n repeat row n - 1: a row
        // of A only ever influences the same row of the product, and nobody reads those rows of the result.
        if (warp_active) {
            const int planes = comp ? 2 : 1;
            const uint32_t stg = smem_u32(q_stage + (size_t)lg * kQStage);
#pragma unroll
            for (int pl = 0; pl < 2; ++pl) {
                if (pl < planes) {
#pragma unroll
                    for (int it = 0; it < 16; ++it) {
                        const int rr = it * 2 + (lane >> 4);
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(stg + rr * 256 + (((lane & 15) ^ (rr & 15)) << 4)),
                                     "r"(g[pl][it].x), "r"(g[pl][it].y), "r"(g[pl][it].z), "r"(g[pl][it].w) : "memory");
                    }
                    __syncwarp();
                    uint32_t qr[64];
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];"
                                     : "=r"(qr[4 * c]), "=r"(qr[4 * c + 1]), "=r"(qr[4 * c + 2]), "=r"(qr[4 * c + 3])
                                     : "r"(stg + lane * 256 + ((c ^ (lane & 15)) << 4)) : "memory");
                    }
                    __syncwarp();                         // the buffer is reused for the lo plane
                    tc_st32(tlane + kColQ + 64 * pl, qr);
                    tc_st32(tlane + kColQ + 64 * pl + 32, qr + 32);
                }
            }
            tc_wait_st();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&ctl.q_full));
        const float scale_log2 = 1.4426950408889634f * rsqrtf((float)kHd);
        // Online softmax with a lazy reference: the weights of a row are 2^(s - ref), and ref only moves
        // (with a rescale of the row's running sum and of its outputs in TMEM) when a tile's maximum
        // exceeds it by more than kSlack, so that the outputs can stay and accumulate in TMEM across the
        // tiles; weights then reach at most 2^kSlack, harmless in fp32 and in hi + lo bf16.
        constexpr float kSlack = 8.f;
        float ref = -INFINITY, l = 0.f;

        for (int i = 0; i < T; ++i) {
            const int t = t_begin + i, b = i & 1;
            const int key0 = t * kKeyTile;
            if (!mbar_wait_warp(smem_u32(&ctl.s_full[b]), (uint32_t)(i >> 1) & 1u, abort_flag, lane, wait_limit)) { failed = true; break; }
            tc_fence_after();
            if (trace && tid == 64 && cta < 256 && i == 0) trace[(size_t)cta * 16 + 2] = global_timer_ns();
            float sc[kKeyTile];
            if (warp_active) tc_ld64(tlane + (uint32_t)b * kKeyTile, sc);
            // Visibility of the tile's 64 keys for this row, one bit each: prefix keys always, tree keys by
            // the row's ancestor-or-self bits (bits of nodes that do not exist are never set).
            float tmax = -INFINITY;
            if (warp_active) {
                if (key0 + kKeyTile > P) {
                    const uint64_t alo = (uint64_t)a4[0] | ((uint64_t)a4[1] << 32), ahi = (uint64_t)a4[2] | ((uint64_t)a4[3] << 32);
                    const int sh = key0 - P;              // node index of the tile's first key
                    uint64_t vis;
                    if (sh >= 64) vis = ahi >> (sh - 64);
                    else if (sh > 0) vis = (alo >> sh) | (ahi << (64 - sh));
                    else if (sh == 0) vis = alo;
                    else vis = (alo << (-sh)) | ((1ull << (-sh)) - 1ull);
                    const uint32_t v0 = (uint32_t)vis, v1 = (uint32_t)(vis >> 32);
#pragma unroll
                    for (int j = 0; j < kKeyTile; ++j) {
                        const bool on = (((j < 32 ? v0 : v1) >> (j & 31)) & 1u) != 0;
                        sc[j] = on ? sc[j] : -INFINITY;
                    }
                }
#pragma unroll
                for (int j = 0; j < kKeyTile; ++j) tmax = fmaxf(tmax, sc[j]);
                tmax *= scale_log2;                       // scores stay raw; the scale goes into the exponent below
            }
            // P buffer b was last read by the P V of tile i - 2
            if (i > 1) {
                if (!mbar_wait_warp(smem_u32(&ctl.o_full[b]), (uint32_t)((i - 2) >> 1) & 1u, abort_flag, lane, wait_limit)) { failed = true; break; }
            }
            if (warp_active) {
                const bool move = tmax > ref + kSlack || (ref == -INFINITY && tmax > -INFINITY);
                if (__any_sync(0xffffffffu, move)) {
                    // the outputs in TMEM are about to be rescaled: the P V of tile i - 1 must have retired
                    if (i > 0 && !mbar_wait_warp(smem_u32(&ctl.o_full[b ^ 1]), (uint32_t)((i - 1) >> 1) & 1u, abort_flag, lane, wait_limit)) { failed = true; break; }
                    tc_fence_after();
                    const float factor = !move ? 1.f : (ref == -INFINITY ? 0.f : ex2(ref - tmax));
                    if (move) ref = tmax;
                    l *= factor;
                    if (i > 0) {
#pragma unroll
                        for (int hcol = 0; hcol < 2; ++hcol) {
                            float ov[64];
                            tc_ld64(tlane + kColO + hcol * 64, ov);
#pragma unroll
                            for (int j = 0; j < 64; ++j) ov[j] *= factor;
                            tc_st64(tlane + kColO + hcol * 64, ov);
                        }
                    }
                }
                const float nr0 = (ref == -INFINITY) ? 0.f : -ref;   // no visible key so far: every weight is 0 anyway
                float rs = 0.f;
                uint32_t hi[32], lo[32];                  // packed pairs of consecutive keys: the A operand of P V
#pragma unroll
                for (int e = 0; e < kKeyTile / 2; ++e) {
                    const float p0 = ex2(fmaf(sc[2 * e], scale_log2, nr0));
                    const float p1 = ex2(fmaf(sc[2 * e + 1], scale_log2, nr0));
                    rs += p0 + p1;
                    pack_split(p0, p1, hi[e], lo[e]);
                }
                tc_st32(tlane + kColP + 64 * (uint32_t)b, hi);
                if (comp) tc_st32(tlane + kColP + 64 * (uint32_t)b + 32, lo);
                tc_wait_st();
                l += rs;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl.p_full[b]));
        }
        // the last two tiles' P V
        for (int i = max(0, T - 2); i < T && !failed; ++i)
            if (!mbar_wait_warp(smem_u32(&ctl.o_full[i & 1]), (uint32_t)(i >> 1) & 1u, abort_flag, lane, wait_limit)) failed = true;
        tc_fence_after();
        if (trace && tid == 64 && cta < 256) trace[(size_t)cta * 16 + 3] = global_timer_ns();
        // every copy has landed and every MMA has retired (the last o_full): the ring is free for the
        // partial of this CTA: per row 128 outputs, reference, sum
        if (!failed && warp_active) {
            float *pr = part + (size_t)row * kWsRow;
#pragma unroll
            for (int hcol = 0; hcol < 2; ++hcol) {
                float ov[64];
                if (T > 0) {
                    tc_ld64(tlane + kColO + hcol * 64, ov);
                } else {
#pragma unroll
                    for (int j = 0; j < 64; ++j) ov[j] = 0.f;
                }
                if (row < n) {
#pragma unroll
                    for (int j = 0; j < 64; j += 4)
                        *reinterpret_cast<float4 *>(pr + hcol * 64 + j) = make_float4(ov[j], ov[j + 1], ov[j + 2], ov[j + 3]);
                }
            }
            if (row < n) *reinterpret_cast<float2 *>(pr + kHd) = make_float2(ref, l);
        }
        }
        tc_fence_before();
    }
    if (failed) {
        ctl.abort_flag = 1;
        atomicCAS(status, 0, LLMCAD_ERR_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
    // (the softmax warps have passed the grid dependency, so the status word is final for every thread)
    const bool bad = ctl.abort_flag != 0 || *reinterpret_cast<const volatile int32_t *>(status) != 0;

    // four outputs of one row, normalised, as bf16 hi (and lo) to global memory
    auto store4 = [&](int row, int dim, float4 a, float inv) {
        uint32_t h0, l0, h1, l1;
        pack_split(a.x * inv, a.y * inv, h0, l0);
        pack_split(a.z * inv, a.w * inv, h1, l1);
        __nv_bfloat16 *dst = o + ((size_t)row * n_heads + head) * kHd + dim;
        *reinterpret_cast<uint2 *>(dst) = make_uint2(h0, h1);
        if (comp) *reinterpret_cast<uint2 *>(dst + lo_off) = make_uint2(l0, l1);
    };
    if (splits == 1) {
        if (!bad) {
            for (int idx = tid; idx < n * (kHd / 4); idx += kT5Threads) {
                const int row = idx / (kHd / 4), dim = (idx % (kHd / 4)) * 4;
                const float L = part[(size_t)row * kWsRow + kHd + 1];
                store4(row, dim, *reinterpret_cast<const float4 *>(part + (size_t)row * kWsRow + dim), L > 0.f ? 1.f / L : 0.f);
            }
        }
        if (done_ctr != nullptr) {
            __syncthreads();
            if (tid == 0) dep_arrive(done_ctr);
        }
        if (trace && tid == 0 && cta < 256) trace[(size_t)cta * 16 + 12] = global_timer_ns();
        return;
    }

    if (trace && tid == 0 && cta < 256) trace[(size_t)cta * 16 + 4] = global_timer_ns();
    cg::cluster_group cluster = cg::this_cluster();
    cluster.sync();                                          // all partials of this head are written
    if (trace && tid == 0 && cta < 256) trace[(size_t)cta * 16 + 5] = global_timer_ns();
    if (!bad) {
        if (splits <= 2) merge_splits<2, 4>(part, cluster, splits, split, n, n_heads, head, o, lo_off, comp, tid);
        else if (splits <= 4) merge_splits<4, 2>(part, cluster, splits, split, n, n_heads, head, o, lo_off, comp, tid);
        else merge_splits<kMaxSplits, 1>(part, cluster, splits, split, n, n_heads, head, o, lo_off, comp, tid);
    }
    if (trace && tid == 0 && cta < 256) trace[(size_t)cta * 16 + 6] = global_timer_ns();
    if (done_ctr != nullptr) {
        __syncthreads();                                     // this CTA's rows of the output are written
        if (tid == 0) dep_arrive(done_ctr);
    }
    cluster.sync();                                          // peers may still be reading this CTA's partial
    if (trace && tid == 0 && cta < 256) trace[(size_t)cta * 16 + 12] = global_timer_ns();
}

bool attention_prefers_t5(int n)
{
    static const int min_n = [] { const char *e = getenv("LLMCAD_ATTN_T5_MIN_N"); return e ? atoi(e) : 33; }();
    return min_n > 0 && n >= min_n;
}

cudaError_t launch_attention_t5(const void *q, const void *k, const void *v, int n_heads, int hd, int kv_stride, int P,
                                int n, const uint32_t *anc, void *o, int n_sms, int32_t *status, cudaStream_t st,
                                int *launched, unsigned long long *trace, int comp, const void *kv_lo, int n_tree, int q_first, uint64_t wait_limit_ns,
                                const AttnSync *sync)
{
    if (n_tree <= 0) n_tree = n;
    if (hd != kHd || n < 1 || n > 128 || P + n_tree > kv_stride) return cudaErrorInvalidValue;
    if (comp && kv_lo == nullptr) return cudaErrorInvalidValue;
    const int n_keys = P + n_tree;
    const int n_tiles = (n_keys + kKeyTile - 1) / kKeyTile;
    int splits = n_sms / n_heads;
    if (splits > kMaxSplits) splits = kMaxSplits;
    if (splits > n_tiles) splits = n_tiles;
    if (splits < 1) splits = 1;
    const int tiles_per_split = (n_tiles + splits - 1) / splits;
    splits = (n_tiles + tiles_per_split - 1) / tiles_per_split;      // no split without a tile

    CUtensorMap mk, mv, ml;
    {
        const uint64_t dims[3] = {(uint64_t)kHd, (uint64_t)n_keys, (uint64_t)n_heads};
        const uint64_t strides[2] = {(uint64_t)kHd * 2, (uint64_t)kv_stride * kHd * 2};
        const uint32_t box[3] = {64, 64, 1};
        if (!make_tensor_map_bf16_3d(&mk, k, dims, strides, box)) return cudaErrorInvalidValue;
        if (!make_tensor_map_bf16_3d(&mv, v, dims, strides, box)) return cudaErrorInvalidValue;
    }
    if (comp) {
        const uint64_t dims[3] = {(uint64_t)kHd, (uint64_t)n, (uint64_t)2 * n_heads};
        const uint64_t strides[2] = {(uint64_t)kHd * 2, (uint64_t)kLoRows * kHd * 2};
        const uint32_t box[3] = {64, 64, 1};
        if (!make_tensor_map_bf16_3d(&ml, kv_lo, dims, strides, box)) return cudaErrorInvalidValue;
    } else {
        ml = mk;      // never dereferenced without compensation
    }
    static PerDeviceOnce attr_set;
    if (attr_set.needed()) {
        cudaError_t e = cudaFuncSetAttribute(attention_t5_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(attention_t5_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        if (e != cudaSuccess) return e;
        attr_set.mark();
    }
    LaunchCfg lc(dim3(splits, n_heads), dim3(kT5Threads), kSmemBytes, st, splits);
    if (launched) *launched = 1;
    DepWait dep{nullptr, 0, wait_limit_ns};
    uint32_t *done = nullptr;
    if (sync != nullptr) {
        dep = DepWait{sync->dep_ctr, sync->dep_target, wait_limit_ns};
        done = sync->done_ctr;
        sync->arrivals = (uint32_t)(splits * n_heads);
    }
    return cudaLaunchKernelEx(&lc.cfg, attention_t5_kernel, (const __nv_bfloat16 *)q, mk, mv, ml, n_heads, P, n, anc, (__nv_bfloat16 *)o, splits,
                              tiles_per_split, status, trace, comp, n_tree, q_first, wait_limit_ns, dep, done);
}

}  // namespace llmcad
