// Tree-masked attention on tensor cores (bf16, head_dim 128).
//
// Per head the keys are the prefix slots 0..P-1 (visible to every node) followed by the tree
// nodes at slots P..P+n-1, of which node i sees the ones whose bit is set in its ancestor-or-self
// row (the mask table of Sec. 3.2 "Tree decoder"). The prefix K/V bytes dominate, and a layer has
// few heads, so the key range of each head is split over the CTAs of one thread-block cluster
// (grid = splits x heads, cluster = the splits of a head, about one CTA per SM in total): each
// CTA streams its key range once through a four-stage cp.async ring in shared memory, keeps an
// online softmax per query row and ends with an unnormalised partial (max, sum, output) per row.
// The splits of a head are merged through distributed shared memory: query row r belongs to CTA
// r % splits of the cluster. With few nodes (<= 32, the common tree) every CTA pushes its partial
// rows into a receive buffer in the owner's shared memory (remote stores are posted, remote loads
// pay a round trip each), one cluster barrier follows, and the owner merges what it received and
// writes the bf16 output; larger trees, whose receive buffers would not fit beside the key ring,
// keep their partial at home and the owners fetch the rows after the barrier. No global
// workspace, no atomics.
//
// Inside a CTA warp w owns query rows 16w..16w+15 (n <= 128 nodes -> at most 8 warps busy);
// QK^T and PV are mma.sync m16n8k16 bf16 with fp32 accumulation, scores never leave registers.
#include <cooperative_groups.h>

#include "attention_tc.cuh"

namespace cg = cooperative_groups;

namespace llmcad {

namespace {

constexpr int kHd = 128;
constexpr int kKeyTile = 64;
constexpr int kAtThreads = 256;
constexpr int kRowBytes = kHd * 2;            // 256-byte rows = 16 chunks of 16 bytes
// partial row: 128 outputs, max, sum, padding. 136 floats: rows start on 16 bytes, and the eight rows a
// warp stores at once (fragment layout: lane / 4 = row) start in banks 8 apart, so that its 8-byte stores
// do not collide (with 130 floats they did, four ways, and the stores took longer than the merge itself).
constexpr int kWsRow = kHd + 8;
constexpr int kMaxSplits = 8;                 // portable cluster size
constexpr int kMaxStages = 4;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// 16-byte chunk c of row r lives at chunk c ^ (r & 7): ldmatrix reads of 8 consecutive rows at one
// logical chunk then touch 8 different bank groups.
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return (uint32_t)(row * kRowBytes + ((chunk ^ (row & 7)) << 4)); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid)
{
    const int sz = valid ? 16 : 0;  // size 0: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4_t(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
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

}  // namespace

// GROUPS key groups per CTA: warp w works on query tile w % q_tiles and on the keys
// [g * 64/GROUPS, (g+1) * 64/GROUPS) of every 64-key tile, g = w / q_tiles. With few tree nodes
// (n <= 32: two query tiles) a single warp per query tile would leave most of the SM idle and its
// dependent mma chain would set the pace; splitting the keys of a tile over four warps cuts the
// per-tile latency four-fold. Each warp keeps its own running softmax; the groups are merged in
// shared memory at the end, then the cluster merges the splits.
//
// COMP (the verification pass): queries arrive as bf16 hi + lo planes and the output leaves as hi +
// lo planes (kLoRows rows apart, see common.cuh), and the softmax weights are split into hi + lo as
// well, so that Q K^T and P V each take two MMAs per fragment. The keys and values of the tree nodes
// themselves, which the QKV GEMM has just rounded into the cache, come with their remainders in a
// side buffer kv_lo ([2][H][kLoRows][128]: K then V, indexed by node); the tiles that contain tree
// keys add Q K_lo^T and P V_lo. Only the prefix K/V, which are bf16 by definition, stay as they are.
template <int GROUPS, bool COMP>
__global__ void __launch_bounds__(kAtThreads)
attention_tc_kernel(const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k,
                    const __nv_bfloat16 *__restrict__ v, int n_heads, int kv_stride, int P, int n, int n_pad,
                    const uint32_t *__restrict__ anc, __nv_bfloat16 *o, int splits, int tiles_base, int tiles_rem,
                    const int32_t *status, unsigned long long *trace, const __nv_bfloat16 *__restrict__ kv_lo,
                    int n_tree, int q_first, DepWait dep, uint32_t *done_ctr, int recv_off)
{
    // PUSH: partial rows travel to their owners (see the head of the file); recv_off = where the receive
    // buffer starts in this CTA's shared memory, [splits][rows per CTA][kWsRow] floats behind everything else
    constexpr bool PUSH = GROUPS == 4;
    // n query rows = the tree nodes q_first .. q_first + n - 1 (all of them in a verification pass,
    // the new ones when a tree is extended); the keys are the prefix and all n_tree tree nodes
    // ring depth: with 128 nodes and the lo planes three stages are what fits in shared memory
    constexpr int kStages = (COMP && GROUPS == 1) ? 3 : kMaxStages;
    constexpr int KW = kKeyTile / GROUPS;     // keys per warp per tile: 64, 32 or 16
    constexpr int NT = KW / 8;                // 8-key score tiles per warp per tile
    const int cta = blockIdx.y * gridDim.x + blockIdx.x;
    if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 0] = global_timer_ns();
    pdl_launch_dependents();
    // first cluster barrier, arrival: its completion tells that every CTA of the cluster is running, which a
    // store into a peer's shared memory requires; waited for just before the first such store
    if (PUSH) asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
    extern __shared__ __align__(128) uint8_t sm[];
    uint8_t *s_q = sm;                                      // [n_pad][256 B], with COMP followed by the lo plane
    uint8_t *s_k = s_q + (size_t)(COMP ? 2 : 1) * n_pad * kRowBytes;   // [kStages][64][256 B]
    uint8_t *s_v = s_k + kStages * kKeyTile * kRowBytes;    // [kStages][64][256 B]
    // COMP: remainders of the tree nodes' K and V, [n_pad + 1][256 B] each, row = node; the extra row is zero
    uint8_t *s_kl = s_v + kStages * kKeyTile * kRowBytes;
    uint8_t *s_vl = s_kl + (size_t)(n_pad + 1) * kRowBytes;

    const size_t lo_off = (size_t)kLoRows * n_heads * kHd;  // elements from a hi plane of q / o to its lo plane
    const int split = blockIdx.x, head = blockIdx.y;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_keys = P + n_tree;
    const int n_tiles = (n_keys + kKeyTile - 1) / kKeyTile;
    // the first tiles_rem splits walk one tile more than the others: the tiles with the tree nodes, which cost
    // more (remainders, mask) and cannot be requested before the grid dependency, fall to a short split
    const int t_begin = split * tiles_base + min(split, tiles_rem);
    const int t_end = min(n_tiles, t_begin + tiles_base + (split < tiles_rem ? 1 : 0));
    const __nv_bfloat16 *kh = k + (size_t)head * kv_stride * kHd;
    const __nv_bfloat16 *vh = v + (size_t)head * kv_stride * kHd;

    auto load_tile = [&](int t, int buf) {
        const int key0 = t * kKeyTile;
        uint8_t *dk = s_k + (size_t)buf * kKeyTile * kRowBytes, *dv = s_v + (size_t)buf * kKeyTile * kRowBytes;
        for (int c = tid; c < kKeyTile * 16; c += kAtThreads) {
            const int r = c >> 4, ch = c & 15;
            const int key = key0 + r;
            const bool ok = key < n_keys;
            const size_t off = (size_t)(ok ? key : 0) * kHd + ch * 8;
            cp_async16(smem_u32(dk) + swz(r, ch), kh + off, ok);
            cp_async16(smem_u32(dv) + swz(r, ch), vh + off, ok);
        }
    };

    // The prefix keys and values were written by earlier passes: the first tiles that lie wholly in
    // the prefix are requested before the grid dependency, while the QKV GEMM of this layer is still
    // finishing; the queries, the tree nodes' K/V and the status word wait for it.
    bool early[kStages - 1];
#pragma unroll
    for (int st = 0; st < kStages - 1; ++st) {
        early[st] = t_begin + st < t_end && (t_begin + st + 1) * kKeyTile <= P;
        if (early[st]) load_tile(t_begin + st, st);
    }
    // the queries and the tree nodes' K/V are final: grid dependency, or the producer's completion counter
    if (dep.ctr == nullptr) pdl_wait();
    else {
        if (threadIdx.x == 0) dep_wait_thread(dep);      // a wait that runs out lets the pass go on: the status word tells
        __syncthreads();
    }
    if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 1] = global_timer_ns();
    // queries of this head (rows >= n are zero) and the remaining first key tiles
    for (int c = tid; c < n_pad * 16; c += kAtThreads) {
        const int r = c >> 4, ch = c & 15;
        const bool ok = r < n;
        const size_t off = ((size_t)(ok ? r : 0) * n_heads + head) * kHd + ch * 8;
        cp_async16(smem_u32(s_q) + swz(r, ch), q + off, ok);
        if (COMP) cp_async16(smem_u32(s_q) + n_pad * kRowBytes + swz(r, ch), q + lo_off + off, ok);
    }
    if (COMP && t_end * kKeyTile > P) {         // this CTA's key range reaches the tree nodes
        const __nv_bfloat16 *kl = kv_lo + (size_t)head * kLoRows * kHd;
        const __nv_bfloat16 *vl = kl + (size_t)n_heads * kLoRows * kHd;
        for (int c = tid; c < (n_pad + 1) * 16; c += kAtThreads) {
            const int r = c >> 4, ch = c & 15;
            const bool ok = r < n;
            const size_t off = (size_t)(ok ? r : 0) * kHd + ch * 8;
            cp_async16(smem_u32(s_kl) + swz(r, ch), kl + off, ok);
            cp_async16(smem_u32(s_vl) + swz(r, ch), vl + off, ok);
        }
    }
#pragma unroll
    for (int st = 0; st < kStages - 1; ++st) {
        if (t_begin + st < t_end && !early[st]) load_tile(t_begin + st, st);
        cp_commit();                            // group 0 also carries the queries and everything requested early
    }
    // The status word is looked at only now, with the copies above already on their way (they read buffers that
    // exist whatever an earlier phase found): a refused pass waits for them and leaves.
    if (*reinterpret_cast<const volatile int32_t *>(status)) {   // uniform over the grid: set only by kernels that ran before this one
        cp_wait<0>();          // nothing may still be writing this CTA's shared memory when it exits
        if (threadIdx.x == 0) dep_arrive(done_ctr);
        return;
    }

    const int q_tiles = n_pad >> 4;
    const int qt = warp % q_tiles, kg = warp / q_tiles;
    const bool active = kg < GROUPS;
    const int row0 = qt * 16 + (lane >> 2), row1 = row0 + 8;   // the two query rows this thread holds
    uint32_t anc0[4] = {0, 0, 0, 0}, anc1[4] = {0, 0, 0, 0};
    if (active) {
        for (int w = 0; w < 4; ++w) {
            if (row0 < n) anc0[w] = __ldcg(anc + (q_first + row0) * 4 + w);     // L2: written earlier in this pass
            if (row1 < n) anc1[w] = __ldcg(anc + (q_first + row1) * 4 + w);
        }
    }

    const float scale_log2 = 1.4426950408889634f * rsqrtf((float)kHd);
    uint32_t qf[8][4];
    float oacc[16][4];
#pragma unroll
    for (int j = 0; j < 16; ++j) oacc[j][0] = oacc[j][1] = oacc[j][2] = oacc[j][3] = 0.f;
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    for (int t = t_begin; t < t_end; ++t) {
        const int buf = (t - t_begin) % kStages;
        cp_wait<kStages - 2>();
        __syncthreads();                       // tile t (and Q) visible; everyone is done with tile t-1's buffer
        if (trace && threadIdx.x == 0 && cta < 256 && t == t_begin) trace[(size_t)cta * 16 + 2] = global_timer_ns();
        if (t + kStages - 1 < t_end) load_tile(t + kStages - 1, (t + kStages - 1 - t_begin) % kStages);
        cp_commit();
        if (t == t_begin && active) {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                ldsm4(smem_u32(s_q) + swz(qt * 16 + (lane & 15), ks * 2 + (lane >> 4)), qf[ks]);
        }
        if (!active) continue;
        const uint32_t kb = smem_u32(s_k) + buf * kKeyTile * kRowBytes;
        const uint32_t vb = smem_u32(s_v) + buf * kKeyTile * kRowBytes;
        const int key_off = kg * KW;           // this warp's keys inside the tile

        // ---- S = Q K^T for this warp's KW keys: NT score tiles of 8 keys
        float s[NT][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t ql[4];
            if (COMP) ldsm4(smem_u32(s_q) + n_pad * kRowBytes + swz(qt * 16 + (lane & 15), ks * 2 + (lane >> 4)), ql);
#pragma unroll
            for (int np = 0; np < NT / 2; ++np) {
                uint32_t b[4];
                const int key = key_off + np * 16 + (lane & 7) + ((lane >> 4) << 3);
                ldsm4(kb + swz(key, ks * 2 + ((lane >> 3) & 1)), b);
                mma_bf16(s[2 * np], qf[ks], b[0], b[1]);
                mma_bf16(s[2 * np + 1], qf[ks], b[2], b[3]);
                if (COMP) {
                    mma_bf16(s[2 * np], ql, b[0], b[1]);
                    mma_bf16(s[2 * np + 1], ql, b[2], b[3]);
                }
            }
        }
        const int key_base = t * kKeyTile + key_off;
        const bool needs_mask = key_base + KW > P;          // this warp's keys reach into the tree nodes
        // row of the lo buffers that holds the remainder of key `key` (the zero row for prefix keys)
        auto lo_row = [&](int key) { const int node = key - P - q_first; return (node >= 0 && node < n) ? node : n_pad; };
        if (COMP && needs_mask) {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
                for (int np = 0; np < NT / 2; ++np) {
                    uint32_t b[4];
                    const int row = lo_row(key_base + np * 16 + (lane & 7) + ((lane >> 4) << 3));
                    ldsm4(smem_u32(s_kl) + swz(row, ks * 2 + ((lane >> 3) & 1)), b);
                    mma_bf16(s[2 * np], qf[ks], b[0], b[1]);
                    mma_bf16(s[2 * np + 1], qf[ks], b[2], b[3]);
                }
            }
        }
        // ---- scale, mask (tree region and the ragged end only), online softmax
        float tmax0 = -INFINITY, tmax1 = -INFINITY;
#pragma unroll
        for (int j = 0; j < NT; ++j) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float val = s[j][e] * scale_log2;
                if (needs_mask) {
                    const int key = key_base + j * 8 + ((lane & 3) << 1) + (e & 1);
                    if (key >= P) {
                        const int node = key - P;
                        const uint32_t *a = (e < 2) ? anc0 : anc1;
                        const bool vis = node < n_tree && ((a[node >> 5] >> (node & 31)) & 1u);
                        if (!vis) val = -INFINITY;
                    }
                }
                s[j][e] = val;
                if (e < 2) tmax0 = fmaxf(tmax0, val); else tmax1 = fmaxf(tmax1, val);
            }
        }
        tmax0 = fmaxf(tmax0, __shfl_xor_sync(0xffffffffu, tmax0, 1));
        tmax0 = fmaxf(tmax0, __shfl_xor_sync(0xffffffffu, tmax0, 2));
        tmax1 = fmaxf(tmax1, __shfl_xor_sync(0xffffffffu, tmax1, 1));
        tmax1 = fmaxf(tmax1, __shfl_xor_sync(0xffffffffu, tmax1, 2));
        const float mn0 = fmaxf(m0, tmax0), mn1 = fmaxf(m1, tmax1);
        // a row that has seen no visible key yet keeps max = -inf: use 0 as the reference to avoid inf - inf
        const float ref0 = (mn0 == -INFINITY) ? 0.f : mn0, ref1 = (mn1 == -INFINITY) ? 0.f : mn1;
        const float alpha0 = exp2f(m0 - ref0), alpha1 = exp2f(m1 - ref1);
        m0 = mn0; m1 = mn1;
        float rs0 = 0.f, rs1 = 0.f;
        uint32_t pa[NT / 2][4], pl[COMP ? NT / 2 : 1][4];
#pragma unroll
        for (int j = 0; j < NT; ++j) {
            const float p0 = exp2f(s[j][0] - ref0), p1 = exp2f(s[j][1] - ref0);
            const float p2 = exp2f(s[j][2] - ref1), p3 = exp2f(s[j][3] - ref1);
            rs0 += p0 + p1; rs1 += p2 + p3;
            if (COMP) {
                pack_split(p0, p1, pa[j >> 1][(j & 1) * 2 + 0], pl[COMP ? j >> 1 : 0][(j & 1) * 2 + 0]);
                pack_split(p2, p3, pa[j >> 1][(j & 1) * 2 + 1], pl[COMP ? j >> 1 : 0][(j & 1) * 2 + 1]);
            } else {
                pa[j >> 1][(j & 1) * 2 + 0] = pack_bf16(p0, p1);
                pa[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
            }
        }
        l0 = l0 * alpha0 + rs0; l1 = l1 * alpha1 + rs1;
#pragma unroll
        for (int j = 0; j < 16; ++j) { oacc[j][0] *= alpha0; oacc[j][1] *= alpha0; oacc[j][2] *= alpha1; oacc[j][3] *= alpha1; }
        // ---- O += P V: k = KW keys (steps of 16), n = 128 dims (8 pairs of n-tiles)
#pragma unroll
        for (int kk = 0; kk < NT / 2; ++kk) {
#pragma unroll
            for (int dp = 0; dp < 8; ++dp) {
                uint32_t b[4];
                const int key = key_off + kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                ldsm4_t(vb + swz(key, dp * 2 + (lane >> 4)), b);
                mma_bf16(oacc[2 * dp], pa[kk], b[0], b[1]);
                mma_bf16(oacc[2 * dp + 1], pa[kk], b[2], b[3]);
                if (COMP) {
                    mma_bf16(oacc[2 * dp], pl[COMP ? kk : 0], b[0], b[1]);
                    mma_bf16(oacc[2 * dp + 1], pl[COMP ? kk : 0], b[2], b[3]);
                }
            }
        }
        if (COMP && needs_mask) {
#pragma unroll
            for (int kk = 0; kk < NT / 2; ++kk) {
#pragma unroll
                for (int dp = 0; dp < 8; ++dp) {
                    uint32_t b[4];
                    const int row = lo_row(key_base + kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3));
                    ldsm4_t(smem_u32(s_vl) + swz(row, dp * 2 + (lane >> 4)), b);
                    mma_bf16(oacc[2 * dp], pa[kk], b[0], b[1]);
                    mma_bf16(oacc[2 * dp + 1], pa[kk], b[2], b[3]);
                }
            }
        }
    }
    cp_wait<0>();
    if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 3] = global_timer_ns();

    // ---- row sums over the four threads of a row
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    // ---- every warp leaves its unnormalised partial (outputs, max, sum) in shared memory (the
    // K/V ring is done): wpart[kg][row][kWsRow]
    __syncthreads();
    float *wpart = reinterpret_cast<float *>(sm);
    if (active) {
        float *wp = wpart + (size_t)kg * n_pad * kWsRow;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const int dim = j * 8 + ((lane & 3) << 1);
            *reinterpret_cast<float2 *>(wp + (size_t)row0 * kWsRow + dim) = make_float2(oacc[j][0], oacc[j][1]);
            *reinterpret_cast<float2 *>(wp + (size_t)row1 * kWsRow + dim) = make_float2(oacc[j][2], oacc[j][3]);
        }
        if ((lane & 3) == 0) {
            *reinterpret_cast<float2 *>(wp + (size_t)row0 * kWsRow + kHd) = make_float2(m0, l0);
            *reinterpret_cast<float2 *>(wp + (size_t)row1 * kWsRow + kHd) = make_float2(m1, l1);
        }
    }
    __syncthreads();
    // The CTA's partial of four outputs of a row, merged over its key groups in group order:
    // out = sum_g O_g 2^(m_g - M), l = sum_g l_g 2^(m_g - M), M = max_g m_g.
    auto merged4 = [&](int row, int dim, float2 &ML) {
        float mg[GROUPS], M = -INFINITY, L = 0.f;
#pragma unroll
        for (int g = 0; g < GROUPS; ++g) { mg[g] = wpart[((size_t)g * n_pad + row) * kWsRow + kHd]; M = fmaxf(M, mg[g]); }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int g = 0; g < GROUPS; ++g) {
            const float w = (mg[g] == -INFINITY) ? 0.f : exp2f(mg[g] - M);
            const float4 vv = *reinterpret_cast<const float4 *>(wpart + ((size_t)g * n_pad + row) * kWsRow + dim);
            L += wpart[((size_t)g * n_pad + row) * kWsRow + kHd + 1] * w;
            acc.x += vv.x * w; acc.y += vv.y * w; acc.z += vv.z * w; acc.w += vv.w * w;
        }
        ML = make_float2(M, L);
        return acc;
    };
    // four outputs of one row, normalised, as bf16 hi (and lo) to global memory
    auto store4 = [&](int row, int dim, float4 acc, float inv) {
        uint32_t h0, l0w, h1, l1w;
        pack_split(acc.x * inv, acc.y * inv, h0, l0w);
        pack_split(acc.z * inv, acc.w * inv, h1, l1w);
        __nv_bfloat16 *dst = o + ((size_t)row * n_heads + head) * kHd + dim;
        *reinterpret_cast<uint2 *>(dst) = make_uint2(h0, h1);
        if (COMP) *reinterpret_cast<uint2 *>(dst + lo_off) = make_uint2(l0w, l1w);
    };

    if (splits == 1) {
        for (int idx = tid; idx < n * (kHd / 4); idx += kAtThreads) {
            const int row = idx / (kHd / 4), dim = (idx % (kHd / 4)) * 4;
            float2 ML;
            const float4 acc = merged4(row, dim, ML);
            store4(row, dim, acc, ML.y > 0.f ? 1.f / ML.y : 0.f);
        }
        if (done_ctr != nullptr) {
            __syncthreads();
            if (threadIdx.x == 0) dep_arrive(done_ctr);
        }
        if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 12] = global_timer_ns();
        return;
    }

    cg::cluster_group cluster = cg::this_cluster();
    if (PUSH) {
        // ---- rows to their owners: row r -> CTA r % splits, slot [this split][r / splits] of its receive buffer
        float *recv = reinterpret_cast<float *>(sm + recv_off);
        const int rows_cap = (n_pad + splits - 1) / splits;
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");     // every CTA of the cluster is running
        for (int idx = tid; idx < n * (kHd / 4); idx += kAtThreads) {
            const int row = idx / (kHd / 4), dim = (idx % (kHd / 4)) * 4;
            float2 ML;
            const float4 acc = merged4(row, dim, ML);
            float *dst = cluster.map_shared_rank(recv, row % splits) + ((size_t)split * rows_cap + row / splits) * kWsRow;
            *reinterpret_cast<float4 *>(dst + dim) = acc;
            if (dim == 0) *reinterpret_cast<float2 *>(dst + kHd) = ML;
        }
        if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 4] = global_timer_ns();
        // second cluster barrier: the stores above are released by the arrival and acquired by the wait
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
        asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
        if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 5] = global_timer_ns();
        // ---- merge over the splits, in split order: out = sum_s O_s 2^(m_s - M) / sum_s l_s 2^(m_s - M)
        const int my_rows = (n - split + splits - 1) / splits;   // rows split, split + splits, ... below n
        for (int idx = tid; idx < my_rows * (kHd / 4); idx += kAtThreads) {
            const int lr = idx / (kHd / 4), dim = (idx % (kHd / 4)) * 4;
            float ms[kMaxSplits], M = -INFINITY, L = 0.f;
#pragma unroll
            for (int sp = 0; sp < kMaxSplits; ++sp) {
                ms[sp] = sp < splits ? recv[((size_t)sp * rows_cap + lr) * kWsRow + kHd] : -INFINITY;
                M = fmaxf(M, ms[sp]);
            }
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int sp = 0; sp < kMaxSplits; ++sp) {
                if (sp < splits) {
                    const float *src = recv + ((size_t)sp * rows_cap + lr) * kWsRow;
                    const float w = (ms[sp] == -INFINITY) ? 0.f : exp2f(ms[sp] - M);
                    const float4 vv = *reinterpret_cast<const float4 *>(src + dim);
                    L += src[kHd + 1] * w;
                    acc.x += vv.x * w; acc.y += vv.y * w; acc.z += vv.z * w; acc.w += vv.w * w;
                }
            }
            store4(split + lr * splits, dim, acc, L > 0.f ? 1.f / L : 0.f);
        }
        if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 6] = global_timer_ns();
        if (done_ctr != nullptr) {
            __syncthreads();                                     // this CTA's rows of the output are written
            if (threadIdx.x == 0) dep_arrive(done_ctr);
        }
        // (nobody reads this CTA's shared memory from outside, and what peers stored into it arrived before the
        // barrier let go: the CTA may leave)
        if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 12] = global_timer_ns();
        return;
    }

    // ---- larger trees: the merged partial of the CTA stays at home, part[row][kWsRow]
    float *part = (GROUPS > 1) ? wpart + (size_t)GROUPS * n_pad * kWsRow : wpart;
    if (GROUPS > 1) {
        for (int idx = tid; idx < n_pad * (kHd / 4); idx += kAtThreads) {
            const int row = idx / (kHd / 4), dim = (idx % (kHd / 4)) * 4;
            float2 ML;
            const float4 acc = merged4(row, dim, ML);
            *reinterpret_cast<float4 *>(part + (size_t)row * kWsRow + dim) = acc;
            if (dim == 0) *reinterpret_cast<float2 *>(part + (size_t)row * kWsRow + kHd) = ML;
        }
    }
    if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 4] = global_timer_ns();
    cluster.sync();                                          // all partials of this head are written
    if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 5] = global_timer_ns();
    // ---- merge rows split, split + splits, ...: out = sum_s O_s 2^(m_s - M) / sum_s l_s 2^(m_s - M)
    const float *peer[kMaxSplits];
#pragma unroll
    for (int sp = 0; sp < kMaxSplits; ++sp) peer[sp] = sp < splits ? cluster.map_shared_rank(part, sp) : part;
    const int my_rows = (n - split + splits - 1) / splits;   // rows split, split+splits, ... below n
    for (int idx = tid; idx < my_rows * (kHd / 4); idx += kAtThreads) {
        const int row = split + (idx / (kHd / 4)) * splits, dim = (idx % (kHd / 4)) * 4;
        float2 ml[kMaxSplits];
        float4 ov[kMaxSplits];
#pragma unroll
        for (int sp = 0; sp < kMaxSplits; ++sp) {
            if (sp < splits) {
                ml[sp] = *reinterpret_cast<const float2 *>(peer[sp] + (size_t)row * kWsRow + kHd);
                ov[sp] = *reinterpret_cast<const float4 *>(peer[sp] + (size_t)row * kWsRow + dim);
            } else {
                ml[sp] = make_float2(-INFINITY, 0.f);
                ov[sp] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        float M = -INFINITY;
#pragma unroll
        for (int sp = 0; sp < kMaxSplits; ++sp) M = fmaxf(M, ml[sp].x);
        float L = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int sp = 0; sp < kMaxSplits; ++sp) {
            const float w = (ml[sp].x == -INFINITY) ? 0.f : exp2f(ml[sp].x - M);
            L += ml[sp].y * w;
            acc.x += ov[sp].x * w; acc.y += ov[sp].y * w; acc.z += ov[sp].z * w; acc.w += ov[sp].w * w;
        }
        store4(row, dim, acc, L > 0.f ? 1.f / L : 0.f);
    }
    if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 6] = global_timer_ns();
    if (done_ctr != nullptr) {
        __syncthreads();                                     // this CTA's rows of the output are written
        if (threadIdx.x == 0) dep_arrive(done_ctr);
    }
    cluster.sync();                                          // peers may still be reading this CTA's partial
    if (trace && threadIdx.x == 0 && cta < 256) trace[(size_t)cta * 16 + 12] = global_timer_ns();
}

size_t attention_tc_workspace_bytes(int n_heads, int n_sms)
{
    (void)n_heads; (void)n_sms;
    return 256;   // the merge runs through distributed shared memory; no global workspace is needed
}

cudaError_t launch_attention_tc(const void *q, const void *k, const void *v, int n_heads, int hd, int kv_stride, int P,
                                int n, const uint32_t *anc, void *o, float *ws, uint32_t *counters, int n_sms,
                                int32_t *status, cudaStream_t st, int *launched, unsigned long long *trace, int comp,
                                const void *kv_lo, int n_tree, int q_first, const AttnSync *sync)
{
    if (n_tree <= 0) n_tree = n;
    (void)ws; (void)counters;
    if (hd != kHd) return cudaErrorInvalidValue;
    const int n_pad = (n + 15) / 16 * 16;
    const int n_tiles = (P + n_tree + kKeyTile - 1) / kKeyTile;
    // one CTA per SM is resident (register file): aim for a single wave of heads x splits CTAs
    int splits = n_sms / n_heads;
    if (splits > kMaxSplits) splits = kMaxSplits;
    if (splits > n_tiles) splits = n_tiles;
    if (splits < 1) splits = 1;
    const int tiles_base = n_tiles / splits, tiles_rem = n_tiles % splits;   // the first tiles_rem splits take one tile more
    const int q_tiles = n_pad / 16;
    const int groups = q_tiles <= 2 ? 4 : (q_tiles <= 4 ? 2 : 1);
    if (comp && kv_lo == nullptr) return cudaErrorInvalidValue;
    const int stages = (comp && groups == 1) ? 3 : kMaxStages;
    const size_t ring = (size_t)(comp ? 2 : 1) * n_pad * kRowBytes + (size_t)2 * stages * kKeyTile * kRowBytes +
                        (comp ? (size_t)2 * (n_pad + 1) * kRowBytes : 0);
    const size_t part = (size_t)(groups > 1 ? groups + 1 : 1) * n_pad * kWsRow * sizeof(float);
    const size_t recv_off = ((ring > part ? ring : part) + 127) / 128 * 128;
    // with four key groups (<= 32 nodes) the rows are pushed to their owners: [splits][rows per CTA][kWsRow] behind the rest
    const size_t recv = groups == 4 ? (size_t)splits * ((n_pad + splits - 1) / splits) * kWsRow * sizeof(float) : 0;
    const size_t smem = recv_off + recv;
    typedef void (*Kern)(const __nv_bfloat16 *, const __nv_bfloat16 *, const __nv_bfloat16 *, int, int, int, int, int,
                         const uint32_t *, __nv_bfloat16 *, int, int, int, const int32_t *, unsigned long long *,
                         const __nv_bfloat16 *, int, int, DepWait, uint32_t *, int);
    static const Kern kerns[2][3] = {{attention_tc_kernel<1, false>, attention_tc_kernel<2, false>, attention_tc_kernel<4, false>},
                                     {attention_tc_kernel<1, true>, attention_tc_kernel<2, true>, attention_tc_kernel<4, true>}};
    static PerDeviceOnce attr_set;
    if (attr_set.needed()) {
        // 128 nodes, hi + lo; with <= 32 nodes: a deeper ring, and the receive buffer behind it
        const int max_smem = 2 * 128 * kRowBytes + 2 * 3 * kKeyTile * kRowBytes + 2 * 129 * kRowBytes + 128;
        for (int c = 0; c < 2; ++c)
            for (int g = 0; g < 3; ++g) {
                cudaError_t e = cudaFuncSetAttribute(kerns[c][g], cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
                // the largest shared-memory split of the SM, so that the next GEMM's streaming CTA can settle beside this kernel's
                if (e == cudaSuccess) e = cudaFuncSetAttribute(kerns[c][g], cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
                if (e != cudaSuccess) return e;
            }
        attr_set.mark();
    }
    LaunchCfg lc(dim3(splits, n_heads), dim3(kAtThreads), smem, st, splits);
    if (launched) *launched = 1;
    Kern kern = kerns[comp ? 1 : 0][groups == 4 ? 2 : (groups == 2 ? 1 : 0)];
    DepWait dep{nullptr, 0, kDefaultWaitLimitNs};
    uint32_t *done = nullptr;
    if (sync != nullptr) {
        dep = DepWait{sync->dep_ctr, sync->dep_target, sync->wait_limit_ns ? sync->wait_limit_ns : kDefaultWaitLimitNs};
        done = sync->done_ctr;
        sync->arrivals = (uint32_t)(splits * n_heads);
    }
    return cudaLaunchKernelEx(&lc.cfg, kern, (const __nv_bfloat16 *)q, (const __nv_bfloat16 *)k,
                              (const __nv_bfloat16 *)v, n_heads, kv_stride, P, n, n_pad, anc, (__nv_bfloat16 *)o, splits,
                              tiles_base, tiles_rem, (const int32_t *)status, trace, (const __nv_bfloat16 *)kv_lo, n_tree, q_first, dep, done,
                              (int)recv_off);
}

}  // namespace llmcad
