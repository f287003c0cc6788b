// C ABI of the library (see include/llmcad.h): contexts, weight packing, and the host-side
// sequencing of one verification pass. All arithmetic of the pass runs in the kernels of the
// other translation units; this file only validates arguments and enqueues them in order.
#include <cuda.h>

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/llmcad_profile.h"
#include "attention_tc.cuh"
#include "common.cuh"
#include "gemm_tc.cuh"

using namespace llmcad;

namespace {

thread_local char g_cuda_err[256] = "";

bool cuda_ok(cudaError_t e, const char *what)
{
    if (e == cudaSuccess) return true;
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", what, cudaGetErrorString(e));
    return false;
}

#define CUDA_TRY(expr)                                             \
    do {                                                           \
        if (!cuda_ok((expr), #expr)) return LLMCAD_ERR_CUDA;       \
    } while (0)

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct PackedLayout {
    size_t attn_norm, wqkv, wo, ffn_norm, wgu, wdown, layer_bytes;  // offsets inside one layer
    size_t tok_embed, final_norm, lm_head, total;                   // offsets from the start of the buffer
};

// The tensor-core path streams weights as pre-swizzled 16 KB tiles (pack.cu); the plain-ALU
// path reads them row-major.
bool want_tiled(const llmcad_config &c)
{
    return c.dtype == LLMCAD_BF16 && !(c.flags & LLMCAD_FLAG_SIMT_GEMM) && c.d_model % 128 == 0;
}

PackedLayout packed_layout(const llmcad_config &c)
{
    const size_t e = c.dtype == LLMCAD_F32 ? 4 : 2;
    const size_t d = c.d_model, f = c.d_ffn, v = c.vocab;
    const bool tiled = want_tiled(c);
    const bool w4 = tiled && (c.flags & LLMCAD_FLAG_INT4_WEIGHTS);     // the layer matrices only; the lm_head stays bf16
    auto mat_head = [&](size_t n_out, size_t n_in) { return tiled ? tiled_weight_bytes((int)n_out, (int)n_in) : n_out * n_in * e; };
    auto mat = [&](size_t n_out, size_t n_in) { return w4 ? tiled_weight_int4_bytes((int)n_out, (int)n_in) : mat_head(n_out, n_in); };
    PackedLayout L{};
    size_t o = 0;
    L.attn_norm = o; o = align_up(o + d * e, 1024);
    L.wqkv = o;      o = align_up(o + 3 * mat(d, d), 1024);
    L.wo = o;        o = align_up(o + mat(d, d), 1024);
    L.ffn_norm = o;  o = align_up(o + d * e, 1024);
    L.wgu = o;       o = align_up(o + 2 * mat(f, d), 1024);
    L.wdown = o;     o = align_up(o + mat(d, f), 1024);
    L.layer_bytes = o;
    o = L.layer_bytes * (size_t)c.n_layers;
    L.tok_embed = o;  o = align_up(o + v * d * e, 1024);
    L.final_norm = o; o = align_up(o + d * e, 1024);
    L.lm_head = o;    o = align_up(o + mat_head(v, d), 1024);
    L.total = o;
    return L;
}

int check_config(const llmcad_config *c)
{
    if (c == nullptr) return LLMCAD_ERR_INVALID_ARG;
    if (c->n_layers < 0 || c->d_model <= 0 || c->n_heads <= 0 || c->head_dim <= 0 || c->d_ffn <= 0 || c->vocab <= 0 ||
        c->max_seq <= 0 || c->max_tree <= 0)
        return LLMCAD_ERR_INVALID_ARG;
    if (c->dtype != LLMCAD_F32 && c->dtype != LLMCAD_BF16) return LLMCAD_ERR_UNSUPPORTED;
    if (c->max_tree > LLMCAD_MAX_TREE) return LLMCAD_ERR_UNSUPPORTED;
    if (c->head_dim != 64 && c->head_dim != 128) return LLMCAD_ERR_UNSUPPORTED;
    if (c->n_heads * c->head_dim != c->d_model) return LLMCAD_ERR_UNSUPPORTED;
    if (c->d_model % 8 || c->d_ffn % 8) return LLMCAD_ERR_UNSUPPORTED;
    // INT4 weights: the tensor-core path only, groups of 64 input columns
    if ((c->flags & LLMCAD_FLAG_INT4_WEIGHTS) && (!want_tiled(*c) || c->d_model % 64 || c->d_ffn % 64)) return LLMCAD_ERR_UNSUPPORTED;
    return LLMCAD_OK;
}

}  // namespace

constexpr int kSyncCounters = 2048;

struct llmcad_ctx {
    llmcad_config cfg;
    PackedLayout lay;
    int n_sms = 0;
    size_t elem = 2;
    bool tc_gemm = false, tc_attn = false;
    bool w4 = false;          // the layer matrices are held as INT4 tiles (LLMCAD_FLAG_INT4_WEIGHTS)
    // Tensor-core path: activations travel as bf16 hi + lo planes (common.cuh); a tuning aid
    // (LLMCAD_COMP=0) turns the lo planes off.
    bool comp = false;
    // activations of up to 128 nodes; xn, q, att and h hold two planes of 128 rows (hi, lo)
    float *x = nullptr;       // residual stream [128][d] fp32
    void *xn = nullptr;       // normalised GEMM input [2][128][d]
    void *q = nullptr;        // rotated queries [2][128][d]
    void *att = nullptr;      // attention output [2][128][d]
    void *h = nullptr;        // SwiGLU output [2][128][f]
    void *kv_lo = nullptr;    // bf16 remainders of the current layer's tree keys and values [2][H][128][hd]
    float *logits = nullptr;  // [128][V], used when the caller does not want logits
    TreeBuffers tb{};
    int32_t *ibuf = nullptr;  // tokens[128], parent[128], argmax[128], path[128], scalars[8], chain[128]
    float *partials = nullptr;            // segment workspace of the tensor-core GEMMs
    size_t partial_floats = 0;
    float *ssq[2] = {nullptr, nullptr};   // partial sums of squares for the folded attention / FFN norms
    float *attn_ws = nullptr;
    uint32_t *attn_counters = nullptr;
    // completion counters through which the kernels of a tensor-core pass hand over (common.cuh): one per
    // kernel, taken in launch order, all zeroed at the start of a forward. Off by default: measured on B200
    // (7B shape, 32 nodes) the hand-over through counters costs 4 % of the pass against grid dependencies
    // (a release after a burst of stores takes 2-4 us under the weight stream; the grid dependency's flush
    // takes 1.3). LLMCAD_SYNC_COUNTERS=1 (tuning aid, read at creation) switches it on.
    uint32_t *sync_ctrs = nullptr;
    int sync_next = 0;
    bool use_counters = false;
    uint32_t *next_ctr() { return (use_counters && sync_next < kSyncCounters) ? sync_ctrs + sync_next++ : nullptr; }
    int64_t launches = 0;
    uint64_t wait_limit_ns = kDefaultWaitLimitNs;   // bound of every device-side wait (llmcad_set_wait_limit_ns)
    unsigned long long *trace = nullptr;   // optional timeline buffer (llmcad_set_gemm_trace): [launch][256][16]
    int trace_launch = 0, trace_capacity = 0;
    unsigned long long *next_trace()
    {
        if (trace == nullptr || trace_launch >= trace_capacity) return nullptr;
        return trace + (size_t)(trace_launch++) * 256 * 16;
    }
    const void *maps_for = nullptr;    // packed weight buffer of the current call
    CUtensorMap act_maps[9][3];        // [n_pad/16][xn, att, h]
    bool act_ready[9] = {false, false, false, false, false, false, false, false, false};
    // optional per-launch timing (events around every GEMM / attention launch)
    bool timing = false;
    struct Timed { int kind; cudaEvent_t a, b; };
    std::vector<Timed> timed;
    std::vector<cudaEvent_t> event_pool;

    int32_t *tokens_dev() const { return ibuf; }
    int32_t *parent_dev() const { return ibuf + 128; }
    int32_t *argmax_dev() const { return ibuf + 256; }
    int32_t *path_dev() const { return ibuf + 384; }
    int32_t *scalars_dev() const { return ibuf + 512; }
    int32_t *chain_dev() const { return ibuf + 520; }
};

namespace {

// Brackets one launch with events when kernel timing is on.
struct TimedLaunch {
    llmcad_ctx *ctx;
    cudaStream_t st;
    cudaEvent_t a = nullptr, b = nullptr;
    int kind;
    TimedLaunch(llmcad_ctx *c, int k, cudaStream_t s) : ctx(c), st(s), kind(k)
    {
        if (!ctx->timing) return;
        a = take();
        b = take();
        if (a && b) cudaEventRecord(a, st);
    }
    ~TimedLaunch()
    {
        if (!ctx->timing || !a || !b) return;
        cudaEventRecord(b, st);
        ctx->timed.push_back({kind, a, b});
    }
    cudaEvent_t take()
    {
        if (!ctx->event_pool.empty()) {
            cudaEvent_t e = ctx->event_pool.back();
            ctx->event_pool.pop_back();
            return e;
        }
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
        return e;
    }
};

int ensure_weight_maps(llmcad_ctx *ctx, const void *packed)
{
    // the pass reads its weights as pre-swizzled tiles through plain bulk copies, so there is no
    // tensor map to encode for them: remember which packed buffer the chains address
    ctx->maps_for = packed;
    return LLMCAD_OK;
}

int ensure_act_maps(llmcad_ctx *ctx, int n_pad)
{
    const int slot = n_pad / 16;
    if (!ctx->tc_gemm || ctx->act_ready[slot]) return LLMCAD_OK;
    const llmcad_config &c = ctx->cfg;
    bool ok = true;
    const uint32_t planes = ctx->comp ? 2 : 1;
    ok &= make_act_map_bf16(&ctx->act_maps[slot][0], ctx->xn, 128, c.d_model, n_pad, planes, kLoRows);
    ok &= make_act_map_bf16(&ctx->act_maps[slot][1], ctx->att, 128, c.d_model, n_pad, planes, kLoRows);
    ok &= make_act_map_bf16(&ctx->act_maps[slot][2], ctx->h, 128, c.d_ffn, n_pad, planes, kLoRows);
    if (!ok) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled failed for an activation buffer");
        return LLMCAD_ERR_CUDA;
    }
    ctx->act_ready[slot] = true;
    return LLMCAD_OK;
}

// One tensor-core GEMM of the pass: the streaming kernel and its finishing kernel.
struct TcGemm {
    GemmMaps maps;
    GemmParams p;
    TcGemm() { p = GemmParams{}; }
    // W is `which` (0 qkv, 1 o, 2 gate/up, 3 down) of layer l, or the lm_head when l < 0;
    // act selects the activation buffer it multiplies (0 normalised stream, 1 attention output, 2 SwiGLU output)
    static const char *weight_ptr(llmcad_ctx *ctx, int l, int which)
    {
        const char *base = static_cast<const char *>(ctx->maps_for);
        if (l < 0) return base + ctx->lay.lm_head;
        const char *lb = base + ctx->lay.layer_bytes * (size_t)l;
        return lb + (which == 0 ? ctx->lay.wqkv : which == 1 ? ctx->lay.wo : which == 2 ? ctx->lay.wgu : ctx->lay.wdown);
    }
    void set(llmcad_ctx *ctx, int l, int which, int act, int n_in, const EpiParams &ep, int n_pad)
    {
        maps.x = ctx->act_maps[n_pad / 16][act];
        p.g = make_gemm_desc(n_in, ep, weight_ptr(ctx, l, which), ctx->w4 && l >= 0);
        p.n_pad = n_pad;
        p.comp = ctx->comp ? 1 : 0;
    }
    int launch(llmcad_ctx *ctx, int32_t *status, cudaStream_t st)
    {
        p.partials = ctx->partials;
        p.status = status;
        p.wait_limit_ns = ctx->wait_limit_ns;
        p.trace = ctx->next_trace();
        int launched = 0;
        TimedLaunch tl(ctx, 0, st);
        const cudaError_t e = launch_gemm_tc(maps, p, ctx->n_sms, ctx->partial_floats, st, &launched);
        ctx->launches += launched;
        if (e == cudaErrorInvalidValue && launched == 0) return LLMCAD_ERR_UNSUPPORTED;   // more tiles than the workspace holds
        CUDA_TRY(e);
        return LLMCAD_OK;
    }
};

// One GEMM of the plain-ALU path: W is `which` of layer l (or the lm_head when l < 0).
int run_gemm(llmcad_ctx *ctx, const void *packed, int l, int which, int act, int n_in, const EpiParams &ep, int n_pad,
             int32_t *status, cudaStream_t st)
{
    (void)n_pad;
    const char *base = static_cast<const char *>(packed);
    const void *xin = act == 0 ? ctx->xn : act == 1 ? ctx->att : ctx->h;
    ctx->launches++;
    TimedLaunch tl(ctx, 0, st);
    const void *W;
    if (l < 0) W = base + ctx->lay.lm_head;
    else {
        const char *lb = base + ctx->lay.layer_bytes * (size_t)l;
        W = lb + (which == 0 ? ctx->lay.wqkv : which == 1 ? ctx->lay.wo : which == 2 ? ctx->lay.wgu : ctx->lay.wdown);
    }
    CUDA_TRY(launch_gemm_simt(W, xin, ctx->cfg.dtype, n_in, ep, status, st));
    return LLMCAD_OK;
}

// comp: q carries a lo plane kLoRows rows after the hi plane, and o gets one too (the pass);
// the single-step entry points work on plain bf16 buffers.
int run_attention(llmcad_ctx *ctx, const void *q, const void *k, const void *v, int kv_stride, int P, int n, void *o,
                  bool comp, int32_t *status, cudaStream_t st, int n_tree = 0, int q_first = 0, const AttnSync *sync = nullptr)
{
    const llmcad_config &c = ctx->cfg;
    TimedLaunch tl(ctx, 1, st);
    if (ctx->tc_attn) {
        int launched = 0;
        const bool t5 = (c.flags & LLMCAD_FLAG_T5_ATTN) ? true
                        : (c.flags & LLMCAD_FLAG_MMA_ATTN) ? false : attention_prefers_t5(n);
        if (t5) {
            CUDA_TRY(launch_attention_t5(q, k, v, c.n_heads, c.head_dim, kv_stride, P, n, ctx->tb.anc, o, ctx->n_sms, status, st,
                                         &launched, ctx->next_trace(), comp ? 1 : 0, ctx->kv_lo, n_tree, q_first, ctx->wait_limit_ns, sync));
            ctx->launches += launched;
            return LLMCAD_OK;
        }
        CUDA_TRY(launch_attention_tc(q, k, v, c.n_heads, c.head_dim, kv_stride, P, n, ctx->tb.anc, o, ctx->attn_ws,
                                     ctx->attn_counters, ctx->n_sms, status, st, &launched, ctx->next_trace(), comp ? 1 : 0,
                                     ctx->kv_lo, n_tree, q_first, sync));
        ctx->launches += launched;
        return LLMCAD_OK;
    }
    if (sizeof(float) * (size_t)(c.head_dim + P + (n_tree > 0 ? n_tree : n)) > 200 * 1024) return LLMCAD_ERR_UNSUPPORTED;
    ctx->launches++;
    CUDA_TRY(launch_attention_simt(q, k, v, c.dtype, c.n_heads, c.head_dim, kv_stride, P, n, ctx->tb.anc, o, status, st, n_tree,
                                   q_first));
    return LLMCAD_OK;
}

// Decoder forward over the nodes n_old .. n_tree-1 of a tree of n_tree nodes (all of them when
// n_old = 0): tree prep of the whole tree, embedding, all layers; K/V of node i go to cache slot
// P+i, where the nodes below n_old already have theirs. When logits != nullptr the final norm and
// lm_head run too (one row per processed node).
int run_forward(llmcad_ctx *ctx, const void *packed, void *kv_cache, int P, const int32_t *tokens,
                const int32_t *parent, int n_tree, float *logits, int32_t *status, cudaStream_t st, int n_old = 0)
{
    const llmcad_config &c = ctx->cfg;
    const int d = c.d_model, f = c.d_ffn, hd = c.head_dim, H = c.n_heads, S = c.max_seq;
    const int n = n_tree - n_old;                    // nodes this call computes
    const int n_pad = (n + 15) / 16 * 16;
    const int32_t *new_tokens = tokens + n_old;
    const char *base = static_cast<const char *>(packed);
    int rc;
    if ((rc = ensure_weight_maps(ctx, packed)) != LLMCAD_OK) return rc;
    if ((rc = ensure_act_maps(ctx, n_pad)) != LLMCAD_OK) return rc;

    CUDA_TRY(launch_tree_prep(parent, tokens, n_tree, P, c.vocab, hd, c.rope_base, ctx->tb, status, st));
    ctx->launches += 2;
    const float2 *rope_new = ctx->tb.rope_cs + (size_t)n_old * (hd / 2);
    const size_t kv_layer = (size_t)2 * H * S * hd * ctx->elem;

    if (ctx->tc_gemm) {
        // Tensor-core path. The RMSNorms are folded into the GEMMs: whoever produces the residual
        // stream (the embedding gather, the O and down GEMMs) also writes gain * x in bf16 and
        // partial sums of squares; the consuming GEMM scales its accumulators by the per-node
        // rsqrt(mean(x^2) + eps). Activations travel as bf16 hi + lo planes (ctx->comp).
        const int tiles4 = 4 * ((d + 127) / 128);
        CUDA_TRY(launch_embed_norm(base + ctx->lay.tok_embed, new_tokens, n, d,
                                   c.n_layers > 0 ? base + ctx->lay.attn_norm : base + ctx->lay.final_norm, ctx->x, ctx->xn,
                                   ctx->ssq[0], ctx->comp ? 1 : 0, status, st));
        auto qkv_ep = [&](int l, int parts) {
            char *kl = static_cast<char *>(kv_cache) + kv_layer * (size_t)l;
            EpiParams ep{};
            ep.n = n; ep.mode = EPI_QKV; ep.n_out = 3 * d; ep.q_out = ctx->q; ep.k_cache = kl; ep.v_cache = kl + kv_layer / 2;
            ep.rope_cs = rope_new; ep.d = d; ep.hd = hd; ep.S = S; ep.P = P + n_old;
            ep.ssq_in = ctx->ssq[0]; ep.ssq_in_parts = parts; ep.norm_d = d; ep.eps = c.rms_eps;
            ep.comp = ctx->comp ? 1 : 0; ep.kv_lo = ctx->kv_lo;
            return ep;
        };
        auto head_ep = [&](int parts) {
            EpiParams ep{};
            ep.n = n; ep.mode = EPI_PLAIN; ep.n_out = c.vocab; ep.y = logits; ep.ldy = c.vocab;
            ep.ssq_in = ctx->ssq[0]; ep.ssq_in_parts = parts; ep.norm_d = d; ep.eps = c.rms_eps;
            return ep;
        };
        // the GEMMs of the pass in order; attention runs before the O GEMM of every layer
        struct Spec { int l, which, act, n_in; EpiParams ep; bool attention_first; };
        std::vector<Spec> specs;
        if (c.n_layers > 0) specs.push_back({0, 0, 0, d, qkv_ep(0, 1), false});
        else if (logits != nullptr) specs.push_back({-1, 0, 0, d, head_ep(1), false});
        for (int l = 0; l < c.n_layers; ++l) {
            const char *lb = base + ctx->lay.layer_bytes * (size_t)l;
            const bool last = l + 1 == c.n_layers;
            const char *next_gain = last ? base + ctx->lay.final_norm : lb + ctx->lay.layer_bytes + ctx->lay.attn_norm;
            EpiParams ep{};
            ep.n = n; ep.mode = EPI_RESID; ep.n_out = d; ep.x = ctx->x;
            ep.xg_out = ctx->xn; ep.gain_next = lb + ctx->lay.ffn_norm; ep.ssq_out = ctx->ssq[1];
            ep.comp = ctx->comp ? 1 : 0;
            specs.push_back({l, 1, 1, d, ep, true});

            ep = EpiParams{}; ep.n = n; ep.mode = EPI_SWIGLU; ep.n_out = f; ep.h = ctx->h;
            ep.ssq_in = ctx->ssq[1]; ep.ssq_in_parts = tiles4; ep.norm_d = d; ep.eps = c.rms_eps;
            ep.comp = ctx->comp ? 1 : 0;
            specs.push_back({l, 2, 0, d, ep, false});

            ep = EpiParams{}; ep.n = n; ep.mode = EPI_RESID; ep.n_out = d; ep.x = ctx->x;
            ep.xg_out = ctx->xn; ep.gain_next = next_gain; ep.ssq_out = ctx->ssq[0];
            ep.comp = ctx->comp ? 1 : 0;
            specs.push_back({l, 3, 2, f, ep, false});

            if (!last) specs.push_back({l + 1, 0, 0, d, qkv_ep(l + 1, tiles4), false});
            else if (logits != nullptr) specs.push_back({-1, 0, 0, d, head_ep(tiles4), false});
        }
        std::vector<TcGemm> gemms(specs.size());
        for (size_t i = 0; i < specs.size(); ++i)
            gemms[i].set(ctx, specs[i].l, specs[i].which, specs[i].act, specs[i].n_in, specs[i].ep, n_pad);
        // Hand-over between the kernels: completion counters (one per kernel, zeroed here) where both sides are
        // tensor-core kernels of this library, the grid dependency otherwise. `dep` is what the next kernel
        // waits for: null after the embedding kernel and after a plain-ALU attention kernel.
        ctx->sync_next = 0;
        if (ctx->use_counters) CUDA_TRY(cudaMemsetAsync(ctx->sync_ctrs, 0, kSyncCounters * sizeof(uint32_t), st));
        const uint32_t *dep = nullptr;
        uint32_t dep_target = 0;
        for (size_t i = 0; i < specs.size(); ++i) {
            if (specs[i].attention_first) {
                char *kl = static_cast<char *>(kv_cache) + kv_layer * (size_t)specs[i].l;
                AttnSync sync{dep, dep_target, ctx->tc_attn ? ctx->next_ctr() : nullptr, ctx->wait_limit_ns, 0};
                const bool with_sync = ctx->tc_attn && sync.done_ctr != nullptr;
                // without the tensor-core attention kernel the lo plane of att stays zero, as allocated
                if ((rc = run_attention(ctx, ctx->q, kl, kl + kv_layer / 2, S, P, n, ctx->att, ctx->comp && ctx->tc_attn, status, st,
                                        n_tree, n_old, with_sync ? &sync : nullptr)) != LLMCAD_OK) return rc;
                dep = with_sync ? sync.done_ctr : nullptr;
                dep_target = sync.arrivals;
            }
            GemmParams &gp = gemms[i].p;
            gp.dep_ctr = dep; gp.dep_target = dep_target;
            gp.s_done = ctx->next_ctr();
            gp.f_done = gp.s_done != nullptr ? ctx->next_ctr() : nullptr;
            if (gp.f_done == nullptr) gp.s_done = nullptr;
            if ((rc = gemms[i].launch(ctx, status, st)) != LLMCAD_OK) return rc;
            dep = gp.f_done;
            dep_target = (uint32_t)gp.f_grid;
        }
        return LLMCAD_OK;
    }

    CUDA_TRY(launch_embed(base + ctx->lay.tok_embed, c.dtype, new_tokens, n, d, ctx->x, status, st));
    for (int l = 0; l < c.n_layers; ++l) {
        const char *lb = base + ctx->lay.layer_bytes * (size_t)l;
        char *kl = static_cast<char *>(kv_cache) + kv_layer * (size_t)l;
        char *vl = kl + kv_layer / 2;
        EpiParams ep{};
        ep.n = n;

        CUDA_TRY(launch_rmsnorm(ctx->x, lb + ctx->lay.attn_norm, c.dtype, n, d, c.rms_eps, ctx->xn, status, st));
        ctx->launches++;
        ep.mode = EPI_QKV; ep.n_out = 3 * d; ep.q_out = ctx->q; ep.k_cache = kl; ep.v_cache = vl;
        ep.rope_cs = rope_new; ep.d = d; ep.hd = hd; ep.S = S; ep.P = P + n_old;
        if ((rc = run_gemm(ctx, packed, l, 0, 0, d, ep, n_pad, status, st)) != LLMCAD_OK) return rc;

        if ((rc = run_attention(ctx, ctx->q, kl, vl, S, P, n, ctx->att, false, status, st, n_tree, n_old)) != LLMCAD_OK) return rc;

        ep = EpiParams{}; ep.n = n; ep.mode = EPI_RESID; ep.n_out = d; ep.x = ctx->x;
        if ((rc = run_gemm(ctx, packed, l, 1, 1, d, ep, n_pad, status, st)) != LLMCAD_OK) return rc;

        CUDA_TRY(launch_rmsnorm(ctx->x, lb + ctx->lay.ffn_norm, c.dtype, n, d, c.rms_eps, ctx->xn, status, st));
        ctx->launches++;
        ep = EpiParams{}; ep.n = n; ep.mode = EPI_SWIGLU; ep.n_out = f; ep.h = ctx->h;
        if ((rc = run_gemm(ctx, packed, l, 2, 0, d, ep, n_pad, status, st)) != LLMCAD_OK) return rc;

        ep = EpiParams{}; ep.n = n; ep.mode = EPI_RESID; ep.n_out = d; ep.x = ctx->x;
        if ((rc = run_gemm(ctx, packed, l, 3, 2, f, ep, n_pad, status, st)) != LLMCAD_OK) return rc;
    }
    if (logits != nullptr) {
        CUDA_TRY(launch_rmsnorm(ctx->x, base + ctx->lay.final_norm, c.dtype, n, d, c.rms_eps, ctx->xn, status, st));
        ctx->launches++;
        EpiParams ep{};
        ep.n = n; ep.mode = EPI_PLAIN; ep.n_out = c.vocab; ep.y = logits; ep.ldy = c.vocab;
        if ((rc = run_gemm(ctx, packed, -1, 0, 0, d, ep, n_pad, status, st)) != LLMCAD_OK) return rc;
    }
    return LLMCAD_OK;
}

int check_pass_args(const llmcad_ctx *ctx, const void *packed, const void *kv, int P, const void *tok, const void *par, int n)
{
    if (ctx == nullptr || packed == nullptr || kv == nullptr || tok == nullptr || par == nullptr) return LLMCAD_ERR_INVALID_ARG;
    // bulk copies of weight tiles and 8/16-byte vector stores into the cache: the header asks for 256-byte alignment
    if ((reinterpret_cast<uintptr_t>(packed) & 255) != 0 || (reinterpret_cast<uintptr_t>(kv) & 255) != 0) return LLMCAD_ERR_INVALID_ARG;
    if (n < 1 || P < 0) return LLMCAD_ERR_INVALID_ARG;
    if (n > ctx->cfg.max_tree) return LLMCAD_ERR_UNSUPPORTED;
    if ((long long)P + n > ctx->cfg.max_seq) return LLMCAD_ERR_CAPACITY;
    return LLMCAD_OK;
}

}  // namespace

// =============================================================================================
extern "C" {

int llmcad_version(void) { return 100; }

const char *llmcad_strerror(int code)
{
    switch (code) {
    case LLMCAD_OK: return "ok";
    case LLMCAD_ERR_INVALID_ARG: return "invalid argument";
    case LLMCAD_ERR_UNSUPPORTED: return "unsupported size, shape or dtype";
    case LLMCAD_ERR_CAPACITY: return "prefix_len + n exceeds the cache capacity";
    case LLMCAD_ERR_CUDA: return "CUDA call failed";
    case LLMCAD_ERR_BAD_TREE: return "malformed tree (parent_idx)";
    case LLMCAD_ERR_BAD_TOKEN: return "token id out of range";
    case LLMCAD_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case LLMCAD_ERR_NAN: return "NaN logit";
    case LLMCAD_ERR_CHECK: return "a device-side bounds check of the debug build failed";
    default: return "unknown error";
    }
}

const char *llmcad_last_cuda_error(void) { return g_cuda_err; }

size_t llmcad_kv_cache_bytes(const llmcad_config *cfg)
{
    if (check_config(cfg) != LLMCAD_OK) return 0;
    const size_t e = cfg->dtype == LLMCAD_F32 ? 4 : 2;
    return (size_t)cfg->n_layers * 2 * cfg->n_heads * cfg->max_seq * cfg->head_dim * e;
}

size_t llmcad_packed_weight_bytes(const llmcad_config *cfg)
{
    if (check_config(cfg) != LLMCAD_OK) return 0;
    return packed_layout(*cfg).total;
}

int llmcad_create(const llmcad_config *cfg, llmcad_ctx **out)
{
    if (out == nullptr) return LLMCAD_ERR_INVALID_ARG;
    *out = nullptr;
    int rc = check_config(cfg);
    if (rc != LLMCAD_OK) return rc;
    int dev = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    cudaDeviceProp prop;
    CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
    llmcad_ctx *ctx = new (std::nothrow) llmcad_ctx();
    if (ctx == nullptr) return LLMCAD_ERR_INVALID_ARG;
    ctx->cfg = *cfg;
    ctx->lay = packed_layout(*cfg);
    ctx->n_sms = prop.multiProcessorCount;
    ctx->elem = cfg->dtype == LLMCAD_F32 ? 4 : 2;
    const bool sm100 = prop.major == 10;
    ctx->tc_gemm = want_tiled(*cfg);
    ctx->w4 = ctx->tc_gemm && (cfg->flags & LLMCAD_FLAG_INT4_WEIGHTS);
    if (ctx->tc_gemm && !sm100) {   // the tensor-core kernels are sm_100a only
        delete ctx;
        snprintf(g_cuda_err, sizeof(g_cuda_err), "device is not sm_100");
        return LLMCAD_ERR_CUDA;
    }
    ctx->tc_attn = cfg->dtype == LLMCAD_BF16 && cfg->head_dim == 128 && !(cfg->flags & LLMCAD_FLAG_SIMT_ATTN);
    {
        const char *e = getenv("LLMCAD_COMP");
        ctx->comp = ctx->tc_gemm && !(e != nullptr && atoi(e) == 0);
    }

    const size_t d = cfg->d_model, f = cfg->d_ffn, hd = cfg->head_dim;
    auto alloc = [&](void **p, size_t bytes) {
        if (!cuda_ok(cudaMalloc(p, bytes), "cudaMalloc")) return false;
        return cuda_ok(cudaMemset(*p, 0, bytes), "cudaMemset");
    };
    bool ok = true;
    ok = ok && alloc((void **)&ctx->x, 128 * d * 4);
    ok = ok && alloc(&ctx->xn, 2 * kLoRows * d * ctx->elem);
    ok = ok && alloc(&ctx->q, 2 * kLoRows * d * ctx->elem);
    ok = ok && alloc(&ctx->att, 2 * kLoRows * d * ctx->elem);
    ok = ok && alloc(&ctx->h, 2 * kLoRows * f * ctx->elem);
    ok = ok && alloc(&ctx->kv_lo, 2 * kLoRows * d * ctx->elem);
    ok = ok && alloc((void **)&ctx->logits, (size_t)128 * cfg->vocab * 4);
    ok = ok && alloc((void **)&ctx->tb.depth, 128 * 4);
    ok = ok && alloc((void **)&ctx->tb.pos, 128 * 4);
    ok = ok && alloc((void **)&ctx->tb.anc, 128 * 16);
    ok = ok && alloc((void **)&ctx->tb.rope_cs, 128 * (hd / 2) * sizeof(float2));
    ok = ok && alloc((void **)&ctx->ibuf, (520 + 128) * 4);
    {
        // segment workspace: the GEMM with the most tiles of this model (or 256 tiles, for the single-GEMM entry points)
        int max_tiles = 256;
        for (size_t rows : {3 * d, f, (size_t)cfg->vocab})
            if ((int)((rows + 127) / 128) > max_tiles) max_tiles = (int)((rows + 127) / 128);
        const int max_pad = (cfg->max_tree + 15) / 16 * 16;
        ctx->partial_floats = ctx->tc_gemm ? gemm_tc_partial_floats(ctx->n_sms, max_tiles, max_pad) : 64;
        ok = ok && alloc((void **)&ctx->partials, ctx->partial_floats * 4);
    }
    const size_t ssq_floats = (size_t)4 * ((d + 127) / 128) * LLMCAD_MAX_TREE;
    ok = ok && alloc((void **)&ctx->ssq[0], ssq_floats * 4);
    ok = ok && alloc((void **)&ctx->ssq[1], ssq_floats * 4);
    ok = ok && alloc((void **)&ctx->attn_ws, attention_tc_workspace_bytes(cfg->n_heads, ctx->n_sms));
    ok = ok && alloc((void **)&ctx->attn_counters, (size_t)cfg->n_heads * 8 * 4);
    ok = ok && alloc((void **)&ctx->sync_ctrs, kSyncCounters * sizeof(uint32_t));
    {
        const char *e = getenv("LLMCAD_SYNC_COUNTERS");
        ctx->use_counters = e != nullptr && atoi(e) != 0;
    }
    if (ok) {
        std::vector<int32_t> chain(128);
        for (int i = 0; i < 128; ++i) chain[i] = i - 1;
        ok = cuda_ok(cudaMemcpy(ctx->chain_dev(), chain.data(), 128 * 4, cudaMemcpyHostToDevice), "cudaMemcpy");
    }
    if (!ok) {
        llmcad_destroy(ctx);
        return LLMCAD_ERR_CUDA;
    }
    *out = ctx;
    return LLMCAD_OK;
}

void llmcad_destroy(llmcad_ctx *ctx)
{
    if (ctx == nullptr) return;
    void *ptrs[] = {ctx->x, ctx->xn, ctx->q, ctx->att, ctx->h, ctx->kv_lo, ctx->logits, ctx->tb.depth, ctx->tb.pos, ctx->tb.anc,
                    ctx->tb.rope_cs, ctx->ibuf, ctx->partials, ctx->attn_ws, ctx->attn_counters, ctx->sync_ctrs, ctx->ssq[0],
                    ctx->ssq[1]};
    for (void *p : ptrs)
        if (p != nullptr) cudaFree(p);
    for (auto &t : ctx->timed) { cudaEventDestroy(t.a); cudaEventDestroy(t.b); }
    for (auto e : ctx->event_pool) cudaEventDestroy(e);
    delete ctx;
}

int llmcad_pack_layer(llmcad_ctx *ctx, int32_t layer, const llmcad_layer_weights *src, void *packed, void *stream)
{
    if (ctx == nullptr || src == nullptr || packed == nullptr) return LLMCAD_ERR_INVALID_ARG;
    if (layer < 0 || layer >= ctx->cfg.n_layers) return LLMCAD_ERR_INVALID_ARG;
    if (!src->attn_norm || !src->wq || !src->wk || !src->wv || !src->wo || !src->ffn_norm || !src->w_gate || !src->w_up ||
        !src->w_down)
        return LLMCAD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t e = ctx->elem, d = ctx->cfg.d_model, f = ctx->cfg.d_ffn;
    char *lb = static_cast<char *>(packed) + ctx->lay.layer_bytes * (size_t)layer;
    auto cp = [&](size_t off, const void *s, size_t bytes) {
        return cudaMemcpyAsync(lb + off, s, bytes, cudaMemcpyDeviceToDevice, st);
    };
    if (ctx->w4) {
        // quantised on the way in: INT4 codes and power-of-two group scales, tiled for the streaming kernel
        const size_t t_dd = tiled_weight_int4_bytes((int)d, (int)d), t_fd = tiled_weight_int4_bytes((int)f, (int)d);
        CUDA_TRY(cp(ctx->lay.attn_norm, src->attn_norm, d * e));
        CUDA_TRY(cp(ctx->lay.ffn_norm, src->ffn_norm, d * e));
        CUDA_TRY(launch_tile_weight_int4(src->wq, (int)d, (int)d, lb + ctx->lay.wqkv, st));
        CUDA_TRY(launch_tile_weight_int4(src->wk, (int)d, (int)d, lb + ctx->lay.wqkv + t_dd, st));
        CUDA_TRY(launch_tile_weight_int4(src->wv, (int)d, (int)d, lb + ctx->lay.wqkv + 2 * t_dd, st));
        CUDA_TRY(launch_tile_weight_int4(src->wo, (int)d, (int)d, lb + ctx->lay.wo, st));
        CUDA_TRY(launch_tile_weight_int4(src->w_gate, (int)f, (int)d, lb + ctx->lay.wgu, st));
        CUDA_TRY(launch_tile_weight_int4(src->w_up, (int)f, (int)d, lb + ctx->lay.wgu + t_fd, st));
        CUDA_TRY(launch_tile_weight_int4(src->w_down, (int)d, (int)f, lb + ctx->lay.wdown, st));
        return LLMCAD_OK;
    }
    if (ctx->tc_gemm) {
        const size_t t_dd = tiled_weight_bytes((int)d, (int)d), t_fd = tiled_weight_bytes((int)f, (int)d);
        CUDA_TRY(cp(ctx->lay.attn_norm, src->attn_norm, d * e));
        CUDA_TRY(cp(ctx->lay.ffn_norm, src->ffn_norm, d * e));
        CUDA_TRY(launch_tile_weight(src->wq, (int)d, (int)d, lb + ctx->lay.wqkv, st));
        CUDA_TRY(launch_tile_weight(src->wk, (int)d, (int)d, lb + ctx->lay.wqkv + t_dd, st));
        CUDA_TRY(launch_tile_weight(src->wv, (int)d, (int)d, lb + ctx->lay.wqkv + 2 * t_dd, st));
        CUDA_TRY(launch_tile_weight(src->wo, (int)d, (int)d, lb + ctx->lay.wo, st));
        CUDA_TRY(launch_tile_weight(src->w_gate, (int)f, (int)d, lb + ctx->lay.wgu, st));
        CUDA_TRY(launch_tile_weight(src->w_up, (int)f, (int)d, lb + ctx->lay.wgu + t_fd, st));
        CUDA_TRY(launch_tile_weight(src->w_down, (int)d, (int)f, lb + ctx->lay.wdown, st));
        return LLMCAD_OK;
    }
    CUDA_TRY(cp(ctx->lay.attn_norm, src->attn_norm, d * e));
    CUDA_TRY(cp(ctx->lay.wqkv, src->wq, d * d * e));
    CUDA_TRY(cp(ctx->lay.wqkv + d * d * e, src->wk, d * d * e));
    CUDA_TRY(cp(ctx->lay.wqkv + 2 * d * d * e, src->wv, d * d * e));
    CUDA_TRY(cp(ctx->lay.wo, src->wo, d * d * e));
    CUDA_TRY(cp(ctx->lay.ffn_norm, src->ffn_norm, d * e));
    CUDA_TRY(cp(ctx->lay.wgu, src->w_gate, f * d * e));
    CUDA_TRY(cp(ctx->lay.wgu + f * d * e, src->w_up, f * d * e));
    CUDA_TRY(cp(ctx->lay.wdown, src->w_down, d * f * e));
    return LLMCAD_OK;
}

int llmcad_pack_globals(llmcad_ctx *ctx, const llmcad_global_weights *src, void *packed, void *stream)
{
    if (ctx == nullptr || src == nullptr || packed == nullptr) return LLMCAD_ERR_INVALID_ARG;
    if (!src->tok_embed || !src->final_norm || !src->lm_head) return LLMCAD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t e = ctx->elem, d = ctx->cfg.d_model, v = ctx->cfg.vocab;
    char *b = static_cast<char *>(packed);
    CUDA_TRY(cudaMemcpyAsync(b + ctx->lay.tok_embed, src->tok_embed, v * d * e, cudaMemcpyDeviceToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(b + ctx->lay.final_norm, src->final_norm, d * e, cudaMemcpyDeviceToDevice, st));
    if (ctx->tc_gemm) CUDA_TRY(launch_tile_weight(src->lm_head, (int)v, (int)d, b + ctx->lay.lm_head, st));
    else CUDA_TRY(cudaMemcpyAsync(b + ctx->lay.lm_head, src->lm_head, v * d * e, cudaMemcpyDeviceToDevice, st));
    return LLMCAD_OK;
}

int llmcad_verify_tree(llmcad_ctx *ctx, const void *packed, void *kv_cache, int32_t prefix_len,
                       const int32_t *tree_tokens, const int32_t *parent_idx, int32_t n, const llmcad_result *out,
                       void *stream)
{
    int rc = check_pass_args(ctx, packed, kv_cache, prefix_len, tree_tokens, parent_idx, n);
    if (rc != LLMCAD_OK) return rc;
    if (out == nullptr || out->argmax == nullptr || out->accepted_path == nullptr || out->scalars == nullptr)
        return LLMCAD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const llmcad_config &c = ctx->cfg;
    int32_t *status = out->scalars + LLMCAD_S_STATUS;
    float *logits = out->logits != nullptr ? out->logits : ctx->logits;
    CUDA_TRY(cudaMemsetAsync(out->scalars, 0, 8 * sizeof(int32_t), st));
    if ((rc = run_forward(ctx, packed, kv_cache, prefix_len, tree_tokens, parent_idx, n, logits, status, st)) != LLMCAD_OK)
        return rc;
    CUDA_TRY(launch_argmax(logits, n, c.vocab, out->argmax, status, st));
    CUDA_TRY(launch_accept(parent_idx, tree_tokens, out->argmax, n, prefix_len, out->accepted_path, out->scalars, st));
    CUDA_TRY(launch_compact(kv_cache, c.dtype, c.n_layers, c.n_heads, c.max_seq, c.head_dim, prefix_len,
                            out->accepted_path, out->scalars, st));
    ctx->launches += 3;
    return LLMCAD_OK;
}

int llmcad_verify_tree_host(llmcad_ctx *ctx, const void *packed, void *kv_cache, int32_t prefix_len,
                            const int32_t *tree_tokens, const int32_t *parent_idx, int32_t n,
                            const llmcad_host_result *out, void *stream)
{
    int rc = check_pass_args(ctx, packed, kv_cache, prefix_len, tree_tokens, parent_idx, n);
    if (rc != LLMCAD_OK) return rc;
    if (out == nullptr || out->argmax == nullptr || out->accepted_path == nullptr || out->scalars == nullptr)
        return LLMCAD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CUDA_TRY(cudaMemcpyAsync(ctx->tokens_dev(), tree_tokens, n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(ctx->parent_dev(), parent_idx, n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    llmcad_result dev{};
    dev.logits = out->logits != nullptr ? ctx->logits : nullptr;
    dev.argmax = ctx->argmax_dev();
    dev.accepted_path = ctx->path_dev();
    dev.scalars = ctx->scalars_dev();
    rc = llmcad_verify_tree(ctx, packed, kv_cache, prefix_len, ctx->tokens_dev(), ctx->parent_dev(), n, &dev, stream);
    if (rc != LLMCAD_OK) return rc;
    // argmax[128], path[128] and scalars[8] are contiguous in the context's integer buffer
    CUDA_TRY(cudaMemcpyAsync(out->argmax, ctx->argmax_dev(), n * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaMemcpyAsync(out->accepted_path, ctx->path_dev(), n * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaMemcpyAsync(out->scalars, ctx->scalars_dev(), 8 * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    if (out->logits != nullptr)
        CUDA_TRY(cudaMemcpyAsync(out->logits, ctx->logits, (size_t)n * ctx->cfg.vocab * sizeof(float), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    return LLMCAD_OK;
}

int llmcad_prefill(llmcad_ctx *ctx, const void *packed, void *kv_cache, int32_t prefix_len, const int32_t *tokens,
                   int32_t n, float *last_logits, void *stream)
{
    if (ctx == nullptr || packed == nullptr || kv_cache == nullptr || tokens == nullptr) return LLMCAD_ERR_INVALID_ARG;
    if (n < 1 || prefix_len < 0) return LLMCAD_ERR_INVALID_ARG;
    if ((long long)prefix_len + n > ctx->cfg.max_seq) return LLMCAD_ERR_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t *status = ctx->scalars_dev() + LLMCAD_S_STATUS;
    CUDA_TRY(cudaMemsetAsync(ctx->scalars_dev(), 0, 8 * sizeof(int32_t), st));
    const int chunk = ctx->cfg.max_tree;
    for (int done = 0; done < n; done += chunk) {
        const int m = n - done < chunk ? n - done : chunk;
        const bool last = done + m == n;
        // a chain whose "prefix" is everything before it; every node is committed, nothing to roll back
        int rc = run_forward(ctx, packed, kv_cache, prefix_len + done, tokens + done, ctx->chain_dev(), m,
                             (last && last_logits != nullptr) ? ctx->logits : nullptr, status, st);
        if (rc != LLMCAD_OK) return rc;
        if (last && last_logits != nullptr)
            CUDA_TRY(cudaMemcpyAsync(last_logits, ctx->logits + (size_t)(m - 1) * ctx->cfg.vocab,
                                     (size_t)ctx->cfg.vocab * sizeof(float), cudaMemcpyDeviceToDevice, st));
    }
    return LLMCAD_OK;
}

int llmcad_extend_tree(llmcad_ctx *ctx, const void *packed, void *kv_cache, int32_t prefix_len, const int32_t *tree_tokens,
                       const int32_t *parent_idx, int32_t n_old, int32_t n_tree, int32_t top_k, float *logits,
                       int32_t *topk_ids, float *topk_probs, int32_t *status, void *stream)
{
    int rc = check_pass_args(ctx, packed, kv_cache, prefix_len, tree_tokens, parent_idx, n_tree);
    if (rc != LLMCAD_OK) return rc;
    if (status == nullptr || n_old < 0 || n_old >= n_tree || top_k < 0 || top_k > LLMCAD_MAX_TOPK) return LLMCAD_ERR_INVALID_ARG;
    if (top_k > 0 && (topk_ids == nullptr || topk_probs == nullptr)) return LLMCAD_ERR_INVALID_ARG;
    if (top_k > ctx->cfg.vocab) return LLMCAD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float *lg = logits != nullptr ? logits : ctx->logits;
    CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
    if ((rc = run_forward(ctx, packed, kv_cache, prefix_len, tree_tokens, parent_idx, n_tree, lg, status, st, n_old)) != LLMCAD_OK)
        return rc;
    if (top_k > 0) {
        CUDA_TRY(launch_topk_softmax(lg, n_tree - n_old, ctx->cfg.vocab, top_k, topk_ids, topk_probs, status, st));
        ctx->launches++;
    }
    return LLMCAD_OK;
}

int llmcad_tree_prep(const int32_t *parent_idx, int32_t n, int32_t prefix_len, int32_t *depth, int32_t *pos,
                     uint32_t *anc, int32_t *status, void *stream)
{
    if (!parent_idx || !depth || !pos || !anc || !status) return LLMCAD_ERR_INVALID_ARG;
    if (n < 1 || prefix_len < 0) return LLMCAD_ERR_INVALID_ARG;
    if (n > LLMCAD_MAX_TREE) return LLMCAD_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
    TreeBuffers tb{depth, pos, anc, nullptr};
    CUDA_TRY(launch_tree_prep(parent_idx, nullptr, n, prefix_len, 0, 0, 0.f, tb, status, st));
    return LLMCAD_OK;
}

int llmcad_accept_compact(llmcad_ctx *ctx, void *kv_cache, int32_t prefix_len, const int32_t *tree_tokens,
                          const int32_t *parent_idx, const int32_t *argmax, int32_t n, int32_t *accepted_path,
                          int32_t *scalars, void *stream)
{
    if (!ctx || !tree_tokens || !parent_idx || !argmax || !accepted_path || !scalars) return LLMCAD_ERR_INVALID_ARG;
    if (n < 1 || prefix_len < 0) return LLMCAD_ERR_INVALID_ARG;
    if (n > ctx->cfg.max_tree) return LLMCAD_ERR_UNSUPPORTED;
    if ((long long)prefix_len + n > ctx->cfg.max_seq) return LLMCAD_ERR_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const llmcad_config &c = ctx->cfg;
    CUDA_TRY(cudaMemsetAsync(scalars, 0, 8 * sizeof(int32_t), st));
    // the search trusts the tree: validate it first (a malformed tree lands in scalars[status])
    CUDA_TRY(launch_tree_prep(parent_idx, tree_tokens, n, prefix_len, c.vocab, c.head_dim, c.rope_base, ctx->tb,
                              scalars + LLMCAD_S_STATUS, st));
    CUDA_TRY(launch_accept(parent_idx, tree_tokens, argmax, n, prefix_len, accepted_path, scalars, st));
    ctx->launches += 2;
    if (kv_cache != nullptr) {
        CUDA_TRY(launch_compact(kv_cache, c.dtype, c.n_layers, c.n_heads, c.max_seq, c.head_dim, prefix_len, accepted_path,
                                scalars, st));
        ctx->launches++;
    }
    return LLMCAD_OK;
}

int llmcad_tree_attention(llmcad_ctx *ctx, const void *q, const void *k, const void *v, int32_t kv_stride,
                          int32_t prefix_len, const int32_t *parent_idx, int32_t n, void *o, void *stream)
{
    if (!ctx || !q || !k || !v || !parent_idx || !o) return LLMCAD_ERR_INVALID_ARG;
    if (n < 1 || prefix_len < 0 || kv_stride < prefix_len + n) return LLMCAD_ERR_INVALID_ARG;
    if (n > ctx->cfg.max_tree) return LLMCAD_ERR_UNSUPPORTED;
    // the tensor-core kernels move rows as 16-byte vectors and bulk copies
    if (ctx->tc_attn && ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) |
                          reinterpret_cast<uintptr_t>(o)) & 15) != 0)
        return LLMCAD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t *status = ctx->scalars_dev() + LLMCAD_S_STATUS;
    CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
    TreeBuffers tb = ctx->tb;
    tb.rope_cs = nullptr;
    CUDA_TRY(launch_tree_prep(parent_idx, nullptr, n, prefix_len, 0, 0, 0.f, tb, status, st));
    ctx->launches++;
    return run_attention(ctx, q, k, v, kv_stride, prefix_len, n, o, false, status, st);
}

int llmcad_skinny_gemm(llmcad_ctx *ctx, const void *w, const void *x, float *y, int32_t n_out, int32_t n_in, int32_t n,
                       void *stream)
{
    if (!ctx || !w || !x || !y) return LLMCAD_ERR_INVALID_ARG;
    if (n_out < 1 || n_in < 1 || n < 1) return LLMCAD_ERR_INVALID_ARG;
    if (n > ctx->cfg.max_tree || n_in % 8) return LLMCAD_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t *status = ctx->scalars_dev() + LLMCAD_S_STATUS;
    CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
    EpiParams ep{};
    ep.mode = EPI_PLAIN; ep.n = n; ep.n_out = n_out; ep.y = y; ep.ldy = n_out;
    if (ctx->tc_gemm) {
        const int n_pad = (n + 15) / 16 * 16;
        TcGemm g;
        // rows of x beyond n are outside the tensor: the copy engine fills them with zeros
        if (!make_tensor_map_bf16(&g.maps.w, w, n_out, n_in, 128) || !make_act_map_bf16(&g.maps.x, x, n, n_in, n_pad, 1, n)) {
            snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled failed");
            return LLMCAD_ERR_CUDA;
        }
        g.p.g = make_gemm_desc(n_in, ep);
        g.p.n_pad = n_pad;
        return g.launch(ctx, status, st);
    }
    ctx->launches++;
    TimedLaunch tl(ctx, 0, st);
    CUDA_TRY(launch_gemm_simt(w, x, ctx->cfg.dtype, n_in, ep, status, st));
    return LLMCAD_OK;
}

size_t llmcad_tiled_weight_bytes(int32_t n_out, int32_t n_in)
{
    if (n_out < 1 || n_in < 1) return 0;
    return tiled_weight_bytes(n_out, n_in);
}

int llmcad_tile_weight(const void *w, int32_t n_out, int32_t n_in, void *tiled, void *stream)
{
    if (!w || !tiled) return LLMCAD_ERR_INVALID_ARG;
    if (n_out < 1 || n_in < 1) return LLMCAD_ERR_INVALID_ARG;
    if (n_in % 8) return LLMCAD_ERR_UNSUPPORTED;
    CUDA_TRY(launch_tile_weight(w, n_out, n_in, tiled, static_cast<cudaStream_t>(stream)));
    return LLMCAD_OK;
}

int llmcad_skinny_gemm_tiled(llmcad_ctx *ctx, const void *w_tiled, const void *x, float *y, int32_t n_out, int32_t n_in,
                             int32_t n, void *stream)
{
    if (!ctx || !w_tiled || !x || !y) return LLMCAD_ERR_INVALID_ARG;
    if (n_out < 1 || n_in < 1 || n < 1) return LLMCAD_ERR_INVALID_ARG;
    if (n > ctx->cfg.max_tree || n_in % 8 || !ctx->tc_gemm) return LLMCAD_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t *status = ctx->scalars_dev() + LLMCAD_S_STATUS;
    CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
    EpiParams ep{};
    ep.mode = EPI_PLAIN; ep.n = n; ep.n_out = n_out; ep.y = y; ep.ldy = n_out;
    const int n_pad = (n + 15) / 16 * 16;
    TcGemm g;
    if (!make_act_map_bf16(&g.maps.x, x, n, n_in, n_pad, 1, n)) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled failed");
        return LLMCAD_ERR_CUDA;
    }
    g.p.g = make_gemm_desc(n_in, ep, w_tiled);
    g.p.n_pad = n_pad;
    return g.launch(ctx, status, st);
}

int llmcad_quantize_int4(const void *w, int32_t n_out, int32_t n_in, int8_t *q, int8_t *e, void *stream)
{
    if (!w || !q || !e) return LLMCAD_ERR_INVALID_ARG;
    if (n_out < 1 || n_in < 1) return LLMCAD_ERR_INVALID_ARG;
    if (n_in % 64) return LLMCAD_ERR_UNSUPPORTED;
    CUDA_TRY(launch_quantize_int4_plain(w, n_out, n_in, q, e, static_cast<cudaStream_t>(stream)));
    return LLMCAD_OK;
}

size_t llmcad_tiled_weight_int4_bytes(int32_t n_out, int32_t n_in)
{
    if (n_out < 1 || n_in < 1 || n_in % 64) return 0;
    return tiled_weight_int4_bytes(n_out, n_in);
}

int llmcad_tile_weight_int4(const void *w, int32_t n_out, int32_t n_in, void *tiled, void *stream)
{
    if (!w || !tiled) return LLMCAD_ERR_INVALID_ARG;
    if (n_out < 1 || n_in < 1) return LLMCAD_ERR_INVALID_ARG;
    if (n_in % 64) return LLMCAD_ERR_UNSUPPORTED;
    CUDA_TRY(launch_tile_weight_int4(w, n_out, n_in, tiled, static_cast<cudaStream_t>(stream)));
    return LLMCAD_OK;
}

int llmcad_skinny_gemm_tiled_int4(llmcad_ctx *ctx, const void *w_tiled, const void *x, float *y, int32_t n_out, int32_t n_in,
                                  int32_t n, void *stream)
{
    if (!ctx || !w_tiled || !x || !y) return LLMCAD_ERR_INVALID_ARG;
    if (n_out < 1 || n_in < 1 || n < 1) return LLMCAD_ERR_INVALID_ARG;
    if (n > ctx->cfg.max_tree || n_in % 64 || !ctx->tc_gemm) return LLMCAD_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t *status = ctx->scalars_dev() + LLMCAD_S_STATUS;
    CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
    EpiParams ep{};
    ep.mode = EPI_PLAIN; ep.n = n; ep.n_out = n_out; ep.y = y; ep.ldy = n_out;
    const int n_pad = (n + 15) / 16 * 16;
    TcGemm g;
    if (!make_act_map_bf16(&g.maps.x, x, n, n_in, n_pad, 1, n)) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "cuTensorMapEncodeTiled failed");
        return LLMCAD_ERR_CUDA;
    }
    g.p.g = make_gemm_desc(n_in, ep, w_tiled, true);
    g.p.n_pad = n_pad;
    return g.launch(ctx, status, st);
}

int llmcad_set_kernel_timing(llmcad_ctx *ctx, int32_t enable)
{
    if (ctx == nullptr) return LLMCAD_ERR_INVALID_ARG;
    ctx->timing = enable != 0;
    return LLMCAD_OK;
}

int llmcad_get_kernel_timing(llmcad_ctx *ctx, int32_t kind, double *total_ms, int64_t *n_launches)
{
    if (ctx == nullptr || total_ms == nullptr || n_launches == nullptr) return LLMCAD_ERR_INVALID_ARG;
    double ms = 0.0;
    int64_t cnt = 0;
    std::vector<llmcad_ctx::Timed> rest;
    for (auto &t : ctx->timed) {
        if (t.kind != kind) { rest.push_back(t); continue; }
        CUDA_TRY(cudaEventSynchronize(t.b));
        float f = 0.f;
        CUDA_TRY(cudaEventElapsedTime(&f, t.a, t.b));
        ms += f;
        ++cnt;
        ctx->event_pool.push_back(t.a);
        ctx->event_pool.push_back(t.b);
    }
    ctx->timed.swap(rest);
    *total_ms = ms;
    *n_launches = cnt;
    return LLMCAD_OK;
}

int llmcad_set_gemm_trace(llmcad_ctx *ctx, uint64_t *trace, int32_t capacity)
{
    if (ctx == nullptr) return LLMCAD_ERR_INVALID_ARG;
    ctx->trace = reinterpret_cast<unsigned long long *>(trace);
    ctx->trace_launch = 0;
    ctx->trace_capacity = trace ? capacity : 0;
    return LLMCAD_OK;
}

int llmcad_last_status(llmcad_ctx *ctx, void *stream)
{
    if (ctx == nullptr) return LLMCAD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t v = 0;
    CUDA_TRY(cudaMemcpyAsync(&v, ctx->scalars_dev() + LLMCAD_S_STATUS, sizeof(v), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    return v;
}

int llmcad_tree_confidence(const double *branch_conf, int32_t n_branches, double *t_c)
{
    if (branch_conf == nullptr || t_c == nullptr || n_branches < 1) return LLMCAD_ERR_INVALID_ARG;
    double best = 0.0;
    for (int32_t i = 0; i < n_branches; ++i) {
        if (!(branch_conf[i] > 0.0 && branch_conf[i] <= 1.0)) return LLMCAD_ERR_INVALID_ARG;
        best = branch_conf[i] > best ? branch_conf[i] : best;
    }
    *t_c = best;
    return LLMCAD_OK;
}

int llmcad_update_threshold(double alpha, int32_t n_correct, int32_t n_all, double tree_confidence, double *alpha_next)
{
    if (alpha_next == nullptr || !(alpha > 0.0) || n_all < 0 || n_correct < 0 || n_correct > n_all) return LLMCAD_ERR_INVALID_ARG;
    if (!(tree_confidence > 0.0 && tree_confidence <= 1.0)) return LLMCAD_ERR_INVALID_ARG;
    if (n_all == 0) *alpha_next = alpha;                       // nothing was verified
    else if (n_correct == n_all) *alpha_next = 0.5 * alpha;    // no error: trust the draft model more
    else *alpha_next = alpha * exp(-log(tree_confidence) * (double)(n_all - n_correct) / (double)n_all);
    return LLMCAD_OK;
}

int llmcad_tree_branches(const int32_t *parent_idx, const double *node_conf, int32_t n, int32_t *leaf,
                         double *cum_conf, int32_t *branch_len, int32_t *n_branches)
{
    if (parent_idx == nullptr || node_conf == nullptr || leaf == nullptr || cum_conf == nullptr ||
        branch_len == nullptr || n_branches == nullptr || n < 1 || n > LLMCAD_MAX_TREE)
        return LLMCAD_ERR_INVALID_ARG;
    if (parent_idx[0] != -1) return LLMCAD_ERR_INVALID_ARG;
    bool inner[LLMCAD_MAX_TREE] = {};
    double cum[LLMCAD_MAX_TREE];
    int32_t depth[LLMCAD_MAX_TREE];
    cum[0] = 1.0;
    depth[0] = 0;
    for (int32_t i = 1; i < n; ++i) {                         // parents come first: one sweep
        const int32_t par = parent_idx[i];
        if (par < 0 || par >= i || !(node_conf[i] > 0.0 && node_conf[i] <= 1.0)) return LLMCAD_ERR_INVALID_ARG;
        inner[par] = true;
        cum[i] = cum[par] * node_conf[i];
        depth[i] = depth[par] + 1;
    }
    int32_t nb = 0;
    for (int32_t i = 0; i < n; ++i) {
        if (inner[i]) continue;
        leaf[nb] = i;
        cum_conf[nb] = cum[i];
        branch_len[nb] = depth[i];
        ++nb;
    }
    *n_branches = nb;
    return LLMCAD_OK;
}

int llmcad_branch_pacer(const double *cum_conf, const int32_t *branch_len, int32_t n_branches, double m_tokens,
                        double *f, int32_t *next_branch)
{
    if (cum_conf == nullptr || branch_len == nullptr || f == nullptr || next_branch == nullptr || n_branches < 1 ||
        !(m_tokens >= 0.0))
        return LLMCAD_ERR_INVALID_ARG;
    double total = 0.0;
    for (int32_t i = 0; i < n_branches; ++i) {
        if (!(cum_conf[i] > 0.0 && cum_conf[i] <= 1.0) || branch_len[i] < 0) return LLMCAD_ERR_INVALID_ARG;
        total += cum_conf[i];
    }
    int32_t best = 0;
    for (int32_t x = 0; x < n_branches; ++x) {
        f[x] = m_tokens * (cum_conf[x] / total) - (double)branch_len[x];
        if (f[x] > f[best]) best = x;
    }
    *next_branch = best;
    return LLMCAD_OK;
}

int64_t llmcad_launch_count(const llmcad_ctx *ctx) { return ctx ? ctx->launches : 0; }

int llmcad_set_wait_limit_ns(llmcad_ctx *ctx, uint64_t ns)
{
    if (ctx == nullptr) return LLMCAD_ERR_INVALID_ARG;
    ctx->wait_limit_ns = ns ? ns : kDefaultWaitLimitNs;
    return LLMCAD_OK;
}

int llmcad_selftest_wait_timeout(llmcad_ctx *ctx, void *stream)
{
    if (ctx == nullptr) return LLMCAD_ERR_INVALID_ARG;
    if (!ctx->tc_gemm || ctx->cfg.vocab < 160) return LLMCAD_ERR_UNSUPPORTED;
    if (ctx->wait_limit_ns > 100000000ull) return LLMCAD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t *status = ctx->scalars_dev() + LLMCAD_S_STATUS;
    CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
    const int n_pad = 16;
    int rc = ensure_act_maps(ctx, n_pad);
    if (rc != LLMCAD_OK) return rc;
    // A 256 x 128 GEMM on 16 nodes. Weights: the first 64 KB of the context's logits buffer read as
    // four pre-swizzled tiles (any bit pattern will do); input: the normalised activations; output:
    // plain fp32 rows further up in the same buffer.
    EpiParams ep{};
    ep.mode = EPI_PLAIN; ep.n = n_pad; ep.n_out = 256; ep.ldy = 256;
    ep.y = ctx->logits + (64 * 1024) / sizeof(float);
    TcGemm g;
    g.maps.x = ctx->act_maps[n_pad / 16][0];
    g.p.g = make_gemm_desc(128, ep, ctx->logits);
    g.p.n_pad = n_pad;
    g.p.comp = ctx->comp ? 1 : 0;
    // the activation copies are withheld: the ring stages never fill, and every role of the streaming
    // kernel runs into the wait limit
    g.p.withhold_act = 1;
    rc = g.launch(ctx, status, st);
    if (rc != LLMCAD_OK) return rc;
    int32_t v = 0;
    CUDA_TRY(cudaMemcpyAsync(&v, status, sizeof(v), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(cudaStreamSynchronize(st));
    return v;
}

}  // extern "C"
