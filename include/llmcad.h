/*
 * llmcad.h -- C ABI of the B200 (sm_100a) token-tree verification library.
 *
 * One call of llmcad_verify_tree() is the target model's single-pass verification
 * of a draft token tree (LLMCad, arXiv 2309.04255, Sec. 3.2 "Token tree
 * verification and rectification"): a LLaMA-style decoder forward over all N tree
 * nodes at once, each node at position prefix_len + depth and attending to the
 * prefix KV cache plus its own ancestors (the mask table of Sec. 3.2 "Tree
 * decoder"), then the depth-first search for the longest verified root-to-node
 * path, then the rollback of the cache to that path.
 *
 * Conventions
 *   - Every pointer marked DEVICE is memory of the current CUDA device, owned by
 *     the caller and only borrowed for the duration of the enqueued work. Every
 *     pointer marked HOST is ordinary host memory.
 *   - `stream` arguments are a cudaStream_t passed as void*. Calls enqueue work on
 *     that stream and return without synchronising unless stated otherwise.
 *   - A context is not thread-safe and serves one stream at a time.
 *   - Return value: LLMCAD_OK or a negative host-detected error. Errors found on
 *     the device (malformed tree, token id out of range, a wait that ran out) are
 *     written to scalars[LLMCAD_S_STATUS]; all later phases of that pass then do
 *     nothing: the cache below prefix_len is untouched and new_prefix_len equals
 *     prefix_len. Kernels never trap and never wait without a limit.
 *   - There is no CPU fallback: every step below runs in CUDA kernels of this
 *     library, and every entry point fails with LLMCAD_ERR_CUDA when no device is
 *     usable.
 *
 * Model (the LLaMA shape): pre-norm residual blocks, RMSNorm, no biases, n_kv_heads
 * = n_heads, rotary position embedding on interleaved pairs (x[2t], x[2t+1]) with
 * angle pos * rope_base^(-2t/head_dim), softmax scale 1/sqrt(head_dim), SwiGLU
 * FFN, separate embedding and lm_head. Weights are row-major [out][in].
 * dtype bf16: weights and cached K/V are bf16; residual stream, accumulators,
 * softmax, norms and logits are fp32. Every activation that enters a tensor-core
 * product (GEMM inputs, queries, softmax weights, attention outputs, and within a
 * pass the tree nodes' own K/V) travels as two bf16 planes, hi = bf16(v) and
 * lo = bf16(v - hi), i.e. with 16 significant bits: plain bf16 activations do not
 * stay inside 2e-2 of the largest logit over tens of layers. The cache receives the
 * hi plane of K/V only. dtype fp32: all fp32.
 *
 * KV cache layout: [n_layers][2 (K,V)][n_heads][max_seq][head_dim] in the model
 * dtype. Slots 0..prefix_len-1 hold the prefix; during a pass the tree nodes'
 * rows sit at slots prefix_len..prefix_len+N-1; after the pass slots
 * 0..new_prefix_len-1 hold prefix + verified path, the rest is unspecified.
 */
#ifndef LLMCAD_H
#define LLMCAD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LLMCAD_MAX_TREE 128

enum {
    LLMCAD_OK = 0,
    LLMCAD_ERR_INVALID_ARG = -1, /* NULL pointer, non-positive size, N < 1 */
    LLMCAD_ERR_UNSUPPORTED = -2, /* N > max_tree or > 128, head_dim not 64/128, unknown dtype, odd sizes */
    LLMCAD_ERR_CAPACITY = -3,    /* prefix_len + N > max_seq */
    LLMCAD_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed (see llmcad_last_cuda_error) */
    /* device-detected, reported in scalars[LLMCAD_S_STATUS] */
    LLMCAD_ERR_BAD_TREE = 1,  /* parent_idx[0] != -1, or parent_idx[i] not in [0, i) */
    LLMCAD_ERR_BAD_TOKEN = 2, /* token id outside [0, vocab) */
    LLMCAD_ERR_TIMEOUT = 3,   /* a bounded device-side wait ran out */
    LLMCAD_ERR_NAN = 4,       /* a logit was NaN */
    LLMCAD_ERR_CHECK = 5      /* debug build (-DLLMCAD_CHECKS) only: a device-side bounds check failed; the access was skipped */
};

enum { LLMCAD_F32 = 0, LLMCAD_BF16 = 1 };

/* flags of llmcad_config */
enum {
    LLMCAD_FLAG_SIMT_GEMM = 1, /* use the plain-ALU GEMM even for bf16 (debugging aid) */
    LLMCAD_FLAG_SIMT_ATTN = 2, /* use the plain-ALU attention even for bf16 (debugging aid) */
    LLMCAD_FLAG_T5_ATTN = 4,   /* bf16, head_dim 128: tcgen05 attention kernel for every tree size (default: above 32 nodes) */
    LLMCAD_FLAG_MMA_ATTN = 8,  /* bf16, head_dim 128: mma.sync attention kernel for every tree size */
    LLMCAD_FLAG_INT4_WEIGHTS = 16 /* bf16 contexts: the seven matrices of every layer are held as INT4 (see llmcad_quantize_int4) */
};

/* indices into the scalars[8] output */
enum {
    LLMCAD_S_ACCEPTED_LEN = 0,   /* nodes on the verified path, root included (>= 1) */
    LLMCAD_S_NEXT_TOKEN = 1,     /* target's output at the last verified node */
    LLMCAD_S_NEW_PREFIX_LEN = 2, /* prefix_len + accepted_len */
    LLMCAD_S_N_CORRECT = 3,      /* verified draft tokens = accepted_len - 1 */
    LLMCAD_S_N_ALL = 4,          /* draft tokens on the longest branch through the last verified node */
    LLMCAD_S_RECTIFIED = 5,      /* 1 if the last verified node had draft children (all wrong) */
    LLMCAD_S_STATUS = 6,         /* 0 or a device-detected error */
    LLMCAD_S_RESERVED = 7
};

typedef struct llmcad_ctx llmcad_ctx;

typedef struct {
    int32_t n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
    int32_t max_seq;  /* cache capacity in slots */
    int32_t max_tree; /* largest N this context will see, <= LLMCAD_MAX_TREE */
    float rms_eps, rope_base;
    int32_t dtype; /* LLMCAD_F32 or LLMCAD_BF16 */
    int32_t flags;
} llmcad_config;

/* Unpacked weights of one layer, DEVICE pointers, row-major [out][in]. */
typedef struct {
    const void *attn_norm; /* [d] */
    const void *wq, *wk, *wv, *wo; /* [d][d] */
    const void *ffn_norm;  /* [d] */
    const void *w_gate, *w_up; /* [f][d] */
    const void *w_down;    /* [d][f] */
} llmcad_layer_weights;

typedef struct {
    const void *tok_embed;  /* [V][d] */
    const void *final_norm; /* [d] */
    const void *lm_head;    /* [V][d] */
} llmcad_global_weights;

/* Outputs of a pass: DEVICE pointers, caller-owned. */
typedef struct {
    float *logits;          /* [N][vocab] fp32, or NULL when not wanted */
    int32_t *argmax;        /* [N]: lowest index of each node's maximum logit */
    int32_t *accepted_path; /* [max_tree]: node indices of the verified path, root first */
    int32_t *scalars;       /* [8], see LLMCAD_S_* */
} llmcad_result;

/* The same outputs in HOST memory, for llmcad_verify_tree_host. */
typedef struct {
    float *logits;          /* [N][vocab] or NULL */
    int32_t *argmax;        /* [N] */
    int32_t *accepted_path; /* [max_tree] */
    int32_t *scalars;       /* [8] */
} llmcad_host_result;

int llmcad_version(void);
const char *llmcad_strerror(int code);
/* Text of the last CUDA error this library saw on the calling thread's context. */
const char *llmcad_last_cuda_error(void);

/* Create a context for one model shape on the current device. Allocates the
 * context's own workspaces (activations of max_tree nodes, partial tiles, attention
 * partials: a few tens of MB). Fails with LLMCAD_ERR_CUDA without a usable GPU. */
int llmcad_create(const llmcad_config *cfg, llmcad_ctx **out);
void llmcad_destroy(llmcad_ctx *ctx);

/* Bytes of the KV cache / of the packed weight buffer for this configuration.
 * The caller allocates both as DEVICE memory, 256-byte aligned (the pass refuses other pointers
 * with LLMCAD_ERR_INVALID_ARG: weight tiles travel as bulk copies, K/V rows as vector stores). */
size_t llmcad_kv_cache_bytes(const llmcad_config *cfg);
size_t llmcad_packed_weight_bytes(const llmcad_config *cfg);

/* One-time packing into the layout the kernels stream: per layer attn_norm,
 * [wq;wk;wv] as one [3d][d] matrix, wo, ffn_norm, [w_gate;w_up] as one [2f][d]
 * matrix, w_down; then tok_embed, final_norm, lm_head. In bf16 contexts every matrix
 * is stored as pre-swizzled 16 KB tiles (see llmcad_tile_weight below), in fp32
 * contexts row-major. Device-to-device work on `stream`; the sources may be freed
 * once the stream has run it.
 * llmcad_pack_layer packs layer `layer`; llmcad_pack_globals the three shared
 * tensors. All of them must have been called before the first pass. */
int llmcad_pack_layer(llmcad_ctx *ctx, int32_t layer, const llmcad_layer_weights *src /*HOST struct of DEVICE ptrs*/,
                      void *packed /*DEVICE*/, void *stream);
int llmcad_pack_globals(llmcad_ctx *ctx, const llmcad_global_weights *src, void *packed /*DEVICE*/, void *stream);

/* Sec. 3.2: one verification pass.
 *   packed       DEVICE, from the pack calls
 *   kv_cache     DEVICE, layout above; slots < prefix_len are read, slots
 *                prefix_len .. prefix_len+N-1 are written, then the verified path is
 *                moved to slots prefix_len .. new_prefix_len-1
 *   tree_tokens  DEVICE int32[N]; node 0 is the root: the last committed token whose
 *                K/V is not in the cache yet; it is always verified
 *   parent_idx   DEVICE int32[N], parent_idx[0] = -1, 0 <= parent_idx[i] < i
 *   out          HOST struct of DEVICE pointers
 * Asynchronous on `stream`. */
int llmcad_verify_tree(llmcad_ctx *ctx, const void *packed, void *kv_cache, int32_t prefix_len,
                       const int32_t *tree_tokens, const int32_t *parent_idx, int32_t n,
                       const llmcad_result *out, void *stream);

/* The same pass for callers holding HOST buffers: copies tokens and parents to the
 * device, runs the pass, copies argmax, path, scalars (and logits when out->logits
 * is not NULL) back, and synchronises `stream` before returning. The host buffers
 * should be pinned for the copies to be asynchronous; pageable memory works too. */
int llmcad_verify_tree_host(llmcad_ctx *ctx, const void *packed, void *kv_cache, int32_t prefix_len,
                            const int32_t *tree_tokens /*HOST*/, const int32_t *parent_idx /*HOST*/, int32_t n,
                            const llmcad_host_result *out, void *stream);

/* Fill cache slots prefix_len .. prefix_len+n-1 from n tokens (a chain-shaped tree
 * whose nodes are all committed): the "examine them sequentially" case of Sec. 3.2
 * run in one shot. Any n >= 1; processed in chunks of max_tree. last_logits, when
 * not NULL, receives the fp32 logits [vocab] at the last token (DEVICE). */
int llmcad_prefill(llmcad_ctx *ctx, const void *packed, void *kv_cache, int32_t prefix_len,
                   const int32_t *tokens /*DEVICE*/, int32_t n, float *last_logits /*DEVICE or NULL*/, void *stream);

/* ---- single steps of the pass, exported for parity tests and kernel benchmarks ---- */

/* Mask table of Sec. 3.2 "Tree decoder": depth[i], pos[i] = prefix_len + depth[i] and
 * the ancestor-or-self bitmask anc[i][4] (bit j of the 128-bit row i set iff node j is
 * i or an ancestor of i). status receives 0 or LLMCAD_ERR_BAD_TREE. All DEVICE. */
int llmcad_tree_prep(const int32_t *parent_idx, int32_t n, int32_t prefix_len, int32_t *depth, int32_t *pos,
                     uint32_t *anc /*[n][4]*/, int32_t *status, void *stream);

/* Depth-first verified-sequence search and rollback of Sec. 3.2 on a given argmax
 * array: writes accepted_path and scalars, and moves the verified nodes' K/V rows
 * of every layer from slot prefix_len+path[j] to slot prefix_len+j.
 * kv_cache may be NULL (search only). All DEVICE. */
int llmcad_accept_compact(llmcad_ctx *ctx, void *kv_cache, int32_t prefix_len, const int32_t *tree_tokens,
                          const int32_t *parent_idx, const int32_t *argmax, int32_t n,
                          int32_t *accepted_path, int32_t *scalars, void *stream);

/* Tree-masked attention alone (one layer), the masked self-attention of Sec. 3.2 "Tree
 * decoder": node i attends to every prefix slot and to the tree nodes whose bit is set in
 * row i of the mask table (itself and its ancestors), softmax scale 1/sqrt(hd).
 * q [n][H][hd]; k, v [H][kv_stride][hd] with the prefix at slots 0..prefix_len-1 and the
 * tree nodes at prefix_len..prefix_len+n-1; o [n][H][hd]. dtype as in llmcad_config. All
 * DEVICE; in bf16 contexts q, k, v and o must be 16-byte aligned (LLMCAD_ERR_INVALID_ARG
 * otherwise). A malformed parent_idx lands in the context's status word
 * (llmcad_last_status) and leaves o untouched. */
int llmcad_tree_attention(llmcad_ctx *ctx, const void *q, const void *k, const void *v, int32_t kv_stride,
                          int32_t prefix_len, const int32_t *parent_idx, int32_t n, void *o, void *stream);

/* Skinny GEMM alone: y[n][n_out] (fp32) = x[n][n_in] W[n_out][n_in]^T with W and x in
 * the context's dtype; the weight-streaming step of Sec. 3.2's one-shot verification
 * (parameters visited once for all n tokens). n <= max_tree. All DEVICE. */
int llmcad_skinny_gemm(llmcad_ctx *ctx, const void *w, const void *x, float *y, int32_t n_out, int32_t n_in,
                       int32_t n, void *stream);

/* For the entry points that have no scalars output (prefill, tree_attention, skinny_gemm):
 * synchronises `stream` and returns the context's own device status word of the last such
 * call: 0, a device-detected LLMCAD_ERR_* (> 0), or LLMCAD_ERR_CUDA. */
int llmcad_last_status(llmcad_ctx *ctx, void *stream);

/* The tensor-core path streams each weight matrix as a sequence of 16 KB tiles (128 rows x 64
 * columns, tile-row major then k-block, 128-byte rows with the 16-byte chunk c of row r stored
 * at position c ^ (r & 7)), so that one bulk copy moves a tile from HBM into shared memory in
 * the form the MMA reads. llmcad_pack_layer / llmcad_pack_globals produce this layout inside the
 * packed buffer; these two calls expose it for a single row-major bf16 matrix [n_out][n_in]
 * (DEVICE), n_in a multiple of 8. */
size_t llmcad_tiled_weight_bytes(int32_t n_out, int32_t n_in);
int llmcad_tile_weight(const void *w, int32_t n_out, int32_t n_in, void *tiled /*DEVICE*/, void *stream);
/* llmcad_skinny_gemm on a matrix in that layout (bf16 contexts only). */
int llmcad_skinny_gemm_tiled(llmcad_ctx *ctx, const void *w_tiled, const void *x, float *y, int32_t n_out, int32_t n_in,
                             int32_t n, void *stream);

/* INT4 weights (Sec. 4.1: the target model runs with INT4 group-quantised weights). Format of this
 * library, where the paper only names the precision: symmetric codes q in [-8, 7], one scale per row and
 * group of 64 consecutive input columns, the scale a power of two 2^e with e the smallest integer such
 * that max|w| <= 7 * 2^e over the group (-126 for a group of zeros), q = w / 2^e rounded to nearest,
 * halves to even. Every dequantised weight q * 2^e is a value bf16 holds exactly, so a pass with INT4
 * weights is the bf16 pass over the dequantised weights, bit for bit, at a quarter of the weight bytes.
 * A context created with LLMCAD_FLAG_INT4_WEIGHTS (bf16, d_model and d_ffn multiples of 64) quantises
 * the layer matrices inside llmcad_pack_layer and streams them as INT4 tiles, which the GEMM kernel
 * expands to bf16 tiles in shared memory; embedding and lm_head stay bf16.
 * llmcad_quantize_int4: codes and exponents of a row-major bf16 matrix [n_out][n_in] (DEVICE), n_in a
 * multiple of 64, as plain arrays q [n_out][n_in] and e [n_out][n_in / 64] (DEVICE int8).
 * llmcad_tile_weight_int4 / llmcad_tiled_weight_int4_bytes: the same quantisation in the layout the GEMM
 * streams (4224 bytes per tile of 128 rows and 64 columns: 128 x 8 words of eight codes, 128 exponents).
 * llmcad_skinny_gemm_tiled_int4: llmcad_skinny_gemm on a matrix in that layout (bf16 contexts only). */
int llmcad_quantize_int4(const void *w, int32_t n_out, int32_t n_in, int8_t *q, int8_t *e, void *stream);
size_t llmcad_tiled_weight_int4_bytes(int32_t n_out, int32_t n_in);
int llmcad_tile_weight_int4(const void *w, int32_t n_out, int32_t n_in, void *tiled /*DEVICE*/, void *stream);
int llmcad_skinny_gemm_tiled_int4(llmcad_ctx *ctx, const void *w_tiled, const void *x, float *y, int32_t n_out, int32_t n_in,
                                  int32_t n, void *stream);

/* Tree attention without any allocation. (The paper has no counterpart: this entry point exists
 * for the way the library is embedded, not for the method.)
 *
 * Who needs it: code that may not allocate device memory -- a plug-in loaded into a server that
 * gave the whole device to its own memory pool at start-up, or a latency-critical loop where a
 * device-synchronising cudaMalloc is not allowed. llmcad_tree_attention() needs a context, and
 * llmcad_create() allocates; this variant needs no context and calls no cudaMalloc, cudaFree or
 * other allocating routine, ever. Its scratch (per-node depth, position, ancestor bit rows, a
 * status word: 4 KB) is a static device array inside the library image; every GPU that loads the
 * library holds those 4 KB until the process exits.
 *
 * Same computation and layouts as llmcad_tree_attention, bf16, head_dim 128 only:
 * q, o [n][n_heads][128]; k, v [n_heads][kv_stride][128]; parent_idx int32[n]; all DEVICE,
 * caller-owned, q, k, v and o 16-byte aligned (LLMCAD_ERR_INVALID_ARG otherwise). status_out
 * (DEVICE int32, may be NULL) receives 0 or LLMCAD_ERR_BAD_TREE; a malformed tree leaves o untouched.
 * Limits: n <= 128 (what the static scratch holds) -- larger n is refused with
 * LLMCAD_ERR_UNSUPPORTED and a message in llmcad_noalloc_last_error(); n_heads <= 65535.
 *
 * The first call on a device looks up the device address of the static array (with that device
 * current); make that first call before starting any stream capture. All calls share the one
 * array, which keeps the previous call's contents (the status word is cleared on the stream at
 * the start of every call): two calls whose work overlaps on the GPU -- different streams
 * without ordering, or several host threads -- race on it. Calls on one stream are safe.
 * Asynchronous on `stream`. */
int llmcad_tree_attention_noalloc(const void *q, const void *k, const void *v, int32_t n_heads, int32_t kv_stride,
                                  int32_t prefix_len, const int32_t *parent_idx, int32_t n, void *o,
                                  int32_t *status_out, void *stream);
const char *llmcad_noalloc_last_error(void);

/* Tree extension: the tree decoder of Sec. 3.2 on the generating side. A token tree grows by a few
 * nodes at a time; the K/V of its first n_old nodes are already in cache slots prefix_len ..
 * prefix_len + n_old - 1 of every layer (from earlier calls of this function with the same prefix;
 * llmcad_verify_tree moves the cache, so a tree is not extended across it). The call computes the
 * decoder forward of the nodes n_old .. n_tree-1 only, each at position prefix_len + depth and
 * attending to the prefix and its own ancestors among ALL n_tree nodes (same mask table), writes
 * their K/V to slots prefix_len + n_old .. prefix_len + n_tree - 1, and returns per new node the
 * fp32 logits (logits [n_tree - n_old][vocab], optional) and the top_k most probable next tokens
 * with their softmax probabilities (topk_ids, topk_probs [n_tree - n_old][top_k], descending, ties
 * to the lower id; top_k in 0..LLMCAD_MAX_TOPK): the confidences that the branch rule (a successor
 * above a threshold opens a branch) and the cumulative branch confidences are made of. tree_tokens
 * and parent_idx describe the whole tree (n_tree entries, parent_idx[i] < i, root -1); all pointers
 * but ctx are device pointers; *status receives 0 or a device-detected error. n_old = 0 starts a
 * tree. Asynchronous on `stream`. */
#define LLMCAD_MAX_TOPK 8
int llmcad_extend_tree(llmcad_ctx *ctx, const void *packed_weights, void *kv_cache, int32_t prefix_len,
                       const int32_t *tree_tokens, const int32_t *parent_idx, int32_t n_old, int32_t n_tree, int32_t top_k,
                       float *logits, int32_t *topk_ids, float *topk_probs, int32_t *status, void *stream);

/* Host-side scalars of the fallback decision (Sec. 3.3); plain arithmetic, no device work.
 * llmcad_tree_confidence: T_c = max_i C_i over the n_branches cumulative confidences of a token
 * tree (host array, each in (0, 1]). llmcad_update_threshold: the self-adaptive threshold of
 * Eq. 3 after one verification: n_correct = scalars[LLMCAD_S_N_CORRECT], n_all =
 * scalars[LLMCAD_S_N_ALL] of that pass, tree_confidence = T_c of the verified tree;
 * *alpha_next = alpha / 2 when n_correct == n_all, else alpha / T_c^((n_all - n_correct) / n_all);
 * n_all == 0 (a tree of the root alone) leaves alpha unchanged. LLMCAD_ERR_INVALID_ARG for null
 * pointers, n_branches < 1, alpha <= 0, n_correct outside [0, n_all] or a confidence outside (0, 1]. */
int llmcad_tree_confidence(const double *branch_conf, int32_t n_branches, double *t_c);
int llmcad_update_threshold(double alpha, int32_t n_correct, int32_t n_all, double tree_confidence, double *alpha_next);

/* Host-side scalars of the confidence-based branch pacer (Sec. 3.2, Eq. 1-2); plain arithmetic, no
 * device work, all pointers host pointers.
 * llmcad_tree_branches: the branches of a token tree, one per leaf (root-to-leaf paths), leaves in
 * ascending node order. parent_idx[n] as for llmcad_verify_tree (parent_idx[0] = -1,
 * parent_idx[i] < i); node_conf[n] = the confidence with which the generating model proposed each
 * node's token, in (0, 1] (entry 0, the root, is the last committed token and is ignored). Outputs,
 * each with room for n entries: leaf[b] = node index of the branch's leaf, cum_conf[b] = product
 * of the confidences of the branch's draft tokens (1 for a tree of the root alone), branch_len[b] =
 * number of draft tokens on it (the leaf's depth); *n_branches = number of entries written.
 * llmcad_branch_pacer: f[x] = m_tokens * cum_conf[x] / sum_i cum_conf[i] - branch_len[x] for each
 * of the n_branches branches (Eq. 1): the share of m_tokens tokens that the branch's confidence
 * entitles it to, minus the tokens it holds. *next_branch = the branch with the largest f, the
 * lower index on ties: giving the next token to any other branch would lower an f that is already
 * smaller, so this choice keeps min_x f(x) (Eq. 2) as large as possible (max-min fairness).
 * LLMCAD_ERR_INVALID_ARG for null pointers, n < 1 or n > LLMCAD_MAX_TREE, an invalid parent_idx,
 * n_branches < 1, a negative length or m_tokens, or a confidence outside (0, 1]. */
int llmcad_tree_branches(const int32_t *parent_idx, const double *node_conf, int32_t n, int32_t *leaf,
                         double *cum_conf, int32_t *branch_len, int32_t *n_branches);
int llmcad_branch_pacer(const double *cum_conf, const int32_t *branch_len, int32_t n_branches, double m_tokens,
                        double *f, int32_t *next_branch);

#ifdef __cplusplus
}
#endif
#endif /* LLMCAD_H */
