/*
 * CPU oracle for token-tree verification by a LLaMA-style target model.
 *
 * THIS IS TEST INFRASTRUCTURE. It is a plain, slow, obviously-correct statement
 * of what the verification pass computes, used only by the tests, the smoke
 * check and the benchmark's cpu_baseline leg. The product path never calls it
 * and shares no code, header, table or constant with it.
 *
 * Arithmetic: weights are read as fp32 (bf16 weights are widened exactly by the
 * caller); every activation, accumulator, softmax and angle is fp64.
 *
 * What it follows (paper: LLMCad, arXiv 2309.04255):
 *   - tree decoder mask table, Sec. 3.2 "Tree decoder": a query takes into
 *     account only the earlier positions of its own branch;
 *   - non-autoregressive verification, Sec. 3.2 "Token tree verification and
 *     rectification": the target examines all draft tokens in one pass and the
 *     result equals examining them sequentially;
 *   - depth-first verified-sequence search and rollback/rectify, same section.
 * The decoder itself (pre-norm RMSNorm, rotary positions on interleaved pairs,
 * SwiGLU, no biases) is the LLaMA shape the benchmark configs name; the paper
 * only says "decoder layers with masked self-attention, LayerNorm, Linear"
 * (Sec. 2.1). Those conventions are pinned by the tests against a library
 * implementation of the LLaMA decoder.
 *
 * Pins (tests/test_oracle_pins.py): mask example of Sec. 3.2, acceptance example
 * of Fig. 7's text, chain tree == sequential decoding (oracle/sequential.c),
 * every node == its root-to-node path run as a sequence through a library
 * decoder, acceptance == sequential greedy check, closed forms of each step.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
    double rms_eps, rope_base;
} orc_config;

enum { ORC_OK = 0, ORC_BAD_TREE = 1, ORC_BAD_TOKEN = 2 };

/* Sec. 3.2 "Tree decoder": mask table. anc[i*n+j] = 1 iff node j is node i
 * itself or one of its ancestors (the "previous positions on the same branch").
 * Node i sits at sequence position prefix_len + depth[i]. */
int orc_tree_prep(const int *parent_idx, int n, int prefix_len, int *depth, int *pos, unsigned char *anc)
{
    if (n < 1 || parent_idx[0] != -1) return ORC_BAD_TREE;
    for (int i = 1; i < n; ++i)
        if (parent_idx[i] < 0 || parent_idx[i] >= i) return ORC_BAD_TREE;
    memset(anc, 0, (size_t)n * n);
    for (int i = 0; i < n; ++i) {
        int p = parent_idx[i];
        depth[i] = (p < 0) ? 0 : depth[p] + 1;
        pos[i] = prefix_len + depth[i];
        if (p >= 0)
            for (int j = 0; j < n; ++j) anc[(size_t)i * n + j] = anc[(size_t)p * n + j];
        anc[(size_t)i * n + i] = 1;
    }
    return ORC_OK;
}

/* x[i] = E[token_i] */
int orc_embed(const orc_config *c, const float *E, const int *tokens, int n, double *x)
{
    for (int i = 0; i < n; ++i) {
        if (tokens[i] < 0 || tokens[i] >= c->vocab) return ORC_BAD_TOKEN;
        for (int k = 0; k < c->d_model; ++k) x[(size_t)i * c->d_model + k] = E[(size_t)tokens[i] * c->d_model + k];
    }
    return ORC_OK;
}

/* out[i] = x[i] / sqrt(mean(x[i]^2) + eps) * g */
void orc_rmsnorm(const double *x, const float *g, int n, int d, double eps, double *out)
{
    for (int i = 0; i < n; ++i) {
        double ss = 0.0;
        for (int k = 0; k < d; ++k) ss += x[(size_t)i * d + k] * x[(size_t)i * d + k];
        double r = 1.0 / sqrt(ss / d + eps);
        for (int k = 0; k < d; ++k) out[(size_t)i * d + k] = x[(size_t)i * d + k] * r * g[k];
    }
}

/* y[i][o] = sum_k W[o][k] x[i][k]; W row-major [n_out][n_in] */
void orc_linear(const float *W, int n_out, int n_in, const double *x, int n, double *y)
{
#pragma omp parallel for schedule(static)
    for (int o = 0; o < n_out; ++o) {
        const float *w = W + (size_t)o * n_in;
        for (int i = 0; i < n; ++i) {
            const double *xi = x + (size_t)i * n_in;
            double acc = 0.0;
            for (int k = 0; k < n_in; ++k) acc += (double)w[k] * xi[k];
            y[(size_t)i * n_out + o] = acc;
        }
    }
}

/* Rotary position embedding on interleaved pairs (v[2t], v[2t+1]) of every head:
 * angle = pos * base^(-2t/hd). */
void orc_rope(double *v, const int *pos, int n, int n_heads, int hd, double base)
{
    for (int i = 0; i < n; ++i)
        for (int h = 0; h < n_heads; ++h)
            for (int t = 0; t < hd / 2; ++t) {
                double ang = (double)pos[i] * pow(base, -2.0 * t / hd);
                double cs = cos(ang), sn = sin(ang);
                double *p = v + ((size_t)i * n_heads + h) * hd + 2 * t;
                double a = p[0], b = p[1];
                p[0] = a * cs - b * sn;
                p[1] = a * sn + b * cs;
            }
}

/* Tree-masked attention. Node i, head h: softmax over every prefix slot and over
 * the tree nodes j with anc[i][j] of q.k / sqrt(hd), then the same weights on V.
 * pk, pv: [H][P][hd] prefix rows; tk, tv, q, o: [n][H*hd]. Masked keys take no
 * part at all (weight exactly 0). */
void orc_tree_attention(const double *q, const double *pk, const double *pv, int P,
                        const double *tk, const double *tv, const unsigned char *anc,
                        int n, int n_heads, int hd, double *o)
{
    const int d = n_heads * hd;
    const double scale = 1.0 / sqrt((double)hd);
#pragma omp parallel for collapse(2) schedule(static)
    for (int i = 0; i < n; ++i)
        for (int h = 0; h < n_heads; ++h) {
            const double *qi = q + (size_t)i * d + (size_t)h * hd;
            double *s = (double *)malloc(sizeof(double) * (size_t)(P + n));
            double mx = -INFINITY;
            for (int t = 0; t < P; ++t) {
                const double *k = pk + ((size_t)h * P + t) * hd;
                double acc = 0.0;
                for (int e = 0; e < hd; ++e) acc += qi[e] * k[e];
                s[t] = acc * scale;
                if (s[t] > mx) mx = s[t];
            }
            for (int j = 0; j < n; ++j) {
                if (!anc[(size_t)i * n + j]) { s[P + j] = -INFINITY; continue; }
                const double *k = tk + (size_t)j * d + (size_t)h * hd;
                double acc = 0.0;
                for (int e = 0; e < hd; ++e) acc += qi[e] * k[e];
                s[P + j] = acc * scale;
                if (s[P + j] > mx) mx = s[P + j];
            }
            double den = 0.0;
            for (int t = 0; t < P + n; ++t) {
                s[t] = (s[t] == -INFINITY) ? 0.0 : exp(s[t] - mx);
                den += s[t];
            }
            double *oi = o + (size_t)i * d + (size_t)h * hd;
            for (int e = 0; e < hd; ++e) oi[e] = 0.0;
            for (int t = 0; t < P; ++t) {
                const double *v = pv + ((size_t)h * P + t) * hd;
                double w = s[t] / den;
                for (int e = 0; e < hd; ++e) oi[e] += w * v[e];
            }
            for (int j = 0; j < n; ++j) {
                if (s[P + j] == 0.0) continue;
                const double *v = tv + (size_t)j * d + (size_t)h * hd;
                double w = s[P + j] / den;
                for (int e = 0; e < hd; ++e) oi[e] += w * v[e];
            }
            free(s);
        }
}

/* One decoder layer over all tree nodes. x [n][d] is updated in place; tree_k and
 * tree_v [n][d] receive this layer's (rotated) keys and values of the tree nodes. */
void orc_layer(const orc_config *c,
               const float *attn_norm, const float *wq, const float *wk, const float *wv, const float *wo,
               const float *ffn_norm, const float *w_gate, const float *w_up, const float *w_down,
               const double *prefix_k, const double *prefix_v, int P,
               const int *pos, const unsigned char *anc, int n,
               double *x, double *tree_k, double *tree_v)
{
    const int d = c->d_model, f = c->d_ffn;
    double *xn = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *q = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *att = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *tmp = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *g = (double *)malloc(sizeof(double) * (size_t)n * f);
    double *u = (double *)malloc(sizeof(double) * (size_t)n * f);

    orc_rmsnorm(x, attn_norm, n, d, c->rms_eps, xn);
    orc_linear(wq, d, d, xn, n, q);
    orc_linear(wk, d, d, xn, n, tree_k);
    orc_linear(wv, d, d, xn, n, tree_v);
    orc_rope(q, pos, n, c->n_heads, c->head_dim, c->rope_base);
    orc_rope(tree_k, pos, n, c->n_heads, c->head_dim, c->rope_base);
    orc_tree_attention(q, prefix_k, prefix_v, P, tree_k, tree_v, anc, n, c->n_heads, c->head_dim, att);
    orc_linear(wo, d, d, att, n, tmp);
    for (size_t t = 0; t < (size_t)n * d; ++t) x[t] += tmp[t];

    orc_rmsnorm(x, ffn_norm, n, d, c->rms_eps, xn);
    orc_linear(w_gate, f, d, xn, n, g);
    orc_linear(w_up, f, d, xn, n, u);
    for (size_t t = 0; t < (size_t)n * f; ++t) g[t] = g[t] / (1.0 + exp(-g[t])) * u[t];
    orc_linear(w_down, d, f, g, n, tmp);
    for (size_t t = 0; t < (size_t)n * d; ++t) x[t] += tmp[t];

    free(xn); free(q); free(att); free(tmp); free(g); free(u);
}

/* logits[i] = rmsnorm(x[i]) W_lm^T */
void orc_head(const orc_config *c, const float *final_norm, const float *lm_head, const double *x, int n, double *logits)
{
    double *xn = (double *)malloc(sizeof(double) * (size_t)n * c->d_model);
    orc_rmsnorm(x, final_norm, n, c->d_model, c->rms_eps, xn);
    orc_linear(lm_head, c->vocab, c->d_model, xn, n, logits);
    free(xn);
}

/* greedy choice of the target at each node: lowest index of the maximum */
void orc_argmax(const double *logits, int n, int vocab, int *out)
{
    for (int i = 0; i < n; ++i) {
        int best = 0;
        for (int t = 1; t < vocab; ++t)
            if (logits[(size_t)i * vocab + t] > logits[(size_t)i * vocab + best]) best = t;
        out[i] = best;
    }
}

/* Depth-first verified-sequence search (Sec. 3.2). A child is correct when its
 * draft token equals the target's output at its parent; the correct token tree is
 * what remains reachable from the root through correct children; the verified
 * sequence is its longest root-to-node path (ties: lowest node index). The
 * target's output at the last verified node is the next token: the rectified token
 * when that node had draft children (all of them wrong), a free extra token
 * otherwise.
 * result[0..5] = accepted_len, next_token, n_correct, n_all, rectified, (unused). */
typedef struct { const int *parent, *tok, *amax; int n; int *first_child, *next_sib, *depth; int best, best_depth; } dfs_t;

static void dfs_visit(dfs_t *s, int u, int du)
{
    s->depth[u] = du;
    if (du > s->best_depth || (du == s->best_depth && u < s->best)) { s->best = u; s->best_depth = du; }
    for (int c = s->first_child[u]; c >= 0; c = s->next_sib[c])
        if (s->tok[c] == s->amax[u]) dfs_visit(s, c, du + 1);
}

static int deepest_below(const int *first_child, const int *next_sib, int u)
{
    int best = 0;
    for (int c = first_child[u]; c >= 0; c = next_sib[c]) {
        int h = 1 + deepest_below(first_child, next_sib, c);
        if (h > best) best = h;
    }
    return best;
}

void orc_accept(const int *parent_idx, const int *tokens, const int *argmax, int n, int *path, int *result)
{
    int *first_child = (int *)malloc(sizeof(int) * n), *next_sib = (int *)malloc(sizeof(int) * n);
    int *depth = (int *)malloc(sizeof(int) * n);
    for (int i = 0; i < n; ++i) first_child[i] = next_sib[i] = -1;
    for (int i = n - 1; i >= 1; --i) { /* prepend in reverse so lists are in index order */
        next_sib[i] = first_child[parent_idx[i]];
        first_child[parent_idx[i]] = i;
    }
    dfs_t s = { parent_idx, tokens, argmax, n, first_child, next_sib, depth, 0, -1 };
    dfs_visit(&s, 0, 0);
    int len = s.best_depth + 1;
    for (int u = s.best, j = len - 1; j >= 0; --j, u = parent_idx[u]) path[j] = u;
    result[0] = len;
    result[1] = argmax[s.best];
    result[2] = len - 1;
    result[3] = s.best_depth + deepest_below(first_child, next_sib, s.best);
    result[4] = first_child[s.best] >= 0;
    result[5] = 0;
    free(first_child); free(next_sib); free(depth);
}

/* Rollback (Sec. 3.2): the cache keeps the prefix rows followed by the rows of the
 * verified nodes in path order. prefix [H][P][hd], tree [n][H*hd] -> out [H][P+len][hd] */
void orc_compact(const double *prefix, const double *tree, int P, int n_heads, int hd,
                 const int *path, int len, double *out)
{
    const int d = n_heads * hd;
    for (int h = 0; h < n_heads; ++h) {
        for (int t = 0; t < P; ++t)
            memcpy(out + ((size_t)h * (P + len) + t) * hd, prefix + ((size_t)h * P + t) * hd, sizeof(double) * hd);
        for (int j = 0; j < len; ++j)
            memcpy(out + ((size_t)h * (P + len) + P + j) * hd, tree + (size_t)path[j] * d + (size_t)h * hd, sizeof(double) * hd);
    }
}

/* Fallback scalars (Sec. 3.3). Tree-cumulative confidence: the largest cumulative confidence over
 * the branches of a token tree. */
double orc_tree_confidence(const double *branch_conf, int n_branches)
{
    double t = branch_conf[0];
    for (int i = 1; i < n_branches; ++i)
        if (branch_conf[i] > t) t = branch_conf[i];
    return t;
}

/* Self-adaptive threshold, Eq. 3: after a verification with n_correct correct draft tokens out of
 * n_all on the most matching branch, alpha is halved when all were correct and otherwise divided
 * by T_c^((n_all - n_correct) / n_all). A verification without draft tokens (n_all = 0) leaves it. */
double orc_alpha_update(double alpha, int n_correct, int n_all, double t_c)
{
    if (n_all == 0) return alpha;
    if (n_correct == n_all) return alpha * 0.5;
    return alpha / pow(t_c, (double)(n_all - n_correct) / (double)n_all);
}

/* Confidences of the generating side (Sec. 3.2: a candidate whose confidence exceeds a threshold
 * opens a branch): the softmax of a node's logits, and its k largest entries in descending order
 * (ties: lower token id first). */
void orc_topk_softmax(const double *logits, int n, int vocab, int k, int *ids, double *probs)
{
    double *p = (double *)malloc(sizeof(double) * (size_t)vocab);
    for (int i = 0; i < n; ++i) {
        const double *row = logits + (size_t)i * vocab;
        double mx = row[0], sum = 0.0;
        for (int t = 1; t < vocab; ++t) if (row[t] > mx) mx = row[t];
        for (int t = 0; t < vocab; ++t) { p[t] = exp(row[t] - mx); sum += p[t]; }
        for (int t = 0; t < vocab; ++t) p[t] /= sum;
        for (int r = 0; r < k; ++r) {
            int best = -1;
            for (int t = 0; t < vocab; ++t) {
                int taken = 0;
                for (int q = 0; q < r; ++q) if (ids[(size_t)i * k + q] == t) taken = 1;
                if (!taken && (best < 0 || row[t] > row[best])) best = t;
            }
            ids[(size_t)i * k + r] = best;
            probs[(size_t)i * k + r] = p[best];
        }
    }
    free(p);
}

/* Branches of a token tree (Sec. 3.2): one per leaf, the path from the root to that leaf. For the
 * leaves in ascending node order: the leaf, the cumulative confidence of the branch (the product
 * of the confidences of its tokens) and the number of draft tokens on it. The root is the last
 * committed token, not a draft token: it counts in neither. Returns the number of branches. */
int orc_tree_branches(const int *parent, const double *node_conf, int n, int *leaf, double *cum_conf, int *branch_len)
{
    int nb = 0;
    for (int i = 0; i < n; ++i) {
        int has_child = 0;
        for (int j = i + 1; j < n; ++j)
            if (parent[j] == i) has_child = 1;
        if (has_child) continue;
        double c = 1.0;
        int len = 0;
        for (int a = i; parent[a] >= 0; a = parent[a]) {
            c *= node_conf[a];
            ++len;
        }
        leaf[nb] = i;
        cum_conf[nb] = c;
        branch_len[nb] = len;
        ++nb;
    }
    return nb;
}

/* Confidence-based branch pacer, Eq. 1-2. With N branches, M tokens to share out, branch x
 * holding T_x tokens at cumulative confidence C_x:  f(x) = M * C_x / sum_i C_i - T_x, the share
 * of the M tokens that the branch's confidence entitles it to minus what it has. Max-min fairness
 * keeps the smallest f as large as possible, so the next token goes to the branch whose f is
 * largest (every other choice lowers an f that is already smaller); ties go to the lower index.
 * Fills f[0..N) and returns that branch. */
int orc_branch_pacer(const double *cum_conf, const int *branch_len, int n_branches, double m_tokens, double *f)
{
    double total = 0.0;
    for (int i = 0; i < n_branches; ++i) total += cum_conf[i];
    int next = 0;
    for (int x = 0; x < n_branches; ++x) {
        f[x] = m_tokens * (cum_conf[x] / total) - (double)branch_len[x];
        if (f[x] > f[next]) next = x;
    }
    return next;
}

/* INT4 group quantisation of the weights (Sec. 4.1: the target model's weights are held as INT4
 * through group-wise post-training quantisation). Reading, where the paper only names the format:
 * symmetric codes q in [-8, 7], one scale per row and group of `group` consecutive input columns,
 * the scale a power of two 2^e, e the smallest integer with max|w| <= 7 * 2^e over the group (a
 * group of zeros gets e = -126), q = w / 2^e rounded to the nearest integer, halves to even.
 * Power-of-two scales make every dequantised weight q * 2^e a value bf16 holds exactly, so the
 * quantised model is an ordinary model over those weights and the rest of the oracle applies
 * unchanged. w: [rows][cols] fp32, cols a multiple of group; q: [rows][cols] int8;
 * e: [rows][cols / group] int8. */
void orc_quantize_int4(const float *w, int rows, int cols, int group, signed char *q, signed char *e)
{
    const int ng = cols / group;
    for (int r = 0; r < rows; ++r)
        for (int g = 0; g < ng; ++g) {
            const float *x = w + (size_t)r * cols + (size_t)g * group;
            double m = 0.0;
            for (int c = 0; c < group; ++c)
                if (fabs((double)x[c]) > m) m = fabs((double)x[c]);
            int ex = -126;
            if (m > 0.0) {
                ex = -126;
                while (ex < 127 && m > 7.0 * ldexp(1.0, ex)) ++ex;    /* smallest e with m <= 7 * 2^e */
            }
            e[(size_t)r * ng + g] = (signed char)ex;
            for (int c = 0; c < group; ++c) {
                double v = nearbyint(ldexp((double)x[c], -ex));   /* default rounding mode: to nearest, halves to even */
                if (v > 7.0) v = 7.0;
                if (v < -8.0) v = -8.0;
                q[(size_t)r * cols + (size_t)g * group + c] = (signed char)v;
            }
        }
}

/* The weights a quantised model computes with: w[r][c] = q[r][c] * 2^e[r][c / group]. */
void orc_dequantize_int4(const signed char *q, const signed char *e, int rows, int cols, int group, float *w)
{
    const int ng = cols / group;
    for (int r = 0; r < rows; ++r)
        for (int c = 0; c < cols; ++c)
            w[(size_t)r * cols + c] = (float)ldexp((double)q[(size_t)r * cols + c], e[(size_t)r * ng + c / group]);
}
