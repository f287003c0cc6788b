/*
 * Ordinary autoregressive decoding, one token per step, with an ordinary causal
 * KV cache. TEST INFRASTRUCTURE: this is the "examining them sequentially" side of
 * the paper's statement that one-shot verification gives the same result as
 * sequential verification (Sec. 3.2, "Token tree verification and
 * rectification"). It is written separately from oracle.c (own loops, own cache
 * layout, no shared helper) so that a chain-shaped tree run through the tree
 * oracle can be checked against it step by step, and so that it can itself be
 * checked against a library LLaMA decoder.
 *
 * Cache layout: kc, vc [n_layers][max_seq][d_model] fp64; the token consumed at
 * step t is written at row t and attends to rows 0..t.
 */
#include <math.h>
#include <stdlib.h>

typedef struct {
    int n_layers, d_model, n_heads, head_dim, d_ffn, vocab;
    double rms_eps, rope_base;
} seq_config;

typedef struct {
    const float *attn_norm, *wq, *wk, *wv, *wo, *ffn_norm, *w_gate, *w_up, *w_down;
} seq_layer;

static void matvec(const float *W, int n_out, int n_in, const double *x, double *y)
{
#pragma omp parallel for schedule(static)
    for (int o = 0; o < n_out; ++o) {
        double acc = 0.0;
        for (int k = 0; k < n_in; ++k) acc += (double)W[(size_t)o * n_in + k] * x[k];
        y[o] = acc;
    }
}

static void norm(const double *x, const float *g, int d, double eps, double *y)
{
    double ss = 0.0;
    for (int k = 0; k < d; ++k) ss += x[k] * x[k];
    double r = 1.0 / sqrt(ss / d + eps);
    for (int k = 0; k < d; ++k) y[k] = g[k] * (x[k] * r);
}

static void rotate(double *v, int t, int n_heads, int hd, double base)
{
    for (int h = 0; h < n_heads; ++h)
        for (int p = 0; p < hd; p += 2) {
            double freq = 1.0 / pow(base, (double)p / hd);
            double c = cos(t * freq), s = sin(t * freq);
            double re = v[h * hd + p], im = v[h * hd + p + 1];
            v[h * hd + p] = re * c - im * s;
            v[h * hd + p + 1] = re * s + im * c;
        }
}

/* Consume `token` at position t (rows 0..t-1 of the cache are already filled),
 * write row t of every layer's cache, return logits[vocab]. */
int seq_decode_step(const seq_config *c, const float *tok_embed, const seq_layer *layers,
                    const float *final_norm, const float *lm_head,
                    double *kc, double *vc, int max_seq, int t, int token, double *logits)
{
    const int d = c->d_model, f = c->d_ffn, hd = c->head_dim, H = c->n_heads;
    if (token < 0 || token >= c->vocab || t < 0 || t >= max_seq) return 1;
    double *x = (double *)malloc(sizeof(double) * d), *xn = (double *)malloc(sizeof(double) * d);
    double *q = (double *)malloc(sizeof(double) * d), *a = (double *)malloc(sizeof(double) * d);
    double *r = (double *)malloc(sizeof(double) * d);
    double *g = (double *)malloc(sizeof(double) * f), *u = (double *)malloc(sizeof(double) * f);
    double *w = (double *)malloc(sizeof(double) * (t + 1));
    for (int k = 0; k < d; ++k) x[k] = tok_embed[(size_t)token * d + k];

    for (int l = 0; l < c->n_layers; ++l) {
        const seq_layer *L = &layers[l];
        double *K = kc + (size_t)l * max_seq * d, *V = vc + (size_t)l * max_seq * d;
        norm(x, L->attn_norm, d, c->rms_eps, xn);
        matvec(L->wq, d, d, xn, q);
        matvec(L->wk, d, d, xn, K + (size_t)t * d);
        matvec(L->wv, d, d, xn, V + (size_t)t * d);
        rotate(q, t, H, hd, c->rope_base);
        rotate(K + (size_t)t * d, t, H, hd, c->rope_base);
        for (int h = 0; h < H; ++h) {
            double top = -INFINITY, z = 0.0;
            for (int s = 0; s <= t; ++s) {
                double dot = 0.0;
                for (int e = 0; e < hd; ++e) dot += q[h * hd + e] * K[(size_t)s * d + h * hd + e];
                w[s] = dot / sqrt((double)hd);
                if (w[s] > top) top = w[s];
            }
            for (int s = 0; s <= t; ++s) { w[s] = exp(w[s] - top); z += w[s]; }
            for (int e = 0; e < hd; ++e) {
                double acc = 0.0;
                for (int s = 0; s <= t; ++s) acc += w[s] * V[(size_t)s * d + h * hd + e];
                a[h * hd + e] = acc / z;
            }
        }
        matvec(L->wo, d, d, a, r);
        for (int k = 0; k < d; ++k) x[k] += r[k];
        norm(x, L->ffn_norm, d, c->rms_eps, xn);
        matvec(L->w_gate, f, d, xn, g);
        matvec(L->w_up, f, d, xn, u);
        for (int k = 0; k < f; ++k) g[k] = u[k] * g[k] / (1.0 + exp(-g[k]));
        matvec(L->w_down, d, f, g, r);
        for (int k = 0; k < d; ++k) x[k] += r[k];
    }
    norm(x, final_norm, d, c->rms_eps, xn);
    matvec(lm_head, c->vocab, d, xn, logits);
    free(x); free(xn); free(q); free(a); free(r); free(g); free(u); free(w);
    return 0;
}
