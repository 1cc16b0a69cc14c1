/*
 * cats_ref.c -- CPU oracle for the tree-verification forward of CATS-style
 * self-speculative decoding (Stage 3 of Algorithm 1: the target model scores a
 * draft token tree in one pass, walks the longest accepted path and rolls the
 * KV cache back along it).
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, obviously
 * correct restatement of what the path computes.  Only the test-suite, the
 * smoke check and the benchmark's CPU-baseline leg may call it; the CUDA
 * library shares no code with it and neither includes the other.
 *
 * Arithmetic: every sum (dot products, softmax, norms) is accumulated in fp64
 * in ascending index order.  The "rounding contract" of the GPU path is
 * mirrored at the points where the GPU stores a 16-bit value:
 *   - GEMM inputs (normalised hidden states, attention output, SwiGLU output)
 *     are rounded to bf16 once;
 *   - q and k are rotated (RoPE) from the unrounded sums and rounded to bf16
 *     once; v is rounded once; the KV cache holds those bf16 values;
 *   - the residual stream and the logits are fp32.
 * cats_ref_set_contract(0) switches every bf16 rounding off ("pure" mode), so
 * the oracle can be pinned against float64 library implementations.
 *
 * Parity status: every function below is pinned by tests/test_oracle_*.py
 * (brute force, closed forms, torch float64 library ops, a HuggingFace LLaMA
 * forward with an explicit 4-D mask, Algorithm 1's own walk).  The size of the
 * deviation between contract mode and pure mode is "parity unpinned": the
 * paper states no tolerance for 16-bit inference.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC cats_ref.c -o libcats_ref.so -lm
 * (no fused multiply-add: products and sums are rounded separately on every host)
 * OpenMP is used over independent output rows only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define CATS_REF_MAX_T 128

typedef struct {
    int32_t hidden, n_heads, head_dim, ffn, vocab, n_layers, max_seq;
    float rms_eps, rope_base;
} cats_ref_cfg;

typedef struct {
    const uint16_t *attn_norm, *wq, *wk, *wv, *wo, *mlp_norm, *w_gate, *w_up, *w_down;
} cats_ref_layer_weights;

static int g_contract = 1;
static int g_accum32 = 0;

void cats_ref_set_contract(int on) { g_contract = on ? 1 : 0; }
int cats_ref_get_contract(void) { return g_contract; }

/* Sensitivity probe, off by default: accumulate the projections' dot products in fp32 (sequential,
 * ascending k) instead of fp64.  Every bf16 rounding point of the contract is a discontinuity: two
 * evaluations whose sums differ in the last fp32 bits round a small fraction of the activations to
 * neighbouring bf16 values, and those one-ulp flips spread through attention and the MLPs.  Running
 * the oracle both ways measures how far two equally valid evaluations of the same contract drift
 * apart -- the floor below which no GPU-vs-oracle deviation can be expected to fall. */
void cats_ref_set_accum32(int on) { g_accum32 = on ? 1 : 0; }

/* ---- bf16 <-> fp32 (round to nearest even) ---------------------------- */

float cats_ref_bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

uint16_t cats_ref_f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* NaN stays NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/* value -> value rounded at a contract point (identity in pure mode) */
static double rnd16(double x) {
    if (!g_contract) return x;
    return (double)cats_ref_bf16_to_f32(cats_ref_f32_to_bf16((float)x));
}

/* ---- O1: ancestor mask, depth, position ids (Fig. 4 caption: tree mask; ---
 * Algorithm 1, BuildTree / mask=T.tree_mask).  Node 0 is the root (the last
 * committed token); parent[i] < i.  mask[i] has bit j set iff j is i or an
 * ancestor of i; pos[i] = prefix_len + depth[i].
 * Returns 0, or -2 for a malformed parent array. */
int cats_ref_build_tree_mask(const int32_t *parent, int32_t T, int32_t prefix_len,
                             uint64_t *mask /*[T][2]*/, int32_t *pos, int32_t *depth) {
    if (T < 1 || T > CATS_REF_MAX_T) return -1;
    if (parent[0] != -1) return -2;
    for (int i = 1; i < T; ++i)
        if (parent[i] < 0 || parent[i] >= i) return -2;
    for (int i = 0; i < T; ++i) {
        uint64_t m0 = 0, m1 = 0;
        int d = 0;
        int j = i;
        while (j != -1) { /* walk up to the root, marking each node met */
            if (j < 64) m0 |= (uint64_t)1 << j; else m1 |= (uint64_t)1 << (j - 64);
            j = parent[j];
            if (j != -1) ++d;
        }
        mask[2 * i] = m0;
        mask[2 * i + 1] = m1;
        if (depth) depth[i] = d;
        pos[i] = prefix_len + d;
    }
    return 0;
}

/* ---- RMSNorm: y = g * x * rsqrt(mean(x^2) + eps)  (decoder family of the
 * paper's models: LLaMA-2 / Vicuna).  out is fp64 holding contract-rounded
 * values. */
void cats_ref_rmsnorm(const float *x, const uint16_t *g, int32_t T, int32_t H, float eps,
                      double *out /*[T][H]*/) {
    for (int t = 0; t < T; ++t) {
        double ss = 0.0;
        for (int i = 0; i < H; ++i) ss += (double)x[(size_t)t * H + i] * (double)x[(size_t)t * H + i];
        double r = 1.0 / sqrt(ss / (double)H + (double)eps);
        for (int i = 0; i < H; ++i)
            out[(size_t)t * H + i] = rnd16((double)cats_ref_bf16_to_f32(g[i]) * ((double)x[(size_t)t * H + i] * r));
    }
}

/* ---- Linear: y[t][o] = sum_k W[o][k] * x[t][k], W bf16 [n_out][n_in]
 * (nn.Linear layout), fp64 sums in ascending k.  The loop nest keeps, for one
 * output row, all T running sums side by side; each sum still adds its terms
 * in ascending k.  linear_row is compiled for a few vector widths; the order
 * of additions inside each acc[t] is the same in all of them. */
__attribute__((target_clones("avx512f", "avx2", "default")))
static void linear_row_f32(const uint16_t *w, int32_t n_in, const double *xT, int32_t T, double *acc) {
    float facc[CATS_REF_MAX_T];
    for (int t = 0; t < T; ++t) facc[t] = 0.0f;
    for (int k = 0; k < n_in; ++k) {
        float wk = cats_ref_bf16_to_f32(w[k]);
        const double *xk = xT + (size_t)k * T;
        for (int t = 0; t < T; ++t) facc[t] += wk * (float)xk[t];
    }
    for (int t = 0; t < T; ++t) acc[t] = (double)facc[t];
}

__attribute__((target_clones("avx512f", "avx2", "default")))
static void linear_row(const uint16_t *w, int32_t n_in, const double *xT, int32_t T, double *acc) {
    for (int t = 0; t < T; ++t) acc[t] = 0.0;
    for (int k = 0; k < n_in; ++k) {
        double wk = (double)cats_ref_bf16_to_f32(w[k]);
        const double *xk = xT + (size_t)k * T;
        for (int t = 0; t < T; ++t) acc[t] += wk * xk[t];
    }
}

void cats_ref_linear(const uint16_t *W, int32_t n_out, int32_t n_in, const double *x /*[T][n_in]*/,
                     int32_t T, double *y /*[T][n_out]*/) {
    double *xT = (double *)malloc((size_t)n_in * T * sizeof(double));
    for (int t = 0; t < T; ++t)
        for (int k = 0; k < n_in; ++k) xT[(size_t)k * T + t] = x[(size_t)t * n_in + k];
#pragma omp parallel for schedule(static)
    for (int o = 0; o < n_out; ++o) {
        double acc[CATS_REF_MAX_T];
        if (g_accum32) linear_row_f32(W + (size_t)o * n_in, n_in, xT, T, acc);
        else linear_row(W + (size_t)o * n_in, n_in, xT, T, acc);
        for (int t = 0; t < T; ++t) y[(size_t)t * n_out + o] = acc[t];
    }
    free(xT);
}

/* ---- RoPE, rotate-half pairing (i, i + hd/2), inv_freq_i = base^(-2i/hd),
 * angle = pos * inv_freq_i.  In place on one head vector of fp64 values. */
void cats_ref_rope_head(double *x, int32_t hd, int32_t pos, double base) {
    int half = hd / 2;
    for (int i = 0; i < half; ++i) {
        double inv_freq = pow(base, -2.0 * (double)i / (double)hd);
        double ang = (double)pos * inv_freq;
        double c = cos(ang), s = sin(ang);
        double a = x[i], b = x[i + half];
        x[i] = a * c - b * s;
        x[i + half] = b * c + a * s;
    }
}

int cats_ref_tree_attention_rows(const double *q, const float *kc, const float *vc, const uint64_t *mask,
                                 int32_t nq, int32_t T, int32_t P, int32_t nh, int32_t hd,
                                 int64_t kv_row_stride, double scale, double *out, double *probs);

/* ---- O3 attention (tree-masked): node i of head h attends to every prefix
 * row [0,P) and to tree row P+j iff bit j of mask[i] is set; softmax of
 * scale * q.k over the visible columns; out = sum p * v.
 * q [T][nh][hd] fp64; kc/vc float caches with row stride kv_row_stride
 * elements, head h at column offset h*hd; out [T][nh][hd] fp64 (rounded at the
 * contract point).  probs (optional) [nh][T][P+T] receives the probabilities,
 * exact zeros at masked columns. */
int cats_ref_tree_attention(const double *q, const float *kc, const float *vc, const uint64_t *mask,
                            int32_t T, int32_t P, int32_t nh, int32_t hd, int64_t kv_row_stride,
                            double scale, double *out, double *probs) {
    return cats_ref_tree_attention_rows(q, kc, vc, mask, T, T, P, nh, hd, kv_row_stride, scale, out, probs);
}

/* The same attention for nq query rows that need not be all T tree nodes: query
 * i carries its own 128-bit visibility row mask[i] over the T tree rows P..P+T-1
 * (Stage 2 of Algorithm 1 re-forwards only the correction nodes, with the
 * tree mask applied; the other tree rows are already in the cache).
 * q, out [nq][nh][hd]; probs (optional) [nh][nq][P+T]. */
int cats_ref_tree_attention_rows(const double *q, const float *kc, const float *vc, const uint64_t *mask,
                                 int32_t nq, int32_t T, int32_t P, int32_t nh, int32_t hd,
                                 int64_t kv_row_stride, double scale, double *out, double *probs) {
    if (T < 1 || T > CATS_REF_MAX_T || nq < 1 || nq > T || P < 0) return -1;
    int S = P + T;
#pragma omp parallel for schedule(static) collapse(2)
    for (int h = 0; h < nh; ++h) {
        for (int i = 0; i < nq; ++i) {
            double *s = (double *)malloc((size_t)S * sizeof(double));
            unsigned char *vis = (unsigned char *)malloc((size_t)S);
            const double *qi = q + ((size_t)i * nh + h) * hd;
            double m = -INFINITY;
            for (int c = 0; c < S; ++c) {
                int visible;
                if (c < P) visible = 1;
                else {
                    int j = c - P;
                    visible = (int)((mask[2 * i + (j >> 6)] >> (j & 63)) & 1u);
                }
                vis[c] = (unsigned char)visible;
                if (!visible) continue;
                const float *kr = kc + (size_t)c * kv_row_stride + (size_t)h * hd;
                double d = 0.0;
                for (int e = 0; e < hd; ++e) d += qi[e] * (double)kr[e];
                s[c] = d * scale;
                if (s[c] > m) m = s[c];
            }
            double l = 0.0;
            for (int c = 0; c < S; ++c)
                if (vis[c]) { s[c] = exp(s[c] - m); l += s[c]; }
            double *oi = out + ((size_t)i * nh + h) * hd;
            for (int e = 0; e < hd; ++e) oi[e] = 0.0;
            for (int c = 0; c < S; ++c) {
                double p = vis[c] ? s[c] / l : 0.0;
                if (probs) probs[((size_t)h * nq + i) * S + c] = p;
                if (!vis[c]) continue;
                const float *vr = vc + (size_t)c * kv_row_stride + (size_t)h * hd;
                for (int e = 0; e < hd; ++e) oi[e] += p * (double)vr[e];
            }
            for (int e = 0; e < hd; ++e) oi[e] = rnd16(oi[e]);
            free(s);
            free(vis);
        }
    }
    return 0;
}

static double silu(double x) { return x / (1.0 + exp(-x)); }

/* ---- O3: one decoder layer over the T tree nodes (Algorithm 1, Stage 3:
 * H_tgt <- M(T.hidden_states, mask=T.tree_mask, KV_M); Section 3.2, final
 * verification: all tree nodes in one batch under the tree mask).
 * resid [T][H] fp32 in/out.  kc, vc: this layer's caches, float
 * [max_seq][nh*hd]; rows [0,P) are the committed prefix, rows P+i are written
 * here.  q_out (optional) [T][nh*hd] fp64 receives the rotated, rounded q. */
int cats_ref_verify_layer(const cats_ref_cfg *cfg, const cats_ref_layer_weights *w, float *resid,
                          float *kc, float *vc, const uint64_t *mask, const int32_t *pos,
                          int32_t T, int32_t P, double *q_out) {
    int H = cfg->hidden, nh = cfg->n_heads, hd = cfg->head_dim, F = cfg->ffn;
    int D = nh * hd;
    if (T < 1 || T > CATS_REF_MAX_T || P < 0 || P + T > cfg->max_seq || (hd & 1)) return -1;
    double *xn = (double *)malloc((size_t)T * H * sizeof(double));
    double *q = (double *)malloc((size_t)T * D * sizeof(double));
    double *k = (double *)malloc((size_t)T * D * sizeof(double));
    double *v = (double *)malloc((size_t)T * D * sizeof(double));
    double *o = (double *)malloc((size_t)T * D * sizeof(double));
    double *y = (double *)malloc((size_t)T * H * sizeof(double));
    double *g = (double *)malloc((size_t)T * F * sizeof(double));
    double *u = (double *)malloc((size_t)T * F * sizeof(double));

    /* attention block */
    cats_ref_rmsnorm(resid, w->attn_norm, T, H, cfg->rms_eps, xn);
    cats_ref_linear(w->wq, D, H, xn, T, q);
    cats_ref_linear(w->wk, D, H, xn, T, k);
    cats_ref_linear(w->wv, D, H, xn, T, v);
    for (int t = 0; t < T; ++t) {
        for (int h = 0; h < nh; ++h) {
            cats_ref_rope_head(q + (size_t)t * D + (size_t)h * hd, hd, pos[t], (double)cfg->rope_base);
            cats_ref_rope_head(k + (size_t)t * D + (size_t)h * hd, hd, pos[t], (double)cfg->rope_base);
        }
        for (int e = 0; e < D; ++e) {
            q[(size_t)t * D + e] = rnd16(q[(size_t)t * D + e]);
            kc[(size_t)(P + t) * D + e] = (float)rnd16(k[(size_t)t * D + e]);
            vc[(size_t)(P + t) * D + e] = (float)rnd16(v[(size_t)t * D + e]);
        }
    }
    if (q_out) memcpy(q_out, q, (size_t)T * D * sizeof(double));
    cats_ref_tree_attention(q, kc, vc, mask, T, P, nh, hd, D, 1.0 / sqrt((double)hd), o, NULL);
    cats_ref_linear(w->wo, H, D, o, T, y);
    for (size_t i = 0; i < (size_t)T * H; ++i) resid[i] = (float)((double)resid[i] + y[i]);

    /* MLP block (SwiGLU) */
    cats_ref_rmsnorm(resid, w->mlp_norm, T, H, cfg->rms_eps, xn);
    cats_ref_linear(w->w_gate, F, H, xn, T, g);
    cats_ref_linear(w->w_up, F, H, xn, T, u);
    for (size_t i = 0; i < (size_t)T * F; ++i) g[i] = rnd16(silu(g[i]) * u[i]);
    cats_ref_linear(w->w_down, H, F, g, T, y);
    for (size_t i = 0; i < (size_t)T * H; ++i) resid[i] = (float)((double)resid[i] + y[i]);

    free(xn); free(q); free(k); free(v); free(o); free(y); free(g); free(u);
    return 0;
}

/* ---- O3 over a subset of the tree (Algorithm 1, Stage 2: the correction
 * tokens go through layers 1..L_SV again with the tree mask applied; the
 * main-chain nodes already have their K/V in these layers).
 * nodes[0..m) are tree node indices, strictly ascending; resid [m][H] holds the
 * hidden states of those nodes only.  The K/V of node nodes[j] is written to
 * cache row P + nodes[j]; every other cache row is read-only.  Node nodes[j]
 * attends to the prefix and to the tree rows its mask row names, which must
 * be rows of active nodes or rows cached earlier. */
int cats_ref_verify_layer_nodes(const cats_ref_cfg *cfg, const cats_ref_layer_weights *w, float *resid,
                                float *kc, float *vc, const uint64_t *mask /*[T][2]*/, const int32_t *pos /*[T]*/,
                                const int32_t *nodes, int32_t m, int32_t T, int32_t P) {
    int H = cfg->hidden, nh = cfg->n_heads, hd = cfg->head_dim, F = cfg->ffn;
    int D = nh * hd;
    if (T < 1 || T > CATS_REF_MAX_T || m < 1 || m > T || P < 0 || P + T > cfg->max_seq || (hd & 1)) return -1;
    for (int j = 0; j < m; ++j)
        if (nodes[j] < 0 || nodes[j] >= T || (j > 0 && nodes[j] <= nodes[j - 1])) return -2;
    double *xn = (double *)malloc((size_t)m * H * sizeof(double));
    double *q = (double *)malloc((size_t)m * D * sizeof(double));
    double *k = (double *)malloc((size_t)m * D * sizeof(double));
    double *v = (double *)malloc((size_t)m * D * sizeof(double));
    double *o = (double *)malloc((size_t)m * D * sizeof(double));
    double *y = (double *)malloc((size_t)m * H * sizeof(double));
    double *g = (double *)malloc((size_t)m * F * sizeof(double));
    double *u = (double *)malloc((size_t)m * F * sizeof(double));
    uint64_t *mrows = (uint64_t *)malloc((size_t)m * 2 * sizeof(uint64_t));

    cats_ref_rmsnorm(resid, w->attn_norm, m, H, cfg->rms_eps, xn);
    cats_ref_linear(w->wq, D, H, xn, m, q);
    cats_ref_linear(w->wk, D, H, xn, m, k);
    cats_ref_linear(w->wv, D, H, xn, m, v);
    for (int j = 0; j < m; ++j) {
        int n = nodes[j];
        for (int h = 0; h < nh; ++h) {
            cats_ref_rope_head(q + (size_t)j * D + (size_t)h * hd, hd, pos[n], (double)cfg->rope_base);
            cats_ref_rope_head(k + (size_t)j * D + (size_t)h * hd, hd, pos[n], (double)cfg->rope_base);
        }
        for (int e = 0; e < D; ++e) {
            q[(size_t)j * D + e] = rnd16(q[(size_t)j * D + e]);
            kc[(size_t)(P + n) * D + e] = (float)rnd16(k[(size_t)j * D + e]);
            vc[(size_t)(P + n) * D + e] = (float)rnd16(v[(size_t)j * D + e]);
        }
        mrows[2 * j] = mask[2 * n];
        mrows[2 * j + 1] = mask[2 * n + 1];
    }
    cats_ref_tree_attention_rows(q, kc, vc, mrows, m, T, P, nh, hd, D, 1.0 / sqrt((double)hd), o, NULL);
    cats_ref_linear(w->wo, H, D, o, m, y);
    for (size_t i = 0; i < (size_t)m * H; ++i) resid[i] = (float)((double)resid[i] + y[i]);

    cats_ref_rmsnorm(resid, w->mlp_norm, m, H, cfg->rms_eps, xn);
    cats_ref_linear(w->w_gate, F, H, xn, m, g);
    cats_ref_linear(w->w_up, F, H, xn, m, u);
    for (size_t i = 0; i < (size_t)m * F; ++i) g[i] = rnd16(silu(g[i]) * u[i]);
    cats_ref_linear(w->w_down, H, F, g, m, y);
    for (size_t i = 0; i < (size_t)m * H; ++i) resid[i] = (float)((double)resid[i] + y[i]);

    free(xn); free(q); free(k); free(v); free(o); free(y); free(g); free(u); free(mrows);
    return 0;
}

/* ---- O2: hidden states of the tree tokens from the embedding table. */
void cats_ref_embed(const uint16_t *E /*[V][H]*/, const int32_t *tokens, int32_t T, int32_t H, float *resid) {
    for (int t = 0; t < T; ++t)
        for (int i = 0; i < H; ++i) resid[(size_t)t * H + i] = cats_ref_bf16_to_f32(E[(size_t)tokens[t] * H + i]);
}

/* ---- O4: final norm, LM head, per-node argmax (Algorithm 1: p_tgt =
 * softmax(H(H_tgt)); softmax is monotone, so greedy acceptance needs only the
 * argmax of the logits).  Ties: lowest vocabulary index.  margin[i] = top1 -
 * top2.  logits [T][V] fp32 (optional). */
int cats_ref_lm_head_argmax(const cats_ref_cfg *cfg, const uint16_t *final_norm, const uint16_t *w_lm,
                            const float *resid, int32_t T, float *logits, int32_t *argmax, float *margin) {
    int H = cfg->hidden, V = cfg->vocab;
    if (T < 1 || T > CATS_REF_MAX_T) return -1;
    double *xn = (double *)malloc((size_t)T * H * sizeof(double));
    double *lg = (double *)malloc((size_t)T * V * sizeof(double));
    cats_ref_rmsnorm(resid, final_norm, T, H, cfg->rms_eps, xn);
    cats_ref_linear(w_lm, V, H, xn, T, lg);
    for (int t = 0; t < T; ++t) {
        float best = -INFINITY, second = -INFINITY;
        int bi = -1;
        for (int vv = 0; vv < V; ++vv) {
            float x = (float)lg[(size_t)t * V + vv];
            if (logits) logits[(size_t)t * V + vv] = x;
            if (x > best) { second = best; best = x; bi = vv; }
            else if (x > second) second = x;
        }
        argmax[t] = bi;
        if (margin) margin[t] = best - second;
    }
    free(xn); free(lg);
    return 0;
}

/* ---- O5: greedy longest-accepted-path walk (Algorithm 1, the walk step
 * of Stage 3, and the bonus token).  A child is accepted
 * iff its token equals the target's argmax at its parent; among equal sibling
 * tokens the lowest node index wins.  path[0] = 0 (root); out_tokens holds the
 * accepted draft tokens followed by the bonus token; n_out == path_len. */
int cats_ref_accept_path(const int32_t *parent, const int32_t *tokens, const int32_t *argmax, int32_t T,
                         int32_t *path, int32_t *path_len, int32_t *out_tokens, int32_t *n_out) {
    if (T < 1 || T > CATS_REF_MAX_T) return -1;
    int cur = 0, len = 0, no = 0;
    path[len++] = 0;
    for (;;) {
        int want = argmax[cur];
        int next = -1;
        for (int j = cur + 1; j < T; ++j)
            if (parent[j] == cur && tokens[j] == want) { next = j; break; }
        if (next < 0) break;
        out_tokens[no++] = want;
        path[len++] = next;
        cur = next;
    }
    out_tokens[no++] = argmax[cur]; /* bonus token */
    *path_len = len;
    *n_out = no;
    return 0;
}

/* ---- O5b: typical (relaxed) acceptance, the second criterion Acc of
 * Algorithm 1 ("greedy or typical"; the tables' "relaxed (temperature = 0.7)"
 * setting), as the cited Medusa work defines it: with p = softmax(logits / t)
 * at the parent, a child token x is acceptable iff
 *     p(x) > min(eps, delta * exp(-H(p))),      H(p) = -sum_v p_v log p_v.
 * Per-node statistics by their definitions, in fp64:
 *   lse[n]     = log sum_v exp(logits[n][v] / t)
 *   entropy[n] = H(softmax(logits[n] / t))
 *   cand_logit[i] = logits[parent[i]][tokens[i]]   (0 for the root)
 *   prob[i]    = p_parent(i)(tokens[i])            (optional, fp64; 0 for the root)
 * lse, entropy and cand_logit are delivered as fp32 (what the walk consumes). */
int cats_ref_typical_stats(const float *logits, int32_t T, int32_t V, double temperature,
                           const int32_t *parent, const int32_t *tokens, float *lse, float *entropy,
                           float *cand_logit, double *prob) {
    if (T < 1 || T > CATS_REF_MAX_T || V < 1 || !(temperature > 0.0)) return -1;
    double *lse64 = (double *)malloc((size_t)T * sizeof(double));
    for (int n = 0; n < T; ++n) {
        const float *l = logits + (size_t)n * V;
        double m = -INFINITY;
        for (int v = 0; v < V; ++v) {
            double z = (double)l[v] / temperature;
            if (z > m) m = z;
        }
        double Z = 0.0;
        for (int v = 0; v < V; ++v) Z += exp((double)l[v] / temperature - m);
        lse64[n] = m + log(Z);
        double H = 0.0;
        for (int v = 0; v < V; ++v) {
            double lp = (double)l[v] / temperature - lse64[n];
            double pv = exp(lp);
            if (pv > 0.0) H -= pv * lp;
        }
        lse[n] = (float)lse64[n];
        entropy[n] = (float)H;
    }
    for (int i = 0; i < T; ++i) {
        int pa = parent[i];
        if (i == 0 || pa < 0 || pa >= i || tokens[i] < 0 || tokens[i] >= V) {
            cand_logit[i] = 0.f;
            if (prob) prob[i] = 0.0;
            continue;
        }
        float c = logits[(size_t)pa * V + tokens[i]];
        cand_logit[i] = c;
        if (prob) prob[i] = exp((double)c / temperature - lse64[pa]);
    }
    free(lse64);
    return 0;
}

/* The walk of Algorithm 1 with a per-node verdict: starting at the root, take
 * the first acceptable child in node order (on a CATS tree: the main draft
 * token d_a, else the correction at that position), stop when none is; the
 * bonus token is the argmax at the last accepted node. */
static int walk_with_verdicts(const int32_t *parent, const int32_t *tokens, const int32_t *argmax,
                              const unsigned char *ok, int32_t T, int32_t *path, int32_t *path_len,
                              int32_t *out_tokens, int32_t *n_out) {
    int cur = 0, len = 0, no = 0;
    path[len++] = 0;
    for (;;) {
        int next = -1;
        for (int j = cur + 1; j < T; ++j)
            if (parent[j] == cur && ok[j]) { next = j; break; }
        if (next < 0) break;
        out_tokens[no++] = tokens[next];
        path[len++] = next;
        cur = next;
    }
    out_tokens[no++] = argmax[cur];
    *path_len = len;
    *n_out = no;
    return 0;
}

/* Typical acceptance straight from the definition, in fp64, on the logits. */
int cats_ref_accept_path_typical_def(const int32_t *parent, const int32_t *tokens, const int32_t *argmax,
                                     const float *logits, int32_t T, int32_t V, double temperature,
                                     double eps, double delta, int32_t *path, int32_t *path_len,
                                     int32_t *out_tokens, int32_t *n_out) {
    if (T < 1 || T > CATS_REF_MAX_T) return -1;
    float lse[CATS_REF_MAX_T], H[CATS_REF_MAX_T], cand[CATS_REF_MAX_T];
    double prob[CATS_REF_MAX_T];
    unsigned char ok[CATS_REF_MAX_T];
    /* entropy again in fp64 here, so that the verdict does not pass through fp32 */
    int rc = cats_ref_typical_stats(logits, T, V, temperature, parent, tokens, lse, H, cand, prob);
    if (rc) return rc;
    ok[0] = 0;
    for (int i = 1; i < T; ++i) {
        int pa = parent[i];
        const float *l = logits + (size_t)pa * V;
        double m = -INFINITY, Z = 0.0, Hd = 0.0;
        for (int v = 0; v < V; ++v) if ((double)l[v] / temperature > m) m = (double)l[v] / temperature;
        for (int v = 0; v < V; ++v) Z += exp((double)l[v] / temperature - m);
        for (int v = 0; v < V; ++v) {
            double lp = (double)l[v] / temperature - m - log(Z);
            if (exp(lp) > 0.0) Hd -= exp(lp) * lp;
        }
        double thr = delta * exp(-Hd);
        if (eps < thr) thr = eps;
        ok[i] = (unsigned char)(prob[i] > thr);
    }
    return walk_with_verdicts(parent, tokens, argmax, ok, T, path, path_len, out_tokens, n_out);
}

/* The same walk from the fp32 statistics, with the verdict taken in the log
 * domain in fp32 and a fixed operation order, so that any implementation given
 * the same inputs reaches the same verdict bit for bit:
 *     logp = fma(cand_logit[i], inv_temperature, -lse[parent])        (one rounding)
 *     thr  = min(log_eps, log_delta - entropy[parent])
 *     acceptable iff logp > thr          (log is monotone: the same criterion). */
int cats_ref_accept_path_typical(const int32_t *parent, const int32_t *tokens, const int32_t *argmax,
                                 const float *cand_logit, const float *lse, const float *entropy, int32_t T,
                                 float inv_temperature, float log_eps, float log_delta, int32_t *path,
                                 int32_t *path_len, int32_t *out_tokens, int32_t *n_out) {
    if (T < 1 || T > CATS_REF_MAX_T) return -1;
    unsigned char ok[CATS_REF_MAX_T];
    ok[0] = 0;
    for (int i = 1; i < T; ++i) {
        int pa = parent[i];
        if (pa < 0 || pa >= i) return -2;
        float logp = fmaf(cand_logit[i], inv_temperature, -lse[pa]);
        volatile float d = log_delta - entropy[pa];
        float thr = fminf(log_eps, d);
        ok[i] = (unsigned char)(logp > thr);
    }
    return walk_with_verdicts(parent, tokens, argmax, ok, T, path, path_len, out_tokens, n_out);
}

/* ---- O6: KV rollback along the accepted path (Algorithm 1, last step of
 * the cycle).  For every layer, K and V: row
 * P+path[k] moves to row P+k, k ascending, in place.  src/dst (optional)
 * receive the row index lists.  The cache element type is opaque: elem_bytes
 * bytes per element. */
int cats_ref_compact_kv(void *kcache, void *vcache, int32_t n_layers, int64_t layer_stride_elems,
                        int64_t row_elems, int32_t elem_bytes, int32_t prefix_len, const int32_t *path,
                        int32_t path_len, int32_t *new_len, int32_t *src, int32_t *dst) {
    if (path_len < 1 || path_len > CATS_REF_MAX_T) return -1;
    for (int k = 0; k < path_len; ++k) {
        if (path[k] < k || (k > 0 && path[k] <= path[k - 1])) return -2;
        if (src) src[k] = prefix_len + path[k];
        if (dst) dst[k] = prefix_len + k;
    }
    size_t rb = (size_t)row_elems * elem_bytes;
    for (int l = 0; l < n_layers; ++l) {
        for (int which = 0; which < 2; ++which) {
            unsigned char *base = (unsigned char *)(which ? vcache : kcache) +
                                  (size_t)l * layer_stride_elems * elem_bytes;
            for (int k = 0; k < path_len; ++k) {
                if (path[k] == k) continue;
                memmove(base + (size_t)(prefix_len + k) * rb, base + (size_t)(prefix_len + path[k]) * rb, rb);
            }
        }
    }
    *new_len = prefix_len + path_len;
    return 0;
}

/* ---- Whole Stage-3 forward: embedding (or caller's hidden states), layers
 * [0, n_layers), head, argmax.  weights: array of n_layers structs.  kc/vc:
 * [n_layers][max_seq][nh*hd] float.  If hidden_in != NULL it is used instead
 * of the embedding gather.  resid_out (optional) [T][H]. */
int cats_ref_verify_forward(const cats_ref_cfg *cfg, const cats_ref_layer_weights *weights,
                            const uint16_t *embed, const uint16_t *final_norm, const uint16_t *w_lm,
                            const int32_t *parent, const int32_t *tokens, const float *hidden_in,
                            int32_t T, int32_t P, float *kc, float *vc, float *logits, int32_t *argmax,
                            float *margin, float *resid_out) {
    int H = cfg->hidden;
    uint64_t mask[2 * CATS_REF_MAX_T];
    int32_t pos[CATS_REF_MAX_T], depth[CATS_REF_MAX_T];
    int rc = cats_ref_build_tree_mask(parent, T, P, mask, pos, depth);
    if (rc) return rc;
    float *resid = (float *)malloc((size_t)T * H * sizeof(float));
    if (hidden_in) memcpy(resid, hidden_in, (size_t)T * H * sizeof(float));
    else cats_ref_embed(embed, tokens, T, H, resid);
    size_t lstride = (size_t)cfg->max_seq * cfg->n_heads * cfg->head_dim;
    for (int l = 0; l < cfg->n_layers; ++l) {
        rc = cats_ref_verify_layer(cfg, &weights[l], resid, kc + l * lstride, vc + l * lstride, mask, pos, T, P, NULL);
        if (rc) { free(resid); return rc; }
    }
    rc = cats_ref_lm_head_argmax(cfg, final_norm, w_lm, resid, T, logits, argmax, margin);
    if (resid_out) memcpy(resid_out, resid, (size_t)T * H * sizeof(float));
    free(resid);
    return rc;
}
