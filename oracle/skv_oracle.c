/*
 * skv_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of what the routed decode path computes,
 * written from the paper's definitions so that it can be checked against the
 * paper by eye.  Only the tests, the smoke check and the benchmark's CPU
 * baseline leg may call it.  It shares no code, header, table or constant
 * with the CUDA library and knows nothing about pages, splits or tiles.
 *
 * State (Algorithm 1, "Standard Inference"): one dense K store and one dense
 * V store PER LAYER, owner or not, laid out [B][n_max][Hkv][D] and kept as the
 * bf16 bit patterns that were appended (bf16 -> fp64 widening is exact).
 *
 * Operations:
 *   oracle_append       "Update K_l, V_l" of Algorithm 1: write rows of layer l.
 *   oracle_decode_attn  Eq. (3.1): Output_l = Attn(Q_l, K_l', V_l') with the
 *                       source layer l' = r[l] taken BY INDEXING the per-layer
 *                       stores (Eq. (3.2) / Algorithm 2 say which l' to use).
 *                       Attn is scaled dot-product softmax attention; query
 *                       head h reads KV head floor(h / (Hq/Hkv)).
 *   oracle_attn_rows    Pre-fill (Section 3.1.1 "processing the initial prompt of T
 *                       tokens in parallel"): Eq. (3.1) for many query tokens at
 *                       once, each a row (sequence b, position pos) that attends
 *                       the source layer's tokens 0..pos of its sequence (a
 *                       decoder is causal).  One decode step is the special case
 *                       of one row per sequence at pos = seq_len - 1.
 *   oracle_rcla_map     Section 3.2 (R-CLA, training time): per layer and forward pass
 *                       d ~ Bernoulli(p); d = 1 keeps the layer's own K,V, d = 0 takes
 *                       a layer drawn uniformly from those before it.  The random
 *                       numbers are inputs (u for the coin, v for the choice).
 *   oracle_rdcla_map    Section 4.2 ablation (RD-CLA@k): the fixed groups of k layers,
 *                       but each layer flips a coin between the group's first layer
 *                       and its own K,V.
 *   oracle_mu           Eq. (3.2): owner set S -> map mu (0-based layers).
 *   oracle_group_map    Section 4.3: groups of g consecutive layers share the
 *                       first layer's cache.
 *   oracle_cache_bytes  Section 1 footnote / Figure 1 caption / Section 3.1.1:
 *                       2 x #cached layers x #kv_heads x head_dim x bytes/elt
 *                       per token, times the number of tokens.
 *
 * Pinned by tests/test_oracle_pins.py (paper's printed values, closed forms,
 * library attention in fp64, brute force).  OpenMP is used over independent
 * (sequence, head) pairs for wall-clock timing only; it changes no result.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int L, Hq, Hkv, D, B;
    int64_t n_max;
    int32_t *r;          /* [L] routing map, 0-based, r[l] <= l */
    uint16_t **K;        /* [L] -> [B][n_max][Hkv][D] bf16 bits, NULL until first append */
    uint16_t **V;
} oracle_t;

static double bf16_to_f64(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

oracle_t *oracle_create(int L, const int32_t *r, int Hq, int Hkv, int D, int B, int64_t n_max)
{
    if (L <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || B <= 0 || n_max <= 0 || Hq % Hkv != 0)
        return NULL;
    for (int l = 0; l < L; ++l)
        if (r[l] < 0 || r[l] > l)
            return NULL;
    oracle_t *o = (oracle_t *)calloc(1, sizeof *o);
    if (!o) return NULL;
    o->L = L; o->Hq = Hq; o->Hkv = Hkv; o->D = D; o->B = B; o->n_max = n_max;
    o->r = (int32_t *)malloc(sizeof(int32_t) * (size_t)L);
    o->K = (uint16_t **)calloc((size_t)L, sizeof *o->K);
    o->V = (uint16_t **)calloc((size_t)L, sizeof *o->V);
    memcpy(o->r, r, sizeof(int32_t) * (size_t)L);
    return o;
}

void oracle_destroy(oracle_t *o)
{
    if (!o) return;
    for (int l = 0; l < o->L; ++l) { free(o->K[l]); free(o->V[l]); }
    free(o->K); free(o->V); free(o->r); free(o);
}

static size_t row_index(const oracle_t *o, int64_t b, int64_t t)
{
    return ((size_t)b * (size_t)o->n_max + (size_t)t) * (size_t)o->Hkv * (size_t)o->D;
}

/* "Update": rows K[i], V[i] ([Hkv][D] bf16 bits) become token pos[i] of
 * sequence seq_idx[i] in layer `layer`'s own store.  No routing here: every
 * layer keeps its own cache, as in Algorithm 1.  Later rows overwrite earlier
 * ones at the same (sequence, position). */
int oracle_append(oracle_t *o, int layer, const uint16_t *K, const uint16_t *V,
                  const int64_t *seq_idx, const int64_t *pos, int64_t n_tok)
{
    if (!o || layer < 0 || layer >= o->L) return -1;
    size_t row = (size_t)o->Hkv * (size_t)o->D;
    if (!o->K[layer]) {
        size_t elems = (size_t)o->B * (size_t)o->n_max * row;
        o->K[layer] = (uint16_t *)calloc(elems, sizeof(uint16_t));
        o->V[layer] = (uint16_t *)calloc(elems, sizeof(uint16_t));
        if (!o->K[layer] || !o->V[layer]) return -2;
    }
    for (int64_t i = 0; i < n_tok; ++i) {
        if (seq_idx[i] < 0 || seq_idx[i] >= o->B || pos[i] < 0 || pos[i] >= o->n_max) return -3;
        size_t at = row_index(o, seq_idx[i], pos[i]);
        memcpy(o->K[layer] + at, K + (size_t)i * row, row * sizeof(uint16_t));
        memcpy(o->V[layer] + at, V + (size_t)i * row, row * sizeof(uint16_t));
    }
    return 0;
}

/* Read back one stored row (bit patterns) of a layer's own store. */
int oracle_read(const oracle_t *o, int layer, int64_t b, int64_t t, uint16_t *K_row, uint16_t *V_row)
{
    if (!o || layer < 0 || layer >= o->L || !o->K[layer]) return -1;
    if (b < 0 || b >= o->B || t < 0 || t >= o->n_max) return -3;
    size_t row = (size_t)o->Hkv * (size_t)o->D, at = row_index(o, b, t);
    memcpy(K_row, o->K[layer] + at, row * sizeof(uint16_t));
    memcpy(V_row, o->V[layer] + at, row * sizeof(uint16_t));
    return 0;
}

/* Softmax weights of query head h of sequence b over the first n cached
 * tokens of the source layer r[layer]:  w_t = exp(s_t - max s) / sum(...),
 * s_t = scale * <Q[b,h,:], K_src[b,t,kv(h),:]>. */
static int weights_of(const oracle_t *o, int layer, const uint16_t *Q, int b, int h,
                      int64_t n, double scale, double *w)
{
    int src = o->r[layer];
    const uint16_t *Ks = o->K[src];
    if (!Ks) return -1;
    int G = o->Hq / o->Hkv, kv = h / G, D = o->D;
    const uint16_t *q = Q + ((size_t)b * (size_t)o->Hq + (size_t)h) * (size_t)D;
    double smax = -INFINITY;
    for (int64_t t = 0; t < n; ++t) {
        const uint16_t *k = Ks + row_index(o, b, t) + (size_t)kv * (size_t)D;
        double s = 0.0;
        for (int d = 0; d < D; ++d) s += bf16_to_f64(q[d]) * bf16_to_f64(k[d]);
        s *= scale;
        w[t] = s;
        if (s > smax) smax = s;
    }
    double denom = 0.0;
    for (int64_t t = 0; t < n; ++t) { w[t] = exp(w[t] - smax); denom += w[t]; }
    for (int64_t t = 0; t < n; ++t) w[t] /= denom;
    return 0;
}

int oracle_attn_weights(const oracle_t *o, int layer, const uint16_t *Q, int b, int h,
                        int64_t n, double scale, double *w_out)
{
    if (!o || layer < 0 || layer >= o->L || b < 0 || b >= o->B || h < 0 || h >= o->Hq) return -1;
    if (n < 0 || n > o->n_max) return -3;
    return weights_of(o, layer, Q, b, h, n, scale, w_out);
}

/* Eq. (3.1) with l' = r[layer]:  out[b,h,:] = sum_t w_t * V_src[b,t,kv(h),:]
 * over t < seq_lens[b]; a sequence of length 0 gives a zero row.
 * Q: [B][Hq][D] bf16 bits; out: [B][Hq][D] fp64 (not rounded). */
int oracle_decode_attn(const oracle_t *o, int layer, const uint16_t *Q, const int32_t *seq_lens,
                       double scale, double *out)
{
    if (!o || layer < 0 || layer >= o->L) return -1;
    int src = o->r[layer];
    if (!o->K[src] || !o->V[src]) return -1;
    int G = o->Hq / o->Hkv, D = o->D;
    for (int b = 0; b < o->B; ++b)
        if (seq_lens[b] < 0 || seq_lens[b] > o->n_max) return -3;
    int fail = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < o->B; ++b) {
        for (int h = 0; h < o->Hq; ++h) {
            int64_t n = seq_lens[b];
            double *y = out + ((size_t)b * (size_t)o->Hq + (size_t)h) * (size_t)D;
            for (int d = 0; d < D; ++d) y[d] = 0.0;
            if (n == 0) continue;
            double *w = (double *)malloc(sizeof(double) * (size_t)n);
            if (!w || weights_of(o, layer, Q, b, h, n, scale, w) != 0) {
#pragma omp atomic write
                fail = 1;
                free(w);
                continue;
            }
            int kv = h / G;
            for (int64_t t = 0; t < n; ++t) {
                const uint16_t *v = o->V[src] + row_index(o, b, t) + (size_t)kv * (size_t)D;
                for (int d = 0; d < D; ++d) y[d] += w[t] * bf16_to_f64(v[d]);
            }
            free(w);
        }
    }
    return fail ? -2 : 0;
}

/* Eq. (3.1) with l' = r[layer] for n_q query tokens processed in parallel (pre-fill):
 * row i is a token of sequence q_seq[i] at position q_pos[i]; a decoder is causal, so it
 * attends the source layer's tokens t = 0 .. q_pos[i] of that sequence:
 *   s_t = scale * <Q[i,h,:], K_src[q_seq[i], t, kv(h), :]>,  w = softmax(s),
 *   out[i,h,:] = sum_t w_t * V_src[q_seq[i], t, kv(h), :].
 * Q: [n_q][Hq][D] bf16 bits; out: [n_q][Hq][D] fp64 (not rounded). */
int oracle_attn_rows(const oracle_t *o, int layer, const uint16_t *Q, const int64_t *q_seq, const int64_t *q_pos,
                     int64_t n_q, double scale, double *out)
{
    if (!o || layer < 0 || layer >= o->L) return -1;
    int src = o->r[layer];
    if (!o->K[src] || !o->V[src]) return -1;
    int G = o->Hq / o->Hkv, D = o->D;
    for (int64_t i = 0; i < n_q; ++i)
        if (q_seq[i] < 0 || q_seq[i] >= o->B || q_pos[i] < 0 || q_pos[i] >= o->n_max) return -3;
    int fail = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int64_t i = 0; i < n_q; ++i) {
        for (int h = 0; h < o->Hq; ++h) {
            int64_t b = q_seq[i], n = q_pos[i] + 1;
            int kv = h / G;
            const uint16_t *q = Q + ((size_t)i * (size_t)o->Hq + (size_t)h) * (size_t)D;
            double *y = out + ((size_t)i * (size_t)o->Hq + (size_t)h) * (size_t)D;
            double *s = (double *)malloc(sizeof(double) * (size_t)n);
            if (!s) {
#pragma omp atomic write
                fail = 1;
                continue;
            }
            double smax = -INFINITY;
            for (int64_t t = 0; t < n; ++t) {
                const uint16_t *k = o->K[src] + row_index(o, b, t) + (size_t)kv * (size_t)D;
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += bf16_to_f64(q[d]) * bf16_to_f64(k[d]);
                s[t] = scale * acc;
                if (s[t] > smax) smax = s[t];
            }
            double denom = 0.0;
            for (int64_t t = 0; t < n; ++t) { s[t] = exp(s[t] - smax); denom += s[t]; }
            for (int d = 0; d < D; ++d) y[d] = 0.0;
            for (int64_t t = 0; t < n; ++t) {
                const uint16_t *v = o->V[src] + row_index(o, b, t) + (size_t)kv * (size_t)D;
                double w = s[t] / denom;
                for (int d = 0; d < D; ++d) y[d] += w * bf16_to_f64(v[d]);
            }
            free(s);
        }
    }
    return fail ? -2 : 0;
}

/* Section 3.2, one forward pass of R-CLA training, 0-based layers: for every layer l draw
 * d ~ Bernoulli(p_self) as (u[l] < p_self); d = 1: the layer attends its own K,V (map[l] = l);
 * d = 0: it attends layer l' uniform on {0, .., l-1}, taken as floor(v[l] * l).  Layer 0 has no
 * layer before it and always attends itself.  u, v in [0, 1). */
int oracle_rcla_map(int L, double p_self, const double *u, const double *v, int32_t *map_out)
{
    if (L <= 0 || p_self < 0.0 || p_self > 1.0) return -1;
    for (int l = 0; l < L; ++l) {
        if (u[l] < 0.0 || u[l] >= 1.0 || v[l] < 0.0 || v[l] >= 1.0) return -1;
        if (l == 0 || u[l] < p_self) {
            map_out[l] = l;
        } else {
            int pick = (int)floor(v[l] * (double)l);
            if (pick > l - 1) pick = l - 1;
            map_out[l] = pick;
        }
    }
    return 0;
}

/* Section 4.2 ablation, RD-CLA@k: groups of k consecutive layers share the first one's K,V as in
 * CLA@k, but at each forward step each layer flips a coin: u[l] < p_self keeps its own K,V,
 * otherwise it attends the first layer of its group. */
int oracle_rdcla_map(int L, int k, double p_self, const double *u, int32_t *map_out)
{
    if (L <= 0 || k <= 0 || p_self < 0.0 || p_self > 1.0) return -1;
    for (int l = 0; l < L; ++l) {
        if (u[l] < 0.0 || u[l] >= 1.0) return -1;
        map_out[l] = (u[l] < p_self) ? l : (l / k) * k;
    }
    return 0;
}

/* Eq. (3.2), 0-based: mu(l) = l if l in S, else the largest member of S below
 * l.  Returns -1 when some layer has no owner at or below it (mu undefined). */
int oracle_mu(int L, const int32_t *owners, int n_owners, int32_t *mu_out)
{
    for (int l = 0; l < L; ++l) {
        int best = -1;
        for (int i = 0; i < n_owners; ++i) {
            int j = owners[i];
            if (j < 0 || j >= L) return -1;
            if (j == l) { best = l; break; }
            if (j < l && j > best) best = j;
        }
        if (best < 0) return -1;
        mu_out[l] = best;
    }
    return 0;
}

/* Section 4.3: every g consecutive layers share the cache of the first one. */
int oracle_group_map(int L, int g, int32_t *r_out)
{
    if (g <= 0) return -1;
    for (int l = 0; l < L; ++l) r_out[l] = (l / g) * g;
    return 0;
}

/* Number of layers that keep a cache: those that read their own. */
int oracle_count_owners(int L, const int32_t *r)
{
    int c = 0;
    for (int l = 0; l < L; ++l) c += (r[l] == l);
    return c;
}

/* 2 (K and V) x #cached layers x #kv_heads x head_dim x bytes per element,
 * for n_tokens tokens (Section 1 footnote with #layers -> |S|; M = L(T+t)S of
 * Section 3.1.1). */
int64_t oracle_cache_bytes(int L, const int32_t *r, int Hkv, int D, int bytes_per_elt, int64_t n_tokens)
{
    return (int64_t)2 * oracle_count_owners(L, r) * Hkv * D * bytes_per_elt * n_tokens;
}
