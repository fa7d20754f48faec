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
 *   oracle_append_fp8   the same Update through an FP8 (E4M3, per-row scale) quantiser; the
 *                       attention then sees the dequantised values (scheme stated below).
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
    double **Kq;         /* [L] -> same shape, fp64: layers appended through the fp8 quantiser hold their */
    double **Vq;         /*        DEQUANTISED values here instead (code value x row scale), NULL otherwise */
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
    o->Kq = (double **)calloc((size_t)L, sizeof *o->Kq);
    o->Vq = (double **)calloc((size_t)L, sizeof *o->Vq);
    memcpy(o->r, r, sizeof(int32_t) * (size_t)L);
    return o;
}

void oracle_destroy(oracle_t *o)
{
    if (!o) return;
    for (int l = 0; l < o->L; ++l) { free(o->K[l]); free(o->V[l]); free(o->Kq[l]); free(o->Vq[l]); }
    free(o->K); free(o->V); free(o->Kq); free(o->Vq); free(o->r); free(o);
}

static int has_store(const oracle_t *o, int l) { return o->Kq[l] || o->K[l]; }

/* element of a layer's K (or V) store as fp64: exact bf16 value, or the dequantised fp8 value */
static double k_at(const oracle_t *o, int l, size_t i) { return o->Kq[l] ? o->Kq[l][i] : bf16_to_f64(o->K[l][i]); }
static double v_at(const oracle_t *o, int l, size_t i) { return o->Vq[l] ? o->Vq[l][i] : bf16_to_f64(o->V[l][i]); }

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
    if (o->Kq[layer]) return -4;                          /* a layer is either bf16 or fp8, not both */
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

/* ---- fp8 pages (quantisation is orthogonal to depth-wise sharing: Section 2, Section 5) ----------
 * The paper names KV quantisation as composable with its method and fixes no scheme.  The one used
 * here: OCP FP8 E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, subnormals, largest
 * finite value 448, no infinities) with one fp32 scale per (token, kv head) row, separately for K
 * and V:   amax = max |x| over the row;  scale = amax / 448;  code = E4M3(x * (448 / amax)),
 * round to nearest even, saturating at +-448; a row of zeros has scale 0 and zero codes.  The
 * divisions and the product are single fp32 operations (both sides take the decision in fp32).
 * The value the attention sees is  code value x scale. */

/* value of an E4M3 code (NaN codes 0x7f / 0xff never come out of the quantiser) */
static double e4m3_value(uint8_t c)
{
    int sign = c >> 7, e = (c >> 3) & 15, m = c & 7;
    double v = (e == 0) ? ldexp((double)m, -9) : ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/* fp32 -> E4M3, round to nearest even, saturating */
static uint8_t e4m3_encode(float y)
{
    uint8_t sign = (y < 0.0f || (y == 0.0f && 1.0f / y < 0.0f)) ? 0x80 : 0x00;
    double a = fabs((double)y);
    if (a >= 464.0) return sign | 0x7e;                 /* >= the midpoint above 448 (and beyond): saturate */
    if (a < ldexp(1.0, -6)) {                           /* subnormal range: multiples of 2^-9 */
        double q = a * 512.0;                           /* exact */
        double f = floor(q);
        double r = q - f;
        int n = (int)f;
        if (r > 0.5 || (r == 0.5 && (n & 1))) ++n;      /* ties to even */
        return sign | (uint8_t)n;                       /* n = 8 is the smallest normal, code 0x08 */
    }
    int e;
    double fr = frexp(a, &e);                           /* a = fr * 2^e, fr in [0.5, 1) */
    double mant = fr * 2.0;                             /* [1, 2) */
    int ex = e - 1;                                     /* a = mant * 2^ex */
    double q = (mant - 1.0) * 8.0;                      /* exact in fp64 */
    double f = floor(q);
    double r = q - f;
    int n = (int)f;
    if (r > 0.5 || (r == 0.5 && (n & 1))) ++n;
    if (n == 8) { n = 0; ++ex; }
    int code = ((ex + 7) << 3) | n;
    if (code > 0x7e) code = 0x7e;
    return sign | (uint8_t)code;
}

/* Quantise n rows of D bf16 values: codes [n][D], scales [n]. */
void oracle_quantize_e4m3(const uint16_t *x, int64_t n, int D, uint8_t *codes, float *scales)
{
    for (int64_t i = 0; i < n; ++i) {
        const uint16_t *row = x + (size_t)i * (size_t)D;
        float amax = 0.0f;
        for (int d = 0; d < D; ++d) {
            float v = (float)fabs(bf16_to_f64(row[d]));
            if (v > amax) amax = v;
        }
        volatile float inv = amax > 0.0f ? 448.0f / amax : 0.0f;
        volatile float sc = amax / 448.0f;
        scales[i] = sc;
        for (int d = 0; d < D; ++d) {
            volatile float y = (float)bf16_to_f64(row[d]) * inv;     /* one fp32 product */
            codes[(size_t)i * (size_t)D + (size_t)d] = e4m3_encode(y);
        }
    }
}

double oracle_e4m3_value(int code) { return e4m3_value((uint8_t)code); }

/* "Update" through the quantiser: the layer's store receives the DEQUANTISED rows (code value x
 * scale, exact in fp64); optionally hands back the codes and scales ([n][Hkv][D] and [n][Hkv]). */
int oracle_append_fp8(oracle_t *o, int layer, const uint16_t *K, const uint16_t *V,
                      const int64_t *seq_idx, const int64_t *pos, int64_t n_tok,
                      uint8_t *K_codes, uint8_t *V_codes, float *K_scales, float *V_scales)
{
    if (!o || layer < 0 || layer >= o->L) return -1;
    if (o->K[layer]) return -4;                          /* a layer is either bf16 or fp8, not both */
    size_t row = (size_t)o->Hkv * (size_t)o->D;
    if (!o->Kq[layer]) {
        size_t elems = (size_t)o->B * (size_t)o->n_max * row;
        o->Kq[layer] = (double *)calloc(elems, sizeof(double));
        o->Vq[layer] = (double *)calloc(elems, sizeof(double));
        if (!o->Kq[layer] || !o->Vq[layer]) return -2;
    }
    uint8_t *ck = (uint8_t *)malloc(row), *cv = (uint8_t *)malloc(row);
    float *sk = (float *)malloc(sizeof(float) * (size_t)o->Hkv), *sv = (float *)malloc(sizeof(float) * (size_t)o->Hkv);
    if (!ck || !cv || !sk || !sv) { free(ck); free(cv); free(sk); free(sv); return -2; }
    int rc = 0;
    for (int64_t i = 0; i < n_tok && rc == 0; ++i) {
        if (seq_idx[i] < 0 || seq_idx[i] >= o->B || pos[i] < 0 || pos[i] >= o->n_max) { rc = -3; break; }
        oracle_quantize_e4m3(K + (size_t)i * row, o->Hkv, o->D, ck, sk);
        oracle_quantize_e4m3(V + (size_t)i * row, o->Hkv, o->D, cv, sv);
        size_t at = row_index(o, seq_idx[i], pos[i]);
        for (int h = 0; h < o->Hkv; ++h)
            for (int d = 0; d < o->D; ++d) {
                size_t j = (size_t)h * (size_t)o->D + (size_t)d;
                o->Kq[layer][at + j] = e4m3_value(ck[j]) * (double)sk[h];
                o->Vq[layer][at + j] = e4m3_value(cv[j]) * (double)sv[h];
            }
        if (K_codes) memcpy(K_codes + (size_t)i * row, ck, row);
        if (V_codes) memcpy(V_codes + (size_t)i * row, cv, row);
        if (K_scales) memcpy(K_scales + (size_t)i * (size_t)o->Hkv, sk, sizeof(float) * (size_t)o->Hkv);
        if (V_scales) memcpy(V_scales + (size_t)i * (size_t)o->Hkv, sv, sizeof(float) * (size_t)o->Hkv);
    }
    free(ck); free(cv); free(sk); free(sv);
    return rc;
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
    if (!has_store(o, src)) return -1;
    int G = o->Hq / o->Hkv, kv = h / G, D = o->D;
    const uint16_t *q = Q + ((size_t)b * (size_t)o->Hq + (size_t)h) * (size_t)D;
    double smax = -INFINITY;
    for (int64_t t = 0; t < n; ++t) {
        size_t k0 = row_index(o, b, t) + (size_t)kv * (size_t)D;
        double s = 0.0;
        for (int d = 0; d < D; ++d) s += bf16_to_f64(q[d]) * k_at(o, src, k0 + (size_t)d);
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
    if (!has_store(o, src)) return -1;
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
                size_t v0 = row_index(o, b, t) + (size_t)kv * (size_t)D;
                for (int d = 0; d < D; ++d) y[d] += w[t] * v_at(o, src, v0 + (size_t)d);
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
    if (!has_store(o, src)) return -1;
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
                size_t k0 = row_index(o, b, t) + (size_t)kv * (size_t)D;
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += bf16_to_f64(q[d]) * k_at(o, src, k0 + (size_t)d);
                s[t] = scale * acc;
                if (s[t] > smax) smax = s[t];
            }
            double denom = 0.0;
            for (int64_t t = 0; t < n; ++t) { s[t] = exp(s[t] - smax); denom += s[t]; }
            for (int d = 0; d < D; ++d) y[d] = 0.0;
            for (int64_t t = 0; t < n; ++t) {
                size_t v0 = row_index(o, b, t) + (size_t)kv * (size_t)D;
                double w = s[t] / denom;
                for (int d = 0; d < D; ++d) y[d] += w * v_at(o, src, v0 + (size_t)d);
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
