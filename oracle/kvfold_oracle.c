/*
 * KV-Fold fold-step oracle: plain, slow, fp64 CPU code.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may include, link or
 * call this file; it exists so that the CUDA library can be checked against an
 * independent statement of what the paper's fold step computes.  It shares no
 * code, table or constant with the CUDA library.
 *
 * What is computed (paper Section 2, "KV-Fold" paragraph, the recurrence
 * (K,V)^(t) = F((K,V)^(t-1), x_t) and the foldl form that follows it, and
 * Figure "KV-Fold" for the append / unchanged-prefix statement):
 *
 *   - queries come from the new chunk only;
 *   - the new tokens get positions continued from the absolute position of the
 *     chunk's first token, and RoPE is applied at those positions;
 *   - the chunk's rotated keys and its values are appended to the accumulated
 *     per-layer cache, rows of earlier chunks are never touched again;
 *   - every query attends to all rows of earlier chunks and, inside its own
 *     chunk, to the rows up to and including itself (this is what makes the
 *     fold equal to the paper's FULL condition, one causal pass over the
 *     whole sequence);
 *   - grouped-query attention: query head h reads KV head h / (H / Hkv).
 *
 * All arithmetic is fp64; exp, log, cos, sin, pow are libm's.  There is no
 * blocking, no running ("online") softmax, no fusion: scores for one query
 * row are written out in full, the maximum is subtracted, the row is
 * exponentiated, summed and normalised, and the weighted sum of value rows is
 * taken.  OpenMP is used only across independent (query row, head) pairs.
 *
 * Sink + window variant (the paper's comparison with StreamingLLM: a few sink
 * tokens kept from the start plus a sliding window of recent tokens, eviction
 * that leaves the kept rows at their original positions, no RoPE re-anchoring).
 * With okvf_cache_set_window(n_sink, window) the step behaves as if, after every
 * chunk, all rows had been evicted except the first n_sink and the last
 * `window`: a chunk that starts at row P sees rows r < n_sink, rows
 * P - window <= r < P, and its own rows causally.  Nothing is deleted here (the
 * arrays keep every row); invisible rows get weight exactly zero.
 *
 * Quantised storage (the paper's Discussion: a per-step round trip
 * bf16 -> intN -> bf16 of the stored K/V; the scheme itself is not given).
 * Reading taken here: symmetric int8 per stored row (one token of one KV head),
 * applied once, when the row is appended (a second round trip of an already
 * quantised row would return the same codes up to ties).  With
 * okvf_cache_set_quant(c, bits) (bits = 8 or 4, the two widths the paper
 * reports) a key row is rotated in fp32 (the dtype-faithful operation order),
 * then for the row x[0..d), with Q = 127 for int8 and Q = 7 for int4:
 *     amax = max |x_j|      inv = Q / amax        scale = amax / Q
 *     code_j = clamp(rint(x_j * inv), -Q, Q)      (all in fp32, ties to even)
 *     stored value = bf16(code_j * scale)         (fp32 product, then bf16)
 * and a value row goes through the same three lines unrotated; amax = 0 gives
 * codes 0 and scale 0.  The decision that produces an integer is taken in
 * fp32, the precision the CUDA library takes it in; the attention over the
 * stored values stays in fp64.
 *
 * Readings taken where the paper is silent (each is a build-wide reading):
 *   - RoPE pairs element j with element j + d/2 (rotate-half); the
 *     "interleaved" switch pairs (2j, 2j+1) instead;
 *   - theta = pos * base^(-2j/d), or pos * inv_freq[j] when a table is given;
 *   - keys are cached after rotation, values are cached as given;
 *   - softmax scale defaults to 1/sqrt(d).
 *
 * Every function here is pinned by tests that do not call it back: dense-mask
 * brute force written with complex-number rotations, fold == one causal pass
 * for every chunking, closed forms (first token, constant V, zero Q running
 * mean, position shift invariance, planted key), the paper's printed cache
 * sizes for the accounting function, and a half-ulp bound for the
 * dtype-faithful rotation.  No function is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct okvf_cache {
    int n_q_heads, n_kv_heads, head_dim, interleaved;
    int64_t capacity, len;
    int64_t n_sink, window; /* window <= 0: every earlier row is visible */
    int quant_bits;         /* 0: rows are stored as given; 8 / 4: int8 / int4 round trip at append */
    double scale;
    double *inv_freq; /* [head_dim/2] */
    double *K;        /* [n_kv_heads][capacity][head_dim], rotated keys */
    double *V;        /* [n_kv_heads][capacity][head_dim] */
} okvf_cache;

/* inv_freq[j] = base^(-2j/d)  (RoFormer's frequencies, cited by Section 2). */
void okvf_inv_freq(double rope_base, int head_dim, double *out) {
    for (int j = 0; j < head_dim / 2; ++j)
        out[j] = pow(rope_base, -2.0 * (double)j / (double)head_dim);
}

okvf_cache *okvf_cache_create(int n_q_heads, int n_kv_heads, int head_dim, int64_t capacity,
                              double rope_base, double softmax_scale, int interleaved,
                              const double *inv_freq_or_null) {
    if (n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads != 0) return NULL;
    if (head_dim <= 0 || head_dim % 2 != 0 || capacity <= 0) return NULL;
    okvf_cache *c = (okvf_cache *)calloc(1, sizeof(okvf_cache));
    if (!c) return NULL;
    c->n_q_heads = n_q_heads;
    c->n_kv_heads = n_kv_heads;
    c->head_dim = head_dim;
    c->interleaved = interleaved;
    c->capacity = capacity;
    c->len = 0; /* the empty accumulator (emptyset, emptyset) of the foldl form */
    c->scale = softmax_scale != 0.0 ? softmax_scale : 1.0 / sqrt((double)head_dim);
    c->inv_freq = (double *)malloc(sizeof(double) * (size_t)(head_dim / 2));
    size_t plane = (size_t)n_kv_heads * (size_t)capacity * (size_t)head_dim;
    c->K = (double *)malloc(sizeof(double) * plane);
    c->V = (double *)malloc(sizeof(double) * plane);
    if (!c->inv_freq || !c->K || !c->V) {
        free(c->inv_freq); free(c->K); free(c->V); free(c);
        return NULL;
    }
    if (inv_freq_or_null) memcpy(c->inv_freq, inv_freq_or_null, sizeof(double) * (size_t)(head_dim / 2));
    else okvf_inv_freq(rope_base, head_dim, c->inv_freq);
    return c;
}

void okvf_cache_destroy(okvf_cache *c) {
    if (!c) return;
    free(c->inv_freq); free(c->K); free(c->V); free(c);
}

int64_t okvf_cache_len(const okvf_cache *c) { return c->len; }
void okvf_cache_reset(okvf_cache *c) { c->len = 0; }
/* Quantised storage (see the header): bits = 0, 8 or 4.  Returns 0, or 1 for other values. */
int okvf_cache_set_quant(okvf_cache *c, int bits) {
    if (bits != 0 && bits != 8 && bits != 4) return 1;
    c->quant_bits = bits;
    return 0;
}
/* Sink + window variant (see the header); window <= 0 switches it off. */
void okvf_cache_set_window(okvf_cache *c, int64_t n_sink, int64_t window) {
    c->n_sink = n_sink < 0 ? 0 : n_sink;
    c->window = window;
}
const double *okvf_cache_k(const okvf_cache *c) { return c->K; }
const double *okvf_cache_v(const okvf_cache *c) { return c->V; }

/* Bytes of K and V held for `tokens` tokens of one layer: the per-token figure
 * of Section 5 (KV heads x head_dim x (K,V) x bytes per element). */
int64_t okvf_cache_bytes(int n_kv_heads, int head_dim, int64_t tokens, int elem_bytes) {
    return (int64_t)2 * n_kv_heads * head_dim * elem_bytes * tokens;
}

/* RoPE on one head vector of length d at position pos, fp64. */
static void rope_vec(const double *x, double *y, int d, int64_t pos, const double *inv_freq,
                     int interleaved) {
    int half = d / 2;
    for (int j = 0; j < half; ++j) {
        double theta = (double)pos * inv_freq[j];
        double c = cos(theta), s = sin(theta);
        int a = interleaved ? 2 * j : j;
        int b = interleaved ? 2 * j + 1 : j + half;
        y[a] = x[a] * c - x[b] * s;
        y[b] = x[b] * c + x[a] * s;
    }
}

/* x, y: [n][heads][d]; token i is rotated at position pos0 + i. */
void okvf_rope_fp64(const double *x, int64_t n, int heads, int d, int64_t pos0,
                    const double *inv_freq, int interleaved, double *y) {
    for (int64_t i = 0; i < n; ++i)
        for (int h = 0; h < heads; ++h)
            rope_vec(x + ((size_t)i * heads + h) * d, y + ((size_t)i * heads + h) * d, d, pos0 + i,
                     inv_freq, interleaved);
}

/* Round an fp32 value to bf16 (round to nearest, ties to even), returned as the
 * fp32 value that the bf16 pattern stands for.  NaN is not expected. */
static float round_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    u &= 0xFFFF0000u;
    memcpy(&f, &u, 4);
    return f;
}

/*
 * "Dtype-faithful" rotation: the bit pattern the cache must hold.
 * theta and its cosine and sine are taken in fp64 and rounded once to fp32;
 * the rotation is then two fp32 operations per output: the cross product is
 * rounded to fp32 first, then one fused multiply-add:
 *     lo' = fma(x_lo, c, -(x_hi * s))        hi' = fma(x_hi, c, (x_lo * s))
 * and, for a bf16 cache, one round-to-nearest-even to bf16.
 * (This file must be compiled with -ffp-contract=off so that the compiler
 * fuses nothing else.)
 */
void okvf_rope_faithful(const float *x, int64_t n, int heads, int d, int64_t pos0,
                        const double *inv_freq, int interleaved, int to_bf16, float *y) {
    int half = d / 2;
    for (int64_t i = 0; i < n; ++i) {
        for (int j = 0; j < half; ++j) {
            double theta = (double)(pos0 + i) * inv_freq[j];
            float c = (float)cos(theta), s = (float)sin(theta);
            int a = interleaved ? 2 * j : j;
            int b = interleaved ? 2 * j + 1 : j + half;
            for (int h = 0; h < heads; ++h) {
                const float *xv = x + ((size_t)i * heads + h) * d;
                float *yv = y + ((size_t)i * heads + h) * d;
                float cross_lo = xv[b] * s;
                float cross_hi = xv[a] * s;
                float lo = fmaf(xv[a], c, -cross_lo);
                float hi = fmaf(xv[b], c, cross_hi);
                yv[a] = to_bf16 ? round_bf16(lo) : lo;
                yv[b] = to_bf16 ? round_bf16(hi) : hi;
            }
        }
    }
}

/*
 * Round trip of one row x[0..d) (fp32 in) through `bits`-bit codes (8 or 4): codes (optional, as
 * int32), the row's scale and the stored values y (the bf16 values, held in fp32).  See the header
 * for the arithmetic.
 */
void okvf_quant_row(const float *x, int d, int bits, int32_t *codes, float *scale_out, float *y) {
    const float Q = bits == 4 ? 7.0f : 127.0f;
    float amax = 0.0f;
    for (int j = 0; j < d; ++j) {
        float a = fabsf(x[j]);
        if (a > amax) amax = a;
    }
    float inv = amax > 0.0f ? Q / amax : 0.0f;
    float scale = amax / Q;
    for (int j = 0; j < d; ++j) {
        float r = rintf(x[j] * inv); /* default rounding mode: to nearest, ties to even */
        if (r > Q) r = Q;
        if (r < -Q) r = -Q;
        if (codes) codes[j] = (int32_t)r;
        if (y) y[j] = round_bf16(r * scale);
    }
    if (scale_out) *scale_out = scale;
}

/*
 * One fold step.
 *   q      [n][H][d]    queries of the new chunk, before rotation
 *   k_new  [n][Hkv][d]  keys of the new chunk, before rotation
 *   v_new  [n][Hkv][d]  values of the new chunk
 *   pos0   absolute position of the chunk's first token
 *   rows   optional list of in-chunk query indices to evaluate (NULL: all n);
 *          the append always covers the whole chunk
 *   out    [n_out][H][d]  attention output for the evaluated rows
 *   lse    [n_out][H]     optional: log of the softmax denominator (natural log)
 *   rowsum [n_out][H]     optional: sum of the normalised weights (should be 1)
 * Returns 0, or 1 bad argument, 2 capacity exceeded (nothing is changed then).
 */
int okvf_fold_step(okvf_cache *c, const double *q, const double *k_new, const double *v_new,
                   int64_t n, int64_t pos0, const int32_t *rows, int64_t n_rows, double *out,
                   double *lse, double *rowsum) {
    if (!c || !q || !k_new || !v_new || !out || n <= 0) return 1;
    if (c->len + n > c->capacity) return 2;
    const int H = c->n_q_heads, Hkv = c->n_kv_heads, d = c->head_dim, G = H / Hkv;
    const int64_t P = c->len, cap = c->capacity;
    if (rows)
        for (int64_t o = 0; o < n_rows; ++o)
            if (rows[o] < 0 || rows[o] >= n) return 1;

    /* append: rotated keys and raw values become rows P .. P+n-1 */
    for (int64_t i = 0; i < n; ++i) {
        for (int g = 0; g < Hkv; ++g) {
            size_t dst = ((size_t)g * cap + (size_t)(P + i)) * d;
            size_t src = ((size_t)i * Hkv + g) * d;
            if (c->quant_bits != 0) {
                /* the row as the library holds it: fp32 rotation in the faithful order, int8 round
                 * or int4 round trip, bf16; the value row likewise without the rotation */
                float xf[512], rot[512], st[512];
                if (d > 512) return 1;
                for (int e = 0; e < d; ++e) xf[e] = (float)k_new[src + e];
                okvf_rope_faithful(xf, 1, 1, d, pos0 + i, c->inv_freq, c->interleaved, 0, rot);
                okvf_quant_row(rot, d, c->quant_bits, NULL, NULL, st);
                for (int e = 0; e < d; ++e) c->K[dst + e] = (double)st[e];
                for (int e = 0; e < d; ++e) xf[e] = (float)v_new[src + e];
                okvf_quant_row(xf, d, c->quant_bits, NULL, NULL, st);
                for (int e = 0; e < d; ++e) c->V[dst + e] = (double)st[e];
                continue;
            }
            rope_vec(k_new + src, c->K + dst, d, pos0 + i, c->inv_freq, c->interleaved);
            memcpy(c->V + dst, v_new + src, sizeof(double) * (size_t)d);
        }
    }

    const int64_t n_out = rows ? n_rows : n;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int64_t o = 0; o < n_out; ++o) {
        for (int h = 0; h < H; ++h) {
            const int64_t i = rows ? rows[o] : o;
            const int g = h / G;
            const int64_t visible = P + i + 1; /* whole prefix, then rows 0..i of the chunk */
            double *qr = (double *)malloc(sizeof(double) * (size_t)d);
            double *s = (double *)malloc(sizeof(double) * (size_t)visible);
            rope_vec(q + ((size_t)i * H + h) * d, qr, d, pos0 + i, c->inv_freq, c->interleaved);
            const double *Kg = c->K + (size_t)g * cap * d;
            const double *Vg = c->V + (size_t)g * cap * d;
            double m = -INFINITY;
            for (int64_t r = 0; r < visible; ++r) {
                /* sink + window: an earlier chunk's row survives eviction only as a sink or
                 * among the last `window` rows before this chunk */
                if (c->window > 0 && r < P && r >= c->n_sink && r < P - c->window) {
                    s[r] = -INFINITY;
                    continue;
                }
                double acc = 0.0;
                for (int e = 0; e < d; ++e) acc += qr[e] * Kg[(size_t)r * d + e];
                s[r] = acc * c->scale;
                if (s[r] > m) m = s[r];
            }
            double l = 0.0;
            for (int64_t r = 0; r < visible; ++r) {
                s[r] = exp(s[r] - m);
                l += s[r];
            }
            double *dst = out + ((size_t)o * H + h) * d;
            for (int e = 0; e < d; ++e) dst[e] = 0.0;
            double wsum = 0.0;
            for (int64_t r = 0; r < visible; ++r) {
                double w = s[r] / l;
                wsum += w;
                for (int e = 0; e < d; ++e) dst[e] += w * Vg[(size_t)r * d + e];
            }
            if (lse) lse[(size_t)o * H + h] = m + log(l);
            if (rowsum) rowsum[(size_t)o * H + h] = wsum;
            free(qr);
            free(s);
        }
    }
    c->len = P + n; /* the accumulator handed to the next step */
    return 0;
}
