/*
 * matkv_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * Plain, slow, fp64 CPU statement of what the MatKV attention path computes.
 * It shares no code, header, table or helper with the CUDA library and is
 * called only from the tests, the smoke check and the benchmark's CPU-baseline
 * leg.
 *
 * What is computed (paper, Section III-B "Materializing and Retrieving KV
 * Caches" and Section IV "Avoiding Prefill Using KV in SSD"): the precomputed
 * K,V of the retrieved document chunks are placed BEFORE the query, each chunk
 * having been materialised alone with its tokens at positions 0..len-1, and
 * only the query (and what is generated after it) attends to them.  On this
 * path the result is therefore exact softmax attention of each query row over
 * the key/value set
 *
 *     chunk_0 || chunk_1 || ... || chunk_{n-1} || tail[0 .. v)
 *
 * where the chunk bytes are used verbatim (no re-rotation, no cross-chunk
 * mask: every chunk token is visible) and `tail` holds the K,V of the query
 * suffix and of the generated tokens, of which query row i sees the first
 * v_i (causal inside the tail).  Grouped-query attention: query head h reads
 * KV head floor(h / G), G = Hq / Hkv.  The paper prints no formula for
 * attention; the definition used is the textbook one:
 *
 *     s_j = scale * <q, K_j>,  m = max_j s_j,
 *     p_j = exp(s_j - m) / sum_j exp(s_j - m),
 *     o   = sum_j p_j V_j,     lse = m + ln sum_j exp(s_j - m).
 *
 * Three separately written evaluators:
 *   O1  matkv_oracle_attend_walk   walks the segments in place, two passes;
 *   O2  matkv_oracle_attend_brute  copies the visible set into flat arrays,
 *                                   full score matrix with a boolean mask;
 *   O3  matkv_oracle_attend_merge  attention per segment, then the
 *                                   log-sum-exp merge of the per-segment
 *                                   results (the identity that lets
 *                                   independently materialised chunks compose).
 *
 * Inputs are bf16 bit patterns (uint16_t), widened exactly to double.
 * Chunk blob layout: [L][2 (K then V)][Hkv][len][D], contiguous.
 * Tail layout for one (request, layer): [Hkv][cap][D].
 * Query layout: [n_q][Hq][D].  Outputs: o [n_q][Hq][D], lse [n_q][Hq], double.
 * A row with an empty visible set gets o = 0 and lse = -inf.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t n_layers, n_q_heads, n_kv_heads, head_dim;
    double scale;
} matkv_oracle_shape;

static double widen(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* K (kv=0) or V (kv=1) row `t` of (layer, kv head g) inside one chunk blob */
static const uint16_t *blob_row(const matkv_oracle_shape *sh, const uint16_t *blob, int32_t len,
                                int32_t layer, int kv, int32_t g, int32_t t) {
    size_t slab = ((size_t)layer * 2 + (size_t)kv) * (size_t)sh->n_kv_heads + (size_t)g;
    return blob + (slab * (size_t)len + (size_t)t) * (size_t)sh->head_dim;
}

static double dot_row(const uint16_t *q, const uint16_t *k, int32_t D) {
    double s = 0.0;
    for (int32_t d = 0; d < D; ++d) s += widen(q[d]) * widen(k[d]);
    return s;
}

/* ---- O1: segment walk ---------------------------------------------------- */
int matkv_oracle_attend_walk(const matkv_oracle_shape *sh, int32_t layer, int32_t n_seg,
                             const uint16_t *const *seg_blob, const int32_t *seg_len,
                             const uint16_t *tail_k, const uint16_t *tail_v, int32_t tail_cap,
                             int32_t n_q, const uint16_t *q, const int32_t *visible, double *o,
                             double *lse) {
    const int32_t D = sh->head_dim, Hq = sh->n_q_heads, Hkv = sh->n_kv_heads, G = Hq / Hkv;
    int64_t n_chunk_tok = 0;
    for (int32_t c = 0; c < n_seg; ++c) n_chunk_tok += seg_len[c];
    double *s = (double *)malloc(sizeof(double) * (size_t)(n_chunk_tok + tail_cap + 1));
    if (!s) return -1;
    for (int32_t i = 0; i < n_q; ++i) {
        const int32_t v = visible[i];
        if (v < 0 || v > tail_cap) { free(s); return -2; }
        for (int32_t h = 0; h < Hq; ++h) {
            const int32_t g = h / G;
            const uint16_t *qv = q + ((size_t)i * Hq + h) * D;
            double *oo = o + ((size_t)i * Hq + h) * D;
            /* pass 1: scores and their maximum */
            int64_t n = 0;
            double m = -INFINITY;
            for (int32_t c = 0; c < n_seg; ++c)
                for (int32_t t = 0; t < seg_len[c]; ++t) {
                    s[n] = sh->scale * dot_row(qv, blob_row(sh, seg_blob[c], seg_len[c], layer, 0, g, t), D);
                    if (s[n] > m) m = s[n];
                    ++n;
                }
            for (int32_t t = 0; t < v; ++t) {
                s[n] = sh->scale * dot_row(qv, tail_k + ((size_t)g * tail_cap + t) * D, D);
                if (s[n] > m) m = s[n];
                ++n;
            }
            for (int32_t d = 0; d < D; ++d) oo[d] = 0.0;
            if (n == 0) { lse[(size_t)i * Hq + h] = -INFINITY; continue; }
            /* pass 2: weights, normaliser, weighted sum of V */
            double z = 0.0;
            for (int64_t j = 0; j < n; ++j) { s[j] = exp(s[j] - m); z += s[j]; }
            n = 0;
            for (int32_t c = 0; c < n_seg; ++c)
                for (int32_t t = 0; t < seg_len[c]; ++t) {
                    const uint16_t *vr = blob_row(sh, seg_blob[c], seg_len[c], layer, 1, g, t);
                    const double p = s[n++] / z;
                    for (int32_t d = 0; d < D; ++d) oo[d] += p * widen(vr[d]);
                }
            for (int32_t t = 0; t < v; ++t) {
                const uint16_t *vr = tail_v + ((size_t)g * tail_cap + t) * D;
                const double p = s[n++] / z;
                for (int32_t d = 0; d < D; ++d) oo[d] += p * widen(vr[d]);
            }
            lse[(size_t)i * Hq + h] = m + log(z);
        }
    }
    free(s);
    return 0;
}

/* ---- O2: brute force on a materialised concatenation ---------------------- */
int matkv_oracle_attend_brute(const matkv_oracle_shape *sh, int32_t layer, int32_t n_seg,
                              const uint16_t *const *seg_blob, const int32_t *seg_len,
                              const uint16_t *tail_k, const uint16_t *tail_v, int32_t tail_cap,
                              int32_t n_q, const uint16_t *q, const int32_t *visible, double *o,
                              double *lse) {
    const int32_t D = sh->head_dim, Hq = sh->n_q_heads, Hkv = sh->n_kv_heads, G = Hq / Hkv;
    int64_t n_chunk_tok = 0;
    int32_t vmax = 0;
    for (int32_t c = 0; c < n_seg; ++c) n_chunk_tok += seg_len[c];
    for (int32_t i = 0; i < n_q; ++i) {
        if (visible[i] < 0 || visible[i] > tail_cap) return -2;
        if (visible[i] > vmax) vmax = visible[i];
    }
    const int64_t n_kv = n_chunk_tok + vmax;
    uint16_t *Kf = (uint16_t *)malloc(sizeof(uint16_t) * (size_t)(n_kv + 1) * D);
    uint16_t *Vf = (uint16_t *)malloc(sizeof(uint16_t) * (size_t)(n_kv + 1) * D);
    double *S = (double *)malloc(sizeof(double) * (size_t)n_q * (size_t)(n_kv + 1));
    unsigned char *mask = (unsigned char *)malloc((size_t)n_q * (size_t)(n_kv + 1));
    if (!Kf || !Vf || !S || !mask) { free(Kf); free(Vf); free(S); free(mask); return -1; }
    /* the mask depends on the row only: all chunk tokens, then a causal tail */
    for (int32_t i = 0; i < n_q; ++i)
        for (int64_t j = 0; j < n_kv; ++j)
            mask[(size_t)i * n_kv + j] = (j < n_chunk_tok) || (j - n_chunk_tok < visible[i]);
    for (int32_t g = 0; g < Hkv; ++g) {
        /* concatenate the chunks' rows, then the tail's, by plain copies */
        int64_t at = 0;
        for (int32_t c = 0; c < n_seg; ++c) {
            memcpy(Kf + at * D, blob_row(sh, seg_blob[c], seg_len[c], layer, 0, g, 0), sizeof(uint16_t) * (size_t)seg_len[c] * D);
            memcpy(Vf + at * D, blob_row(sh, seg_blob[c], seg_len[c], layer, 1, g, 0), sizeof(uint16_t) * (size_t)seg_len[c] * D);
            at += seg_len[c];
        }
        if (vmax > 0) {
            memcpy(Kf + at * D, tail_k + (size_t)g * tail_cap * D, sizeof(uint16_t) * (size_t)vmax * D);
            memcpy(Vf + at * D, tail_v + (size_t)g * tail_cap * D, sizeof(uint16_t) * (size_t)vmax * D);
        }
        for (int32_t hh = 0; hh < G; ++hh) {
            const int32_t h = g * G + hh;
            for (int32_t i = 0; i < n_q; ++i)
                for (int64_t j = 0; j < n_kv; ++j)
                    S[(size_t)i * n_kv + j] = sh->scale * dot_row(q + ((size_t)i * Hq + h) * D, Kf + j * D, D);
            for (int32_t i = 0; i < n_q; ++i) {
                double *oo = o + ((size_t)i * Hq + h) * D;
                double m = -INFINITY, z = 0.0;
                for (int32_t d = 0; d < D; ++d) oo[d] = 0.0;
                for (int64_t j = 0; j < n_kv; ++j)
                    if (mask[(size_t)i * n_kv + j] && S[(size_t)i * n_kv + j] > m) m = S[(size_t)i * n_kv + j];
                if (m == -INFINITY) { lse[(size_t)i * Hq + h] = -INFINITY; continue; }
                for (int64_t j = 0; j < n_kv; ++j)
                    if (mask[(size_t)i * n_kv + j]) z += exp(S[(size_t)i * n_kv + j] - m);
                for (int64_t j = 0; j < n_kv; ++j) {
                    if (!mask[(size_t)i * n_kv + j]) continue;
                    const double p = exp(S[(size_t)i * n_kv + j] - m) / z;
                    for (int32_t d = 0; d < D; ++d) oo[d] += p * widen(Vf[j * D + d]);
                }
                lse[(size_t)i * Hq + h] = m + log(z);
            }
        }
    }
    free(Kf); free(Vf); free(S); free(mask);
    return 0;
}

/* ---- log-sum-exp merge of partial attentions ------------------------------ */
/* parts: o_part [n_parts][D], lse_part [n_parts]; parts with lse = -inf are empty. */
void matkv_oracle_lse_merge(int32_t n_parts, int32_t D, const double *o_part, const double *lse_part,
                            double *o, double *lse) {
    double m = -INFINITY, z = 0.0;
    for (int32_t c = 0; c < n_parts; ++c)
        if (lse_part[c] > m) m = lse_part[c];
    for (int32_t d = 0; d < D; ++d) o[d] = 0.0;
    if (m == -INFINITY) { *lse = -INFINITY; return; }
    for (int32_t c = 0; c < n_parts; ++c)
        if (lse_part[c] != -INFINITY) z += exp(lse_part[c] - m);
    *lse = m + log(z);
    for (int32_t c = 0; c < n_parts; ++c) {
        if (lse_part[c] == -INFINITY) continue;
        const double w = exp(lse_part[c] - *lse);
        for (int32_t d = 0; d < D; ++d) o[d] += w * o_part[(size_t)c * D + d];
    }
}

/* attention of one query vector over one contiguous run of rows */
static void attend_run(const matkv_oracle_shape *sh, const uint16_t *qv, const uint16_t *k,
                       const uint16_t *v, int32_t n, double *o, double *lse) {
    const int32_t D = sh->head_dim;
    for (int32_t d = 0; d < D; ++d) o[d] = 0.0;
    if (n <= 0) { *lse = -INFINITY; return; }
    double *s = (double *)malloc(sizeof(double) * (size_t)n);
    double m = -INFINITY, z = 0.0;
    for (int32_t t = 0; t < n; ++t) {
        s[t] = sh->scale * dot_row(qv, k + (size_t)t * D, D);
        if (s[t] > m) m = s[t];
    }
    for (int32_t t = 0; t < n; ++t) z += exp(s[t] - m);
    for (int32_t t = 0; t < n; ++t) {
        const double p = exp(s[t] - m) / z;
        for (int32_t d = 0; d < D; ++d) o[d] += p * widen(v[(size_t)t * D + d]);
    }
    *lse = m + log(z);
    free(s);
}

/* ---- O3: per-segment attention + merge ------------------------------------ */
int matkv_oracle_attend_merge(const matkv_oracle_shape *sh, int32_t layer, int32_t n_seg,
                              const uint16_t *const *seg_blob, const int32_t *seg_len,
                              const uint16_t *tail_k, const uint16_t *tail_v, int32_t tail_cap,
                              int32_t n_q, const uint16_t *q, const int32_t *visible, double *o,
                              double *lse) {
    const int32_t D = sh->head_dim, Hq = sh->n_q_heads, Hkv = sh->n_kv_heads, G = Hq / Hkv;
    double *po = (double *)malloc(sizeof(double) * (size_t)(n_seg + 1) * D);
    double *pl = (double *)malloc(sizeof(double) * (size_t)(n_seg + 1));
    if (!po || !pl) { free(po); free(pl); return -1; }
    for (int32_t i = 0; i < n_q; ++i) {
        if (visible[i] < 0 || visible[i] > tail_cap) { free(po); free(pl); return -2; }
        for (int32_t h = 0; h < Hq; ++h) {
            const int32_t g = h / G;
            const uint16_t *qv = q + ((size_t)i * Hq + h) * D;
            for (int32_t c = 0; c < n_seg; ++c)
                attend_run(sh, qv, blob_row(sh, seg_blob[c], seg_len[c], layer, 0, g, 0),
                           blob_row(sh, seg_blob[c], seg_len[c], layer, 1, g, 0), seg_len[c],
                           po + (size_t)c * D, pl + c);
            attend_run(sh, qv, tail_k + (size_t)g * tail_cap * D, tail_v + (size_t)g * tail_cap * D,
                       visible[i], po + (size_t)n_seg * D, pl + n_seg);
            matkv_oracle_lse_merge(n_seg + 1, D, po, pl, o + ((size_t)i * Hq + h) * D,
                                   lse + (size_t)i * Hq + h);
        }
    }
    free(po); free(pl);
    return 0;
}

/* ---- optional rotary position embedding (test-only feature) --------------- */
/* Rotate-half pairing (d, d + D/2), angle pos * theta^(-2d/D); input and output are
 * bf16 bits, the rotation is done in fp64 and rounded to bf16 nearest-even, which
 * is what a model would have handed to the attention path.  n_vec vectors of D. */
static uint16_t narrow_rne(double x) {
    float f = (float)x; /* double -> float is correctly rounded; bf16 keeps 8 bits so   */
    uint32_t u;         /* double rounding could differ only on exact fp32 ties: accept */
    memcpy(&u, &f, sizeof u);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

void matkv_oracle_rope(int32_t n_vec, int32_t D, double theta, const int64_t *pos,
                       const uint16_t *in, uint16_t *out) {
    const int32_t half = D / 2;
    for (int32_t i = 0; i < n_vec; ++i)
        for (int32_t d = 0; d < half; ++d) {
            const double ang = (double)pos[i] * pow(theta, -2.0 * (double)d / (double)D);
            const double c = cos(ang), s = sin(ang);
            const double a = widen(in[(size_t)i * D + d]), b = widen(in[(size_t)i * D + d + half]);
            out[(size_t)i * D + d] = narrow_rne(a * c - b * s);
            out[(size_t)i * D + d + half] = narrow_rne(b * c + a * s);
        }
}

/* ---- fp8 chunk codec (compressed store; the paper names KV compression as the lever on storage cost,
 *      "Total Cost of Ownership" discussion, without fixing a format) -------------------------------------
 * Format taken here: every block of up to 64 consecutive tokens of one (layer, K or V, KV head) slab, i.e.
 * up to 64 x D values, shares one power-of-two scale 2^e (e an int8); each value is stored as an e4m3 code
 * (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities, largest finite 448; the two NaN codes
 * 0x7f / 0xff are never produced).  A stored value stands for  value(code) * 2^e,  which is always exactly
 * representable in bf16, so attention over a compressed chunk is attention over ordinary bf16 numbers.
 *   e      = the smallest integer with  amax * 2^-e <= 448  (amax = largest magnitude in the block),
 *            0 for an all-zero block, clamped to [-127, 127];
 *   code   = the e4m3 number nearest to  x * 2^-e,  ties to the code with an even mantissa.
 * Inputs must be finite. */
double matkv_oracle_e4m3_value(uint8_t code) {
    const int s = code >> 7, E = (code >> 3) & 15, M = code & 7;
    const double mag = E == 0 ? ldexp((double)M, -9) : ldexp(1.0 + (double)M / 8.0, E - 7);
    return s ? -mag : mag;
}

/* nearest e4m3 code by exhaustive search over the 127 finite magnitudes (0x00 .. 0x7e) */
uint8_t matkv_oracle_e4m3_encode(double x) {
    const double a = fabs(x);
    int best = 0;
    double best_d = a; /* distance to code 0 */
    for (int c = 1; c <= 0x7e; ++c) {
        const double d = fabs(a - matkv_oracle_e4m3_value((uint8_t)c));
        if (d < best_d || (d == best_d && (c & 1) == 0)) { /* a tie is between neighbours: keep the even one */
            best_d = d;
            best = c;
        }
    }
    if (best == 0) return 0; /* zero carries no sign */
    return (uint8_t)(best | (x < 0 ? 0x80 : 0));
}

int32_t matkv_oracle_fp8_block_exponent(double amax) {
    if (amax == 0.0) return 0;
    int32_t e = -200;
    while (ldexp(amax, -e) > 448.0) ++e;
    if (e < -127) e = -127;
    if (e > 127) e = 127;
    return e;
}

/* One block: n_el bf16 values -> n_el codes and the block's exponent. */
void matkv_oracle_fp8_quantize_block(int64_t n_el, const uint16_t *x, uint8_t *codes, int8_t *e_out) {
    double amax = 0.0;
    for (int64_t i = 0; i < n_el; ++i) amax = fmax(amax, fabs(widen(x[i])));
    const int32_t e = matkv_oracle_fp8_block_exponent(amax);
    for (int64_t i = 0; i < n_el; ++i) codes[i] = matkv_oracle_e4m3_encode(ldexp(widen(x[i]), -e));
    *e_out = (int8_t)e;
}

/* A whole chunk blob [L][2][Hkv][len][D] bf16 -> codes of the same shape and exponents [L][2][Hkv][ceil(len/64)]. */
void matkv_oracle_fp8_quantize_blob(const matkv_oracle_shape *sh, int32_t len, const uint16_t *blob, uint8_t *codes,
                                    int8_t *exps) {
    const int32_t D = sh->head_dim, nb = (len + 63) / 64;
    const int64_t n_slab = (int64_t)sh->n_layers * 2 * sh->n_kv_heads;
    for (int64_t s = 0; s < n_slab; ++s)
        for (int32_t b = 0; b < nb; ++b) {
            const int32_t t0 = b * 64, nt = len - t0 < 64 ? len - t0 : 64;
            const int64_t off = (s * len + t0) * D;
            matkv_oracle_fp8_quantize_block((int64_t)nt * D, blob + off, codes + off, exps + s * nb + b);
        }
}

/* ... and back: bf16 bit patterns of value(code) * 2^e (exact). */
void matkv_oracle_fp8_dequantize_blob(const matkv_oracle_shape *sh, int32_t len, const uint8_t *codes, const int8_t *exps,
                                      uint16_t *blob) {
    const int32_t D = sh->head_dim, nb = (len + 63) / 64;
    const int64_t n_slab = (int64_t)sh->n_layers * 2 * sh->n_kv_heads;
    for (int64_t s = 0; s < n_slab; ++s)
        for (int32_t t = 0; t < len; ++t)
            for (int32_t d = 0; d < D; ++d) {
                const int64_t i = (s * len + t) * D + d;
                blob[i] = narrow_rne(ldexp(matkv_oracle_e4m3_value(codes[i]), exps[s * nb + t / 64]));
            }
}
