/*
 * CPU oracle (fp64, single-threaded, no blocking, no fusion).  See
 * kvbfp_oracle.h for the role of this file and the passages it follows.
 * TEST INFRASTRUCTURE ONLY: nothing in the CUDA library links or calls it.
 */
#include "kvbfp_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ inputs */

/* Widen one input element to double (exact for f32 and bf16). */
static double load_elem(const void* base, int dt, int64_t i) {
    if (dt == ORACLE_F32) return (double)((const float*)base)[i];
    if (dt == ORACLE_F64) return ((const double*)base)[i];
    /* bf16 = upper half of an IEEE binary32 */
    uint32_t bits = (uint32_t)((const uint16_t*)base)[i] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static int format_ok(const oracle_format* f) {
    if (!f) return 0;
    if (f->batch < 1 || f->n_kv_heads < 1 || f->head_dim < 1 || f->max_seq < 1) return 0;
    if (f->block < 1 || f->head_dim % f->block != 0) return 0;
    if (f->mant_bits < 2 || f->mant_bits > 8) return 0;
    if ((f->head_dim * f->mant_bits) % 8 != 0) return 0;
    return 1;
}

size_t oracle_row_mant_bytes(const oracle_format* f) {
    return (size_t)f->head_dim * (size_t)f->mant_bits / 8;
}
size_t oracle_row_exp_bytes(const oracle_format* f) {
    return (size_t)(f->head_dim / f->block);
}

/* ------------------------------------------------- Eq. (1) and the BFP cast */

/* The exponent byte stores E + 127 where 2^E is the power of two at or below
 * the block's largest magnitude (E clamped below at -127).  The mantissa's unit
 * weight is 2^(E - (p-2)), so the largest element lands in [2^(p-2), 2^(p-1)). */
double oracle_bfp_value(int M, int e8, int p) {
    return ldexp((double)M, e8 - 127 - (p - 2));
}

int oracle_bfp_cast_block(const double* x, int n, int p, int* e8_out, int* M_out) {
    const int qmax = (1 << (p - 1)) - 1;
    double amax = 0.0;
    for (int j = 0; j < n; ++j) {
        if (!isfinite(x[j])) return ORACLE_NONFINITE;
        double a = fabs(x[j]);
        if (a > amax) amax = a;
    }
    int E = -127;
    if (amax > 0.0) {
        int ex;
        (void)frexp(amax, &ex);     /* amax = m * 2^ex, m in [0.5, 1)  =>  floor(log2 amax) = ex-1 */
        E = ex - 1;
        if (E < -127) E = -127;
    }
    if (E > 127) return ORACLE_NONFINITE;   /* beyond binary32 range: not a valid input */
    const int e = E - (p - 2);
    for (int j = 0; j < n; ++j) {
        double t = ldexp(x[j], -e);          /* exact power-of-two scaling */
        double r = nearbyint(t);             /* default rounding mode: to nearest, ties to even */
        if (r > (double)qmax) r = (double)qmax;
        if (r < (double)-qmax) r = (double)-qmax;
        M_out[j] = (int)r;
    }
    *e8_out = E + 127;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ packing */

void oracle_pack_mantissas(const int* M, int count, int p, uint8_t* bytes) {
    size_t nbytes = ((size_t)count * (size_t)p + 7) / 8;
    memset(bytes, 0, nbytes);
    const unsigned mask = (1u << p) - 1u;
    for (int j = 0; j < count; ++j) {
        unsigned field = (unsigned)(M[j] + (1 << (p - 1))) & mask;   /* excess-2^(p-1) code, p bits */
        for (int k = 0; k < p; ++k) {
            size_t bit = (size_t)j * (size_t)p + (size_t)k;
            if ((field >> k) & 1u) bytes[bit >> 3] |= (uint8_t)(1u << (bit & 7));
        }
    }
}

void oracle_unpack_mantissas(const uint8_t* bytes, int count, int p, int* M) {
    for (int j = 0; j < count; ++j) {
        unsigned field = 0;
        for (int k = 0; k < p; ++k) {
            size_t bit = (size_t)j * (size_t)p + (size_t)k;
            field |= (unsigned)((bytes[bit >> 3] >> (bit & 7)) & 1u) << k;
        }
        M[j] = (int)field - (1 << (p - 1));   /* excess-2^(p-1) code */
    }
}

/* ------------------------------------------------------ Algorithm 1, steps 1-4 */

int oracle_channel_stat(const void* x, int dt, int64_t n_tokens, int n_heads, int head_dim,
                        int stat_kind, double* stat_out) {
    if (!x || !stat_out || n_tokens < 0 || n_heads < 1 || head_dim < 1) return ORACLE_INVALID;
    const int64_t C = (int64_t)n_heads * head_dim;
    for (int64_t c = 0; c < C; ++c) stat_out[c] = 0.0;
    for (int64_t t = 0; t < n_tokens; ++t) {
        for (int64_t c = 0; c < C; ++c) {
            double v = load_elem(x, dt, t * C + c);
            if (!isfinite(v)) return ORACLE_NONFINITE;
            if (stat_kind == ORACLE_STAT_MAXABS) {
                double a = fabs(v);
                if (a > stat_out[c]) stat_out[c] = a;
            } else {
                stat_out[c] += v * v;
            }
        }
    }
    if (stat_kind == ORACLE_STAT_L2)
        for (int64_t c = 0; c < C; ++c) stat_out[c] = sqrt(stat_out[c]);
    return ORACLE_OK;
}

void oracle_argsort_stable(const double* stat, int d, int32_t* perm, int32_t* inv_perm) {
    /* insertion sort on (stat, index): stable, ascending */
    for (int j = 0; j < d; ++j) perm[j] = j;
    for (int j = 1; j < d; ++j) {
        int32_t cur = perm[j];
        int k = j - 1;
        while (k >= 0 && stat[perm[k]] > stat[cur]) {
            perm[k + 1] = perm[k];
            --k;
        }
        perm[k + 1] = cur;
    }
    if (inv_perm)
        for (int j = 0; j < d; ++j) inv_perm[perm[j]] = j;
}

int oracle_calibrate(const void* x, int dt, int64_t n_tokens, int n_heads, int head_dim,
                     int stat_kind, double* stat_out, int32_t* perm_out, int32_t* inv_perm_out) {
    if (!perm_out) return ORACLE_INVALID;
    const int64_t C = (int64_t)n_heads * head_dim;
    double* stat = stat_out ? stat_out : (double*)malloc((size_t)C * sizeof(double));
    if (!stat) return ORACLE_INVALID;
    int rc = oracle_channel_stat(x, dt, n_tokens, n_heads, head_dim, stat_kind, stat);
    if (rc == ORACLE_OK) {
        for (int h = 0; h < n_heads; ++h)
            oracle_argsort_stable(stat + (int64_t)h * head_dim, head_dim,
                                  perm_out + (int64_t)h * head_dim,
                                  inv_perm_out ? inv_perm_out + (int64_t)h * head_dim : NULL);
    }
    if (!stat_out) free(stat);
    return rc;
}

void oracle_fold_perm(const double* w, int n_heads, int head_dim, int64_t d_in,
                      const int32_t* perm, double* out) {
    for (int h = 0; h < n_heads; ++h)
        for (int j = 0; j < head_dim; ++j) {
            const double* src = w + ((int64_t)h * head_dim + perm[(int64_t)h * head_dim + j]) * d_in;
            double* dst = out + ((int64_t)h * head_dim + j) * d_in;
            for (int64_t i = 0; i < d_in; ++i) dst[i] = src[i];
        }
}

/* -------------------------------------------------------------- cache write */

static int append_one(const oracle_format* f, uint8_t* mant, uint8_t* exp8, const void* x_new,
                      int dt, int n_new, const int32_t* start_pos, const int32_t* perm) {
    const int d = f->head_dim, n = f->block, p = f->mant_bits, H = f->n_kv_heads;
    const size_t row_m = oracle_row_mant_bytes(f), row_e = oracle_row_exp_bytes(f);
    double* row = (double*)malloc((size_t)d * sizeof(double));
    int* M = (int*)malloc((size_t)d * sizeof(int));
    int rc = ORACLE_OK;
    for (int b = 0; b < f->batch && rc == ORACLE_OK; ++b) {
        if (start_pos[b] < 0 || (int64_t)start_pos[b] + n_new > f->max_seq) { rc = ORACLE_CAPACITY; break; }
        for (int t = 0; t < n_new && rc == ORACLE_OK; ++t)
            for (int h = 0; h < H && rc == ORACLE_OK; ++h) {
                const int64_t src = (((int64_t)b * n_new + t) * H + h) * d;
                /* Algorithm 1 step 3 at run time: permuted channel j holds original channel perm[h][j] */
                for (int j = 0; j < d; ++j) {
                    int c = perm ? perm[(int64_t)h * d + j] : j;
                    row[j] = load_elem(x_new, dt, src + c);
                }
                const int64_t pos = ((int64_t)b * H + h) * f->max_seq + start_pos[b] + t;
                for (int blk = 0; blk < d / n && rc == ORACLE_OK; ++blk) {
                    int e8;
                    rc = oracle_bfp_cast_block(row + blk * n, n, p, &e8, M + blk * n);
                    if (rc == ORACLE_OK) exp8[pos * (int64_t)row_e + blk] = (uint8_t)e8;
                }
                if (rc == ORACLE_OK) oracle_pack_mantissas(M, d, p, mant + pos * (int64_t)row_m);
            }
    }
    free(row);
    free(M);
    return rc;
}

int oracle_append(const oracle_format* f, uint8_t* k_mant, uint8_t* k_exp, uint8_t* v_mant,
                  uint8_t* v_exp, const void* k_new, const void* v_new, int dt, int n_new,
                  const int32_t* start_pos, const int32_t* perm_k, const int32_t* perm_v) {
    if (!format_ok(f) || !start_pos || n_new < 0) return ORACLE_INVALID;
    int rc = ORACLE_OK;
    if (k_new) {
        if (!k_mant || !k_exp) return ORACLE_INVALID;
        rc = append_one(f, k_mant, k_exp, k_new, dt, n_new, start_pos, perm_k);
    }
    if (rc == ORACLE_OK && v_new) {
        if (!v_mant || !v_exp) return ORACLE_INVALID;
        rc = append_one(f, v_mant, v_exp, v_new, dt, n_new, start_pos, perm_v);
    }
    return rc;
}

/* ------------------------------------------------------------------ dequant */

/* Dequantise one stored row into stored (permuted) channel order. */
static void dequant_row(const oracle_format* f, const uint8_t* mant_row, const uint8_t* exp_row,
                        int* Mtmp, double* out) {
    const int d = f->head_dim, n = f->block, p = f->mant_bits;
    oracle_unpack_mantissas(mant_row, d, p, Mtmp);
    for (int j = 0; j < d; ++j) out[j] = oracle_bfp_value(Mtmp[j], exp_row[j / n], p);
}

int oracle_dequant(const oracle_format* f, const uint8_t* mant, const uint8_t* exp8, int b,
                   int h, int t0, int n_tok, const int32_t* perm, double* out) {
    if (!format_ok(f) || !mant || !exp8 || !out) return ORACLE_INVALID;
    if (b < 0 || b >= f->batch || h < 0 || h >= f->n_kv_heads) return ORACLE_INVALID;
    if (t0 < 0 || n_tok < 0 || (int64_t)t0 + n_tok > f->max_seq) return ORACLE_CAPACITY;
    const int d = f->head_dim;
    const size_t row_m = oracle_row_mant_bytes(f), row_e = oracle_row_exp_bytes(f);
    int* M = (int*)malloc((size_t)d * sizeof(int));
    double* row = (double*)malloc((size_t)d * sizeof(double));
    for (int t = 0; t < n_tok; ++t) {
        const int64_t pos = ((int64_t)b * f->n_kv_heads + h) * f->max_seq + t0 + t;
        dequant_row(f, mant + pos * (int64_t)row_m, exp8 + pos * (int64_t)row_e, M, row);
        for (int j = 0; j < d; ++j) {
            int c = perm ? perm[(int64_t)h * d + j] : j;   /* stored slot j came from channel c */
            out[(int64_t)t * d + c] = row[j];
        }
    }
    free(M);
    free(row);
    return ORACLE_OK;
}

/* ---------------------------------------------------------------- attention */

/* Attention over the cache; theta != NULL: the dequantised key row of token t is rotated to position t
 * (Eq. (4) with the tables of Algorithm 1 step 5, one set of d entries per KV head) before the product. */
static int decode_attn_impl(const oracle_format* f, const uint8_t* k_mant, const uint8_t* k_exp,
                            const uint8_t* v_mant, const uint8_t* v_exp, const void* q, int q_dt,
                            int n_q_heads, const int32_t* seq_lens, const int32_t* perm_k,
                            const int32_t* inv_perm_v, double softmax_scale, int q_mant_bits,
                            const double* theta, const int32_t* partner, const double* sign,
                            double* out) {
    if (!format_ok(f) || !k_mant || !k_exp || !v_mant || !v_exp || !q || !seq_lens || !out)
        return ORACLE_INVALID;
    if (n_q_heads < 1 || n_q_heads % f->n_kv_heads != 0) return ORACLE_INVALID;
    if (q_mant_bits != 0 && (q_mant_bits < 2 || q_mant_bits > 24)) return ORACLE_INVALID;
    const int d = f->head_dim, H = f->n_kv_heads, G = n_q_heads / H, n = f->block;
    const size_t row_m = oracle_row_mant_bytes(f), row_e = oracle_row_exp_bytes(f);
    const double scale = softmax_scale > 0.0 ? softmax_scale : 1.0 / sqrt((double)d);
    int rc = ORACLE_OK;
    int* M = (int*)malloc((size_t)d * sizeof(int));
    double* qp = (double*)malloc((size_t)d * sizeof(double));
    double* krow = (double*)malloc((size_t)d * sizeof(double));
    double* krot = (double*)malloc((size_t)d * sizeof(double));
    double* o = (double*)malloc((size_t)d * sizeof(double));
    for (int b = 0; b < f->batch && rc == ORACLE_OK; ++b) {
        const int len = seq_lens[b];
        if (len < 0 || len > f->max_seq) { rc = ORACLE_CAPACITY; break; }
        double* s = (double*)malloc((size_t)(len > 0 ? len : 1) * sizeof(double));
        for (int hq = 0; hq < n_q_heads && rc == ORACLE_OK; ++hq) {
            const int g = hq / G;   /* KV head shared by this query head */
            /* Eq. (3): pi(q) */
            for (int j = 0; j < d; ++j) {
                int c = perm_k ? perm_k[(int64_t)g * d + j] : j;
                qp[j] = load_elem(q, q_dt, ((int64_t)b * n_q_heads + hq) * d + c);
                if (!isfinite(qp[j])) rc = ORACLE_NONFINITE;
            }
            if (rc != ORACLE_OK) break;
            if (q_mant_bits) {   /* BFP query: same block size, wider mantissa */
                for (int blk = 0; blk < d / n; ++blk) {
                    int e8;
                    rc = oracle_bfp_cast_block(qp + blk * n, n, q_mant_bits, &e8, M + blk * n);
                    if (rc != ORACLE_OK) break;
                    for (int j = 0; j < n; ++j)
                        qp[blk * n + j] = oracle_bfp_value(M[blk * n + j], e8, q_mant_bits);
                }
                if (rc != ORACLE_OK) break;
            }
            double* dst = out + ((int64_t)b * n_q_heads + hq) * d;
            if (len == 0) {
                for (int c = 0; c < d; ++c) dst[c] = 0.0;
                continue;
            }
            const int64_t base = ((int64_t)b * H + g) * f->max_seq;
            double smax = -INFINITY;
            for (int t = 0; t < len; ++t) {
                dequant_row(f, k_mant + (base + t) * (int64_t)row_m, k_exp + (base + t) * (int64_t)row_e, M, krow);
                const double* kt = krow;
                if (theta) {   /* Sec. III par. 2: the rotary embedding is applied after the read-back */
                    oracle_rope_apply(d, (double)t, theta + (int64_t)g * d, partner + (int64_t)g * d,
                                      sign + (int64_t)g * d, krow, krot);
                    kt = krot;
                }
                double acc = 0.0;
                for (int j = 0; j < d; ++j) acc += qp[j] * kt[j];
                s[t] = scale * acc;
                if (s[t] > smax) smax = s[t];
            }
            double denom = 0.0;
            for (int t = 0; t < len; ++t) {
                s[t] = exp(s[t] - smax);
                denom += s[t];
            }
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int t = 0; t < len; ++t) {
                dequant_row(f, v_mant + (base + t) * (int64_t)row_m, v_exp + (base + t) * (int64_t)row_e, M, krow);
                double w = s[t] / denom;
                for (int c = 0; c < d; ++c) o[c] += w * krow[c];
            }
            /* stored V slot j holds original channel perm_v[j]; out[c] = o[inv_perm_v[c]] */
            for (int c = 0; c < d; ++c) {
                int j = inv_perm_v ? inv_perm_v[(int64_t)g * d + c] : c;
                dst[c] = o[j];
            }
        }
        free(s);
    }
    free(M);
    free(qp);
    free(krow);
    free(krot);
    free(o);
    return rc;
}

int oracle_decode_attn(const oracle_format* f, const uint8_t* k_mant, const uint8_t* k_exp,
                       const uint8_t* v_mant, const uint8_t* v_exp, const void* q, int q_dt,
                       int n_q_heads, const int32_t* seq_lens, const int32_t* perm_k,
                       const int32_t* inv_perm_v, double softmax_scale, int q_mant_bits,
                       double* out) {
    return decode_attn_impl(f, k_mant, k_exp, v_mant, v_exp, q, q_dt, n_q_heads, seq_lens, perm_k,
                            inv_perm_v, softmax_scale, q_mant_bits, NULL, NULL, NULL, out);
}

int oracle_decode_attn_rope(const oracle_format* f, const uint8_t* k_mant, const uint8_t* k_exp,
                            const uint8_t* v_mant, const uint8_t* v_exp, const void* q, int q_dt,
                            int n_q_heads, const int32_t* seq_lens, const int32_t* perm_k,
                            const int32_t* inv_perm_v, double softmax_scale, const double* theta,
                            const int32_t* partner, const double* sign, double* out) {
    if (!theta || !partner || !sign) return ORACLE_INVALID;
    return decode_attn_impl(f, k_mant, k_exp, v_mant, v_exp, q, q_dt, n_q_heads, seq_lens, perm_k,
                            inv_perm_v, softmax_scale, 0, theta, partner, sign, out);
}

/* --------------------------------------------------------- rotary embedding */

void oracle_rope_tables(int d, double base, int half_split, double* theta, int32_t* partner,
                        double* sign) {
    /* theta_i = base^(-2(i-1)/d), i = 1..d/2 (RoFormer).  Interleaved layout of
     * Eq. (4): channels (2i-1, 2i) form pair i; the half-split layout of the
     * footnote pairs channel i with channel i + d/2. */
    const int half = d / 2;
    for (int c = 0; c < d; ++c) {
        int i = half_split ? (c % half) : (c / 2);
        theta[c] = pow(base, -2.0 * (double)i / (double)d);
        if (half_split) {
            partner[c] = (c < half) ? c + half : c - half;
            sign[c] = (c < half) ? -1.0 : 1.0;
        } else {
            partner[c] = (c % 2 == 0) ? c + 1 : c - 1;
            sign[c] = (c % 2 == 0) ? -1.0 : 1.0;
        }
    }
}

void oracle_rope_permute_tables(int d, const int32_t* perm, const int32_t* inv_perm,
                                const double* theta, const int32_t* partner, const double* sign,
                                double* theta_p, int32_t* partner_p, double* sign_p) {
    /* Algorithm 1 step 5.  Slot j of the permuted vector holds channel perm[j];
     * its partner channel partner[perm[j]] now sits in slot inv_perm[partner[perm[j]]]. */
    for (int j = 0; j < d; ++j) {
        theta_p[j] = theta[perm[j]];
        sign_p[j] = sign[perm[j]];
        partner_p[j] = inv_perm[partner[perm[j]]];
    }
}

void oracle_rope_apply(int d, double m, const double* theta, const int32_t* partner,
                       const double* sign, const double* x, double* y) {
    for (int c = 0; c < d; ++c)
        y[c] = x[c] * cos(m * theta[c]) + sign[c] * x[partner[c]] * sin(m * theta[c]);
}
