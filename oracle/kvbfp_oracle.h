/*
 * CPU oracle for the Block-Floating-Point KV cache with K-sort.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, single-threaded fp64
 * restatement of what the paper defines.  It shares no code, header, table or
 * helper with the CUDA library, and the CUDA library never calls it.  Only the
 * tests, the smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * All pointers are HOST pointers.  Status codes: 0 ok, 1 invalid argument,
 * 4 capacity exceeded, 7 non-finite input.
 *
 * Paper passages followed (Trukhanov & Soloveychik, "Accurate Block
 * Quantization in LLMs with Outliers"):
 *   Sec. II-B, Eq. (1)      BFP block: n integers M_i in [-(2^(p-1)-1), 2^(p-1)-1]
 *                           and one b-bit exponent e; values 2^e * M_i.
 *   Sec. II-B (last par.)   cast = exponent from the largest |x| of the block,
 *                           scale by it, round to the closest integer in range.
 *   Sec. II-C, Eq. (2),(3)  a joint channel permutation of q and k leaves q.k
 *                           unchanged.
 *   Sec. II-D, Eq. (4)      element-wise rotary embedding.
 *   Sec. III, Algorithm 1   per head: channel statistic, argsort, permute W_k,
 *                           W_q, and (step 5) the RoPE frequency / partner /
 *                           sign vectors.
 *   Sec. III (par. 2)       keys stored per head as 4-bit mantissas with one
 *                           shared exponent per block of 32/64/128; at decode
 *                           the keys are read back and multiplied with pi(q);
 *                           q may be held as BFP16 (8-bit mantissas).
 *   Sec. IV                 rounding to the nearest.
 *
 * Parity unpinned: the perplexities of Table I (they need trained weights and
 * a text corpus).  Every function below is pinned by closed forms, invariants
 * or brute force in the CPU test-suite.
 */
#ifndef KVBFP_ORACLE_H
#define KVBFP_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { ORACLE_OK = 0, ORACLE_INVALID = 1, ORACLE_CAPACITY = 4, ORACLE_NONFINITE = 7 };
enum { ORACLE_F32 = 0, ORACLE_BF16 = 1, ORACLE_F64 = 2 };
enum { ORACLE_STAT_MAXABS = 0, ORACLE_STAT_L2 = 1 };

typedef struct {
    int32_t batch;
    int32_t n_kv_heads;
    int32_t head_dim;
    int32_t max_seq;
    int32_t block;      /* n: elements sharing one exponent, divides head_dim */
    int32_t mant_bits;  /* p: mantissa width, sign included, 2..8             */
} oracle_format;

/* Bytes of one token row of mantissas / exponents. */
size_t oracle_row_mant_bytes(const oracle_format* f);
size_t oracle_row_exp_bytes(const oracle_format* f);

/* Eq. (1): value of mantissa M in a block whose stored exponent byte is e8. */
double oracle_bfp_value(int M, int e8, int p);

/* Cast one block of n doubles (Sec. II-B).  Writes the exponent byte and n mantissas. */
int oracle_bfp_cast_block(const double* x, int n, int p, int* e8_out, int* M_out);

/* p-bit fields holding M + 2^(p-1) (excess code), element j in bits [j*p, (j+1)*p) of a
 * little-endian bit stream. */
void oracle_pack_mantissas(const int* M, int count, int p, uint8_t* bytes);
void oracle_unpack_mantissas(const uint8_t* bytes, int count, int p, int* M);

/* Algorithm 1 step 1 (statistic per head channel) over x[T][H][d]. */
int oracle_channel_stat(const void* x, int dt, int64_t n_tokens, int n_heads, int head_dim,
                        int stat_kind, double* stat_out);
/* Algorithm 1 step 2: ascending, equal statistics keep channel order. */
void oracle_argsort_stable(const double* stat, int d, int32_t* perm, int32_t* inv_perm);
int oracle_calibrate(const void* x, int dt, int64_t n_tokens, int n_heads, int head_dim,
                     int stat_kind, double* stat_out, int32_t* perm_out, int32_t* inv_perm_out);

/* Algorithm 1 steps 3-4: gather the rows of a per-head weight slab
 * w[H][d][d_in] by perm[H][d]:  out[h][j][:] = w[h][perm[h][j]][:]. */
void oracle_fold_perm(const double* w, int n_heads, int head_dim, int64_t d_in,
                      const int32_t* perm, double* out);

/* Cache write (Sec. II-A, Sec. III par. 2): permute, cast, pack, store. */
int oracle_append(const oracle_format* f, uint8_t* k_mant, uint8_t* k_exp, uint8_t* v_mant,
                  uint8_t* v_exp, const void* k_new, const void* v_new, int dt, int n_new,
                  const int32_t* start_pos, const int32_t* perm_k, const int32_t* perm_v);

/* Eq. (1) over stored rows; perm != NULL scatters back to original channels. */
int oracle_dequant(const oracle_format* f, const uint8_t* mant, const uint8_t* exp8, int b,
                   int h, int t0, int n_tok, const int32_t* perm, double* out);

/* Exact attention in fp64 over the dequantised cache (Sec. III par. 2).
 * q_mant_bits == 0 keeps q as given; otherwise pi(q) is first cast to BFP with
 * that mantissa width and the cache's block size (BFP16 query of Sec. IV). */
int oracle_decode_attn(const oracle_format* f, const uint8_t* k_mant, const uint8_t* k_exp,
                       const uint8_t* v_mant, const uint8_t* v_exp, const void* q, int q_dt,
                       int n_q_heads, const int32_t* seq_lens, const int32_t* perm_k,
                       const int32_t* inv_perm_v, double softmax_scale, int q_mant_bits,
                       double* out);

/* The same over a cache of keys stored BEFORE the rotary embedding (Sec. III par. 2: the embedding is applied
 * to the keys after they are read back): the dequantised key row of token t is rotated to position t by
 * Eq. (4), with tables in stored order (Algorithm 1 step 5; [n_kv_heads * head_dim] each), and then
 * multiplied with pi(q).  q is taken as given: already rotated to its own position by the caller. */
int oracle_decode_attn_rope(const oracle_format* f, const uint8_t* k_mant, const uint8_t* k_exp,
                            const uint8_t* v_mant, const uint8_t* v_exp, const void* q, int q_dt,
                            int n_q_heads, const int32_t* seq_lens, const int32_t* perm_k,
                            const int32_t* inv_perm_v, double softmax_scale, const double* theta,
                            const int32_t* partner, const double* sign, double* out);

/* Eq. (4): rotary embedding of x[d] at position m, in place.
 * theta[d], partner[d] (0-based index of the element whose value is taken for
 * the sine term) and sign[d] describe the layout; Algorithm 1 step 5 permutes
 * them with oracle_rope_permute_tables. */
void oracle_rope_tables(int d, double base, int half_split, double* theta, int32_t* partner,
                        double* sign);
void oracle_rope_permute_tables(int d, const int32_t* perm, const int32_t* inv_perm,
                                const double* theta, const int32_t* partner, const double* sign,
                                double* theta_p, int32_t* partner_p, double* sign_p);
void oracle_rope_apply(int d, double m, const double* theta, const int32_t* partner,
                       const double* sign, const double* x, double* y);

#ifdef __cplusplus
}
#endif
#endif
