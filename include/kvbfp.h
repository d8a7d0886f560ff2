/*
 * kvbfp — a KV cache in Block Floating Point (BFP) with K-sort channel
 * permutation, for NVIDIA B200 (sm_100a).  C ABI; no CUDA or framework types.
 *
 * Method: N. Trukhanov, I. Soloveychik, "Accurate Block Quantization in LLMs
 * with Outliers".  A BFP block is n signed p-bit integer mantissas M_i sharing
 * one 8-bit exponent e, with values 2^e * M_i (Sec. II-B, Eq. (1)).  Key
 * channels are reordered once, per head, by a permutation pi found from a
 * per-channel magnitude statistic (Sec. II-C, Sec. III Algorithm 1); q is
 * permuted the same way, which leaves q.k unchanged (Eq. (2), (3)).
 *
 * Conventions for every call
 *  - Pointers are DEVICE pointers unless the parameter says "host".  Structs
 *    (kvbfp_format, kvbfp_cache) live in host memory and are read during the call.
 *  - The caller owns every buffer.  The library allocates nothing and keeps no
 *    state between calls except one 4-byte status word per device.
 *  - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL is the
 *    default stream) of the CURRENT device; results are valid once the stream
 *    has been synchronised.
 *  - Argument errors are found on the host before anything is enqueued and are
 *    returned as a status.  Data-dependent conditions (non-finite input, a
 *    position beyond the cache capacity, a sequence longer than the hint) set
 *    bits in the device status word, skip the offending work, and never trap;
 *    read them with kvbfp_device_status().
 *  - Tensors are dense, row-major, last index fastest, 16-byte aligned.
 *
 * Storage layout (the paper does not fix one; this is the library's own):
 *  - mantissa plane  [batch, n_kv_heads, max_seq, row_m] bytes, row_m = head_dim*p/8;
 *    a row is a little-endian bit stream, stored slot j in bits [j*p, (j+1)*p),
 *    holding M + 2^(p-1) (excess code: 0 is stored as 8, 32 or 128; p = 4: low nibble is the even
 *    slot);
 *  - exponent plane  [batch, n_kv_heads, max_seq, row_e] bytes, row_e = head_dim/n;
 *    byte i belongs to slots [i*n, (i+1)*n) and holds E + 127, where 2^E is the
 *    largest power of two not above the block's largest magnitude (E >= -127);
 *    the mantissa's unit weight is 2^(E - (p-2)).  255 is never written.
 *  - "slot" = position after the permutation: slot j of head h holds original
 *    channel perm[h*head_dim + j].
 */
#ifndef KVBFP_H
#define KVBFP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    KVBFP_OK = 0,
    KVBFP_ERR_INVALID_ARG = 1,  /* null pointer, bad count, inconsistent sizes          */
    KVBFP_ERR_UNSUPPORTED = 2,  /* a format or shape the kernels are not built for       */
    KVBFP_ERR_ALIGNMENT = 3,    /* a pointer that is not 16-byte aligned                 */
    KVBFP_ERR_CAPACITY = 4,     /* more tokens than the cache holds (host-visible cases) */
    KVBFP_ERR_WORKSPACE = 5,    /* workspace missing or too small                        */
    KVBFP_ERR_CUDA = 6          /* a CUDA runtime call or a launch failed                */
} kvbfp_status;

typedef enum { KVBFP_F32 = 0, KVBFP_BF16 = 1 } kvbfp_dtype;
typedef enum { KVBFP_STAT_MAXABS = 0, KVBFP_STAT_L2 = 1 } kvbfp_stat;

/* Bits of the device status word. */
enum {
    KVBFP_FLAG_NONFINITE = 1u,     /* an input element was Inf or NaN                        */
    KVBFP_FLAG_POSITION = 2u,      /* append: start_pos + n_new beyond max_seq, the sequence's rows are skipped;
                                      decode: a seq_len beyond max_seq is read as max_seq, a negative one as 0 */
    KVBFP_FLAG_LEN_HINT = 4u,      /* a seq_len exceeded max_len_hint: tokens past it unread */
    KVBFP_FLAG_WAIT_TIMEOUT = 8u   /* an on-chip copy did not complete within its wait bound */
};

/* Which decode kernel to run. */
enum {
    KVBFP_DECODE_AUTO = 0,     /* the fastest tensor-core kernel for the format                       */
    KVBFP_DECODE_SIMT = 1,     /* fp32 FMA on the plain ALUs, one query head at a time                */
    KVBFP_DECODE_MMA = 2,      /* same as AUTO: grouped queries as the N operand of warp-level MMAs   */
    KVBFP_DECODE_MMA_BF16 = 3  /* the generic bf16 tensor-core kernel (all mantissa widths).  AUTO uses the
                                  integer-score kernels for 4 bits, for 8 bits with blocks of 32 or more and for
                                  6 bits with blocks of 32 or more and one query head per kv head, and this one
                                  otherwise (6 bits with grouped query heads or blocks of 16; 8 bits with blocks
                                  of 16).  Its conversion leaves the bf16 range for cache values of magnitude
                                  2^120 and above; the other kernels have no such limit. */
};
/* Optional, or-ed into `flags`: tokens per sequence chunk (a multiple of 128; 0 = chosen by the
 * library from the batch size and the sequence bound). */
#define KVBFP_DECODE_CHUNK(tokens) (((uint32_t)(tokens) / 128u) << 8)

/* BFP format and cache geometry (Sec. II-B: block size n, mantissa precision p, b = 8). */
typedef struct {
    int32_t batch;
    int32_t n_kv_heads;
    int32_t head_dim;   /* 128 */
    int32_t max_seq;    /* capacity in tokens per (batch, head); a multiple of 16 */
    int32_t block;      /* n: 16, 32, 64 or 128; divides head_dim */
    int32_t mant_bits;  /* p: 4, 6 or 8, sign included; mantissas lie in [-(2^(p-1)-1), 2^(p-1)-1] */
} kvbfp_format;

/* The cache is four caller-owned planes (see "Storage layout"). */
typedef struct {
    kvbfp_format fmt;
    uint8_t* k_mant;
    uint8_t* k_exp;
    uint8_t* v_mant;
    uint8_t* v_exp;
} kvbfp_cache;

/* Library version, major*10000 + minor*100 + patch. */
int32_t kvbfp_version(void);

/* Text of a status code (static storage, never NULL). */
const char* kvbfp_status_string(kvbfp_status s);

/* Text of the last CUDA error seen by this thread inside the library (thread-local storage;
 * empty string if none). */
const char* kvbfp_last_cuda_error(void);

/* Sizes in bytes of ONE mantissa plane and ONE exponent plane of `fmt` (host pointers out).
 * Bits per stored element are p + 8/n (Sec. III: BFP12 = 4-bit mantissas + the shared byte). */
kvbfp_status kvbfp_plane_bytes(const kvbfp_format* fmt, size_t* mant_bytes, size_t* exp_bytes);

/*
 * K-sort, Algorithm 1 steps 1-2 (Sec. III), run once before inference.
 *   x            [n_tokens, n_heads, head_dim] of `dt`: calibration keys, or W_k transposed so
 *                that the reduced axis comes first
 *   stat         KVBFP_STAT_MAXABS: stat[h,c] = max_t |x[t,h,c]|   (exact)
 *                KVBFP_STAT_L2:     stat[h,c] = sqrt(sum_t x^2), summed in fp64 (Algorithm 1 step 1)
 *   stat_out     [n_heads*head_dim] f32, required
 *   perm_out     [n_heads*head_dim] i32: slot j of head h holds channel perm_out[h*d+j]; ascending
 *                statistic, equal statistics in channel order (stable)
 *   inv_perm_out [n_heads*head_dim] i32 or NULL: inv_perm[h*d + perm[h*d+j]] = j
 *   workspace    KVBFP_STAT_L2 only: n_heads*head_dim*8 bytes for the fp64 sums; NULL for MAXABS
 * Non-finite inputs set KVBFP_FLAG_NONFINITE; the permutation is then unspecified but valid.
 */
kvbfp_status kvbfp_calibrate(const void* x, kvbfp_dtype dt, int64_t n_tokens, int32_t n_heads,
                             int32_t head_dim, kvbfp_stat stat, float* stat_out, int32_t* perm_out,
                             int32_t* inv_perm_out, void* workspace, size_t workspace_bytes,
                             void* stream);

/*
 * Algorithm 1 steps 3-4: fold a permutation into a projection weight, once, offline.
 *   w   [n_heads*head_dim, d_in] of `dt` (rows = output channels of W_k or W_q)
 *   out [n_heads*head_dim, d_in] of `dt`, out[h*d + j, :] = w[h*d + perm[h*d+j], :]; out != w
 * With folded weights the run-time gathers are not needed: pass perm_k = NULL to append/decode.
 */
kvbfp_status kvbfp_fold_perm(const void* w, kvbfp_dtype dt, int32_t n_heads, int32_t head_dim,
                             int64_t d_in, const int32_t* perm, void* out, void* stream);

/*
 * Cache write (Sec. II-A; Sec. III par. 2): permute each new row, take the shared exponent of each
 * block from its largest magnitude, round mantissas to nearest (ties to even), clamp to the
 * symmetric range, pack, store (Sec. II-B last paragraph).
 *   k_new, v_new [batch, n_new, n_kv_heads, head_dim] of `dt`; either may be NULL (plane untouched)
 *   start_pos    [batch] i32: row t of sequence b goes to position start_pos[b] + t
 *   perm_k/v     [n_kv_heads*head_dim] i32 or NULL (identity, e.g. when folded into the weights)
 * A sequence whose rows would pass max_seq is skipped whole and sets KVBFP_FLAG_POSITION.
 */
kvbfp_status kvbfp_append(const kvbfp_cache* cache, const void* k_new, const void* v_new,
                          kvbfp_dtype dt, int32_t n_new, const int32_t* start_pos,
                          const int32_t* perm_k, const int32_t* perm_v, void* stream);

/*
 * Eq. (1): rows [t0, t0+n_tok) of (b, h) of one plane pair back to numbers (exact in f32 and bf16).
 *   b, h  a sequence and a head, or -1 for all of them (one launch either way)
 *   perm  [n_kv_heads*head_dim] i32 or NULL.  NULL: out[.., t, j] = slot j;
 *         else out[.., t, perm[h*d+j]] = slot j (original channel order)
 *   out   device, of out_dt: [n_tok, head_dim] for one (b, h); with h = -1 the heads come after the tokens,
 *         [n_tok, n_kv_heads, head_dim]; with b = -1 the sequences come first, [batch, n_tok, ..] -- the layout
 *         kvbfp_append takes its rows in
 * Errors: rows past max_seq -> KVBFP_ERR_CAPACITY; nothing is written then.
 */
kvbfp_status kvbfp_dequant(const kvbfp_format* fmt, const uint8_t* mant, const uint8_t* exp8,
                           int32_t b, int32_t h, int32_t t0, int32_t n_tok, const int32_t* perm,
                           void* out, kvbfp_dtype out_dt, void* stream);

/*
 * Algorithm 1 step 5 (Sec. III): rotary-embedding tables in stored (slot) order, so that rows that are already
 * permuted can be rotated (Sec. II-D, Eq. (4)) without undoing K-sort.  Slot j of head h holds channel
 * c = perm[h*d+j]; the tables give that channel's frequency, the slot of its rotation partner and the sine sign.
 *   perm, inv_perm  [n_heads*head_dim] i32, both NULL for the identity
 *   base            frequency base (10000 in RoFormer); theta_i = base^(-2i/d)
 *   half_split      0: pairs of neighbouring channels (2i, 2i+1), the layout of Eq. (4);
 *                   1: pairs (i, i + d/2), the layout of the open-source Llama code (footnote to Sec. III)
 *   theta_out       [n_heads*head_dim] f64;  partner_out [n_heads*head_dim] i32;  sign_out [n_heads*head_dim] f32
 */
kvbfp_status kvbfp_rope_tables(const int32_t* perm, const int32_t* inv_perm, int32_t n_heads,
                               int32_t head_dim, double base, int32_t half_split, double* theta_out,
                               int32_t* partner_out, float* sign_out, void* stream);

/*
 * Eq. (4) in table form on rows in slot order: y[j] = x[j] cos(m theta_j) + sign_j x[partner_j] sin(m theta_j),
 * m = positions[row].  The angle is formed and reduced in fp64, the rotation itself is fp32 (about 1e-7 relative).
 *   x, y       [n_rows, n_heads, head_dim] of `dt`, y != x
 *   positions  [n_rows] i32
 */
kvbfp_status kvbfp_rope_apply(const void* x, kvbfp_dtype dt, int64_t n_rows, int32_t n_heads,
                              int32_t head_dim, const int32_t* positions, const double* theta,
                              const int32_t* partner, const float* sign, void* y, void* stream);

/* Bytes of workspace kvbfp_decode_attn needs for this cache geometry (0 on invalid arguments). */
size_t kvbfp_decode_workspace_bytes(const kvbfp_format* fmt, int32_t n_q_heads);

/*
 * One decode step of attention read straight from the packed cache (Sec. II-A; Sec. III par. 2:
 * keys are read back and multiplied with pi(q)): scores = scale * pi(q).K^T over tokens
 * t < seq_lens[b], softmax, times V; K/V are dequantised in registers, never written back.
 *   q              [batch, n_q_heads, head_dim] of q_dt, original channel order
 *   n_q_heads      multiple of n_kv_heads; query head hq reads KV head hq / (n_q_heads/n_kv_heads)
 *   seq_lens       [batch] i32
 *   max_len_hint   host-known upper bound of seq_lens (0 = max_seq); sizes the launch only
 *   perm_k         permutation the keys were appended with (NULL = identity); q is gathered by it
 *   inv_perm_v     inverse of the permutation V was appended with (NULL = identity):
 *                  out[c] = o_slot[inv_perm_v[g*d + c]]
 *   softmax_scale  0 means 1/sqrt(head_dim)
 *   q_mant_bits    0: q used as given.  8: pi(q) is first cast to BFP with 8-bit mantissas and the
 *                  cache's block size (the BFP16 query of Sec. IV)
 *   out            [batch, n_q_heads, head_dim] f32; zeros where seq_lens[b] == 0
 *   workspace      at least kvbfp_decode_workspace_bytes() bytes, contents need no initialisation
 *   flags          KVBFP_DECODE_* [| KVBFP_DECODE_CHUNK(tokens)]
 * The sequence is split into chunks handled independently; a second kernel merges the per-chunk
 * (max, sum, output) triples with log-sum-exp weights.
 */
kvbfp_status kvbfp_decode_attn(const kvbfp_cache* cache, const void* q, kvbfp_dtype q_dt,
                               int32_t n_q_heads, const int32_t* seq_lens, int32_t max_len_hint,
                               const int32_t* perm_k, const int32_t* inv_perm_v,
                               float softmax_scale, int32_t q_mant_bits, float* out,
                               void* workspace, size_t workspace_bytes, uint32_t flags,
                               void* stream);

/*
 * kvbfp_decode_attn over a cache whose keys were stored BEFORE the rotary embedding (Sec. III par. 2: the
 * embedding is applied to the keys after they are read back from the cache; Sec. II-D, Eq. (4); tables in
 * stored order per Algorithm 1 step 5).  Token t's dequantised key row is rotated to position t, in registers,
 * before the product with pi(q):  k'[j] = k[j] cos(t theta_j) + sign_j k[partner_j] sin(t theta_j).
 *   q                    as in kvbfp_decode_attn, already rotated to its own position by the caller
 *   theta, partner, sign [n_kv_heads*head_dim] f64 / i32 / f32 as written by kvbfp_rope_tables for the
 *                        permutation the keys were appended with (partners share a frequency and have
 *                        opposite signs; other tables give unspecified results)
 *   flags                KVBFP_DECODE_AUTO or KVBFP_DECODE_SIMT (the fp32 kernel is the only one that rotates:
 *                        KVBFP_ERR_UNSUPPORTED otherwise); chunks are capped at 512 tokens
 * Everything else (workspace, lengths, V side, merge, errors) as in kvbfp_decode_attn.  No BFP query cast.
 */
kvbfp_status kvbfp_decode_attn_rope(const kvbfp_cache* cache, const void* q, kvbfp_dtype q_dt,
                                    int32_t n_q_heads, const int32_t* seq_lens, int32_t max_len_hint,
                                    const int32_t* perm_k, const int32_t* inv_perm_v, float softmax_scale,
                                    const double* theta, const int32_t* partner, const float* sign,
                                    float* out, void* workspace, size_t workspace_bytes, uint32_t flags,
                                    void* stream);

/*
 * kvbfp_decode_attn for callers that must not allocate device memory (the paper has no counterpart:
 * this is a deployment aid, not a step of the method).  Who needs it: code that runs after a serving
 * process has frozen its memory pool, plug-ins that are handed tensors but no allocator, and loops
 * that cannot afford the device-wide synchronisation an allocation or a free may cause.  It computes
 * exactly what kvbfp_decode_attn computes and takes the same arguments minus the workspace, which
 * lives in a fixed array inside the library image instead.
 *  - Limit: the array is kvbfp_static_scratch_bytes() = 32 MiB.  A geometry whose
 *    kvbfp_decode_workspace_bytes() is larger is refused with KVBFP_ERR_WORKSPACE and nothing is
 *    enqueued; use kvbfp_decode_attn with your own workspace then.  Every GPU on which the library is
 *    loaded gives up those 32 MiB until the process exits.
 *  - The call allocates nothing: no cudaMalloc, cudaFree or allocating library routine.
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *    that device current) and keeps it; make that first call before any stream capture begins.
 *  - All calls on a device share the one array, which still holds the previous call's partial
 *    results.  Nothing in it has to start at zero (each call writes every value it later reads), but
 *    two calls that overlap on the GPU — different streams, or one stream while another still runs —
 *    race on it and produce garbage.  Serialise them, or give the concurrent ones their own
 *    workspace through kvbfp_decode_attn.
 */
size_t kvbfp_static_scratch_bytes(void);
kvbfp_status kvbfp_decode_attn_static(const kvbfp_cache* cache, const void* q, kvbfp_dtype q_dt,
                                      int32_t n_q_heads, const int32_t* seq_lens,
                                      int32_t max_len_hint, const int32_t* perm_k,
                                      const int32_t* inv_perm_v, float softmax_scale,
                                      int32_t q_mant_bits, float* out, uint32_t flags, void* stream);

/*
 * One whole decode step for a caller whose new token lives in HOST memory (Sec. II-A: per step only
 * the new token's q, k, v are computed; the rest is read from the cache): brings k_new, v_new and q
 * to the device, appends the token (kvbfp_append with n_new = 1), runs kvbfp_decode_attn, brings the
 * result back and synchronises `stream`, so out_host is valid on return.
 *   k_new_host, v_new_host  host [batch, 1, n_kv_heads, head_dim] of `dt`, 16-byte aligned
 *   q_host                  host [batch, n_q_heads, head_dim] of `dt`, 16-byte aligned
 *   out_host                host [batch, n_q_heads, head_dim] f32, 16-byte aligned
 *   start_pos, seq_lens     device [batch] i32, as in kvbfp_append / kvbfp_decode_attn
 *   staging                 device scratch of at least kvbfp_step_staging_bytes() bytes
 * How the bytes cross the bus: when all four host buffers are page-locked memory that the current device can
 * address (cudaHostAlloc / cudaHostRegister; the call asks cudaPointerGetAttributes), the kernels read the new
 * token and the query from them, and write the result to out_host, in place -- the same bytes cross the bus, without
 * separate copy commands.  Otherwise (pageable memory) the call falls back to cudaMemcpyAsync through `staging`.
 * All other parameters as in kvbfp_append and kvbfp_decode_attn.
 */
size_t kvbfp_step_staging_bytes(const kvbfp_format* fmt, int32_t n_q_heads, kvbfp_dtype dt);
kvbfp_status kvbfp_decode_step_host(const kvbfp_cache* cache, const void* k_new_host,
                                    const void* v_new_host, const void* q_host, kvbfp_dtype dt,
                                    int32_t n_q_heads, const int32_t* start_pos,
                                    const int32_t* seq_lens, int32_t max_len_hint,
                                    const int32_t* perm_k, const int32_t* perm_v,
                                    const int32_t* inv_perm_v, float softmax_scale,
                                    float* out_host, void* staging, size_t staging_bytes,
                                    void* workspace, size_t workspace_bytes, uint32_t flags,
                                    void* stream);

/*
 * Diagnostic: the bounded barrier wait of the staged decode kernels, on its own.  Launches one warp that waits on a
 * barrier whose bytes arrive (must succeed) and on one whose bytes nothing ever sends: after `tries` tries of at most
 * `hint_ns` nanoseconds each (tries <= 1000, hint_ns <= 1 000 000: one second at the most) that wait gives up,
 * KVBFP_FLAG_WAIT_TIMEOUT is raised in the device status word and the kernel returns normally -- the same thing a
 * decode kernel does when an on-chip copy does not complete.  Nothing traps and the context stays usable; read the
 * flag with kvbfp_device_status.  (No counterpart in the paper.)
 */
kvbfp_status kvbfp_selftest_wait_timeout(uint32_t tries, uint32_t hint_ns, void* stream);

/*
 * Diagnostics of the work split behind kvbfp_decode_attn (host only: nothing is launched, no device is touched).
 * The persistent kernels lay the sequence pieces ("items") of all (batch, kv head) pairs out pair-major, cut them
 * into one contiguous range per resident warp, and let every range write one partial result per pair it touches;
 * the merge finds those partial results again with the same integer arithmetic.  These calls expose that arithmetic
 * as the kernels use it, so that it can be checked on its own.
 *   kvbfp_split_plan         for `pairs` pairs of at most `len_cap` tokens in chunks of `chunk` tokens (a multiple of
 *                            128), items of `fine_tokens` tokens (a multiple of 16 that divides the chunk; the
 *                            kernels ask for 64) where the plan allows them, on a device that holds
 *                            `capacity_blocks` thread blocks of `warps_per_block` warps:
 *                            out6 = {grid, n_warps, item_tokens, items_per_pair, range_items, range_extra}
 *   kvbfp_split_range_start  first item of range w (the first range_extra ranges hold range_items + 1 items)
 *   kvbfp_split_range_of     the range that holds item x
 *   kvbfp_split_partial_slot the chunk-sized slot (n_chunks per pair) that receives the partial result of a run
 *                            whose first item within its pair is `item`
 */
kvbfp_status kvbfp_split_plan(int32_t pairs, int32_t len_cap, int32_t chunk, int32_t fine_tokens,
                              int32_t capacity_blocks, int32_t warps_per_block, int32_t* out6);
int32_t kvbfp_split_range_start(int32_t w, int32_t range_items, int32_t range_extra);
int32_t kvbfp_split_range_of(int32_t x, int32_t range_items, int32_t range_extra);
int32_t kvbfp_split_partial_slot(int32_t item, int32_t item_tokens, int32_t chunk, int32_t n_chunks);

/*
 * Profiling aid.  After this call, every kvbfp_decode_attn issued from the calling thread records
 * `start_event` just before and `stop_event` just after its main kernel (the one that streams the
 * cache), on the call's stream.  Both are cudaEvent_t passed as void*; (NULL, NULL) switches it off.
 */
kvbfp_status kvbfp_profile_decode_events(void* start_event, void* stop_event);

/*
 * Synchronises `stream`, copies the device status word of the current device to *flags_out (host
 * pointer) and clears it.
 */
kvbfp_status kvbfp_device_status(uint32_t* flags_out, void* stream);

/* Number of kernels the library has launched from this process so far (all devices). */
uint64_t kvbfp_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* KVBFP_H */
