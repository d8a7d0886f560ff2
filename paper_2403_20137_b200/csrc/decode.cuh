// Internal interface between the decode entry point and its kernels.
#pragma once
#include "common.cuh"

namespace kvbfp {

// One partial result per (batch, query head, chunk): PSTRIDE floats =
// o[128] (sum of 2^(s-m) * V over the chunk, stored-slot order), m (running max, log2 units), l (sum).
constexpr int kPartStride = kHeadDim + 4;
constexpr int kMinChunk = 128;     // tokens; chunk sizes are multiples of this

struct DecodeArgs {
    kvbfp_format fmt;
    const uint8_t *k_mant, *k_exp, *v_mant, *v_exp;
    const void* q;            // [B, Hq, d]
    int q_is_bf16;
    int n_q_heads;
    const int32_t* seq_lens;
    const int32_t* perm_k;
    const int32_t* inv_perm_v;
    float scale_log2e;        // softmax scale * log2(e)
    int q_mant_bits;
    float* out;
    uint32_t* qfrag;          // workspace region for the tensor-core kernel's B fragments
    float* partials;          // workspace region [B, Hq, n_chunks, kPartStride]
    int chunk;                // tokens per chunk
    int n_chunks;
    int len_cap;              // min(max_len_hint, max_seq)
    int item_tokens;          // persistent kernel: tokens per work item (divides chunk) and items per (batch, kv head)
    int items_per_pair;
    int range_items;          // persistent kernel: items of a warp's range; the first `range_extra` ranges hold one more
    int range_extra;
    // keys cached before the rotary embedding (fp32 kernel only): tables in stored order, [n_kv_heads * head_dim]
    const double* rope_theta;
    const int32_t* rope_partner;
    const float* rope_sign;
    uint32_t* status;
};

kvbfp_status launch_decode_simt(const DecodeArgs& a, cudaStream_t s);
kvbfp_status launch_decode_mma(const DecodeArgs& a, cudaStream_t s);    // bf16, every mantissa width
// How the persistent kernel cut the work, for the merge: the items (pair-major pieces of `item_tokens` tokens,
// `items_per_pair` per (batch, kv head)) were split into `n_warps` contiguous ranges of `range_items` items, the
// first `range_extra` of them one item longer.  n_warps == 0: no ranges,
// every chunk has its own partial.
struct Split {
    int n_warps = 0;
    int item_tokens = 0;
    int items_per_pair = 0;
    int range_items = 0;      // range w starts at item  w * range_items + min(w, range_extra)
    int range_extra = 0;
};
// First item of range w, and the range that holds item x (32-bit: the launcher refuses 2^31 items and more).
__host__ __device__ __forceinline__ int range_start(int w, int range_items, int range_extra) {
    return w * range_items + (w < range_extra ? w : range_extra);
}
__host__ __device__ __forceinline__ int range_of(int x, int range_items, int range_extra) {
    const int big = range_extra * (range_items + 1);             // items held by the longer ranges
    return x < big ? x / (range_items + 1) : range_extra + (x - big) / range_items;
}
// Slot (chunk-sized, n_chunks per pair) that receives the partial of a run whose first item within its pair
// is `item`.  Items are whole chunks, or chunk / R tokens with R = 2 or more: then slot = ceil(item / R), at most
// the last one.  Runs of a pair start at item 0 and at range boundaries, which lie a whole range apart: with ranges
// of 2R - 1 items or more, two starts never round up to the same slot, and a start that is clamped to the last slot
// (item > (n_chunks - 1) R) has its predecessor at or below (n_chunks - 2) R, i.e. in an earlier slot -- provided a
// pair has two slots or more: with a single chunk per pair every start would share slot 0, so plan_persistent()
// never cuts such pairs finer than chunks.
__host__ __device__ __forceinline__ int partial_slot(int item, int item_tokens, int chunk, int n_chunks) {
    if (item_tokens == chunk) return item;
    const int R = chunk / item_tokens;
    const int s = (item + R - 1) / R;
    return s < n_chunks ? s : n_chunks - 1;
}
// Work split of a persistent kernel (host side).  Items are pieces of fine_tokens tokens (chunk / R, a multiple of the
// 16 tokens that copies start on) when the library chose the chunking (chunk == kMinChunk), a pair has two chunks or
// more, and every warp still gets 2R + 1 or more items on average, so 2R at the least (partial_slot() then keeps the
// runs' partial results apart); whole chunks otherwise.  The kernels ask for kItemTokens = 64, their tile: with
// 16-token items the ranges come out more evenly (two warps then differ by a quarter of a tile, not a whole one), but
// every run then ends in a partial tile that is copied and worked on like a whole one, and the launch was 1-2 %
// slower.  The items are cut into one contiguous range per warp of min(capacity, blocks needed) thread blocks.
// Fills the range fields of `b` and `split`, returns the grid.
constexpr int kItemTokens = 64;
inline kvbfp_status plan_persistent(const DecodeArgs& a, int fine_tokens, int capacity_blocks, int warps_per_block,
                                    DecodeArgs* b, Split* split, int* grid) {
    *b = a;
    const int64_t pairs = (int64_t)a.fmt.batch * a.fmt.n_kv_heads;
    b->item_tokens = a.chunk;
    b->items_per_pair = a.n_chunks;
    if (fine_tokens >= 16 && fine_tokens % 16 == 0 && fine_tokens < a.chunk && a.chunk % fine_tokens == 0) {   // (copies start on 16-token groups)
        const int R = a.chunk / fine_tokens;
        const int fine_per_pair = (a.len_cap + fine_tokens - 1) / fine_tokens;
        if (a.chunk == kMinChunk && a.n_chunks >= 2 &&
            pairs * fine_per_pair >= (int64_t)(2 * R + 1) * capacity_blocks * warps_per_block) {
            b->item_tokens = fine_tokens;
            b->items_per_pair = fine_per_pair;
        }
    }
    const int64_t n_items = pairs * b->items_per_pair;
    if (n_items >= (int64_t)1 << 31) return KVBFP_ERR_UNSUPPORTED;         // item indices are 32-bit in the kernels
    const int64_t want = (n_items + warps_per_block - 1) / warps_per_block;
    *grid = (int)(want < capacity_blocks ? want : capacity_blocks);
    split->n_warps = *grid * warps_per_block;
    split->item_tokens = b->item_tokens;
    split->items_per_pair = b->items_per_pair;
    b->range_items = split->range_items = (int)(n_items / split->n_warps);
    b->range_extra = split->range_extra = (int)(n_items % split->n_warps);
    return KVBFP_OK;
}
// The items of one (batch, kv head) that fall into a warp's item range (persistent kernels).
struct Run {
    int b, hk;
    int chunk0;        // first item within the pair: the slot of the chunk it lies in receives the partial result
    int n_items;       // items covered (>= 1)
    int n_tok;         // tokens that exist in them (0: nothing to do)
    int n_tiles;
    int64_t row0;      // first row in the planes
};
// 4-bit mantissas: integer scores + fp16 P.V, persistent
kvbfp_status launch_decode_mma4(const DecodeArgs& a, cudaStream_t s, Split* split);
// 8-bit mantissas, blocks of 32 slots or more: integer scores on the stored bytes + fp16 P.V, persistent
kvbfp_status launch_decode_mma8(const DecodeArgs& a, cudaStream_t s, Split* split);
// 6-bit mantissas, one query head per kv head, blocks of 32 slots or more: integer scores + fp16 P.V on the stored
// bytes and their masked copies, persistent
kvbfp_status launch_decode_mma6(const DecodeArgs& a, cudaStream_t s, Split* split);
size_t qfrag_bytes(const kvbfp_format& f, int n_q_heads);
// Events the caller asked to have recorded around the main decode kernel (nullptr = none).
void profile_events(cudaEvent_t* start, cudaEvent_t* stop);

}  // namespace kvbfp
