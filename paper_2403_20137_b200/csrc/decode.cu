// Decode-attention entry point: argument checks, sequence chunking, and the log-sum-exp merge of the
// per-chunk partial results (the split over sequence length).
#include <math.h>

#include "decode.cuh"

namespace kvbfp {
namespace {

// One warp per (batch, query head): out = sum_i 2^(m_i - m) o_i / sum_i 2^(m_i - m) l_i over the partial
// results of the row.  n_warps == 0: every chunk that holds tokens has its own partial (item = chunk).
// n_warps > 0: the items (pair-major pieces of item_tokens tokens) were cut into n_warps contiguous ranges and
// each range wrote one partial per (batch, kv head) it touches, at the slot of the chunk in which its first
// item there lies; the same integer arithmetic as in the kernel finds those slots.
// SPLIT: a thread block per row, its four warps take every fourth partial and their results are merged through
// shared memory (rows with many partials: long sequences cut into many ranges); else four rows per thread block.
template <bool SPLIT>
__global__ void __launch_bounds__(128) lse_merge(const float* __restrict__ partials, const int32_t* __restrict__ seq_lens,
                                                 const int32_t* __restrict__ inv_perm_v, float* __restrict__ out,
                                                 int n_rows, int n_q_heads, int group, int n_chunks, int chunk,
                                                 int len_cap, int n_warps, int item_tokens, int items_per_pair,
                                                 int range_items, int range_extra) {
    constexpr int D = kHeadDim;
    __shared__ float so[4][D];
    __shared__ float sml[4][2];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = SPLIT ? blockIdx.x : blockIdx.x * 4 + warp;           // b * Hq + hq
    pdl_wait();
    pdl_trigger();
    if (row >= n_rows) return;
    const int b = row / n_q_heads, hq = row % n_q_heads;
    const int len_raw = seq_lens[b];        // (on its way while the slots are worked out and the partials asked for)
    const float* base = partials + (int64_t)row * n_chunks * kPartStride;
    const int first = (b * (n_q_heads / group) + hq / group) * items_per_pair;   // first item of the pair
    // The partials of the row: with n_warps == 0 one per item that holds tokens; else one per range that holds such
    // items of the pair -- the ranges are consecutive, and the k-th of them starts inside the pair at the first item
    // of range w0 + k (the first one at item 0), so every lane finds its own partial without walking the others.
    // Where the partials lie does not depend on the sequence's length, only how many of them there are: the loads
    // go out for as many as the longest sequence allowed would have, and those beyond the real count are dropped
    // unread (their slots hold whatever an earlier call left there).
    const int nc_max = (len_cap + item_tokens - 1) / item_tokens;
    int w0 = 0, n_part_max = nc_max;
    if (n_warps > 0 && nc_max > 0) {
        w0 = range_of(first, range_items, range_extra);
        n_part_max = range_of(first + nc_max - 1, range_items, range_extra) - w0 + 1;
    }
    // this warp's share of them: all, or every fourth one starting at its own number
    auto share = [&](int n) { return SPLIT ? (n > warp ? (n - warp + 3) >> 2 : 0) : n; };
    const int n_sub_max = share(n_part_max);
    int n_part = -1;                         // (of the warp's share) known once the length has arrived
    float m = -INFINITY, l = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k0 = 0; k0 < n_sub_max; k0 += 32) {
        // a lane per partial: its slot, maximum and sum
        const int kk = k0 + lane;
        const bool may = kk < n_sub_max;
        const int k = SPLIT ? 4 * kk + warp : kk;
        int item = k;
        if (n_warps > 0) item = max(range_start(w0 + (may ? k : 0), range_items, range_extra) - first, 0);
        const int slot = may ? partial_slot(item, item_tokens, chunk, n_chunks) : 0;
        const float* pk = base + (int64_t)slot * kPartStride;
        const float mk_raw = may ? pk[D] : -INFINITY;
        const float lk_raw = may ? pk[D + 1] : 0.f;
        // the first eight vectors of this batch: every lane its four channels
        float4 o0[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int sj = __shfl_sync(0xffffffffu, slot, u);
            o0[u] = (k0 + u < n_sub_max) ? *reinterpret_cast<const float4*>(base + (int64_t)sj * kPartStride + lane * 4)
                                          : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (n_part < 0) {
            const int len = len_raw < 0 ? 0 : (len_raw > len_cap ? len_cap : len_raw);
            const int nc = (len + item_tokens - 1) / item_tokens;        // items that hold tokens
            n_part = nc;
            if (n_warps > 0 && nc > 0) n_part = range_of(first + nc - 1, range_items, range_extra) - w0 + 1;
            n_part = share(n_part);
        }
        if (k0 >= n_part) break;
        // the weights of the batch against the common maximum
        const bool have = kk < n_part;
        const float mk = have ? mk_raw : -INFINITY;
        const float lk = have ? lk_raw : 0.f;
        float mn = mk;
#pragma unroll
        for (int off = 16; off; off >>= 1) mn = fmaxf(mn, __shfl_xor_sync(0xffffffffu, mn, off));
        mn = fmaxf(mn, m);
        const float a1 = (m == -INFINITY) ? 0.f : exp2f(m - mn);
        const float ak = (mk == -INFINITY) ? 0.f : exp2f(mk - mn);
        float ls = ak * lk;
#pragma unroll
        for (int off = 16; off; off >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, off);
        acc.x *= a1; acc.y *= a1; acc.z *= a1; acc.w *= a1;
        l = l * a1 + ls;
        m = mn;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float aj = __shfl_sync(0xffffffffu, ak, u);              // 0 for lanes without a partial
            if (aj != 0.f) {                                               // (a dropped slot may hold anything)
                acc.x += aj * o0[u].x; acc.y += aj * o0[u].y; acc.z += aj * o0[u].z; acc.w += aj * o0[u].w;
            }
        }
        // the rest of the batch, eight loads at a time: lane j's slot and weight go round
        const int cnt = min(32, n_part - k0);
        for (int j0 = 8; j0 < cnt; j0 += 8) {
            float4 oi[8];
            float aj[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int sj = __shfl_sync(0xffffffffu, slot, (j0 + u) & 31);
                aj[u] = __shfl_sync(0xffffffffu, ak, (j0 + u) & 31);       // 0 for lanes without a partial
                oi[u] = (j0 + u < cnt) ? *reinterpret_cast<const float4*>(base + (int64_t)sj * kPartStride + lane * 4)
                                       : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                acc.x += aj[u] * oi[u].x; acc.y += aj[u] * oi[u].y; acc.z += aj[u] * oi[u].z; acc.w += aj[u] * oi[u].w;
            }
        }
    }
    if (SPLIT) {       // the four warps' results into warp 0
        *reinterpret_cast<float4*>(&so[warp][lane * 4]) = acc;
        if (lane == 0) { sml[warp][0] = m; sml[warp][1] = l; }
        __syncthreads();
        if (warp != 0) return;
        float mn = fmaxf(fmaxf(sml[0][0], sml[1][0]), fmaxf(sml[2][0], sml[3][0]));
        acc = make_float4(0.f, 0.f, 0.f, 0.f);
        l = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float a = (sml[w][0] == -INFINITY) ? 0.f : exp2f(sml[w][0] - mn);
            const float4 o = *reinterpret_cast<const float4*>(&so[w][lane * 4]);
            acc.x += a * o.x; acc.y += a * o.y; acc.z += a * o.z; acc.w += a * o.w;
            l += a * sml[w][1];
        }
        __syncwarp();                                   // so[0] is reused below
    }
    const float inv = (l > 0.f) ? 1.f / l : 0.f;
    float* dst = out + (int64_t)row * D;
    if (!inv_perm_v) {
        *reinterpret_cast<float4*>(dst + lane * 4) = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
    } else {
        so[warp][lane * 4 + 0] = acc.x * inv; so[warp][lane * 4 + 1] = acc.y * inv;
        so[warp][lane * 4 + 2] = acc.z * inv; so[warp][lane * 4 + 3] = acc.w * inv;
        __syncwarp();
        const int32_t* ip = inv_perm_v + (hq / group) * D;
#pragma unroll
        for (int k = 0; k < 4; ++k) dst[lane + 32 * k] = so[warp][ip[lane + 32 * k] & (D - 1)];
    }
}

inline int max_chunks(const kvbfp_format& f) { return (f.max_seq + kMinChunk - 1) / kMinChunk; }

thread_local cudaEvent_t t_ev_start = nullptr, t_ev_stop = nullptr;

}  // namespace

void profile_events(cudaEvent_t* start, cudaEvent_t* stop) {
    *start = t_ev_start;
    *stop = t_ev_stop;
}

size_t qfrag_bytes(const kvbfp_format& f, int n_q_heads) {
    const int group = n_q_heads / f.n_kv_heads;
    const int nt = (group + 3) / 4;                  // four query heads per 8-column MMA tile
    const size_t frag = (size_t)f.batch * f.n_kv_heads * nt * 8 * 32 * 2 * sizeof(uint32_t);
    const size_t qexp = ((size_t)f.batch * n_q_heads * 8 * sizeof(int32_t) + 255) & ~(size_t)255;   // per-query exponents and biases
    return frag + qexp;
}

}  // namespace kvbfp

extern "C" size_t kvbfp_decode_workspace_bytes(const kvbfp_format* fmt, int32_t n_q_heads) {
    using namespace kvbfp;
    if (check_format(fmt) != KVBFP_OK || n_q_heads < 1 || n_q_heads % fmt->n_kv_heads != 0) return 0;
    size_t part = (size_t)fmt->batch * n_q_heads * max_chunks(*fmt) * kPartStride * sizeof(float);
    return qfrag_bytes(*fmt, n_q_heads) + part;
}

namespace kvbfp {
namespace {
// The decode entry points: argument checks, chunking, main kernel, merge.  rope_theta != nullptr: keys are rotated
// to their positions after the read-back (fp32 kernel).
kvbfp_status decode_common(const kvbfp_cache* cache, const void* q, kvbfp_dtype q_dt, int32_t n_q_heads,
                           const int32_t* seq_lens, int32_t max_len_hint, const int32_t* perm_k,
                           const int32_t* inv_perm_v, float softmax_scale, int32_t q_mant_bits,
                           const double* rope_theta, const int32_t* rope_partner, const float* rope_sign,
                           float* out, void* workspace, size_t workspace_bytes, uint32_t flags, void* stream) {
    if (!cache) return KVBFP_ERR_INVALID_ARG;
    const kvbfp_format& f = cache->fmt;
    kvbfp_status st = check_format(&f);
    if (st != KVBFP_OK) return st;
    if (!cache->k_mant || !cache->k_exp || !cache->v_mant || !cache->v_exp || !q || !seq_lens || !out)
        return KVBFP_ERR_INVALID_ARG;
    if (n_q_heads < 1 || n_q_heads % f.n_kv_heads != 0) return KVBFP_ERR_INVALID_ARG;
    const int group = n_q_heads / f.n_kv_heads;
    if (group > 8) return KVBFP_ERR_UNSUPPORTED;
    if ((int64_t)f.batch * n_q_heads > (1 << 28)) return KVBFP_ERR_UNSUPPORTED;     // row counts are 32-bit in the kernels
    if (q_dt != KVBFP_F32 && q_dt != KVBFP_BF16) return KVBFP_ERR_INVALID_ARG;
    if (q_mant_bits != 0 && q_mant_bits != 8) return KVBFP_ERR_UNSUPPORTED;
    if (max_len_hint < 0 || !(softmax_scale >= 0.f) || isinf(softmax_scale)) return KVBFP_ERR_INVALID_ARG;
    uint32_t impl = flags & 0xffu, chunk_units = (flags >> 8) & 0xfffu;
    if (impl > KVBFP_DECODE_MMA_BF16 || (flags >> 20)) return KVBFP_ERR_INVALID_ARG;
    if (rope_theta) {
        if (impl != KVBFP_DECODE_AUTO && impl != KVBFP_DECODE_SIMT) return KVBFP_ERR_UNSUPPORTED;
        impl = KVBFP_DECODE_SIMT;
        // the rotation is carried from token to token in fp32: short chunks keep that chain short
        if (chunk_units == 0 || chunk_units > 4) chunk_units = 4;
    }
    const void* ptrs[] = {cache->k_mant, cache->k_exp, cache->v_mant, cache->v_exp, q, out, workspace, perm_k, inv_perm_v,
                          rope_theta, rope_partner, rope_sign};
    for (const void* p : ptrs)
        if (p && !aligned16(p)) return KVBFP_ERR_ALIGNMENT;
    const size_t need = kvbfp_decode_workspace_bytes(&f, n_q_heads);
    if (!workspace || workspace_bytes < need) return KVBFP_ERR_WORKSPACE;

    DecodeArgs a;
    a.fmt = f;
    a.k_mant = cache->k_mant; a.k_exp = cache->k_exp; a.v_mant = cache->v_mant; a.v_exp = cache->v_exp;
    a.q = q; a.q_is_bf16 = (q_dt == KVBFP_BF16); a.n_q_heads = n_q_heads;
    a.seq_lens = seq_lens; a.perm_k = perm_k; a.inv_perm_v = inv_perm_v;
    const float scale = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)f.head_dim);
    a.scale_log2e = scale * 1.4426950408889634f;
    a.q_mant_bits = q_mant_bits;
    a.rope_theta = rope_theta; a.rope_partner = rope_partner; a.rope_sign = rope_sign;
    a.out = out;
    a.qfrag = static_cast<uint32_t*>(workspace);
    a.partials = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + qfrag_bytes(f, n_q_heads));
    a.len_cap = (max_len_hint > 0 && max_len_hint < f.max_seq) ? max_len_hint : f.max_seq;

    // Sequence chunking: enough independent (batch, kv head, chunk) items to keep every warp slot of
    // the machine busy for a few rounds, chunks in multiples of kMinChunk tokens.
    const bool tensor_default = impl != KVBFP_DECODE_SIMT && impl != KVBFP_DECODE_MMA_BF16;
    const bool use_mma4 = tensor_default && f.mant_bits == 4;
    const bool use_mma8 = tensor_default && f.mant_bits == 8 && f.block >= 32;
    const bool use_mma6 = tensor_default && f.mant_bits == 6 && f.block >= 32 && group == 1;
    int chunk;
    if (chunk_units) {
        chunk = (int)chunk_units * kMinChunk;
    } else if (use_mma4 || use_mma8 || use_mma6) {
        chunk = kMinChunk;      // the persistent kernel balances by item count: finest items, one partial per range
    } else {
        const int64_t pairs = (int64_t)f.batch * f.n_kv_heads;
        int n_sm = 0;
        st = sm_count(&n_sm);
        if (st != KVBFP_OK) return st;
        const int64_t target_items = (int64_t)n_sm * 16 * 4;
        int64_t want = (target_items + pairs - 1) / pairs;
        if (want < 1) want = 1;
        int64_t per = (a.len_cap + want - 1) / want;
        chunk = (int)(((per + kMinChunk - 1) / kMinChunk) * kMinChunk);
        if (chunk < kMinChunk) chunk = kMinChunk;
    }
    a.chunk = chunk;
    a.n_chunks = (a.len_cap + chunk - 1) / chunk;
    st = status_word(&a.status);
    if (st != KVBFP_OK) return st;

    cudaStream_t s = (cudaStream_t)stream;
    a.item_tokens = a.chunk;
    a.items_per_pair = a.n_chunks;
    Split split;
    split.item_tokens = a.chunk;
    split.items_per_pair = a.n_chunks;
    if (impl == KVBFP_DECODE_SIMT) st = launch_decode_simt(a, s);
    else if (use_mma4) st = launch_decode_mma4(a, s, &split);
    else if (use_mma8) st = launch_decode_mma8(a, s, &split);
    else if (use_mma6) st = launch_decode_mma6(a, s, &split);
    else st = launch_decode_mma(a, s);
    if (st != KVBFP_OK) return st;
    const int n_rows = f.batch * n_q_heads;
    // partials per row, at most: a thread block per row where there are many (its warps share them)
    const int per_row = split.n_warps > 0 ? (split.items_per_pair + (split.range_items > 0 ? split.range_items : 1) - 1) /
                                                (split.range_items > 0 ? split.range_items : 1) + 1
                                          : a.n_chunks;
    if (per_row > 8)
        (void)launch_pdl(lse_merge<true>, dim3(n_rows), dim3(128), 0, s, (const float*)a.partials, seq_lens, inv_perm_v, out,
                         n_rows, n_q_heads, group, a.n_chunks, a.chunk, a.len_cap, split.n_warps, split.item_tokens,
                         split.items_per_pair, split.range_items, split.range_extra);
    else
        (void)launch_pdl(lse_merge<false>, dim3((n_rows + 3) / 4), dim3(128), 0, s, (const float*)a.partials, seq_lens, inv_perm_v, out,
                         n_rows, n_q_heads, group, a.n_chunks, a.chunk, a.len_cap, split.n_warps, split.item_tokens,
                         split.items_per_pair, split.range_items, split.range_extra);
    KVBFP_LAUNCH_CHECK("lse_merge");
    return KVBFP_OK;
}
}  // namespace
}  // namespace kvbfp

extern "C" kvbfp_status kvbfp_decode_attn(const kvbfp_cache* cache, const void* q, kvbfp_dtype q_dt,
                                          int32_t n_q_heads, const int32_t* seq_lens, int32_t max_len_hint,
                                          const int32_t* perm_k, const int32_t* inv_perm_v, float softmax_scale,
                                          int32_t q_mant_bits, float* out, void* workspace, size_t workspace_bytes,
                                          uint32_t flags, void* stream) {
    return kvbfp::decode_common(cache, q, q_dt, n_q_heads, seq_lens, max_len_hint, perm_k, inv_perm_v, softmax_scale,
                                q_mant_bits, nullptr, nullptr, nullptr, out, workspace, workspace_bytes, flags, stream);
}

extern "C" kvbfp_status kvbfp_decode_attn_rope(const kvbfp_cache* cache, const void* q, kvbfp_dtype q_dt,
                                               int32_t n_q_heads, const int32_t* seq_lens, int32_t max_len_hint,
                                               const int32_t* perm_k, const int32_t* inv_perm_v, float softmax_scale,
                                               const double* theta, const int32_t* partner, const float* sign,
                                               float* out, void* workspace, size_t workspace_bytes, uint32_t flags,
                                               void* stream) {
    if (!theta || !partner || !sign) return KVBFP_ERR_INVALID_ARG;
    return kvbfp::decode_common(cache, q, q_dt, n_q_heads, seq_lens, max_len_hint, perm_k, inv_perm_v, softmax_scale, 0,
                                theta, partner, sign, out, workspace, workspace_bytes, flags, stream);
}

// ---- diagnostics: the split arithmetic itself, callable from the host ----------------------------------------
extern "C" kvbfp_status kvbfp_split_plan(int32_t pairs, int32_t len_cap, int32_t chunk, int32_t fine_tokens,
                                         int32_t capacity_blocks, int32_t warps_per_block, int32_t* out6) {
    using namespace kvbfp;
    if (!out6 || pairs < 1 || len_cap < 1 || chunk < kMinChunk || chunk % kMinChunk != 0 || fine_tokens < 1 ||
        capacity_blocks < 1 || warps_per_block < 1)
        return KVBFP_ERR_INVALID_ARG;
    DecodeArgs a{};
    a.fmt.batch = pairs;
    a.fmt.n_kv_heads = 1;
    a.len_cap = len_cap;
    a.chunk = chunk;
    a.n_chunks = (len_cap + chunk - 1) / chunk;
    DecodeArgs b;
    Split split;
    int grid = 0;
    const kvbfp_status st = plan_persistent(a, fine_tokens, capacity_blocks, warps_per_block, &b, &split, &grid);
    if (st != KVBFP_OK) return st;
    out6[0] = grid; out6[1] = split.n_warps; out6[2] = split.item_tokens; out6[3] = split.items_per_pair;
    out6[4] = split.range_items; out6[5] = split.range_extra;
    return KVBFP_OK;
}
extern "C" int32_t kvbfp_split_range_start(int32_t w, int32_t range_items, int32_t range_extra) {
    return kvbfp::range_start(w, range_items, range_extra);
}
extern "C" int32_t kvbfp_split_range_of(int32_t x, int32_t range_items, int32_t range_extra) {
    return kvbfp::range_of(x, range_items, range_extra);
}
extern "C" int32_t kvbfp_split_partial_slot(int32_t item, int32_t item_tokens, int32_t chunk, int32_t n_chunks) {
    return kvbfp::partial_slot(item, item_tokens, chunk, n_chunks);
}

extern "C" kvbfp_status kvbfp_profile_decode_events(void* start_event, void* stop_event) {
    if ((start_event == nullptr) != (stop_event == nullptr)) return KVBFP_ERR_INVALID_ARG;
    kvbfp::t_ev_start = (cudaEvent_t)start_event;
    kvbfp::t_ev_stop = (cudaEvent_t)stop_event;
    return KVBFP_OK;
}

extern "C" size_t kvbfp_step_staging_bytes(const kvbfp_format* fmt, int32_t n_q_heads, kvbfp_dtype dt) {
    using namespace kvbfp;
    if (check_format(fmt) != KVBFP_OK || n_q_heads < 1 || (dt != KVBFP_F32 && dt != KVBFP_BF16)) return 0;
    const size_t es = dt == KVBFP_F32 ? 4 : 2;
    const size_t kv = (size_t)fmt->batch * fmt->n_kv_heads * fmt->head_dim * es;
    const size_t qb = (size_t)fmt->batch * n_q_heads * fmt->head_dim * es;
    const size_t ob = (size_t)fmt->batch * n_q_heads * fmt->head_dim * sizeof(float);
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    return up(kv) * 2 + up(qb) + up(ob);
}

extern "C" kvbfp_status kvbfp_decode_step_host(const kvbfp_cache* cache, const void* k_new_host,
                                               const void* v_new_host, const void* q_host, kvbfp_dtype dt,
                                               int32_t n_q_heads, const int32_t* start_pos, const int32_t* seq_lens,
                                               int32_t max_len_hint, const int32_t* perm_k, const int32_t* perm_v,
                                               const int32_t* inv_perm_v, float softmax_scale, float* out_host,
                                               void* staging, size_t staging_bytes, void* workspace,
                                               size_t workspace_bytes, uint32_t flags, void* stream) {
    using namespace kvbfp;
    if (!cache || !k_new_host || !v_new_host || !q_host || !out_host || !start_pos || !seq_lens)
        return KVBFP_ERR_INVALID_ARG;
    const size_t need = kvbfp_step_staging_bytes(&cache->fmt, n_q_heads, dt);
    if (need == 0) return KVBFP_ERR_INVALID_ARG;
    if (!staging || staging_bytes < need) return KVBFP_ERR_WORKSPACE;
    if (!aligned16(staging)) return KVBFP_ERR_ALIGNMENT;
    const kvbfp_format& f = cache->fmt;
    const size_t es = dt == KVBFP_F32 ? 4 : 2;
    const size_t kv = (size_t)f.batch * f.n_kv_heads * f.head_dim * es;
    const size_t qb = (size_t)f.batch * n_q_heads * f.head_dim * es;
    const size_t ob = (size_t)f.batch * n_q_heads * f.head_dim * sizeof(float);
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    uint8_t* base = static_cast<uint8_t*>(staging);
    uint8_t *dk = base, *dv = base + up(kv), *dq = base + 2 * up(kv), *dout = base + 2 * up(kv) + up(qb);
    cudaStream_t s = (cudaStream_t)stream;
    // Page-locked host buffers that this device can address are read and written by the kernels themselves.
    const void* hp[4] = {k_new_host, v_new_host, q_host, out_host};
    void* mapped[4] = {nullptr, nullptr, nullptr, nullptr};
    bool in_place = true;
    for (int i = 0; i < 4 && in_place; ++i) {
        cudaPointerAttributes at;
        const cudaError_t e = cudaPointerGetAttributes(&at, hp[i]);
        if (e != cudaSuccess) (void)cudaGetLastError();
        in_place = e == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer != nullptr &&
                   aligned16(at.devicePointer);
        mapped[i] = in_place ? at.devicePointer : nullptr;
    }
    if (in_place) {
        kvbfp_status st = kvbfp_append(cache, mapped[0], mapped[1], dt, 1, start_pos, perm_k, perm_v, stream);
        if (st != KVBFP_OK) return st;
        st = kvbfp_decode_attn(cache, mapped[2], dt, n_q_heads, seq_lens, max_len_hint, perm_k, inv_perm_v, softmax_scale,
                               0, static_cast<float*>(mapped[3]), workspace, workspace_bytes, flags, stream);
        if (st != KVBFP_OK) return st;
        KVBFP_CUDA(cudaStreamSynchronize(s));
        return KVBFP_OK;
    }
    KVBFP_CUDA(cudaMemcpyAsync(dk, k_new_host, kv, cudaMemcpyHostToDevice, s));
    KVBFP_CUDA(cudaMemcpyAsync(dv, v_new_host, kv, cudaMemcpyHostToDevice, s));
    KVBFP_CUDA(cudaMemcpyAsync(dq, q_host, qb, cudaMemcpyHostToDevice, s));
    kvbfp_status st = kvbfp_append(cache, dk, dv, dt, 1, start_pos, perm_k, perm_v, stream);
    if (st != KVBFP_OK) return st;
    st = kvbfp_decode_attn(cache, dq, dt, n_q_heads, seq_lens, max_len_hint, perm_k, inv_perm_v, softmax_scale, 0,
                           reinterpret_cast<float*>(dout), workspace, workspace_bytes, flags, stream);
    if (st != KVBFP_OK) return st;
    KVBFP_CUDA(cudaMemcpyAsync(out_host, dout, ob, cudaMemcpyDeviceToHost, s));
    KVBFP_CUDA(cudaStreamSynchronize(s));
    return KVBFP_OK;
}
