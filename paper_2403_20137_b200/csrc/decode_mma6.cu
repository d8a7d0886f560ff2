// Decode attention over a 6-bit BFP cache, one query head per kv head, blocks of 32 slots or more: integer
// tensor-core MMAs for the scores and fp16 tensor-core MMAs for P.V, both on the stored bytes with one mask per word
// (Sec. III par. 2 of the paper: keys are read back from the cache and multiplied with pi(q); Sec. II-B: the inner
// product of two BFP blocks is an integer product plus an exponent addition).
//
// Same launch design as the 4-bit kernel: work items laid out pair-major and cut into one contiguous range per
// resident warp (persistent), "runs" with one partial result each, a private ring of shared-memory stages per warp
// filled by 1-D bulk asynchronous copies, no block-wide barrier in the loop.
//
// Four 6-bit fields (excess-32 code, f = M + 32) fill three bytes:
//     b0 = f0 + 64 (f1 mod 4),   b1 = (f1 div 4) + 16 (f2 mod 16),   b2 = (f2 div 16) + 4 f3.
// Fields are never widened.  With the masked bytes m0 = b0 & 0x3F = f0, m1 = b1 & 0x0F = f1 div 4, m2 = b2 & 0x03 =
// f2 div 16 the sum q0 f0 + q1 f1 + q2 f2 + q3 f3 is linear in (b, m):
//     b0 (q1/64) + b1 (q2/16) + b2 (q3/4) + m0 (q0 - q1/64) + m1 (4 q1 - q2/16) + m2 (16 q2 - q3/4),
// so a packed word and the same word under one constant mask (the mask repeats every three words) are the two
// unsigned-byte operands of the MMAs, in the scores and in P.V alike.
//   Scores: the six coefficients of a 3-byte group differ by up to 2^10 (2^8 after the masked bytes are taken times
//   four), so they are cast to 24-bit fixed point with their block's exponent and split into THREE signed byte
//   digits, C = 65536 d2 + 256 d1 + d0.  The MMA columns keep the blocks apart (column = (block, digit), zeros
//   outside the block, two 8-column tiles), so one accumulator set per tile collects all blocks of a token and lane
//   (g, t) ends up with the three digit sums of (token g, block t).  The contribution of the excess-32 offsets (every
//   field 32: bytes 32, 8, 130, masked 32, 8, 2) is subtracted per digit, the digits are recombined, and one fp32
//   multiply applies 2^(e_k - 127) * scale * log2(e) * 2^(qe - 27).
//   P.V: a byte under a zero exponent field is the fp16 subnormal byte * 2^-24, so the V bytes need no arithmetic
//   either; the weight of (token, block) = softmax weight x 2^(e_v - D + 7), D a reference exponent byte raised tile
//   by tile, is formed in fp32 and travels as (hi, lo) fp16 halves in column (block, half).  Row "whole byte" and
//   row "masked byte" of every byte accumulate separately; the fields' sums are recombined once per run and the
//   offsets are taken out through the sum of the weights.
#include <math.h>

#include <atomic>
#include <type_traits>

#include "decode.cuh"
#include "ptx.cuh"

namespace kvbfp {
namespace {

constexpr int kWarps = 4;
constexpr int kMT = 4;                  // 16-token MMA row tiles per stage
constexpr int kTile = 16 * kMT;         // tokens per stage
constexpr int kStages = 2;
constexpr int kMinCtas = 2;
constexpr int D = kHeadDim;
constexpr int ROW_M = D * 6 / 8;        // 96 bytes of mantissas per token row
constexpr int kTopShiftH = 7;           // weight of a block at the reference exponent is 2^kTopShiftH (times the softmax
                                        // weight, at most 2^8, before it is cut into fp16 halves)
constexpr int kFlushStages = 4;         // stages between two removals of the excess-code offsets
constexpr int kDvHeadroom = 2;          // binades left above a tile's largest V exponent when the reference moves
constexpr int kFixBits = 23;            // coefficients are cast to round(c * 2^(kFixBits - qe)), |c| * 2^-qe < 0.99
                                        // (three signed byte digits hold up to 127.5 * 2^16)

// byte t (= byte index mod 3) of a 3-byte group: mask of its low field part, and its value when every field is 32
__host__ __device__ constexpr uint32_t low_mask(int t) { return t == 0 ? 0x3Fu : t == 1 ? 0x0Fu : 0x03u; }
__host__ __device__ constexpr int raw_at_zero(int t) { return t == 0 ? 32 : t == 1 ? 8 : 130; }
__host__ __device__ constexpr int low_at_zero(int t) { return t == 0 ? 32 : t == 1 ? 8 : 2; }
// mask of the low field parts of a word whose first byte has type s
__host__ __device__ constexpr uint32_t word_mask(int s) {
    return low_mask(s % 3) | (low_mask((s + 1) % 3) << 8) | (low_mask((s + 2) % 3) << 16) | (low_mask((s + 3) % 3) << 24);
}

template <int N>
struct Geo6 {
    static constexpr int ROW_E = D / N;
    static constexpr int KM_OFF = 0;
    static constexpr int VM_OFF = kTile * ROW_M;
    static constexpr int KE_OFF = 2 * kTile * ROW_M;
    static constexpr int VE_OFF = KE_OFF + kTile * ROW_E;
    static constexpr int STAGE_BYTES = 2 * kTile * (ROW_M + ROW_E);
    static constexpr int WARP_BYTES = kStages * STAGE_BYTES;
    static constexpr int DIG_OFF = kWarps * WARP_BYTES;                 // per warp: [kind][digit][ROW_M] signed bytes
    static constexpr int DIG_WARP = 2 * 3 * ROW_M;
    static constexpr int BAR_OFF = DIG_OFF + kWarps * DIG_WARP;
    static constexpr int SMEM_BYTES = BAR_OFF + kWarps * kStages * 8;
};

template <int N>
__global__ void __launch_bounds__(kWarps * 32, kMinCtas) decode_mma6(DecodeArgs a) {
    pdl_wait();
    using G_ = Geo6<N>;
    constexpr int ROW_E = G_::ROW_E;
    constexpr int NBLK = D / N;                       // blocks of a row
    constexpr int BLK_BYTES = N * 6 / 8;              // 24, 48 or 96
    constexpr int BLK_LANES = N / 4;                  // 3-byte groups (= lanes of the set-up) per block
    extern __shared__ __align__(128) uint8_t smem[];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int Hkv = a.fmt.n_kv_heads;
    const int wglob = blockIdx.x * kWarps + warp;
    const int i0 = range_start(wglob, a.range_items, a.range_extra);                  // this warp's items
    const int i1 = i0 + a.range_items + (wglob < a.range_extra ? 1 : 0);
    auto get_run = [&](int it) -> Run {
        Run r;
        const int pair = it / a.items_per_pair;
        r.chunk0 = it - pair * a.items_per_pair;
        r.b = pair / Hkv;
        r.hk = pair - r.b * Hkv;
        r.n_items = min(i1 - it, a.items_per_pair - r.chunk0);
        int len = a.seq_lens[r.b];
        if (len > a.fmt.max_seq || len < 0) {
            if (lane == 0 && r.chunk0 == 0 && r.hk == 0) raise_flag(a.status, KVBFP_FLAG_POSITION);
            len = len < 0 ? 0 : a.fmt.max_seq;
        }
        if (len > a.len_cap) {
            if (lane == 0 && r.chunk0 == 0 && r.hk == 0) raise_flag(a.status, KVBFP_FLAG_LEN_HINT);
            len = a.len_cap;
        }
        const int tok0 = r.chunk0 * a.item_tokens;
        const int64_t tok1 = (int64_t)(r.chunk0 + r.n_items) * a.item_tokens;
        r.n_tok = max(0, (int)min((int64_t)len, tok1) - tok0);
        r.n_tiles = (r.n_tok + kTile - 1) / kTile;
        r.row0 = (int64_t)pair * a.fmt.max_seq + tok0;
        return r;
    };

    uint8_t* wsm = smem + warp * G_::WARP_BYTES;
    int8_t* dig = reinterpret_cast<int8_t*>(smem + G_::DIG_OFF + warp * G_::DIG_WARP);
    const uint32_t wsm_u32 = smem_u32(wsm);
    const uint32_t bar0 = smem_u32(smem + G_::BAR_OFF + warp * kStages * 8);
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    // ---- producer: lanes 0..3 each own one of the four spans of a stage (K mantissas, V mantissas,
    // K exponents, V exponents).  The cursor (p_run, p_tile) runs ahead of the consumer by kStages tiles.
    const uint8_t* my_base = lane == 0 ? a.k_mant : lane == 1 ? a.v_mant : lane == 2 ? a.k_exp : a.v_exp;
    const int my_row_bytes = (lane < 2) ? ROW_M : ROW_E;
    const uint32_t my_dst = wsm_u32 + (lane == 0 ? G_::KM_OFF : lane == 1 ? G_::VM_OFF : lane == 2 ? G_::KE_OFF : G_::VE_OFF);
    int p_next = i0;
    Run pr;
    pr.n_tiles = 0;
    int p_tile = 0;
    auto issue_next = [&](int stage) {
        while (p_tile >= pr.n_tiles) {               // next run that has tokens
            if (p_next >= i1) return;
            pr = get_run(p_next);
            p_next += pr.n_items;
            p_tile = 0;
        }
        if (lane < 4) {
            const int off = p_tile * kTile;
            const int rows = min(kTile, ((pr.n_tok + 15) & ~15) - off);    // whole 16-token groups; stays below max_seq
            const uint32_t bar = bar0 + 8 * stage;
            if (lane == 0) mbar_expect_tx(bar, (uint32_t)(2 * rows * (ROW_M + ROW_E)));
            __syncwarp(0xfu);
            bulk_g2s(my_dst + stage * G_::STAGE_BYTES, my_base + (pr.row0 + off) * my_row_bytes, rows * my_row_bytes, bar);
        }
        ++p_tile;
    };
    for (int s = 0; s < kStages; ++s) issue_next(s);
    if (i0 >= i1) return;

    // per-lane constants
    // K: addresses for the 8 x 16-byte matrix loads: lane i names token row i % 8 (+ 8 for odd matrices) of matrix
    // i / 8; matrices 0, 1 = tokens 0..7 and 8..15 of 16-byte piece 2j, matrices 2, 3 = the same tokens of piece 2j + 1
    const int lm_off = G_::KM_OFF + (8 * ((lane >> 3) & 1) + (lane & 7)) * ROW_M + 16 * (lane >> 4);
    // word 4 p + t of a row (piece p, this lane's word) starts with a byte of type (p + t) mod 3
    const uint32_t mk0 = t % 3 == 0 ? word_mask(0) : t % 3 == 1 ? word_mask(1) : word_mask(2);         // pieces 0, 3
    const uint32_t mk1 = (t + 1) % 3 == 0 ? word_mask(0) : (t + 1) % 3 == 1 ? word_mask(1) : word_mask(2);   // pieces 1, 4
    const uint32_t mk2 = (t + 2) % 3 == 0 ? word_mask(0) : (t + 2) % 3 == 1 ? word_mask(1) : word_mask(2);   // pieces 2, 5
    // V: bytes [12g, 12g + 12) (slots 16g..16g+15, all in block 16g / N) of tokens t, t + 4, t + 8, t + 12
    const int v_off = G_::VM_OFF + t * ROW_M + 12 * g;
    // softmax weights travel from the lanes that computed them (token = lane / 4 and + 8, block = lane % 4)
    const int src_lo = 4 * t + (g >> 1), src_hi = 4 * (t + 4) + (g >> 1);
    const uint32_t half_sel = (g & 1) ? 0x7632u : 0x5410u;     // odd columns carry the lo halves
    constexpr int tb_mask = NBLK - 1;

    int stage = 0;
    uint32_t parity = 0;
    bool timed_out = false;

    for (int c_next = i0; c_next < i1 && !timed_out;) {
        const Run cr = get_run(c_next);
        c_next += cr.n_items;
        if (cr.n_tok == 0) continue;

        // ---- run set-up: the query coefficients, by this warp and for this (batch, kv head) -------------------
        // Lane L owns the 3-byte group L of a row: slots 4L..4L+3.
        uint32_t qb[2][3][2][2];          // B fragments [8-column tile][piece pair][whole / masked][piece of the pair]
        float qfac_h;                     // factor and digit offsets of this lane's block (block t)
        int qbias_h[3];
        {
            float v[4];
            {
                int ch[4];
                if (a.perm_k) {
                    const int4 p = __ldg(reinterpret_cast<const int4*>(a.perm_k + cr.hk * D + 4 * lane));
                    ch[0] = p.x; ch[1] = p.y; ch[2] = p.z; ch[3] = p.w;
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) ch[j] = 4 * lane + j;
                }
                const int64_t q_row = (int64_t)cr.b * Hkv + cr.hk;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t idx = q_row * D + (ch[j] & (D - 1));
                    v[j] = a.q_is_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(a.q)[idx]) : static_cast<const float*>(a.q)[idx];
                }
            }
            if (a.q_mant_bits) {          // BFP query (Sec. IV): blocks of N slots, 8-bit mantissas
                uint32_t am = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) am = max(am, __float_as_uint(v[j]) & 0x7fffffffu);
#pragma unroll
                for (int off = BLK_LANES >> 1; off; off >>= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
                int e8 = (int)(am >> 23);
                if (e8 == 255) { raise_flag(a.status, KVBFP_FLAG_NONFINITE); e8 = 254; }
                const int k = 127 - e8 + 6, k1 = k >> 1, k2 = k - k1;
                const float w = unit_weight(e8, 8);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float tv = (v[j] * pow2i(k1)) * pow2i(k2);
                    v[j] = rintf(fminf(fmaxf(tv, -127.f), 127.f)) * w;
                }
            }
            // coefficients of the whole bytes (c[0][type]) and of the masked bytes (c[1][type]).  The masked bytes are
            // small (at most 63, 15, 3) and enter the MMAs times four (the masked word shifted left by two bits, which
            // moves nothing across a byte): their coefficients, the largest of the six, shrink by four, and with them
            // the rounding unit that all six share -- it is the whole bytes, up to 255, that this unit multiplies
            float c[2][3];
            c[0][0] = v[1] * 0.015625f;  c[0][1] = v[2] * 0.0625f;  c[0][2] = v[3] * 0.25f;
            c[1][0] = (v[0] - c[0][0]) * 0.25f;  c[1][1] = v[1] - c[0][1] * 0.25f;  c[1][2] = 4.f * v[2] - c[0][2] * 0.25f;
            uint32_t am = 0;
#pragma unroll
            for (int kind = 0; kind < 2; ++kind)
#pragma unroll
                for (int ty = 0; ty < 3; ++ty) am = max(am, __float_as_uint(c[kind][ty]) & 0x7fffffffu);
#pragma unroll
            for (int off = BLK_LANES >> 1; off; off >>= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
            int e = (int)(am >> 23);
            if (e == 255) { raise_flag(a.status, KVBFP_FLAG_NONFINITE); e = 254; }
            // |c| * 2^-qe < 0.99: one more binade when the largest magnitude sits in the top percent of its own
            const int qe = (am == 0) ? 0 : e - 126 + ((am & 0x7fffffu) >= 0x7e0000u ? 1 : 0);
            const int sh = kFixBits - qe, h1 = sh / 2, h2 = sh - h1;  // two exact factors
            int bias[3] = {0, 0, 0};
            __syncwarp();                                             // (earlier readers of the digit bytes are done)
#pragma unroll
            for (int kind = 0; kind < 2; ++kind)
#pragma unroll
                for (int ty = 0; ty < 3; ++ty) {
                    const int C = __float2int_rn((c[kind][ty] * pow2i(h1)) * pow2i(h2));
                    const int C1 = (C + 128) >> 8, d0 = C - 256 * C1;           // C = 65536 d2 + 256 d1 + d0
                    const int d2 = (C1 + 128) >> 8, d1 = C1 - 256 * d2;
                    const int at0 = kind ? 4 * low_at_zero(ty) : raw_at_zero(ty);
                    bias[0] += at0 * d0; bias[1] += at0 * d1; bias[2] += at0 * d2;
                    dig[(kind * 3 + 0) * ROW_M + 3 * lane + ty] = (int8_t)d0;
                    dig[(kind * 3 + 1) * ROW_M + 3 * lane + ty] = (int8_t)d1;
                    dig[(kind * 3 + 2) * ROW_M + 3 * lane + ty] = (int8_t)d2;
                }
#pragma unroll
            for (int off = BLK_LANES >> 1; off; off >>= 1) {
#pragma unroll
                for (int d = 0; d < 3; ++d) bias[d] += __shfl_xor_sync(0xffffffffu, bias[d], off);
            }
            const float fac = pow2_split(a.scale_log2e, qe - kFixBits - 4);     // (2^-4: unit of a 6-bit mantissa)
            const int lead = (t < NBLK ? t : 0) * BLK_LANES;
            const float fac_t = __shfl_sync(0xffffffffu, fac, lead);
            qfac_h = t < NBLK ? fac_t : 0.f;
#pragma unroll
            for (int d = 0; d < 3; ++d) {
                const int b_t = __shfl_sync(0xffffffffu, bias[d], lead);
                qbias_h[d] = t < NBLK ? b_t : 0;
            }
            __syncwarp();
            // B fragments.  Tile 0: column g = (block g/2, digit d2 for even g, d1 for odd g); tile 1: column g = (block
            // g/2, digit d0) for even g, nothing for odd g.  A word of four bytes never straddles a block.
#pragma unroll
            for (int j = 0; j < 3; ++j)
#pragma unroll
                for (int kind = 0; kind < 2; ++kind)
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const int byte0 = 16 * (2 * j + half) + 4 * t;
                        const bool mine = byte0 / BLK_BYTES == (g >> 1);
                        const int8_t* base = dig + kind * 3 * ROW_M + byte0;
                        const uint32_t w2 = *reinterpret_cast<const uint32_t*>(base + 2 * ROW_M);
                        const uint32_t w1 = *reinterpret_cast<const uint32_t*>(base + 1 * ROW_M);
                        const uint32_t w0 = *reinterpret_cast<const uint32_t*>(base);
                        qb[0][j][kind][half] = mine ? ((g & 1) ? w1 : w2) : 0u;
                        qb[1][j][kind][half] = (mine && !(g & 1)) ? w0 : 0u;
                    }
        }

        // The V side finds its reference exponent on the way: every tile is checked against the current one
        // before it is used, and the reference is raised (the accumulators scaled down by the exact power of
        // two) when a tile holds a larger exponent byte.  The first tile of a run always raises it.
        int dv = 0;
        uint32_t dv_probe = 0x7FFF7FFFu;          // (0x7FFF - dv) in both halves: adding a byte > dv sets bit 15
        int wexp = 127 + kTopShiftH;              // exponent byte e gives the fp32 weight 2^(e - dv + kTopShiftH) = bits (e + wexp) << 23
        float wsum = 0.f;                         // this lane's weights (tokens g, g + 8, block t) since the last removal of the offsets
        int since_flush = 0;
        float o[12][4];                           // byte i of the lane's twelve: rows "whole byte" ([0], [1]) and "masked byte" ([2], [3])
#pragma unroll
        for (int r = 0; r < 12; ++r)
#pragma unroll
            for (int k = 0; k < 4; ++k) o[r][k] = 0.f;
        float m_run = -INFINITY, l_run = 0.f;

        constexpr int VE_WORDS = kTile * ROW_E / 4;      // V exponent bytes of a stage, in words
        auto raise_dv = [&](const uint8_t* st, int n_live) {
            const int n_bytes = min(n_live, kTile) * ROW_E;
            uint32_t m = 0;
            for (int w = lane; w < VE_WORDS; w += 32) {
                uint32_t x = *reinterpret_cast<const uint32_t*>(st + G_::VE_OFF + 4 * w);
                const int left = n_bytes - 4 * w;
                if (left < 4) x = left <= 0 ? 0u : (x & ((1u << (8 * left)) - 1u));
                m = vmaxu4(m, x);
            }
#pragma unroll
            for (int off = 16; off; off >>= 1) m = vmaxu4(m, __shfl_xor_sync(0xffffffffu, m, off));
            m = vmaxu4(m, m >> 16);
            m = vmaxu4(m, m >> 8);
            const int dt = (int)(m & 0xffu);
            if (dt > dv) {
                const int nd = min(dt + kDvHeadroom, 255);
                const float f = pow2_split(1.f, dv - nd);       // exact; underflows to 0 only with the sums it scales
#pragma unroll
                for (int r = 0; r < 12; ++r)
#pragma unroll
                    for (int k = 0; k < 4; ++k) o[r][k] *= f;
                dv = nd;
                dv_probe = (0x7FFFu - (uint32_t)nd) * 0x00010001u;
                wexp = 127 + kTopShiftH - nd;
                wsum *= f;
            }
        };
        // the V bytes enter the MMAs as they are stored, so per unit of weight every row carries the value its byte
        // has when all fields are 32 too much; taken out of the hi-half column of the sums every few stages, while
        // they are still small next to what they are taken from
        auto flush_offsets = [&]() {
            float w = wsum;
            w += __shfl_xor_sync(0xffffffffu, w, 4);
            w += __shfl_xor_sync(0xffffffffu, w, 8);
            w += __shfl_xor_sync(0xffffffffu, w, 16);
            w *= -5.9604644775390625e-8f;             // 2^-24: the bytes are fp16 subnormals
#pragma unroll
            for (int r = 0; r < 12; ++r) {
                o[r][0] += w * (float)raw_at_zero(r % 3);
                o[r][2] += w * (float)low_at_zero(r % 3);
            }
            wsum = 0.f;
            since_flush = 0;
        };

        // one stage of kTile tokens; FULL = every row of the tile exists
        auto tile_body = [&](const uint8_t* st, int n_live, auto full_tag) {
            constexpr bool FULL = decltype(full_tag)::value;
            // ---- V exponent bytes against the reference: even and odd bytes in 16-bit lanes, bit 15 = "larger"
            if (FULL) {
                uint32_t f = 0;
#pragma unroll
                for (int i = 0; i < (VE_WORDS + 31) / 32; ++i) {
                    const int w = lane + 32 * i;
                    if (VE_WORDS % 32 == 0 || w < VE_WORDS) {
                        const uint32_t x = *reinterpret_cast<const uint32_t*>(st + G_::VE_OFF + 4 * w);
                        f |= ((x & 0x00FF00FFu) + dv_probe) | (prmt(x, 0u, 0x4341u) + dv_probe);
                    }
                }
                if (__any_sync(0xffffffffu, (f & 0x80008000u) != 0u)) raise_dv(st, n_live);
            } else {
                raise_dv(st, n_live);         // rows past the end may hold anything: masked there
            }
            // ---- scores ---------------------------------------------------------
            float sc[kMT][2];
#pragma unroll
            for (int mt = 0; mt < kMT; ++mt) {
                if (!FULL && mt * 16 >= n_live) {
                    sc[mt][0] = sc[mt][1] = -INFINITY;
                    continue;
                }
                const uint32_t ka = smem_u32(st) + lm_off + mt * 16 * ROW_M;
                int acc0[4], acc1[4];
#pragma unroll
                for (int j = 0; j < 3; ++j) {
                    uint32_t u[4];            // tokens g, g + 8 of pieces 2j and 2j + 1: bytes 4t..4t+3 of each
                    ldmatrix_x4(u[0], u[1], u[2], u[3], ka + 32 * j);
                    const uint32_t ma = (2 * j) % 3 == 0 ? mk0 : (2 * j) % 3 == 1 ? mk1 : mk2;
                    const uint32_t mb = (2 * j + 1) % 3 == 0 ? mk0 : (2 * j + 1) % 3 == 1 ? mk1 : mk2;
                    if (j == 0) {
                        mma_u8s8_k32_first(acc0, u[0], u[1], u[2], u[3], qb[0][j][0][0], qb[0][j][0][1], 0, 0);
                        mma_u8s8_k32_first(acc1, u[0], u[1], u[2], u[3], qb[1][j][0][0], qb[1][j][0][1], 0, 0);
                    } else {
                        mma_u8s8_k32(acc0, u[0], u[1], u[2], u[3], qb[0][j][0][0], qb[0][j][0][1]);
                        mma_u8s8_k32(acc1, u[0], u[1], u[2], u[3], qb[1][j][0][0], qb[1][j][0][1]);
                    }
                    const uint32_t l0 = (u[0] & ma) << 2, l1 = (u[1] & ma) << 2, l2 = (u[2] & mb) << 2, l3 = (u[3] & mb) << 2;
                    mma_u8s8_k32(acc0, l0, l1, l2, l3, qb[0][j][1][0], qb[0][j][1][1]);
                    mma_u8s8_k32(acc1, l0, l1, l2, l3, qb[1][j][1][0], qb[1][j][1][1]);
                }
                // digits recombined (the lower two in integers, the top one in fp32: the whole would not fit 32 bits),
                // times 2^(e_k - 127) * factor for block t; then the four blocks of a token are added across the lanes t
                // (an exponent byte of 0 counts as weight 0)
                const uint32_t e0 = st[G_::KE_OFF + (mt * 16 + g) * ROW_E + (t & tb_mask)];
                const uint32_t e1 = st[G_::KE_OFF + (mt * 16 + g + 8) * ROW_E + (t & tb_mask)];
                const float lo0 = __int2float_rn(256 * (acc0[1] - qbias_h[1]) + (acc1[0] - qbias_h[0]));
                const float lo1 = __int2float_rn(256 * (acc0[3] - qbias_h[1]) + (acc1[2] - qbias_h[0]));
                float s0 = fmaf(__int2float_rn(acc0[0] - qbias_h[2]), 65536.f, lo0) * (__uint_as_float(e0 << 23) * qfac_h);
                float s1 = fmaf(__int2float_rn(acc0[2] - qbias_h[2]), 65536.f, lo1) * (__uint_as_float(e1 << 23) * qfac_h);
                s0 += __shfl_xor_sync(0xffffffffu, s0, 1);
                s1 += __shfl_xor_sync(0xffffffffu, s1, 1);
                s0 += __shfl_xor_sync(0xffffffffu, s0, 2);
                s1 += __shfl_xor_sync(0xffffffffu, s1, 2);
                if (!FULL) {       // select, not arithmetic: rows past the end may hold anything
                    if (mt * 16 + g >= n_live) s0 = -INFINITY;
                    if (mt * 16 + g + 8 >= n_live) s1 = -INFINITY;
                }
                sc[mt][0] = s0; sc[mt][1] = s1;
            }

            // ---- running softmax (reference point moves only in big steps) ------
            float mx = -INFINITY;
#pragma unroll
            for (int mt = 0; mt < kMT; ++mt) mx = fmaxf(mx, fmaxf(sc[mt][0], sc[mt][1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
            if (__any_sync(0xffffffffu, mx > m_run + 8.f)) {
                const float m_new = fmaxf(m_run, mx);
                const float alpha = (m_run == -INFINITY) ? 0.f : ex2_approx(m_run - m_new);
                m_run = m_new;
                l_run *= alpha;
                wsum *= alpha;
#pragma unroll
                for (int r = 0; r < 12; ++r)
#pragma unroll
                    for (int k = 0; k < 4; ++k) o[r][k] *= alpha;
            }

            // ---- P.V ------------------------------------------------------------
#pragma unroll
            for (int mt = 0; mt < kMT; ++mt) {
                if (!FULL && mt * 16 >= n_live) continue;
                const float p0 = ex2_approx(sc[mt][0] - m_run);
                const float p1 = ex2_approx(sc[mt][1] - m_run);
                l_run += p0 + p1;
                const int ev0 = st[G_::VE_OFF + (mt * 16 + g) * ROW_E + (t & tb_mask)];
                const int ev1 = st[G_::VE_OFF + (mt * 16 + g + 8) * ROW_E + (t & tb_mask)];
                float w0 = p0 * __int_as_float(max(ev0 + wexp, 0) << 23);
                float w1 = p1 * __int_as_float(max(ev1 + wexp, 0) << 23);
                if (!FULL) {       // rows past the end may hold any exponent byte: select, not arithmetic
                    if (mt * 16 + g >= n_live) w0 = 0.f;
                    if (mt * 16 + g + 8 >= n_live) w1 = 0.f;
                }
                wsum += w0 + w1;
                const float h0 = __uint_as_float(__float_as_uint(w0) & 0xffffe000u);
                const float h1 = __uint_as_float(__float_as_uint(w1) & 0xffffe000u);
                const uint32_t q0 = pack_f16x2_rn(h0, w0 - h0), q1 = pack_f16x2_rn(h1, w1 - h1);
                // B fragment for lane (g, t): column g = (block g/2, half g%2); tokens t, t+4 | t+8, t+12
                const uint32_t v0 = __shfl_sync(0xffffffffu, q0, src_lo);
                const uint32_t v1 = __shfl_sync(0xffffffffu, q0, src_hi);
                const uint32_t v2 = __shfl_sync(0xffffffffu, q1, src_lo);
                const uint32_t v3 = __shfl_sync(0xffffffffu, q1, src_hi);
                const uint32_t pb0 = prmt(v0, v1, half_sel), pb1 = prmt(v2, v3, half_sel);
                uint32_t vw[4][3];
#pragma unroll
                for (int k = 0; k < 4; ++k)
#pragma unroll
                    for (int j = 0; j < 3; ++j)
                        vw[k][j] = *reinterpret_cast<const uint32_t*>(st + v_off + (mt * 16 + 4 * k) * ROW_M + 4 * j);
#pragma unroll
                for (int x = 0; x < 6; ++x) {         // byte pair (2x, 2x+1) of the lane's twelve bytes
                    const uint32_t sel = (x & 1) ? 0x7632u : 0x5410u;
                    const uint32_t XA = prmt(vw[0][x >> 1], vw[1][x >> 1], sel);      // [tok.b, tok.b', tok'.b, tok'.b']
                    const uint32_t XB = prmt(vw[2][x >> 1], vw[3][x >> 1], sel);
                    const uint32_t me = low_mask((2 * x) % 3) * 0x00010001u, mo = low_mask((2 * x + 1) % 3) * 0x00010001u;
                    const uint32_t a_e = XA & 0x00FF00FFu, a_o = prmt(XA, 0u, 0x4341u);
                    const uint32_t b_e = XB & 0x00FF00FFu, b_o = prmt(XB, 0u, 0x4341u);
                    mma_f16(o[2 * x], a_e, XA & me, b_e, XB & me, pb0, pb1);
                    mma_f16(o[2 * x + 1], a_o, a_o & mo, b_o, b_o & mo, pb0, pb1);
                }
            }
        };

        for (int it = 0; it < cr.n_tiles; ++it) {
            if (!mbar_wait_bounded(bar0 + 8 * stage, parity)) { timed_out = true; break; }
            const uint8_t* st = wsm + stage * G_::STAGE_BYTES;
            const int n_live = cr.n_tok - it * kTile;        // tokens of this tile that exist (may exceed kTile)
            if (n_live >= kTile) tile_body(st, n_live, std::true_type{});
            else tile_body(st, n_live, std::false_type{});
            if (++since_flush == kFlushStages) flush_offsets();
            __syncwarp();
            issue_next(stage);
            if (++stage == kStages) { stage = 0; parity ^= 1u; }
        }
        if (timed_out) break;

        // ---- partial result of the run, at the slot of its first chunk ----------------------------
        // lane (g, t) holds, for the bytes 12g..12g+11 of the row, the sums weighted for block t: the lanes whose t
        // is the block of those bytes write them out.  With R = row "whole byte" and L = row "masked byte" of the
        // three bytes of a group:  f0 = L0, f1 = 4 L1 + (R0 - L0)/64, f2 = 16 L2 + (R1 - L1)/16, f3 = (R2 - L2)/4.
        flush_offsets();
        float l = l_run;
        l += __shfl_xor_sync(0xffffffffu, l, 4);
        l += __shfl_xor_sync(0xffffffffu, l, 8);
        l += __shfl_xor_sync(0xffffffffu, l, 16);
        if (t == (16 * g) / N) {
            // 2^24 undoes the subnormal scaling of the bytes (kept apart from the other factor: their product can
            // leave the fp32 range)
            const float vfac = pow2_split(1.f, dv - 131 - kTopShiftH);
            float* dst = a.partials + (((int64_t)cr.b * a.n_q_heads + cr.hk) * a.n_chunks + partial_slot(cr.chunk0, a.item_tokens, a.chunk, a.n_chunks)) * kPartStride;
#pragma unroll
            for (int m4 = 0; m4 < 4; ++m4) {
                float R[3], L[3];
#pragma unroll
                for (int i = 0; i < 3; ++i) {
                    R[i] = (o[3 * m4 + i][0] + o[3 * m4 + i][1]) * 16777216.f;
                    L[i] = (o[3 * m4 + i][2] + o[3 * m4 + i][3]) * 16777216.f;
                }
                float4 v;
                v.x = L[0] * vfac;
                v.y = (4.f * L[1] + (R[0] - L[0]) * 0.015625f) * vfac;
                v.z = (16.f * L[2] + (R[1] - L[1]) * 0.0625f) * vfac;
                v.w = ((R[2] - L[2]) * 0.25f) * vfac;
                reinterpret_cast<float4*>(dst + 16 * g)[m4] = v;
            }
            if (g == 0) { dst[D] = m_run; dst[D + 1] = l; }
        }
    }

    // the merge kernel is released only here: its thread blocks, dispatched while this kernel still streams, slowed
    // the SMs they landed on, and with one range per warp the slowest SM sets the time of the launch
    pdl_trigger();
    if (timed_out) {
        // give the copies still in flight a bounded chance to land before the shared memory is released
        if (lane == 0) raise_flag(a.status, KVBFP_FLAG_WAIT_TIMEOUT);
        for (int s = 0; s < kStages; ++s) {
            (void)mbar_wait_bounded(bar0 + 8 * s, 0);
            (void)mbar_wait_bounded(bar0 + 8 * s, 1);
        }
    }
}

template <int N>
kvbfp_status launch2(const DecodeArgs& a, cudaStream_t s, Split* split) {
    using G_ = Geo6<N>;
    static std::atomic<int> resident[64];   // thread blocks that fit the whole device, per device (0 = not asked yet)
    int dev = 0;
    KVBFP_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return KVBFP_ERR_UNSUPPORTED;
    if (!resident[dev].load(std::memory_order_acquire)) {
        KVBFP_CUDA(cudaFuncSetAttribute(decode_mma6<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, G_::SMEM_BYTES));
        int per_sm = 0, n_sm = 0;
        KVBFP_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_mma6<N>, kWarps * 32, G_::SMEM_BYTES));
        KVBFP_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
        if (per_sm < 1 || n_sm < 1) return KVBFP_ERR_CUDA;
        resident[dev].store(per_sm * n_sm, std::memory_order_release);
    }
    DecodeArgs b;
    int grid = 0;
    const kvbfp_status st = plan_persistent(a, kItemTokens, resident[dev].load(std::memory_order_relaxed), kWarps, &b, split, &grid);
    if (st != KVBFP_OK) return st;
    cudaEvent_t ev0, ev1;
    profile_events(&ev0, &ev1);
    if (ev0) KVBFP_CUDA(cudaEventRecord(ev0, s));
    (void)launch_pdl(decode_mma6<N>, dim3(grid), dim3(kWarps * 32), G_::SMEM_BYTES, s, b);
    KVBFP_LAUNCH_CHECK("decode_mma6");
    if (ev1) KVBFP_CUDA(cudaEventRecord(ev1, s));
    return KVBFP_OK;
}

}  // namespace

// 6-bit mantissas, one query head per kv head, blocks of 32 slots or more.
kvbfp_status launch_decode_mma6(const DecodeArgs& a, cudaStream_t s, Split* split) {
    switch (a.fmt.block) {
        case 32: return launch2<32>(a, s, split);
        case 64: return launch2<64>(a, s, split);
        case 128: return launch2<128>(a, s, split);
    }
    return KVBFP_ERR_UNSUPPORTED;
}

}  // namespace kvbfp
