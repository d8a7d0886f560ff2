// Decode attention over a 4-bit BFP cache: integer tensor-core MMAs for the scores, fp16 tensor-core MMAs
// with two mantissas per operand element for P.V
// (Sec. III par. 2 of the paper: keys are read back from the cache and multiplied with pi(q);
// Sec. II-B: a block's values are integer mantissas times one power of two).
//
// Work split.  The (batch, kv head, 128-token chunk) items are laid out pair-major and cut into one
// contiguous range per resident warp; the kernel is persistent (one launch fills the machine once).
// A warp walks its range as "runs" -- the chunks of one (batch, kv head) that fall into the range --
// keeping one set of accumulators per run and writing one partial result per run, at the slot of the
// run's first chunk.  Each warp has a private ring of shared-memory stages (an mbarrier per stage counts the
// bytes): the K and V mantissa tiles of 64 tokens arrive by tiled 2-D asynchronous copies over tensor maps of the
// two planes (rows of 128 bytes = two tokens, 16-byte pieces swizzled so that every fragment load below is free of
// bank conflicts), the exponent bytes by 1-D bulk copies; lanes 0..3 issue one piece each.  The copies run ahead
// across run boundaries, so a new run starts with its first tiles already on chip.  There is no block-wide
// barrier in the loop; every warp fetches its own tiles.
//
// Unpacking is what limits this kernel (instruction issue, not memory).  A packed byte holds
// two mantissas in excess-8 code: B = 16*(M_hi+8) + (M_lo+8).  fp16 path (P.V with several query heads; scores only
// for blocks of 16): fp16 has a 10-bit fraction, so the whole byte can be put under the bits of 1024.0 with one byte
// permute: the element
// 1024 + B.  A second element with the high nibble masked away and bit 7 set, 1024 + 128 + (M_lo+8),
// comes from one logic op.  One f16x2 fma per register with the block's power of two removes the
// common bias 1160 and applies the weight, exactly:
//     kind 1:  (16*M_hi + M_lo) * w        kind 2:  M_lo * w
// The two mantissas are then separated by linearity instead of by shifts:
//   scores:  q_hi*M_hi + q_lo*M_lo = (q_hi/16) * kind1 + (q_lo - q_hi/16) * kind2, so the query
//            fragment simply carries those two coefficients at the two k positions;
//   output:  the row of kind 1 accumulates 16*o_hi + o_lo and the row of kind 2 accumulates o_lo;
//            o_hi = (row1 - row2)/16 once, when the run's partial result is written.
//
// Scores for blocks of 32 slots or more use the integer tensor-core path instead (Sec. II-B of the paper:
// the inner product of two BFP blocks is an integer product plus an exponent addition); see "integer scores" below.
//
// Range of the fp16 path.  fp16 cannot hold 2^e for every exponent byte, so each run keeps a reference exponent
// byte D of its rows (of V, and of K when the scores use fp16) and uses the weights 2^(e - D + 5): the largest block gets
// 2^5 (the bias product 1160 * 2^5 still fits fp16), blocks more than 2^29 below the largest one of
// the run are flushed to zero (their contribution is below 2^-29 of it), and the common factor
// 2^(D - 134) is applied in fp32 to the partial output (and to fp16 scores).  The weights come from a
// shared-memory table addressed by exponent byte from a per-run base, so the subtraction costs
// nothing.  q and the softmax weights are carried as (hi, lo) fp16 pairs (q after a per-head
// power-of-two normalisation), accumulation is fp32.
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
constexpr int kMinCtas = 3;             // resident thread blocks per SM with several query heads in one 8-column tile; two
                                        // tiles (groups of 5 to 8 heads) run two blocks per SM: with three they spill, and
                                        // measured 9 % slower
constexpr int kMinCtasSingle = 2;       // one query head per kv head: two blocks (8 warps) per SM with up to 255 registers
                                        // measured 4 % faster than three (0.91 against 0.87 of the copy bandwidth on the
                                        // same box); grouped heads the other way round (0.73 against 0.76)
constexpr int D = kHeadDim;
constexpr int ROW_M = D / 2;            // 64 bytes of mantissas per token row
constexpr int kTopShift = 5;            // weight of the run's largest block is 2^kTopShift
constexpr int kTopShiftH = 7;           // the same in the single-head path, whose weights multiply the softmax weights
                                        // (at most 2^8) before they are cut into fp16 halves: 2^15 at the most
constexpr int kFlushStages = 4;         // single-head path: stages between two removals of the excess-code offsets
constexpr int kDvHeadroom = 2;          // binades left above a tile's largest V exponent when the reference moves
constexpr int kLutEntries = 512;        // index = exponent byte - D + 255, D = largest valid exponent byte

constexpr uint32_t kMagic = 0x64646464u;        // 0x64 = high byte of fp16 1024.0
constexpr uint32_t kBias = 0xE488E488u;         // fp16 -1160.0 twice

// Byte `byte` (0..63) of a row: low nibble = slot 2*byte, high nibble = slot 2*byte+1.
// K side, k position kk (0..3 = k 2t, 2t+1, 2t+8, 2t+9) of k-step ks for lane column t:
//   byte = 16t + 4(ks/2) + 2(ks%2) + (kk%2), kind 1 (whole byte) for kk < 2, kind 2 (low nibble) for kk >= 2.

// ------------------------------------------------------------------ query fragments
// One warp per (batch, kv head, n-tile).  Writes, in MMA B-fragment order, the (hi, lo) fp16 halves of
// the coefficients c1 = q_hi/16 (whole byte) and c2 = q_lo - q_hi/16 (low nibble), normalised per query
// head by a power of two 2^qe, and qe itself.
__global__ void __launch_bounds__(32) make_qfrag4(DecodeArgs a, int NT, int32_t* qmeta) {
    pdl_wait();
    pdl_trigger();
    const int N = a.fmt.block;
    const int lane = threadIdx.x, gp = lane >> 2, tp = lane & 3;
    const int item = blockIdx.x;
    const int nt = item % NT, hk = (item / NT) % a.fmt.n_kv_heads, b = item / NT / a.fmt.n_kv_heads;
    const int G = a.n_q_heads / a.fmt.n_kv_heads;
    __shared__ float sq[4][D];       // pi(q) of the four query heads of this n-tile, then the coefficients
    __shared__ int sqe[4];
    for (int i = lane; i < 4 * D; i += 32) {
        const int qq = 4 * nt + i / D, slot = i % D;
        float v = 0.f;
        if (qq < G) {
            const int ch = a.perm_k ? (a.perm_k[hk * D + slot] & (D - 1)) : slot;
            const int64_t idx = ((int64_t)b * a.n_q_heads + hk * G + qq) * D + ch;
            v = a.q_is_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(a.q)[idx]) : static_cast<const float*>(a.q)[idx];
        }
        sq[i / D][slot] = v;
    }
    __syncwarp();
    if (a.q_mant_bits) {   // BFP query (Sec. IV): blocks of N slots, 8-bit mantissas
        const int nblk = D / N;
        for (int i = lane; i < 4 * nblk; i += 32) {
            float* blk = &sq[i / nblk][(i % nblk) * N];
            uint32_t am = 0;
            for (int j = 0; j < N; ++j) am = max(am, __float_as_uint(blk[j]) & 0x7fffffffu);
            int e8 = (int)(am >> 23);
            if (e8 == 255) { raise_flag(a.status, KVBFP_FLAG_NONFINITE); e8 = 254; }
            const int k = 127 - e8 + 6, k1 = k >> 1, k2 = k - k1;
            const float w = unit_weight(e8, 8);
            for (int j = 0; j < N; ++j) {
                float tv = (blk[j] * pow2i(k1)) * pow2i(k2);
                blk[j] = rintf(fminf(fmaxf(tv, -127.f), 127.f)) * w;
            }
        }
        __syncwarp();
    }
    // coefficients in place: slot 2j <- c2 (low nibble), slot 2j+1 <- c1 (whole byte); per-head exponent.
    // Lane l owns bytes l and l + 32 (slots 2l, 2l+1, 2l+64, 2l+65).
    for (int qq = 0; qq < 4; ++qq) {
        const float c1a = sq[qq][2 * lane + 1] * 0.0625f, c2a = sq[qq][2 * lane] - c1a;
        const float c1b = sq[qq][2 * lane + 65] * 0.0625f, c2b = sq[qq][2 * lane + 64] - c1b;
        uint32_t am = max(max(__float_as_uint(c1a) & 0x7fffffffu, __float_as_uint(c2a) & 0x7fffffffu),
                          max(__float_as_uint(c1b) & 0x7fffffffu, __float_as_uint(c2b) & 0x7fffffffu));
#pragma unroll
        for (int off = 16; off; off >>= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
        int e = (int)(am >> 23);
        if (e == 255) { if (lane == 0) raise_flag(a.status, KVBFP_FLAG_NONFINITE); e = 254; }
        const int qe = (am == 0) ? 0 : e - 126;               // |c| * 2^-qe < 1
        // scale by 2^-qe in two exact steps (qe in [-126, 128])
        const int h1 = (-qe) / 2, h2 = (-qe) - h1;
        const float f1 = pow2i(h1), f2 = pow2i(h2);
        sq[qq][2 * lane] = (c2a * f1) * f2;       sq[qq][2 * lane + 1] = (c1a * f1) * f2;
        sq[qq][2 * lane + 64] = (c2b * f1) * f2;  sq[qq][2 * lane + 65] = (c1b * f1) * f2;
        if (lane == 0) sqe[qq] = qe;
    }
    __syncwarp();
    if (lane < 4 && 4 * nt + lane < G) qmeta[((int64_t)b * a.n_q_heads + hk * G + 4 * nt + lane) * 8] = sqe[lane];

    const int qi = 4 * nt + (gp >> 1), part = gp & 1;
    uint32_t* dst = a.qfrag + (int64_t)item * (8 * 32 * 2);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        uint32_t reg[2];
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {         // rr = 0: kind 1 (k 2t, 2t+1); rr = 1: kind 2 (k 2t+8, 2t+9)
            uint32_t h[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int byte = 16 * tp + 4 * (ks >> 1) + 2 * (ks & 1) + e;
                const float v = sq[gp >> 1][2 * byte + (rr == 0 ? 1 : 0)];
                const __half hi = __float2half_rn(v);
                __half out = part ? __float2half_rn(v - __half2float(hi)) : hi;
                if (qi >= G) out = __ushort_as_half(0);
                h[e] = __half_as_ushort(out);
            }
            reg[rr] = h[0] | (h[1] << 16);
        }
        const int wd = 2 * ks;
        dst[((wd >> 2) * 32 + lane) * 4 + (wd & 3)] = reg[0];
        dst[((wd >> 2) * 32 + lane) * 4 + (wd & 3) + 1] = reg[1];
    }
}

// ---- integer scores (blocks of 32 slots or more) --------------------------------------------------------------
// The K bytes enter unsigned-byte x signed-byte MMAs twice: as they are, and as the packed 32-bit word shifted left
// by four bits WITHOUT a mask: byte i of that is 16 * lo_i + hi_(i-1) (nothing for i = 0), still linear in the
// nibbles.  The two coefficient rows a (whole byte) and b (shifted word) therefore solve, per word and from its last
// byte down,
//     16 a_i + b_(i+1) = q_hi_i,   a_i + 16 b_i = q_lo_i        (b_4 = 0)
// They are cast to 15-bit fixed point, C = round(c * 2^(14 - qe)), with the exponent qe of their block and written as
// two signed byte digits, C = 256 * d1 + d0, which sit in two MMA columns; the two 32-bit sums of a (token, block) are
// recombined exactly, the constant contribution of the excess-8 offsets (136 per whole byte, 136 per shifted byte
// but 128 for byte 0 of a word) goes into the accumulator beforehand, and one fp32 multiply-add applies
// 2^(e_k - 127) * scale * log2(e) * 2^(qe - 16) per (token, block) (the factor 2^-2 of the mantissa unit included).

// With one query head per kv head these coefficients are formed inside the main kernel, by the warp itself at the
// start of each run and in registers: the query row is 512 bytes, and a launch of its own for it cost more than the
// arithmetic.  With several heads a small kernel writes them out beforehand (make_qfrag4i).

// What lane L = lane % 16 holds of one query head after query_word(): the digit bytes of packed word L (bytes
// 4L..4L+3 of a row, slots 8L..8L+7), four per register, for the whole-byte row (a) and the shifted-word row (b), and
// the factor and the offsets' contribution of the block the word lies in.  Lanes 16..31 do the same for a head of their
// own (or mirror lanes 0..15).
struct QWord {
    uint32_t a_d1, a_d0, b_d1, b_d0;
    float fac;        // scale * log2(e) * 2^(qe - 16)
    int bias;         // 136 * sum(C of whole bytes) + 136 * sum(C of shifted bytes), 128 for byte 0 of a word
};
// Channels of the eight slots of this lane's word (the permutation of kv head hk, or the identity).
__device__ __forceinline__ void query_channels(const DecodeArgs& a, int hk, int lane, int (&ch)[8]) {
    const int L = lane & 15;
    if (a.perm_k) {
        const int4 p0 = __ldg(reinterpret_cast<const int4*>(a.perm_k + hk * D + 8 * L));
        const int4 p1 = __ldg(reinterpret_cast<const int4*>(a.perm_k + hk * D + 8 * L) + 1);
        ch[0] = p0.x; ch[1] = p0.y; ch[2] = p0.z; ch[3] = p0.w; ch[4] = p1.x; ch[5] = p1.y; ch[6] = p1.z; ch[7] = p1.w;
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) ch[j] = 8 * L + j;
    }
}
// pi(q) of those slots for row q_row of q (!live: a head that does not exist, all zeros).
__device__ __forceinline__ void query_values(const DecodeArgs& a, int64_t q_row, bool live, const int (&ch)[8], float (&v)[8]) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        v[j] = 0.f;
        if (live) {
            const int64_t idx = q_row * D + (ch[j] & (D - 1));
            v[j] = a.q_is_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(a.q)[idx]) : static_cast<const float*>(a.q)[idx];
        }
    }
}
// The coefficient rows of one query head from its values v (each half warp may work on a head of its own: nothing
// crosses the halves); with q_mant_bits first the BFP16 cast of Sec. IV (blocks of N slots, 8-bit mantissas).
template <int N>
__device__ __forceinline__ QWord query_word(const DecodeArgs& a, float (&v)[8]) {
    constexpr int wpb = N / 8;                 // 4-byte words (= lanes) per block
    if (a.q_mant_bits) {
        uint32_t am = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) am = max(am, __float_as_uint(v[j]) & 0x7fffffffu);
#pragma unroll
        for (int off = wpb >> 1; off; off >>= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
        int e8 = (int)(am >> 23);
        if (e8 == 255) { raise_flag(a.status, KVBFP_FLAG_NONFINITE); e8 = 254; }
        const int k = 127 - e8 + 6, k1 = k >> 1, k2 = k - k1;
        const float w = unit_weight(e8, 8);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float tv = (v[j] * pow2i(k1)) * pow2i(k2);
            v[j] = rintf(fminf(fmaxf(tv, -127.f), 127.f)) * w;
        }
    }
    // byte i of the word: low nibble = slot 2i, high nibble = slot 2i + 1; solved from the last byte down
    float ca[4], cb[4];
    uint32_t am = 0;
    float b_next = 0.f;
#pragma unroll
    for (int i = 3; i >= 0; --i) {
        ca[i] = (v[2 * i + 1] - b_next) * 0.0625f;
        cb[i] = (v[2 * i] - ca[i]) * 0.0625f;
        b_next = cb[i];
        am = max(am, max(__float_as_uint(ca[i]) & 0x7fffffffu, __float_as_uint(cb[i]) & 0x7fffffffu));
    }
#pragma unroll
    for (int off = wpb >> 1; off; off >>= 1) am = max(am, __shfl_xor_sync(0xffffffffu, am, off));
    int e = (int)(am >> 23);
    if (e == 255) { raise_flag(a.status, KVBFP_FLAG_NONFINITE); e = 254; }
    const int qe = (am == 0) ? 0 : e - 126;                   // |c| * 2^-qe < 1
    const int sh = 14 - qe, h1 = sh / 2, h2 = sh - h1;        // two exact factors (sh in [-114, 140])
    QWord w;
    w.a_d1 = w.a_d0 = w.b_d1 = w.b_d0 = 0u;
    w.bias = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int Ca = __float2int_rn((ca[i] * pow2i(h1)) * pow2i(h2));
        const int Cb = __float2int_rn((cb[i] * pow2i(h1)) * pow2i(h2));
        w.bias += 136 * Ca + (i == 0 ? 128 : 136) * Cb;
        const int a1 = (Ca + 128) >> 8, a0 = Ca - 256 * a1;   // C = 256 * d1 + d0, both signed bytes
        const int b1 = (Cb + 128) >> 8, b0 = Cb - 256 * b1;
        w.a_d1 |= ((uint32_t)a1 & 0xffu) << (8 * i);  w.a_d0 |= ((uint32_t)a0 & 0xffu) << (8 * i);
        w.b_d1 |= ((uint32_t)b1 & 0xffu) << (8 * i);  w.b_d0 |= ((uint32_t)b0 & 0xffu) << (8 * i);
    }
#pragma unroll
    for (int off = wpb >> 1; off; off >>= 1) w.bias += __shfl_xor_sync(0xffffffffu, w.bias, off);
    w.fac = pow2_split(a.scale_log2e, qe - 16);
    return w;
}

// Several query heads per kv head: one warp per (batch, kv head, n-tile) writes the B fragments of the 32-byte-deep
// MMAs -- word 2 * seg + kind covers the bytes [16 seg, 16 seg + 16) of a row (kind 0: whole bytes, kind 1: shifted
// words); lane (g, t) holds bytes 4t..4t+3 for column g = (query g/2, digit g%2: 0 = d1, 1 = d0) -- and, per query
// head, qmeta[8 q + 2 blk] = factor (float bits), qmeta[8 q + 2 blk + 1] = offsets' contribution.  The two half warps
// take the query heads (0, 1) of the n-tile, then (2, 3); all loads go out first.
template <int N>
__global__ void __launch_bounds__(128) make_qfrag4i(DecodeArgs a, int NT, int32_t* qmeta) {
    pdl_wait();
    pdl_trigger();
    constexpr int NBLK = D / N;
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int item = blockIdx.x * 4 + (threadIdx.x >> 5);
    if (item >= a.fmt.batch * a.fmt.n_kv_heads * NT) return;
    const int nt = item % NT, hk = (item / NT) % a.fmt.n_kv_heads, b = item / NT / a.fmt.n_kv_heads;
    const int Gq = a.n_q_heads / a.fmt.n_kv_heads;
    // The four query rows of the n-tile are parked in shared memory by 16-byte loads that do not wait for the
    // permutation's indices, and pi(q) is gathered from there (one memory round trip instead of two).
    __shared__ __align__(16) float srow[4][4][D];                 // [warp][head of the n-tile][channel], raw bits
    const int es = a.q_is_bf16 ? 2 : 4;
    const int pieces = 4 * D * es / 16;                           // 16-byte pieces of the four rows: 64 or 128
    uint8_t* park = reinterpret_cast<uint8_t*>(&srow[threadIdx.x >> 5][0][0]);
    uint4 raw[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int pc = lane + 32 * i;                             // piece pc: head pc / (pieces / 4), piece of its row
        raw[i] = make_uint4(0u, 0u, 0u, 0u);
        if (pc < pieces) {
            const int hq = pc / (pieces / 4), off = pc % (pieces / 4);
            const int qi = 4 * nt + hq;
            if (qi < Gq)
                raw[i] = __ldg(reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(a.q) +
                                                              ((int64_t)b * a.n_q_heads + hk * Gq + qi) * D * es) + off);
        }
    }
    int ch[8];
    float qv[2][8];
    query_channels(a, hk, lane, ch);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int pc = lane + 32 * i;
        if (pc < pieces) {
            const int hq = pc / (pieces / 4), off = pc % (pieces / 4);
            *reinterpret_cast<uint4*>(park + hq * (D * 4) + off * 16) = raw[i];     // (rows 512 bytes apart either way)
        }
    }
    __syncwarp();
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
        const int hq = 2 * pass + (lane >> 4);
        const uint8_t* row = park + hq * (D * 4);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int c = ch[j] & (D - 1);
            qv[pass][j] = a.q_is_bf16 ? __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(row)[c] << 16)
                                      : reinterpret_cast<const float*>(row)[c];
        }
    }
    uint32_t qi8[8];
#pragma unroll
    for (int pass = 0; pass < 2; ++pass) {
        const QWord w = query_word<N>(a, qv[pass]);
#pragma unroll
        for (int hw = 0; hw < 2; ++hw) {          // the head worked out by half warp hw in this pass
            const int qq = 2 * pass + hw;
            const bool mine = (g >> 1) == qq;
#pragma unroll
            for (int m = 0; m < 8; ++m) {
                const int seg = m >> 1, kind = m & 1;
                const uint32_t d1 = __shfl_sync(0xffffffffu, kind ? w.b_d1 : w.a_d1, 16 * hw + 4 * seg + t);
                const uint32_t d0 = __shfl_sync(0xffffffffu, kind ? w.b_d0 : w.a_d0, 16 * hw + 4 * seg + t);
                if (mine) qi8[m] = (g & 1) ? d0 : d1;
            }
            const int qi = 4 * nt + qq;
            if (qi < Gq && (lane & 15) % (N / 8) == 0 && (lane >> 4) == hw) {      // block leaders of that half warp
                int32_t* meta = qmeta + ((int64_t)b * a.n_q_heads + hk * Gq + qi) * 8;
                const int k = (lane & 15) / (N / 8);
                meta[2 * k] = __float_as_int(w.fac);
                meta[2 * k + 1] = w.bias;
            }
        }
    }
    static_assert(NBLK >= 1, "");
    uint32_t* dst = a.qfrag + (int64_t)item * (8 * 32);
#pragma unroll
    for (int m = 0; m < 8; ++m) dst[((m >> 2) * 32 + lane) * 4 + (m & 3)] = qi8[m];
}

// ------------------------------------------------------------------ main kernel
// Shared memory of a thread block.  The mantissa tiles come first: every (warp, stage) has a K tile and a V tile of
// kTile token rows x 64 bytes, each 4 KiB and aligned to 1 KiB.  They are filled by tiled 2-D copies that take the
// plane as rows of 128 bytes (two tokens: whole 128-byte lines move) and swizzle the 16-byte pieces of such a row,
// piece ^ (row % 8): token rows are 64 bytes apart, so without it the same piece of tokens g and g + 2 would sit in the
// same banks.  Exponent bytes, the weight table and the barriers follow.
constexpr int kTileBytes = kTile * ROW_M;
template <int N>
struct Geo4 {
    static constexpr int ROW_E = D / N;
    static constexpr int MANT_STAGE = 2 * kTileBytes;                   // K tile, V tile
    static constexpr int KM_OFF = 0;
    static constexpr int VM_OFF = kTileBytes;
    static constexpr int EXP_OFF = kWarps * kStages * MANT_STAGE;       // per (warp, stage): K bytes, V bytes
    static constexpr int EXP_STAGE = 2 * kTile * ROW_E;
    static constexpr int KE_OFF = 0;
    static constexpr int VE_OFF = kTile * ROW_E;
    static constexpr int LUT_OFF = EXP_OFF + kWarps * kStages * EXP_STAGE;   // uint2[kLutEntries]
    static constexpr int BAR_OFF = LUT_OFF + kLutEntries * 8;
    static constexpr int SMEM_BYTES = BAR_OFF + kWarps * kStages * 8;
};
// Offset of 16-byte piece `piece` (0..3) of token row `tok` inside a swizzled tile.
__device__ __forceinline__ int swz(int tok, int piece) {
    return (tok >> 1) * 128 + (((4 * (tok & 1) + piece) ^ ((tok >> 1) & 7)) << 4);
}
// P.V: lane column t holds tokens tok4(t, 0..3) of a 16-token row tile as the k positions (2t, 2t+1, 2t+8, 2t+9) of the
// MMA.  Which tokens is free (the softmax weights are brought along); these make the 8-byte V loads of a half warp
// (tokens tok4(0..3, k), pieces 0 and 1 or 2 and 3) fall into distinct banks of the swizzled tile.
__host__ __device__ constexpr int tok4(int t, int k) { return (t & 1) + 4 * (t >> 1) + 2 * (k & 1) + 8 * (k >> 1); }

// Largest of the first `bytes` bytes of a 16-byte-aligned span in global memory, over the warp.  Whole
// 16-byte vectors are loaded (the span is padded to a multiple of 16 inside the plane); bytes past
// `bytes` are masked out.
__device__ __forceinline__ int warp_max_byte(const uint8_t* p, int bytes, int lane) {
    uint32_t m = 0;
    const uint4* v = reinterpret_cast<const uint4*>(p);
    const int n_vec = (bytes + 15) >> 4;
    auto masked = [&](uint4 x, int i) -> uint32_t {
        const int left = bytes - 16 * i;                 // valid bytes in this vector (may exceed 16)
        if (left < 16) {
            uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int r = left - 4 * k;
                w[k] = r >= 4 ? w[k] : (r <= 0 ? 0u : (w[k] & ((1u << (8 * r)) - 1u)));
            }
            x = make_uint4(w[0], w[1], w[2], w[3]);
        }
        return vmaxu4(vmaxu4(x.x, x.y), vmaxu4(x.z, x.w));
    };
    // eight vectors per lane in flight at a time: the pass is latency, not bandwidth
    for (int i0 = lane; i0 < n_vec; i0 += 8 * 32) {
        uint4 x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = i0 + 32 * u;
            x[u] = i < n_vec ? __ldg(v + i) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) m = vmaxu4(m, masked(x[u], i0 + 32 * u));
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) m = vmaxu4(m, __shfl_xor_sync(0xffffffffu, m, off));
    m = vmaxu4(m, m >> 16);
    m = vmaxu4(m, m >> 8);
    return (int)(m & 0xffu);
}

// MHA: one query head per kv head and blocks of 32 slots or more -- the MMA columns separate the blocks of a row
// instead of the query heads (see make_qfrag4h), in the scores and in P.V.
template <int N, int NT, bool MHA>
__global__ void __launch_bounds__(kWarps * 32, MHA ? kMinCtasSingle : (NT == 1 ? kMinCtas : 2))
decode_mma4(DecodeArgs a, const int32_t* __restrict__ qmeta, const __grid_constant__ CUtensorMap k_map,
            const __grid_constant__ CUtensorMap v_map) {
    using G_ = Geo4<N>;
    constexpr int ROW_E = G_::ROW_E;
    constexpr int NBK = (N == 16) ? 2 : 1;            // blocks inside a K lane chunk of 32 slots
    constexpr bool KI = (N >= 32);                    // integer MMA path for the scores
    constexpr int NBLK = KI ? D / N : 1;              // blocks of a row (integer path)
    static_assert(!MHA || (KI && NT == 1), "the single-head path is built on the integer scores");
    extern __shared__ __align__(1024) uint8_t smem[];         // the swizzle pattern is a function of the address
    pdl_wait();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int Hkv = a.fmt.n_kv_heads, Gq = a.n_q_heads / Hkv;
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

    if (smem_u32(smem) & 1023u) {        // never expected: the tiles would be read with the wrong pattern
        if (threadIdx.x == 0) raise_flag(a.status, KVBFP_FLAG_WAIT_TIMEOUT);
        return;                          // (the whole block, before any copy is issued)
    }
    uint8_t* wsm = smem + warp * kStages * G_::MANT_STAGE;                          // this warp's mantissa tiles
    uint8_t* wse = smem + G_::EXP_OFF + warp * kStages * G_::EXP_STAGE;             // and exponent bytes
    const uint32_t wsm_u32 = smem_u32(wsm), wse_u32 = smem_u32(wse);
    const uint32_t bar0 = smem_u32(smem + G_::BAR_OFF + warp * kStages * 8);
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) mbar_init(bar0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    // ---- producer: lanes 0..3 each own one of the four pieces of a stage: the K and V mantissa tiles (tiled copies of
    // kTile whole rows: rows past the sequence are never used, rows past the plane arrive as zeros) and the K and V
    // exponent bytes (1-D copies of the 16-token groups that hold tokens).  The cursor (p_run, p_tile) runs ahead of
    // the consumer by kStages tiles.
    const uint8_t* my_exp = lane == 2 ? a.k_exp : a.v_exp;
    const CUtensorMap* my_map = lane == 0 ? &k_map : &v_map;
    const uint32_t my_dst = lane < 2 ? wsm_u32 + (lane == 0 ? G_::KM_OFF : G_::VM_OFF)
                                     : wse_u32 + (lane == 2 ? G_::KE_OFF : G_::VE_OFF);
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
            if (lane == 0) mbar_expect_tx(bar, (uint32_t)(2 * kTileBytes + 2 * rows * ROW_E));
            __syncwarp(0xfu);
            if (lane < 2) tensor_g2s_2d(my_dst + stage * G_::MANT_STAGE, my_map, 0, (int)((pr.row0 + off) >> 1), bar);
            else bulk_g2s(my_dst + stage * G_::EXP_STAGE, my_exp + (pr.row0 + off) * ROW_E, rows * ROW_E, bar);
        }
        ++p_tile;
    };
    for (int s = 0; s < kStages; ++s) issue_next(s);

    // (the table is filled while the first copies are in flight)
    // weight table: entry i = (2^(i - 255 + kTopShift) twice as f16x2, the same times -1160); entries
    // above 255 belong to rows that are masked later (past the end of the run) and only have to exist
    uint2* lut = reinterpret_cast<uint2*>(smem + G_::LUT_OFF);
    if (!MHA)
        for (int i = threadIdx.x; i < kLutEntries; i += kWarps * 32) {
            const uint32_t s2 = (i <= 255 ? pow2_f16(i - 255 + kTopShift) : 0u) * 0x00010001u;
            lut[i] = make_uint2(s2, mul_f16x2(s2, kBias));
        }
    __syncthreads();
    if (i0 >= i1) return;

    // per-lane byte offsets inside a stage (mantissa tiles swizzled, see Geo4)
    const int k_off = G_::KM_OFF + swz(g, t);                  // 16 bytes [16t, 16t + 16) of token g,
    const int k_off8 = G_::KM_OFF + swz(g + 8, t);             // of token g + 8
    // integer scores: addresses for the 8 x 16-byte matrix loads.  Lane i names token row i % 8 of matrix i / 8;
    // matrices 0, 1 = tokens 0..7 and 8..15 of 16-byte piece 0 (piece j: address ^ (j << 4)), matrices 2, 3 (loads
    // of four) = the same tokens of piece 1
    const int lm_off = G_::KM_OFF + swz(8 * ((lane >> 3) & 1) + (lane & 7), lane >> 4);
    const int kei_off = G_::KE_OFF + g * ROW_E;
    const int ke_off = G_::KE_OFF + g * ROW_E + ((N == 16) ? 2 * t : (N == 32) ? t : (N == 64) ? (t >> 1) : 0);
    int v_off[4], ve_off[4];                                   // bytes [8g, 8g + 8) of rows tok4(t, k)
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        v_off[k] = G_::VM_OFF + swz(tok4(t, k), g >> 1) + 8 * (g & 1);
        ve_off[k] = G_::VE_OFF + tok4(t, k) * ROW_E + (16 * g) / N;
    }
    // softmax weights travel from the lanes that computed them (token = lane / 4 and + 8, column pair = lane % 4)
    const int src_lo = 4 * tok4(t, 0) + (g >> 1), src_hi = 4 * tok4(t, 1) + (g >> 1);
    const uint32_t half_sel = (g & 1) ? 0x7632u : 0x5410u;     // odd columns carry the lo halves

    int stage = 0;
    uint32_t parity = 0;
    bool timed_out = false;

    for (int c_next = i0; c_next < i1 && !timed_out;) {
        const Run cr = get_run(c_next);
        c_next += cr.n_items;
        if (cr.n_tok == 0) continue;

        // ---- run set-up: exponent references, query fragments, score factors ------------------
        uint2 qf[NT][8];                  // fp16 path: B fragments of the coefficients
        float kfac[NT];
        uint32_t qi8[NT][8];              // integer path: B fragments of the coefficient digits
        float qfac[NT][NBLK];             //   scale * log2(e) * 2^(qe - 14) per block
        int qbias[NT][NBLK];              //   offset contribution per block
        float qfac_h = 0.f;               // single-head path: factor and offsets of this lane's block (block t)
        int qbias_h = 0;
        {
            const uint4* src = reinterpret_cast<const uint4*>(a.qfrag);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                if (MHA) {
                    // B fragments: word 4 j + 2 kind + half covers bytes 16 (2j + half) + 4t .. + 3 (MMA j takes the 16-byte
                    // pieces 2j and 2j + 1 of a row); column g = (block g / 2, digit g % 2), zeros outside its block
                    int ch[8];
                    float qv[8];
                    query_channels(a, cr.hk, lane, ch);
                    query_values(a, (int64_t)cr.b * Hkv + cr.hk, true, ch, qv);
                    const QWord w = query_word<N>(a, qv);
#pragma unroll
                    for (int wd = 0; wd < 8; ++wd) {
                        const int j = wd >> 2, kind = (wd >> 1) & 1, half = wd & 1;
                        const int src_lane = 4 * (2 * j + half) + t;
                        const uint32_t d1 = __shfl_sync(0xffffffffu, kind ? w.b_d1 : w.a_d1, src_lane);
                        const uint32_t d0 = __shfl_sync(0xffffffffu, kind ? w.b_d0 : w.a_d0, src_lane);
                        const bool mine = (16 * (2 * j + half)) / (N / 2) == (g >> 1);
                        qi8[0][wd] = mine ? ((g & 1) ? d0 : d1) : 0u;
                    }
                    // this lane's block is block t (blocks that do not exist: factor 0, offsets 0)
                    const int lead = (t < NBLK ? t : 0) * (N / 8);
                    const float fac = __shfl_sync(0xffffffffu, w.fac, lead);
                    const int bias = __shfl_sync(0xffffffffu, w.bias, lead);
                    qfac_h = t < NBLK ? fac : 0.f;
                    qbias_h = t < NBLK ? bias : 0;
                } else if (KI) {
                    // several query heads: fragments and per-block factors come from make_qfrag4i (forming them here, at the
                    // start of a run, cost this kernel 8 % on long sequences: four heads' worth of dependent loads
                    // before the first tile can be used)
                    const uint4* s8 = src + (((int64_t)cr.b * Hkv + cr.hk) * NT + nt) * (2 * 32);
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const uint4 v = __ldg(s8 + j * 32 + lane);
                        qi8[nt][4 * j] = v.x; qi8[nt][4 * j + 1] = v.y; qi8[nt][4 * j + 2] = v.z; qi8[nt][4 * j + 3] = v.w;
                    }
                    const int qn = 4 * nt + t;
                    const int32_t* meta = qmeta + ((int64_t)cr.b * a.n_q_heads + cr.hk * Gq + (qn < Gq ? qn : 0)) * 8;
#pragma unroll
                    for (int k = 0; k < NBLK; ++k) {
                        qfac[nt][k] = __int_as_float(meta[2 * k]);
                        qbias[nt][k] = meta[2 * k + 1];
                    }
                } else {
                    const int qn = 4 * nt + t;
                    const int32_t* meta = qmeta + ((int64_t)cr.b * a.n_q_heads + cr.hk * Gq + (qn < Gq ? qn : 0)) * 8;
                    const uint4* s16 = src + (((int64_t)cr.b * Hkv + cr.hk) * NT + nt) * (4 * 32);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint4 v = __ldg(s16 + j * 32 + lane);
                        qf[nt][2 * j] = make_uint2(v.x, v.y);
                        qf[nt][2 * j + 1] = make_uint2(v.z, v.w);
                    }
                    kfac[nt] = (float)(qn < Gq ? meta[0] : 0);      // the query's exponent; completed below
                }
            }
        }
        // (after the fragment loads were issued, so that the two latencies overlap)
        const int dk = KI ? 0 : warp_max_byte(a.k_exp + cr.row0 * ROW_E, cr.n_tok * ROW_E, lane);
        const uint2* lutk = lut + (255 - dk);
        // The V side finds its reference exponent on the way: every tile is checked against the current one
        // before it is used, and the reference is raised (the accumulators scaled down by the exact power of
        // two) when a tile holds a larger exponent byte.  The first tile of a run always raises it.
        int dv = 0;
        uint32_t dv_probe = 0x7FFF7FFFu;          // (0x7FFF - dv) in both halves: adding a byte > dv sets bit 15
        const uint2* lutv = lut + 255;
        // single-head path: exponent byte e gives the fp32 weight 2^(e - dv + kTopShiftH) = bits (e + wexp) << 23;
        // wsum collects this lane's weights (tokens g, g + 8 of every row tile, block t) since the last removal of
        // the excess-code offsets from the sums
        int wexp = 127 + kTopShiftH;
        float wsum = 0.f;
        int since_flush = 0;
        if (!KI) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) kfac[nt] = pow2_split(a.scale_log2e, dk - 129 - kTopShift + (int)kfac[nt]);
        }
        float o[NT][8][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int r = 0; r < 8; ++r)
#pragma unroll
                for (int k = 0; k < 4; ++k) o[nt][r][k] = 0.f;
        float m_run[NT], l_run[NT];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) { m_run[nt] = -INFINITY; l_run[nt] = 0.f; }

        constexpr int VE_WORDS = kTile * ROW_E / 4;      // V exponent bytes of a stage, in words
        // slow path of the check: largest V exponent byte among the tile's live rows; raise the reference to it
        // (plus some headroom, so that small upward steps do not come back here)
        auto raise_dv = [&](const uint8_t* se, int n_live) {
            const int n_bytes = min(n_live, kTile) * ROW_E;
            uint32_t m = 0;
            for (int w = lane; w < VE_WORDS; w += 32) {
                uint32_t x = *reinterpret_cast<const uint32_t*>(se + G_::VE_OFF + 4 * w);
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
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int r = 0; r < 8; ++r)
#pragma unroll
                        for (int k = 0; k < 4; ++k) o[nt][r][k] *= f;
                dv = nd;
                dv_probe = (0x7FFFu - (uint32_t)nd) * 0x00010001u;
                lutv = lut + (255 - nd);
                wexp = 127 + kTopShiftH - nd;
                wsum *= f;
            }
        };
        // single-head path: the V bytes enter the MMAs as they are stored, so row "whole byte" carries 136 and row
        // "low nibble" 8 per unit of weight too much; taken out of the hi-half column of the sums every few stages,
        // while they are still small next to what they are taken from
        auto flush_offsets = [&]() {
            float w = wsum;
            w += __shfl_xor_sync(0xffffffffu, w, 4);
            w += __shfl_xor_sync(0xffffffffu, w, 8);
            w += __shfl_xor_sync(0xffffffffu, w, 16);
            const float c1 = w * (-136.f * 5.9604644775390625e-8f), c2 = w * (-8.f * 5.9604644775390625e-8f);   // 2^-24: the bytes are fp16 subnormals
#pragma unroll
            for (int r = 0; r < 8; ++r) { o[0][r][0] += c1; o[0][r][2] += c2; }
            wsum = 0.f;
            since_flush = 0;
        };

        // one stage of kTile tokens; FULL = every row of the tile exists
        auto tile_body = [&](const uint8_t* st, const uint8_t* se, int n_live, auto full_tag) {
            constexpr bool FULL = decltype(full_tag)::value;
            // ---- V exponent bytes against the reference: even and odd bytes in 16-bit lanes, bit 15 = "larger"
            if (FULL) {
                uint32_t f = 0;
#pragma unroll
                for (int i = 0; i < (VE_WORDS + 31) / 32; ++i) {
                    const int w = lane + 32 * i;
                    if (VE_WORDS % 32 == 0 || w < VE_WORDS) {
                        const uint32_t x = *reinterpret_cast<const uint32_t*>(se + G_::VE_OFF + 4 * w);
                        f |= ((x & 0x00FF00FFu) + dv_probe) | (prmt(x, 0u, 0x4341u) + dv_probe);
                    }
                }
                if (__any_sync(0xffffffffu, (f & 0x80008000u) != 0u)) raise_dv(se, n_live);
            } else {
                raise_dv(se, n_live);         // rows past the end may hold anything: masked there
            }
            // ---- scores ---------------------------------------------------------
            float sc[kMT][NT][2];
#pragma unroll
            for (int mt = 0; mt < kMT; ++mt) {
                if (!FULL && mt * 16 >= n_live) {
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) sc[mt][nt][0] = sc[mt][nt][1] = -INFINITY;
                    continue;
                }
                if (MHA) {
                    // ---- single head: each MMA takes two 16-byte pieces of the token rows (lane t: bytes 4t..4t+3 of each);
                    // the columns keep the blocks apart, so all four MMAs go to one accumulator set
                    const uint32_t ka = smem_u32(st) + lm_off + mt * 16 * ROW_M;
                    uint32_t u[4], v[4];          // tokens g, g + 8 of pieces 0, 1 (u) and 2, 3 (v): bytes 4t..4t+3 of each
                    ldmatrix_x4(u[0], u[1], u[2], u[3], ka);
                    ldmatrix_x4(v[0], v[1], v[2], v[3], ka ^ 32u);
                    int acc[4];
                    mma_u8s8_k32_first(acc, u[0], u[1], u[2], u[3], qi8[0][0], qi8[0][1], 0, 0);
                    mma_u8s8_k32(acc, v[0], v[1], v[2], v[3], qi8[0][4], qi8[0][5]);
                    mma_u8s8_k32(acc, u[0] << 4, u[1] << 4, u[2] << 4, u[3] << 4, qi8[0][2], qi8[0][3]);
                    mma_u8s8_k32(acc, v[0] << 4, v[1] << 4, v[2] << 4, v[3] << 4, qi8[0][6], qi8[0][7]);
                    // (256 * hi-digit sum + lo-digit sum) * 2^(e_k - 127) * (scale * 2^(qe - 16)) for block t, then the
                    // four blocks of a token are added across the lanes t (an exponent byte of 0 counts as weight 0)
                    constexpr int tb_mask = NBLK - 1;
                    const uint32_t e0 = se[G_::KE_OFF + (mt * 16 + g) * ROW_E + (t & tb_mask)];
                    const uint32_t e1 = se[G_::KE_OFF + (mt * 16 + g + 8) * ROW_E + (t & tb_mask)];
                    float s0 = __int2float_rn(256 * acc[0] + (acc[1] - qbias_h)) * (__uint_as_float(e0 << 23) * qfac_h);
                    float s1 = __int2float_rn(256 * acc[2] + (acc[3] - qbias_h)) * (__uint_as_float(e1 << 23) * qfac_h);
                    s0 += __shfl_xor_sync(0xffffffffu, s0, 1);
                    s1 += __shfl_xor_sync(0xffffffffu, s1, 1);
                    s0 += __shfl_xor_sync(0xffffffffu, s0, 2);
                    s1 += __shfl_xor_sync(0xffffffffu, s1, 2);
                    sc[mt][0][0] = s0; sc[mt][0][1] = s1;
                } else if (KI) {
                    // ---- integer path, several query heads: per 16-byte segment one 32-byte-deep MMA takes the bytes
                    // as they are (k 0..15) and the words shifted left by four bits (k 16..31; see make_qfrag4i)
                    int acc[NT][NBLK][4];
                    const uint32_t ka = smem_u32(st) + lm_off + mt * 16 * ROW_M;
                    constexpr int SEG_PER_BLK = 4 / NBLK;
#pragma unroll
                    for (int seg = 0; seg < 4; ++seg) {
                        const int blk = seg / SEG_PER_BLK;
                        uint32_t wa, wb;          // bytes 16 seg + 4t .. + 3 of tokens g and g + 8
                        ldmatrix_x2(wa, wb, ka ^ (uint32_t)(seg << 4));
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            if (seg % SEG_PER_BLK == 0)   // first MMA of a block starts from zero
                                mma_u8s8_k32_first(acc[nt][blk], wa, wb, wa << 4, wb << 4, qi8[nt][2 * seg], qi8[nt][2 * seg + 1],
                                                   0, 0);
                            else
                                mma_u8s8_k32(acc[nt][blk], wa, wb, wa << 4, wb << 4, qi8[nt][2 * seg], qi8[nt][2 * seg + 1]);
                        }
                    }
                    // (256 * hi-digit sum + lo-digit sum) * 2^(e_k - 127) * (scale * 2^(qe - 16)), per block (an exponent
                    // byte of 0 counts as weight 0)
                    uint32_t ew0, ew1;            // the exponent bytes of tokens g and g + 8
                    if (ROW_E == 4) {
                        ew0 = *reinterpret_cast<const uint32_t*>(se + kei_off + mt * 16 * ROW_E);
                        ew1 = *reinterpret_cast<const uint32_t*>(se + kei_off + (mt * 16 + 8) * ROW_E);
                    } else if (ROW_E == 2) {
                        ew0 = *reinterpret_cast<const uint16_t*>(se + kei_off + mt * 16 * ROW_E);
                        ew1 = *reinterpret_cast<const uint16_t*>(se + kei_off + (mt * 16 + 8) * ROW_E);
                    } else {
                        ew0 = se[kei_off + mt * 16 * ROW_E];
                        ew1 = se[kei_off + (mt * 16 + 8) * ROW_E];
                    }
                    float s0[NT], s1[NT];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) s0[nt] = s1[nt] = 0.f;
#pragma unroll
                    for (int k = 0; k < NBLK; ++k) {
                        const float w0 = __uint_as_float(((ew0 >> (8 * k)) & 0xffu) << 23);
                        const float w1 = __uint_as_float(((ew1 >> (8 * k)) & 0xffu) << 23);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            // (the offsets' constant contribution is taken out here: as the accumulator's start value
                            // it would tie up four registers per block for the whole loop)
                            const float f0 = __int2float_rn(256 * acc[nt][k][0] + (acc[nt][k][1] - qbias[nt][k]));
                            const float f1 = __int2float_rn(256 * acc[nt][k][2] + (acc[nt][k][3] - qbias[nt][k]));
                            s0[nt] = fmaf(f0, w0 * qfac[nt][k], s0[nt]);
                            s1[nt] = fmaf(f1, w1 * qfac[nt][k], s1[nt]);
                        }
                    }
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) { sc[mt][nt][0] = s0[nt]; sc[mt][nt][1] = s1[nt]; }
                } else {
                    const uint4 xa = *reinterpret_cast<const uint4*>(st + k_off + mt * 16 * ROW_M);
                    const uint4 xb = *reinterpret_cast<const uint4*>(st + k_off8 + mt * 16 * ROW_M);
                    const uint32_t wa[4] = {xa.x, xa.y, xa.z, xa.w}, wb[4] = {xb.x, xb.y, xb.z, xb.w};
                    uint2 la[NBK], lb[NBK];
    #pragma unroll
                    for (int k = 0; k < NBK; ++k) {
                        la[k] = lutk[se[ke_off + mt * 16 * ROW_E + k]];
                        lb[k] = lutk[se[ke_off + (mt * 16 + 8) * ROW_E + k]];
                    }
                    float acc[NT][2][4];
    #pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int kb = (NBK == 2) ? (i >> 1) : 0;
                        // bytes 4i..4i+3 of the lane chunk: kind 1 by byte permute, kind 2 by one logic op
                        const uint32_t a1_01 = prmt(wa[i], kMagic, 0x4140u), a1_23 = prmt(wa[i], kMagic, 0x4342u);
                        const uint32_t b1_01 = prmt(wb[i], kMagic, 0x4140u), b1_23 = prmt(wb[i], kMagic, 0x4342u);
                        const uint32_t a2_01 = lop3<0x6A>(a1_01, 0xFF0FFF0Fu, 0x00800080u), a2_23 = lop3<0x6A>(a1_23, 0xFF0FFF0Fu, 0x00800080u);
                        const uint32_t b2_01 = lop3<0x6A>(b1_01, 0xFF0FFF0Fu, 0x00800080u), b2_23 = lop3<0x6A>(b1_23, 0xFF0FFF0Fu, 0x00800080u);
                        const uint32_t A0 = fma_f16x2(a1_01, la[kb].x, la[kb].y), A1 = fma_f16x2(b1_01, lb[kb].x, lb[kb].y);
                        const uint32_t A2 = fma_f16x2(a2_01, la[kb].x, la[kb].y), A3 = fma_f16x2(b2_01, lb[kb].x, lb[kb].y);
                        const uint32_t B0 = fma_f16x2(a1_23, la[kb].x, la[kb].y), B1 = fma_f16x2(b1_23, lb[kb].x, lb[kb].y);
                        const uint32_t B2 = fma_f16x2(a2_23, la[kb].x, la[kb].y), B3 = fma_f16x2(b2_23, lb[kb].x, lb[kb].y);
    #pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            const uint2 q0 = qf[nt][2 * i], q1 = qf[nt][2 * i + 1];
                            if (i == 0) {
                                mma_f16_first(acc[nt][0], A0, A1, A2, A3, q0.x, q0.y);
                                mma_f16_first(acc[nt][1], B0, B1, B2, B3, q1.x, q1.y);
                            } else {
                                mma_f16(acc[nt][0], A0, A1, A2, A3, q0.x, q0.y);
                                mma_f16(acc[nt][1], B0, B1, B2, B3, q1.x, q1.y);
                            }
                        }
                    }
    #pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        sc[mt][nt][0] = ((acc[nt][0][0] + acc[nt][0][1]) + (acc[nt][1][0] + acc[nt][1][1])) * kfac[nt];
                        sc[mt][nt][1] = ((acc[nt][0][2] + acc[nt][0][3]) + (acc[nt][1][2] + acc[nt][1][3])) * kfac[nt];
                    }
                }
                if (!FULL) {       // select, not arithmetic: rows past the end may hold anything
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        if (mt * 16 + g >= n_live) sc[mt][nt][0] = -INFINITY;
                        if (mt * 16 + g + 8 >= n_live) sc[mt][nt][1] = -INFINITY;
                    }
                }
            }

            // ---- running softmax (reference point moves only in big steps) ------
            bool grow = false;
            float tmax[NT];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                float mx = -INFINITY;
#pragma unroll
                for (int mt = 0; mt < kMT; ++mt) mx = fmaxf(mx, fmaxf(sc[mt][nt][0], sc[mt][nt][1]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                tmax[nt] = mx;
                grow |= mx > m_run[nt] + 8.f;
            }
            if (__any_sync(0xffffffffu, grow)) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const float m_new = fmaxf(m_run[nt], tmax[nt]);
                    const float alpha = (m_run[nt] == -INFINITY) ? 0.f : ex2_approx(m_run[nt] - m_new);
                    m_run[nt] = m_new;
                    l_run[nt] *= alpha;
                    if (MHA) wsum *= alpha;
#pragma unroll
                    for (int r = 0; r < 8; ++r)
#pragma unroll
                        for (int k = 0; k < 4; ++k) o[nt][r][k] *= alpha;
                }
            }

            // ---- P.V ------------------------------------------------------------
#pragma unroll
            for (int mt = 0; mt < kMT; ++mt) {
                if (!FULL && mt * 16 >= n_live) continue;
                if (MHA) {
                    // ---- single head: the weight of (token, block t) = softmax weight x 2^(e_v - dv + kTopShiftH) is
                    // formed here, in fp32, and travels as (hi, lo) fp16 halves in column (block, half); the V bytes
                    // need no arithmetic at all: a byte under a zero exponent field is the fp16 subnormal byte * 2^-24
                    constexpr int tb_mask = NBLK - 1;
                    const float p0 = ex2_approx(sc[mt][0][0] - m_run[0]);
                    const float p1 = ex2_approx(sc[mt][0][1] - m_run[0]);
                    l_run[0] += p0 + p1;
                    const int ev0 = se[G_::VE_OFF + (mt * 16 + g) * ROW_E + (t & tb_mask)];
                    const int ev1 = se[G_::VE_OFF + (mt * 16 + g + 8) * ROW_E + (t & tb_mask)];
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
                    // B fragment for lane (g, t): column g = (block g/2, half g%2); tokens tok4(t, 0), tok4(t, 1) | tok4(t, 2), tok4(t, 3)
                    const uint32_t v0 = __shfl_sync(0xffffffffu, q0, src_lo);
                    const uint32_t v1 = __shfl_sync(0xffffffffu, q0, src_hi);
                    const uint32_t v2 = __shfl_sync(0xffffffffu, q1, src_lo);
                    const uint32_t v3 = __shfl_sync(0xffffffffu, q1, src_hi);
                    const uint32_t pb0 = prmt(v0, v1, half_sel), pb1 = prmt(v2, v3, half_sel);
                    uint2 vw[4];
#pragma unroll
                    for (int k = 0; k < 4; ++k) vw[k] = *reinterpret_cast<const uint2*>(st + v_off[k] + mt * 16 * ROW_M);
#pragma unroll
                    for (int x = 0; x < 4; ++x) {         // byte pair (2x, 2x+1) of the lane's eight bytes
                        const uint32_t wA0 = (x < 2) ? vw[0].x : vw[0].y, wA1 = (x < 2) ? vw[1].x : vw[1].y;
                        const uint32_t wB0 = (x < 2) ? vw[2].x : vw[2].y, wB1 = (x < 2) ? vw[3].x : vw[3].y;
                        const uint32_t sel = (x & 1) ? 0x7632u : 0x5410u;
                        const uint32_t XA = prmt(wA0, wA1, sel), XB = prmt(wB0, wB1, sel);     // [tok.b, tok.b', tok'.b, tok'.b']
                        const uint32_t a1e = XA & 0x00FF00FFu, a1o = prmt(XA, 0u, 0x4341u);
                        const uint32_t b1e = XB & 0x00FF00FFu, b1o = prmt(XB, 0u, 0x4341u);
                        mma_f16(o[0][2 * x], a1e, XA & 0x000F000Fu, b1e, XB & 0x000F000Fu, pb0, pb1);
                        mma_f16(o[0][2 * x + 1], a1o, a1o & 0x000F000Fu, b1o, b1o & 0x000F000Fu, pb0, pb1);
                    }
                    continue;
                }
                // softmax weights of this lane's tokens (g and g+8), then the B fragment of P^T for lane (g, t):
                // column g = (query g/2, half g%2); tokens tok4(t, 0), tok4(t, 1) | tok4(t, 2), tok4(t, 3)
                uint32_t pb[NT][2];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const float p0 = ex2_approx(sc[mt][nt][0] - m_run[nt]);
                    const float p1 = ex2_approx(sc[mt][nt][1] - m_run[nt]);
                    l_run[nt] += p0 + p1;
                    // (hi, lo) fp16 halves of each weight, packed in one register before they travel: hi = the
                    // value cut to 11 significant bits (exact in fp16), lo = the rest
                    const float h0 = __uint_as_float(__float_as_uint(p0) & 0xffffe000u);
                    const float h1 = __uint_as_float(__float_as_uint(p1) & 0xffffe000u);
                    const uint32_t w0 = pack_f16x2_rn(h0, p0 - h0), w1 = pack_f16x2_rn(h1, p1 - h1);
                    const uint32_t v0 = __shfl_sync(0xffffffffu, w0, src_lo);   // token tok4(t, 0)
                    const uint32_t v1 = __shfl_sync(0xffffffffu, w0, src_hi);   // token tok4(t, 1)
                    const uint32_t v2 = __shfl_sync(0xffffffffu, w1, src_lo);   // token tok4(t, 2) = tok4(t, 0) + 8
                    const uint32_t v3 = __shfl_sync(0xffffffffu, w1, src_hi);   // token tok4(t, 3) = tok4(t, 1) + 8
                    pb[nt][0] = prmt(v0, v1, half_sel);      // this column's half of the first token pair
                    pb[nt][1] = prmt(v2, v3, half_sel);      // and of the second
                }
                // V pieces: bytes [8g, 8g+8) (slots 16g..16g+15) of tokens tok4(t, 0..3) of this row tile
                uint2 vw[4];
                uint2 lv[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    vw[k] = *reinterpret_cast<const uint2*>(st + v_off[k] + mt * 16 * ROW_M);
                    lv[k] = lutv[se[ve_off[k] + mt * 16 * ROW_E]];
                }
                if (!FULL) {       // rows past the end contribute exactly zero
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (mt * 16 + tok4(t, k) >= n_live) lv[k] = make_uint2(0u, 0u);
                }
                const uint32_t sA = prmt(lv[0].x, lv[1].x, 0x7610u), cA = prmt(lv[0].y, lv[1].y, 0x7610u);
                const uint32_t sB = prmt(lv[2].x, lv[3].x, 0x7610u), cB = prmt(lv[2].y, lv[3].y, 0x7610u);
#pragma unroll
                for (int x = 0; x < 4; ++x) {         // byte pair (2x, 2x+1) of the lane's eight bytes
                    const uint32_t wA0 = (x < 2) ? vw[0].x : vw[0].y, wA1 = (x < 2) ? vw[1].x : vw[1].y;
                    const uint32_t wB0 = (x < 2) ? vw[2].x : vw[2].y, wB1 = (x < 2) ? vw[3].x : vw[3].y;
                    const uint32_t sel = (x & 1) ? 0x7632u : 0x5410u;
                    const uint32_t XA = prmt(wA0, wA1, sel), XB = prmt(wB0, wB1, sel);     // [tok.b, tok.b', tok'.b, tok'.b']
                    // kind 1 for the even byte by mask-or, for the odd byte by byte permute; kind 2 from kind 1
                    const uint32_t a1e = lop3<0xEA>(XA, 0x00FF00FFu, 0x64006400u), a1o = prmt(XA, kMagic, 0x4341u);
                    const uint32_t b1e = lop3<0xEA>(XB, 0x00FF00FFu, 0x64006400u), b1o = prmt(XB, kMagic, 0x4341u);
                    const uint32_t a2e = lop3<0x6A>(a1e, 0xFF0FFF0Fu, 0x00800080u), a2o = lop3<0x6A>(a1o, 0xFF0FFF0Fu, 0x00800080u);
                    const uint32_t b2e = lop3<0x6A>(b1e, 0xFF0FFF0Fu, 0x00800080u), b2o = lop3<0x6A>(b1o, 0xFF0FFF0Fu, 0x00800080u);
                    const uint32_t E0 = fma_f16x2(a1e, sA, cA), E1 = fma_f16x2(a2e, sA, cA);
                    const uint32_t E2 = fma_f16x2(b1e, sB, cB), E3 = fma_f16x2(b2e, sB, cB);
                    const uint32_t O0 = fma_f16x2(a1o, sA, cA), O1 = fma_f16x2(a2o, sA, cA);
                    const uint32_t O2 = fma_f16x2(b1o, sB, cB), O3 = fma_f16x2(b2o, sB, cB);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        mma_f16(o[nt][2 * x], E0, E1, E2, E3, pb[nt][0], pb[nt][1]);
                        mma_f16(o[nt][2 * x + 1], O0, O1, O2, O3, pb[nt][0], pb[nt][1]);
                    }
                }
            }
        };

        for (int it = 0; it < cr.n_tiles; ++it) {
            if (!mbar_wait_bounded(bar0 + 8 * stage, parity)) { timed_out = true; break; }
            const uint8_t* st = wsm + stage * G_::MANT_STAGE;
            const uint8_t* se = wse + stage * G_::EXP_STAGE;
            const int n_live = cr.n_tok - it * kTile;        // tokens of this tile that exist (may exceed kTile)
            if (n_live >= kTile) tile_body(st, se, n_live, std::true_type{});
            else tile_body(st, se, n_live, std::false_type{});
            if (MHA && ++since_flush == kFlushStages) flush_offsets();
            __syncwarp();
            issue_next(stage);
            if (++stage == kStages) { stage = 0; parity ^= 1u; }
        }
        if (timed_out) break;

        // ---- partial result of the run, at the slot of its first chunk ----------------------------
        // row of kind 1 = 16*o_hi + o_lo, row of kind 2 = o_lo; common factor 2^(dv - 129 - kTopShift)
        if (MHA) {
            // lane (g, t) holds, for the bytes 8g..8g+7 of the row, the sums weighted for block t: the lanes whose t
            // is the block of those bytes write them out.  2^24 undoes the subnormal scaling of the bytes.
            flush_offsets();
            const float vfac = pow2_split(1.f, dv - 129 - kTopShiftH);      // (2^24 apart: their product can leave the fp32 range)
            const float vfac16 = vfac * 0.0625f;
            float l = l_run[0];
            l += __shfl_xor_sync(0xffffffffu, l, 4);
            l += __shfl_xor_sync(0xffffffffu, l, 8);
            l += __shfl_xor_sync(0xffffffffu, l, 16);
            if (t == (16 * g) / N) {
                float* dst = a.partials + (((int64_t)cr.b * a.n_q_heads + cr.hk) * a.n_chunks + partial_slot(cr.chunk0, a.item_tokens, a.chunk, a.n_chunks)) * kPartStride;
#pragma unroll
                for (int r4 = 0; r4 < 4; ++r4) {
                    const float w0 = (o[0][2 * r4][0] + o[0][2 * r4][1]) * 16777216.f, l0 = (o[0][2 * r4][2] + o[0][2 * r4][3]) * 16777216.f;
                    const float w1 = (o[0][2 * r4 + 1][0] + o[0][2 * r4 + 1][1]) * 16777216.f, l1 = (o[0][2 * r4 + 1][2] + o[0][2 * r4 + 1][3]) * 16777216.f;
                    float4 v;
                    v.x = l0 * vfac;            // slot 16g + 4r4     (low nibble of byte 2r4)
                    v.y = (w0 - l0) * vfac16;   // slot 16g + 4r4 + 1 (high nibble of byte 2r4)
                    v.z = l1 * vfac;
                    v.w = (w1 - l1) * vfac16;
                    reinterpret_cast<float4*>(dst + 16 * g)[r4] = v;
                }
                if (g == 0) { dst[D] = m_run[0]; dst[D + 1] = l; }
            }
        } else {
        const float vfac = pow2_split(1.f, dv - 129 - kTopShift);
        const float vfac16 = vfac * 0.0625f;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            float l = l_run[nt];
            l += __shfl_xor_sync(0xffffffffu, l, 4);
            l += __shfl_xor_sync(0xffffffffu, l, 8);
            l += __shfl_xor_sync(0xffffffffu, l, 16);
            const int qi = 4 * nt + t;
            if (qi < Gq) {
                float* dst = a.partials + (((int64_t)cr.b * a.n_q_heads + cr.hk * Gq + qi) * a.n_chunks + partial_slot(cr.chunk0, a.item_tokens, a.chunk, a.n_chunks)) * kPartStride;
#pragma unroll
                for (int r4 = 0; r4 < 4; ++r4) {
                    const float w0 = o[nt][2 * r4][0] + o[nt][2 * r4][1], l0 = o[nt][2 * r4][2] + o[nt][2 * r4][3];
                    const float w1 = o[nt][2 * r4 + 1][0] + o[nt][2 * r4 + 1][1], l1 = o[nt][2 * r4 + 1][2] + o[nt][2 * r4 + 1][3];
                    float4 v;
                    v.x = l0 * vfac;            // slot 16g + 4r4     (low nibble of byte 2r4)
                    v.y = (w0 - l0) * vfac16;   // slot 16g + 4r4 + 1 (high nibble of byte 2r4)
                    v.z = l1 * vfac;
                    v.w = (w1 - l1) * vfac16;
                    reinterpret_cast<float4*>(dst + 16 * g)[r4] = v;
                }
                if (g == 0) { dst[D] = m_run[nt]; dst[D + 1] = l; }
            }
        }
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

template <int N, int NT, bool MHA>
kvbfp_status launch3(const DecodeArgs& a, cudaStream_t s, Split* split) {
    using G_ = Geo4<N>;
    static std::atomic<int> resident[64];   // thread blocks that fit the whole device, per device (0 = not asked yet;
                                            // two host threads asking at once store the same number)
    int dev = 0;
    KVBFP_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return KVBFP_ERR_UNSUPPORTED;
    if (!resident[dev].load(std::memory_order_acquire)) {
        KVBFP_CUDA(cudaFuncSetAttribute(decode_mma4<N, NT, MHA>, cudaFuncAttributeMaxDynamicSharedMemorySize, G_::SMEM_BYTES));
        int per_sm = 0, n_sm = 0;
        KVBFP_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_mma4<N, NT, MHA>, kWarps * 32, G_::SMEM_BYTES));
        KVBFP_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
        if (per_sm < 1 || n_sm < 1) return KVBFP_ERR_CUDA;
        resident[dev].store(per_sm * n_sm, std::memory_order_release);
    }
    // per-query exponents and biases (8 words each) sit behind the fragments in the query region of the workspace
    int32_t* qmeta = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(a.qfrag) +
                                               (size_t)a.fmt.batch * a.fmt.n_kv_heads * NT * 8 * 32 * 2 * sizeof(uint32_t));
    const int n_pre = a.fmt.batch * a.fmt.n_kv_heads * NT;
    if (N < 32) {
        (void)launch_pdl(make_qfrag4, dim3(n_pre), dim3(32), 0, s, a, NT, qmeta);
        KVBFP_LAUNCH_CHECK("make_qfrag4");
    } else if (!MHA) {    // (with one query head per kv head the main kernel forms the query coefficients itself)
        (void)launch_pdl(make_qfrag4i<(N >= 32 ? N : 32)>, dim3((n_pre + 3) / 4), dim3(128), 0, s, a, NT, qmeta);
        KVBFP_LAUNCH_CHECK("make_qfrag4i");
    }
    DecodeArgs b;
    int grid = 0;
    const kvbfp_status st = plan_persistent(a, kItemTokens, resident[dev].load(std::memory_order_relaxed), kWarps, &b, split, &grid);
    if (st != KVBFP_OK) return st;
    // tensor maps of the two mantissa planes (this device's memory; rows of two tokens, boxes of kTile tokens)
    // (a decode loop passes the same planes step after step: the last pair of maps is kept per host thread)
    struct MapCache { const void *k = nullptr, *v = nullptr; uint64_t rows = 0; int dev = -1; CUtensorMap k_map, v_map; };
    static thread_local MapCache mc;
    const uint64_t n_rows = (uint64_t)a.fmt.batch * a.fmt.n_kv_heads * a.fmt.max_seq;
    if (mc.k != a.k_mant || mc.v != a.v_mant || mc.rows != n_rows || mc.dev != dev) {
        mc.k = nullptr;
        kvbfp_status ms = make_row_map(&mc.k_map, a.k_mant, n_rows / 2, 2 * ROW_M, kTile / 2);
        if (ms == KVBFP_OK) ms = make_row_map(&mc.v_map, a.v_mant, n_rows / 2, 2 * ROW_M, kTile / 2);
        if (ms != KVBFP_OK) return ms;
        mc.k = a.k_mant; mc.v = a.v_mant; mc.rows = n_rows; mc.dev = dev;
    }
    const CUtensorMap& k_map = mc.k_map;
    const CUtensorMap& v_map = mc.v_map;
    cudaEvent_t ev0, ev1;
    profile_events(&ev0, &ev1);
    if (ev0) KVBFP_CUDA(cudaEventRecord(ev0, s));
    (void)launch_pdl(decode_mma4<N, NT, MHA>, dim3(grid), dim3(kWarps * 32), G_::SMEM_BYTES, s, b, (const int32_t*)qmeta, k_map, v_map);
    KVBFP_LAUNCH_CHECK("decode_mma4");
    if (ev1) KVBFP_CUDA(cudaEventRecord(ev1, s));
    return KVBFP_OK;
}

template <int N>
kvbfp_status launch2(const DecodeArgs& a, cudaStream_t s, Split* split) {
    const int G = a.n_q_heads / a.fmt.n_kv_heads;
    if (N >= 32 && G == 1) return launch3<N, 1, (N >= 32)>(a, s, split);
    return (G <= 4) ? launch3<N, 1, false>(a, s, split) : launch3<N, 2, false>(a, s, split);
}

}  // namespace

kvbfp_status launch_decode_mma4(const DecodeArgs& a, cudaStream_t s, Split* split) {
    switch (a.fmt.block) {
        case 16: return launch2<16>(a, s, split);
        case 32: return launch2<32>(a, s, split);
        case 64: return launch2<64>(a, s, split);
        case 128: return launch2<128>(a, s, split);
    }
    return KVBFP_ERR_UNSUPPORTED;
}

}  // namespace kvbfp
