// Decode attention over the packed BFP cache with warp-level bf16 tensor-core MMAs
// (Sec. III par. 2 of the paper: keys are read back from the cache and multiplied with pi(q);
// Sec. II-B: a block's values are integer mantissas times one power of two).
//
// Work split.  One warp owns one (batch, kv head, chunk of the sequence) item and all query heads
// that share the kv head, so K and V are read from HBM once per group.  Each warp runs its own
// ring of shared-memory stages filled by 1-D bulk asynchronous copies (one elected lane issues
// them, an mbarrier per stage counts the bytes); there is no block-wide barrier in the loop.
//
// Arithmetic.  A mantissa field is turned into a bf16 number without an integer-to-float
// conversion: the stored field (an unsigned offset, M + 2^(P-1)) is or-ed under the bits of
// 128.0, giving 128 + offset exactly; one bf16x2 fma with the block's power-of-two weight removes
// the bias and applies 2^e in the same instruction, exactly (the result M * 2^e has at most 7
// significant bits).  Scores:  S[16 tokens x 8 cols] += K[16 x 16 slots] . Q[16 slots x 8 cols],
// where the 8 columns are four query heads times (hi, lo) bf16 halves of q, so q keeps ~16 bits.
// Output: O^T[16 slots x 8 cols] += V^T[16 slots x 16 tokens] . P^T[16 tokens x 8 cols], with the
// softmax weights split into hi/lo halves the same way.  Accumulators are fp32.
//
// Range.  The bias product (136, 160 or 2304 units of the block's weight for 4-, 6- and 8-bit mantissas) is a bf16
// intermediate of about 2^5 times the block's largest value, so cache values of magnitude 2^120 and above are
// outside this kernel's range (they give infinities); the fp32 kernel and the 4- and 8-bit integer-score kernels
// have no such limit.
//
// The integer pipe (logic ops, shifts, byte permutes) is what limits this kernel: every field is
// extracted with one three-input logic instruction and block weights come from a 256-entry table in
// shared memory instead of being rebuilt from the exponent byte.
#include <math.h>

#include <atomic>

#include "decode.cuh"
#include "ptx.cuh"

namespace kvbfp {
namespace {

constexpr int kWarps = 4;
constexpr int kMT = 2;             // 16-token MMA row tiles per stage
constexpr int kStages = 3;         // shared-memory stages per warp
constexpr int kMinCtas = 1;        // resident thread blocks per SM the register allocation must allow
constexpr int kTile = 16 * kMT;        // tokens per stage

// bf16 bit pattern of 2^(e8 - 127 - (P-2)); subnormal results down to 2^-133 are exact.
template <int P>
__device__ __forceinline__ uint32_t weight_bf16(uint32_t e8) {
    const int f = (int)e8 - (P - 2);
    return f >= 1 ? ((uint32_t)f << 7) : (0x40u >> (-f));
}

// Format constants of the "or under 128.0" conversion.  The stored field is M + 2^(P-1) (P = 4, 6);
// the value built is 128 + 2^(P-1) + M, so the bias to remove is `bias`.
template <int P> struct Fmt;
template <> struct Fmt<4> { static constexpr uint32_t mask = 0x000F000Fu, magic = 0x43004300u, bias = 0xC308C308u; };  // -136
template <> struct Fmt<6> { static constexpr uint32_t mask = 0x003F003Fu, magic = 0x43004300u, bias = 0xC320C320u; };  // -160
template <> struct Fmt<8> { static constexpr uint32_t mask = 0x000F000Fu, magic = 0x43004300u, bias = 0xC510C510u; };  // -2304

// Per-row (or per token pair) weights ready for the conversion fma's.
struct Wgt {
    uint32_t s;     // (2^e, 2^e') as bf16x2
    uint32_t c;     // -bias * s
    uint32_t s16;   // 16 * s   (8-bit mantissas only)
};
template <int P>
__device__ __forceinline__ Wgt make_wgt(uint32_t s2, uint32_t c2) {
    Wgt w;
    w.s = s2;
    w.c = c2;
    w.s16 = (P == 8) ? mul_bf16x2(s2, 0x41804180u) : 0u;   // 16.0
    return w;
}

// x holds two fields at bits [0, P) and [16, 16+P) (P = 4, 6), or two bytes at bits [0,8) and [16,24) (P = 8).
template <int P>
__device__ __forceinline__ uint32_t cvt_pair(uint32_t x, const Wgt& w) {
    if (P == 8) {
        // byte = M + 128 = 16*H + L with both nibbles unsigned
        uint32_t lo = lop3<0xEA>(x, 0x000F000Fu, 0x43004300u);         // (x & m) | 128.0  = 128 + L
        uint32_t hi = lop3<0xEA>(x >> 4, 0x000F000Fu, 0x43004300u);    // (x & m) | 128.0  = 128 + H
        uint32_t v = fma_bf16x2(hi, w.s16, w.c);                       // (16H - 256) * 2^e, exact
        return fma_bf16x2(lo, w.s, v);                                 // (16H + L - 128) * 2^e = M * 2^e, exact
    }
    return fma_bf16x2(lop3<0xEA>(x, Fmt<P>::mask, Fmt<P>::magic), w.s, w.c);   // (x & mask) | 128.0 in one op
}

// Slot (within the 128-slot row) that the K-side unpack puts at k-position kk of k-step ks for lane
// column t; kk = 0..3 stands for k = 2t, 2t+1, 2t+8, 2t+9 of the m16n8k16 fragment.
template <int P>
__host__ __device__ __forceinline__ int k_slot(int ks, int t, int kk) {
    if (P == 4) return 32 * t + 8 * (ks >> 1) + 2 * (ks & 1) + (kk >> 1) + 4 * (kk & 1);
    if (P == 8) return 32 * t + 4 * ks + 2 * (kk & 1) + (kk >> 1);
    return 32 * t + 4 * ks + kk;
}

// Two A registers (k = 2t..2t+1 and k = 2t+8..2t+9) of k-steps ks and ks+1 (ks even) from a lane's
// 32-slot chunk w[P].
template <int P>
__device__ __forceinline__ void k_pairs2(const uint32_t (&w)[P], int ks, const Wgt& wg,
                                         uint32_t (&r)[4]) {
    if (P == 4) {
        uint32_t x4, x8, x12;
        x4 = w[ks >> 1] >> 4; x8 = w[ks >> 1] >> 8; x12 = w[ks >> 1] >> 12;
        r[0] = cvt_pair<4>(w[ks >> 1], wg);
        r[1] = cvt_pair<4>(x4, wg);
        r[2] = cvt_pair<4>(x8, wg);
        r[3] = cvt_pair<4>(x12, wg);
    } else if (P == 8) {
        r[0] = cvt_pair<8>(w[ks], wg);
        r[1] = cvt_pair<8>(w[ks] >> 8, wg);
        r[2] = cvt_pair<8>(w[ks + 1], wg);
        r[3] = cvt_pair<8>(w[ks + 1] >> 8, wg);
    } else {
        uint32_t f[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int bit = 6 * (4 * ks + j), word = bit >> 5, s = bit & 31;
            f[j] = (s + 6 > 32) ? __funnelshift_r(w[word], w[(word + 1) % P], s) : (w[word] >> s);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) r[j] = cvt_pair<6>(prmt(f[2 * j], f[2 * j + 1], 0x5410u), wg);
    }
}

// V side: registers for MMA row pairs r and r+1 (r even): (slot 2r, 2r+1, 2r+2, 2r+3) x (token pair),
// from the two tokens' 16-slot pieces wa, wb (P/2 words each).
template <int P>
__device__ __forceinline__ void v_pairs2(const uint32_t* wa, const uint32_t* wb, int r, const Wgt& wg,
                                         uint32_t (&o)[4]) {
    if (P == 4) {
        // word i = slots 8i..8i+7; halfword h of word i = slots 8i+4h..8i+4h+3 = rows 2r..2r+3 with r = 4i+2h
        const uint32_t x = prmt(wa[r >> 2], wb[r >> 2], ((r >> 1) & 1) ? 0x7632u : 0x5410u);
        uint32_t x4, x8, x12;
        x4 = x >> 4; x8 = x >> 8; x12 = x >> 12;
        o[0] = cvt_pair<4>(x, wg);
        o[1] = cvt_pair<4>(x4, wg);
        o[2] = cvt_pair<4>(x8, wg);
        o[3] = cvt_pair<4>(x12, wg);
    } else if (P == 8) {
        // word i = slots 4i..4i+3; slots 2r..2r+3 = word r>>1
        const uint32_t xl = prmt(wa[r >> 1], wb[r >> 1], 0x5410u), xh = prmt(wa[r >> 1], wb[r >> 1], 0x7632u);
        o[0] = cvt_pair<8>(xl, wg);
        o[1] = cvt_pair<8>(xl >> 8, wg);
        o[2] = cvt_pair<8>(xh, wg);
        o[3] = cvt_pair<8>(xh >> 8, wg);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int bit = 6 * (2 * r + j), word = bit >> 5, s = bit & 31;
            const uint32_t fa = (s + 6 > 32) ? __funnelshift_r(wa[word], wa[(word + 1) % 3], s) : (wa[word] >> s);
            const uint32_t fb = (s + 6 > 32) ? __funnelshift_r(wb[word], wb[(word + 1) % 3], s) : (wb[word] >> s);
            o[j] = cvt_pair<6>(prmt(fa, fb, 0x5410u), wg);
        }
    }
}

// ------------------------------------------------------------------ query fragments
// One warp per (batch, kv head, n-tile): writes the B fragments of pi(q) for the score MMAs,
// [item][j = 0..3][lane][4 words], word 4j+k = (k-step 2j + k/2, register k%2).
template <int P>
__global__ void __launch_bounds__(32) make_qfrag(DecodeArgs a, int NT) {
    constexpr int D = kHeadDim;
    const int N = a.fmt.block;
    const int lane = threadIdx.x, gp = lane >> 2, tp = lane & 3;
    const int item = blockIdx.x;
    const int nt = item % NT, g = (item / NT) % a.fmt.n_kv_heads, b = item / NT / a.fmt.n_kv_heads;
    const int G = a.n_q_heads / a.fmt.n_kv_heads;
    const int qi = 4 * nt + (gp >> 1), part = gp & 1;
    __shared__ float sq[4][D];       // pi(q) of the four query heads of this n-tile
    for (int i = lane; i < 4 * D; i += 32) {
        const int qq = 4 * nt + i / D, slot = i % D;
        float v = 0.f;
        if (qq < G) {
            const int ch = a.perm_k ? (a.perm_k[g * D + slot] & (D - 1)) : slot;
            const int64_t idx = ((int64_t)b * a.n_q_heads + g * G + qq) * D + ch;
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
    uint32_t* dst = a.qfrag + (int64_t)item * (8 * 32 * 2);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        uint32_t reg[2];
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) {
            uint32_t h[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const float v = sq[gp >> 1][k_slot<P>(ks, tp, 2 * rr + e)];
                __nv_bfloat16 hi = __float2bfloat16_rn(v);
                __nv_bfloat16 out = part ? __float2bfloat16_rn(v - __bfloat162float(hi)) : hi;
                if (qi >= G) out = __ushort_as_bfloat16(0);
                h[e] = __bfloat16_as_ushort(out);
            }
            reg[rr] = h[0] | (h[1] << 16);
        }
        const int wd = 2 * ks;                       // word index of reg[0]
        dst[((wd >> 2) * 32 + lane) * 4 + (wd & 3)] = reg[0];
        dst[((wd >> 2) * 32 + lane) * 4 + (wd & 3) + 1] = reg[1];
    }
}

// ------------------------------------------------------------------ main kernel
template <int P, int N>
struct Geo {
    static constexpr int D = kHeadDim;
    static constexpr int ROW_M = D * P / 8, ROW_E = D / N;
    static constexpr int STAGES = kStages;
    static constexpr int KM_OFF = 0;
    static constexpr int VM_OFF = kTile * ROW_M;
    static constexpr int KE_OFF = 2 * kTile * ROW_M;
    static constexpr int VE_OFF = KE_OFF + kTile * ROW_E;
    static constexpr int STAGE_BYTES = 2 * kTile * (ROW_M + ROW_E);
    static constexpr int WARP_BYTES = STAGES * STAGE_BYTES;
    static constexpr int LUT_OFF = kWarps * WARP_BYTES;                 // uint2[256]
    static constexpr int BAR_OFF = LUT_OFF + 256 * 8;
    template <int NT> static constexpr int smem_bytes() { return BAR_OFF + kWarps * STAGES * 8; }
};

template <int P, int N, int NT>
__global__ void __launch_bounds__(kWarps * 32, kMinCtas) decode_mma(DecodeArgs a) {
    using G_ = Geo<P, N>;
    constexpr int D = kHeadDim, ROW_M = G_::ROW_M, ROW_E = G_::ROW_E, STAGES = G_::STAGES;
    constexpr int NBK = (N == 16) ? 2 : 1;            // blocks inside a K lane chunk of 32 slots
    extern __shared__ __align__(128) uint8_t smem[];

    // weight table: entry e = (2^(e-127-(P-2)) twice as bf16x2, the same times the negated bias)
    uint2* lut = reinterpret_cast<uint2*>(smem + G_::LUT_OFF);
    for (int e = threadIdx.x; e < 256; e += kWarps * 32) {
        const uint32_t s2 = weight_bf16<P>((uint32_t)e) * 0x00010001u;
        lut[e] = make_uint2(s2, mul_bf16x2(s2, Fmt<P>::bias));
    }
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int Hkv = a.fmt.n_kv_heads, Gq = a.n_q_heads / Hkv;
    const int64_t item = (int64_t)blockIdx.x * kWarps + warp;
    const int64_t n_items = (int64_t)a.fmt.batch * Hkv * a.n_chunks;
    if (item >= n_items) return;
    const int chunk_id = (int)(item % a.n_chunks);
    const int hk = (int)((item / a.n_chunks) % Hkv);
    const int b = (int)(item / a.n_chunks / Hkv);

    int len = a.seq_lens[b];
    if (len > a.fmt.max_seq || len < 0) {
        if (lane == 0 && chunk_id == 0 && hk == 0) raise_flag(a.status, KVBFP_FLAG_POSITION);
        len = len < 0 ? 0 : a.fmt.max_seq;
    }
    if (len > a.len_cap) {
        if (lane == 0 && chunk_id == 0 && hk == 0) raise_flag(a.status, KVBFP_FLAG_LEN_HINT);
        len = a.len_cap;
    }
    const int t0 = chunk_id * a.chunk;
    if (t0 >= len) return;
    const int t1 = min(len, t0 + a.chunk);
    const int n_tiles = (t1 - t0 + kTile - 1) / kTile;

    uint8_t* wsm = smem + warp * G_::WARP_BYTES;
    const uint32_t wsm_u32 = smem_u32(wsm);
    const uint32_t bar0 = smem_u32(smem + G_::BAR_OFF + warp * STAGES * 8);
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) mbar_init(bar0 + 8 * s, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    const int64_t row0 = ((int64_t)b * Hkv + hk) * a.fmt.max_seq + t0;
    const uint8_t* gkm = a.k_mant + row0 * ROW_M;
    const uint8_t* gvm = a.v_mant + row0 * ROW_M;
    const uint8_t* gke = a.k_exp + row0 * ROW_E;
    const uint8_t* gve = a.v_exp + row0 * ROW_E;
    const int n_tok = t1 - t0;
    auto issue = [&](int stage, int tile) {      // lane 0 only
        const int off = tile * kTile;
        int rows = n_tok - off;
        rows = rows >= kTile ? kTile : ((rows + 15) & ~15);     // whole 16-token groups; stays below max_seq
        const uint32_t bar = bar0 + 8 * stage;
        const uint32_t dst = wsm_u32 + stage * G_::STAGE_BYTES;
        mbar_expect_tx(bar, (uint32_t)(2 * rows * (ROW_M + ROW_E)));
        bulk_g2s(dst + G_::KM_OFF, gkm + off * ROW_M, rows * ROW_M, bar);
        bulk_g2s(dst + G_::VM_OFF, gvm + off * ROW_M, rows * ROW_M, bar);
        bulk_g2s(dst + G_::KE_OFF, gke + off * ROW_E, rows * ROW_E, bar);
        bulk_g2s(dst + G_::VE_OFF, gve + off * ROW_E, rows * ROW_E, bar);
    };
    if (lane == 0) {
        for (int s = 0; s < STAGES && s < n_tiles; ++s) issue(s, s);
    }

    // B fragments of pi(q): 16 registers per n-tile
    uint2 qf[NT][8];
    {
        const uint4* src = reinterpret_cast<const uint4*>(a.qfrag) + (((int64_t)b * Hkv + hk) * NT) * (4 * 32);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint4 v = __ldg(src + (nt * 4 + j) * 32 + lane);
                qf[nt][2 * j] = make_uint2(v.x, v.y);
                qf[nt][2 * j + 1] = make_uint2(v.z, v.w);
            }
    }
#define QF(nt, ks) (qf[nt][ks])

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

    // per-lane byte offsets inside a stage
    const int k_off = G_::KM_OFF + g * ROW_M + t * (4 * P);                       // + mt*16*ROW_M, + 8*ROW_M
    const int ke_off = G_::KE_OFF + g * ROW_E + ((N == 16) ? 2 * t : (N == 32) ? t : (N == 64) ? (t >> 1) : 0);
    const int v_off = G_::VM_OFF + t * ROW_M + g * (2 * P);                       // + (mt*16 + 4k)*ROW_M
    const int ve_off = G_::VE_OFF + t * ROW_E + (16 * g) / N;
    const int src_lo = 4 * t + (g >> 1), src_hi = 4 * (t + 4) + (g >> 1);
    const bool odd_col = (g & 1) != 0;

    bool timed_out = false;
    for (int it = 0; it < n_tiles; ++it) {
        const int stage = it % STAGES;
        const uint32_t parity = (uint32_t)(it / STAGES) & 1u;
        if (!mbar_wait_bounded(bar0 + 8 * stage, parity)) { timed_out = true; break; }
        const uint8_t* st = wsm + stage * G_::STAGE_BYTES;
        const int n_live = n_tok - it * kTile;        // tokens of this tile that exist (may exceed kTile)
        const bool full = n_live >= kTile;

        // ---- scores -------------------------------------------------------------
        float sc[kMT][NT][2];
#pragma unroll
        for (int mt = 0; mt < kMT; ++mt) {
            if (mt * 16 >= n_live) {
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) sc[mt][nt][0] = sc[mt][nt][1] = -INFINITY;
                continue;
            }
            uint32_t wa[P], wb[P];
            {
                const uint8_t* pa = st + k_off + mt * 16 * ROW_M;
                const uint8_t* pb = pa + 8 * ROW_M;
                if (P == 6) {
#pragma unroll
                    for (int i = 0; i < 3; ++i) {
                        uint2 x = reinterpret_cast<const uint2*>(pa)[i], y = reinterpret_cast<const uint2*>(pb)[i];
                        wa[2 * i] = x.x; wa[2 * i + 1] = x.y; wb[2 * i] = y.x; wb[2 * i + 1] = y.y;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < P / 4; ++i) {
                        uint4 x = reinterpret_cast<const uint4*>(pa)[i], y = reinterpret_cast<const uint4*>(pb)[i];
                        wa[4 * i] = x.x; wa[4 * i + 1] = x.y; wa[4 * i + 2] = x.z; wa[4 * i + 3] = x.w;
                        wb[4 * i] = y.x; wb[4 * i + 1] = y.y; wb[4 * i + 2] = y.z; wb[4 * i + 3] = y.w;
                    }
                }
            }
            Wgt ga[NBK], gb[NBK];
#pragma unroll
            for (int k = 0; k < NBK; ++k) {
                const uint2 la = lut[st[ke_off + mt * 16 * ROW_E + k]];
                const uint2 lb = lut[st[ke_off + (mt * 16 + 8) * ROW_E + k]];
                ga[k] = make_wgt<P>(la.x, la.y);
                gb[k] = make_wgt<P>(lb.x, lb.y);
            }
            constexpr int NACC = 2;     // two independent accumulator chains for the score MMAs
            float acc[NT][NACC][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int c = 0; c < NACC; ++c) acc[nt][c][0] = acc[nt][c][1] = acc[nt][c][2] = acc[nt][c][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 8; ks += 2) {
                const int kb = (NBK == 2) ? (ks >> 2) : 0;
                uint32_t ra[4], rb[4];
                k_pairs2<P>(wa, ks, ga[kb], ra);
                k_pairs2<P>(wb, ks, gb[kb], rb);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const uint2 q0 = QF(nt, ks), q1 = QF(nt, ks + 1);
                    mma_bf16(acc[nt][0], ra[0], rb[0], ra[1], rb[1], q0.x, q0.y);
                    mma_bf16(acc[nt][NACC - 1], ra[2], rb[2], ra[3], rb[3], q1.x, q1.y);
                }
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                float s0 = acc[nt][0][0] + acc[nt][0][1], s1 = acc[nt][0][2] + acc[nt][0][3];
                if (NACC == 2) {
                    s0 += acc[nt][1][0] + acc[nt][1][1];
                    s1 += acc[nt][1][2] + acc[nt][1][3];
                }
                sc[mt][nt][0] = s0 * a.scale_log2e;
                sc[mt][nt][1] = s1 * a.scale_log2e;
            }
            if (!full) {       // select, not arithmetic: rows past the end may hold anything
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    if (mt * 16 + g >= n_live) sc[mt][nt][0] = -INFINITY;
                    if (mt * 16 + g + 8 >= n_live) sc[mt][nt][1] = -INFINITY;
                }
            }
        }

        // ---- running softmax (reference point moves only in big steps) ----------
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
#pragma unroll
                for (int r = 0; r < 8; ++r)
#pragma unroll
                    for (int k = 0; k < 4; ++k) o[nt][r][k] *= alpha;
            }
        }

        // ---- P.V ----------------------------------------------------------------
#pragma unroll
        for (int mt = 0; mt < kMT; ++mt) {
            if (mt * 16 >= n_live) continue;
            // softmax weights of this lane's tokens (g and g+8), then the B fragment of P^T for lane (g, t):
            // column g = (query g/2, half g%2); tokens t, t+4 | t+8, t+12
            uint32_t pb[NT][2];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const float p0 = ex2_approx(sc[mt][nt][0] - m_run[nt]);
                const float p1 = ex2_approx(sc[mt][nt][1] - m_run[nt]);
                l_run[nt] += p0 + p1;
                const float v0 = __shfl_sync(0xffffffffu, p0, src_lo);   // token t
                const float v1 = __shfl_sync(0xffffffffu, p0, src_hi);   // token t+4
                const float v2 = __shfl_sync(0xffffffffu, p1, src_lo);   // token t+8
                const float v3 = __shfl_sync(0xffffffffu, p1, src_hi);   // token t+12
                // hi half = the value cut to its upper 16 bits (an exact bf16); lo half = the rest
                const uint32_t u0 = __float_as_uint(v0), u1 = __float_as_uint(v1);
                const uint32_t u2 = __float_as_uint(v2), u3 = __float_as_uint(v3);
                const uint32_t hiA = prmt(u0, u1, 0x7632u), hiB = prmt(u2, u3, 0x7632u);
                const uint32_t loA = pack_bf16x2_rn(v0 - __uint_as_float(u0 & 0xffff0000u), v1 - __uint_as_float(u1 & 0xffff0000u));
                const uint32_t loB = pack_bf16x2_rn(v2 - __uint_as_float(u2 & 0xffff0000u), v3 - __uint_as_float(u3 & 0xffff0000u));
                pb[nt][0] = odd_col ? loA : hiA;
                pb[nt][1] = odd_col ? loB : hiB;
            }
            // V pieces: slots [16g, 16g+16) of tokens t, t+4, t+8, t+12 of this row tile
            constexpr int VW = P / 2;      // words per token piece
            uint32_t vw[4][VW];
            uint32_t ev[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint8_t* pv = st + v_off + (mt * 16 + 4 * k) * ROW_M;
                if (P == 4) {
                    uint2 x = *reinterpret_cast<const uint2*>(pv);
                    vw[k][0] = x.x; vw[k][1] = x.y;
                } else if (P == 6) {
#pragma unroll
                    for (int i = 0; i < 3; ++i) vw[k][i] = reinterpret_cast<const uint32_t*>(pv)[i];
                } else {
                    uint4 x = *reinterpret_cast<const uint4*>(pv);
                    vw[k][0] = x.x; vw[k][1] = x.y; vw[k][2] = x.z; vw[k][3] = x.w;
                }
                ev[k] = st[ve_off + (mt * 16 + 4 * k) * ROW_E];
            }
            uint2 lv[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) lv[k] = lut[ev[k]];
            if (!full) {       // rows past the end contribute exactly zero
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (mt * 16 + t + 4 * k >= n_live) lv[k] = make_uint2(0u, 0u);
            }
            const Wgt gA = make_wgt<P>(prmt(lv[0].x, lv[1].x, 0x7610u), prmt(lv[0].y, lv[1].y, 0x7610u));
            const Wgt gB = make_wgt<P>(prmt(lv[2].x, lv[3].x, 0x7610u), prmt(lv[2].y, lv[3].y, 0x7610u));
#pragma unroll
            for (int r = 0; r < 8; r += 2) {
                uint32_t xa[4], xb[4];
                v_pairs2<P>(vw[0], vw[1], r, gA, xa);
                v_pairs2<P>(vw[2], vw[3], r, gB, xb);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    mma_bf16(o[nt][r], xa[0], xa[1], xb[0], xb[1], pb[nt][0], pb[nt][1]);
                    mma_bf16(o[nt][r + 1], xa[2], xa[3], xb[2], xb[3], pb[nt][0], pb[nt][1]);
                }
            }
        }

        __syncwarp();
        if (lane == 0 && it + STAGES < n_tiles) issue(stage, it + STAGES);
    }

    if (timed_out) {
        // give the copies still in flight a bounded chance to land before the shared memory is released
        if (lane == 0) raise_flag(a.status, KVBFP_FLAG_WAIT_TIMEOUT);
        for (int s = 0; s < STAGES; ++s) {
            (void)mbar_wait_bounded(bar0 + 8 * s, 0);
            (void)mbar_wait_bounded(bar0 + 8 * s, 1);
        }
        return;
    }

    // ---- per-chunk partial results ------------------------------------------------
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        float l = l_run[nt];
        l += __shfl_xor_sync(0xffffffffu, l, 4);
        l += __shfl_xor_sync(0xffffffffu, l, 8);
        l += __shfl_xor_sync(0xffffffffu, l, 16);
        const int qi = 4 * nt + t;
        if (qi < Gq) {
            float* dst = a.partials + (((int64_t)b * a.n_q_heads + hk * Gq + qi) * a.n_chunks + chunk_id) * kPartStride;
#pragma unroll
            for (int r4 = 0; r4 < 4; ++r4) {
                float4 v;
                v.x = o[nt][2 * r4][0] + o[nt][2 * r4][1];
                v.y = o[nt][2 * r4][2] + o[nt][2 * r4][3];
                v.z = o[nt][2 * r4 + 1][0] + o[nt][2 * r4 + 1][1];
                v.w = o[nt][2 * r4 + 1][2] + o[nt][2 * r4 + 1][3];
                reinterpret_cast<float4*>(dst + 16 * g)[r4] = v;
            }
            if (g == 0) { dst[D] = m_run[nt]; dst[D + 1] = l; }
        }
    }
}

template <int P, int N, int NT>
kvbfp_status launch3(const DecodeArgs& a, cudaStream_t s) {
    using G_ = Geo<P, N>;
    static std::atomic<bool> attr_set[64];      // per device; setting the attribute twice is harmless
    int dev = 0;
    KVBFP_CUDA(cudaGetDevice(&dev));
    if (dev >= 0 && dev < 64 && !attr_set[dev].load(std::memory_order_acquire)) {
        KVBFP_CUDA(cudaFuncSetAttribute(decode_mma<P, N, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, G_::template smem_bytes<NT>()));
        attr_set[dev].store(true, std::memory_order_release);
    }
    const int n_pre = a.fmt.batch * a.fmt.n_kv_heads * NT;
    make_qfrag<P><<<n_pre, 32, 0, s>>>(a, NT);
    KVBFP_LAUNCH_CHECK("make_qfrag");
    const int64_t n_items = (int64_t)a.fmt.batch * a.fmt.n_kv_heads * a.n_chunks;
    if ((n_items + kWarps - 1) / kWarps > 0x7fffffffLL) return KVBFP_ERR_UNSUPPORTED;     // more thread blocks than a grid holds
    const int grid = (int)((n_items + kWarps - 1) / kWarps);
    cudaEvent_t ev0, ev1;
    profile_events(&ev0, &ev1);
    if (ev0) KVBFP_CUDA(cudaEventRecord(ev0, s));
    decode_mma<P, N, NT><<<grid, kWarps * 32, G_::template smem_bytes<NT>(), s>>>(a);
    KVBFP_LAUNCH_CHECK("decode_mma");
    if (ev1) KVBFP_CUDA(cudaEventRecord(ev1, s));
    return KVBFP_OK;
}

template <int P, int N>
kvbfp_status launch2(const DecodeArgs& a, cudaStream_t s) {
    const int G = a.n_q_heads / a.fmt.n_kv_heads;
    return (G <= 4) ? launch3<P, N, 1>(a, s) : launch3<P, N, 2>(a, s);
}

template <int P>
kvbfp_status launch1(const DecodeArgs& a, cudaStream_t s) {
    switch (a.fmt.block) {
        case 16: return launch2<P, 16>(a, s);
        case 32: return launch2<P, 32>(a, s);
        case 64: return launch2<P, 64>(a, s);
        case 128: return launch2<P, 128>(a, s);
    }
    return KVBFP_ERR_UNSUPPORTED;
}

}  // namespace

kvbfp_status launch_decode_mma(const DecodeArgs& a, cudaStream_t s) {
    switch (a.fmt.mant_bits) {
        case 4: return launch1<4>(a, s);
        case 6: return launch1<6>(a, s);
        case 8: return launch1<8>(a, s);
    }
    return KVBFP_ERR_UNSUPPORTED;
}

}  // namespace kvbfp
