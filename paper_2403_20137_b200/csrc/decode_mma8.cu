// Decode attention over an 8-bit BFP cache (blocks of 32 slots or more): integer tensor-core MMAs for the
// scores on the stored bytes as they are, fp16 tensor-core MMAs for P.V
// (Sec. III par. 2 of the paper: keys are read back from the cache and multiplied with pi(q);
// Sec. II-B: the inner product of two BFP blocks is an integer product plus an exponent addition).
//
// Same launch design as the 4-bit kernel: work items laid out pair-major and cut into one contiguous range per
// resident warp (persistent), "runs" with one partial result each, a private ring of shared-memory stages per
// warp (each warp fetches its own tiles), no block-wide barrier in the loop.  The K and V byte tiles come by tiled 2-D
// asynchronous copies over tensor maps of the two planes (a row = one token = 128 bytes, 128-byte swizzle: the
// 16-byte piece p of row r lands at piece p ^ (r % 8)), which makes the fragment loads below conflict-free; the
// exponent bytes come by 1-D bulk copies.
//
// A stored byte is B = M + 128 (excess code), so nothing has to be unpacked.
//   Scores: the bytes are the unsigned operand of a byte MMA.  The query block is cast to 15-bit fixed point
//   C = round(q * 2^(14 - qe)) with the block's own exponent qe and split into two signed byte digits,
//   C = 256 d1 + d0, which sit in two MMA columns; 256 * sum(B d1) + sum(B d0) - 128 * sum(C) = sum(M C) exactly
//   (the last term enters as the accumulator's start value), and one fp32 multiply-add applies
//   2^(e_k - 133) * 2^(qe - 14) * scale per (token, block).
//   P.V: a byte is put under the bits of fp16 1024.0 by a byte permute or a mask-or (1024 + B, exact); one f16x2
//   fma with the block's power of two removes the bias 1152 and applies the weight, exactly (|M| < 2^7).  The
//   weights are 2^(e - D + 5) relative to a reference exponent byte D that the warp raises tile by tile (see the
//   4-bit kernel); 2^(D - 138) is applied in fp32 to the partial result.  Softmax weights are (hi, lo) fp16 pairs.
#include <math.h>

#include <atomic>
#include <type_traits>

#include "decode.cuh"
#include "ptx.cuh"

namespace kvbfp {
namespace {

constexpr int kWarps = 4;
constexpr int kMT = 2;                  // 16-token MMA row tiles per stage
constexpr int kTile = 16 * kMT;         // tokens per stage
constexpr int kStages = 2;
constexpr int D = kHeadDim;
constexpr int ROW_M = D;                // one byte per slot
constexpr int kTopShift = 5;            // weight of a block at the reference exponent is 2^kTopShift
constexpr int kDvHeadroom = 2;
constexpr int kLutEntries = 512;
constexpr uint32_t kMagic = 0x64646464u;        // 0x64 = high byte of fp16 1024.0
constexpr uint32_t kBias = 0xE480E480u;         // fp16 -1152.0 twice

// ------------------------------------------------------------------ query fragments
// One 128-thread block per (batch, kv head, n-tile of four query heads); thread s = slot s.  Fragment m (0..7) of an
// n-tile covers row bytes {32 (m/2) + 8 t + 4 (m%2) + e : t, e = 0..3}: lane (g, t) of the main kernel reads eight
// consecutive bytes per 32-byte group, the first four feed MMA m = even, the last four MMA m = odd.  Column
// g = (query g/2, digit g%2: 0 = d1, 1 = d0).  qmeta[query][2 blk] = scale * log2(e) * 2^(qe - 14) as float bits,
// qmeta[query][2 blk + 1] = 128 * sum(C) of the block.
__global__ void __launch_bounds__(128) make_qfrag8i(DecodeArgs a, int NT, int32_t* qmeta) {
    pdl_wait();
    pdl_trigger();
    const int N = a.fmt.block, nblk = D / N;
    const int s = threadIdx.x, blk = s / N;
    const int item = blockIdx.x;
    const int nt = item % NT, hk = (item / NT) % a.fmt.n_kv_heads, b = item / NT / a.fmt.n_kv_heads;
    const int G = a.n_q_heads / a.fmt.n_kv_heads;
    __shared__ int sC[4][D];
    __shared__ uint32_t smax[2][4][4];
    __shared__ int sbias[4][4];
    if (s < 32) reinterpret_cast<uint32_t*>(smax)[s] = 0u;
    if (s < 16) reinterpret_cast<int*>(sbias)[s] = 0;
    __syncthreads();
    const int ch = a.perm_k ? (a.perm_k[hk * D + s] & (D - 1)) : s;
    float v[4];
#pragma unroll
    for (int qq = 0; qq < 4; ++qq) {
        v[qq] = 0.f;
        if (4 * nt + qq < G) {
            const int64_t idx = ((int64_t)b * a.n_q_heads + hk * G + 4 * nt + qq) * D + ch;
            v[qq] = a.q_is_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(a.q)[idx]) : static_cast<const float*>(a.q)[idx];
        }
    }
    if (a.q_mant_bits) {   // BFP query (Sec. IV): blocks of N slots, 8-bit mantissas
#pragma unroll
        for (int qq = 0; qq < 4; ++qq) {
            const uint32_t mx = __reduce_max_sync(0xffffffffu, __float_as_uint(v[qq]) & 0x7fffffffu);
            if ((s & 31) == 0) atomicMax(&smax[0][qq][blk], mx);
        }
        __syncthreads();
#pragma unroll
        for (int qq = 0; qq < 4; ++qq) {
            int e8 = (int)(smax[0][qq][blk] >> 23);
            if (e8 == 255) { raise_flag(a.status, KVBFP_FLAG_NONFINITE); e8 = 254; }
            const int k = 127 - e8 + 6, k1 = k >> 1, k2 = k - k1;
            const float tv = (v[qq] * pow2i(k1)) * pow2i(k2);
            v[qq] = rintf(fminf(fmaxf(tv, -127.f), 127.f)) * unit_weight(e8, 8);
        }
    }
#pragma unroll
    for (int qq = 0; qq < 4; ++qq) {
        const uint32_t mx = __reduce_max_sync(0xffffffffu, __float_as_uint(v[qq]) & 0x7fffffffu);
        if ((s & 31) == 0) atomicMax(&smax[1][qq][blk], mx);
    }
    __syncthreads();
#pragma unroll
    for (int qq = 0; qq < 4; ++qq) {
        const uint32_t am = smax[1][qq][blk];
        int e = (int)(am >> 23);
        if (e == 255) { raise_flag(a.status, KVBFP_FLAG_NONFINITE); e = 254; }
        const int qe = (am == 0) ? 0 : e - 126;               // |q| * 2^-qe < 1
        const int sh = 14 - qe, h1 = sh / 2, h2 = sh - h1;    // two exact factors
        const int C = __float2int_rn((v[qq] * pow2i(h1)) * pow2i(h2));
        sC[qq][s] = C;
        const int bsum = __reduce_add_sync(0xffffffffu, 128 * C);
        if ((s & 31) == 0) atomicAdd(&sbias[qq][blk], bsum);
        if (s % N == 0 && 4 * nt + qq < G)
            qmeta[((int64_t)b * a.n_q_heads + hk * G + 4 * nt + qq) * 8 + 2 * blk] = __float_as_int(pow2_split(a.scale_log2e, qe - 14));
    }
    __syncthreads();
    if (s < 4 * nblk) {
        const int qq = s / nblk, k = s % nblk;
        if (4 * nt + qq < G) qmeta[((int64_t)b * a.n_q_heads + hk * G + 4 * nt + qq) * 8 + 2 * k + 1] = sbias[qq][k];
    }
    const int lane = s & 31, gp = lane >> 2, tp = lane & 3;
    const int qq = gp >> 1, digit = gp & 1, qi = 4 * nt + qq;
    uint32_t* dst = a.qfrag + (int64_t)item * (8 * 32);
#pragma unroll
    for (int mm = 0; mm < 2; ++mm) {
        const int m = (s >> 5) + 4 * mm;
        uint32_t reg = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int C = sC[qq][32 * (m >> 1) + 8 * tp + 4 * (m & 1) + e];
            const int d1 = (C + 128) >> 8, d0 = C - 256 * d1;
            const int dsel = (qi < G) ? (digit ? d0 : d1) : 0;
            reg |= ((uint32_t)dsel & 0xffu) << (8 * e);
        }
        dst[((m >> 2) * 32 + lane) * 4 + (m & 3)] = reg;
    }
}

// ------------------------------------------------------------------ main kernel
constexpr int kTileBytes = kTile * ROW_M;      // 4 KiB: a whole number of 1 KiB swizzle periods
template <int N>
struct Geo8 {
    static constexpr int ROW_E = D / N;
    // mantissa tiles first (1 KiB-aligned: the swizzle pattern is a function of the address), then the exponent bytes
    static constexpr int MANT_STAGE = 2 * kTileBytes;                   // K tile, V tile
    static constexpr int KM_OFF = 0;
    static constexpr int VM_OFF = kTileBytes;
    static constexpr int EXP_OFF = kWarps * kStages * MANT_STAGE;       // per (warp, stage): K bytes, V bytes
    static constexpr int EXP_STAGE = 2 * kTile * ROW_E;
    static constexpr int KE_OFF = 0;
    static constexpr int VE_OFF = kTile * ROW_E;
    static constexpr int LUT_OFF = EXP_OFF + kWarps * kStages * EXP_STAGE;   // uint2[kLutEntries]
    static constexpr int LUTF_OFF = LUT_OFF + kLutEntries * 8;          // float[256]
    static constexpr int BAR_OFF = LUTF_OFF + 256 * 4;
    static constexpr int SMEM_BYTES = BAR_OFF + kWarps * kStages * 8;
};
// Tokens of a 16-token row tile whose V bytes lane (g, t) loads for P.V, k = 0..3: 2t, 2t+1, 2t+8, 2t+9 -- the MMA's
// own order of the contraction index, and rows whose numbers mod 8 differ in bits 1 and 2 across t, so that the
// eight lanes of a quarter warp (two values of g, four of t) read eight different swizzled pieces.
__device__ __forceinline__ int tok8(int t, int k) { return 2 * t + (k & 1) + 4 * (k & 2); }

template <int N, int NT>
__global__ void __launch_bounds__(kWarps * 32, 3) decode_mma8(DecodeArgs a, const int32_t* __restrict__ qmeta,
                                                              const __grid_constant__ CUtensorMap k_map,
                                                              const __grid_constant__ CUtensorMap v_map) {
    pdl_wait();
    using G_ = Geo8<N>;
    constexpr int ROW_E = G_::ROW_E;
    constexpr int NBLK = D / N;                       // blocks of a row
    constexpr int GRP_PER_BLK = 4 / NBLK;             // 32-byte groups per block
    extern __shared__ __align__(1024) uint8_t smem[];         // the swizzle pattern is a function of the address

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

    // ---- producer: lanes 0..3 each own one of the four pieces of a stage: the K and V byte tiles (tiled copies of
    // kTile whole rows: rows past the sequence are never used, rows past the plane arrive as zeros) and the K and V
    // exponent bytes (1-D copies of the 16-token groups that hold tokens)
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
            if (lane < 2) tensor_g2s_2d(my_dst + stage * G_::MANT_STAGE, my_map, 0, (int)(pr.row0 + off), bar);
            else bulk_g2s(my_dst + stage * G_::EXP_STAGE, my_exp + (pr.row0 + off) * ROW_E, rows * ROW_E, bar);
        }
        ++p_tile;
    };
    for (int s = 0; s < kStages; ++s) issue_next(s);

    // (the tables are filled while the first copies are in flight)
    // fp16 weight table: entry i = (2^(i - 255 + kTopShift) twice, the same times -1152); entries above 255 belong
    // to rows that are masked later and only have to exist
    uint2* lut = reinterpret_cast<uint2*>(smem + G_::LUT_OFF);
    for (int i = threadIdx.x; i < kLutEntries; i += kWarps * 32) {
        const uint32_t s2 = (i <= 255 ? pow2_f16(i - 255 + kTopShift) : 0u) * 0x00010001u;
        lut[i] = make_uint2(s2, mul_f16x2(s2, kBias));
    }
    float* lutf = reinterpret_cast<float*>(smem + G_::LUTF_OFF);      // 2^(e - 133): weight of a mantissa unit
    for (int i = threadIdx.x; i < 256; i += kWarps * 32) lutf[i] = unit_weight(i, 8);
    __syncthreads();
    if (i0 >= i1) return;

    // per-lane byte offsets inside a stage (mantissa tiles swizzled: byte b of row r sits at b ^ ((r % 8) << 4))
    int k_sw[4];                                               // this lane's eight bytes of each 32-byte group, rows g and g + 8
#pragma unroll
    for (int grp = 0; grp < 4; ++grp) k_sw[grp] = G_::KM_OFF + g * ROW_M + ((t * 8 + 32 * grp) ^ (g << 4));
    const int kei_off = G_::KE_OFF + g * ROW_E;
    int v_off[4], ve_off[4];                                   // bytes [16g, 16g + 16) of rows tok8(t, k)
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int r = tok8(t, k);
        v_off[k] = G_::VM_OFF + r * ROW_M + ((g ^ (r & 7)) << 4);
        ve_off[k] = G_::VE_OFF + r * ROW_E + (16 * g) / N;
    }
    // softmax weights travel from the lanes that computed them (token = lane / 4 and + 8, column pair = lane % 4)
    const int src_lo = 4 * tok8(t, 0) + (g >> 1), src_hi = 4 * tok8(t, 1) + (g >> 1);
    const uint32_t half_sel = (g & 1) ? 0x7632u : 0x5410u;     // odd columns carry the lo halves

    int stage = 0;
    uint32_t parity = 0;
    bool timed_out = false;

    for (int c_next = i0; c_next < i1 && !timed_out;) {
        const Run cr = get_run(c_next);
        c_next += cr.n_items;
        if (cr.n_tok == 0) continue;

        // ---- run set-up: query fragments, score factors, V reference exponent
        uint32_t qi8[NT][8];              // B fragments of the coefficient digits
        float qfac[NT][NBLK];             // scale * log2(e) * 2^(qe - 14) per block
        int qbias[NT][NBLK];              // 128 * sum(C) per block
        {
            const uint4* src = reinterpret_cast<const uint4*>(a.qfrag);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int qn = 4 * nt + t;
                const int32_t* meta = qmeta + ((int64_t)cr.b * a.n_q_heads + cr.hk * Gq + (qn < Gq ? qn : 0)) * 8;
                const uint4* s8 = src + (((int64_t)cr.b * Hkv + cr.hk) * NT + nt) * (2 * 32);
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const uint4 v = __ldg(s8 + j * 32 + lane);
                    qi8[nt][4 * j] = v.x; qi8[nt][4 * j + 1] = v.y; qi8[nt][4 * j + 2] = v.z; qi8[nt][4 * j + 3] = v.w;
                }
#pragma unroll
                for (int k = 0; k < NBLK; ++k) {
                    qfac[nt][k] = __int_as_float(meta[2 * k]);
                    qbias[nt][k] = meta[2 * k + 1];
                }
            }
        }
        int dv = 0;                               // reference exponent byte of the V weights, raised on the way
        uint32_t dv_probe = 0x7FFF7FFFu;          // (0x7FFF - dv) in both halves: adding a byte > dv sets bit 15
        const uint2* lutv = lut + 255;
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
                const float f = pow2_split(1.f, dv - nd);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int r = 0; r < 8; ++r)
#pragma unroll
                        for (int k = 0; k < 4; ++k) o[nt][r][k] *= f;
                dv = nd;
                dv_probe = (0x7FFFu - (uint32_t)nd) * 0x00010001u;
                lutv = lut + (255 - nd);
            }
        };

        // one stage of kTile tokens; FULL = every row of the tile exists
        auto tile_body = [&](const uint8_t* st, const uint8_t* se, int n_live, auto full_tag) {
            constexpr bool FULL = decltype(full_tag)::value;
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
                int acc[NT][NBLK][4];
                const uint8_t* pa = st + mt * 16 * ROW_M;
#pragma unroll
                for (int grp = 0; grp < 4; ++grp) {        // 32-byte groups of the row; this lane's eight bytes of each
                    const uint2 wa = *reinterpret_cast<const uint2*>(pa + k_sw[grp]);
                    const uint2 wb = *reinterpret_cast<const uint2*>(pa + 8 * ROW_M + k_sw[grp]);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        if (grp % GRP_PER_BLK == 0)   // first MMA of a block: the offsets' constant contribution goes in as C
                            mma_u8s8_first(acc[nt][grp / GRP_PER_BLK], wa.x, wb.x, qi8[nt][2 * grp], 0, -qbias[nt][grp / GRP_PER_BLK]);
                        else
                            mma_u8s8(acc[nt][grp / GRP_PER_BLK], wa.x, wb.x, qi8[nt][2 * grp]);
                        mma_u8s8(acc[nt][grp / GRP_PER_BLK], wa.y, wb.y, qi8[nt][2 * grp + 1]);
                    }
                }
                float s0[NT], s1[NT];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) s0[nt] = s1[nt] = 0.f;
#pragma unroll
                for (int k = 0; k < NBLK; ++k) {
                    const float w0 = lutf[se[kei_off + mt * 16 * ROW_E + k]];
                    const float w1 = lutf[se[kei_off + (mt * 16 + 8) * ROW_E + k]];
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        const float f0 = __int2float_rn(256 * acc[nt][k][0] + acc[nt][k][1]);
                        const float f1 = __int2float_rn(256 * acc[nt][k][2] + acc[nt][k][3]);
                        s0[nt] = fmaf(f0, w0 * qfac[nt][k], s0[nt]);
                        s1[nt] = fmaf(f1, w1 * qfac[nt][k], s1[nt]);
                    }
                }
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) { sc[mt][nt][0] = s0[nt]; sc[mt][nt][1] = s1[nt]; }
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
                // B fragment of P^T for lane (g, t): column g = (query g/2, half g%2); tokens 2t, 2t+1 | 2t+8, 2t+9
                uint32_t pb[NT][2];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const float p0 = ex2_approx(sc[mt][nt][0] - m_run[nt]);
                    const float p1 = ex2_approx(sc[mt][nt][1] - m_run[nt]);
                    l_run[nt] += p0 + p1;
                    const float h0 = __uint_as_float(__float_as_uint(p0) & 0xffffe000u);
                    const float h1 = __uint_as_float(__float_as_uint(p1) & 0xffffe000u);
                    const uint32_t w0 = pack_f16x2_rn(h0, p0 - h0), w1 = pack_f16x2_rn(h1, p1 - h1);
                    const uint32_t v0 = __shfl_sync(0xffffffffu, w0, src_lo);   // token 2t
                    const uint32_t v1 = __shfl_sync(0xffffffffu, w0, src_hi);   // token 2t+1
                    const uint32_t v2 = __shfl_sync(0xffffffffu, w1, src_lo);   // token 2t+8
                    const uint32_t v3 = __shfl_sync(0xffffffffu, w1, src_hi);   // token 2t+9
                    pb[nt][0] = prmt(v0, v1, half_sel);
                    pb[nt][1] = prmt(v2, v3, half_sel);
                }
                // V pieces: bytes [16g, 16g+16) (slots 16g..16g+15) of tokens tok8(t, 0..3) of this row tile
                uint4 vw[4];
                uint2 lv[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    vw[k] = *reinterpret_cast<const uint4*>(st + v_off[k] + mt * 16 * ROW_M);
                    lv[k] = lutv[se[ve_off[k] + mt * 16 * ROW_E]];
                }
                if (!FULL) {       // rows past the end contribute exactly zero
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (mt * 16 + tok8(t, k) >= n_live) lv[k] = make_uint2(0u, 0u);
                }
                const uint32_t sA = prmt(lv[0].x, lv[1].x, 0x7610u), cA = prmt(lv[0].y, lv[1].y, 0x7610u);
                const uint32_t sB = prmt(lv[2].x, lv[3].x, 0x7610u), cB = prmt(lv[2].y, lv[3].y, 0x7610u);
#pragma unroll
                for (int r = 0; r < 8; ++r) {         // byte pair (2r, 2r+1) of the lane's sixteen bytes = output rows g, g+8
                    const uint32_t wA0 = r < 2 ? vw[0].x : r < 4 ? vw[0].y : r < 6 ? vw[0].z : vw[0].w;
                    const uint32_t wA1 = r < 2 ? vw[1].x : r < 4 ? vw[1].y : r < 6 ? vw[1].z : vw[1].w;
                    const uint32_t wB0 = r < 2 ? vw[2].x : r < 4 ? vw[2].y : r < 6 ? vw[2].z : vw[2].w;
                    const uint32_t wB1 = r < 2 ? vw[3].x : r < 4 ? vw[3].y : r < 6 ? vw[3].z : vw[3].w;
                    const uint32_t sel = (r & 1) ? 0x7632u : 0x5410u;
                    const uint32_t XA = prmt(wA0, wA1, sel), XB = prmt(wB0, wB1, sel);     // [tok.b, tok.b', tok'.b, tok'.b']
                    const uint32_t ae = lop3<0xEA>(XA, 0x00FF00FFu, 0x64006400u), ao = prmt(XA, kMagic, 0x4341u);
                    const uint32_t be = lop3<0xEA>(XB, 0x00FF00FFu, 0x64006400u), bo = prmt(XB, kMagic, 0x4341u);
                    const uint32_t E0 = fma_f16x2(ae, sA, cA), O0 = fma_f16x2(ao, sA, cA);
                    const uint32_t E2 = fma_f16x2(be, sB, cB), O2 = fma_f16x2(bo, sB, cB);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) mma_f16(o[nt][r], E0, O0, E2, O2, pb[nt][0], pb[nt][1]);
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
            __syncwarp();
            issue_next(stage);
            if (++stage == kStages) { stage = 0; parity ^= 1u; }
        }
        if (timed_out) break;

        // ---- partial result of the run: output row g of row tile r is slot 16g + 2r, row g+8 is slot 16g + 2r + 1
        const float vfac = pow2_split(1.f, dv - 133 - kTopShift);
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
                    float4 v;
                    v.x = (o[nt][2 * r4][0] + o[nt][2 * r4][1]) * vfac;
                    v.y = (o[nt][2 * r4][2] + o[nt][2 * r4][3]) * vfac;
                    v.z = (o[nt][2 * r4 + 1][0] + o[nt][2 * r4 + 1][1]) * vfac;
                    v.w = (o[nt][2 * r4 + 1][2] + o[nt][2 * r4 + 1][3]) * vfac;
                    reinterpret_cast<float4*>(dst + 16 * g)[r4] = v;
                }
                if (g == 0) { dst[D] = m_run[nt]; dst[D + 1] = l; }
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

template <int N, int NT>
kvbfp_status launch3(const DecodeArgs& a, cudaStream_t s, Split* split) {
    using G_ = Geo8<N>;
    static std::atomic<int> resident[64];   // thread blocks that fit the whole device, per device (0 = not asked yet;
                                            // two host threads asking at once store the same number)
    int dev = 0;
    KVBFP_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return KVBFP_ERR_UNSUPPORTED;
    if (!resident[dev].load(std::memory_order_acquire)) {
        KVBFP_CUDA(cudaFuncSetAttribute(decode_mma8<N, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, G_::SMEM_BYTES));
        int per_sm = 0, n_sm = 0;
        KVBFP_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode_mma8<N, NT>, kWarps * 32, G_::SMEM_BYTES));
        KVBFP_CUDA(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
        if (per_sm < 1 || n_sm < 1) return KVBFP_ERR_CUDA;
        resident[dev].store(per_sm * n_sm, std::memory_order_release);
    }
    int32_t* qmeta = reinterpret_cast<int32_t*>(reinterpret_cast<uint8_t*>(a.qfrag) +
                                               (size_t)a.fmt.batch * a.fmt.n_kv_heads * NT * 8 * 32 * 2 * sizeof(uint32_t));
    const int n_pre = a.fmt.batch * a.fmt.n_kv_heads * NT;
    (void)launch_pdl(make_qfrag8i, dim3(n_pre), dim3(128), 0, s, a, NT, qmeta);
    KVBFP_LAUNCH_CHECK("make_qfrag8i");
    DecodeArgs b;
    int grid = 0;
    const kvbfp_status st = plan_persistent(a, kItemTokens, resident[dev].load(std::memory_order_relaxed), kWarps, &b, split, &grid);
    if (st != KVBFP_OK) return st;
    // tensor maps of the two byte planes (this device's memory; rows of one token, boxes of kTile tokens); a decode
    // loop passes the same planes step after step: the last pair of maps is kept per host thread
    struct MapCache { const void *k = nullptr, *v = nullptr; uint64_t rows = 0; int dev = -1; CUtensorMap k_map, v_map; };
    static thread_local MapCache mc;
    const uint64_t n_rows = (uint64_t)a.fmt.batch * a.fmt.n_kv_heads * a.fmt.max_seq;
    if (mc.k != a.k_mant || mc.v != a.v_mant || mc.rows != n_rows || mc.dev != dev) {
        mc.k = nullptr;
        kvbfp_status ms = make_row_map(&mc.k_map, a.k_mant, n_rows, ROW_M, kTile);
        if (ms == KVBFP_OK) ms = make_row_map(&mc.v_map, a.v_mant, n_rows, ROW_M, kTile);
        if (ms != KVBFP_OK) return ms;
        mc.k = a.k_mant; mc.v = a.v_mant; mc.rows = n_rows; mc.dev = dev;
    }
    cudaEvent_t ev0, ev1;
    profile_events(&ev0, &ev1);
    if (ev0) KVBFP_CUDA(cudaEventRecord(ev0, s));
    (void)launch_pdl(decode_mma8<N, NT>, dim3(grid), dim3(kWarps * 32), G_::SMEM_BYTES, s, b, (const int32_t*)qmeta, mc.k_map, mc.v_map);
    KVBFP_LAUNCH_CHECK("decode_mma8");
    if (ev1) KVBFP_CUDA(cudaEventRecord(ev1, s));
    return KVBFP_OK;
}

template <int N>
kvbfp_status launch2(const DecodeArgs& a, cudaStream_t s, Split* split) {
    const int G = a.n_q_heads / a.fmt.n_kv_heads;
    return (G <= 4) ? launch3<N, 1>(a, s, split) : launch3<N, 2>(a, s, split);
}

}  // namespace

kvbfp_status launch_decode_mma8(const DecodeArgs& a, cudaStream_t s, Split* split) {
    switch (a.fmt.block) {
        case 32: return launch2<32>(a, s, split);
        case 64: return launch2<64>(a, s, split);
        case 128: return launch2<128>(a, s, split);
    }
    return KVBFP_ERR_UNSUPPORTED;
}

}  // namespace kvbfp
