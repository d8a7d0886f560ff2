// Cache write: permute, shared exponent, round, clamp, pack, store (Sec. II-B last paragraph,
// Sec. III par. 2 of the paper; Algorithm 1 step 3 applied at run time as a gather).
//
// Sixteen lanes own one (token, head) row of 128 channels, eight stored slots per lane.  A block of n slots
// is held by n/8 neighbouring lanes; its largest magnitude is found with xor-shuffles on the IEEE bit
// patterns (integer compare = exact).  Rounding to nearest-even is one fused multiply-add with
// 1.5 * 2^23 + 2^(p-1): the integer M + 2^(p-1), which is the stored field, appears in the low bits of
// the sum.  Two kernels share this: append_quant_pack for single tokens (a thread block takes sixteen
// tokens per step and each 16-lane group walks the heads of its token), append_rows for runs of tokens
// (further down: a thread block per (sequence, head), rows staged through shared memory).
#include <atomic>
#include <type_traits>

#include "common.cuh"
#include "ptx.cuh"

namespace kvbfp {
namespace {

constexpr int kThreads = 256;
constexpr int kTokPerCta = kThreads / 16;

struct AppendArgs {
    const void* src[2];      // k_new, v_new (nullptr = skip)
    uint8_t* mant[2];
    uint8_t* exp8[2];
    const int32_t* perm[2];
    const int32_t* start_pos;
    int32_t batch, n_new, n_heads, max_seq;
    uint32_t* status;
};

// Eight consecutive channels of a row (no permutation): one or two 16-byte loads.
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p)), b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 a = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
// Eight channels picked by the permutation from the row parked in shared memory.
__device__ __forceinline__ void gather8(const float* row, const int (&idx)[8], float (&v)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = row[idx[i]];
}
__device__ __forceinline__ void gather8(const __nv_bfloat16* row, const int (&idx)[8], float (&v)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
        v[i] = __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(row)[idx[i]] << 16);
}

template <int P, int N, typename T>
__global__ void __launch_bounds__(kThreads) append_quant_pack(AppendArgs a) {
    constexpr int D = kHeadDim;
    constexpr int ROW_M = D * P / 8, ROW_E = D / N;
    constexpr int LANES_PER_BLOCK = N / 8;
    constexpr int QMAX = (1 << (P - 1)) - 1, EXC = 1 << (P - 1);
    constexpr float MAGIC = 12582912.f + (float)EXC;            // 1.5 * 2^23 + 2^(p-1)
    constexpr uint32_t MAGIC_BITS = 0x4B400000u;                // bits of 1.5 * 2^23: sum bits - this = field

    pdl_wait();
    pdl_trigger();
    const int which = blockIdx.y;
    const T* src = static_cast<const T*>(a.src[which]);
    if (!src) return;
    const int32_t* perm = a.perm[which];
    const int sub = threadIdx.x & 15;          // lane within the row
    const int tloc = threadIdx.x >> 4;         // token within the thread block's step
    // a permuted row is parked in shared memory by 16-byte loads that do not wait for the permutation, and picked
    // apart from there (the gather straight from global memory was a second round trip behind the index loads)
    __shared__ __align__(16) T srow[kTokPerCta][D];
    const int H = a.n_heads;
    const int64_t n_tok = (int64_t)a.batch * a.n_new;

    for (int64_t bt0 = (int64_t)blockIdx.x * kTokPerCta; bt0 < n_tok; bt0 += (int64_t)gridDim.x * kTokPerCta) {
        const int64_t bt = bt0 + tloc;
        const bool live = bt < n_tok;
        int b = 0, t = 0, sp = 0;
        bool fits = false;
        if (live) {
            b = (int)(bt / a.n_new);
            t = (int)(bt - (int64_t)b * a.n_new);
            sp = a.start_pos[b];
            fits = sp >= 0 && (int64_t)sp + a.n_new <= a.max_seq;
            if (!fits && t == 0 && sub == 0) raise_flag(a.status, KVBFP_FLAG_POSITION);   // sequence skipped whole
        }
        const T* tok = src + (live ? bt : 0) * H * D;
        for (int h = blockIdx.z; h < H; h += gridDim.z) {      // heads are also spread over thread blocks when tokens are few
            float v[8];
            if (perm) {      // Algorithm 1 step 3: slot j takes channel perm[h][j]
                const int4* pp = reinterpret_cast<const int4*>(perm + h * D + sub * 8);
                const int4 p0 = __ldg(pp), p1 = __ldg(pp + 1);
                const int idx[8] = {p0.x & (D - 1), p0.y & (D - 1), p0.z & (D - 1), p0.w & (D - 1),
                                    p1.x & (D - 1), p1.y & (D - 1), p1.z & (D - 1), p1.w & (D - 1)};
                constexpr int VEC = 8 * (int)sizeof(T) / 16;            // 16-byte pieces of the lane's eight channels
                const uint4* rp = reinterpret_cast<const uint4*>(tok + h * D + sub * 8);
                uint4 raw[VEC];
#pragma unroll
                for (int i = 0; i < VEC; ++i) raw[i] = __ldg(rp + i);
                __syncwarp();                                   // the row parked before this one has been read
#pragma unroll
                for (int i = 0; i < VEC; ++i) reinterpret_cast<uint4*>(&srow[tloc][sub * 8])[i] = raw[i];
                __syncwarp();
                gather8(&srow[tloc][0], idx, v);
            } else {
                load8(tok + h * D + sub * 8, v);
            }
            // shared exponent: the biased exponent field of the block's largest magnitude
            uint32_t amax = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) amax = max(amax, __float_as_uint(v[i]) & 0x7fffffffu);
#pragma unroll
            for (int off = 1; off < LANES_PER_BLOCK; off <<= 1)
                amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, off));
            int e8 = (int)(amax >> 23);
            if (e8 == 255) {            // Inf or NaN somewhere in the block
                if (live) raise_flag(a.status, KVBFP_FLAG_NONFINITE);
                e8 = 254;
            }
            // t = x * 2^(127 - e8 + p - 2) through two exact power-of-two factors; the second multiply is fused
            // with the rounding add, and the clamp to +-(2^(p-1) - 1) acts on the rounded sum
            const int k = 127 - e8 + (P - 2);
            const int k1 = k >> 1, k2 = k - k1;
            const float s1 = pow2i(k1), s2 = pow2i(k2);
            uint32_t f[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float r = fmaf(v[i] * s1, s2, MAGIC);                          // to nearest, ties to even
                r = fminf(fmaxf(r, MAGIC - (float)QMAX), MAGIC + (float)QMAX);  // NaN falls to the lower bound
                f[i] = __float_as_uint(r);
            }
            if (!live || !fits) continue;
            const int64_t pos = ((int64_t)b * H + h) * a.max_seq + sp + t;
            uint8_t* mrow = a.mant[which] + pos * ROW_M;
            if (P == 4) {
                // sum of (bits_i - MAGIC_BITS) * 16^i, with the constant part taken off once (arithmetic mod 2^32)
                uint32_t w = f[7];
#pragma unroll
                for (int i = 6; i >= 0; --i) w = w * 16u + f[i];
                reinterpret_cast<uint32_t*>(mrow)[sub] = w - MAGIC_BITS * 0x11111111u;
            } else if (P == 6) {
                uint64_t w = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) w |= (uint64_t)((f[i] - MAGIC_BITS) & 0x3fu) << (6 * i);
                uint16_t* o = reinterpret_cast<uint16_t*>(mrow + sub * 6);
                o[0] = (uint16_t)w;
                o[1] = (uint16_t)(w >> 16);
                o[2] = (uint16_t)(w >> 32);
            } else {
                uint32_t lo = 0, hi = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    lo |= ((f[i] - MAGIC_BITS) & 0xffu) << (8 * i);
                    hi |= ((f[i + 4] - MAGIC_BITS) & 0xffu) << (8 * i);
                }
                reinterpret_cast<uint2*>(mrow)[sub] = make_uint2(lo, hi);
            }
            if ((sub % LANES_PER_BLOCK) == 0) a.exp8[which][pos * ROW_E + sub / LANES_PER_BLOCK] = (uint8_t)e8;
        }
    }
}

// ---- runs of tokens (prefill): rows staged through shared memory ----------------------------------------------
//
// A thread block keeps one (sequence, head) and walks token tiles, so all row arithmetic is done once per block
// and the eight source channels of a lane (Algorithm 1 step 3) are fixed shared-memory addresses.  A warp owns two
// token rows per tile and a ring of four stages: every lane sends its part of the row straight to shared memory
// with asynchronous 16-byte copies, several tiles ahead of the cast, and waits on its own copy groups.
//
// bf16 rows with 4- or 6-bit fields are cast on pairs of bf16 numbers: everything the cast does to a bf16 number
// stays inside bf16 -- the two power-of-two factors are exact, and 192 + 2^(p-1) + M with |M| <= 2^(p-1) lies in
// [128, 256], where bf16 has unit spacing, so the fused multiply-add rounds to nearest-even exactly as the fp32
// form does, and the field is the sum's bits minus the bits of 192.  The other formats take the fp32 form.
__device__ __forceinline__ uint32_t bf2_max(uint32_t a, uint32_t b) {       // a NaN loses against a number
    uint32_t d; asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b)); return d;
}
__device__ __forceinline__ uint32_t bf2_min(uint32_t a, uint32_t b) {
    uint32_t d; asm("min.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b)); return d;
}
__device__ __forceinline__ uint32_t bf2_max_nan(uint32_t a, uint32_t b) {   // a NaN wins (comes out as 0x7fff)
    uint32_t d; asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b)); return d;
}
template <int OFF>
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr) {
    uint32_t v; asm volatile("ld.shared.u16 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(OFF) : "memory"); return v;
}
template <int OFF>
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v; asm volatile("ld.shared.b32 %0, [%1+%2];" : "=r"(v) : "r"(addr), "n"(OFF) : "memory"); return v;
}
template <int OFF>
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
    uint4 c;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4+%5];" : "=r"(c.x), "=r"(c.y), "=r"(c.z), "=r"(c.w)
                 : "r"(addr), "n"(OFF) : "memory");
    return c;
}

constexpr int kRing = 4;                       // stages per warp

template <int P, int N, typename T>
__global__ void __launch_bounds__(kThreads) append_rows(AppendArgs a, int chunks) {
    constexpr int D = kHeadDim, kWarps = kThreads / 32;
    constexpr bool BF16 = sizeof(T) == 2;
    constexpr bool PACKED = BF16 && P != 8;
    constexpr int ROW_IN = D * (int)sizeof(T);                    // 256 or 512 bytes
    constexpr int ROW_B = ROW_IN + 64;      // the second row sits 16 banks off the first: both lane groups read the
                                            // same channel numbers at the same time
    constexpr int STAGE_BYTES = 2 * ROW_IN + 128;
    constexpr int LANE_IN = 8 * (int)sizeof(T);                   // the lane's own 16 or 32 bytes of a row
    constexpr int ROW_M = D * P / 8, ROW_E = D / N;
    constexpr int LANES_PER_BLOCK = N / 8;
    constexpr int EXC = 1 << (P - 1), QMAX = EXC - 1;
    __shared__ __align__(128) uint8_t ring[kWarps * kRing * STAGE_BYTES];

    pdl_wait();
    pdl_trigger();
    const int which = blockIdx.y;
    const T* src = static_cast<const T*>(which ? a.src[1] : a.src[0]);
    if (!src) return;
    const int32_t* perm = which ? a.perm[1] : a.perm[0];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane & 15, grp = lane >> 4;
    const int H = a.n_heads;
    // the thread block's head (fastest: blocks that run together read the heads of the same tokens), sequence
    // and first tile; everything that follows from these is the same in all its threads
    const int h = blockIdx.x % H;
    const int b = (blockIdx.x / H) % a.batch;
    const int chunk = blockIdx.x / (H * a.batch);
    const int sp = a.start_pos[b];
    if (sp < 0 || (int64_t)sp + a.n_new > a.max_seq) {            // sequence skipped whole
        if (threadIdx.x == 0 && chunk == 0) raise_flag(a.status, KVBFP_FLAG_POSITION);
        return;
    }
    const int t_first = chunk * kTokPerCta + 2 * warp;            // the warp's first row of its first tile
    const int t_step = chunks * kTokPerCta;
    const int64_t pos0 = ((int64_t)b * H + h) * a.max_seq + sp + t_first + grp;
    uint8_t* mrow = (which ? a.mant[1] : a.mant[0]) + pos0 * ROW_M + sub * P;       // eight fields of P bits = P bytes per lane
    uint8_t* erow = (which ? a.exp8[1] : a.exp8[0]) + pos0 * ROW_E + sub / LANES_PER_BLOCK;

    const uint32_t my_row = smem_u32(ring) + warp * (kRing * STAGE_BYTES) + grp * ROW_B;

    // ---- copies: the lane's bytes of its group's row, one group of copies per tile (empty once the rows end,
    // so that "all but the newest kRing - 1 groups have landed" always means the stage about to be read)
    const uint4* p_in = reinterpret_cast<const uint4*>(src + (((int64_t)b * a.n_new + t_first + grp) * H + h) * D + sub * 8);
    const int64_t p_in_step = (int64_t)t_step * H * (ROW_IN / 16);
    int p_t = t_first + grp;
    auto issue_next = [&](int stage) {
        if (p_t < a.n_new) {
            const uint32_t dst = my_row + sub * LANE_IN + stage * STAGE_BYTES;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(p_in) : "memory");
            if (!BF16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 16), "l"(p_in + 1) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        p_t += t_step;
        p_in += p_in_step;
    };
#pragma unroll
    for (int s = 0; s < kRing; ++s) issue_next(s);

    // where the lane's eight slots find their channels in the staged row; without a permutation the lane keeps
    // its own bytes
    uint32_t at[8];
    if (perm) {
        const int4* pp = reinterpret_cast<const int4*>(perm + h * D + sub * 8);
        const int4 p0 = __ldg(pp), p1 = __ldg(pp + 1);
        const int idx[8] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) at[i] = my_row + (int)sizeof(T) * (idx[i] & (D - 1));
    }

    int t = t_first;                 // row of lane group 0; group 1 has t + 1
    auto cast_stage = [&](auto stage_c) {
        constexpr int OFF = decltype(stage_c)::value * STAGE_BYTES;
        asm volatile("cp.async.wait_group %0;" ::"n"(kRing - 1) : "memory");
        __syncwarp();                                  // the other lanes' parts of the rows are in place too
        const bool live = t + grp < a.n_new;
        int e8;
        uint32_t f[PACKED ? 4 : 8];     // the fields, still above their base: bf16 pairs or fp32 sums
        if constexpr (PACKED) {
            // P = 4 pairs slot j with slot j + 4 (their fields are 16 bits apart in the packed word), P = 6 pairs
            // neighbours
            if (perm) {
                uint32_t e[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) e[i] = lds_u16<OFF>(at[i]);
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    f[j] = P == 4 ? __byte_perm(e[j], e[j + 4], 0x5410) : __byte_perm(e[2 * j], e[2 * j + 1], 0x5410);
            } else {
                const uint4 c = lds_v4<OFF>(my_row + sub * LANE_IN);
                if (P == 4) {
                    f[0] = __byte_perm(c.x, c.z, 0x5410); f[1] = __byte_perm(c.x, c.z, 0x7632);
                    f[2] = __byte_perm(c.y, c.w, 0x5410); f[3] = __byte_perm(c.y, c.w, 0x7632);
                } else {
                    f[0] = c.x; f[1] = c.y; f[2] = c.z; f[3] = c.w;
                }
            }
            __syncwarp();                                  // every lane holds its part: the stage can be refilled
            issue_next(decltype(stage_c)::value);
            // shared exponent: the exponent field of the block's largest magnitude
            uint32_t m2 = bf2_max_nan(bf2_max_nan(f[0] & 0x7fff7fffu, f[1] & 0x7fff7fffu),
                                      bf2_max_nan(f[2] & 0x7fff7fffu, f[3] & 0x7fff7fffu));
#pragma unroll
            for (int off = 1; off < LANES_PER_BLOCK; off <<= 1) m2 = bf2_max_nan(m2, __shfl_xor_sync(0xffffffffu, m2, off));
            e8 = (int)(max(m2 & 0xffffu, m2 >> 16) >> 7);
        } else {
            if (perm) {
#pragma unroll
                for (int i = 0; i < 8; ++i) f[i] = BF16 ? lds_u16<OFF>(at[i]) << 16 : lds_u32<OFF>(at[i]);
            } else if (BF16) {
                const uint4 c = lds_v4<OFF>(my_row + sub * LANE_IN);
                const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) { f[2 * i] = w[i] << 16; f[2 * i + 1] = w[i] & 0xffff0000u; }
            } else {
                const uint4 c0 = lds_v4<OFF>(my_row + sub * LANE_IN), c1 = lds_v4<OFF + 16>(my_row + sub * LANE_IN);
                f[0] = c0.x; f[1] = c0.y; f[2] = c0.z; f[3] = c0.w; f[4] = c1.x; f[5] = c1.y; f[6] = c1.z; f[7] = c1.w;
            }
            __syncwarp();
            issue_next(decltype(stage_c)::value);
            uint32_t amax = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) amax = max(amax, f[i] & 0x7fffffffu);
#pragma unroll
            for (int off = 1; off < LANES_PER_BLOCK; off <<= 1) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, off));
            e8 = (int)(amax >> 23);
        }
        if (e8 == 255) {            // Inf or NaN somewhere in the block
            if (live) raise_flag(a.status, KVBFP_FLAG_NONFINITE);
            e8 = 254;
        }
        // x * 2^(127 - e8 + p - 2) through two exact power-of-two factors, the second one fused with the rounding
        // add (to nearest, ties to even); the clamp acts on the rounded sum; NaN falls to the lower bound
        const int k = 127 - e8 + (P - 2);
        const int k1 = k >> 1, k2 = k - k1;
        if constexpr (PACKED) {
            constexpr uint32_t BASE = 0x43404340u;                       // bf16 192.0 twice
            constexpr uint32_t MAGIC = BASE + EXC * 0x10001u;            // 192 + 2^(p-1)
            constexpr uint32_t LO = MAGIC - QMAX * 0x10001u, HI = MAGIC + QMAX * 0x10001u;
            const uint32_t s1 = ((uint32_t)(k1 + 127) << 7) * 0x10001u, s2 = ((uint32_t)(k2 + 127) << 7) * 0x10001u;
#pragma unroll
            for (int j = 0; j < 4; ++j) f[j] = bf2_min(bf2_max(fma_bf16x2(mul_bf16x2(f[j], s1), s2, MAGIC), LO), HI);
            if (live) {
                if (P == 4) {
                    // sum of (bits_j - BASE) * 16^j, the constant part taken off once (arithmetic mod 2^32)
                    const uint32_t o = ((f[3] * 16u + f[2]) * 16u + f[1]) * 16u + f[0];
                    *reinterpret_cast<uint32_t*>(mrow) = o - BASE * 0x1111u;
                } else {
                    uint32_t t12[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t c = f[j] - BASE;
                        t12[j] = (c | (c >> 10)) & 0xfffu;
                    }
                    const uint32_t lo = t12[0] + (t12[1] << 12) + (t12[2] << 24);
                    const uint32_t hi = (t12[2] >> 8) + (t12[3] << 4);
                    uint16_t* o = reinterpret_cast<uint16_t*>(mrow);
                    o[0] = (uint16_t)lo;
                    o[1] = (uint16_t)(lo >> 16);
                    o[2] = (uint16_t)hi;
                }
            }
        } else {
            constexpr float MAGIC = 12582912.f + (float)EXC;            // 1.5 * 2^23 + 2^(p-1)
            constexpr uint32_t MAGIC_BITS = 0x4B400000u;                // bits of 1.5 * 2^23: sum bits - this = field
            const float s1 = pow2i(k1), s2 = pow2i(k2);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float r = fmaf(__uint_as_float(f[i]) * s1, s2, MAGIC);
                r = fminf(fmaxf(r, MAGIC - (float)QMAX), MAGIC + (float)QMAX);
                f[i] = __float_as_uint(r);
            }
            if (live) {
                if (P == 4) {
                    uint32_t w = f[7];
#pragma unroll
                    for (int i = 6; i >= 0; --i) w = w * 16u + f[i];
                    *reinterpret_cast<uint32_t*>(mrow) = w - MAGIC_BITS * 0x11111111u;
                } else if (P == 6) {
                    uint64_t w = 0;
#pragma unroll
                    for (int i = 0; i < 8; ++i) w |= (uint64_t)((f[i] - MAGIC_BITS) & 0x3fu) << (6 * i);
                    uint16_t* o = reinterpret_cast<uint16_t*>(mrow);
                    o[0] = (uint16_t)w;
                    o[1] = (uint16_t)(w >> 16);
                    o[2] = (uint16_t)(w >> 32);
                } else {
                    uint32_t lo = 0, hi = 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        lo |= ((f[i] - MAGIC_BITS) & 0xffu) << (8 * i);
                        hi |= ((f[i + 4] - MAGIC_BITS) & 0xffu) << (8 * i);
                    }
                    *reinterpret_cast<uint2*>(mrow) = make_uint2(lo, hi);
                }
            }
        }
        if (live && (sub % LANES_PER_BLOCK) == 0) *erow = (uint8_t)e8;
        t += t_step;
        mrow += (int64_t)t_step * ROW_M;
        erow += (int64_t)t_step * ROW_E;
    };
    // the rows of a warp only grow: once its first row lies beyond the sequence it is done
    while (t < a.n_new) {
        cast_stage(std::integral_constant<int, 0>{});
        if (t >= a.n_new) break;
        cast_stage(std::integral_constant<int, 1>{});
        if (t >= a.n_new) break;
        cast_stage(std::integral_constant<int, 2>{});
        if (t >= a.n_new) break;
        cast_stage(std::integral_constant<int, 3>{});
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// Runs of at least one tile per sequence take the staged kernel; single tokens (the decode step) stay with the
// general one, whose lane groups each find their own sequence.
template <int P, int N, typename T>
kvbfp_status launch_rows(const AppendArgs& a, cudaStream_t s) {
    const int tiles = (a.n_new + kTokPerCta - 1) / kTokPerCta;            // per sequence
    int n_sm = 0;
    const kvbfp_status st = sm_count(&n_sm);
    if (st != KVBFP_OK) return st;
    // thread blocks over the sides that have rows: one resident wave where blocks of one (sequence, head) fill at
    // least 15/16 of it, else about eight waves of shorter blocks, which even out; no block shorter than 16 tiles
    static std::atomic<int> per_sm{0};              // (two host threads asking at once store the same number)
    int bps = per_sm.load(std::memory_order_relaxed);
    if (bps == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, append_rows<P, N, T>, kThreads, 0) != cudaSuccess || bps < 1)
            return KVBFP_ERR_CUDA;
        per_sm.store(bps, std::memory_order_relaxed);
    }
    const int sides = (a.src[0] ? 1 : 0) + (a.src[1] ? 1 : 0);
    const int64_t per_chunk = (int64_t)a.n_heads * a.batch * sides;
    const int64_t resident = (int64_t)n_sm * bps;
    int64_t chunks = resident / per_chunk;                              // one wave, if blocks of equal length fill it
    if (chunks * per_chunk * 16 < resident * 15 || chunks > tiles / 16) {
        chunks = (8 * resident + per_chunk - 1) / per_chunk;
        if (chunks > tiles / 16) chunks = tiles / 16;
    }
    if (chunks < 1) chunks = 1;
    if (per_chunk * chunks > 0x7fffffffLL) return KVBFP_ERR_UNSUPPORTED;
    dim3 grid((unsigned)(per_chunk / sides * chunks), 2, 1);
    (void)launch_pdl(append_rows<P, N, T>, grid, dim3(kThreads), 0, s, a, (int)chunks);
    KVBFP_LAUNCH_CHECK("append_rows");
    return KVBFP_OK;
}

template <int P, int N, typename T>
kvbfp_status launch(const AppendArgs& a, int64_t n_rows, cudaStream_t s) {
    if (a.n_new >= kTokPerCta && a.n_new <= (1 << 30)) return launch_rows<P, N, T>(a, s);
    const int64_t n_tok = (int64_t)a.batch * a.n_new;
    const int64_t want = (n_tok + kTokPerCta - 1) / kTokPerCta;
    int n_sm = 0;
    const kvbfp_status st = sm_count(&n_sm);
    if (st != KVBFP_OK) return st;
    const int gx = (int)(want < n_sm * 16 ? want : n_sm * 16);
    (void)n_rows;
    int hs = (int)((n_sm * 4 + gx - 1) / gx);             // enough thread blocks to fill the machine
    if (hs > a.n_heads) hs = a.n_heads;
    if (hs < 1) hs = 1;
    dim3 grid(gx, 2, hs);
    (void)launch_pdl(append_quant_pack<P, N, T>, grid, dim3(kThreads), 0, s, a);
    KVBFP_LAUNCH_CHECK("append_quant_pack");
    return KVBFP_OK;
}

template <int P, typename T>
kvbfp_status launch_n(int n, const AppendArgs& a, int64_t n_rows, cudaStream_t s) {
    switch (n) {
        case 16: return launch<P, 16, T>(a, n_rows, s);
        case 32: return launch<P, 32, T>(a, n_rows, s);
        case 64: return launch<P, 64, T>(a, n_rows, s);
        case 128: return launch<P, 128, T>(a, n_rows, s);
    }
    return KVBFP_ERR_UNSUPPORTED;
}

template <typename T>
kvbfp_status launch_p(int p, int n, const AppendArgs& a, int64_t n_rows, cudaStream_t s) {
    switch (p) {
        case 4: return launch_n<4, T>(n, a, n_rows, s);
        case 6: return launch_n<6, T>(n, a, n_rows, s);
        case 8: return launch_n<8, T>(n, a, n_rows, s);
    }
    return KVBFP_ERR_UNSUPPORTED;
}

}  // namespace
}  // namespace kvbfp

extern "C" kvbfp_status kvbfp_append(const kvbfp_cache* cache, const void* k_new, const void* v_new,
                                     kvbfp_dtype dt, int32_t n_new, const int32_t* start_pos,
                                     const int32_t* perm_k, const int32_t* perm_v, void* stream) {
    using namespace kvbfp;
    if (!cache) return KVBFP_ERR_INVALID_ARG;
    kvbfp_status st = check_format(&cache->fmt);
    if (st != KVBFP_OK) return st;
    if (!start_pos || n_new < 0 || (!k_new && !v_new)) return KVBFP_ERR_INVALID_ARG;
    if (dt != KVBFP_F32 && dt != KVBFP_BF16) return KVBFP_ERR_INVALID_ARG;
    if (k_new && (!cache->k_mant || !cache->k_exp)) return KVBFP_ERR_INVALID_ARG;
    if (v_new && (!cache->v_mant || !cache->v_exp)) return KVBFP_ERR_INVALID_ARG;
    if (n_new > cache->fmt.max_seq) return KVBFP_ERR_CAPACITY;
    const void* ptrs[] = {k_new, v_new, cache->k_mant, cache->k_exp, cache->v_mant, cache->v_exp, perm_k, perm_v};
    for (const void* p : ptrs)
        if (p && !aligned16(p)) return KVBFP_ERR_ALIGNMENT;
    if (n_new == 0) return KVBFP_OK;

    AppendArgs a;
    a.src[0] = k_new; a.src[1] = v_new;
    a.mant[0] = cache->k_mant; a.mant[1] = cache->v_mant;
    a.exp8[0] = cache->k_exp; a.exp8[1] = cache->v_exp;
    a.perm[0] = perm_k; a.perm[1] = perm_v;
    a.start_pos = start_pos;
    a.batch = cache->fmt.batch; a.n_new = n_new; a.n_heads = cache->fmt.n_kv_heads;
    a.max_seq = cache->fmt.max_seq;
    st = status_word(&a.status);
    if (st != KVBFP_OK) return st;
    const int64_t n_rows = (int64_t)a.batch * n_new * a.n_heads;
    if (n_rows >= ((int64_t)1 << 31)) return KVBFP_ERR_UNSUPPORTED;     // 2^31 rows of 128 channels would be half a terabyte
    cudaStream_t s = (cudaStream_t)stream;
    if (dt == KVBFP_F32) return launch_p<float>(cache->fmt.mant_bits, cache->fmt.block, a, n_rows, s);
    return launch_p<__nv_bfloat16>(cache->fmt.mant_bits, cache->fmt.block, a, n_rows, s);
}
