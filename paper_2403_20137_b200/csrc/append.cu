// Cache write: permute, shared exponent, round, clamp, pack, store (Sec. II-B last paragraph,
// Sec. III par. 2 of the paper; Algorithm 1 step 3 applied at run time as a gather).
//
// Sixteen lanes own one (token, head) row of 128 channels, eight stored slots per lane; a thread block
// takes sixteen tokens per step and each 16-lane group walks the heads of its token, so no index has to
// be divided per row.  A block of n slots is held by n/8 neighbouring lanes; its largest magnitude is
// found with xor-shuffles on the IEEE bit patterns (integer compare = exact).  Rounding to nearest-even
// is one fused multiply-add with 1.5 * 2^23 + 2^(p-1): the integer M + 2^(p-1), which is the stored
// field, appears in the low bits of the sum.
#include "common.cuh"

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
// Eight channels picked by the permutation, straight from the row (it sits in L1 after the first touch).
__device__ __forceinline__ void gather8(const float* row, const int (&idx)[8], float (&v)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __ldg(row + idx[i]);
}
__device__ __forceinline__ void gather8(const __nv_bfloat16* row, const int (&idx)[8], float (&v)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
        v[i] = __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(row) + idx[i]) << 16);
}

template <int P, int N, typename T>
__global__ void __launch_bounds__(kThreads) append_quant_pack(AppendArgs a) {
    constexpr int D = kHeadDim;
    constexpr int ROW_M = D * P / 8, ROW_E = D / N;
    constexpr int LANES_PER_BLOCK = N / 8;
    constexpr int QMAX = (1 << (P - 1)) - 1, EXC = 1 << (P - 1);
    constexpr float MAGIC = 12582912.f + (float)EXC;            // 1.5 * 2^23 + 2^(p-1)
    constexpr uint32_t MAGIC_BITS = 0x4B400000u;                // bits of 1.5 * 2^23: sum bits - this = field

    const int which = blockIdx.y;
    const T* src = static_cast<const T*>(a.src[which]);
    if (!src) return;
    const int32_t* perm = a.perm[which];
    const int sub = threadIdx.x & 15;          // lane within the row
    const int tloc = threadIdx.x >> 4;         // token within the thread block's step
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
                gather8(tok + h * D, idx, v);
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

template <int P, int N, typename T>
kvbfp_status launch(const AppendArgs& a, int64_t n_rows, cudaStream_t s) {
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
    append_quant_pack<P, N, T><<<grid, kThreads, 0, s>>>(a);
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
