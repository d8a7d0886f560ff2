// Eq. (1) of the paper: stored mantissas times 2^e back to numbers, optionally in the original channel order.
//
// A thread block takes a tile of 64 token rows of one (batch, head): the packed rows are contiguous in their
// plane and come in with 16-byte loads into shared memory, the exponent bytes as the fp32 weights 2^(e - 127 - (p-2))
// they stand for (worked out once per block of a row, not once per element); every thread then owns four output channels of a row
// (so a warp writes one row with one 16-byte store per lane, fully coalesced) and picks the fields of those
// channels out of the staged row -- with a permutation that is a gather through the inverse permutation, which
// the block builds once in shared memory.  One launch covers any rectangle (sequences x heads x tokens).
#include "common.cuh"

namespace kvbfp {
namespace {

constexpr int kTileTok = 64;
constexpr int kThreads = 256;

template <typename T>
__device__ __forceinline__ void store4(T* dst, float a, float b, float c, float d);
template <>
__device__ __forceinline__ void store4<float>(float* dst, float a, float b, float c, float d) {
    *reinterpret_cast<float4*>(dst) = make_float4(a, b, c, d);
}
template <>
__device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* dst, float a, float b, float c, float d) {
    // M * 2^k with |M| <= 127 has at most 7 significant bits: truncation is exact
    const uint32_t lo = (__float_as_uint(a) >> 16) | (__float_as_uint(b) & 0xffff0000u);
    const uint32_t hi = (__float_as_uint(c) >> 16) | (__float_as_uint(d) & 0xffff0000u);
    *reinterpret_cast<uint2*>(dst) = make_uint2(lo, hi);
}

struct DequantArgs {
    const uint8_t *mant, *exp8;
    const int32_t* perm;          // [n_kv_heads, head_dim] or nullptr
    void* out;
    int n_kv_heads, max_seq, block_log2;
    int b0, nb, h0, nh, t0, n_tok;
    int tiles;                    // tiles per (batch, head)
    int64_t out_seq_stride, out_tok_stride, out_head_stride;      // in elements
};

template <int P, typename T, bool PERM>
__global__ void __launch_bounds__(kThreads) dequant_tile(DequantArgs a) {
    constexpr int D = kHeadDim, ROW_M = D * P / 8;
    __shared__ __align__(16) uint8_t smant[kTileTok * ROW_M + 16];      // (+16: the two-byte read of the last field)
    __shared__ float sw[kTileTok * 8];                                   // weight of one mantissa unit per (row, block)
    __shared__ int sinv[D];
    const int tid = threadIdx.x, lane = tid & 31, sub = tid >> 5;
    const int tile = blockIdx.x % a.tiles;
    const int pair = blockIdx.x / a.tiles;
    const int hh = pair % a.nh, bb = pair / a.nh;
    const int h = a.h0 + hh, b = a.b0 + bb;
    const int row_e = D >> a.block_log2;
    const int tok0 = tile * kTileTok;
    const int rows = min(kTileTok, a.n_tok - tok0);
    const int64_t row0 = ((int64_t)b * a.n_kv_heads + h) * a.max_seq + a.t0 + tok0;

    const uint4* src = reinterpret_cast<const uint4*>(a.mant + row0 * ROW_M);
    for (int i = tid; i < rows * (ROW_M / 16); i += kThreads) reinterpret_cast<uint4*>(smant)[i] = __ldg(src + i);
    const uint8_t* esrc = a.exp8 + row0 * row_e;
    for (int i = tid; i < rows * row_e; i += kThreads) sw[i] = unit_weight(__ldg(esrc + i), P);
    if (PERM && tid < D) sinv[a.perm[h * D + tid] & (D - 1)] = tid;
    __syncthreads();

    // the four channels of this thread: where their fields sit in a staged row
    int byte[4], sh[4], eb[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int c = 4 * lane + j;
        const int slot = PERM ? sinv[c] : c;
        byte[j] = (slot * P) >> 3;
        sh[j] = (slot * P) & 7;
        eb[j] = slot >> a.block_log2;
    }
    T* out = static_cast<T*>(a.out) + bb * a.out_seq_stride + hh * a.out_head_stride + 4 * lane;
    for (int r = sub; r < rows; r += kThreads / 32) {
        const uint8_t* mrow = smant + r * ROW_M;
        float v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t w = mrow[byte[j]];
            if (P == 6) w |= (uint32_t)mrow[byte[j] + 1] << 8;        // a 6-bit field may straddle two bytes
            const int m = (int)((w >> sh[j]) & ((1u << P) - 1u)) - (1 << (P - 1));
            v[j] = (float)m * sw[r * row_e + eb[j]];
        }
        store4<T>(out + (int64_t)(tok0 + r) * a.out_tok_stride, v[0], v[1], v[2], v[3]);
    }
}

template <int P, typename T>
void launch2(const DequantArgs& a, int grid, cudaStream_t s) {
    if (a.perm) dequant_tile<P, T, true><<<grid, kThreads, 0, s>>>(a);
    else dequant_tile<P, T, false><<<grid, kThreads, 0, s>>>(a);
}
template <typename T>
void launch1(const DequantArgs& a, int p, int grid, cudaStream_t s) {
    if (p == 4) launch2<4, T>(a, grid, s);
    else if (p == 6) launch2<6, T>(a, grid, s);
    else launch2<8, T>(a, grid, s);
}

}  // namespace
}  // namespace kvbfp

extern "C" kvbfp_status kvbfp_dequant(const kvbfp_format* fmt, const uint8_t* mant, const uint8_t* exp8,
                                      int32_t b, int32_t h, int32_t t0, int32_t n_tok,
                                      const int32_t* perm, void* out, kvbfp_dtype out_dt, void* stream) {
    using namespace kvbfp;
    kvbfp_status st = check_format(fmt);
    if (st != KVBFP_OK) return st;
    if (!mant || !exp8 || !out) return KVBFP_ERR_INVALID_ARG;
    if (b < -1 || b >= fmt->batch || h < -1 || h >= fmt->n_kv_heads || t0 < 0 || n_tok < 0) return KVBFP_ERR_INVALID_ARG;
    if ((int64_t)t0 + n_tok > fmt->max_seq) return KVBFP_ERR_CAPACITY;
    if (out_dt != KVBFP_F32 && out_dt != KVBFP_BF16) return KVBFP_ERR_INVALID_ARG;
    if (!aligned16(mant) || !aligned16(exp8) || !aligned16(out) || (perm && !aligned16(perm))) return KVBFP_ERR_ALIGNMENT;
    if (n_tok == 0) return KVBFP_OK;
    DequantArgs a;
    a.mant = mant; a.exp8 = exp8; a.perm = perm; a.out = out;
    a.n_kv_heads = fmt->n_kv_heads; a.max_seq = fmt->max_seq;
    a.block_log2 = fmt->block == 16 ? 4 : fmt->block == 32 ? 5 : fmt->block == 64 ? 6 : 7;
    a.b0 = b < 0 ? 0 : b; a.nb = b < 0 ? fmt->batch : 1;
    a.h0 = h < 0 ? 0 : h; a.nh = h < 0 ? fmt->n_kv_heads : 1;
    a.t0 = t0; a.n_tok = n_tok;
    a.tiles = (n_tok + kTileTok - 1) / kTileTok;
    a.out_head_stride = kHeadDim;
    a.out_tok_stride = (int64_t)a.nh * kHeadDim;
    a.out_seq_stride = (int64_t)n_tok * a.out_tok_stride;
    const int64_t grid = (int64_t)a.tiles * a.nb * a.nh;
    if (grid > 0x7fffffffLL) return KVBFP_ERR_UNSUPPORTED;
    cudaStream_t s = (cudaStream_t)stream;
    if (out_dt == KVBFP_F32) launch1<float>(a, fmt->mant_bits, (int)grid, s);
    else launch1<__nv_bfloat16>(a, fmt->mant_bits, (int)grid, s);
    KVBFP_LAUNCH_CHECK("dequant_tile");
    return KVBFP_OK;
}
