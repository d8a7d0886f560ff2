// Eq. (1) of the paper: stored mantissas times 2^e back to numbers, optionally scattered to the
// original channel order.  One thread per (token, group of eight slots).
#include "common.cuh"

namespace kvbfp {
namespace {

template <typename T>
__device__ __forceinline__ T from_float(float x);
template <>
__device__ __forceinline__ float from_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) {
    // M * 2^k with |M| <= 127 has at most 7 significant bits: truncation is exact
    return __ushort_as_bfloat16((unsigned short)(__float_as_uint(x) >> 16));
}

template <typename T>
__global__ void __launch_bounds__(256) dequant_rows(const uint8_t* __restrict__ mant,
                                                    const uint8_t* __restrict__ exp8, int64_t row0,
                                                    int n_tok, int p, int n, const int32_t* __restrict__ perm,
                                                    T* __restrict__ out) {
    constexpr int D = kHeadDim;
    const int row_m = D * p / 8, row_e = D / n;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)n_tok * (D / 8)) return;
    const int t = (int)(i / (D / 8)), grp = (int)(i % (D / 8));
    const uint8_t* mrow = mant + (row0 + t) * row_m;
    const float w = unit_weight(exp8[(row0 + t) * row_e + (grp * 8) / n], p);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int slot = grp * 8 + j;
        const int m = extract_field(mrow, slot * p, p);
        const int c = perm ? (perm[slot] & (D - 1)) : slot;
        out[(int64_t)t * D + c] = from_float<T>((float)m * w);
    }
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
    if (b < 0 || b >= fmt->batch || h < 0 || h >= fmt->n_kv_heads || t0 < 0 || n_tok < 0) return KVBFP_ERR_INVALID_ARG;
    if ((int64_t)t0 + n_tok > fmt->max_seq) return KVBFP_ERR_CAPACITY;
    if (out_dt != KVBFP_F32 && out_dt != KVBFP_BF16) return KVBFP_ERR_INVALID_ARG;
    if (!aligned16(mant) || !aligned16(exp8) || !aligned16(out) || (perm && !aligned16(perm))) return KVBFP_ERR_ALIGNMENT;
    if (n_tok == 0) return KVBFP_OK;
    const int64_t row0 = ((int64_t)b * fmt->n_kv_heads + h) * fmt->max_seq + t0;
    const int64_t n_thr = (int64_t)n_tok * (kHeadDim / 8);
    const int grid = (int)((n_thr + 255) / 256);
    const int32_t* hp = perm ? perm + (int64_t)h * kHeadDim : nullptr;
    cudaStream_t s = (cudaStream_t)stream;
    if (out_dt == KVBFP_F32)
        dequant_rows<float><<<grid, 256, 0, s>>>(mant, exp8, row0, n_tok, fmt->mant_bits, fmt->block, hp, (float*)out);
    else
        dequant_rows<__nv_bfloat16><<<grid, 256, 0, s>>>(mant, exp8, row0, n_tok, fmt->mant_bits, fmt->block, hp,
                                                         (__nv_bfloat16*)out);
    KVBFP_LAUNCH_CHECK("dequant_rows");
    return KVBFP_OK;
}
