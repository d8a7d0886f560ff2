// Rotary embeddings in the permuted channel order: Eq. (4) of the paper (Sec. II-D) in table form, and
// Algorithm 1 step 5 (Sec. III), which permutes the frequency vector, the partner indices and the sine
// signs so that a row that is already in stored (slot) order can be rotated without undoing K-sort.
#include <math.h>

#include "common.cuh"

namespace kvbfp {
namespace {

// One thread per (head, slot): slot j holds channel c = perm[j]; its partner channel i[c] sits in slot
// inv_perm[i[c]].  Interleaved layout (Eq. (4)): pairs (2i, 2i+1); half-split layout (the footnote to
// Sec. III): pairs (i, i + d/2).  theta_i = base^(-2i/d).
__global__ void __launch_bounds__(kHeadDim) rope_tables(const int32_t* __restrict__ perm, const int32_t* __restrict__ inv_perm,
                                                        int d, double base, int half_split, double* __restrict__ theta,
                                                        int32_t* __restrict__ partner, float* __restrict__ sign) {
    const int h = blockIdx.x, j = threadIdx.x;
    const int c = perm ? (perm[h * d + j] & (d - 1)) : j;
    const int half = d / 2;
    const int pair = half_split ? (c % half) : (c / 2);
    int pc;
    float sg;
    if (half_split) { pc = c < half ? c + half : c - half; sg = c < half ? -1.f : 1.f; }
    else { pc = (c & 1) ? c - 1 : c + 1; sg = (c & 1) ? 1.f : -1.f; }
    theta[h * d + j] = pow(base, -2.0 * (double)pair / (double)d);
    partner[h * d + j] = inv_perm ? (inv_perm[h * d + pc] & (d - 1)) : pc;
    sign[h * d + j] = sg;
}

template <typename T> __device__ __forceinline__ float ld(const T* p);
template <> __device__ __forceinline__ float ld<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void st(T* p, float v);
template <> __device__ __forceinline__ void st<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void st<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// y[j] = x[j] cos(m theta_j) + sign_j x[partner_j] sin(m theta_j).  The angle is formed and reduced to [-pi, pi]
// in fp64 (positions reach tens of thousands of radians, beyond what an fp32 product resolves); sine, cosine and
// the two products are fp32.  A thread keeps one (head, slot) and walks kRopeRows rows, so the tables are read once.
constexpr int kRopeRows = 32;
template <typename T>
__global__ void __launch_bounds__(kHeadDim) rope_apply(const T* __restrict__ x, const int32_t* __restrict__ pos, int64_t n_rows,
                                                       int n_heads, const double* __restrict__ theta,
                                                       const int32_t* __restrict__ partner, const float* __restrict__ sign,
                                                       T* __restrict__ y) {
    constexpr int D = kHeadDim;
    const int h = blockIdx.y, j = threadIdx.x;
    const double th = theta[h * D + j];
    const int pj = partner[h * D + j] & (D - 1);
    const float sg = sign[h * D + j];
    const int64_t r0 = (int64_t)blockIdx.x * kRopeRows;
    const int64_t r1 = r0 + kRopeRows < n_rows ? r0 + kRopeRows : n_rows;
#pragma unroll 4
    for (int64_t row = r0; row < r1; ++row) {
        const T* xr = x + (row * n_heads + h) * D;
        float sn, cs;
        sincos_reduced((double)pos[row] * th, &sn, &cs);
        const float v = fmaf(ld<T>(xr + j), cs, sg * ld<T>(xr + pj) * sn);
        st<T>(y + (row * n_heads + h) * D + j, v);
    }
}

}  // namespace
}  // namespace kvbfp

extern "C" kvbfp_status kvbfp_rope_tables(const int32_t* perm, const int32_t* inv_perm, int32_t n_heads,
                                          int32_t head_dim, double base, int32_t half_split, double* theta_out,
                                          int32_t* partner_out, float* sign_out, void* stream) {
    using namespace kvbfp;
    if (!theta_out || !partner_out || !sign_out || n_heads < 1 || !(base > 1.0)) return KVBFP_ERR_INVALID_ARG;
    if ((perm == nullptr) != (inv_perm == nullptr)) return KVBFP_ERR_INVALID_ARG;
    if (head_dim != kHeadDim) return KVBFP_ERR_UNSUPPORTED;
    const void* ptrs[] = {perm, inv_perm, theta_out, partner_out, sign_out};
    for (const void* p : ptrs)
        if (p && !aligned16(p)) return KVBFP_ERR_ALIGNMENT;
    rope_tables<<<n_heads, kHeadDim, 0, (cudaStream_t)stream>>>(perm, inv_perm, head_dim, base, half_split ? 1 : 0,
                                                               theta_out, partner_out, sign_out);
    KVBFP_LAUNCH_CHECK("rope_tables");
    return KVBFP_OK;
}

extern "C" kvbfp_status kvbfp_rope_apply(const void* x, kvbfp_dtype dt, int64_t n_rows, int32_t n_heads,
                                         int32_t head_dim, const int32_t* positions, const double* theta,
                                         const int32_t* partner, const float* sign, void* y, void* stream) {
    using namespace kvbfp;
    if (!x || !y || x == y || !positions || !theta || !partner || !sign || n_rows < 0 || n_heads < 1)
        return KVBFP_ERR_INVALID_ARG;
    if (head_dim != kHeadDim || n_heads > 65535 || n_rows > 0x7fffffff) return KVBFP_ERR_UNSUPPORTED;
    if (dt != KVBFP_F32 && dt != KVBFP_BF16) return KVBFP_ERR_INVALID_ARG;
    const void* ptrs[] = {x, y, positions, theta, partner, sign};
    for (const void* p : ptrs)
        if (!aligned16(p)) return KVBFP_ERR_ALIGNMENT;
    if (n_rows == 0) return KVBFP_OK;
    dim3 grid((unsigned)((n_rows + kRopeRows - 1) / kRopeRows), (unsigned)n_heads);
    cudaStream_t s = (cudaStream_t)stream;
    if (dt == KVBFP_F32)
        rope_apply<float><<<grid, kHeadDim, 0, s>>>((const float*)x, positions, n_rows, n_heads, theta, partner, sign, (float*)y);
    else
        rope_apply<__nv_bfloat16><<<grid, kHeadDim, 0, s>>>((const __nv_bfloat16*)x, positions, n_rows, n_heads, theta, partner,
                                                            sign, (__nv_bfloat16*)y);
    KVBFP_LAUNCH_CHECK("rope_apply");
    return KVBFP_OK;
}
