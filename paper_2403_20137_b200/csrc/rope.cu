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

// y[j] = x[j] cos(m theta_j) + sign_j x[partner_j] sin(m theta_j).  Angles are formed and reduced to [-pi, pi] in
// fp64 (positions reach tens of thousands of radians, beyond what an fp32 product resolves); sine, cosine and the
// products are fp32.
//
// A thread block keeps one head and walks tiles of kRopeTile rows, which it stages in shared memory with 16-byte
// loads, rotates in place and writes back with 16-byte stores.  Tables as kvbfp_rope_tables makes them pair the
// slots up (partner of partner = self, one frequency, opposite signs): the block lists the 64 pairs once, a thread
// owns a pair and half of the rows, and one sine/cosine serves both slots.  Where the positions of a tile count up
// by one (a run of tokens), the angle of row r is the tile's first angle plus r * theta: one exact sine/cosine per
// pair and tile, turned by the tabulated (cos, sin)(r * theta) with one complex product -- the same accuracy as a
// direct evaluation (no chain of products).  Other tiles evaluate every (row, pair) directly; tables that do not
// pair up take the slot-by-slot form.
constexpr int kRopeTile = 32;
constexpr int kRopeThreads = 128;

template <typename T> __device__ __forceinline__ float ld(const T* p);
template <> __device__ __forceinline__ float ld<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void st(T* p, float v);
template <> __device__ __forceinline__ void st<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void st<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename T>
__global__ void __launch_bounds__(kRopeThreads) rope_apply(const T* __restrict__ x, const int32_t* __restrict__ pos, int64_t n_rows,
                                                           int n_heads, const double* __restrict__ theta,
                                                           const int32_t* __restrict__ partner, const float* __restrict__ sign,
                                                           T* __restrict__ y, int n_tiles, int chunks) {
    constexpr int D = kHeadDim, HALF = D / 2;
    constexpr int VEC_ROW = D * (int)sizeof(T) / 16;            // 16-byte pieces of a row
    __shared__ __align__(16) T tile[kRopeTile * D];
    __shared__ float2 turn[kRopeTile][HALF];                    // (cos, sin)(r * theta) of pair i
    __shared__ int pair_a[HALF], pair_b[HALF];
    __shared__ int s_pos[kRopeTile];
    __shared__ int n_pairs;
    const int tid = threadIdx.x;
    const int h = blockIdx.x % n_heads, chunk = blockIdx.x / n_heads;

    // ---- the head's tables: do they pair the slots up?
    const int my_partner = partner[h * D + tid] & (D - 1);
    const float my_sign = sign[h * D + tid];
    const double my_theta = theta[h * D + tid];
    if (tid == 0) n_pairs = 0;
    const bool well = my_partner != tid && (partner[h * D + my_partner] & (D - 1)) == tid && sign[h * D + my_partner] == -my_sign &&
                      theta[h * D + my_partner] == my_theta && (my_sign == 1.f || my_sign == -1.f);
    const bool paired = __syncthreads_and(well);
    if (paired && my_sign < 0.f) {                              // the slot whose product with the sine is subtracted
        const int k = atomicAdd(&n_pairs, 1);
        pair_a[k] = tid;
        pair_b[k] = my_partner;
    }
    __syncthreads();
    const int pi = tid & (HALF - 1), half_rows = tid / HALF;    // pair, and which half of the rows
    int sa = 0, sb = 0;
    double th = 0.0;
    if (paired) {
        sa = pair_a[pi]; sb = pair_b[pi];
        th = theta[h * D + sa];
    }
    bool have_turn = false;                                     // the table is made when the first counting tile comes

    for (int t = chunk; t < n_tiles; t += chunks) {
        const int64_t row0 = (int64_t)t * kRopeTile;
        const int rows = (int)min((int64_t)kRopeTile, n_rows - row0);
        __syncthreads();                                        // the tile before this one has been written out
        for (int e = tid; e < rows * VEC_ROW; e += kRopeThreads) {
            const int r = e / VEC_ROW, v = e % VEC_ROW;
            reinterpret_cast<uint4*>(tile)[r * VEC_ROW + v] =
                __ldg(reinterpret_cast<const uint4*>(x + ((row0 + r) * n_heads + h) * D) + v);
        }
        if (tid < rows) s_pos[tid] = pos[row0 + tid];
        __syncthreads();
        const bool counting = __syncthreads_and(tid >= rows || s_pos[tid] == s_pos[0] + tid) && rows > 2;
        if (paired && counting && !have_turn) {
            for (int e = tid; e < kRopeTile * HALF; e += kRopeThreads) {
                const int r = e / HALF, i = e % HALF;
                float sn, cs;
                sincos_reduced((double)r * theta[h * D + pair_a[i]], &sn, &cs);
                turn[r][i] = make_float2(cs, sn);
            }
            have_turn = true;
            __syncthreads();
        }
        if (paired) {
            float c0 = 1.f, s0 = 0.f;
            if (counting) sincos_reduced((double)s_pos[0] * th, &s0, &c0);
            for (int r = half_rows; r < rows; r += kRopeThreads / HALF) {
                float cs, sn;
                if (counting) {
                    const float2 w = turn[r][pi];
                    cs = c0 * w.x - s0 * w.y;
                    sn = s0 * w.x + c0 * w.y;
                } else {
                    sincos_reduced((double)s_pos[r] * th, &sn, &cs);
                }
                const float xa = ld<T>(tile + r * D + sa), xb = ld<T>(tile + r * D + sb);
                st<T>(tile + r * D + sa, fmaf(xa, cs, -(xb * sn)));
                st<T>(tile + r * D + sb, fmaf(xb, cs, xa * sn));
            }
            __syncthreads();
            for (int e = tid; e < rows * VEC_ROW; e += kRopeThreads) {
                const int r = e / VEC_ROW, v = e % VEC_ROW;
                reinterpret_cast<uint4*>(y + ((row0 + r) * n_heads + h) * D)[v] = reinterpret_cast<const uint4*>(tile)[r * VEC_ROW + v];
            }
        } else {                                                // slot by slot, straight to the output
            for (int r = 0; r < rows; ++r) {
                float sn, cs;
                sincos_reduced((double)s_pos[r] * my_theta, &sn, &cs);
                const float v = fmaf(ld<T>(tile + r * D + tid), cs, my_sign * ld<T>(tile + r * D + my_partner) * sn);
                st<T>(y + ((row0 + r) * n_heads + h) * D + tid, v);
            }
        }
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
    const int64_t n_tiles = (n_rows + kRopeTile - 1) / kRopeTile;
    int n_sm = 0;
    const kvbfp_status st = sm_count(&n_sm);
    if (st != KVBFP_OK) return st;
    int64_t chunks = ((int64_t)n_sm * 16 + n_heads - 1) / n_heads;        // about two resident waves of thread blocks
    if (chunks > n_tiles) chunks = n_tiles;
    const unsigned grid = (unsigned)(chunks * n_heads);
    cudaStream_t s = (cudaStream_t)stream;
    if (dt == KVBFP_F32)
        rope_apply<float><<<grid, kRopeThreads, 0, s>>>((const float*)x, positions, n_rows, n_heads, theta, partner, sign, (float*)y,
                                                        (int)n_tiles, (int)chunks);
    else
        rope_apply<__nv_bfloat16><<<grid, kRopeThreads, 0, s>>>((const __nv_bfloat16*)x, positions, n_rows, n_heads, theta, partner,
                                                                sign, (__nv_bfloat16*)y, (int)n_tiles, (int)chunks);
    KVBFP_LAUNCH_CHECK("rope_apply");
    return KVBFP_OK;
}
