// K-sort set-up, Algorithm 1 of the paper (Sec. III): step 1 channel statistic, step 2 argsort,
// steps 3-4 row gather of a projection weight.
//
// colstat: x[T][C] is read as a flat array of 16-byte vectors; the grid stride is a multiple of the
// vectors per row, so a thread stays on the same channels and keeps its running statistic in
// registers.  Max-abs is taken on IEEE magnitude bits (integer compare: exact, order-independent).
#include "common.cuh"

namespace kvbfp {
namespace {

constexpr int kThreads = 256;

// ---- step 1, max-abs ----------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(kThreads) colstat_maxabs(const T* __restrict__ x, int64_t n_vec,
                                                           int vec_per_row, uint32_t* __restrict__ stat_bits) {
    constexpr int VEC = 16 / sizeof(T);
    extern __shared__ uint32_t sm_stat[];            // [C] for the channels this CTA can touch
    const int C = vec_per_row * VEC;
    for (int c = threadIdx.x; c < C; c += kThreads) sm_stat[c] = 0;
    __syncthreads();
    const int64_t tid = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * kThreads;       // multiple of vec_per_row
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    uint32_t m0 = 0, m1 = 0, m2 = 0, m3 = 0;
    int64_t i = tid;
    for (; i + 3 * stride < n_vec; i += 4 * stride) {
        uint4 a = __ldg(xv + i), b = __ldg(xv + i + stride), c = __ldg(xv + i + 2 * stride), d = __ldg(xv + i + 3 * stride);
        if (sizeof(T) == 2) {
            m0 = __vmaxu2(__vmaxu2(m0, a.x & 0x7fff7fffu), __vmaxu2(b.x & 0x7fff7fffu, __vmaxu2(c.x & 0x7fff7fffu, d.x & 0x7fff7fffu)));
            m1 = __vmaxu2(__vmaxu2(m1, a.y & 0x7fff7fffu), __vmaxu2(b.y & 0x7fff7fffu, __vmaxu2(c.y & 0x7fff7fffu, d.y & 0x7fff7fffu)));
            m2 = __vmaxu2(__vmaxu2(m2, a.z & 0x7fff7fffu), __vmaxu2(b.z & 0x7fff7fffu, __vmaxu2(c.z & 0x7fff7fffu, d.z & 0x7fff7fffu)));
            m3 = __vmaxu2(__vmaxu2(m3, a.w & 0x7fff7fffu), __vmaxu2(b.w & 0x7fff7fffu, __vmaxu2(c.w & 0x7fff7fffu, d.w & 0x7fff7fffu)));
        } else {
            m0 = max(max(m0, a.x & 0x7fffffffu), max(b.x & 0x7fffffffu, max(c.x & 0x7fffffffu, d.x & 0x7fffffffu)));
            m1 = max(max(m1, a.y & 0x7fffffffu), max(b.y & 0x7fffffffu, max(c.y & 0x7fffffffu, d.y & 0x7fffffffu)));
            m2 = max(max(m2, a.z & 0x7fffffffu), max(b.z & 0x7fffffffu, max(c.z & 0x7fffffffu, d.z & 0x7fffffffu)));
            m3 = max(max(m3, a.w & 0x7fffffffu), max(b.w & 0x7fffffffu, max(c.w & 0x7fffffffu, d.w & 0x7fffffffu)));
        }
    }
    for (; i < n_vec; i += stride) {
        uint4 a = __ldg(xv + i);
        if (sizeof(T) == 2) {
            m0 = __vmaxu2(m0, a.x & 0x7fff7fffu); m1 = __vmaxu2(m1, a.y & 0x7fff7fffu);
            m2 = __vmaxu2(m2, a.z & 0x7fff7fffu); m3 = __vmaxu2(m3, a.w & 0x7fff7fffu);
        } else {
            m0 = max(m0, a.x & 0x7fffffffu); m1 = max(m1, a.y & 0x7fffffffu);
            m2 = max(m2, a.z & 0x7fffffffu); m3 = max(m3, a.w & 0x7fffffffu);
        }
    }
    const int c0 = (int)(tid % vec_per_row) * VEC;
    if (tid < n_vec) {
        uint32_t m[4] = {m0, m1, m2, m3};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (sizeof(T) == 2) {   // widen bf16 magnitudes to binary32 bit patterns
                atomicMax(&sm_stat[c0 + 2 * k], (m[k] & 0xffffu) << 16);
                atomicMax(&sm_stat[c0 + 2 * k + 1], m[k] & 0xffff0000u);
            } else {
                atomicMax(&sm_stat[c0 + k], m[k]);
            }
        }
    }
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += kThreads)
        if (sm_stat[c]) atomicMax(&stat_bits[c], sm_stat[c]);
}

// ---- step 1, sum of squares in fp64 (Euclidean norm of Algorithm 1) ---------------
template <typename T>
__global__ void __launch_bounds__(kThreads) colstat_sumsq(const T* __restrict__ x, int64_t n_vec, int vec_per_row,
                                                          double* __restrict__ sums) {
    constexpr int VEC = 16 / sizeof(T);
    const int64_t tid = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * kThreads;
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    double acc[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) acc[k] = 0.0;
    for (int64_t i = tid; i < n_vec; i += stride) {
        uint4 a = __ldg(xv + i);
        uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (sizeof(T) == 2) {
                double lo = (double)__uint_as_float(w[k] << 16), hi = (double)__uint_as_float(w[k] & 0xffff0000u);
                acc[(2 * k) % VEC] += lo * lo;
                acc[(2 * k + 1) % VEC] += hi * hi;
            } else {
                double v = (double)__uint_as_float(w[k]);
                acc[k % VEC] += v * v;
            }
        }
    }
    if (tid < n_vec) {
        const int c0 = (int)(tid % vec_per_row) * VEC;
#pragma unroll
        for (int k = 0; k < VEC; ++k) atomicAdd(&sums[c0 + k], acc[k]);
    }
}

// ---- step 2: per-head stable argsort by rank counting ------------------------------
// KeyT = uint32_t (binary32 magnitude bits) or double (sums of squares).  One CTA per head.
template <typename KeyT>
__global__ void __launch_bounds__(kHeadDim) head_argsort(const KeyT* __restrict__ keys, float* __restrict__ stat_out,
                                                         int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
                                                         uint32_t* status) {
    constexpr int D = kHeadDim;
    __shared__ KeyT k[D];
    const int h = blockIdx.x, c = threadIdx.x;
    KeyT mine = keys[h * D + c];
    if (sizeof(KeyT) == 8) {     // fp64 sums: publish sqrt as the f32 statistic; NaN/Inf -> flag
        double s = (double)mine;
        if (!(s <= 1.7976931348623157e308) ) { raise_flag(status, KVBFP_FLAG_NONFINITE); mine = (KeyT)0; }
        stat_out[h * D + c] = (float)sqrt(s);
    } else {
        uint32_t bits = (uint32_t)mine;
        if ((bits >> 23) == 255u) raise_flag(status, KVBFP_FLAG_NONFINITE);
    }
    k[c] = mine;
    __syncthreads();
    int rank = 0;
    for (int o = 0; o < D; ++o) rank += (k[o] < mine) || (k[o] == mine && o < c);
    perm[h * D + rank] = c;
    if (inv_perm) inv_perm[h * D + c] = rank;
}

// ---- steps 3-4: gather weight rows ---------------------------------------------------
__global__ void __launch_bounds__(256) fold_rows(const uint8_t* __restrict__ w, uint8_t* __restrict__ out,
                                                 const int32_t* __restrict__ perm, int64_t row_bytes) {
    const int row = blockIdx.x;                     // h*D + j
    const int h = row / kHeadDim;
    const int srow = h * kHeadDim + (perm[row] & (kHeadDim - 1));
    const uint8_t* s = w + (int64_t)srow * row_bytes;
    uint8_t* d = out + (int64_t)row * row_bytes;
    if ((row_bytes & 15) == 0) {
        const int64_t nv = row_bytes >> 4;
        for (int64_t i = threadIdx.x; i < nv; i += blockDim.x)
            reinterpret_cast<uint4*>(d)[i] = __ldg(reinterpret_cast<const uint4*>(s) + i);
    } else {
        for (int64_t i = threadIdx.x; i < row_bytes; i += blockDim.x) d[i] = s[i];
    }
}

template <typename T>
kvbfp_status run_calibrate(const void* x, int64_t n_tokens, int n_heads, kvbfp_stat stat, float* stat_out,
                           int32_t* perm_out, int32_t* inv_perm_out, void* workspace, cudaStream_t s,
                           uint32_t* status) {
    constexpr int VEC = 16 / sizeof(T);
    const int C = n_heads * kHeadDim;
    const int vec_per_row = C / VEC;
    const int64_t n_vec = n_tokens * vec_per_row;
    // grid * kThreads must be a multiple of vec_per_row
    int unit = vec_per_row;
    {   // unit = vec_per_row / gcd(vec_per_row, kThreads)
        int a = vec_per_row, b = kThreads;
        while (b) { int t = a % b; a = b; b = t; }
        unit = vec_per_row / a;
    }
    int64_t want = (n_vec + kThreads - 1) / kThreads;
    int n_sm = 0;
    const kvbfp_status sm_st = sm_count(&n_sm);
    if (sm_st != KVBFP_OK) return sm_st;
    int64_t cap = (int64_t)n_sm * 8;
    int64_t g = want < cap ? want : cap;
    g = ((g + unit - 1) / unit) * unit;
    if (g < unit) g = unit;
    if (stat == KVBFP_STAT_MAXABS) {
        KVBFP_CUDA(cudaMemsetAsync(stat_out, 0, (size_t)C * sizeof(float), s));
        if (n_vec > 0) {
            colstat_maxabs<T><<<(int)g, kThreads, (size_t)C * sizeof(uint32_t), s>>>(
                (const T*)x, n_vec, vec_per_row, reinterpret_cast<uint32_t*>(stat_out));
            KVBFP_LAUNCH_CHECK("colstat_maxabs");
        }
        head_argsort<uint32_t><<<n_heads, kHeadDim, 0, s>>>(reinterpret_cast<const uint32_t*>(stat_out), stat_out,
                                                           perm_out, inv_perm_out, status);
        KVBFP_LAUNCH_CHECK("head_argsort");
    } else {
        double* sums = static_cast<double*>(workspace);
        KVBFP_CUDA(cudaMemsetAsync(sums, 0, (size_t)C * sizeof(double), s));
        if (n_vec > 0) {
            colstat_sumsq<T><<<(int)g, kThreads, 0, s>>>((const T*)x, n_vec, vec_per_row, sums);
            KVBFP_LAUNCH_CHECK("colstat_sumsq");
        }
        head_argsort<double><<<n_heads, kHeadDim, 0, s>>>(sums, stat_out, perm_out, inv_perm_out, status);
        KVBFP_LAUNCH_CHECK("head_argsort");
    }
    return KVBFP_OK;
}

}  // namespace
}  // namespace kvbfp

extern "C" kvbfp_status kvbfp_calibrate(const void* x, kvbfp_dtype dt, int64_t n_tokens, int32_t n_heads,
                                        int32_t head_dim, kvbfp_stat stat, float* stat_out, int32_t* perm_out,
                                        int32_t* inv_perm_out, void* workspace, size_t workspace_bytes,
                                        void* stream) {
    using namespace kvbfp;
    if ((!x && n_tokens != 0) || !stat_out || !perm_out || n_tokens < 0 || n_heads < 1) return KVBFP_ERR_INVALID_ARG;
    if (head_dim != kHeadDim) return KVBFP_ERR_UNSUPPORTED;
    if (n_heads > 96) return KVBFP_ERR_UNSUPPORTED;      // channel table of one CTA: 96*128*4 = 48 KB
    if (dt != KVBFP_F32 && dt != KVBFP_BF16) return KVBFP_ERR_INVALID_ARG;
    if (stat != KVBFP_STAT_MAXABS && stat != KVBFP_STAT_L2) return KVBFP_ERR_INVALID_ARG;
    if ((x && !aligned16(x)) || !aligned16(stat_out) || !aligned16(perm_out) || (inv_perm_out && !aligned16(inv_perm_out)))
        return KVBFP_ERR_ALIGNMENT;
    if (stat == KVBFP_STAT_L2) {
        if (!workspace || workspace_bytes < (size_t)n_heads * head_dim * sizeof(double)) return KVBFP_ERR_WORKSPACE;
        if (!aligned16(workspace)) return KVBFP_ERR_ALIGNMENT;
    }
    uint32_t* status = nullptr;
    kvbfp_status st = status_word(&status);
    if (st != KVBFP_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    if (dt == KVBFP_F32)
        return run_calibrate<float>(x, n_tokens, n_heads, stat, stat_out, perm_out, inv_perm_out, workspace, s, status);
    return run_calibrate<__nv_bfloat16>(x, n_tokens, n_heads, stat, stat_out, perm_out, inv_perm_out, workspace, s, status);
}

extern "C" kvbfp_status kvbfp_fold_perm(const void* w, kvbfp_dtype dt, int32_t n_heads, int32_t head_dim,
                                        int64_t d_in, const int32_t* perm, void* out, void* stream) {
    using namespace kvbfp;
    if (!w || !out || !perm || n_heads < 1 || d_in < 1 || w == out) return KVBFP_ERR_INVALID_ARG;
    if (head_dim != kHeadDim) return KVBFP_ERR_UNSUPPORTED;
    if (dt != KVBFP_F32 && dt != KVBFP_BF16) return KVBFP_ERR_INVALID_ARG;
    if (!aligned16(w) || !aligned16(out) || !aligned16(perm)) return KVBFP_ERR_ALIGNMENT;
    const int64_t row_bytes = d_in * (dt == KVBFP_F32 ? 4 : 2);
    fold_rows<<<n_heads * head_dim, 256, 0, (cudaStream_t)stream>>>((const uint8_t*)w, (uint8_t*)out, perm, row_bytes);
    KVBFP_LAUNCH_CHECK("fold_rows");
    return KVBFP_OK;
}
