// Shared host/device helpers of the kvbfp CUDA library (sm_100a).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvbfp.h"

namespace kvbfp {

constexpr int kHeadDim = 128;

// ---- host side -------------------------------------------------------------

// Records a failed CUDA call for kvbfp_last_cuda_error() and maps it to a status.
kvbfp_status cuda_fail(cudaError_t e, const char* what);
// Address of the device status word of the current device (no allocation: a __device__ symbol).
kvbfp_status status_word(uint32_t** ptr);
void count_launch(int n = 1);
// Number of SMs of the current device (asked once per device); grids are sized in multiples of it.
kvbfp_status sm_count(int* n);

// Tensor map over a plane of byte rows, [n_rows, row_bytes] (row_bytes 64 or 128), copied in boxes of box_rows whole
// rows, swizzled in shared memory: the 16-byte pieces of a row land at piece ^ (row % 8) for rows of 128 bytes and at
// piece ^ ((row / 2) % 4) for rows of 64 bytes, so that the same piece of eight neighbouring rows falls into eight
// different bank groups.  The map covers memory of the current device only.
kvbfp_status make_row_map(CUtensorMap* map, const void* base, uint64_t n_rows, uint32_t row_bytes, uint32_t box_rows);

#define KVBFP_CUDA(call)                                                         \
    do {                                                                         \
        cudaError_t e__ = (call);                                                \
        if (e__ != cudaSuccess) return ::kvbfp::cuda_fail(e__, #call);           \
    } while (0)

#define KVBFP_LAUNCH_CHECK(name)                                                 \
    do {                                                                         \
        cudaError_t e__ = cudaGetLastError();                                    \
        if (e__ != cudaSuccess) return ::kvbfp::cuda_fail(e__, name);            \
        ::kvbfp::count_launch();                                                 \
    } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline kvbfp_status check_format(const kvbfp_format* f) {
    if (!f) return KVBFP_ERR_INVALID_ARG;
    if (f->batch < 1 || f->n_kv_heads < 1 || f->max_seq < 1) return KVBFP_ERR_INVALID_ARG;
    if (f->head_dim != kHeadDim) return KVBFP_ERR_UNSUPPORTED;
    if (f->block != 16 && f->block != 32 && f->block != 64 && f->block != 128) return KVBFP_ERR_UNSUPPORTED;
    if (f->mant_bits != 4 && f->mant_bits != 6 && f->mant_bits != 8) return KVBFP_ERR_UNSUPPORTED;
    if (f->max_seq % 16 != 0) return KVBFP_ERR_INVALID_ARG;
    return KVBFP_OK;
}
inline size_t row_m_bytes(const kvbfp_format& f) { return (size_t)f.head_dim * f.mant_bits / 8; }
inline size_t row_e_bytes(const kvbfp_format& f) { return (size_t)(f.head_dim / f.block); }

// ---- device side -----------------------------------------------------------

// ---- launches that overlap with the kernel before them -----------------------
//
// The kernels of a decode step (cache write, query coefficients, attention, merge) are launched with programmatic
// stream serialization: the next kernel's thread blocks may become resident and run their set-up while the kernel
// before it is still running.  Every such kernel calls pdl_wait() before its first access to global memory (it
// returns once the kernel before it has completed and its writes are visible; at once if the launch had no such
// predecessor) and pdl_trigger() after it, so that at most one kernel waits behind the running one and its blocks
// never compete with blocks of the running kernel that have not started yet: the short kernels right after the
// wait, the persistent decode kernels at their end (waiting blocks on an SM slow its streaming warps down).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t h) { return __uint_as_float(h << 16); }

// 2^k for k in [-126, 127]
__device__ __forceinline__ float pow2i(int k) { return __uint_as_float((uint32_t)(k + 127) << 23); }

// Weight of one mantissa unit, 2^(e8 - 127 - (p-2)), as an fp32 number; exact down to 2^-133
// (subnormal) for e8 = 0, p = 8.
__device__ __forceinline__ float unit_weight(int e8, int p) {
    int f = e8 - (p - 2);                 // biased exponent field of the result
    return f >= 1 ? __uint_as_float((uint32_t)f << 23) : __uint_as_float(1u << (22 + f));
}

// cos and sin of an angle given in fp64 (token position times frequency, up to ~1e6 rad): reduced to [-pi, pi]
// in fp64, evaluated in fp32.
__device__ __forceinline__ void sincos_reduced(double angle, float* sn, float* cs) {
    const double k = rint(angle * 0.15915494309189535);                        // 1 / (2 pi)
    const double r = fma(-k, 2.4492935982947064e-16, fma(-k, 6.283185307179586, angle));   // 2 pi in two terms
    sincosf((float)r, sn, cs);
}

__device__ __forceinline__ void raise_flag(uint32_t* status, uint32_t bit) { atomicOr(status, bit); }

// Mantissa stored in the p-bit field (excess-2^(p-1) code) starting at bit `bit` of a little-endian byte row.
__device__ __forceinline__ int extract_field(const uint8_t* row, int bit, int p) {
    int byte = bit >> 3, sh = bit & 7;
    uint32_t w = row[byte] | ((uint32_t)row[byte + ((sh + p > 8) ? 1 : 0)] << 8);
    return (int)((w >> sh) & ((1u << p) - 1u)) - (1 << (p - 1));
}

}  // namespace kvbfp
