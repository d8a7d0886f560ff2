// Library-wide host state: status word address, error text, launch counter, small queries.
#include <atomic>
#include <cstdio>
#include <cstring>

#include "common.cuh"
#include "ptx.cuh"

namespace kvbfp {

// One status word per device: a __device__ symbol, so nothing is allocated.
__device__ uint32_t g_status_word = 0;

static thread_local char t_err[256] = "";
static std::atomic<uint64_t> g_launches{0};

kvbfp_status cuda_fail(cudaError_t e, const char* what) {
    snprintf(t_err, sizeof t_err, "%s: %s", what, cudaGetErrorString(e));
    (void)cudaGetLastError();   // clear the sticky-less error state
    return KVBFP_ERR_CUDA;
}

void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

kvbfp_status sm_count(int* n) {
    constexpr int kMaxDev = 64;
    static std::atomic<int> cache[kMaxDev];            // per device; 0 = not asked yet
    int dev = 0;
    KVBFP_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDev) return KVBFP_ERR_UNSUPPORTED;
    int v = cache[dev].load(std::memory_order_acquire);
    if (!v) {
        KVBFP_CUDA(cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev));
        if (v < 1) return KVBFP_ERR_CUDA;
        cache[dev].store(v, std::memory_order_release);
    }
    *n = v;
    return KVBFP_OK;
}

kvbfp_status make_row_map(CUtensorMap* map, const void* base, uint64_t n_rows, uint32_t row_bytes, uint32_t box_rows) {
    using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static std::atomic<EncodeFn> encode{nullptr};      // the driver's entry point, asked for once
    EncodeFn fn = encode.load(std::memory_order_acquire);
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        KVBFP_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q));
        if (!p || q != cudaDriverEntryPointSuccess) {
            snprintf(t_err, sizeof t_err, "cuTensorMapEncodeTiled is not available from this driver");
            return KVBFP_ERR_CUDA;
        }
        fn = reinterpret_cast<EncodeFn>(p);
        encode.store(fn, std::memory_order_release);
    }
    if ((row_bytes != 64 && row_bytes != 128) || box_rows < 1 || box_rows > 256 || n_rows < 1 ||
        n_rows > 0x7fffffffull || !aligned16(base))
        return KVBFP_ERR_UNSUPPORTED;
    const cuuint64_t dims[2] = {row_bytes, n_rows};
    const cuuint64_t strides[1] = {row_bytes};
    const cuuint32_t box[2] = {row_bytes, box_rows};
    const cuuint32_t elem[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, elem,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(t_err, sizeof t_err, "cuTensorMapEncodeTiled failed with driver error %d", (int)r);
        return KVBFP_ERR_CUDA;
    }
    return KVBFP_OK;
}

// Self-test of the bounded barrier wait that every staged kernel relies on: one warp, two barriers.  The first
// expects 16 bytes that a bulk copy delivers: its wait must succeed.  The second expects 16 bytes that nothing ever
// sends: its wait must give up after `tries` tries of `hint_ns` each, raise the time-out flag and return -- no trap,
// nothing left in flight, the context stays usable.
__device__ __align__(16) uint8_t g_selftest_bytes[16];
__global__ void __launch_bounds__(32) wait_selftest(uint32_t tries, uint32_t hint_ns, uint32_t* status) {
    __shared__ __align__(16) uint8_t landing[16];
    __shared__ __align__(8) uint64_t bars[2];
    const uint32_t b0 = smem_u32(&bars[0]), b1 = smem_u32(&bars[1]);
    if (threadIdx.x == 0) {
        mbar_init(b0, 1);
        mbar_init(b1, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        mbar_expect_tx(b0, 16u);
        bulk_g2s(smem_u32(landing), g_selftest_bytes, 16u, b0);
        mbar_expect_tx(b1, 16u);                 // bytes that never come
    }
    __syncwarp();
    const bool arrived = mbar_wait_bounded(b0, 0);             // the production bound: the copy lands long before it
    const bool never = mbar_wait_tries(b1, 0, hint_ns, tries);
    if (threadIdx.x == 0) {
        if (!arrived) raise_flag(status, KVBFP_FLAG_NONFINITE);    // (would mean the wait itself is broken)
        if (!never) raise_flag(status, KVBFP_FLAG_WAIT_TIMEOUT);
    }
}

kvbfp_status status_word(uint32_t** ptr) {
    constexpr int kMaxDev = 64;
    static std::atomic<uint32_t*> cache[kMaxDev];      // per device; two threads asking at once store the same address
    int dev = 0;
    KVBFP_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDev) return KVBFP_ERR_UNSUPPORTED;
    if (!cache[dev].load(std::memory_order_acquire)) {
        uint32_t* p = nullptr;
        KVBFP_CUDA(cudaGetSymbolAddress((void**)&p, g_status_word));
        cache[dev].store(p, std::memory_order_release);
    }
    *ptr = cache[dev].load(std::memory_order_relaxed);
    return KVBFP_OK;
}

}  // namespace kvbfp

extern "C" {

int32_t kvbfp_version(void) { return 100; }

const char* kvbfp_status_string(kvbfp_status s) {
    switch (s) {
        case KVBFP_OK: return "ok";
        case KVBFP_ERR_INVALID_ARG: return "invalid argument";
        case KVBFP_ERR_UNSUPPORTED: return "unsupported format or shape";
        case KVBFP_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
        case KVBFP_ERR_CAPACITY: return "cache capacity exceeded";
        case KVBFP_ERR_WORKSPACE: return "workspace missing or too small";
        case KVBFP_ERR_CUDA: return "CUDA error";
    }
    return "unknown status";
}

const char* kvbfp_last_cuda_error(void) { return kvbfp::t_err; }

uint64_t kvbfp_launch_count(void) { return kvbfp::g_launches.load(std::memory_order_relaxed); }

kvbfp_status kvbfp_plane_bytes(const kvbfp_format* fmt, size_t* mant_bytes, size_t* exp_bytes) {
    kvbfp_status st = kvbfp::check_format(fmt);
    if (st != KVBFP_OK) return st;
    size_t rows = (size_t)fmt->batch * fmt->n_kv_heads * fmt->max_seq;
    if (mant_bytes) *mant_bytes = rows * kvbfp::row_m_bytes(*fmt);
    if (exp_bytes) *exp_bytes = rows * kvbfp::row_e_bytes(*fmt);
    return KVBFP_OK;
}

kvbfp_status kvbfp_selftest_wait_timeout(uint32_t tries, uint32_t hint_ns, void* stream) {
    if (tries < 1 || tries > 1000 || hint_ns < 1 || hint_ns > 1000000) return KVBFP_ERR_INVALID_ARG;   // at most a second
    uint32_t* w = nullptr;
    kvbfp_status st = kvbfp::status_word(&w);
    if (st != KVBFP_OK) return st;
    kvbfp::wait_selftest<<<1, 32, 0, (cudaStream_t)stream>>>(tries, hint_ns, w);
    KVBFP_LAUNCH_CHECK("wait_selftest");
    return KVBFP_OK;
}

kvbfp_status kvbfp_device_status(uint32_t* flags_out, void* stream) {
    if (!flags_out) return KVBFP_ERR_INVALID_ARG;
    uint32_t* w = nullptr;
    kvbfp_status st = kvbfp::status_word(&w);
    if (st != KVBFP_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    KVBFP_CUDA(cudaMemcpyAsync(flags_out, w, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    KVBFP_CUDA(cudaMemsetAsync(w, 0, sizeof(uint32_t), s));
    KVBFP_CUDA(cudaStreamSynchronize(s));
    return KVBFP_OK;
}

}  // extern "C"
