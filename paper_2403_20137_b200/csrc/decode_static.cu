// kvbfp_decode_attn_static: decode attention for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a serving loop whose memory
// pool was sized and frozen at start-up, in a plug-in that is handed tensors but no allocator, or
// in code that must not synchronise the device (cudaMalloc and cudaFree may).  kvbfp_decode_attn
// needs a workspace (query fragments and one partial result per sequence chunk); this variant keeps
// that workspace in a fixed array that is part of the library image, so the caller passes inputs
// and outputs only.  The array costs kStaticScratchBytes of device memory on every GPU that loads
// the library, for as long as the process lives.
#include <atomic>
#include "common.cuh"

namespace kvbfp {
namespace {

constexpr size_t kStaticScratchBytes = 32u << 20;   // 32 MiB

// In host code this name is only a handle for the runtime, not a device address: it must be turned
// into one with cudaGetSymbolAddress before a kernel can be given it.
static __device__ __align__(256) uint8_t g_decode_scratch[kStaticScratchBytes];

// Device address of the array on the current device, looked up once per device.
kvbfp_status scratch_address(void** out) {
    constexpr int kMaxDev = 64;
    static std::atomic<void*> cache[kMaxDev];      // two host threads asking at once store the same address
    int dev = 0;
    KVBFP_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDev) return KVBFP_ERR_UNSUPPORTED;
    if (!cache[dev].load(std::memory_order_acquire)) {
        void* p = nullptr;
        KVBFP_CUDA(cudaGetSymbolAddress(&p, g_decode_scratch));
        if (!p) return KVBFP_ERR_CUDA;
        cache[dev].store(p, std::memory_order_release);
    }
    *out = cache[dev].load(std::memory_order_relaxed);
    return KVBFP_OK;
}

}  // namespace
}  // namespace kvbfp

extern "C" size_t kvbfp_static_scratch_bytes(void) { return kvbfp::kStaticScratchBytes; }

extern "C" kvbfp_status kvbfp_decode_attn_static(const kvbfp_cache* cache, const void* q, kvbfp_dtype q_dt,
                                                 int32_t n_q_heads, const int32_t* seq_lens, int32_t max_len_hint,
                                                 const int32_t* perm_k, const int32_t* inv_perm_v,
                                                 float softmax_scale, int32_t q_mant_bits, float* out,
                                                 uint32_t flags, void* stream) {
    using namespace kvbfp;
    if (!cache) return KVBFP_ERR_INVALID_ARG;
    kvbfp_status st = check_format(&cache->fmt);
    if (st != KVBFP_OK) return st;
    if (n_q_heads < 1 || n_q_heads % cache->fmt.n_kv_heads != 0) return KVBFP_ERR_INVALID_ARG;
    const size_t need = kvbfp_decode_workspace_bytes(&cache->fmt, n_q_heads);
    if (need == 0) return KVBFP_ERR_INVALID_ARG;
    if (need > kStaticScratchBytes) return KVBFP_ERR_WORKSPACE;   // geometry too large for the fixed array
    void* scratch = nullptr;
    st = scratch_address(&scratch);
    if (st != KVBFP_OK) return st;
    // The workspace needs no initial contents: every partial result that the merge uses is written by this call
    // first (it may load slots beyond those before it knows the sequence's length, and drops them unused), so
    // nothing has to be cleared between calls.
    return kvbfp_decode_attn(cache, q, q_dt, n_q_heads, seq_lens, max_len_hint, perm_k, inv_perm_v, softmax_scale,
                             q_mant_bits, out, scratch, kStaticScratchBytes, flags, stream);
}
