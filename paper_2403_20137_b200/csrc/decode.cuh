// Internal interface between the decode entry point and its kernels.
#pragma once
#include "common.cuh"

namespace kvbfp {

// One partial result per (batch, query head, chunk): PSTRIDE floats =
// o[128] (sum of 2^(s-m) * V over the chunk, stored-slot order), m (running max, log2 units), l (sum).
constexpr int kPartStride = kHeadDim + 4;
constexpr int kMinChunk = 128;     // tokens; chunk sizes are multiples of this

struct DecodeArgs {
    kvbfp_format fmt;
    const uint8_t *k_mant, *k_exp, *v_mant, *v_exp;
    const void* q;            // [B, Hq, d]
    int q_is_bf16;
    int n_q_heads;
    const int32_t* seq_lens;
    const int32_t* perm_k;
    const int32_t* inv_perm_v;
    float scale_log2e;        // softmax scale * log2(e)
    int q_mant_bits;
    float* out;
    uint32_t* qfrag;          // workspace region for the tensor-core kernel's B fragments
    float* partials;          // workspace region [B, Hq, n_chunks, kPartStride]
    int chunk;                // tokens per chunk
    int n_chunks;
    int len_cap;              // min(max_len_hint, max_seq)
    uint32_t* status;
    // 2^(32-k): multiplying by these and keeping the high word is a right shift by k that runs on the
    // multiply-add pipe instead of the integer pipe (passed at run time so that it stays a multiply)
    uint32_t mulhi4, mulhi8, mulhi12;
};

kvbfp_status launch_decode_simt(const DecodeArgs& a, cudaStream_t s);
kvbfp_status launch_decode_mma(const DecodeArgs& a, cudaStream_t s);    // bf16, every mantissa width
// fp16, 4-bit mantissas, persistent: *n_warps receives the number of warps the items were split over
kvbfp_status launch_decode_mma4(const DecodeArgs& a, cudaStream_t s, int* n_warps);
size_t qfrag_bytes(const kvbfp_format& f, int n_q_heads);
// Events the caller asked to have recorded around the main decode kernel (nullptr = none).
void profile_events(cudaEvent_t* start, cudaEvent_t* stop);

}  // namespace kvbfp
