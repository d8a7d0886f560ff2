// Decode attention on the plain fp32 ALUs, read straight from the packed planes (Sec. III par. 2 of
// the paper: keys are read back from the cache and multiplied with pi(q)).
//
// One warp owns one (batch, query head, chunk) item.  Four neighbouring lanes share a token: lane
// (r, c) = (lane/4, lane%4) holds slots [32c, 32c+32) of token r of each 8-token step, so a warp
// load covers 8 whole rows.  Mantissas are unpacked to integers in registers, the dot product of a
// block is accumulated on the integers and scaled once by the block's 2^e (Sec. II-B: integer
// products, exponents added).  Each 4-lane group keeps its own running softmax maximum; the eight
// groups are merged once at the end of the chunk.
#include <math.h>

#include "decode.cuh"

namespace kvbfp {
namespace {

constexpr int kWarps = 4;

template <int P>
__device__ __forceinline__ void load_chunk(const uint8_t* p, uint32_t (&w)[P]) {
    if (P == 4) {
        uint4 a = __ldg(reinterpret_cast<const uint4*>(p));
        w[0] = a.x; w[1] = a.y; w[2] = a.z; w[3] = a.w;
    } else if (P == 6) {
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            uint2 a = __ldg(reinterpret_cast<const uint2*>(p) + i);
            w[2 * i] = a.x; w[2 * i + 1] = a.y;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            uint4 a = __ldg(reinterpret_cast<const uint4*>(p) + i);
            w[4 * i] = a.x; w[4 * i + 1] = a.y; w[4 * i + 2] = a.z; w[4 * i + 3] = a.w;
        }
    }
}

// Slot i (compile-time) of a lane's 32-slot chunk: the stored field is M + 2^(P-1).
template <int P>
__device__ __forceinline__ float slot_value(const uint32_t (&w)[P], int i) {
    const int bit = i * P, word = bit >> 5, sh = bit & 31;
    uint32_t v = (sh + P > 32) ? __funnelshift_r(w[word], w[(word + 1) % P], sh) : (w[word] >> sh);
    return (float)((int)(v & ((1u << P) - 1u)) - (1 << (P - 1)));
}

// ROPE: the cache holds keys as they were before the rotary embedding (Sec. III par. 2); the rotation of
// token t's key to position t is moved onto the query: q . R_t k = (R_t^T q) . k, and R_t^T q is carried from
// token to token by a fixed rotation (the lane's tokens are 8 apart).
template <int P, int N, bool ROPE>
__global__ void __launch_bounds__(kWarps * 32) decode_simt(DecodeArgs a) {
    constexpr int D = kHeadDim, ROW_M = D * P / 8, ROW_E = D / N;
    constexpr int NB = (N == 16) ? 2 : 1;          // blocks inside one lane's 32 slots
    const int lane = threadIdx.x & 31, r = lane >> 2, c = lane & 3;
    const int Hkv = a.fmt.n_kv_heads, G = a.n_q_heads / Hkv;
    const int64_t item = (int64_t)blockIdx.x * kWarps + (threadIdx.x >> 5);
    const int64_t n_items = (int64_t)a.fmt.batch * a.n_q_heads * a.n_chunks;
    if (item >= n_items) return;
    // neighbouring warps take the query heads that share one KV head, so they read the same rows
    const int qi = (int)(item % G);
    const int chunk_id = (int)((item / G) % a.n_chunks);
    const int g = (int)((item / G / a.n_chunks) % Hkv);
    const int b = (int)(item / G / a.n_chunks / Hkv);
    const int hq = g * G + qi;

    int len = a.seq_lens[b];
    if (len > a.fmt.max_seq || len < 0) {
        if (lane == 0 && chunk_id == 0 && hq == 0) raise_flag(a.status, KVBFP_FLAG_POSITION);
        len = len < 0 ? 0 : a.fmt.max_seq;
    }
    if (len > a.len_cap) {
        if (lane == 0 && chunk_id == 0 && hq == 0) raise_flag(a.status, KVBFP_FLAG_LEN_HINT);
        len = a.len_cap;
    }
    const int t0 = chunk_id * a.chunk;
    if (t0 >= len) return;
    const int t1 = min(len, t0 + a.chunk);

    // pi(q): slot j takes channel perm_k[g][j] (Eq. (3)); the softmax scale and log2(e) ride along
    float q[32];
    {
        const int64_t qbase = ((int64_t)b * a.n_q_heads + hq) * D;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int slot = 32 * c + i;
            const int ch = a.perm_k ? (a.perm_k[g * D + slot] & (D - 1)) : slot;
            q[i] = a.q_is_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(a.q)[qbase + ch])
                               : static_cast<const float*>(a.q)[qbase + ch];
        }
        if (a.q_mant_bits) {   // BFP query (Sec. IV): same block size, 8-bit mantissas
            uint32_t am[2] = {0, 0};
#pragma unroll
            for (int i = 0; i < 32; ++i) am[i >> 4] = max(am[i >> 4], __float_as_uint(q[i]) & 0x7fffffffu);
            if (N >= 32) am[0] = am[1] = max(am[0], am[1]);
            if (N >= 64) am[0] = am[1] = max(am[0], __shfl_xor_sync(0xffffffffu, am[0], 1));
            if (N >= 128) am[0] = am[1] = max(am[0], __shfl_xor_sync(0xffffffffu, am[0], 2));
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                int e8 = (int)(am[i >> 4] >> 23);
                if (e8 == 255) { raise_flag(a.status, KVBFP_FLAG_NONFINITE); e8 = 254; }
                const int k = 127 - e8 + 6, k1 = k >> 1, k2 = k - k1;
                float tv = (q[i] * pow2i(k1)) * pow2i(k2);
                tv = rintf(fminf(fmaxf(tv, -127.f), 127.f));
                q[i] = tv * unit_weight(e8, 8);
            }
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) q[i] *= a.scale_log2e;
    }
    // ROPE state of slot i for the lane's current token t:  q[i] = q_i cos(t th_i) + q'_i sin(t th_i)  (the
    // coefficient of k_i in the score), qw[i] = q'_i cos - q_i sin, with q'_i = -sign_i q_partner(i) (Eq. (4),
    // partners share a frequency and have opposite signs); cos and sin of 8 th_i advance both by 8 tokens.
    // (the step rotation sits in shared memory, one (cos, sin) pair per slot and warp: it only depends on the head,
    // and 64 more registers per lane would leave no room for the prefetched words)
    float qw[ROPE ? 32 : 1];
    __shared__ float2 step_cs[ROPE ? kWarps : 1][ROPE ? 32 * 4 : 1];
    float2* my_cs = &step_cs[ROPE ? (threadIdx.x >> 5) : 0][0];
    if (ROPE) {
        const int64_t qbase = ((int64_t)b * a.n_q_heads + hq) * D;
        const double pos0 = (double)(t0 + r);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int slot = g * D + 32 * c + i;
            const int pj = a.rope_partner[slot] & (D - 1);
            const int ch = a.perm_k ? (a.perm_k[g * D + pj] & (D - 1)) : pj;
            const float qp = (a.q_is_bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(a.q)[qbase + ch])
                                          : static_cast<const float*>(a.q)[qbase + ch]) * a.scale_log2e;
            const float q1 = -a.rope_sign[slot] * qp;
            const double th = a.rope_theta[slot];
            float sn, cs;
            sincos_reduced(pos0 * th, &sn, &cs);
            const float q0 = q[i];
            q[i] = q0 * cs + q1 * sn;
            qw[i] = q1 * cs - q0 * sn;
            if (r == 0) {       // the warp's eight token groups share the head, so one of them fills the table
                float sn8, cs8;
                sincos_reduced(8.0 * th, &sn8, &cs8);
                my_cs[i * 4 + c] = make_float2(cs8, sn8);
            }
        }
        __syncwarp();
    }

    const int64_t row0 = ((int64_t)b * Hkv + g) * a.fmt.max_seq;
    const uint8_t* km = a.k_mant + row0 * ROW_M + c * (4 * P);
    const uint8_t* vm = a.v_mant + row0 * ROW_M + c * (4 * P);
    const uint8_t* ke = a.k_exp + row0 * ROW_E;
    const uint8_t* ve = a.v_exp + row0 * ROW_E;
    const int eb = (N == 16) ? 2 * c : (N == 32) ? c : (N == 64) ? (c >> 1) : 0;   // first block of this lane

    float o[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) o[i] = 0.f;
    float m = -INFINITY, l = 0.f;

    // The packed words and exponent bytes of the lane's next token are loaded before the current token is worked
    // on: with a handful of warps per SM the kernel is otherwise bound by the latency of these loads.
    struct Tok {
        uint32_t k[P], v[P];
        uint32_t ke[NB], ve[NB];
    };
    auto fetch = [&](int tok, Tok& x) {
        if (tok < t1) {
            load_chunk<P>(km + (int64_t)tok * ROW_M, x.k);
            load_chunk<P>(vm + (int64_t)tok * ROW_M, x.v);
#pragma unroll
            for (int blk = 0; blk < NB; ++blk) {
                x.ke[blk] = __ldg(ke + (int64_t)tok * ROW_E + eb + blk);
                x.ve[blk] = __ldg(ve + (int64_t)tok * ROW_E + eb + blk);
            }
        }
    };
    Tok nxt;
    fetch(t0 + r, nxt);
    for (int tb = t0; tb < t1; tb += 8) {
        const int tok = tb + r;
        const bool valid = tok < t1;
        const Tok cur = nxt;
        fetch(tok + 8, nxt);
        float s = 0.f;
        if (valid) {
#pragma unroll
            for (int blk = 0; blk < NB; ++blk) {
                float acc = 0.f;
#pragma unroll
                for (int i = blk * (32 / NB); i < (blk + 1) * (32 / NB); ++i) acc = fmaf(q[i], slot_value<P>(cur.k, i), acc);
                s = fmaf(acc, unit_weight((int)cur.ke[blk], P), s);
            }
        }
        if (ROPE) {       // on to the lane's next token, 8 further
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float u = q[i], w = qw[i];
                const float2 cs = my_cs[i * 4 + c];
                q[i] = fmaf(u, cs.x, w * cs.y);
                qw[i] = fmaf(w, cs.x, -u * cs.y);
            }
        }
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        if (valid) {
            if (s > m + 8.f) {            // lazy rescale: the reference point only moves in big steps
                const float alpha = exp2f(m - s);
                l *= alpha;
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] *= alpha;
                m = s;
            }
            const float p = exp2f(s - m);
            l += p;
#pragma unroll
            for (int blk = 0; blk < NB; ++blk) {
                const float pw = p * unit_weight((int)cur.ve[blk], P);
#pragma unroll
                for (int i = blk * (32 / NB); i < (blk + 1) * (32 / NB); ++i) o[i] = fmaf(pw, slot_value<P>(cur.v, i), o[i]);
            }
        }
    }

    // merge the eight token groups of the warp
    float mm = m;
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, off));
    const float alpha = (m == -INFINITY) ? 0.f : exp2f(m - mm);
    l *= alpha;
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        float v = o[i] * alpha;
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        o[i] = v;
    }
    float* dst = a.partials + (((int64_t)b * a.n_q_heads + hq) * a.n_chunks + chunk_id) * kPartStride;
    if (r == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
            reinterpret_cast<float4*>(dst + 32 * c)[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
        if (c == 0) { dst[D] = mm; dst[D + 1] = l; }
    }
}

template <int P, int N, bool ROPE>
kvbfp_status launch(const DecodeArgs& a, cudaStream_t s) {
    const int64_t n_items = (int64_t)a.fmt.batch * a.n_q_heads * a.n_chunks;
    if ((n_items + kWarps - 1) / kWarps > 0x7fffffffLL) return KVBFP_ERR_UNSUPPORTED;     // more thread blocks than a grid holds
    const int grid = (int)((n_items + kWarps - 1) / kWarps);
    cudaEvent_t ev0, ev1;
    profile_events(&ev0, &ev1);
    if (ev0) KVBFP_CUDA(cudaEventRecord(ev0, s));
    decode_simt<P, N, ROPE><<<grid, kWarps * 32, 0, s>>>(a);
    KVBFP_LAUNCH_CHECK("decode_simt");
    if (ev1) KVBFP_CUDA(cudaEventRecord(ev1, s));
    return KVBFP_OK;
}

template <int P, bool ROPE>
kvbfp_status launch_n(const DecodeArgs& a, cudaStream_t s) {
    switch (a.fmt.block) {
        case 16: return launch<P, 16, ROPE>(a, s);
        case 32: return launch<P, 32, ROPE>(a, s);
        case 64: return launch<P, 64, ROPE>(a, s);
        case 128: return launch<P, 128, ROPE>(a, s);
    }
    return KVBFP_ERR_UNSUPPORTED;
}

template <bool ROPE>
kvbfp_status launch_p(const DecodeArgs& a, cudaStream_t s) {
    switch (a.fmt.mant_bits) {
        case 4: return launch_n<4, ROPE>(a, s);
        case 6: return launch_n<6, ROPE>(a, s);
        case 8: return launch_n<8, ROPE>(a, s);
    }
    return KVBFP_ERR_UNSUPPORTED;
}

}  // namespace

kvbfp_status launch_decode_simt(const DecodeArgs& a, cudaStream_t s) {
    return a.rope_theta ? launch_p<true>(a, s) : launch_p<false>(a, s);
}

}  // namespace kvbfp
