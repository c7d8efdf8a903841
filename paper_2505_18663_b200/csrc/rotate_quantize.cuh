// Online activation transform (Sec. 3.2, Eq. 10): rotate -> auto-scale -> quantize -> pack,
// one kernel, bound by HBM traffic (2K bytes read, K*b/8 + 8 bytes written per token).
//
// General-shape kernel, natural K order.  A warp owns a span of 1024 consecutive channels of
// one token: lane L holds four 16-byte chunks, channels c*256 + 8L + j (c chunk, j in 0..7),
// as 32 fp32 registers.  The Walsh-Hadamard butterflies over channel-index bits 0..log2(B)-1
// run in registers: bits 0-2 inside a chunk, bits 3-7 across lanes with shuffles, bits 8-9
// between chunks.  Blocks smaller than 1024 simply skip the upper stages, so one span holds
// 1024/B whole blocks.  The 1/sqrt(B) normalisation is folded into the scale.
#pragma once

#include "dvdq_common.cuh"

namespace dvdq {

constexpr int kRqSpan = 1024;

template <int LOG2B, int BITS>
__global__ void __launch_bounds__(512)
rq_natural_kernel(const __nv_bfloat16* __restrict__ X, int64_t M, int K, int64_t ldx,
                  uint8_t* __restrict__ codes, float* __restrict__ scales, int32_t* __restrict__ sums,
                  int spans, int tokens_per_cta) {
    __shared__ float s_max[32];
    __shared__ int s_sum[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int tl = warp / spans, sp = warp - tl * spans;
    const int64_t token = (int64_t)blockIdx.x * tokens_per_cta + tl;
    const bool tok_ok = token < M;

    float v[32];
    const __nv_bfloat16* xrow = X + (tok_ok ? token : 0) * ldx;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int e0 = sp * kRqSpan + c * 256 + lane * 8;
        uint4 raw = make_uint4(0u, 0u, 0u, 0u);
        if (tok_ok && e0 < K) raw = __ldg(reinterpret_cast<const uint4*>(xrow + e0));
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {  // a bf16 is the upper half of an fp32
            v[c * 8 + 2 * j] = __uint_as_float(w[j] << 16);
            v[c * 8 + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
        }
    }

    // in-chunk stages: index bits 0,1,2
#pragma unroll
    for (int h = 1; h < 8; h <<= 1) {
        if (h < (1 << LOG2B)) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                if ((i & h) == 0) {
                    const float a = v[i], b = v[i + h];
                    v[i] = a + b;
                    v[i + h] = a - b;
                }
            }
        }
    }
    // cross-lane stages: index bits 3..7 are lane bits 0..4
#pragma unroll
    for (int bit = 3; bit < 8; ++bit) {
        if (bit < LOG2B) {
            const int m = 1 << (bit - 3);
            const bool upper = (lane & m) != 0;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float o = __shfl_xor_sync(0xFFFFFFFFu, v[i], m);
                v[i] = upper ? (o - v[i]) : (v[i] + o);
            }
        }
    }
    // cross-chunk stages: index bits 8,9
#pragma unroll
    for (int bit = 8; bit < 10; ++bit) {
        if (bit < LOG2B) {
            const int h = 8 << (bit - 8);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                if ((i & h) == 0) {
                    const float a = v[i], b = v[i + h];
                    v[i] = a + b;
                    v[i + h] = a - b;
                }
            }
        }
    }

    // per-token absmax (of the un-normalised transform)
    float amax = 0.f;
#pragma unroll
    for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fabsf(v[i]));
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, m));
    if (lane == 0) s_max[warp] = amax;
    __syncthreads();
    amax = 0.f;
    for (int s = 0; s < spans; ++s) amax = fmaxf(amax, s_max[tl * spans + s]);

    constexpr float qmax = (float)((1 << (BITS - 1)) - 1);
    const float inv = amax > 0.f ? qmax / amax : 0.f;

    int q[32];
    int lsum = 0;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        q[i] = __float2int_rn(v[i] * inv);
        lsum += q[i];
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) lsum += __shfl_xor_sync(0xFFFFFFFFu, lsum, m);
    if (lane == 0) s_sum[warp] = lsum;

    // pack + store
    const int64_t row_bytes = act_row_bytes(K, BITS);
    uint8_t* crow = codes + (tok_ok ? token : 0) * row_bytes;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int e0 = sp * kRqSpan + c * 256 + lane * 8;
        const bool ok = tok_ok && e0 < K;
        uint32_t lo = 0u;
#pragma unroll
        for (int j = 0; j < 8; ++j) lo |= ((uint32_t)q[c * 8 + j] & 0xFu) << (4 * j);
        if (ok) *reinterpret_cast<uint32_t*>(crow + (e0 >> 1)) = lo;
        if (BITS == 6) {
            const int a = lane & 1;
            uint32_t hi = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) hi |= (((uint32_t)q[c * 8 + j] >> 4) & 0x3u) << (2 * (4 * (j >> 1) + (j & 1)));
            hi <<= 4 * a;  // hi_field_shift(a, j) = hi_field_shift(0, j) + 4a
            hi |= __shfl_xor_sync(0xFFFFFFFFu, hi, 1);
            if (ok && ((c ^ lane) & 1) == 0) *reinterpret_cast<uint32_t*>(crow + (K >> 1) + ((e0 >> 4) << 2)) = hi;
        }
    }

    __syncthreads();
    if (sp == 0 && lane == 0 && tok_ok) {
        int tsum = 0;
        for (int s = 0; s < spans; ++s) tsum += s_sum[tl * spans + s];
        // s_i = (absmax / sqrt(B)) / qmax
        const float rs = (LOG2B & 1) ? rsqrtf((float)(1 << LOG2B)) : 1.0f / (float)(1 << (LOG2B / 2));
        scales[token] = (amax * rs) / qmax;
        sums[token] = tsum;
    }
}

template <int BITS>
static dvdq_status launch_rq_bits(const void* X, int64_t M, int64_t K, int64_t ldx, int rot_block, void* codes,
                                  float* scales, int32_t* sums, cudaStream_t st) {
    const int spans = (int)((K + kRqSpan - 1) / kRqSpan);
    int tpc = 8 / spans;
    if (tpc < 1) tpc = 1;
    const int threads = spans * tpc * 32;
    const int64_t grid = (M + tpc - 1) / tpc;
    if (grid > 0x7FFFFFFFll) return DVDQ_ERR_SHAPE;
    int log2b = 0;
    while ((1 << log2b) < rot_block) ++log2b;
#define DVDQ_RQ_CASE(L)                                                                                   \
    case L:                                                                                               \
        rq_natural_kernel<L, BITS><<<(unsigned)grid, threads, 0, st>>>(                                   \
            (const __nv_bfloat16*)X, M, (int)K, ldx, (uint8_t*)codes, scales, sums, spans, tpc);          \
        break;
    switch (log2b) {
        DVDQ_RQ_CASE(0)
        DVDQ_RQ_CASE(6)
        DVDQ_RQ_CASE(7)
        DVDQ_RQ_CASE(8)
        DVDQ_RQ_CASE(9)
        DVDQ_RQ_CASE(10)
        default:
            return DVDQ_ERR_ROT_BLOCK;
    }
#undef DVDQ_RQ_CASE
    return cuda_status(cudaGetLastError());
}

inline dvdq_status launch_rotate_quantize(const void* X, int64_t M, int64_t K, int64_t ldx, const dvdq_act_quant& q,
                                          void* codes, float* scales, int32_t* sums, cudaStream_t st) {
    if (M == 0) return DVDQ_OK;
    if (q.bits == 4) return launch_rq_bits<4>(X, M, K, ldx, q.rot_block, codes, scales, sums, st);
    return launch_rq_bits<6>(X, M, K, ldx, q.rot_block, codes, scales, sums, st);
}

}  // namespace dvdq
