// delta-Guided Bit Switching (Sec. 3.3): the two L1 norms of the per-step feature change,
//   num = || F_t - F_{t-1} ||_1,   den = || F_{t-1} ||_1,
// over the model output of a denoising step, and the host-side rule that turns their ratio
// into the activation bit width of the next step.  One pass over both tensors (HBM bound: 4
// bytes per element), fp32 inside a 16-byte chunk, fp64 across chunks, one atomic pair per CTA.
#pragma once

#include "dvdq_common.cuh"

namespace dvdq {

__global__ void __launch_bounds__(256)
gbs_l1_terms_kernel(const __nv_bfloat16* __restrict__ Ft, const __nv_bfloat16* __restrict__ Fp, int64_t n,
                    double* __restrict__ terms) {
    __shared__ double s_num[8], s_den[8];
    double num = 0.0, den = 0.0;
    const int64_t chunks = n / 8;
    const uint4* a4 = reinterpret_cast<const uint4*>(Ft);
    const uint4* b4 = reinterpret_cast<const uint4*>(Fp);
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < chunks; c += (int64_t)gridDim.x * blockDim.x) {
        const uint4 a = __ldg(a4 + c), b = __ldg(b4 + c);
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
        float pn = 0.f, pd = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {  // a bf16 is the upper half of an fp32
            const float a0 = __uint_as_float(aw[j] << 16), a1 = __uint_as_float(aw[j] & 0xFFFF0000u);
            const float b0 = __uint_as_float(bw[j] << 16), b1 = __uint_as_float(bw[j] & 0xFFFF0000u);
            pn += fabsf(a0 - b0) + fabsf(a1 - b1);
            pd += fabsf(b0) + fabsf(b1);
        }
        num += (double)pn;
        den += (double)pd;
    }
    // ragged tail (n not a multiple of 8): one thread of the grid
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t i = chunks * 8; i < n; ++i) {
            const float a = __bfloat162float(Ft[i]), b = __bfloat162float(Fp[i]);
            num += (double)fabsf(a - b);
            den += (double)fabsf(b);
        }
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
        num += __shfl_xor_sync(0xFFFFFFFFu, num, m);
        den += __shfl_xor_sync(0xFFFFFFFFu, den, m);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { s_num[warp] = num; s_den[warp] = den; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double tn = 0.0, td = 0.0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { tn += s_num[w]; td += s_den[w]; }
        atomicAdd(terms, tn);
        atomicAdd(terms + 1, td);
    }
}

}  // namespace dvdq
