// Bounded-init Grid Refinement (Alg. 1, Sec. 3.1): the offline 4-bit weight quantizer that
// produces the (W_q, Delta, z) the GEMM consumes.  The objective || W - Delta (W_q - z) ||_F
// with one (Delta, z) per output channel separates over rows, so one CTA owns one row:
//
//   for every shrink step i: clip bounds lo + i*step, hi - i*step -> MinMax grid of the clipped
//   row -> quantize the UNclipped row -> repeat { Delta = <q,w>/<q,q>, z = clamp(round(mean(W_q)
//   - mean(w)/Delta)), W_q = Quant(w; Delta, z) } until the error improves by less than eps;
//   keep the best grid seen.
//
// Every candidate grid costs ONE pass over the row that returns the squared error and the three
// sums the next refinement needs.  The row sits in shared memory as fp32 (its input type); all
// arithmetic and every rounding decision is fp64 (round half to even), as in the fp64 statement
// of the algorithm this is checked against -- it runs once per model, speed is secondary.
#pragma once

#include "dvdq_common.cuh"

namespace dvdq {

constexpr int kBgrThreads = 256;

struct BgrSums {
    double e2, qw, qq, sq;
};

// Deterministic CTA-wide sum of four doubles; every thread receives the totals.
__device__ __forceinline__ BgrSums bgr_block_sum(BgrSums v, double (*scratch)[4]) {
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
        v.e2 += __shfl_xor_sync(0xFFFFFFFFu, v.e2, m);
        v.qw += __shfl_xor_sync(0xFFFFFFFFu, v.qw, m);
        v.qq += __shfl_xor_sync(0xFFFFFFFFu, v.qq, m);
        v.sq += __shfl_xor_sync(0xFFFFFFFFu, v.sq, m);
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();  // the scratch of the previous call has been read
    if (lane == 0) { scratch[warp][0] = v.e2; scratch[warp][1] = v.qw; scratch[warp][2] = v.qq; scratch[warp][3] = v.sq; }
    __syncthreads();
    BgrSums t = {0.0, 0.0, 0.0, 0.0};
    for (int w = 0; w < kBgrThreads / 32; ++w) { t.e2 += scratch[w][0]; t.qw += scratch[w][1]; t.qq += scratch[w][2]; t.sq += scratch[w][3]; }
    return t;
}

// Quant of Sec. 3.1 of the whole row on the grid (d, z): squared error, <q,w>, <q,q>, sum W_q.
__device__ __forceinline__ BgrSums bgr_pass(const float* row, int K, double d, double z, double (*scratch)[4]) {
    BgrSums s = {0.0, 0.0, 0.0, 0.0};
    for (int k = threadIdx.x; k < K; k += kBgrThreads) {
        const double w = (double)row[k];
        double c = rint(w / d) + z;
        c = fmin(fmax(c, 0.0), 15.0);
        const double q = c - z, r = w - d * q;
        s.e2 += r * r; s.qw += q * w; s.qq += q * q; s.sq += c;
    }
    return bgr_block_sum(s, scratch);
}

__global__ void __launch_bounds__(kBgrThreads)
bgr_kernel(const float* __restrict__ W, int K, int n_steps, double eps, int max_iter,
           uint8_t* __restrict__ Wq, float* __restrict__ delta, int32_t* __restrict__ zero) {
    extern __shared__ float s_row[];
    __shared__ double scratch[kBgrThreads / 32][4];
    const float* src = W + (int64_t)blockIdx.x * K;
    // row statistics: min, max, mean (fp64)
    BgrSums st = {0.0, 0.0, 0.0, 0.0};
    double lo = INFINITY, hi = -INFINITY;
    for (int k = threadIdx.x; k < K; k += kBgrThreads) {
        const float v = src[k];
        s_row[k] = v;
        lo = fmin(lo, (double)v);
        hi = fmax(hi, (double)v);
        st.sq += (double)v;
    }
    // min / max through the same reduction: e2 <- -lo, qw <- hi would add, so reduce them apart
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
        lo = fmin(lo, __shfl_xor_sync(0xFFFFFFFFu, lo, m));
        hi = fmax(hi, __shfl_xor_sync(0xFFFFFFFFu, hi, m));
    }
    __shared__ double s_lo[kBgrThreads / 32], s_hi[kBgrThreads / 32];
    if ((threadIdx.x & 31) == 0) { s_lo[threadIdx.x >> 5] = lo; s_hi[threadIdx.x >> 5] = hi; }
    st = bgr_block_sum(st, scratch);  // contains the barriers that publish s_row, s_lo, s_hi
    for (int w = 0; w < kBgrThreads / 32; ++w) { lo = fmin(lo, s_lo[w]); hi = fmax(hi, s_hi[w]); }
    const double mean = st.sq / (double)K;

    double best_e2 = INFINITY, best_d = 1.0, best_z = 0.0;
    const double step = (hi - lo) / (double)n_steps;
    for (int i = 1; 2 * i < n_steps && hi > lo; ++i) {
        const double lo_c = lo + i * step, hi_c = hi - i * step;
        double d = (hi_c - lo_c) / 15.0;
        double z = fmin(fmax(-rint(lo_c / d), 0.0), 15.0);
        BgrSums s = bgr_pass(s_row, K, d, z, scratch);
        double e2 = s.e2;
        if (e2 < best_e2) { best_e2 = e2; best_d = d; best_z = z; }
        for (int j = 1; j <= max_iter; ++j) {
            if (!(s.qq > 0.0) || !(s.qw > 0.0)) break;
            const double d1 = s.qw / s.qq;
            const double z1 = fmin(fmax(rint(s.sq / (double)K - mean / d1), 0.0), 15.0);
            s = bgr_pass(s_row, K, d1, z1, scratch);
            const double improvement = sqrt(e2) - sqrt(s.e2);
            d = d1; z = z1; e2 = s.e2;
            if (e2 < best_e2) { best_e2 = e2; best_d = d; best_z = z; }
            if (improvement < eps) break;
        }
    }
    if (!(best_e2 < INFINITY)) {  // constant row, or fewer than three shrink steps: plain MinMax
        best_d = fabs(hi) > 0.0 ? fabs(hi) : 1.0;
        best_z = 0.0;
        if (hi > lo) { best_d = (hi - lo) / 15.0; best_z = fmin(fmax(-rint(lo / best_d), 0.0), 15.0); }
    }
    for (int k = threadIdx.x; k < K; k += kBgrThreads) {
        const double c = fmin(fmax(rint((double)s_row[k] / best_d) + best_z, 0.0), 15.0);
        Wq[(int64_t)blockIdx.x * K + k] = (uint8_t)c;
    }
    if (threadIdx.x == 0) {
        delta[blockIdx.x] = (float)best_d;
        zero[blockIdx.x] = (int32_t)best_z;
    }
}

}  // namespace dvdq
