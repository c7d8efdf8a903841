// Offline weight preparation on the GPU (Eq. 10, W^ = Quant(W H); Sec. 3.1 Quant/DeQuant format):
// the rotation W~ = W R along K, and the plain symmetric 4-bit quantizer written straight into
// the packed blob.  Both run once per model, so everything is fp64: the butterflies of a block
// add and subtract bf16 values, which fp64 does without rounding for any realistic exponent
// spread, and the 1/sqrt(B) factor is one multiplication (exact when log2 B is even).  The
// result then agrees with a dense fp64 product bit for bit for B in {64, 256, 1024, 4096} and to
// the last fp64 bit otherwise.
#pragma once

#include "dvdq_common.cuh"

namespace dvdq {

constexpr int kWeightThreads = 512;

// The row of W (bf16, K entries) into shared memory as fp64, transformed block by block:
// log2b butterfly stages, then the orthonormal factor.  All threads of the CTA take part.
__device__ __forceinline__ void rotate_row_fp64(const __nv_bfloat16* __restrict__ w, int K, int log2b, double* s) {
    for (int k = threadIdx.x; k < K; k += blockDim.x) s[k] = (double)__bfloat162float(w[k]);
    __syncthreads();
    for (int st = 0; st < log2b; ++st) {
        const int h = 1 << st;
        for (int p = threadIdx.x; p < K / 2; p += blockDim.x) {
            const int i = ((p >> st) << (st + 1)) | (p & (h - 1));
            const double a = s[i], b = s[i + h];
            s[i] = a + b;
            s[i + h] = a - b;
        }
        __syncthreads();
    }
    if (log2b > 0) {
        const double rs = 1.0 / sqrt((double)(1 << log2b));
        for (int k = threadIdx.x; k < K; k += blockDim.x) s[k] *= rs;
        __syncthreads();
    }
}

// One CTA per output channel: W~[n, :] as fp32 (the input type of the grid-refinement quantizer).
__global__ void rotate_weights_kernel(const __nv_bfloat16* __restrict__ W, int64_t ldw, int K, int log2b,
                                      float* __restrict__ out) {
    extern __shared__ double s_wrow[];
    const int64_t n = blockIdx.x;
    rotate_row_fp64(W + n * ldw, K, log2b, s_wrow);
    for (int k = threadIdx.x; k < K; k += blockDim.x) out[n * (int64_t)K + k] = (float)s_wrow[k];
}

// One CTA per output channel: rotate, Delta_n = max_k |w~_nk| / 7, q = clamp(rne(w~ / Delta), -8, 7),
// stored nibble q (= u - 8 with u = q + 8 and z = 8), Delta as fp32, zero-point rest 0.
__global__ void quantize_weights_symmetric_kernel(const __nv_bfloat16* __restrict__ W, int64_t ldw, int64_t N, int K,
                                                  int log2b, int32_t rot_block, uint8_t* __restrict__ blob) {
    extern __shared__ double s_wrow[];
    __shared__ double s_red[kWeightThreads / 32];
    const int64_t n = blockIdx.x;
    const BlobLayout L = blob_layout(N, K);
    rotate_row_fp64(W + n * ldw, K, log2b, s_wrow);
    double a = 0.0;
    for (int k = threadIdx.x; k < K; k += blockDim.x) a = fmax(a, fabs(s_wrow[k]));
    for (int m = 16; m > 0; m >>= 1) a = fmax(a, __shfl_xor_sync(0xFFFFFFFFu, a, m));
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = a;
    __syncthreads();
    a = 0.0;
    for (int w = 0; w < kWeightThreads / 32; ++w) a = fmax(a, s_red[w]);
    double d = a / 7.0;
    if (!(d > 0.0)) d = 1.0;  // an all-zero row: any step size reproduces it
    uint8_t* row = blob + L.codes_offset + n * (int64_t)(K / 2);
    for (int t = threadIdx.x; t < K / 2; t += blockDim.x) {
        double q0 = rint(s_wrow[2 * t] / d), q1 = rint(s_wrow[2 * t + 1] / d);
        q0 = fmin(fmax(q0, -8.0), 7.0);
        q1 = fmin(fmax(q1, -8.0), 7.0);
        row[t] = (uint8_t)(((int)q0 & 0xF) | (((int)q1 & 0xF) << 4));
    }
    if (threadIdx.x == 0) {
        reinterpret_cast<float*>(blob + L.delta_offset)[n] = (float)d;
        reinterpret_cast<int32_t*>(blob + L.zc_offset)[n] = 0;
        if (n == 0) {
            BlobHeader h;
            h.magic = kBlobMagic; h.version = kBlobVersion; h.N = N; h.K = K;
            h.rot_block = rot_block; h.k_layout = kKLayoutNatural;
            h.codes_offset = L.codes_offset; h.delta_offset = L.delta_offset; h.zc_offset = L.zc_offset;
            *reinterpret_cast<BlobHeader*>(blob) = h;
        }
    }
}

// The packed 4-bit codes of a blob as the GEMM's weight operand: one int8 per code holding 16 x (u - 8)
// (the nibble in the high half of the byte), in the K order in which the GEMM's warps would write
// them into a shared-memory stage: the 32 codes of a 16-byte piece become, word by word, the four
// even-numbered codes then the four odd-numbered ones.  A thread per piece, grid-stride.
__global__ void widen_weights_kernel(const uint8_t* __restrict__ packed, int64_t pieces, uint8_t* __restrict__ operand) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < pieces; i += (int64_t)gridDim.x * blockDim.x) {
        const uint4 p = __ldg(reinterpret_cast<const uint4*>(packed) + i);
        const uint32_t w[4] = {p.x, p.y, p.z, p.w};
        uint32_t e[4], o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { e[j] = (w[j] << 4) & 0xF0F0F0F0u; o[j] = w[j] & 0xF0F0F0F0u; }
        uint4* dst = reinterpret_cast<uint4*>(operand) + 2 * i;
        dst[0] = make_uint4(e[0], o[0], e[1], o[1]);
        dst[1] = make_uint4(e[2], o[2], e[3], o[3]);
    }
}

// The opt-in of a weight kernel to a whole row of fp64 in shared memory, once per device.
template <typename Kern>
static bool weight_kernel_setup(PerDevice<int>& cache, Kern kern) {
    return cache.get([&](int&, int) {
        return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 16384 * (int)sizeof(double)) == cudaSuccess;
    }) != nullptr;
}

}  // namespace dvdq
