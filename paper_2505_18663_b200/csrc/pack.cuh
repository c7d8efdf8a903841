// Format helpers: offline weight packing (Sec. 3.1 Quant/DeQuant format -> device blob) and the
// test/debug converters between natural-order int8 codes and the packed activation layout.
#pragma once

#include "dvdq_common.cuh"

namespace dvdq {

// One thread per output byte: storage positions 2t and 2t+1 of row n.  The stored nibble is
// (u - 8) in two's complement, i.e. u ^ 8, so that the GEMM can widen it with a mask; the
// remaining (8 - z_n) of the zero point is applied in the epilogue from the token's code sum.
__global__ void pack_weights_kernel(const uint8_t* __restrict__ Wq, const float* __restrict__ delta,
                                    const int32_t* __restrict__ zero, int64_t N, int64_t K, int32_t rot_block,
                                    int32_t k_layout, uint8_t* __restrict__ blob) {
    const BlobLayout L = blob_layout(N, K);
    const int64_t half = K / 2;
    const int64_t total = N * half;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t n = t / half, b = t - n * half;
        const uint32_t u0 = Wq[n * K + 2 * b] & 0xFu, u1 = Wq[n * K + 2 * b + 1] & 0xFu;
        blob[L.codes_offset + t] = (uint8_t)((u0 ^ 8u) | ((u1 ^ 8u) << 4));
    }
    for (int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; n < N; n += (int64_t)gridDim.x * blockDim.x) {
        reinterpret_cast<float*>(blob + L.delta_offset)[n] = delta[n];
        reinterpret_cast<int32_t*>(blob + L.zc_offset)[n] = zero[n] - 8;
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        BlobHeader h;
        h.magic = kBlobMagic; h.version = kBlobVersion; h.N = N; h.K = K;
        h.rot_block = rot_block; h.k_layout = k_layout;
        h.codes_offset = L.codes_offset; h.delta_offset = L.delta_offset; h.zc_offset = L.zc_offset;
        *reinterpret_cast<BlobHeader*>(blob) = h;
    }
}

__global__ void unpack_weights_kernel(const uint8_t* __restrict__ blob, int64_t N, int64_t K,
                                      uint8_t* __restrict__ Wq, float* __restrict__ delta, int32_t* __restrict__ zero) {
    const BlobLayout L = blob_layout(N, K);
    const int64_t half = K / 2, total = N * half;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t n = t / half, b = t - n * half;
        const uint32_t v = blob[L.codes_offset + t];
        Wq[n * K + 2 * b] = (uint8_t)((v & 0xFu) ^ 8u);
        Wq[n * K + 2 * b + 1] = (uint8_t)((v >> 4) ^ 8u);
    }
    for (int64_t n = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; n < N; n += (int64_t)gridDim.x * blockDim.x) {
        delta[n] = reinterpret_cast<const float*>(blob + L.delta_offset)[n];
        zero[n] = reinterpret_cast<const int32_t*>(blob + L.zc_offset)[n] + 8;
    }
}

// One thread per group of 16 positions of one token row.
template <int BITS>
__global__ void pack_act_codes_kernel(const int8_t* __restrict__ nat, int64_t M, int64_t K, uint8_t* __restrict__ packed) {
    const int64_t groups = K / 16, total = M * groups;
    const int64_t row_bytes = act_row_bytes(K, BITS);
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = t / groups, m = t - i * groups;
        const int8_t* src = nat + i * K + m * 16;
        uint8_t* row = packed + i * row_bytes;
        if (BITS == 8) {  // per 8 channels: the four even channels, then the four odd ones
            for (int a = 0; a < 2; ++a)
                for (int j = 0; j < 8; ++j) row[m * 16 + 8 * a + 4 * (j & 1) + (j >> 1)] = (uint8_t)src[8 * a + j];
            continue;
        }
        uint32_t lo[2] = {0u, 0u}, hi = 0u;
        for (int a = 0; a < 2; ++a)
            for (int j = 0; j < 8; ++j) {
                const uint32_t c = (uint32_t)(int32_t)src[8 * a + j];
                lo[a] |= (c & 0xFu) << (4 * j);
                hi |= ((c >> 4) & 0x3u) << hi_field_shift(a, j);
            }
        reinterpret_cast<uint32_t*>(row)[2 * m] = lo[0];
        reinterpret_cast<uint32_t*>(row)[2 * m + 1] = lo[1];
        if (BITS == 6) reinterpret_cast<uint32_t*>(row + K / 2)[m] = hi;
    }
}

template <int BITS>
__global__ void unpack_act_codes_kernel(const uint8_t* __restrict__ packed, int64_t M, int64_t K, int8_t* __restrict__ nat) {
    const int64_t groups = K / 16, total = M * groups;
    const int64_t row_bytes = act_row_bytes(K, BITS);
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = t / groups, m = t - i * groups;
        const uint8_t* row = packed + i * row_bytes;
        if (BITS == 8) {
            for (int a = 0; a < 2; ++a)
                for (int j = 0; j < 8; ++j) nat[i * K + m * 16 + 8 * a + j] = (int8_t)row[m * 16 + 8 * a + 4 * (j & 1) + (j >> 1)];
            continue;
        }
        const uint32_t lo[2] = {reinterpret_cast<const uint32_t*>(row)[2 * m], reinterpret_cast<const uint32_t*>(row)[2 * m + 1]};
        const uint32_t hi = (BITS == 6) ? reinterpret_cast<const uint32_t*>(row + K / 2)[m] : 0u;
        for (int a = 0; a < 2; ++a)
            for (int j = 0; j < 8; ++j) {
                uint32_t c = (lo[a] >> (4 * j)) & 0xFu;
                int32_t val;
                if (BITS == 6) {
                    c |= ((hi >> hi_field_shift(a, j)) & 0x3u) << 4;
                    val = (int32_t)(c << 26) >> 26;
                } else {
                    val = (int32_t)(c << 28) >> 28;
                }
                nat[i * K + m * 16 + 8 * a + j] = (int8_t)val;
            }
    }
}

// One warp per (token, block): sum of the codes of `block` consecutive channels (block = K for
// the per-token variant).
__global__ void code_sums_kernel(const int8_t* __restrict__ nat, int64_t M, int64_t K, int64_t block,
                                 int32_t* __restrict__ sums) {
    const int lane = threadIdx.x & 31;
    const int64_t unit = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t per_row = K / block;
    if (unit >= M * per_row) return;
    const int64_t row = unit / per_row, blk = unit - row * per_row;
    int s = 0;
    for (int64_t k = lane; k < block; k += 32) s += nat[row * K + blk * block + k];
    for (int m = 16; m > 0; m >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, m);
    if (lane == 0) sums[unit] = s;
}

inline unsigned grid_for(int64_t work, int threads) {
    int64_t g = (work + threads - 1) / threads;
    if (g < 1) g = 1;
    if (g > 148 * 32) g = 148 * 32;
    return (unsigned)g;
}

}  // namespace dvdq
