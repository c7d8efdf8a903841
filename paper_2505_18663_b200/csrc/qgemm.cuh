// Low-bit GEMM with dequantizing epilogue (Eq. 10, Y = X^ Lambda W^^T; Sec. 3.1 DeQuant).
//
//   acc_in = sum_k c_ik (u_nk - z_n),   y_in = bf16(acc_in * s_i * Delta_n + bias_n)
//
// Persistent, warp-specialised sm_100a kernel, one CTA per SM, output tile 128 tokens x 256
// channels, K consumed in blocks of 128 codes:
//
//   warp 0      TMA producer: packed 4/6-bit activation rows and packed 4-bit weight rows
//               -> shared memory ring (kPackedStages deep), completion on mbarriers.
//   warps 6-13  widen the codes to int8 in shared memory, straight into the 128-byte-swizzled
//               K-major layout tcgen05.mma reads.  A 4-bit two's-complement nibble masked into
//               the HIGH half of a byte is the int8 value 16*code, a 6-bit code shifted to the
//               top of a byte is 4*code; the factor (256 or 64 per product) is an exact shift
//               of the int32 accumulator in the epilogue.  Weights are stored as (u - 8); the
//               rest of the zero point, -(z_n - 8) * sum_k c_ik, is a rank-1 integer correction
//               in the epilogue, so the mainloop never subtracts per-row constants.
//   warp 1      one thread issues tcgen05.mma kind::i8 (128x256x32 per instruction) into one of
//               two 256-column int32 accumulators in tensor memory; tcgen05.commit frees the
//               widened stage and publishes the finished accumulator.
//   warps 2-5   epilogue: tcgen05.ld, shift, zero-point correction, scale, bias, optional
//               tanh-GELU, one bf16 rounding, 16-byte stores.  Runs concurrently with the next
//               tile's mainloop thanks to the second accumulator.
//
// Every wait is bounded (see mbar_wait); a role that gives up raises a shared abort flag and
// all roles walk to the common exit, where tensor memory is released.
#pragma once

#include "dvdq_common.cuh"

namespace dvdq {

constexpr int kBM = 128, kBN = 256, kBK = 128;
constexpr int kWideStages = 2;
constexpr int kUnpackWarps = 8, kEpilogueWarps = 4;
constexpr int kFirstEpilogueWarp = 2, kFirstUnpackWarp = 6;
constexpr int kGemmThreads = (2 + kEpilogueWarps + kUnpackWarps) * 32;
constexpr int kTmemCols = 512;

template <int BITS>
struct GemmSmem {
    static constexpr int kPackedStages = (BITS == 4) ? 4 : 3;     // what fits beside the other buffers
    static constexpr int kALo = kBM * kBK / 2;                    // packed low plane / A4 codes
    static constexpr int kAHi = (BITS == 6) ? kBM * kBK / 4 : 0;  // packed high plane
    static constexpr int kW = kBN * kBK / 2;
    static constexpr int kPackedStage = kALo + kAHi + kW;
    static constexpr int kWideA = kBM * kBK, kWideW = kBN * kBK;
    static constexpr int kWideStage = kWideA + kWideW;
    static constexpr int kWideOff = 0;  // 1024-byte aligned tiles first
    static constexpr int kPackedOff = kWideOff + kWideStages * kWideStage;
    static constexpr int kStageOutOff = kPackedOff + kPackedStages * kPackedStage;  // 1024-byte aligned
    static constexpr int kStageOutPerWarp = 2 * 32 * 64;  // two buffers of 32 rows x 32 bf16
    static constexpr int kConstOff = kStageOutOff + kEpilogueWarps * kStageOutPerWarp;
    static constexpr int kConstPerWarp = 3 * kBN * 4;  // delta, zero-point rest, bias for 256 channels
    static constexpr int kBarOff = kConstOff + kEpilogueWarps * kConstPerWarp;
    static constexpr int kNumBars = 2 * kPackedStages + 2 * kWideStages + 4;
    static constexpr int kMiscOff = kBarOff + kNumBars * 8;
    static constexpr int kTotal = kMiscOff + 16 + 1024;  // + slack for manual 1024-byte alignment
};

__device__ __forceinline__ float gelu_tanh_f32(float y) {
    const float c = 0.7978845608028654f;
    return 0.5f * y * (1.0f + tanhf(c * (y + 0.044715f * y * y * y)));
}

template <int BITS, bool RAW>
__global__ void __launch_bounds__(kGemmThreads, 1)
qgemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmAhi,
             const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmY,
             const float* __restrict__ scales,
             const int32_t* __restrict__ sums, const float* __restrict__ delta, const int32_t* __restrict__ zc,
             const __nv_bfloat16* __restrict__ bias, __nv_bfloat16* __restrict__ Y, int64_t ldy,
             int32_t* __restrict__ acc_out, int64_t ldacc, int M, int N, int K, int act) {
    using S = GemmSmem<BITS>;
    constexpr int kPackedStages = S::kPackedStages;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_n = (N + kBN - 1) / kBN, num_m = (M + kBM - 1) / kBM;
    const int num_tiles = num_m * num_n;
    const int KB = (K + kBK - 1) / kBK;

    const uint32_t bar0 = sbase + S::kBarOff;
    auto pk_full = [&](int s) { return bar0 + 8u * s; };
    auto pk_empty = [&](int s) { return bar0 + 8u * (kPackedStages + s); };
    auto wd_full = [&](int s) { return bar0 + 8u * (2 * kPackedStages + s); };
    auto wd_empty = [&](int s) { return bar0 + 8u * (2 * kPackedStages + kWideStages + s); };
    auto acc_full = [&](int s) { return bar0 + 8u * (2 * kPackedStages + 2 * kWideStages + s); };
    auto acc_empty = [&](int s) { return bar0 + 8u * (2 * kPackedStages + 2 * kWideStages + 2 + s); };
    volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + S::kMiscOff);  // [0] tmem base, [1] abort
    volatile uint32_t* abort_flag = misc + 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPackedStages; ++s) { mbar_init(pk_full(s), 1); mbar_init(pk_empty(s), kUnpackWarps); }
        for (int s = 0; s < kWideStages; ++s) { mbar_init(wd_full(s), kUnpackWarps); mbar_init(wd_empty(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full(s), 1); mbar_init(acc_empty(s), kEpilogueWarps); }
        misc[1] = 0u;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(sbase + S::kMiscOff, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = misc[0];

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&tmA);
            if (BITS == 6) tma_prefetch_desc(&tmAhi);
            tma_prefetch_desc(&tmW);
            uint32_t st = 0, ph = 0, issued = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
                const int m0 = (tile / num_n) * kBM, n0 = (tile % num_n) * kBN;
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(pk_empty(st), ph ^ 1u, abort_flag, kWaitPackedEmpty)) { ok = false; break; }
                    const uint32_t dst = sbase + S::kPackedOff + st * S::kPackedStage;
                    mbar_arrive_expect_tx(pk_full(st), S::kPackedStage);
                    tma_load_2d(dst, &tmA, pk_full(st), kb * (kBK / 2), m0);
                    if (BITS == 6) tma_load_2d(dst + S::kALo, &tmAhi, pk_full(st), kb * (kBK / 4), m0);
                    tma_load_2d(dst + S::kALo + S::kAHi, &tmW, pk_full(st), kb * (kBK / 2), n0);
                    ++issued;
                    if (++st == kPackedStages) { st = 0; ph ^= 1u; }
                }
            }
            if (!ok) {
                // Giving up: let copies already in flight land before the CTA exits (bounded).
                const uint32_t n_out = issued < (uint32_t)kPackedStages ? issued : (uint32_t)kPackedStages;
                for (uint32_t i = 0; i < n_out; ++i) {
                    const uint32_t s = (st + kPackedStages - 1 - i) % kPackedStages;
                    const uint32_t p = (s < st) ? ph : (ph ^ 1u);
                    for (int it = 0; it < (1 << 16) && !mbar_try_wait(pk_full(s), p); ++it) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_s8s8s32(kBM, kBN);
            uint32_t st = 0, ph = 0, lt = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x, ++lt) {
                const uint32_t a = lt & 1u, aph = (lt >> 1) & 1u;
                if (!mbar_wait(acc_empty(a), aph ^ 1u, abort_flag, kWaitAccEmpty)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + a * kBN;
                for (int kb = 0; kb < KB; ++kb) {
                    if (!mbar_wait(wd_full(st), ph, abort_flag, kWaitWideFull)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t wa = sbase + S::kWideOff + st * S::kWideStage;
                    const uint64_t adesc = umma_desc_sw128_kmajor(wa);
                    const uint64_t bdesc = umma_desc_sw128_kmajor(wa + S::kWideA);
#pragma unroll
                    for (int k = 0; k < kBK / 32; ++k)  // +32 bytes along K = +2 in the 16-byte address field
                        tc_mma_i8_ss(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    tc_commit(wd_empty(st));
                    if (++st == kWideStages) { st = 0; ph ^= 1u; }
                }
                if (ok) tc_commit(acc_full(a));
            }
        }
        __syncwarp();
    } else if (warp < kFirstUnpackWarp) {
        // ------------------------------------------------------------ epilogue
        const int q = warp & 3;  // tensor-memory lane quarter this warp may read
        const int ew = warp - kFirstEpilogueWarp;
        float* c_delta = reinterpret_cast<float*>(smem + S::kConstOff + ew * S::kConstPerWarp);
        float* c_zc = c_delta + kBN;    // (z_n - 8) as a float: exact, |.| <= 8
        float* c_bias = c_zc + kBN;
        const uint32_t stg0 = sbase + S::kStageOutOff + ew * S::kStageOutPerWarp;
        uint8_t* stg_ptr = smem + S::kStageOutOff + ew * S::kStageOutPerWarp;
        constexpr int kShift = (BITS == 4) ? 8 : 6;
        if (!RAW && lane == 0) tma_prefetch_desc(&tmY);
        uint32_t lt = 0, nstore = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x, ++lt) {
            const uint32_t a = lt & 1u, aph = (lt >> 1) & 1u;
            const int m0 = (tile / num_n) * kBM, n0 = (tile % num_n) * kBN;
            __syncwarp();
            for (int c = lane; c < kBN; c += 32) {
                const int n = n0 + c;
                const bool okn = n < N;
                c_delta[c] = okn ? delta[n] : 0.f;
                c_zc[c] = okn ? (float)zc[n] : 0.f;
                c_bias[c] = (okn && bias != nullptr) ? __bfloat162float(bias[n]) : 0.f;
            }
            __syncwarp();
            if (!mbar_wait(acc_full(a), aph, abort_flag, kWaitAccFull)) break;
            tc_fence_after();
            const int row = m0 + q * 32 + lane;
            const bool row_ok = row < M;
            const float s_i = (!RAW && row_ok) ? scales[row] : 0.f;
            const int32_t S_i = row_ok ? sums[row] : 0;
            const float S_f = (float)S_i;  // |sum of codes| <= K * 32 < 2^24: exact
#pragma unroll 1
            for (int c = 0; c < kBN / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + a * kBN + c * 32 + ((uint32_t)(q * 32) << 16), r);
                tmem_ld_wait();
                const int nb = n0 + c * 32;
                if (RAW) {
                    int32_t* dst = acc_out + (int64_t)row * ldacc + nb;
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        int4 o;
                        o.x = ((int32_t)r[j] >> kShift) - __float2int_rn(c_zc[c * 32 + j]) * S_i;
                        o.y = ((int32_t)r[j + 1] >> kShift) - __float2int_rn(c_zc[c * 32 + j + 1]) * S_i;
                        o.z = ((int32_t)r[j + 2] >> kShift) - __float2int_rn(c_zc[c * 32 + j + 2]) * S_i;
                        o.w = ((int32_t)r[j + 3] >> kShift) - __float2int_rn(c_zc[c * 32 + j + 3]) * S_i;
                        if (row_ok && nb + j < N) *reinterpret_cast<int4*>(dst + j) = o;
                    }
                } else {
                    // The staging buffer used two chunks ago must have been read by its TMA store.
                    if (lane == 0) tma_store_wait_read<1>();
                    __syncwarp();
                    uint8_t* buf = stg_ptr + (nstore & 1u) * (32 * 64);
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        const float4 d0 = *reinterpret_cast<const float4*>(c_delta + c * 32 + j);
                        const float4 d1 = *reinterpret_cast<const float4*>(c_delta + c * 32 + j + 4);
                        const float4 z0 = *reinterpret_cast<const float4*>(c_zc + c * 32 + j);
                        const float4 z1 = *reinterpret_cast<const float4*>(c_zc + c * 32 + j + 4);
                        const float4 b0 = *reinterpret_cast<const float4*>(c_bias + c * 32 + j);
                        const float4 b1 = *reinterpret_cast<const float4*>(c_bias + c * 32 + j + 4);
                        const float dl[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
                        const float zz[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
                        const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                        float v[8];
#pragma unroll
                        for (int t = 0; t < 8; ++t) {
                            // int -> float without the conversion pipe: |acc >> shift| <= K*32*8 <= 2^22
                            const int32_t sh = (int32_t)r[j + t] >> kShift;
                            float f = __int_as_float(sh + 0x4B400000) - 12582912.0f;
                            f = fmaf(-zz[t], S_f, f);                 // rest of the zero point, exact
                            float y = fmaf(f, s_i * dl[t], bb[t]);
                            if (act == 1) y = gelu_tanh_f32(__bfloat162float(__float2bfloat16_rn(y)));
                            v[t] = y;
                        }
                        uint32_t pk[4];
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            __nv_bfloat162 b2 = __floats2bfloat162_rn(v[2 * t], v[2 * t + 1]);
                            pk[t] = *reinterpret_cast<uint32_t*>(&b2);
                        }
                        // 64-byte rows, 16-byte chunk index XORed with (row >> 1) & 3: the layout a
                        // 64B-swizzled TMA store reads, and conflict-free for this per-row write.
                        const int ch = (j >> 3) ^ ((lane >> 1) & 3);
                        *reinterpret_cast<uint4*>(buf + lane * 64 + ch * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0 && nb < N && m0 + q * 32 < M) {
                        tma_store_2d(&tmY, stg0 + (nstore & 1u) * (32 * 64), nb, m0 + q * 32);
                        tma_store_commit();
                    }
                    ++nstore;
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(a));
        }
        if (!RAW && lane == 0) tma_store_wait_all();
        __syncwarp();
    } else {
        // ------------------------------------------------------------ widen 4/6-bit codes to int8
        const int u = threadIdx.x - kFirstUnpackWarp * 32;  // 0..255
        uint32_t pst = 0, pph = 0, wst = 0, wph = 0;
        bool ok = true;
        for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
            for (int kb = 0; kb < KB; ++kb) {
                if (!mbar_wait(pk_full(pst), pph, abort_flag, kWaitPackedFull)) { ok = false; break; }
                if (!mbar_wait(wd_empty(wst), wph ^ 1u, abort_flag, kWaitWideEmpty)) { ok = false; break; }
                tc_fence_after();
                const uint8_t* pk = smem + S::kPackedOff + pst * S::kPackedStage;
                uint8_t* wdA = smem + S::kWideOff + wst * S::kWideStage;
                uint8_t* wdW = wdA + S::kWideA;
                // activation tile: 128 rows x 4 chunks of 32 codes
#pragma unroll
                for (int it = 0; it < (kBM * 4) / 256; ++it) {
                    const int qi = it * 256 + u, row = qi >> 2, ck = qi & 3;
                    const uint4 p = *reinterpret_cast<const uint4*>(pk + row * (kBK / 2) + ck * 16);
                    const uint32_t w[4] = {p.x, p.y, p.z, p.w};
                    uint32_t e[4], o[4];
                    if (BITS == 4) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) { e[j] = (w[j] << 4) & 0xF0F0F0F0u; o[j] = w[j] & 0xF0F0F0F0u; }
                    } else {
                        const uint2 hp = *reinterpret_cast<const uint2*>(pk + S::kALo + row * (kBK / 4) + ck * 8);
                        const uint32_t h[2] = {hp.x, hp.y};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t hh = h[j >> 1];
                            const int a2 = 2 * (j & 1);
                            e[j] = ((w[j] << 2) & 0x3C3C3C3Cu) | ((hh << (6 - 2 * a2)) & 0xC0C0C0C0u);
                            o[j] = ((w[j] >> 2) & 0x3C3C3C3Cu) | ((hh << (4 - 2 * a2)) & 0xC0C0C0C0u);
                        }
                    }
                    uint8_t* drow = wdA + (row >> 3) * 1024 + (row & 7) * 128;
                    *reinterpret_cast<uint4*>(drow + (((2 * ck) ^ (row & 7)) << 4)) = make_uint4(e[0], o[0], e[1], o[1]);
                    *reinterpret_cast<uint4*>(drow + (((2 * ck + 1) ^ (row & 7)) << 4)) = make_uint4(e[2], o[2], e[3], o[3]);
                }
                // weight tile: 256 rows x 4 chunks of 32 nibbles, stored as (u - 8)
                const uint8_t* pw = pk + S::kALo + S::kAHi;
#pragma unroll
                for (int it = 0; it < (kBN * 4) / 256; ++it) {
                    const int qi = it * 256 + u, row = qi >> 2, ck = qi & 3;
                    const uint4 p = *reinterpret_cast<const uint4*>(pw + row * (kBK / 2) + ck * 16);
                    const uint32_t w[4] = {p.x, p.y, p.z, p.w};
                    uint32_t e[4], o[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) { e[j] = (w[j] << 4) & 0xF0F0F0F0u; o[j] = w[j] & 0xF0F0F0F0u; }
                    uint8_t* drow = wdW + (row >> 3) * 1024 + (row & 7) * 128;
                    *reinterpret_cast<uint4*>(drow + (((2 * ck) ^ (row & 7)) << 4)) = make_uint4(e[0], o[0], e[1], o[1]);
                    *reinterpret_cast<uint4*>(drow + (((2 * ck + 1) ^ (row & 7)) << 4)) = make_uint4(e[2], o[2], e[3], o[3]);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) { mbar_arrive(wd_full(wst)); mbar_arrive(pk_empty(pst)); }
                if (++pst == kPackedStages) { pst = 0; pph ^= 1u; }
                if (++wst == kWideStages) { wst = 0; wph ^= 1u; }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// ------------------------------------------------------------------ host side

typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline PFN_encodeTiled get_encode_tiled() {
    static PFN_encodeTiled fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_encodeTiled>(p);
    }
    return fn;
}

// Byte matrix [rows, row_len] with row pitch `pitch`, tiles of box_rows x box_bytes, no swizzle,
// out-of-range bytes read as zero.
// bf16 matrix [rows, cols] with row pitch ld elements, tiles of 32 x 32, 64-byte swizzle
// (the layout the epilogue stages its output in).
inline bool make_out_map(CUtensorMap* tm, const void* base, uint64_t cols, uint64_t rows, uint64_t ld) {
    PFN_encodeTiled enc = get_encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline bool make_byte_map(CUtensorMap* tm, const void* base, uint64_t row_len, uint64_t rows, uint64_t pitch,
                          uint32_t box_bytes, uint32_t box_rows) {
    PFN_encodeTiled enc = get_encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {row_len, rows};
    const cuuint64_t strides[1] = {pitch};
    const cuuint32_t box[2] = {box_bytes, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BITS, bool RAW>
static dvdq_status launch_qgemm_t(const void* codes, const float* scales, const int32_t* sums, int64_t M,
                                  const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy,
                                  int32_t* acc_out, int64_t ldacc, cudaStream_t st) {
    using S = GemmSmem<BITS>;
    const int64_t K = w.K, N = w.N;
    const BlobLayout L = blob_layout(N, K);
    const uint8_t* blob = static_cast<const uint8_t*>(w.blob);
    const uint64_t pitch = (uint64_t)act_row_bytes(K, BITS);
    CUtensorMap tmA, tmAhi, tmW, tmY;
    if (!make_byte_map(&tmA, codes, (uint64_t)K / 2, (uint64_t)M, pitch, kBK / 2, kBM)) return DVDQ_ERR_CUDA;
    if (BITS == 6) {
        if (!make_byte_map(&tmAhi, static_cast<const uint8_t*>(codes) + K / 2, (uint64_t)K / 4, (uint64_t)M, pitch, kBK / 4, kBM))
            return DVDQ_ERR_CUDA;
    } else {
        tmAhi = tmA;
    }
    if (!make_byte_map(&tmW, blob + L.codes_offset, (uint64_t)K / 2, (uint64_t)N, (uint64_t)K / 2, kBK / 2, kBN)) return DVDQ_ERR_CUDA;

    if (RAW) {
        tmY = tmA;  // unused
    } else if (!make_out_map(&tmY, Y, (uint64_t)N, (uint64_t)M, (uint64_t)ldy)) {
        return DVDQ_ERR_CUDA;
    }

    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return DVDQ_ERR_CUDA;
        if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return DVDQ_ERR_CUDA;
    }
    auto kern = qgemm_kernel<BITS, RAW>;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kTotal) != cudaSuccess) return DVDQ_ERR_CUDA;
        attr_set = true;
    }
    const int64_t tiles = ((M + kBM - 1) / kBM) * ((N + kBN - 1) / kBN);
    const unsigned grid = (unsigned)(tiles < sm_count ? tiles : sm_count);
    kern<<<grid, kGemmThreads, S::kTotal, st>>>(tmA, tmAhi, tmW, tmY, scales, sums,
                                                reinterpret_cast<const float*>(blob + L.delta_offset),
                                                reinterpret_cast<const int32_t*>(blob + L.zc_offset),
                                                static_cast<const __nv_bfloat16*>(bias), static_cast<__nv_bfloat16*>(Y), ldy,
                                                acc_out, ldacc, (int)M, (int)N, (int)K, act);
    return cuda_status(cudaGetLastError());
}

inline dvdq_status launch_qgemm(const void* codes, const float* scales, const int32_t* sums, int64_t M,
                                const dvdq_act_quant& q, const dvdq_weights& w, const void* bias, int act,
                                void* Y, int64_t ldy, int32_t* acc_out, int64_t ldacc, cudaStream_t st) {
    if (M == 0) return DVDQ_OK;
    const bool raw = acc_out != nullptr;
    if (q.bits == 4)
        return raw ? launch_qgemm_t<4, true>(codes, scales, sums, M, w, bias, act, Y, ldy, acc_out, ldacc, st)
                   : launch_qgemm_t<4, false>(codes, scales, sums, M, w, bias, act, Y, ldy, acc_out, ldacc, st);
    return raw ? launch_qgemm_t<6, true>(codes, scales, sums, M, w, bias, act, Y, ldy, acc_out, ldacc, st)
               : launch_qgemm_t<6, false>(codes, scales, sums, M, w, bias, act, Y, ldy, acc_out, ldacc, st);
}

}  // namespace dvdq
