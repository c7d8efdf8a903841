// Low-bit GEMM with dequantizing epilogue (Eq. 10, Y = X^ Lambda W^^T; Sec. 3.1 DeQuant): what the
// GEMM kernels share, and the dispatch between them.
//
//   acc_in = sum_k c_ik (u_nk - z_n),   y_in = bf16(acc_in * s_i * Delta_n + bias_n)
//
// All of them are persistent, warp-specialised sm_100a kernels for CTA PAIRS (cluster of two, one
// CTA per SM) that own an output tile of 256 tokens x 256 channels and issue
// tcgen05.mma.cta_group::2.kind::i8 256x256x32 with both operands in shared memory, K in blocks of
// 128 codes; each CTA holds 128 token rows of the activation operand and 128 of the 256 weight rows.
//   qgemm_ss.cuh   one scale per token: activation codes one int8 each (TMA writes the operand stages)
//                  or packed 4 / 6 bits each (widened into the stages by warps, like the weights)
//   qgemm_fat.cuh  block-wise scales, and the epilogue that is the next layer's rotate-quantize
// Each of them either widens the 4-bit weight codes itself, tile by tile, or (handle with an operand:
// dvdq_widen_weights) reads them one int8 each with TMA.
// A 4-bit two's-complement nibble masked into the HIGH half of a byte is the int8 value 16 x code, a
// 6-bit code shifted to the top of a byte is 4 x code; the factor (16 x 16, 4 x 16 or 16 per
// product) is an exact shift of the int32 accumulator in the epilogue.  Weights are stored as
// (u - 8); the rest of the zero point, -(z_n - 8) * sum_k c_ik, is a rank-1 integer correction in
// the epilogue.  Every wait is bounded (see mbar_wait); a role that gives up raises its CTA's abort
// flag and all roles walk to the common exit, where the pair synchronises and tensor memory is released.
#pragma once

#include "dvdq_common.cuh"

namespace dvdq {

constexpr int kBM = 128;            // token rows per CTA (the pair's tile has 2 * kBM)
constexpr int kBK = 128;            // codes per k-block (one widening step + four MMA instructions)
constexpr int kUnpackGroups = 2;    // widening warps come in groups that take alternate k-blocks
constexpr int kTmemCols = 512;

// tanh-form GELU, 0.5 y (1 + tanh(u)) with u = sqrt(2/pi) (y + 0.044715 y^3), written as
// y / (1 + exp(-2u)): one ex2.approx and one rcp.approx (about 1e-6 relative, far below the bf16
// rounding that follows) instead of a full-precision tanhf in an epilogue that has no cycles to spare.
__device__ __forceinline__ float gelu_tanh_f32(float y) {
    const float k = -2.0f * 0.7978845608028654f * 1.4426950408889634f;  // -2 sqrt(2/pi) log2(e)
    const float e = k * y * fmaf(0.044715f, y * y, 1.0f);                // -2u log2(e)
    float t, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(e));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + t));
    return y * r;
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

// bf16 matrix [rows, cols] with row pitch ld elements, tiles of 32 rows x 64 columns, 128-byte
// swizzle (the layout the epilogue stages its output in).
inline bool make_out_map(CUtensorMap* tm, const void* base, uint64_t cols, uint64_t rows, uint64_t ld) {
    PFN_encodeTiled enc = get_encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {64, 32};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Byte matrix [rows, row_len] with row pitch `pitch`, tiles of box_rows x box_bytes with the given
// swizzle (box_bytes equals the swizzle span, or no swizzle); out-of-range bytes read as zero.
inline bool make_byte_map(CUtensorMap* tm, const void* base, uint64_t row_len, uint64_t rows, uint64_t pitch,
                          uint32_t box_bytes, uint32_t box_rows, CUtensorMapSwizzle swizzle) {
    PFN_encodeTiled enc = get_encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {row_len, rows};
    const cuuint64_t strides[1] = {pitch};
    const cuuint32_t box[2] = {box_bytes, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// One-time set-up of a pair kernel on the current device: the opt-in to its dynamic shared memory and
// the number of CTA pairs the device keeps resident at once (one CTA per SM).  0 on failure.
template <typename Kern>
static int resident_pairs(PerDevice<int>& cache, Kern kern, int threads, int smem_bytes) {
    int* mp = cache.get([&](int& max_pairs, int dev) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess) return false;
        int sm_count = 0;
        if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(sm_count & ~1), 1, 1);
        cfg.blockDim = dim3((unsigned)threads, 1, 1);
        cfg.dynamicSmemBytes = (size_t)smem_bytes;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, kern, &cfg) != cudaSuccess || clusters < 1) return false;
        max_pairs = clusters < sm_count / 2 ? clusters : sm_count / 2;
        return true;
    });
    return mp ? *mp : 0;
}

// qgemm_ss.cuh: activation codes stored one int8 per code
template <bool RAW>
static dvdq_status launch_qgemm_ss(const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                   const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy,
                                   int32_t* acc_out, int64_t ldacc, cudaStream_t st);

template <bool RAW>
static dvdq_status launch_qgemm_ps(int bits, const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                   const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy,
                                   int32_t* acc_out, int64_t ldacc, cudaStream_t st);
// qgemm_fat.cuh: the same with block-wise activation scales
static dvdq_status launch_qgemm_blk(int sb, const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                    const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy, cudaStream_t st);

inline dvdq_status launch_qgemm(const void* codes, const float* scales, const int32_t* sums, int64_t M,
                                const dvdq_act_quant& q, const dvdq_weights& w, const void* bias, int act,
                                void* Y, int64_t ldy, int32_t* acc_out, int64_t ldacc, cudaStream_t st) {
    if (M == 0) return DVDQ_OK;
    // The int32 output does not depend on the scales: it always runs the per-token kernel, which
    // adds up the code sums of a token's groups itself.
    const bool raw = acc_out != nullptr;
    const int spr = q.scale_group != 0 ? (int)(w.K / q.scale_group) : 1;  // code sums (and scales) per token
    const int sb = storage_bits(q);
    if (sb != 4 && sb != 6 && sb != 8) return DVDQ_ERR_BITS;
    if (!raw && q.scale_group != 0) return launch_qgemm_blk(sb, codes, scales, sums, spr, M, w, bias, act, Y, ldy, st);
    if (sb == 8)
        return raw ? launch_qgemm_ss<true>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st)
                   : launch_qgemm_ss<false>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st);
    return raw ? launch_qgemm_ps<true>(sb, codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st)
               : launch_qgemm_ps<false>(sb, codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st);
}

}  // namespace dvdq
