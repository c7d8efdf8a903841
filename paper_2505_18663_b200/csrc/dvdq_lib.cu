// C ABI of the library (see include/dvdq.h): argument validation, size queries and the
// launches of the kernels in rotate_quantize.cuh, pack.cuh, weights.cuh, qgemm.cuh and
// qgemm_ss.cuh.  One translation unit, so that the device status word is a single symbol.
#include "dvdq_common.cuh"

#include "bgr.cuh"
#include "gbs.cuh"
#include "pack.cuh"
#include "qgemm.cuh"
#include "qgemm_ss.cuh"
#include "qgemm_fat.cuh"
#include "rotate_quantize.cuh"
#include "weights.cuh"
#include "diag.cuh"

namespace dvdq {

dvdq_status cuda_status(cudaError_t e) { return e == cudaSuccess ? DVDQ_OK : DVDQ_ERR_CUDA; }

dvdq_status check_device_arch() {
    static PerDevice<int> cache;  // compute-capability major of each device
    int* major = cache.get([](int& m, int dev) {
        return cudaDeviceGetAttribute(&m, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess;
    });
    if (!major) return DVDQ_ERR_CUDA;
    return *major == 10 ? DVDQ_OK : DVDQ_ERR_ARCH;
}

static bool is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }
static bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Shape rules shared by every entry point: K a multiple of 64 (16-byte TMA pitches for both
// code widths and whole 16-code groups of the 6-bit high plane), K <= 16384 (one CTA holds a
// token), rot_block 0 or a power of two in [64, 4096] dividing K.
static dvdq_status validate_k(int64_t K) {
    if (K <= 0 || K % 64 != 0 || K > 16384) return DVDQ_ERR_SHAPE;
    return DVDQ_OK;
}

dvdq_status validate_act_quant(const dvdq_act_quant* q, int64_t K) {
    if (!q) return DVDQ_ERR_NULL;
    if (q->bits != 4 && q->bits != 6 && q->bits != 8) return DVDQ_ERR_BITS;
    if (q->container_bits != 0 && q->container_bits != 8) return DVDQ_ERR_UNSUPPORTED;
    // block-wise scales: one per token and per group of 128, 256 or 1024 consecutive rotated channels
    // (whole k-blocks of the GEMM, which takes them in pairs: K a multiple of 256 and of the group)
    if (q->scale_group != 0 && q->scale_group != 128 && q->scale_group != 256 && q->scale_group != 1024) return DVDQ_ERR_UNSUPPORTED;
    if (q->scale_group != 0 && (K % q->scale_group != 0 || K % 256 != 0)) return DVDQ_ERR_SHAPE;
    if (q->rot_block != 0) {
        if (!is_pow2(q->rot_block) || q->rot_block < 64 || q->rot_block > 4096) return DVDQ_ERR_ROT_BLOCK;
        if (K % q->rot_block != 0) return DVDQ_ERR_ROT_BLOCK;
    }
    return DVDQ_OK;
}

dvdq_status validate_weights(const dvdq_weights* w) {
    if (!w) return DVDQ_ERR_NULL;
    if (w->magic != kBlobMagic || w->version != kBlobVersion || !w->blob) return DVDQ_ERR_BLOB;
    if (w->N <= 0 || w->N % 8 != 0 || validate_k(w->K) != DVDQ_OK) return DVDQ_ERR_BLOB;
    if (w->blob_bytes != (uint64_t)blob_layout(w->N, w->K).total) return DVDQ_ERR_BLOB;
    if (w->k_layout != kKLayoutNatural) return DVDQ_ERR_BLOB;
    if (!aligned(w->blob, 256)) return DVDQ_ERR_ALIGN;
    if (w->operand != nullptr) {
        if (w->operand_bytes != (uint64_t)(w->N * w->K)) return DVDQ_ERR_BLOB;
        if (!aligned(w->operand, 256)) return DVDQ_ERR_ALIGN;
    }
    return DVDQ_OK;
}

struct WorkspacePlan {
    int64_t codes_off, scales_off, sums_off, total;
};
static int64_t scales_per_token(int64_t K, const dvdq_act_quant& q) { return q.scale_group ? K / q.scale_group : 1; }
static WorkspacePlan workspace_plan(int64_t M, int64_t K, const dvdq_act_quant& q) {
    WorkspacePlan p;
    const int64_t per_token = scales_per_token(K, q);
    p.codes_off = 0;
    p.scales_off = align_up(M * act_row_bytes(K, storage_bits(q)), 256);
    p.sums_off = p.scales_off + align_up(M * per_token * 4, 256);
    p.total = p.sums_off + align_up(M * per_token * 4, 256);
    return p;
}

}  // namespace dvdq

using namespace dvdq;

extern "C" {

const char* dvdq_status_string(dvdq_status s) {
    switch (s) {
        case DVDQ_OK: return "ok";
        case DVDQ_ERR_NULL: return "required pointer is NULL";
        case DVDQ_ERR_SHAPE: return "unsupported shape or leading dimension";
        case DVDQ_ERR_BITS: return "activation bit width must be 4, 6 or 8";
        case DVDQ_ERR_ROT_BLOCK: return "rotation block invalid or inconsistent between activations and weights";
        case DVDQ_ERR_ALIGN: return "pointer or pitch not aligned as required";
        case DVDQ_ERR_WORKSPACE: return "workspace too small";
        case DVDQ_ERR_BLOB: return "weight handle was not produced by this library version";
        case DVDQ_ERR_ARCH: return "device is not sm_100";
        case DVDQ_ERR_CUDA: return "CUDA call failed";
        case DVDQ_ERR_DEVICE_TIMEOUT: return "a kernel gave up on a bounded device-side wait";
        case DVDQ_ERR_UNSUPPORTED: return "reserved option is not built";
    }
    return "unknown status";
}

int32_t dvdq_version(void) { return kLibVersion; }

size_t dvdq_act_codes_bytes(int64_t M, int64_t K, int32_t bits) {
    if (M < 0 || validate_k(K) != DVDQ_OK || (bits != 4 && bits != 6 && bits != 8)) return 0;
    return (size_t)(M * act_row_bytes(K, bits));
}

size_t dvdq_act_codes_bytes_q(int64_t M, int64_t K, const dvdq_act_quant* q) {
    if (M < 0 || validate_k(K) != DVDQ_OK || validate_act_quant(q, K) != DVDQ_OK) return 0;
    return (size_t)(M * act_row_bytes(K, storage_bits(*q)));
}

size_t dvdq_act_scales_count(int64_t M, int64_t K, const dvdq_act_quant* q) {
    if (M < 0 || validate_k(K) != DVDQ_OK || validate_act_quant(q, K) != DVDQ_OK) return 0;
    return (size_t)(M * scales_per_token(K, *q));
}

size_t dvdq_weight_blob_bytes(int64_t N, int64_t K) {
    if (N <= 0 || N % 8 != 0 || validate_k(K) != DVDQ_OK) return 0;
    return (size_t)blob_layout(N, K).total;
}

size_t dvdq_weight_operand_bytes(int64_t N, int64_t K) {
    if (N <= 0 || N % 8 != 0 || validate_k(K) != DVDQ_OK) return 0;
    return (size_t)(N * K);
}

size_t dvdq_qlinear_workspace_bytes(int64_t M, int64_t K, const dvdq_act_quant* q) {
    if (M < 0 || validate_k(K) != DVDQ_OK || validate_act_quant(q, K) != DVDQ_OK) return 0;
    return (size_t)workspace_plan(M, K, *q).total;
}

dvdq_status dvdq_rotate_quantize(const void* X, int64_t M, int64_t K, int64_t ldx, const dvdq_act_quant* q,
                                 void* codes_out, float* scales_out, int32_t* code_sums_out, void* stream) {
    if (!q) return DVDQ_ERR_NULL;
    if (M < 0 || validate_k(K) != DVDQ_OK || ldx < K || ldx % 8 != 0) return DVDQ_ERR_SHAPE;
    dvdq_status s = validate_act_quant(q, K);
    if (s != DVDQ_OK) return s;
    if (M == 0) return DVDQ_OK;
    if (!X || !codes_out || !scales_out || !code_sums_out) return DVDQ_ERR_NULL;
    if (!aligned(X, 16) || !aligned(codes_out, 16) || !aligned(scales_out, 4) || !aligned(code_sums_out, 4)) return DVDQ_ERR_ALIGN;
    if ((s = check_device_arch()) != DVDQ_OK) return s;
    return launch_rotate_quantize(X, M, K, ldx, *q, codes_out, scales_out, code_sums_out, (cudaStream_t)stream);
}

dvdq_status dvdq_pack_weights(const uint8_t* Wq, const float* delta, const int32_t* zero, int64_t N, int64_t K,
                              int32_t rot_block, void* blob_out, dvdq_weights* out, void* stream) {
    if (!Wq || !delta || !zero || !blob_out || !out) return DVDQ_ERR_NULL;
    if (N <= 0 || N % 8 != 0 || validate_k(K) != DVDQ_OK) return DVDQ_ERR_SHAPE;
    dvdq_act_quant probe = {4, rot_block, 0};
    dvdq_status s = validate_act_quant(&probe, K);
    if (s != DVDQ_OK) return s;
    if (!aligned(blob_out, 256)) return DVDQ_ERR_ALIGN;
    if ((s = check_device_arch()) != DVDQ_OK) return s;
    pack_weights_kernel<<<grid_for(N * (K / 2), 256), 256, 0, (cudaStream_t)stream>>>(
        Wq, delta, zero, N, K, rot_block, kKLayoutNatural, static_cast<uint8_t*>(blob_out));
    if ((s = cuda_status(cudaGetLastError())) != DVDQ_OK) return s;
    out->magic = kBlobMagic;
    out->version = kBlobVersion;
    out->N = N;
    out->K = K;
    out->rot_block = rot_block;
    out->k_layout = kKLayoutNatural;
    out->blob = blob_out;
    out->blob_bytes = (uint64_t)blob_layout(N, K).total;
    out->operand = nullptr;
    out->operand_bytes = 0;
    return DVDQ_OK;
}

// ---- offline weight preparation on the GPU (Eq. 10: W^ = Quant(W H)) ------------------------

static int log2_of(int32_t b) {
    int l = 0;
    while ((1 << l) < b) ++l;
    return l;
}

static dvdq_status check_weight_prep_args(const void* W, int64_t N, int64_t K, int64_t ldw, int32_t rot_block, const void* out) {
    if (N < 0 || N > 0x7FFFFFFFll || validate_k(K) != DVDQ_OK || ldw < K) return DVDQ_ERR_SHAPE;
    dvdq_act_quant probe = {4, rot_block, 0, 0};
    dvdq_status s = validate_act_quant(&probe, K);
    if (s != DVDQ_OK) return s;
    if (N == 0) return DVDQ_OK;
    if (!W || !out) return DVDQ_ERR_NULL;
    if (!aligned(W, 2)) return DVDQ_ERR_ALIGN;
    return DVDQ_OK;
}

dvdq_status dvdq_rotate_weights(const void* W, int64_t N, int64_t K, int64_t ldw, int32_t rot_block, float* W_rot_out,
                                void* stream) {
    dvdq_status s = check_weight_prep_args(W, N, K, ldw, rot_block, W_rot_out);
    if (s != DVDQ_OK || N == 0) return s;
    if (!aligned(W_rot_out, 4)) return DVDQ_ERR_ALIGN;
    if ((s = check_device_arch()) != DVDQ_OK) return s;
    static PerDevice<int> cache;
    if (!weight_kernel_setup(cache, rotate_weights_kernel)) return DVDQ_ERR_CUDA;
    rotate_weights_kernel<<<(unsigned)N, kWeightThreads, (size_t)K * sizeof(double), (cudaStream_t)stream>>>(
        static_cast<const __nv_bfloat16*>(W), ldw, (int)K, log2_of(rot_block), W_rot_out);
    return cuda_status(cudaGetLastError());
}

dvdq_status dvdq_quantize_weights_symmetric(const void* W, int64_t N, int64_t K, int64_t ldw, int32_t rot_block,
                                            void* blob_out, dvdq_weights* out, void* stream) {
    if (!out) return DVDQ_ERR_NULL;
    if (N <= 0 || N % 8 != 0) return DVDQ_ERR_SHAPE;
    dvdq_status s = check_weight_prep_args(W, N, K, ldw, rot_block, blob_out);
    if (s != DVDQ_OK) return s;
    if (!aligned(blob_out, 256)) return DVDQ_ERR_ALIGN;
    if ((s = check_device_arch()) != DVDQ_OK) return s;
    static PerDevice<int> cache;
    if (!weight_kernel_setup(cache, quantize_weights_symmetric_kernel)) return DVDQ_ERR_CUDA;
    quantize_weights_symmetric_kernel<<<(unsigned)N, kWeightThreads, (size_t)K * sizeof(double), (cudaStream_t)stream>>>(
        static_cast<const __nv_bfloat16*>(W), ldw, N, (int)K, log2_of(rot_block), rot_block, static_cast<uint8_t*>(blob_out));
    if ((s = cuda_status(cudaGetLastError())) != DVDQ_OK) return s;
    out->magic = kBlobMagic;
    out->version = kBlobVersion;
    out->N = N;
    out->K = K;
    out->rot_block = rot_block;
    out->k_layout = kKLayoutNatural;
    out->blob = blob_out;
    out->blob_bytes = (uint64_t)blob_layout(N, K).total;
    out->operand = nullptr;
    out->operand_bytes = 0;
    return DVDQ_OK;
}

dvdq_status dvdq_widen_weights(const dvdq_weights* w, void* operand_out, size_t operand_bytes, dvdq_weights* out, void* stream) {
    if (!out) return DVDQ_ERR_NULL;
    dvdq_weights in;
    if (w) { in = *w; in.operand = nullptr; in.operand_bytes = 0; }
    dvdq_status s = validate_weights(w ? &in : nullptr);
    if (s != DVDQ_OK) return s;
    if (!operand_out) return DVDQ_ERR_NULL;
    if (operand_bytes < (size_t)(in.N * in.K)) return DVDQ_ERR_WORKSPACE;
    if (!aligned(operand_out, 256)) return DVDQ_ERR_ALIGN;
    if ((s = check_device_arch()) != DVDQ_OK) return s;
    const int64_t pieces = in.N * (in.K / 32);
    widen_weights_kernel<<<grid_for(pieces, 256), 256, 0, (cudaStream_t)stream>>>(
        static_cast<const uint8_t*>(in.blob) + blob_layout(in.N, in.K).codes_offset, pieces, static_cast<uint8_t*>(operand_out));
    if ((s = cuda_status(cudaGetLastError())) != DVDQ_OK) return s;
    in.operand = operand_out;
    in.operand_bytes = (uint64_t)(in.N * in.K);
    *out = in;
    return DVDQ_OK;
}

static dvdq_status check_gemm_args(const void* codes, const int32_t* sums, int64_t M, const dvdq_act_quant* q,
                                   const dvdq_weights* w) {
    dvdq_status s = validate_weights(w);
    if (s != DVDQ_OK) return s;
    if ((s = validate_act_quant(q, w->K)) != DVDQ_OK) return s;
    if (q->rot_block != w->rot_block) return DVDQ_ERR_ROT_BLOCK;
    if (M < 0 || M > 0x7FFFFF00ll) return DVDQ_ERR_SHAPE;
    if (M == 0) return DVDQ_OK;
    if (!codes || !sums) return DVDQ_ERR_NULL;
    if (!aligned(codes, 16) || !aligned(sums, 4)) return DVDQ_ERR_ALIGN;
    return check_device_arch();
}

dvdq_status dvdq_qgemm(const void* codes, const float* scales, const int32_t* code_sums, int64_t M,
                       const dvdq_act_quant* q, const dvdq_weights* w, const void* bias, int32_t act,
                       void* Y, int64_t ldy, void* stream) {
    dvdq_status s = check_gemm_args(codes, code_sums, M, q, w);
    if (s != DVDQ_OK) return s;
    if (act != 0 && act != 1) return DVDQ_ERR_UNSUPPORTED;
    if (ldy < w->N || ldy % 8 != 0) return DVDQ_ERR_SHAPE;
    if (M == 0) return DVDQ_OK;
    if (!scales || !Y) return DVDQ_ERR_NULL;
    if (!aligned(Y, 16) || !aligned(scales, 4) || (bias && !aligned(bias, 2))) return DVDQ_ERR_ALIGN;
    return launch_qgemm(codes, scales, code_sums, M, *q, *w, bias, act, Y, ldy, nullptr, 0, (cudaStream_t)stream);
}

dvdq_status dvdq_qgemm_fused_rq(const void* codes, const float* scales, const int32_t* code_sums, int64_t M,
                                const dvdq_act_quant* q, const dvdq_weights* w, const void* bias, int32_t act,
                                const dvdq_act_quant* q_next, void* codes_next, float* scales_next, int32_t* code_sums_next,
                                void* Y_or_null, int64_t ldy, void* stream) {
    dvdq_status s = check_gemm_args(codes, code_sums, M, q, w);
    if (s != DVDQ_OK) return s;
    if (act != 0 && act != 1) return DVDQ_ERR_UNSUPPORTED;
    // this layer: per-token scales; the next layer: N input channels in whole
    // 256-blocks, rotation block = scale group = 256 (what one 256-wide tile owns), codes one int8 each
    if (q->scale_group != 0) return DVDQ_ERR_UNSUPPORTED;
    if (!q_next) return DVDQ_ERR_NULL;
    if (w->N % 256 != 0 || validate_k(w->N) != DVDQ_OK) return DVDQ_ERR_SHAPE;
    if ((s = validate_act_quant(q_next, w->N)) != DVDQ_OK) return s;
    if (q_next->rot_block != 256 || q_next->scale_group != 256 || q_next->container_bits != 8) return DVDQ_ERR_UNSUPPORTED;
    if (Y_or_null && (ldy < w->N || ldy % 8 != 0)) return DVDQ_ERR_SHAPE;
    if (M == 0) return DVDQ_OK;
    if (!scales || !codes_next || !scales_next || !code_sums_next) return DVDQ_ERR_NULL;
    if (!aligned(scales, 4) || !aligned(codes_next, 16) || !aligned(scales_next, 4) || !aligned(code_sums_next, 4) ||
        (Y_or_null && !aligned(Y_or_null, 16)) || (bias && !aligned(bias, 2)))
        return DVDQ_ERR_ALIGN;
    FusedOut fo;
    fo.codes = static_cast<uint8_t*>(codes_next);
    fo.scales = scales_next;
    fo.sums = code_sums_next;
    fo.y_dbg = static_cast<__nv_bfloat16*>(Y_or_null);
    fo.ldy = ldy;
    fo.bits = q_next->bits;
    return launch_qgemm_fused(storage_bits(*q), codes, scales, code_sums, M, *w, bias, act, fo, (cudaStream_t)stream);
}

dvdq_status dvdq_qgemm_int32(const void* codes, const int32_t* code_sums, int64_t M, const dvdq_act_quant* q,
                             const dvdq_weights* w, int32_t* acc_out, int64_t ldacc, void* stream) {
    dvdq_status s = check_gemm_args(codes, code_sums, M, q, w);
    if (s != DVDQ_OK) return s;
    if (ldacc < w->N || ldacc % 4 != 0) return DVDQ_ERR_SHAPE;
    if (M == 0) return DVDQ_OK;
    if (!acc_out) return DVDQ_ERR_NULL;
    if (!aligned(acc_out, 16)) return DVDQ_ERR_ALIGN;
    return launch_qgemm(codes, nullptr, code_sums, M, *q, *w, nullptr, 0, nullptr, 0, acc_out, ldacc, (cudaStream_t)stream);
}

// Everything dvdq_qlinear and dvdq_qlinear_static check before their first launch: the union of
// what dvdq_rotate_quantize and dvdq_qgemm check on their own.
static dvdq_status check_qlinear_args(const void* X, int64_t M, int64_t ldx, const dvdq_act_quant* q, const dvdq_weights* w,
                                      const void* bias, int32_t act, const void* Y, int64_t ldy) {
    dvdq_status s = validate_weights(w);
    if (s != DVDQ_OK) return s;
    if ((s = validate_act_quant(q, w->K)) != DVDQ_OK) return s;
    if (q->rot_block != w->rot_block) return DVDQ_ERR_ROT_BLOCK;
    if (M < 0 || M > 0x7FFFFF00ll) return DVDQ_ERR_SHAPE;
    if (ldx < w->K || ldx % 8 != 0 || ldx > 0x7FFFFFFFll || ldy < w->N || ldy % 8 != 0) return DVDQ_ERR_SHAPE;
    if (act != 0 && act != 1) return DVDQ_ERR_UNSUPPORTED;
    if (M == 0) return DVDQ_OK;
    if (!X || !Y) return DVDQ_ERR_NULL;
    if (!aligned(X, 16) || !aligned(Y, 16) || (bias && !aligned(bias, 2))) return DVDQ_ERR_ALIGN;
    return check_device_arch();
}

constexpr int64_t kWidenOnceMinTokens = 1024;  // four rows of output tiles share one written operand

static dvdq_status qlinear_on_workspace(const void* X, int64_t M, int64_t ldx, const dvdq_act_quant* q, const dvdq_weights* w,
                                        const void* bias, int32_t act, void* Y, int64_t ldy, uint8_t* ws, size_t ws_bytes,
                                        void* stream) {
    const WorkspacePlan p = workspace_plan(M, w->K, *q);
    void* codes = ws + p.codes_off;
    float* scales = reinterpret_cast<float*>(ws + p.scales_off);
    int32_t* sums = reinterpret_cast<int32_t*>(ws + p.sums_off);
    dvdq_status s = launch_rotate_quantize(X, M, w->K, ldx, *q, codes, scales, sums, (cudaStream_t)stream);
    if (s != DVDQ_OK) return s;
    // Room behind the codes for the int8 weight operand, and enough token tiles to share it: written once
    // per call instead of once per tile (same result bits).
    dvdq_weights wide = *w;
    const int64_t operand_off = align_up(p.total, 256);
    if (w->operand == nullptr && M >= kWidenOnceMinTokens &&
        ws_bytes >= (size_t)(operand_off + w->N * w->K)) {
        const int64_t pieces = w->N * (w->K / 32);
        widen_weights_kernel<<<grid_for(pieces, 256), 256, 0, (cudaStream_t)stream>>>(
            static_cast<const uint8_t*>(w->blob) + blob_layout(w->N, w->K).codes_offset, pieces, ws + operand_off);
        if ((s = cuda_status(cudaGetLastError())) != DVDQ_OK) return s;
        wide.operand = ws + operand_off;
        wide.operand_bytes = (uint64_t)(w->N * w->K);
    }
    return launch_qgemm(codes, scales, sums, M, *q, wide, bias, act, Y, ldy, nullptr, 0, (cudaStream_t)stream);
}

dvdq_status dvdq_qlinear(const void* X, int64_t M, int64_t ldx, const dvdq_act_quant* q, const dvdq_weights* w,
                         const void* bias, int32_t act, void* Y, int64_t ldy, void* workspace, size_t workspace_bytes,
                         void* stream) {
    dvdq_status s = check_qlinear_args(X, M, ldx, q, w, bias, act, Y, ldy);
    if (s != DVDQ_OK) return s;
    if (M == 0) return DVDQ_OK;
    if (!workspace) return DVDQ_ERR_NULL;
    if (!aligned(workspace, 256)) return DVDQ_ERR_ALIGN;
    if (workspace_bytes < (size_t)workspace_plan(M, w->K, *q).total) return DVDQ_ERR_WORKSPACE;
    return qlinear_on_workspace(X, M, ldx, q, w, bias, act, Y, ldy, static_cast<uint8_t*>(workspace), workspace_bytes, stream);
}

// Scratch of dvdq_qlinear_static: part of the library image, so no allocation is ever needed.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) uint8_t g_static_scratch[DVDQ_STATIC_SCRATCH_BYTES];

dvdq_status dvdq_qlinear_static(const void* X, int64_t M, int64_t ldx, const dvdq_act_quant* q, const dvdq_weights* w,
                                const void* bias, int32_t act, void* Y, int64_t ldy, void* stream) {
    static PerDevice<void*> scratch_of_device;
    dvdq_status s = check_qlinear_args(X, M, ldx, q, w, bias, act, Y, ldy);
    if (s != DVDQ_OK) return s;
    if (M == 0) return DVDQ_OK;
    if (workspace_plan(M, w->K, *q).total > (int64_t)DVDQ_STATIC_SCRATCH_BYTES) return DVDQ_ERR_WORKSPACE;
    void** ws = scratch_of_device.get([](void*& ptr, int) {  // set-up, once per device, with that device current
        return cudaGetSymbolAddress(&ptr, g_static_scratch) == cudaSuccess && ptr != nullptr;
    });
    if (!ws) return DVDQ_ERR_CUDA;
    return qlinear_on_workspace(X, M, ldx, q, w, bias, act, Y, ldy, static_cast<uint8_t*>(*ws), (size_t)DVDQ_STATIC_SCRATCH_BYTES, stream);
}

dvdq_status dvdq_pack_act_codes(const int8_t* codes_nat, int64_t M, int64_t K, const dvdq_act_quant* q,
                                void* codes_out, int32_t* code_sums_out, void* stream) {
    if (M < 0 || validate_k(K) != DVDQ_OK) return DVDQ_ERR_SHAPE;
    dvdq_status s = validate_act_quant(q, K);
    if (s != DVDQ_OK) return s;
    if (M == 0) return DVDQ_OK;
    if (!codes_nat || !codes_out || !code_sums_out) return DVDQ_ERR_NULL;
    if (!aligned(codes_out, 16)) return DVDQ_ERR_ALIGN;
    if ((s = check_device_arch()) != DVDQ_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    const unsigned g = grid_for(M * (K / 16), 256);
    const int sb = storage_bits(*q);
    if (sb == 4) pack_act_codes_kernel<4><<<g, 256, 0, st>>>(codes_nat, M, K, static_cast<uint8_t*>(codes_out));
    else if (sb == 6) pack_act_codes_kernel<6><<<g, 256, 0, st>>>(codes_nat, M, K, static_cast<uint8_t*>(codes_out));
    else pack_act_codes_kernel<8><<<g, 256, 0, st>>>(codes_nat, M, K, static_cast<uint8_t*>(codes_out));
    const int64_t block = q->scale_group ? q->scale_group : K;
    code_sums_kernel<<<(unsigned)((M * (K / block) * 32 + 255) / 256), 256, 0, st>>>(codes_nat, M, K, block, code_sums_out);
    return cuda_status(cudaGetLastError());
}

dvdq_status dvdq_unpack_act_codes(const void* codes, int64_t M, int64_t K, const dvdq_act_quant* q,
                                  int8_t* codes_nat, void* stream) {
    if (M < 0 || validate_k(K) != DVDQ_OK) return DVDQ_ERR_SHAPE;
    dvdq_status s = validate_act_quant(q, K);
    if (s != DVDQ_OK) return s;
    if (M == 0) return DVDQ_OK;
    if (!codes || !codes_nat) return DVDQ_ERR_NULL;
    if (!aligned(codes, 16)) return DVDQ_ERR_ALIGN;
    if ((s = check_device_arch()) != DVDQ_OK) return s;
    const unsigned g = grid_for(M * (K / 16), 256);
    const int sb = storage_bits(*q);
    if (sb == 4) unpack_act_codes_kernel<4><<<g, 256, 0, (cudaStream_t)stream>>>(static_cast<const uint8_t*>(codes), M, K, codes_nat);
    else if (sb == 6) unpack_act_codes_kernel<6><<<g, 256, 0, (cudaStream_t)stream>>>(static_cast<const uint8_t*>(codes), M, K, codes_nat);
    else unpack_act_codes_kernel<8><<<g, 256, 0, (cudaStream_t)stream>>>(static_cast<const uint8_t*>(codes), M, K, codes_nat);
    return cuda_status(cudaGetLastError());
}

dvdq_status dvdq_unpack_weights(const dvdq_weights* w, uint8_t* Wq, float* delta, int32_t* zero, void* stream) {
    dvdq_status s = validate_weights(w);
    if (s != DVDQ_OK) return s;
    if (!Wq || !delta || !zero) return DVDQ_ERR_NULL;
    if ((s = check_device_arch()) != DVDQ_OK) return s;
    unpack_weights_kernel<<<grid_for(w->N * (w->K / 2), 256), 256, 0, (cudaStream_t)stream>>>(
        static_cast<const uint8_t*>(w->blob), w->N, w->K, Wq, delta, zero);
    return cuda_status(cudaGetLastError());
}

// ---- Bounded-init Grid Refinement (Alg. 1) ------------------------------------------------

dvdq_status dvdq_bgr_quantize(const float* W_rot, int64_t N, int64_t K, int32_t n_steps, double eps, int32_t max_iter,
                              uint8_t* Wq_out, float* delta_out, int32_t* zero_out, void* stream) {
    if (N < 0 || N > 0x7FFFFFFFll || validate_k(K) != DVDQ_OK || n_steps < 1 || max_iter < 0 || !(eps >= 0.0)) return DVDQ_ERR_SHAPE;
    if (N == 0) return DVDQ_OK;
    if (!W_rot || !Wq_out || !delta_out || !zero_out) return DVDQ_ERR_NULL;
    if (!aligned(W_rot, 4) || !aligned(delta_out, 4) || !aligned(zero_out, 4)) return DVDQ_ERR_ALIGN;
    dvdq_status s = check_device_arch();
    if (s != DVDQ_OK) return s;
    const size_t smem = (size_t)K * sizeof(float);
    static PerDevice<int> attr_set;
    if (!attr_set.get([](int&, int) {
            return cudaFuncSetAttribute(bgr_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 16384 * (int)sizeof(float)) == cudaSuccess;
        }))
        return DVDQ_ERR_CUDA;
    bgr_kernel<<<(unsigned)N, kBgrThreads, smem, (cudaStream_t)stream>>>(W_rot, (int)K, n_steps, eps, max_iter, Wq_out,
                                                                         delta_out, zero_out);
    return cuda_status(cudaGetLastError());
}

// ---- delta-Guided Bit Switching (Sec. 3.3) ---------------------------------------------

dvdq_status dvdq_gbs_l1_terms(const void* F_t, const void* F_prev, int64_t n, double* terms_out, void* stream) {
    if (n < 0) return DVDQ_ERR_SHAPE;
    if (!terms_out) return DVDQ_ERR_NULL;
    if (!aligned(terms_out, 8)) return DVDQ_ERR_ALIGN;
    if (n > 0 && (!F_t || !F_prev)) return DVDQ_ERR_NULL;
    if (n > 0 && (!aligned(F_t, 16) || !aligned(F_prev, 16))) return DVDQ_ERR_ALIGN;
    dvdq_status s = check_device_arch();
    if (s != DVDQ_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(terms_out, 0, 2 * sizeof(double), st) != cudaSuccess) return DVDQ_ERR_CUDA;
    if (n == 0) return DVDQ_OK;
    int64_t blocks = (n / 8 + 255) / 256;
    if (blocks < 1) blocks = 1;
    if (blocks > 148 * 8) blocks = 148 * 8;
    gbs_l1_terms_kernel<<<(unsigned)blocks, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(F_t),
                                                          static_cast<const __nv_bfloat16*>(F_prev), n, terms_out);
    return cuda_status(cudaGetLastError());
}

dvdq_status dvdq_gbs_init(dvdq_gbs_state* g, double delta, int32_t b_low, int32_t b_high) {
    if (!g) return DVDQ_ERR_NULL;
    if (!(delta >= 0.0)) return DVDQ_ERR_SHAPE;  // also rejects NaN
    const bool ok_low = b_low == 4 || b_low == 6 || b_low == 8, ok_high = b_high == 4 || b_high == 6 || b_high == 8;
    if (!ok_low || !ok_high || b_low > b_high) return DVDQ_ERR_BITS;
    g->delta = delta;
    g->b_low = b_low;
    g->b_high = b_high;
    g->accumulated = 0.0;
    g->steps = 0;
    g->high_steps = 0;
    return DVDQ_OK;
}

int32_t dvdq_gbs_next_bits(dvdq_gbs_state* g) {
    if (!g) return 0;
    g->steps += 1;
    if (g->accumulated >= g->delta) {  // enough feature change has piled up: one step at b_high, counter back to zero
        g->accumulated = 0.0;
        g->high_steps += 1;
        return g->b_high;
    }
    return g->b_low;
}

dvdq_status dvdq_gbs_observe(dvdq_gbs_state* g, double l1_change, double l1_prev) {
    if (!g) return DVDQ_ERR_NULL;
    if (!(l1_change >= 0.0) || !(l1_prev >= 0.0)) return DVDQ_ERR_SHAPE;
    // an all-zero previous output gives no ratio: count it as no change (0/0) or as a full change (x/0)
    const double rel = l1_prev > 0.0 ? l1_change / l1_prev : (l1_change > 0.0 ? 1.0 : 0.0);
    g->accumulated += rel;
    return DVDQ_OK;
}

// ---- measurement and diagnostics ---------------------------------------------------------------

dvdq_status dvdq_int8_mma_ceiling(int32_t iters, int64_t* ops_out, void* stream) {
    if (iters < 1 || iters > (1 << 20)) return DVDQ_ERR_SHAPE;
    dvdq_status s = check_device_arch();
    if (s != DVDQ_OK) return s;
    static PerDevice<int> cache;
    const int pairs = resident_pairs(cache, int8_ceiling_kernel, kCeilThreads, kCeilSmem);
    if (pairs == 0) return DVDQ_ERR_CUDA;
    int8_ceiling_kernel<<<2 * pairs, kCeilThreads, kCeilSmem, (cudaStream_t)stream>>>(iters);
    if (ops_out) *ops_out = (int64_t)pairs * iters * (kBK / 32) * 2ll * (2 * kBM) * kSsBN * 32;
    return cuda_status(cudaGetLastError());
}

dvdq_status dvdq_debug_wait_timeout(uint64_t limit_ns, void* stream) {
    if (limit_ns == 0 || limit_ns > 1000000000ull) return DVDQ_ERR_SHAPE;  // at most a second
    dvdq_status s = check_device_arch();
    if (s != DVDQ_OK) return s;
    wait_timeout_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(limit_ns);
    return cuda_status(cudaGetLastError());
}

dvdq_status dvdq_last_device_status(uint32_t* detail) {
    uint32_t h[2] = {0u, 0u};
    if (cudaDeviceSynchronize() != cudaSuccess) return DVDQ_ERR_CUDA;
    if (cudaMemcpyFromSymbol(h, g_device_status, sizeof h) != cudaSuccess) return DVDQ_ERR_CUDA;
    if (h[0] != 0u) {
        const uint32_t zero[2] = {0u, 0u};
        if (cudaMemcpyToSymbol(g_device_status, zero, sizeof zero) != cudaSuccess) return DVDQ_ERR_CUDA;
    }
    if (detail) *detail = h[1];
    return (dvdq_status)h[0];
}

}  // extern "C"
