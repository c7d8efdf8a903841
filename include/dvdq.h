/*
 * dvdq.h -- C ABI of the B200 (sm_100a) quantized-linear library for DVD-Quant.
 *
 * The library runs the per-layer hot path of DVD-Quant's quantized inference:
 *
 *   (1) online activation transform (Sec. 3.2 "Auto-scaling Rotated Quantization",
 *       Eq. 10): rotate each token by a block Hadamard matrix, take one absmax
 *       scale per token, round to b-bit signed codes and pack them;
 *   (2) an integer GEMM of those codes against 4-bit weights stored in the
 *       Quant/DeQuant format of Sec. 3.1 (unsigned code, integer zero point and
 *       step size per output channel) with a dequantizing bf16 epilogue,
 *       Y = X^ Lambda W^^T (Eq. 10).
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller unless a
 *     parameter says "host".  The library never allocates device memory.
 *   - Calls are asynchronous on the CUDA stream passed as `cuda_stream`
 *     (a cudaStream_t cast to void*; NULL is the default stream).
 *   - The return value covers host-side argument validation and launch errors.
 *     A kernel that gives up on a device-side wait records that in a status word
 *     read by dvdq_last_device_status().
 *   - Packed code buffers are opaque; use the pack/unpack entry points to read or
 *     write them.  Row-major everywhere; "ld" arguments count ELEMENTS.
 *   - Only sm_100 devices are accepted (DVDQ_ERR_ARCH otherwise).  There is no
 *     fallback path of any kind.
 */
#ifndef DVDQ_H_
#define DVDQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DVDQ_OK = 0,
    DVDQ_ERR_NULL = 1,           /* a required pointer is NULL */
    DVDQ_ERR_SHAPE = 2,          /* M, N, K or a leading dimension is not supported */
    DVDQ_ERR_BITS = 3,           /* activation bit width is not 4, 6 or 8 */
    DVDQ_ERR_ROT_BLOCK = 4,      /* rotation block invalid, or activations and weights disagree on it */
    DVDQ_ERR_ALIGN = 5,          /* a pointer or pitch misses its alignment requirement */
    DVDQ_ERR_WORKSPACE = 6,      /* workspace too small */
    DVDQ_ERR_BLOB = 7,           /* weight handle / blob header is not one this library wrote */
    DVDQ_ERR_ARCH = 8,           /* current device is not sm_100 */
    DVDQ_ERR_CUDA = 9,           /* a CUDA runtime or driver call failed */
    DVDQ_ERR_DEVICE_TIMEOUT = 10,/* a kernel gave up on a bounded device-side wait */
    DVDQ_ERR_UNSUPPORTED = 11    /* an option that is not built (scale_group other than 0, 128, 256, 1024; unknown activation function) */
} dvdq_status;

/* Human-readable name of a status code (static storage, never NULL). */
const char* dvdq_status_string(dvdq_status s);

/*
 * The activation quantizer of Eq. 10, X^ = Q(X H Lambda^-1):
 *   bits        b, the code width: 4 (codes in [-8,7]), 6 (codes in [-32,31]) or 8 (codes in
 *               [-128,127]; the b_high = 8 of Sec. 3.3's bit-width switching, i.e. the W4A8 steps).
 *               The quantizer is symmetric with qmax = 2^(b-1) - 1.
 *   rot_block   B, the order of the Hadamard blocks of the rotation
 *               R = I_{K/B} (x) H_B / sqrt(B); a power of two in [64, 4096] that
 *               divides K.  0 means no rotation (R = I).
 *   scale_group granularity of Lambda: 0 = one absmax scale per token over all K channels;
 *               G = 128, 256 or 1024 = the block-wise variant of Sec. 3.2's last paragraph, one
 *               scale per token and per group of G consecutive rotated channels (whole k-blocks
 *               of the GEMM; K % G == 0 and K % 256 == 0; every group is quantized on its own,
 *               the GEMM rescales per group).  Other values give DVDQ_ERR_UNSUPPORTED.
 *   container_bits  how the codes are kept between the transform and the GEMM (the values are
 *               the same either way): 0 = packed, b bits per code; 8 = one int8 per code.
 *               int8 tensor cores are the narrowest integer ones on sm_100, so packed codes
 *               are widened inside the GEMM; codes kept in bytes go from HBM into the tensor
 *               core's operand layout untouched, which is faster, at K instead of K*b/8 bytes
 *               per token.  Other values give DVDQ_ERR_UNSUPPORTED.
 */
typedef struct {
    int32_t bits;
    int32_t rot_block;
    int32_t scale_group;
    int32_t container_bits;
} dvdq_act_quant;

/*
 * Host-side handle of a packed weight matrix.  Filled by dvdq_pack_weights();
 * `blob` is the device buffer the caller passed there.  Plain data: it may be
 * copied, and it stays valid as long as the device buffer does.
 */
typedef struct {
    uint32_t magic;      /* 'DVDQ' */
    uint32_t version;
    int64_t  N;          /* output channels (rows of W) */
    int64_t  K;          /* input channels */
    int32_t  rot_block;  /* B the weights were rotated with (recorded, not applied) */
    int32_t  k_layout;   /* storage order of the K axis shared with the activation codes */
    const void* blob;    /* device */
    uint64_t blob_bytes;
    const void* operand; /* device, or NULL: the same codes one int8 each (dvdq_widen_weights) */
    uint64_t operand_bytes;
} dvdq_weights;

/* ---- size queries (host only, no CUDA calls) ------------------------------------ */

/* Bytes of the packed activation codes of an [M, K] tensor: M * K * bits / 8. 0 on bad input. */
size_t dvdq_act_codes_bytes(int64_t M, int64_t K, int32_t bits);
/* The same for a quantizer description: M * K * (container_bits ? container_bits : bits) / 8. */
size_t dvdq_act_codes_bytes_q(int64_t M, int64_t K, const dvdq_act_quant* q);
/* Number of scales (and of code sums) of an [M, K] tensor: M, or M * K / scale_group block-wise. 0 on bad input. */
size_t dvdq_act_scales_count(int64_t M, int64_t K, const dvdq_act_quant* q);
/* Bytes of the device blob that dvdq_pack_weights() writes for an [N, K] matrix. 0 on bad input. */
size_t dvdq_weight_blob_bytes(int64_t N, int64_t K);
/* Bytes of the int8 copy of the codes that dvdq_widen_weights() writes for an [N, K] matrix: N * K. 0 on bad input. */
size_t dvdq_weight_operand_bytes(int64_t N, int64_t K);
/* Bytes of the workspace dvdq_qlinear() needs (codes, scales and code sums of X). 0 on bad input. */
size_t dvdq_qlinear_workspace_bytes(int64_t M, int64_t K, const dvdq_act_quant* q);

/* ---- (1) online activation transform: Sec. 3.2, Eq. 10 ---------------------------
 *
 * For every token i (row of X):  x~_i = x_i R  (fast Walsh-Hadamard butterflies in fp32),
 * a_i = max_k |x~_ik|, s_i = a_i / qmax, c_ik = round_half_even(x~_ik / s_i).
 *
 *   X_bf16         [M, K] bf16, row pitch ldx elements; 16-byte aligned, ldx % 8 == 0
 *   codes_out      dvdq_act_codes_bytes_q(M, K, q) bytes, 16-byte aligned (opaque layout)
 *   scales_out     [M] fp32, s_i  (0 for an all-zero token, whose codes are all 0);
 *                  block-wise: [M, K/scale_group], one scale per token and group
 *   code_sums_out  [M] int32, sum_k c_ik (used by the GEMM for the weight zero point);
 *                  block-wise: [M, K/scale_group], the sum over each group
 * K % 64 == 0, K <= 16384.  M == 0 is a no-op.
 */
dvdq_status dvdq_rotate_quantize(const void* X_bf16, int64_t M, int64_t K, int64_t ldx,
                                 const dvdq_act_quant* q, void* codes_out, float* scales_out,
                                 int32_t* code_sums_out, void* cuda_stream);

/* ---- (0) offline weight packing: Sec. 3.1 Quant/DeQuant format, Eq. 10 W^ ----------
 *
 * Takes weights that are ALREADY rotated (W~ = W R, same B as the activations: dvdq_rotate_weights) and
 * quantized to the format W^ = Delta (W_q - z):
 *   Wq     [N, K] uint8, values 0..15 (upper bits ignored)
 *   delta  [N] fp32 step sizes
 *   zero   [N] int32 zero points, 0..15
 *   blob_out  dvdq_weight_blob_bytes(N, K) bytes, 256-byte aligned
 *   out    host handle describing the blob (written synchronously)
 * N % 8 == 0, K % 64 == 0.  rot_block is recorded so that dvdq_qgemm can refuse
 * activations rotated with a different block.
 */
dvdq_status dvdq_pack_weights(const uint8_t* Wq, const float* delta, const int32_t* zero,
                              int64_t N, int64_t K, int32_t rot_block,
                              void* blob_out, dvdq_weights* out /* host */, void* cuda_stream);

/* ---- the weight operand of the GEMM, written once instead of once per tile: Sec. 3.1, Eq. 10 ----
 *
 * The tensor cores take int8 operands, so every GEMM widens the 4-bit codes (u - 8): by default
 * inside the kernel, each output tile for itself.  This call does it once, into a buffer of the
 * caller's: operand_out (device, dvdq_weight_operand_bytes(N, K) = N * K bytes, 256-byte
 * aligned) receives one int8 per code, and *out is *w referring to that buffer as well.  GEMMs
 * given `out` then read the operand with TMA and widen no weights; all results are bit-identical
 * to those with `w`.  The blob stays the format of record (the
 * scales, zero points and 4-bit codes are still read from it); the buffer may be a scratch area
 * that is rewritten before every launch (one call per layer and step costs about 1 % of a GEMM
 * over 65536 tokens) or kept for the life of the weights (at 8 more bits per weight).  A scratch
 * area shared by several layers is safe only while the calls that write and read it are ordered
 * (one stream, or events between streams): nothing in the library orders them.  w and out
 * may be the same object.  dvdq_qgemm_int32 always reads the 4-bit codes. */
dvdq_status dvdq_widen_weights(const dvdq_weights* w /* host */, void* operand_out, size_t operand_bytes,
                               dvdq_weights* out /* host */, void* cuda_stream);

/* ---- (0) offline weight rotation: Eq. 10, W^ = Quant(W H); Sec. 3.2 ------------------------
 *
 * W~ = W R along K with the same R = I_{K/B} (x) H_B / sqrt(B) as the activations, so that
 * X~ W~^T = X W^T.  Butterflies and the normalisation in fp64, one rounding to fp32 at the end.
 *   W_bf16     [N, K] bf16, row pitch ldw elements
 *   W_rot_out  [N, K] fp32, dense: the input of dvdq_bgr_quantize
 * K % 64 == 0, K <= 16384; rot_block as in dvdq_act_quant.  N == 0 is a no-op. */
dvdq_status dvdq_rotate_weights(const void* W_bf16, int64_t N, int64_t K, int64_t ldw, int32_t rot_block,
                                float* W_rot_out, void* cuda_stream);

/* ---- (0) offline, in one call: rotate and quantize symmetrically into a blob -----------------
 *
 * The plain per-output-channel 4-bit quantizer in the format of Sec. 3.1 with the zero point
 * pinned (not the paper's grid refinement, which is dvdq_bgr_quantize): W~ = W R as above, then
 *     Delta_n = max_k |w~_nk| / 7,  W_q = clamp(round(w~ / Delta), -8, 7) + 8,  z_n = 8
 * (fp64, round half to even; an all-zero row gets Delta = 1), written in the layout of
 * dvdq_pack_weights.  blob_out: dvdq_weight_blob_bytes(N, K) bytes, 256-byte aligned; `out`
 * (host) describes it.  N % 8 == 0, N > 0. */
dvdq_status dvdq_quantize_weights_symmetric(const void* W_bf16, int64_t N, int64_t K, int64_t ldw,
                                            int32_t rot_block, void* blob_out,
                                            dvdq_weights* out /* host */, void* cuda_stream);

/* ---- (0') offline weight quantizer: Bounded-init Grid Refinement, Alg. 1 / Sec. 3.1 ---------
 *
 * For every output channel (row) on its own -- the objective || W - Delta (W_q - z) ||_F with
 * one (Delta, z) per row separates over rows -- and for every shrink step i = 1, 2, ... with
 * delta_l = delta_u = (max - min) / n_steps:
 *     clip the row to [min + i delta_l, max - i delta_u]; MinMax grid of the clipped row;
 *     quantize the unclipped row on it; then repeat
 *         Delta' = <W_q - z, w> / <W_q - z, W_q - z>,
 *         z'     = clamp(round(mean(W_q) - mean(w) / Delta'), 0, 15),
 *         W_q'   = clamp(round(w / Delta') + z', 0, 15)
 *     until the row error improves by less than eps (or max_iter rounds); the best grid seen wins.
 * (Alg. 1 as printed reuses one letter for rows and shrink steps, lets its bounds cross, and
 * stops on a test that is true at once; the statement above is the reading built here.)
 *
 *   W_rot      [N, K] fp32, row-major, dense: the weights ALREADY rotated (W~ = W R)
 *   n_steps    shrink steps across the row's range (the paper's n; e.g. 100); eps >= 0; max_iter >= 0
 *   Wq_out     [N, K] uint8 codes 0..15, delta_out [N] fp32, zero_out [N] int32 0..15:
 *              exactly the inputs of dvdq_pack_weights
 * All arithmetic is fp64 (round half to even).  K % 64 == 0, K <= 16384. */
dvdq_status dvdq_bgr_quantize(const float* W_rot, int64_t N, int64_t K, int32_t n_steps, double eps, int32_t max_iter,
                              uint8_t* Wq_out, float* delta_out, int32_t* zero_out, void* cuda_stream);

/* ---- (2) low-bit GEMM + dequantizing epilogue: Eq. 10, Y = X^ Lambda W^^T ----------
 *
 *   acc_in = sum_k c_ik (u_nk - z_n)      exact int32 (tensor cores, int8 operands)
 *   y_in   = bf16( acc_in * s_i * Delta_n + bias_n )   fp32 arithmetic, one rounding
 *   block-wise scales: y_in = bf16( Delta_n * sum_g s_ig * acc_ing + bias_n ), acc_ing the exact
 *   int32 sum over block g, the sum over blocks in fp32
 *   act == 1 applies tanh-GELU to the rounded value and rounds to bf16 again.
 *
 *   codes, scales, code_sums   outputs of dvdq_rotate_quantize for the same M, K, q
 *   w            host handle from dvdq_pack_weights
 *   bias_bf16    [N] bf16 or NULL
 *   Y_bf16       [M, N] bf16, row pitch ldy elements; 16-byte aligned, ldy % 8 == 0
 */
dvdq_status dvdq_qgemm(const void* codes, const float* scales, const int32_t* code_sums,
                       int64_t M, const dvdq_act_quant* q, const dvdq_weights* w /* host */,
                       const void* bias_bf16, int32_t act, void* Y_bf16, int64_t ldy,
                       void* cuda_stream);

/* ---- (2) of one layer fused with (1) of the next: Eq. 10 applied layer after layer --------
 *
 * Where one quantized layer feeds another (Y of this layer is X of the next, Eq. 10 for both),
 * the bf16 output need not exist: this call runs dvdq_qgemm's contraction and epilogue
 * arithmetic (same roundings: bf16, optional tanh-GELU, bf16 again) and then, inside the same
 * kernel, the next layer's activation transform on those bf16 values: x~ = y R with
 * R = I (x) H_256 / 16, one absmax scale per token and per 256 rotated channels, codes
 * c = round_half_even(x~ / s).  It writes what dvdq_rotate_quantize would write for Y:
 *
 *   q           this layer's quantizer: scale_group = 0 (one scale per token); either code layout
 *   q_next      the next layer's: rot_block = 256, scale_group = 256, container_bits = 8,
 *               bits 4, 6 or 8; the next layer's weights must be rotated with B = 256
 *   codes_next      [M, N] one int8 per code (dvdq_act_codes_bytes_q(M, N, q_next) bytes)
 *   scales_next     [M, N / 256] fp32,  code_sums_next [M, N / 256] int32
 *   Y_bf16_or_null  if not NULL, the bf16 output [M, N] (row pitch ldy) is written as well
 * N % 256 == 0 (a 256-wide tile of the GEMM owns whole rotation blocks and scale groups of its
 * rows, which is what makes the fusion possible).  Other options give DVDQ_ERR_UNSUPPORTED. */
dvdq_status dvdq_qgemm_fused_rq(const void* codes, const float* scales, const int32_t* code_sums,
                                int64_t M, const dvdq_act_quant* q, const dvdq_weights* w /* host */,
                                const void* bias_bf16, int32_t act, const dvdq_act_quant* q_next,
                                void* codes_next, float* scales_next, int32_t* code_sums_next,
                                void* Y_bf16_or_null, int64_t ldy, void* cuda_stream);

/* ---- (1)+(2): one quantized linear layer ------------------------------------------
 * workspace: dvdq_qlinear_workspace_bytes(M, K, q) bytes, 256-byte aligned.  Given
 * dvdq_weight_operand_bytes(N, K) + 256 bytes more (and M >= 1024, no operand in `w` already) the call writes the int8 weight operand behind the codes first, as
 * dvdq_widen_weights would, and the GEMM reads it from there: same result bits, faster GEMM. */
dvdq_status dvdq_qlinear(const void* X_bf16, int64_t M, int64_t ldx, const dvdq_act_quant* q,
                         const dvdq_weights* w /* host */, const void* bias_bf16, int32_t act,
                         void* Y_bf16, int64_t ldy, void* workspace, size_t workspace_bytes,
                         void* cuda_stream);

/* ---- (1)+(2) for callers that cannot allocate device memory -------------------------
 *
 * The paper has no counterpart to this entry point; it exists for integration reasons only.
 *
 * Some hosts of this library cannot hand it a workspace: code running inside a region where
 * cudaMalloc is forbidden or would synchronise the device (a plugin called from another
 * framework's execution engine, a real-time loop that must not touch the allocator, a
 * process whose memory pool is owned and sized by someone else).  For them this variant of
 * dvdq_qlinear keeps the intermediate activation codes, scales and code sums in a fixed
 * array that is part of the library image itself: DVDQ_STATIC_SCRATCH_BYTES of device
 * memory, reserved on every GPU that loads the library for as long as the process lives.
 * The call allocates nothing and frees nothing.  Inputs and outputs are still the caller's.
 *
 *   - The problem must fit: dvdq_qlinear_workspace_bytes(M, K, q) <= DVDQ_STATIC_SCRATCH_BYTES,
 *     otherwise DVDQ_ERR_WORKSPACE is returned and nothing is launched.
 *   - The first call on each device looks up the array's device address (once per device,
 *     with that device current).  Make that first call outside any stream capture.
 *   - Every call on a device uses the SAME array.  Calls that may overlap on the GPU (two
 *     streams, two host threads) race on it; serialise them.  The array keeps the previous
 *     call's contents; the call overwrites every byte it later reads, so nothing needs clearing.
 * All other arguments and rules are those of dvdq_qlinear. */
#define DVDQ_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u)
dvdq_status dvdq_qlinear_static(const void* X_bf16, int64_t M, int64_t ldx, const dvdq_act_quant* q,
                                const dvdq_weights* w /* host */, const void* bias_bf16, int32_t act,
                                void* Y_bf16, int64_t ldy, void* cuda_stream);

/* ---- delta-Guided Bit Switching: Sec. 3.3, Eq. "B_{t_i}" ----------------------------------
 *
 * The activation bit width of the whole model is chosen per denoising step from the
 * accumulated relative L1 change of the model output F:
 *     L1(F, t) = || F_t - F_{t-1} ||_1 / || F_{t-1} ||_1,
 *     B_{t_i}  = b_low  while  sum_{t = t_p}^{t_{i-1}} L1(F, t) <  delta,
 *                b_high once   sum                              >= delta  (and the sum restarts at 0).
 * Reading where the paper is silent: before the first output exists the sum is empty (= 0), so
 * the first step runs at b_low unless delta == 0; delta == 0 gives b_high on every step.
 *
 * dvdq_gbs_l1_terms  one pass over F_t and F_{t-1} (bf16, n elements each, 16-byte aligned):
 *                    terms_out[0] = || F_t - F_{t-1} ||_1, terms_out[1] = || F_{t-1} ||_1 as
 *                    fp64 on the DEVICE (two doubles, 8-byte aligned; zeroed by the call).
 * The state and the three functions below live on the HOST; the caller copies the two terms
 * back once per step and feeds them to dvdq_gbs_observe. */
typedef struct {
    double  delta;        /* threshold on the accumulated relative change */
    int32_t b_low;        /* bit width of redundant steps: 4, 6 or 8 */
    int32_t b_high;       /* bit width of critical steps, >= b_low */
    double  accumulated;  /* sum of L1(F, t) since the last reset */
    int64_t steps;        /* decisions taken so far */
    int64_t high_steps;   /* of which b_high */
} dvdq_gbs_state;

dvdq_status dvdq_gbs_l1_terms(const void* F_t_bf16, const void* F_prev_bf16, int64_t n,
                              double* terms_out /* device, [2] */, void* cuda_stream);
dvdq_status dvdq_gbs_init(dvdq_gbs_state* g /* host */, double delta, int32_t b_low, int32_t b_high);
/* Bit width for the step about to run; resets the sum when it answers b_high.  0 if g is NULL. */
int32_t dvdq_gbs_next_bits(dvdq_gbs_state* g /* host */);
/* Adds L1(F, t) = l1_change / l1_prev of the step that just finished.  An all-zero F_{t-1}
 * counts as relative change 1 if F_t differs from it, else 0. */
dvdq_status dvdq_gbs_observe(dvdq_gbs_state* g /* host */, double l1_change, double l1_prev);

/* ---- test / debug entry points (so that no caller depends on the packed layouts) ---- */

/* The raw accumulators of dvdq_qgemm: acc_out [M, N] int32, row pitch ldacc elements. */
dvdq_status dvdq_qgemm_int32(const void* codes, const int32_t* code_sums, int64_t M,
                             const dvdq_act_quant* q, const dvdq_weights* w /* host */,
                             int32_t* acc_out, int64_t ldacc, void* cuda_stream);

/* Natural-order codes [M, K] int8 -> packed buffer (+ code sums); the inverse of the next one. */
dvdq_status dvdq_pack_act_codes(const int8_t* codes_nat, int64_t M, int64_t K,
                                const dvdq_act_quant* q, void* codes_out, int32_t* code_sums_out,
                                void* cuda_stream);
/* Packed buffer -> natural-order codes [M, K] int8. */
dvdq_status dvdq_unpack_act_codes(const void* codes, int64_t M, int64_t K,
                                  const dvdq_act_quant* q, int8_t* codes_nat, void* cuda_stream);
/* Blob -> Wq [N, K] uint8 (0..15), delta [N], zero [N]. */
dvdq_status dvdq_unpack_weights(const dvdq_weights* w /* host */, uint8_t* Wq, float* delta,
                                int32_t* zero, void* cuda_stream);

/* Ceiling of the int8 tensor pipe for the roofline of dvdq_qgemm (Eq. 10's contraction): every
 * CTA pair issues `iters` (1 .. 2^20) k-blocks of four 256 x 256 x 32 tcgen05.mma.kind::i8 on
 * operands that stay in shared memory -- no loads, no widening, no epilogue.  *ops_out (host,
 * may be NULL) receives the integer operations of the launch (2 per multiply-add); time the
 * call with CUDA events on the stream. */
dvdq_status dvdq_int8_mma_ceiling(int32_t iters, int64_t* ops_out /* host */, void* cuda_stream);

/* Exercises the bounded-wait error path without harming the device: one warp waits on a
 * barrier nobody arrives on, gives up after limit_ns (1 .. 1e9) and returns normally; afterwards
 * dvdq_last_device_status() reports DVDQ_ERR_DEVICE_TIMEOUT with detail 8. */
dvdq_status dvdq_debug_wait_timeout(uint64_t limit_ns, void* cuda_stream);

/* Reads (and clears) the device-side status word of the current device; synchronizes
 * the device.  DVDQ_OK, or DVDQ_ERR_DEVICE_TIMEOUT with `detail` (host, may be NULL)
 * set to a code identifying the wait that gave up. */
dvdq_status dvdq_last_device_status(uint32_t* detail /* host */);

/* Library version, for the Python binding's sanity check. */
int32_t dvdq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DVDQ_H_ */
