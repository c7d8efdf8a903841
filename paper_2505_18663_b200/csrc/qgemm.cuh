// Low-bit GEMM with dequantizing epilogue (Eq. 10, Y = X^ Lambda W^^T; Sec. 3.1 DeQuant).
//
//   acc_in = sum_k c_ik (u_nk - z_n),   y_in = bf16(acc_in * s_i * Delta_n + bias_n)
//
// Persistent, warp-specialised sm_100a kernel for CTA PAIRS (cluster of two, one CTA per SM).
// A pair owns an output tile of 256 tokens x 192 channels and issues tcgen05.mma with
// cta_group::2: each CTA holds 128 token rows of the activation operand and 96 of the 192 weight
// rows, so each CTA unpacks only half of the weight tile.  K is consumed in blocks of 128 codes.
// The limiter of this kernel is shared-memory bandwidth (TMA writes, the unpack warps' reads and
// writes, the tensor core's operand reads), which is why
//   * the widened ACTIVATION operand never touches shared memory: the unpack warps write it to
//     tensor memory with tcgen05.st and the MMA takes A from there;
//   * the pair splits the weight tile.
//
// Roles per CTA (22 warps; the unpack warps come in two groups that take alternate k-blocks):
//   warp 0      TMA producer: packed 4/6-bit activation rows (this CTA's 128 tokens) and packed
//               4-bit weight rows (this CTA's 96 channels) -> shared-memory ring.
//   warps 6-13  widen activation codes to int8 and store them to tensor memory (one thread per
//               token row; warp w may touch tensor-memory lanes 32*(w%4)..+31).
//   warps 14-21 widen weight codes to int8 into the 128-byte-swizzled K-major layout in shared memory.
//               A 4-bit two's-complement nibble masked into the HIGH half of a byte is the int8
//               value 16*code, a 6-bit code shifted to the top of a byte is 4*code; the factor
//               (256 or 64 per product) is an exact shift of the int32 accumulator in the
//               epilogue.  Weights are stored as (u - 8); the rest of the zero point,
//               -(z_n - 8) * sum_k c_ik, is a rank-1 integer correction in the epilogue.
//   warp 1      (leader CTA only) one thread issues tcgen05.mma.cta_group::2.kind::i8, 256x192x32
//               per instruction, into one of two 192-column int32 accumulators per CTA;
//               tcgen05.commit signals "stage free" / "accumulator full" to both CTAs.
//   warps 2-5   epilogue of this CTA's 128 rows: tcgen05.ld, shift, zero-point correction, scale,
//               bias, optional tanh-GELU, one bf16 rounding, TMA stores.  Overlaps the next
//               tile's mainloop through the second accumulator.
//
// Tensor memory (512 columns per CTA): [0,192) and [192,384) accumulators, [384,512) four
// activation stages of 32 columns (128 int8 per row).
//
// Every wait is bounded (see mbar_wait); a role that gives up raises its CTA's abort flag and
// all roles walk to the common exit, where the pair synchronises and tensor memory is released.
#pragma once

#include <stdlib.h>

#include "dvdq_common.cuh"

namespace dvdq {

constexpr int kBM = 128;            // token rows per CTA (the pair's tile has 2 * kBM)
constexpr int kBN = 192;            // channels of the pair's tile
constexpr int kBNh = kBN / 2;       // weight rows widened by each CTA
constexpr int kBK = 128;            // codes per k-block (one unpack + four MMA instructions)
constexpr int kPK = 2 * kBK;        // codes per TMA load of activation rows: 128-byte rows (A4), the width TMA moves at full rate
constexpr int kPackedStages = 4, kWideStages = 4;
constexpr int kWPackedStages = 6;   // ring of packed weight half-tiles (one k-block each)
constexpr int kUnpackGroups = 2;   // unpack warps come in groups that take alternate k-blocks
constexpr int kAWarps = 4 * kUnpackGroups, kWWarps = 4 * kUnpackGroups, kEpilogueWarps = 4;
constexpr int kFirstEpilogueWarp = 2, kFirstAWarp = 6, kFirstWWarp = kFirstAWarp + kAWarps;
constexpr int kStageArrivals = (kAWarps + kWWarps) / kUnpackGroups;  // unpack warps that fill one wide stage, per CTA
constexpr int kGemmThreads = (2 + kEpilogueWarps + kAWarps + kWWarps) * 32;
constexpr int kTmemCols = 512;
constexpr int kTmemACol = 2 * kBN;  // first column of the activation stages
constexpr int kAColsPerStage = kBK / 4;
static_assert(kTmemACol + kWideStages * kAColsPerStage <= kTmemCols, "tensor memory budget");
static_assert(kWideStages % 2 == 0, "the MMA warp takes the wide stages in pairs");

// BLK: block-wise activation scales (tile of 128 channels, see the kernel).
template <int BITS, bool BLK>
struct GemmSmem {
    static constexpr int BN = BLK ? 128 : kBN, BNh = BN / 2;
    static constexpr int kWideW = BNh * kBK;                     // int8 weight half-tile, swizzled
    static constexpr int kWideOff = 0;                            // 1024-byte aligned tiles first
    static_assert(BITS == 4 || BITS == 6, "codes stored one int8 each take qgemm_ss_kernel");
    static constexpr int kALo = kBM * kPK / 2;  // A4 codes / A6 low plane (128-byte rows)
    static constexpr int kPStages = kPackedStages;
    static constexpr int kAHi = (BITS == 6) ? kBM * kPK / 4 : 0;  // packed high plane (64-byte rows)
    static constexpr int kPackedStage = kALo + kAHi;              // activation codes of two k-blocks
    static constexpr int kPackedOff = kWideOff + kWideStages * kWideW;
    static constexpr int kStageOutOff = kPackedOff + kPStages * kPackedStage;  // 1024-byte aligned
    static constexpr int kStageOutPerWarp = 2 * 32 * 128;  // two buffers of 32 rows x 64 bf16
    static constexpr int kWPackedOff = kStageOutOff + kEpilogueWarps * kStageOutPerWarp;
    static constexpr int kWPacked = BNh * kBK / 2;              // packed weight half-tile of one k-block (64-byte rows)
    static constexpr int kConstOff = kWPackedOff + kWPackedStages * kWPacked;
    static constexpr int kConstPerWarp = 3 * BN * 4;  // delta, zero-point rest, bias
    static constexpr int kBarOff = kConstOff + kEpilogueWarps * kConstPerWarp;
    static constexpr int kNumBars = 2 * kPackedStages + 2 * kWideStages + 5 + 2 * kWPackedStages;
    static constexpr int kMiscOff = kBarOff + kNumBars * 8;
    static constexpr int kTotal = kMiscOff + 16 + 1024;  // + slack for manual 1024-byte alignment
    static_assert(kWideW % 1024 == 0 && kPackedStage % 1024 == 0, "swizzled tiles need 1024-byte alignment");
    static_assert(kTotal <= 232448, "more than the 227 KB of shared memory a CTA can have");
};

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

template <int BITS, bool RAW, bool BLK>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
qgemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmAhi,
             const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmY,
             const float* __restrict__ scales,
             const int32_t* __restrict__ sums, const float* __restrict__ delta, const int32_t* __restrict__ zc,
             const __nv_bfloat16* __restrict__ bias, __nv_bfloat16* __restrict__ Y, int64_t ldy,
             int32_t* __restrict__ acc_out, int64_t ldacc, int M, int N, int K, int act, int spr) {
    using S = GemmSmem<BITS, BLK>;
    constexpr int BN = S::BN, BNh = S::BNh;  // channels of the pair's tile / weight rows per CTA
    extern __shared__ uint8_t smem_raw[];
    // identical in both CTAs of the pair: the dynamic shared window starts at the same offset
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();       // 0 = leader of the pair
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_n = (N + BN - 1) / BN, num_m = (M + 2 * kBM - 1) / (2 * kBM);
    const int num_tiles = num_m * num_n;
    const int KB2 = (K + kPK - 1) / kPK;  // activation loads per tile; a k-block past K reads zeros
    const int KB = 2 * KB2;
    // one accumulator per tile, or (block-wise scales) one per tile and scale group: spr groups of
    // 128, 256 or 1024 codes per token, i.e. 1, 2 or 8 k-blocks per accumulator (K is a multiple of 256)
    const int NG = BLK ? spr : 1;
    const int KBG = BLK ? KB / spr : KB;  // k-blocks per accumulator

    const uint32_t bar0 = sbase + S::kBarOff;
    auto pk_full = [&](int s) { return bar0 + 8u * s; };
    auto pk_empty = [&](int s) { return bar0 + 8u * (kPackedStages + s); };
    auto wd_full = [&](int s) { return bar0 + 8u * (2 * kPackedStages + s); };                  // leader's copy is used
    auto wd_empty = [&](int s) { return bar0 + 8u * (2 * kPackedStages + kWideStages + s); };   // one per CTA
    auto acc_full = [&](int s) { return bar0 + 8u * (2 * kPackedStages + 2 * kWideStages + s); };      // one per CTA
    auto acc_empty = [&](int s) { return bar0 + 8u * (2 * kPackedStages + 2 * kWideStages + 2 + s); }; // leader's copy
    const uint32_t drain_bar = bar0 + 8u * (2 * kPackedStages + 2 * kWideStages + 4);
    auto wp_full = [&](int s) { return drain_bar + 8u * (1 + s); };
    auto wp_empty = [&](int s) { return drain_bar + 8u * (1 + kWPackedStages + s); };
    volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + S::kMiscOff);  // [0] tmem base, [1] abort
    volatile uint32_t* abort_flag = misc + 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPackedStages; ++s) { mbar_init(pk_full(s), 1); mbar_init(pk_empty(s), kAWarps); }
        for (int s = 0; s < kWideStages; ++s) { mbar_init(wd_full(s), 2 * kStageArrivals); mbar_init(wd_empty(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full(s), 1); mbar_init(acc_empty(s), 2 * kEpilogueWarps); }
        mbar_init(drain_bar, 1);
        for (int s = 0; s < kWPackedStages; ++s) { mbar_init(wp_full(s), 1); mbar_init(wp_empty(s), kWWarps / kUnpackGroups); }
        misc[1] = 0u;
        fence_mbar_init();
    }
    if (warp == 1) {
        // each CTA allocates all of its own tensor memory, so both allocations start at column 0
        tmem_alloc(sbase + S::kMiscOff, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers are initialised before anyone arrives on them
    tc_fence_after();
    const uint32_t tmem_base = misc[0];

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            tma_prefetch_desc(&tmA);
            if (BITS == 6) tma_prefetch_desc(&tmAhi);
            tma_prefetch_desc(&tmW);
            uint32_t st = 0, ph = 0, issued = 0, wst = 0, wph = 0, wissued = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
                const int m0 = (tile / num_n) * (2 * kBM) + (int)rank * kBM;
                const int n0 = (tile % num_n) * BN + (int)rank * BNh;
                for (int sb = 0; ok && sb < KB2; ++sb) {
                    if (!mbar_wait(pk_empty(st), ph ^ 1u, abort_flag, kWaitPackedEmpty)) { ok = false; break; }
                    const uint32_t dst = sbase + S::kPackedOff + st * S::kPackedStage;
                    mbar_arrive_expect_tx(pk_full(st), S::kPackedStage);
                    tma_load_2d(dst, &tmA, pk_full(st), sb * (kPK / 2), m0);
                    if (BITS == 6) tma_load_2d(dst + S::kALo, &tmAhi, pk_full(st), sb * (kPK / 4), m0);
                    ++issued;
                    if (++st == S::kPStages) { st = 0; ph ^= 1u; }
                    for (int h = 0; h < 2; ++h) {  // the weight rows of the two k-blocks this load covers
                        if (!mbar_wait(wp_empty(wst), wph ^ 1u, abort_flag, kWaitPackedEmpty)) { ok = false; break; }
                        mbar_arrive_expect_tx(wp_full(wst), S::kWPacked);
                        tma_load_2d(sbase + S::kWPackedOff + wst * S::kWPacked, &tmW, wp_full(wst), (2 * sb + h) * (kBK / 2), n0);
                        ++wissued;
                        if (++wst == kWPackedStages) { wst = 0; wph ^= 1u; }
                    }
                }
            }
            if (!ok) {
                // Giving up: let copies already in flight land before the CTA exits (bounded).
                const uint32_t n_out = issued < (uint32_t)S::kPStages ? issued : (uint32_t)S::kPStages;
                for (uint32_t i = 0; i < n_out; ++i) {
                    const uint32_t s = (st + S::kPStages - 1 - i) % S::kPStages;
                    const uint32_t p = (s < st) ? ph : (ph ^ 1u);
                    for (int it = 0; it < (1 << 16) && !mbar_try_wait(pk_full(s), p); ++it) {}
                }
                const uint32_t w_out = wissued < (uint32_t)kWPackedStages ? wissued : (uint32_t)kWPackedStages;
                for (uint32_t i = 0; i < w_out; ++i) {
                    const uint32_t s = (wst + kWPackedStages - 1 - i) % kWPackedStages;
                    const uint32_t p = (s < wst) ? wph : (wph ^ 1u);
                    for (int it = 0; it < (1 << 16) && !mbar_try_wait(wp_full(s), p); ++it) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        // The whole warp walks the loop (warp-uniform control flow); one elected lane issues.
        if (rank == 0) {
            constexpr uint32_t idesc = umma_idesc_s8s8s32(2 * kBM, BN);
            uint32_t st = 0, ph = 0, lt = 0;  // lt: accumulators started so far
            uint32_t acc = 0;                  // the accumulator in use (0 or 1)
            bool ok = true;
            // Starts the next accumulator once the epilogue has drained its previous contents.
            auto acquire = [&]() {
                acc = lt & 1u;
                if (!mbar_wait_warp(acc_empty(acc), ((lt >> 1) & 1u) ^ 1u, abort_flag, kWaitAccEmpty)) ok = false;
                tc_fence_after();
                ++lt;
            };
            for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
                // Two k-blocks per trip (KB is even, and so is kWideStages): the tensor core's queue
                // is short, so every cycle this warp spends between two issues is a bubble in the
                // MMA stream; pairing halves the waits, votes and bookkeeping per k-block.  An
                // accumulator covers KBG k-blocks (a power of two, or the whole of K): with KBG = 1
                // the two blocks of a trip go to different accumulators.
                int kin = 0;  // k-blocks issued into the accumulator in use
                if constexpr (!BLK) {
                    acquire();  // one accumulator per tile
                    if (!ok) break;
                }
                for (int kb = 0; ok && kb < KB; kb += 2) {
                    uint32_t acc_h[2];
                    bool first_h[2], last_h[2];
                    if constexpr (BLK) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            first_h[h] = kin == 0;
                            if (first_h[h]) acquire();
                            acc_h[h] = acc;
                            last_h[h] = ++kin == KBG;
                            if (last_h[h]) kin = 0;
                        }
                        if (!ok) break;
                    } else {
                        acc_h[0] = acc_h[1] = acc;
                        first_h[0] = kb == 0;
                        first_h[1] = last_h[0] = false;
                        last_h[1] = kb + 2 >= KB;
                    }
                    if (!mbar_wait_warp(wd_full(st), ph, abort_flag, kWaitWideFull)) { ok = false; break; }
                    if (!mbar_wait_warp(wd_full(st + 1), ph, abort_flag, kWaitWideFull)) { ok = false; break; }
                    tc_fence_after();
                    if (elect_one()) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint32_t d_tmem = tmem_base + acc_h[h] * BN;
                            const uint32_t a_tmem = tmem_base + kTmemACol + (st + h) * kAColsPerStage;
                            const uint64_t bdesc = umma_desc_sw128_kmajor(sbase + S::kWideOff + (st + h) * S::kWideW);
#pragma unroll
                            for (int k = 0; k < kBK / 32; ++k)  // +32 int8 along K = +8 columns of A, +2 in B's 16-byte address field
                                tc_mma_i8_ts_pair(d_tmem, a_tmem + 8u * k, bdesc + 2u * k, idesc, (first_h[h] && k == 0) ? 0u : 1u);
                            tc_commit_pair(wd_empty(st + h), 3);
                            if (last_h[h]) tc_commit_pair(acc_full(acc_h[h]), 3);
                        }
                    }
                    __syncwarp();
                    st += 2;
                    if (st == kWideStages) { st = 0; ph ^= 1u; }
                }
            }
            // nothing issued by this warp may still be running when the pair leaves
            if (elect_one()) tc_commit_pair(drain_bar, 1);
            __syncwarp();
            mbar_wait(drain_bar, 0u, abort_flag, kWaitDrain);
        }
        __syncwarp();
    } else if (warp < kFirstAWarp) {
        // ------------------------------------------------------------ epilogue
        const int q = warp & 3;  // tensor-memory lane quarter this warp may read
        const int ew = warp - kFirstEpilogueWarp;
        const uint32_t c_delta = sbase + S::kConstOff + ew * S::kConstPerWarp;  // shared addresses of float[BN] each
        const uint32_t c_zc = c_delta + BN * 4;    // (z_n - 8) as a float: exact, |.| <= 8
        const uint32_t c_bias = c_zc + BN * 4;
        const uint32_t stg0 = sbase + S::kStageOutOff + ew * S::kStageOutPerWarp;
        constexpr int kShift = (BITS == 4) ? 8 : 6;  // log2 of (A factor 16 or 4) x (W factor 16)
        if (!RAW && lane == 0) tma_prefetch_desc(&tmY);
        if constexpr (BLK) {
            // Block-wise scales: every block of 1024 codes has its own int32 accumulator (the two
            // accumulators alternate) and its own scale per token.  This warp keeps the running
            // fp32 sum over blocks of its 32 rows in tensor-memory columns [256, 384) -- lanes only
            // it touches -- and dequantizes after the last block.  acc_g here is the sum over the
            // stored codes (u - 8); the rest of the zero point is one term per row:
            //     y = Delta_n * (sum_g s_ig acc_g - (z_n - 8) T_i) + bias_n,  T_i = sum_g s_ig S_ig.
            constexpr uint32_t kFloatCol = 2 * BN;
            uint32_t lt = 0, nstore = 0;
            for (int tile = pair; tile < num_tiles; tile += num_pairs) {
                const int m0 = (tile / num_n) * (2 * kBM) + (int)rank * kBM, n0 = (tile % num_n) * BN;
                __syncwarp();
#pragma unroll
                for (int i = 0; i < BN / 32; ++i) {
                    const int c = lane + 32 * i, n = n0 + c;
                    const bool okn = n < N;
                    sts32f(c_delta + 4 * c, okn ? __ldg(delta + n) : 0.f);
                    sts32f(c_zc + 4 * c, okn ? (float)__ldg(zc + n) : 0.f);
                    sts32f(c_bias + 4 * c, (okn && bias != nullptr) ? __bfloat162float(bias[n]) : 0.f);
                }
                __syncwarp();
                const int row = m0 + q * 32 + lane;
                const bool row_ok = row < M;
                const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
                // the zero-point term T_i = sum_g s_ig S_ig (each S_ig is exact in fp32) is added up group by
                // group, from loads issued a group ahead
                float T = 0.f;
                float s_next = row_ok ? __ldg(scales + (int64_t)row * NG) : 0.f;
                float S_next = row_ok ? (float)__ldg(sums + (int64_t)row * NG) : 0.f;
                bool ok = true;
                for (int g = 0; g < NG; ++g, ++lt) {
                    const uint32_t a = lt & 1u, aph = (lt >> 1) & 1u;
                    const float s_k = s_next * (1.0f / (float)(1 << kShift));
                    T = fmaf(s_next, S_next, T);
                    if (g + 1 < NG && row_ok) {
                        s_next = __ldg(scales + (int64_t)row * NG + g + 1);
                        S_next = (float)__ldg(sums + (int64_t)row * NG + g + 1);
                    }
                    if (!mbar_wait(acc_full(a), aph, abort_flag, kWaitAccFull)) { ok = false; break; }
                    tc_fence_after();
                    const bool last = g == NG - 1;
#pragma unroll 1
                    for (int hc = 0; hc < BN / 32; ++hc) {
                        uint32_t r[32], f[32];
                        tmem_ld_32x32(tmem_base + a * BN + hc * 32 + lane_addr, r);
                        if (g > 0) tmem_ld_32x32(tmem_base + kFloatCol + hc * 32 + lane_addr, f);
                        tmem_ld_wait();
#pragma unroll
                        for (int t = 0; t < 32; ++t)  // running sum of s_ig * acc_g (the raw accumulator is 2^kShift x the true one)
                            f[t] = __float_as_uint(fmaf((float)(int32_t)r[t], s_k, g > 0 ? __uint_as_float(f[t]) : 0.f));
                        if (!last) {
                            tmem_st_32x32(tmem_base + kFloatCol + hc * 32 + lane_addr, f);
                            continue;
                        }
                        // last block: dequantize, round, stage 64 columns per TMA store
                        if ((hc & 1) == 0) {
                            if (lane == 0) tma_store_wait_read<1>();
                            __syncwarp();
                        }
                        const uint32_t buf = stg0 + (nstore & 1u) * (32 * 128);
#pragma unroll
                        for (int j = 0; j < 32; j += 8) {
                            const float4 d0 = lds128f(c_delta + 4 * (hc * 32 + j)), d1 = lds128f(c_delta + 4 * (hc * 32 + j + 4));
                            const float4 z0 = lds128f(c_zc + 4 * (hc * 32 + j)), z1 = lds128f(c_zc + 4 * (hc * 32 + j + 4));
                            const float4 b0 = lds128f(c_bias + 4 * (hc * 32 + j)), b1 = lds128f(c_bias + 4 * (hc * 32 + j + 4));
                            const float dl[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
                            const float zz[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
                            const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                            uint32_t pk[4];
#pragma unroll
                            for (int t = 0; t < 8; t += 2) {
                                float y0 = fmaf(fmaf(-zz[t], T, __uint_as_float(f[j + t])), dl[t], bb[t]);
                                float y1 = fmaf(fmaf(-zz[t + 1], T, __uint_as_float(f[j + t + 1])), dl[t + 1], bb[t + 1]);
                                if (act == 1) {
                                    y0 = gelu_tanh_f32(__bfloat162float(__float2bfloat16_rn(y0)));
                                    y1 = gelu_tanh_f32(__bfloat162float(__float2bfloat16_rn(y1)));
                                }
                                __nv_bfloat162 b2 = __floats2bfloat162_rn(y0, y1);
                                pk[t >> 1] = *reinterpret_cast<uint32_t*>(&b2);
                            }
                            const int ch = (4 * (hc & 1) + (j >> 3)) ^ (lane & 7);
                            sts128(buf + lane * 128 + ch * 16, pk[0], pk[1], pk[2], pk[3]);
                        }
                        if (hc & 1) {
                            fence_proxy_async_smem();
                            __syncwarp();
                            const int nb = n0 + (hc >> 1) * 64;
                            if (lane == 0 && nb < N && m0 + q * 32 < M) {
                                tma_store_2d(&tmY, buf, nb, m0 + q * 32);
                                tma_store_commit();
                            }
                            ++nstore;
                        }
                    }
                    // the accumulator is read: the MMA warp may have it back before this warp's
                    // running sums have landed (nobody else touches those columns)
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty(a), 0));
                    if (!last) tmem_st_wait();
                }
                if (!ok) break;
            }
            if (lane == 0) tma_store_wait_all();
            __syncwarp();
        } else {
        uint32_t lt = 0, nstore = 0;
        for (int tile = pair; tile < num_tiles; tile += num_pairs, ++lt) {
            const uint32_t a = lt & 1u, aph = (lt >> 1) & 1u;
            const int m0 = (tile / num_n) * (2 * kBM) + (int)rank * kBM, n0 = (tile % num_n) * BN;
            __syncwarp();
            {   // per-channel constants of this tile: all loads in flight at once, then the stores
                float cd[BN / 32], cz[BN / 32], cb[BN / 32];
#pragma unroll
                for (int i = 0; i < BN / 32; ++i) {
                    const int n = n0 + lane + 32 * i;
                    const bool okn = n < N;
                    cd[i] = okn ? __ldg(delta + n) : 0.f;
                    cz[i] = okn ? (float)__ldg(zc + n) : 0.f;
                    cb[i] = (okn && bias != nullptr) ? __bfloat162float(bias[n]) : 0.f;
                }
#pragma unroll
                for (int i = 0; i < BN / 32; ++i) {
                    const int c = lane + 32 * i;
                    sts32f(c_delta + 4 * c, cd[i]);
                    sts32f(c_zc + 4 * c, cz[i]);
                    sts32f(c_bias + 4 * c, cb[i]);
                }
            }
            __syncwarp();
            if (!mbar_wait(acc_full(a), aph, abort_flag, kWaitAccFull)) break;
            tc_fence_after();
            const int row = m0 + q * 32 + lane;
            const bool row_ok = row < M;
            const float s_i = (!RAW && row_ok) ? scales[row] : 0.f;
            int32_t S_i = row_ok ? sums[(int64_t)row * spr] : 0;
            if (RAW && row_ok)
                for (int g = 1; g < spr; ++g) S_i += sums[(int64_t)row * spr + g];  // spr == 1 unless the scales are block-wise
            const float S_f = (float)S_i;  // |sum of codes| <= K * 32 < 2^24: exact
            const float s_k = s_i * (1.0f / (float)(1 << kShift)), nS_k = -S_f * (float)(1 << kShift);
            const uint64_t s2 = f2_pack(s_k, s_k), negS2 = f2_pack(nS_k, nS_k);
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + a * BN + c * 32 + ((uint32_t)(q * 32) << 16), r);
                tmem_ld_wait();
                const int nb = n0 + c * 32;
                if (RAW) {
                    int32_t* dst = acc_out + (int64_t)row * ldacc + nb;
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const float4 zq = lds128f(c_zc + 4 * (c * 32 + j));
                        int4 o;
                        o.x = ((int32_t)r[j] >> kShift) - __float2int_rn(zq.x) * S_i;
                        o.y = ((int32_t)r[j + 1] >> kShift) - __float2int_rn(zq.y) * S_i;
                        o.z = ((int32_t)r[j + 2] >> kShift) - __float2int_rn(zq.z) * S_i;
                        o.w = ((int32_t)r[j + 3] >> kShift) - __float2int_rn(zq.w) * S_i;
                        if (row_ok && nb + j < N) *reinterpret_cast<int4*>(dst + j) = o;
                    }
                } else {
                    // Two chunks of 32 columns fill one staging buffer of 32 rows x 128 bytes, which
                    // leaves as ONE TMA store (128-byte rows are what TMA moves at full rate).  The
                    // buffer used two stores ago must have been read by its store.
                    if ((c & 1) == 0) {
                        if (lane == 0) tma_store_wait_read<1>();
                        __syncwarp();
                    }
                    const uint32_t buf = stg0 + (nstore & 1u) * (32 * 128);
#pragma unroll
                    for (int j = 0; j < 32; j += 8) {
                        const float4 d0 = lds128f(c_delta + 4 * (c * 32 + j)), d1 = lds128f(c_delta + 4 * (c * 32 + j + 4));
                        const float4 z0 = lds128f(c_zc + 4 * (c * 32 + j)), z1 = lds128f(c_zc + 4 * (c * 32 + j + 4));
                        const float4 b0 = lds128f(c_bias + 4 * (c * 32 + j)), b1 = lds128f(c_bias + 4 * (c * 32 + j + 4));
                        const float dl[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
                        const float zz[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
                        const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                        float v[8];
                        // The raw accumulator is (256 or 64) x the true one: at most 22 significant
                        // bits, so its conversion is exact and the factor moves into the per-row
                        // constants: y = (raw - zz * S * 2^k) * (s * 2^-k * delta) + bias, on fp32 pairs.
#pragma unroll
                        for (int t = 0; t < 8; t += 2) {
                            const uint64_t raw2 = f2_pack((float)(int32_t)r[j + t], (float)(int32_t)r[j + t + 1]);
                            const uint64_t acc2 = f2_fma(f2_pack(zz[t], zz[t + 1]), negS2, raw2);   // exact
                            const uint64_t y2 = f2_fma(acc2, f2_mul(f2_pack(dl[t], dl[t + 1]), s2), f2_pack(bb[t], bb[t + 1]));
                            f2_unpack(y2, v[t], v[t + 1]);
                        }
                        if (act == 1) {
#pragma unroll
                            for (int t = 0; t < 8; ++t) v[t] = gelu_tanh_f32(__bfloat162float(__float2bfloat16_rn(v[t])));
                        }
                        uint32_t pk[4];
#pragma unroll
                        for (int t = 0; t < 4; ++t) {
                            __nv_bfloat162 b2 = __floats2bfloat162_rn(v[2 * t], v[2 * t + 1]);
                            pk[t] = *reinterpret_cast<uint32_t*>(&b2);
                        }
                        // 128-byte rows, 16-byte chunk index XORed with row % 8: the layout a
                        // 128B-swizzled TMA store reads, and conflict-free for this per-row write.
                        const int ch = (4 * (c & 1) + (j >> 3)) ^ (lane & 7);
                        sts128(buf + lane * 128 + ch * 16, pk[0], pk[1], pk[2], pk[3]);
                    }
                    if (c & 1) {
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0 && nb - 32 < N && m0 + q * 32 < M) {
                            tma_store_2d(&tmY, buf, nb - 32, m0 + q * 32);
                            tma_store_commit();
                        }
                        ++nstore;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty(a), 0));
        }
        if (!RAW && lane == 0) tma_store_wait_all();
        __syncwarp();
        }
    } else if (warp < kFirstWWarp) {
        // ------------------------------------------------------------ widen activation codes -> tensor memory
        const int q = warp & 3;
        const uint32_t grp = (uint32_t)(warp - kFirstAWarp) >> 2;
        const int row = q * 32 + lane;                     // row of this CTA's tile = tensor-memory lane
        // One packed stage holds two k-blocks; group g unpacks the g-th half of every row.
        const uint32_t sw_lo = (uint32_t)row & 7u;         // 128-byte-swizzled TMA tile: chunk ^= row % 8
        const uint32_t sw_hi = (uint32_t)(row >> 1) & 3u;  // 64-byte-swizzled TMA tile: chunk ^= (row / 2) % 4
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        uint32_t j = 0;  // k-blocks seen so far; this warp takes those with j % kUnpackGroups == grp
        bool ok = true;
        const uint32_t rt_zero = runtime_zero();
        for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
            for (int kb = 0; kb < KB; ++kb) {
                const uint32_t jj = j++;
                if (jj % kUnpackGroups != grp) continue;
                const uint32_t sb = jj / kUnpackGroups;
                const uint32_t pst = sb % S::kPStages, pph = (sb / S::kPStages) & 1u;
                const uint32_t wst = jj % kWideStages, wph = (jj / kWideStages) & 1u;
                if (!mbar_wait(pk_full(pst), pph, abort_flag, kWaitPackedFull)) { ok = false; break; }
                const uint32_t pk = sbase + S::kPackedOff + pst * S::kPackedStage;
                const uint32_t prow = pk + row * (kPK / 2);
                uint32_t r[32];  // r[2i] / r[2i+1]: even / odd codes of packed word i, the K order the weights use too
                uint32_t h[8];
                uint32_t loaded = 0u;
                if (BITS == 6) {
                    const uint32_t hrow = pk + S::kALo + row * (kPK / 4);
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        const uint4 p = lds128(hrow + (((2u * grp + (uint32_t)c) ^ sw_hi) << 4));
                        h[4 * c] = p.x; h[4 * c + 1] = p.y; h[4 * c + 2] = p.z; h[4 * c + 3] = p.w;
                        loaded ^= p.w;
                    }
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint4 p = lds128(prow + (((4u * grp + (uint32_t)c) ^ sw_lo) << 4));
                    const uint32_t w[4] = {p.x, p.y, p.z, p.w};
                    loaded ^= p.w;
#pragma unroll
                    for (int jw = 0; jw < 4; ++jw) {
                        const int i = 4 * c + jw;
                        if (BITS == 4) {
                            r[2 * i] = (w[jw] << 4) & 0xF0F0F0F0u;
                            r[2 * i + 1] = w[jw] & 0xF0F0F0F0u;
                        } else {
                            const uint32_t hh = h[i >> 1];
                            const int a2 = 2 * (i & 1);
                            r[2 * i] = ((w[jw] << 2) & 0x3C3C3C3Cu) | ((hh << (6 - 2 * a2)) & 0xC0C0C0C0u);
                            r[2 * i + 1] = ((w[jw] >> 2) & 0x3C3C3C3Cu) | ((hh << (4 - 2 * a2)) & 0xC0C0C0C0u);
                        }
                    }
                }
                // the codes are widened in registers before the stage of tensor memory is known to be free
                loaded &= rt_zero;
                __syncwarp();
                if (lane == 0) mbar_arrive_after_loads(pk_empty(pst), loaded);
                if (!mbar_wait(wd_empty(wst), wph ^ 1u, abort_flag, kWaitWideEmpty)) { ok = false; break; }
                tc_fence_after();
                tmem_st_32x32(tmem_base + kTmemACol + wst * kAColsPerStage + lane_addr, r);
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(wd_full(wst), 0));
            }
        }
    } else {
        // ------------------------------------------------------------ widen weight codes -> shared memory
        const uint32_t grp = (uint32_t)(warp - kFirstWWarp) >> 2;
        const int u = (threadIdx.x - kFirstWWarp * 32) & 127;  // thread of its group of four warps
        uint32_t j = 0;
        bool ok = true;
        const uint32_t rt_zero = runtime_zero();
        for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
            for (int kb = 0; kb < KB; ++kb) {
            const uint32_t jj = j++;
            if (jj % kUnpackGroups != grp) continue;
            const uint32_t pst = jj % kWPackedStages, pph = (jj / kWPackedStages) & 1u;
            const uint32_t wst = jj % kWideStages, wph = (jj / kWideStages) & 1u;
            if (!mbar_wait(wp_full(pst), pph, abort_flag, kWaitPackedFull)) { ok = false; break; }
            const uint32_t pw = sbase + S::kWPackedOff + pst * S::kWPacked;
            const uint32_t wdW = sbase + S::kWideOff + wst * S::kWideW;
            // BNh rows x 4 chunks of 32 nibbles, stored as (u - 8); widened in registers before the
            // wide stage is known to be free
            constexpr int kPieces = (BNh * 4) / 128;
            uint32_t e[kPieces][4], o[kPieces][4];
            uint32_t loaded = 0u;
#pragma unroll
            for (int it = 0; it < kPieces; ++it) {
                const int qi = it * 128 + u, row = qi >> 2, ck = qi & 3;
                const uint4 p = lds128(pw + row * (kBK / 2) + ck * 16);
                const uint32_t w[4] = {p.x, p.y, p.z, p.w};
                loaded ^= p.w;
#pragma unroll
                for (int jw = 0; jw < 4; ++jw) { e[it][jw] = (w[jw] << 4) & 0xF0F0F0F0u; o[it][jw] = w[jw] & 0xF0F0F0F0u; }
            }
            loaded &= rt_zero;
            __syncwarp();
            if (lane == 0) mbar_arrive_after_loads(wp_empty(pst), loaded);  // the packed rows are in registers
            if (!mbar_wait(wd_empty(wst), wph ^ 1u, abort_flag, kWaitWideEmpty)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int it = 0; it < kPieces; ++it) {
                const int qi = it * 128 + u, row = qi >> 2, ck = qi & 3;
                const uint32_t drow = wdW + (row >> 3) * 1024 + (row & 7) * 128;
                sts128(drow + (((2 * ck) ^ (row & 7)) << 4), e[it][0], o[it][0], e[it][1], o[it][1]);
                sts128(drow + (((2 * ck + 1) ^ (row & 7)) << 4), e[it][2], o[it][2], e[it][3], o[it][3]);
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(wd_full(wst), 0));
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer may read this CTA's shared and tensor memory until it is done too
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

template <int BITS, bool RAW, bool BLK>
static dvdq_status launch_qgemm_t(const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                  const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy,
                                  int32_t* acc_out, int64_t ldacc, cudaStream_t st) {
    using S = GemmSmem<BITS, BLK>;
    const int64_t K = w.K, N = w.N;
    const BlobLayout L = blob_layout(N, K);
    const uint8_t* blob = static_cast<const uint8_t*>(w.blob);
    const uint64_t pitch = (uint64_t)act_row_bytes(K, BITS);
    CUtensorMap tmA, tmAhi, tmW, tmY;
    if (!make_byte_map(&tmA, codes, (uint64_t)K / 2, (uint64_t)M, pitch, kPK / 2, kBM, CU_TENSOR_MAP_SWIZZLE_128B))
        return DVDQ_ERR_CUDA;
    if (BITS == 6) {
        if (!make_byte_map(&tmAhi, static_cast<const uint8_t*>(codes) + K / 2, (uint64_t)K / 4, (uint64_t)M, pitch,
                           kPK / 4, kBM, CU_TENSOR_MAP_SWIZZLE_64B))
            return DVDQ_ERR_CUDA;
    } else {
        tmAhi = tmA;
    }

    if (!make_byte_map(&tmW, blob + L.codes_offset, (uint64_t)K / 2, (uint64_t)N, (uint64_t)K / 2, kBK / 2, S::BNh,
                       CU_TENSOR_MAP_SWIZZLE_NONE))
        return DVDQ_ERR_CUDA;
    if (RAW) {
        tmY = tmA;  // unused
    } else if (!make_out_map(&tmY, Y, (uint64_t)N, (uint64_t)M, (uint64_t)ldy)) {
        return DVDQ_ERR_CUDA;
    }

    auto kern = qgemm_kernel<BITS, RAW, BLK>;
    static PerDevice<int> cache;
    const int max_pairs = resident_pairs(cache, kern, kGemmThreads, S::kTotal);
    if (max_pairs == 0) return DVDQ_ERR_CUDA;
    const int64_t tiles = ((M + 2 * kBM - 1) / (2 * kBM)) * ((N + S::BN - 1) / S::BN);
    const unsigned pairs = (unsigned)(tiles < max_pairs ? tiles : max_pairs);
    kern<<<2 * pairs, kGemmThreads, S::kTotal, st>>>(tmA, tmAhi, tmW, tmY, scales, sums,
                                                     reinterpret_cast<const float*>(blob + L.delta_offset),
                                                     reinterpret_cast<const int32_t*>(blob + L.zc_offset),
                                                     static_cast<const __nv_bfloat16*>(bias), static_cast<__nv_bfloat16*>(Y), ldy,
                                                     acc_out, ldacc, (int)M, (int)N, (int)K, act, spr);
    return cuda_status(cudaGetLastError());
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
inline bool use_ps_kernel() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("DVDQ_PS"); v = (e && e[0] == '0') ? 0 : 1; }
    return v == 1;
}

// qgemm_fat.cuh: the same with block-wise activation scales
static dvdq_status launch_qgemm_blk(int sb, const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                    const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy, cudaStream_t st);

inline dvdq_status launch_qgemm(const void* codes, const float* scales, const int32_t* sums, int64_t M,
                                const dvdq_act_quant& q, const dvdq_weights& w, const void* bias, int act,
                                void* Y, int64_t ldy, int32_t* acc_out, int64_t ldacc, cudaStream_t st) {
    if (M == 0) return DVDQ_OK;
    // The int32 output does not depend on the scales: it always runs the per-token kernel, which
    // adds up the code sums of a token's blocks itself.
    const bool raw = acc_out != nullptr;
    const int spr = q.scale_group != 0 ? (int)(w.K / q.scale_group) : 1;  // code sums (and scales) per token
    const int sb = storage_bits(q);
    if (!raw && q.scale_group != 0)
        return launch_qgemm_blk(sb, codes, scales, sums, spr, M, w, bias, act, Y, ldy, st);
    if (sb == 8 && (raw || q.scale_group == 0))
        return raw ? launch_qgemm_ss<true>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st)
                   : launch_qgemm_ss<false>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st);
    if ((sb == 4 || sb == 6) && (raw || q.scale_group == 0) && use_ps_kernel())
        return raw ? launch_qgemm_ps<true>(sb, codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st)
                   : launch_qgemm_ps<false>(sb, codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st);
#define DVDQ_GEMM_CASE(B)                                                                                          \
    if (sb == B) {                                                                                                 \
        if (raw) return launch_qgemm_t<B, true, false>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st); \
        if (q.scale_group != 0)                                                                                    \
            return launch_qgemm_t<B, false, true>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st);      \
        return launch_qgemm_t<B, false, false>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st);         \
    }
    DVDQ_GEMM_CASE(4)
    DVDQ_GEMM_CASE(6)
#undef DVDQ_GEMM_CASE
    return DVDQ_ERR_BITS;
}

}  // namespace dvdq
