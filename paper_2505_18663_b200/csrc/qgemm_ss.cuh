// The GEMM with one activation scale per token (Eq. 10):
//
//   acc_in = sum_k c_ik (u_nk - z_n),   y_in = bf16(acc_in * s_i * Delta_n + bias_n).
//
// A CTA pair owns a tile of 256 tokens x 256 channels: tcgen05.mma.cta_group::2.kind::i8
// 256x256x32 with BOTH operands from shared memory (K-major rows of 128 bytes, 128-byte swizzle),
// two 256-column int32 accumulators in tensor memory.  The 4-bit weights are widened to int8 by
// warps (each CTA its 128 of the 256 rows).  The activation codes come in one of two ways (ABITS):
//   8      one int8 per code (8-bit activations, or 4- / 6-bit codes kept in byte containers): TMA
//          puts them into the operand stages as they are and no warp ever touches them;
//   4, 6   packed: TMA fills a ring of packed tiles and eight more warps widen them into the
//          operand stages, exactly as the weight warps do for their operand.
//
// Roles per CTA (16, 20 or 24 warps):
//   warp 0      TMA producer of the activation codes: this CTA's 128 token rows of a k-block,
//               into the operand stages (ring of 6: the depth covers the copy's latency) or into
//               the ring of packed tiles.
//   warp 15     TMA producer of packed weight rows, into a ring for the widening warps.
//   warp 1      (leader CTA) issues the MMAs; tcgen05.commit frees the stage in both CTAs.
//   warps 2-5   epilogue (tcgen05.ld, zero-point term, scales, bias, GELU, bf16, TMA stores), one
//               warp per tensor-memory lane quarter.
//   warps 6-13  widen weight codes into the operand stage (two groups, alternate k-blocks).
//   warp 14     idle: the TMA copies into operand stages of BOTH CTAs of a pair count their bytes on
//               the leader's barrier of the stage (cp.async.bulk.tensor with .cta_group::2), which
//               the leader's producer arms for both, so nobody has to tell the leader that the
//               peer's rows have landed (+1-3 % over a forwarding warp).
//   warps 16-19 (codes in bytes, EW = 8 only) a second epilogue warp per lane quarter; each then
//               takes 128 of the 256 columns.  With one warp per quarter the epilogue, not the MMA,
//               sets the pace of layers with a short K or a GELU (+13..25 % there); where the
//               mainloop sets it, the extra warps only compete with the widening warps (-2..7 %).
//   warps 16-23 (packed codes, EW = 4) widen activation codes into the operand stage (two groups);
//               with EW = 8 the weight warps 6-13 widen both operands of their k-block instead.
// WOP (the weight handle carries the codes one int8 each, dvdq_widen_weights): warp 15's TMA copies
// go straight into a ring of six weight operand stages, counted on the leader's barrier, and no
// warp widens weights; next to packed activation codes warps 6-9 then widen those, as a third group.
// With codes in bytes no warp touches an operand at all then, and one "full" / "empty" barrier per
// stage serves both operands' rings (half the waits and commits of the MMA warp); with packed codes
// and EW = 8 warps 6-13 widen the activation codes only.
// Every wait is bounded (mbar_wait).
#pragma once

#include "qgemm.cuh"

namespace dvdq {

constexpr int kSsBN = 256, kSsBNh = kSsBN / 2;
constexpr int kSsAStages = 6;        // activation tiles of one k-block (filled by TMA: its latency sets the depth)
constexpr int kSsStages = 4;         // widened weight half-tiles of one k-block (filled by warps)
constexpr int kSsWPackedStages = 4;  // ring of packed weight half-tiles
constexpr int kSsFirstWWarp = 6, kSsWWarps = 8, kSsFwdWarp = kSsFirstWWarp + kSsWWarps, kSsWProducerWarp = kSsFwdWarp + 1;
constexpr int kSsFirstEpilogueWarp2 = kSsWProducerWarp + 1;  // a multiple of 4: warp w reads tensor-memory lanes 32 * (w % 4)..
static_assert(kSsFirstEpilogueWarp2 % 4 == 0, "lane quarters");
static_assert(kSsStages % 2 == 0, "the MMA warp takes the weight stages in pairs");

constexpr int kSsFirstAWarp = kSsFirstEpilogueWarp2;  // packed activation codes: eight more warps widen them (no second set of epilogue warps then)
constexpr int kSsAWarps = 8;

// ABITS: how the activation codes arrive.  8: one int8 each, TMA writes the operand stages themselves.
// 4 / 6: packed; TMA fills a ring of packed tiles and warps widen them into the operand stages, as
// for the weights (a 4-bit code masked into the high half of a byte is 16 x code, a 6-bit code
// moved to the top of a byte 4 x code; the factor is shifted out of the accumulator).
// WOP: the weight operand exists in global memory already (one int8 per code, in the operand's K
// order): TMA writes the weight stages too and no warp widens weights.
template <int ABITS, bool WOP = false>
struct SsSmem {
    static constexpr int BN = kSsBN, BNh = BN / 2;
    static constexpr bool kPackedA = ABITS != 8;
    static constexpr int kAStages = kPackedA ? kSsStages : kSsAStages;  // operand stages of the activation tile
    static constexpr int kWStages = WOP ? kSsAStages : kSsStages;       // operand stages of the weight half-tile
    static constexpr int kWPackedStages = WOP ? 0 : kSsWPackedStages;   // ring of packed weight half-tiles
    static constexpr int kWpBars = WOP ? kWStages : kSsWPackedStages;   // "this CTA's TMA copy of weight rows has landed"
    static constexpr int kA = kBM * kBK;              // activation tile of one k-block (int8, swizzled)
    static constexpr int kW = BNh * kBK;              // widened weight half-tile
    static constexpr int kWPacked = BNh * kBK / 2;    // packed weight half-tile (64-byte rows)
    static constexpr int kALo = kPackedA ? kBM * kBK / 2 : 0;            // packed codes / low plane (64-byte rows)
    static constexpr int kAHi = ABITS == 6 ? kBM * kBK / 4 : 0;          // high plane of 6-bit codes (32-byte rows)
    static constexpr int kAPacked = kALo + kAHi;
    static constexpr int kAPackedStages = !kPackedA ? 0 : (ABITS == 6 ? 3 : 4);  // what fits
    static constexpr int kAOff = 0;
    static constexpr int kWOff = kAOff + kAStages * kA;
    static constexpr int kWPackedOff = kWOff + kWStages * kW;
    static constexpr int kAPackedOff = kWPackedOff + kWPackedStages * kWPacked;
    static constexpr int kStageOutOff = kAPackedOff + kAPackedStages * kAPacked;  // 1024-byte aligned
    // 16 KB of staging and 12 KB of constants whether four or eight epilogue warps share them: one
    // buffer of 32 rows x 64 (or 32) bf16 each, and delta / zero-point rest / bias of 256 (or 128) columns
    static constexpr int kStageOutBytes = 4 * 32 * 128;
    static constexpr int kConstOff = kStageOutOff + kStageOutBytes;
    static constexpr int kConstBytes = 4 * 3 * BN * 4;
    static constexpr int kBarOff = kConstOff + kConstBytes;
    static constexpr int kNumBars = 3 * kAStages + 2 * kWStages + 5 + 2 * kWpBars + 2 * kAPackedStages;
    static_assert(kWStages % 2 == 0, "the MMA warp takes the weight stages in pairs");
    static constexpr int kMiscOff = kBarOff + kNumBars * 8;
    static constexpr int kTotal = kMiscOff + 16 + 1024;
    static_assert(kStageOutOff % 1024 == 0, "swizzled tiles need 1024-byte alignment");
    static_assert(kTotal <= 232448, "more than the 227 KB of shared memory a CTA can have");
};

// D[tmem] (+)= A[smem] * B[smem]^T for a CTA pair, int8 operands, int32 accumulators: each CTA
// holds its 128 rows of A and half of B's rows at the same shared-memory offsets.
__device__ __forceinline__ void tc_mma_i8_ss_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

template <int ABITS>
constexpr int ss_warps(int ew) { return ew == 8 ? kSsFirstEpilogueWarp2 + 4 : (ABITS != 8 ? kSsFirstAWarp + kSsAWarps : kSsFirstEpilogueWarp2); }

template <int ABITS, bool RAW, int EW, bool WOP>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(ss_warps<ABITS>(EW) * 32, 1)
qgemm_ss_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmAhi, const __grid_constant__ CUtensorMap tmW,
                const __grid_constant__ CUtensorMap tmY, const float* __restrict__ scales,
                const int32_t* __restrict__ sums, const float* __restrict__ delta, const int32_t* __restrict__ zc,
                const __nv_bfloat16* __restrict__ bias, int32_t* __restrict__ acc_out, int64_t ldacc,
                int M, int N, int K, int act, int spr) {
    using S = SsSmem<ABITS, WOP>;
    constexpr int BN = S::BN, BNh = S::BNh;
    constexpr bool kPackedA = S::kPackedA;
    constexpr int AST = S::kAStages, APS = S::kAPackedStages, WST = S::kWStages, WPB = S::kWpBars;
    // packed codes with the second set of epilogue warps (layers whose epilogue sets the pace): the
    // eight weight warps widen both operands of their k-block instead of eight more warps
    constexpr bool kWidenBoth = kPackedA && EW == 8;
    // both operands by TMA into rings of the same depth: one "full" and one "empty" barrier per stage serve both
    constexpr bool kOneRing = WOP && !kPackedA;
    static_assert(!kOneRing || S::kAStages == S::kWStages, "one ring: the operands' stages advance together");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_n = (N + BN - 1) / BN, num_m = (M + 2 * kBM - 1) / (2 * kBM);
    const int num_tiles = num_m * num_n;
    const int KB = 2 * ((K + 2 * kBK - 1) / (2 * kBK));  // even; a k-block past K reads zeros

    const uint32_t bar0 = sbase + S::kBarOff;
    auto a_full = [&](int s) { return bar0 + 8u * s; };                          // a slot kept for the layout's sake: copies count on a_ready
    auto a_ready = [&](int s) { return bar0 + 8u * (AST + s); };                 // leader's copy: both CTAs' rows of the stage are in place
    auto a_empty = [&](int s) { return bar0 + 8u * (2 * AST + s); };             // one per CTA
    const uint32_t barw = bar0 + 8u * (3 * AST);
    auto ops_full = [&](int s) { return barw + 8u * s; };                        // widened weights; leader's copy is used
    auto ops_empty = [&](int s) { return barw + 8u * (WST + s); };         // one per CTA
    auto acc_full = [&](int s) { return barw + 8u * (2 * WST + s); };      // one per CTA
    auto acc_empty = [&](int s) { return barw + 8u * (2 * WST + 2 + s); }; // leader's copy
    const uint32_t drain_bar = barw + 8u * (2 * WST + 4);
    auto wp_full = [&](int s) { return drain_bar + 8u * (1 + s); };        // this CTA's TMA copy of weight rows (packed ring, or the stage itself)
    auto wp_empty = [&](int s) { return drain_bar + 8u * (1 + WPB + s); };
    auto apk_full = [&](int s) { return drain_bar + 8u * (1 + 2 * WPB + s); };        // packed activation tiles (TMA)
    auto apk_empty = [&](int s) { return drain_bar + 8u * (1 + 2 * WPB + APS + s); };
    volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + S::kMiscOff);  // [0] tmem base, [1] abort
    volatile uint32_t* abort_flag = misc + 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < AST; ++s) {
            mbar_init(a_full(s), 1);
            // packed codes: the widening warps of both CTAs; codes in bytes: the leader's producer arms it for the
            // TMA copies of both CTAs (in the one-ring mode its weight producer as well)
            mbar_init(a_ready(s), kPackedA ? 2 * (kSsAWarps / kUnpackGroups) : kOneRing ? 2 : 1);
            mbar_init(a_empty(s), 1);
        }
        for (int s = 0; s < APS; ++s) { mbar_init(apk_full(s), 1); mbar_init(apk_empty(s), kSsAWarps / kUnpackGroups); }
        for (int s = 0; s < WST; ++s) { mbar_init(ops_full(s), WOP ? 1 : 2 * (kSsWWarps / kUnpackGroups)); mbar_init(ops_empty(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full(s), 1); mbar_init(acc_empty(s), 2 * EW); }
        mbar_init(drain_bar, 1);
        for (int s = 0; s < WPB; ++s) { mbar_init(wp_full(s), 1); mbar_init(wp_empty(s), kSsWWarps / kUnpackGroups); }
        misc[1] = 0u;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(sbase + S::kMiscOff, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = misc[0];

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer, activation rows
        if (lane == 0) {
            tma_prefetch_desc(&tmA);
            if (ABITS == 6) tma_prefetch_desc(&tmAhi);
            // one int8 per code: straight into the operand stages; packed codes: into the ring the widening warps read
            constexpr int kRing = kPackedA ? APS : AST;
            constexpr uint32_t kBytes = kPackedA ? S::kAPacked : S::kA;
            auto ring_full = [&](int s) { return kPackedA ? apk_full(s) : a_full(s); };
            auto ring_empty = [&](int s) { return kPackedA ? apk_empty(s) : a_empty(s); };
            uint32_t st = 0, ph = 0, issued = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
                const int m0 = (tile / num_n) * (2 * kBM) + (int)rank * kBM;
                for (int kb = 0; ok && kb < KB; ++kb) {
                    if (!mbar_wait(ring_empty(st), ph ^ 1u, abort_flag, kWaitWideEmpty)) { ok = false; break; }
                    if (!kPackedA) {
                        // both CTAs' copies count their bytes on the leader's "full" barrier of the stage
                        if (rank == 0) mbar_arrive_expect_tx(a_ready(st), 2 * S::kA);
                        tma_load_2d_pair(sbase + S::kAOff + st * S::kA, &tmA, map_to_cta(a_ready(st), 0), kb * kBK, m0);
                        ++issued;
                        if (++st == kRing) { st = 0; ph ^= 1u; }
                        continue;
                    }
                    mbar_arrive_expect_tx(ring_full(st), kBytes);
                    if (kPackedA) {
                        const uint32_t dst = sbase + S::kAPackedOff + st * S::kAPacked;
                        tma_load_2d(dst, &tmA, ring_full(st), kb * (kBK / 2), m0);
                        if (ABITS == 6) tma_load_2d(dst + S::kALo, &tmAhi, ring_full(st), kb * (kBK / 4), m0);
                    } else {
                        tma_load_2d(sbase + S::kAOff + st * S::kA, &tmA, ring_full(st), kb * kBK, m0);
                    }
                    ++issued;
                    if (++st == kRing) { st = 0; ph ^= 1u; }
                }
            }
            if (!ok && !kPackedA) {
                // Giving up (some wait ran out after seconds): copies issued before that have long landed;
                // a short bounded pause covers the last ones, whose barrier is not this CTA's to poll.
                for (int it = 0; it < 64; ++it) __nanosleep(1000);
            } else if (!ok) {
                // Giving up: let copies already in flight land before the CTA exits (bounded).
                const uint32_t n_out = issued < (uint32_t)kRing ? issued : (uint32_t)kRing;
                for (uint32_t i = 0; i < n_out; ++i) {
                    const uint32_t s = (st + kRing - 1 - i) % kRing;
                    const uint32_t p = (s < st) ? ph : (ph ^ 1u);
                    for (int it = 0; it < (1 << 16) && !mbar_try_wait(ring_full(s), p); ++it) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == kSsWProducerWarp) {
        // ------------------------------------------------------------ TMA producer, packed weight rows
        if (lane == 0) {
            tma_prefetch_desc(&tmW);
            uint32_t wst = 0, wph = 0, wissued = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
                const int n0 = (tile % num_n) * BN + (int)rank * BNh;
                for (int kb = 0; ok && kb < KB; ++kb) {
                    if (WOP) {
                        // straight into the operand stage, which the MMA's commit frees; both CTAs' copies
                        // count their bytes on the leader's "full" barrier of the stage, like the activation rows
                        const uint32_t full = kOneRing ? a_ready(wst) : ops_full(wst);
                        if (!mbar_wait(kOneRing ? a_empty(wst) : ops_empty(wst), wph ^ 1u, abort_flag, kWaitWideEmpty)) { ok = false; break; }
                        if (rank == 0) mbar_arrive_expect_tx(full, 2 * S::kW);
                        tma_load_2d_pair(sbase + S::kWOff + wst * S::kW, &tmW, map_to_cta(full, 0), kb * kBK, n0);
                    } else {
                        if (!mbar_wait(wp_empty(wst), wph ^ 1u, abort_flag, kWaitPackedEmpty)) { ok = false; break; }
                        mbar_arrive_expect_tx(wp_full(wst), S::kWPacked);
                        tma_load_2d(sbase + S::kWPackedOff + wst * S::kWPacked, &tmW, wp_full(wst), kb * (kBK / 2), n0);
                    }
                    ++wissued;
                    if (++wst == WPB) { wst = 0; wph ^= 1u; }
                }
            }
            if (!ok && WOP) {
                for (int it = 0; it < 64; ++it) __nanosleep(1000);
            } else if (!ok) {
                const uint32_t w_out = wissued < (uint32_t)WPB ? wissued : (uint32_t)WPB;
                for (uint32_t i = 0; i < w_out; ++i) {
                    const uint32_t s = (wst + WPB - 1 - i) % WPB;
                    const uint32_t p = (s < wst) ? wph : (wph ^ 1u);
                    for (int it = 0; it < (1 << 16) && !mbar_try_wait(wp_full(s), p); ++it) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        if (rank == 0) {
            constexpr uint32_t idesc = umma_idesc_s8s8s32(2 * kBM, BN);
            uint32_t st = 0, ph = 0, sa = 0, pa = 0, lt = 0;
            bool ok = true;
            for (int tile = pair; ok && tile < num_tiles; tile += num_pairs, ++lt) {
                const uint32_t a = lt & 1u, aph = (lt >> 1) & 1u;
                if (!mbar_wait_warp(acc_empty(a), aph ^ 1u, abort_flag, kWaitAccEmpty)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + a * BN;
                // Two k-blocks per trip: every cycle between two issues is a bubble in the MMA stream
                for (int kb = 0; kb < KB; kb += 2) {
                    // the activation ring may have an odd number of stages: its second stage of the trip can wrap
                    const uint32_t sa1 = sa + 1 == AST ? 0u : sa + 1, pa1 = sa + 1 == AST ? pa ^ 1u : pa;
                    if (!mbar_wait_warp(a_ready(sa), pa, abort_flag, kWaitPackedFull)) { ok = false; break; }
                    if (!kOneRing && !mbar_wait_warp(ops_full(st), ph, abort_flag, kWaitWideFull)) { ok = false; break; }
                    if (!mbar_wait_warp(a_ready(sa1), pa1, abort_flag, kWaitPackedFull)) { ok = false; break; }
                    if (!kOneRing && !mbar_wait_warp(ops_full(st + 1), ph, abort_flag, kWaitWideFull)) { ok = false; break; }
                    tc_fence_after();
                    if (elect_one()) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint64_t adesc = umma_desc_sw128_kmajor(sbase + S::kAOff + (h ? sa1 : sa) * S::kA);
                            const uint64_t bdesc = umma_desc_sw128_kmajor(sbase + S::kWOff + (st + h) * S::kW);
#pragma unroll
                            for (int k = 0; k < kBK / 32; ++k)  // +32 int8 along K = +2 in the 16-byte address field
                                tc_mma_i8_ss_pair(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (kb | h | k) != 0 ? 1u : 0u);
                            if (!kOneRing) tc_commit_pair(ops_empty(st + h), 3);
                            tc_commit_pair(a_empty(h ? sa1 : sa), 3);
                        }
                        if (kb + 2 >= KB) tc_commit_pair(acc_full(a), 3);
                    }
                    __syncwarp();
                    st += 2;
                    if (st == WST) { st = 0; ph ^= 1u; }
                    sa = sa1 + 1;
                    pa = pa1;
                    if (sa == AST) { sa = 0; pa ^= 1u; }
                }
            }
            if (elect_one()) tc_commit_pair(drain_bar, 1);
            __syncwarp();
            mbar_wait(drain_bar, 0u, abort_flag, kWaitDrain);
        }
        __syncwarp();
    } else if (warp < kSsFirstWWarp || (EW == 8 && warp >= kSsFirstEpilogueWarp2)) {
        // ------------------------------------------------------------ epilogue
        const int q = warp & 3;  // tensor-memory lane quarter this warp may read
        const int half = warp >= kSsFirstEpilogueWarp2 ? 1 : 0;  // EW = 8: which 128 of the tile's 256 columns
        const int ew = 4 * half + q;
        constexpr int CW = BN / (EW / 4);           // columns per warp
        constexpr int RB = EW == 8 ? 64 : 128;  // bytes per row of the staging buffer = of a TMA store
        const uint32_t c_delta = sbase + S::kConstOff + ew * (3 * CW * 4);  // shared addresses of float[CW] each
        const uint32_t c_zc = c_delta + CW * 4;    // (z_n - 8) as a float: exact, |.| <= 8
        const uint32_t c_bias = c_zc + CW * 4;
        const uint32_t stg0 = sbase + S::kStageOutOff + ew * (32 * RB);
        constexpr int kShift = ABITS == 4 ? 8 : ABITS == 6 ? 6 : 4;  // log2 of (A factor 16 / 4 / 1) x (W factor 16)
        if (!RAW && lane == 0) tma_prefetch_desc(&tmY);
        uint32_t lt = 0;
        for (int tile = pair; tile < num_tiles; tile += num_pairs, ++lt) {
            const uint32_t a = lt & 1u, aph = (lt >> 1) & 1u;
            const int m0 = (tile / num_n) * (2 * kBM) + (int)rank * kBM, n0 = (tile % num_n) * BN + half * CW;
            __syncwarp();
            {   // per-channel constants of this warp's columns: all loads in flight at once, then the stores
                float cd[CW / 32], cz[CW / 32], cb[CW / 32];
#pragma unroll
                for (int i = 0; i < CW / 32; ++i) {
                    const int n = n0 + lane + 32 * i;
                    const bool okn = n < N;
                    cd[i] = okn ? __ldg(delta + n) : 0.f;
                    cz[i] = okn ? (float)__ldg(zc + n) : 0.f;
                    cb[i] = (okn && bias != nullptr) ? __bfloat162float(bias[n]) : 0.f;
                }
#pragma unroll
                for (int i = 0; i < CW / 32; ++i) {
                    const int c = lane + 32 * i;
                    sts32f(c_delta + 4 * c, cd[i]);
                    sts32f(c_zc + 4 * c, cz[i]);
                    sts32f(c_bias + 4 * c, cb[i]);
                }
            }
            __syncwarp();
            int row;
            bool row_ok;
            float s_i;
            int32_t S_i;
            // With eight epilogue warps the epilogue sets the pace, and a global-memory latency after the
            // wait for the accumulator would be on every tile's critical path: the row's scale and code
            // sum are loaded before it (+1.5-3.5 % on K = 1536).  With four, the mainloop sets the pace.
            if constexpr (EW == 8) {
                row = m0 + q * 32 + lane;
                row_ok = row < M;
                s_i = (!RAW && row_ok) ? scales[row] : 0.f;
                S_i = row_ok ? sums[(int64_t)row * spr] : 0;
                if (RAW && row_ok)
                    for (int g = 1; g < spr; ++g) S_i += sums[(int64_t)row * spr + g];  // spr == 1 unless the scales are block-wise
                if (!mbar_wait(acc_full(a), aph, abort_flag, kWaitAccFull)) break;
                tc_fence_after();
            } else {
                if (!mbar_wait(acc_full(a), aph, abort_flag, kWaitAccFull)) break;
                tc_fence_after();
                row = m0 + q * 32 + lane;
                row_ok = row < M;
                s_i = (!RAW && row_ok) ? scales[row] : 0.f;
                S_i = row_ok ? sums[(int64_t)row * spr] : 0;
                if (RAW && row_ok)
                    for (int g = 1; g < spr; ++g) S_i += sums[(int64_t)row * spr + g];
            }
            const float S_f = (float)S_i;  // |sum of codes| <= K * 32 < 2^24: exact
            const float s_k = s_i * (1.0f / (float)(1 << kShift)), nS_k = -S_f * (float)(1 << kShift);
            const uint64_t s2 = f2_pack(s_k, s_k), negS2 = f2_pack(nS_k, nS_k);
#pragma unroll 1
            for (int c = 0; c < CW / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(tmem_base + a * BN + half * CW + c * 32 + ((uint32_t)(q * 32) << 16), r);
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
                    // RB / 64 chunks of 32 columns fill the staging buffer (32 rows x RB bytes), which
                    // leaves as one TMA store; the previous store must have read the buffer.
                    if (RB == 64 || (c & 1) == 0) {
                        if (lane == 0) tma_store_wait_read<0>();
                        __syncwarp();
                    }
                    const uint32_t buf = stg0;
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
                        // The layout a swizzled TMA store reads, conflict-free for this per-row write:
                        // 128-byte rows, 16-byte chunk index XORed with row % 8, or 64-byte rows, chunk
                        // index XORed with (row / 2) % 4.
                        const int ch = RB == 128 ? (4 * (c & 1) + (j >> 3)) ^ (lane & 7) : (j >> 3) ^ ((lane >> 1) & 3);
                        sts128(buf + lane * RB + ch * 16, pk[0], pk[1], pk[2], pk[3]);
                    }
                    if (RB == 64 || (c & 1)) {
                        const int x0 = RB == 64 ? nb : nb - 32;
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0 && x0 < N && m0 + q * 32 < M) {
                            tma_store_2d(&tmY, buf, x0, m0 + q * 32);
                            tma_store_commit();
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty(a), 0));
        }
        if (!RAW && lane == 0) tma_store_wait_all();
        __syncwarp();

    } else if (WOP && !kWidenBoth && warp < kSsFwdWarp && !(kPackedA && warp < kSsFirstWWarp + 4)) {
        // the weight operand comes by TMA: these warps have no work (but for the first four next to
        // packed activation codes, which join the activation warps below)
    } else if (!(WOP && !kWidenBoth) && warp < kSsFwdWarp) {
        // ------------------------------------------------------------ widen weight codes -> shared memory
        const uint32_t grp = (uint32_t)(warp - kSsFirstWWarp) >> 2;
        const int u = (threadIdx.x - kSsFirstWWarp * 32) & 127;  // thread of its group of four warps
        uint32_t j = 0;
        bool ok = true;
        const uint32_t rt_zero = runtime_zero();
        for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
            for (int kb = 0; kb < KB; ++kb) {
            const uint32_t jj = j++;
            if (jj % kUnpackGroups != grp) continue;
            if constexpr (kWidenBoth) {
                // this CTA's 128 token rows of the k-block first: the same job on the activation rings
                const uint32_t apst = jj % APS, apph = (jj / APS) & 1u;
                const uint32_t awst = jj % AST, awph = (jj / AST) & 1u;
                if (!mbar_wait(apk_full(apst), apph, abort_flag, kWaitPackedFull)) { ok = false; break; }
                const uint32_t pa = sbase + S::kAPackedOff + apst * S::kAPacked;
                const uint32_t wd = sbase + S::kAOff + awst * S::kA;
                constexpr int kAPieces = (kBM * 4) / 128;
                uint4 pl[kAPieces];
                uint2 ph2[kAPieces];
                uint32_t got = 0u;
#pragma unroll
                for (int it = 0; it < kAPieces; ++it) {
                    const int qi = it * 128 + u, row = qi >> 2, ck = qi & 3;
                    pl[it] = lds128(pa + row * (kBK / 2) + ck * 16);
                    got ^= pl[it].w;
                    if (ABITS == 6) {
                        ph2[it] = lds64(pa + S::kALo + row * (kBK / 4) + ck * 8);
                        got ^= ph2[it].y;
                    }
                }
                got &= rt_zero;
                __syncwarp();
                if (lane == 0) mbar_arrive_after_loads(apk_empty(apst), got);
                if (!mbar_wait(a_empty(awst), awph ^ 1u, abort_flag, kWaitWideEmpty)) { ok = false; break; }
                tc_fence_after();
#pragma unroll
                for (int it = 0; it < kAPieces; ++it) {
                    const int qi = it * 128 + u, row = qi >> 2, ck = qi & 3;
                    const uint32_t w[4] = {pl[it].x, pl[it].y, pl[it].z, pl[it].w};
                    uint32_t e[4], o[4];
#pragma unroll
                    for (int jw = 0; jw < 4; ++jw) {
                        if (ABITS == 4) {
                            e[jw] = (w[jw] << 4) & 0xF0F0F0F0u;
                            o[jw] = w[jw] & 0xF0F0F0F0u;
                        } else {
                            const uint32_t hh = (jw >> 1) ? ph2[it].y : ph2[it].x;
                            const int a2 = 2 * (jw & 1);
                            e[jw] = ((w[jw] << 2) & 0x3C3C3C3Cu) | ((hh << (6 - 2 * a2)) & 0xC0C0C0C0u);
                            o[jw] = ((w[jw] >> 2) & 0x3C3C3C3Cu) | ((hh << (4 - 2 * a2)) & 0xC0C0C0C0u);
                        }
                    }
                    const uint32_t drow = wd + (row >> 3) * 1024 + (row & 7) * 128;
                    sts128(drow + (((2 * ck) ^ (row & 7)) << 4), e[0], o[0], e[1], o[1]);
                    sts128(drow + (((2 * ck + 1) ^ (row & 7)) << 4), e[2], o[2], e[3], o[3]);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(a_ready(awst), 0));
            }
            if constexpr (!WOP) {
                const uint32_t pst = jj % WPB, pph = (jj / WPB) & 1u;
                const uint32_t wst = jj % WST, wph = (jj / WST) & 1u;
                if (!mbar_wait(wp_full(pst), pph, abort_flag, kWaitPackedFull)) { ok = false; break; }
                const uint32_t pw = sbase + S::kWPackedOff + pst * S::kWPacked;
                const uint32_t wdW = sbase + S::kWOff + wst * S::kW;
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
                if (!mbar_wait(ops_empty(wst), wph ^ 1u, abort_flag, kWaitWideEmpty)) { ok = false; break; }
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
                if (lane == 0) mbar_arrive_cluster(map_to_cta(ops_full(wst), 0));
            }
            }
        }
    } else if (kPackedA && EW == 4 && (warp >= kSsFirstAWarp || (WOP && warp >= kSsFirstWWarp && warp < kSsFirstWWarp + 4))) {
        // ------------------------------------------------------------ widen activation codes -> shared memory
        // The same job as the weight warps': this CTA's 128 token rows x 128 codes of a k-block, 16 bytes
        // of packed low bits (and 8 bytes of high bits) per piece, into the K-major 128-byte-swizzled stage.
        if constexpr (kPackedA && EW == 4) {
            // with the weight operand by TMA four of the idle weight warps are a third group: +3 % with 6-bit
            // codes, whose widening is the longest chain (next to weight warps at work a third group cost 3 %)
            constexpr uint32_t kAGroups = WOP ? 3 : 2;
            const uint32_t grp = warp >= kSsFirstAWarp ? (uint32_t)(warp - kSsFirstAWarp) >> 2 : 2u;
            const int u = warp >= kSsFirstAWarp ? (threadIdx.x - kSsFirstAWarp * 32) & 127 : (threadIdx.x - kSsFirstWWarp * 32) & 127;
            uint32_t j = 0;
            bool ok = true;
            const uint32_t rt_zero = runtime_zero();
            for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
                for (int kb = 0; kb < KB; ++kb) {
                    const uint32_t jj = j++;
                    if (jj % kAGroups != grp) continue;
                    const uint32_t pst = jj % APS, pph = (jj / APS) & 1u;
                    const uint32_t wst = jj % AST, wph = (jj / AST) & 1u;
                    if (!mbar_wait(apk_full(pst), pph, abort_flag, kWaitPackedFull)) { ok = false; break; }
                    const uint32_t pa = sbase + S::kAPackedOff + pst * S::kAPacked;
                    const uint32_t wd = sbase + S::kAOff + wst * S::kA;
                    constexpr int kPieces = (kBM * 4) / 128;
                    uint32_t e[kPieces][4], o[kPieces][4];
                    uint32_t loaded = 0u;
#pragma unroll
                    for (int it = 0; it < kPieces; ++it) {
                        const int qi = it * 128 + u, row = qi >> 2, ck = qi & 3;
                        const uint4 p = lds128(pa + row * (kBK / 2) + ck * 16);
                        const uint32_t w[4] = {p.x, p.y, p.z, p.w};
                        loaded ^= p.w;
                        if (ABITS == 4) {
#pragma unroll
                            for (int jw = 0; jw < 4; ++jw) { e[it][jw] = (w[jw] << 4) & 0xF0F0F0F0u; o[it][jw] = w[jw] & 0xF0F0F0F0u; }
                        } else {
                            const uint2 hp = lds64(pa + S::kALo + row * (kBK / 4) + ck * 8);  // bits 5:4 of the piece's 32 codes
                            const uint32_t hh[2] = {hp.x, hp.y};
                            loaded ^= hp.y;
#pragma unroll
                            for (int jw = 0; jw < 4; ++jw) {
                                const int a2 = 2 * (jw & 1);
                                e[it][jw] = ((w[jw] << 2) & 0x3C3C3C3Cu) | ((hh[jw >> 1] << (6 - 2 * a2)) & 0xC0C0C0C0u);
                                o[it][jw] = ((w[jw] >> 2) & 0x3C3C3C3Cu) | ((hh[jw >> 1] << (4 - 2 * a2)) & 0xC0C0C0C0u);
                            }
                        }
                    }
                    loaded &= rt_zero;
                    __syncwarp();
                    if (lane == 0) mbar_arrive_after_loads(apk_empty(pst), loaded);  // the packed rows are in registers
                    if (!mbar_wait(a_empty(wst), wph ^ 1u, abort_flag, kWaitWideEmpty)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int it = 0; it < kPieces; ++it) {
                        const int qi = it * 128 + u, row = qi >> 2, ck = qi & 3;
                        const uint32_t drow = wd + (row >> 3) * 1024 + (row & 7) * 128;
                        sts128(drow + (((2 * ck) ^ (row & 7)) << 4), e[it][0], o[it][0], e[it][1], o[it][1]);
                        sts128(drow + (((2 * ck + 1) ^ (row & 7)) << 4), e[it][2], o[it][2], e[it][3], o[it][3]);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(map_to_cta(a_ready(wst), 0));
                }
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

// bf16 matrix [rows, cols] with row pitch ld elements, tiles of 32 rows x 32 columns, 64-byte
// swizzle (the layout this kernel's epilogue stages its output in).
inline bool make_out_map32(CUtensorMap* tm, const void* base, uint64_t cols, uint64_t rows, uint64_t ld) {
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

// Tensor maps of the activation codes: one int8 each -> tiles of 128 tokens x 128 bytes in the operand
// layout (128-byte swizzle); packed -> 64-byte rows of low bits per k-block (and 32-byte rows of
// high bits for 6-bit codes), unswizzled, as the weights.
template <int ABITS>
static bool make_act_maps(const void* codes, int64_t M, int64_t K, CUtensorMap* tmA, CUtensorMap* tmAhi) {
    if (ABITS == 8) {
        if (!make_byte_map(tmA, codes, (uint64_t)K, (uint64_t)M, (uint64_t)K, kBK, kBM, CU_TENSOR_MAP_SWIZZLE_128B)) return false;
        *tmAhi = *tmA;  // unused
        return true;
    }
    const uint64_t pitch = (uint64_t)act_row_bytes(K, ABITS);
    if (!make_byte_map(tmA, codes, (uint64_t)K / 2, (uint64_t)M, pitch, kBK / 2, kBM, CU_TENSOR_MAP_SWIZZLE_NONE)) return false;
    *tmAhi = *tmA;
    if (ABITS == 6 && !make_byte_map(tmAhi, static_cast<const uint8_t*>(codes) + K / 2, (uint64_t)K / 4, (uint64_t)M, pitch, kBK / 4, kBM,
                                     CU_TENSOR_MAP_SWIZZLE_NONE))
        return false;
    return true;
}

template <int ABITS, bool RAW, int EW, bool WOP>
static dvdq_status launch_qgemm_ss_w(const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                   const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy,
                                   int32_t* acc_out, int64_t ldacc, cudaStream_t st) {
    using S = SsSmem<ABITS, WOP>;
    const int64_t K = w.K, N = w.N;
    const BlobLayout L = blob_layout(N, K);
    const uint8_t* blob = static_cast<const uint8_t*>(w.blob);
    CUtensorMap tmA, tmAhi, tmW, tmY;
    if (!make_act_maps<ABITS>(codes, M, K, &tmA, &tmAhi)) return DVDQ_ERR_CUDA;
    if (WOP ? !make_byte_map(&tmW, w.operand, (uint64_t)K, (uint64_t)N, (uint64_t)K, kBK, S::BNh, CU_TENSOR_MAP_SWIZZLE_128B)
            : !make_byte_map(&tmW, blob + L.codes_offset, (uint64_t)K / 2, (uint64_t)N, (uint64_t)K / 2, kBK / 2, S::BNh,
                             CU_TENSOR_MAP_SWIZZLE_NONE))
        return DVDQ_ERR_CUDA;
    if (RAW) {
        tmY = tmA;  // unused
    } else if (!(EW == 8 ? make_out_map32(&tmY, Y, (uint64_t)N, (uint64_t)M, (uint64_t)ldy)
                         : make_out_map(&tmY, Y, (uint64_t)N, (uint64_t)M, (uint64_t)ldy))) {
        return DVDQ_ERR_CUDA;
    }
    constexpr int kThreads = ss_warps<ABITS>(EW) * 32;
    auto kern = qgemm_ss_kernel<ABITS, RAW, EW, WOP>;
    static PerDevice<int> cache;
    const int max_pairs = resident_pairs(cache, kern, kThreads, S::kTotal);
    if (max_pairs == 0) return DVDQ_ERR_CUDA;
    const int64_t tiles = ((M + 2 * kBM - 1) / (2 * kBM)) * ((N + S::BN - 1) / S::BN);
    const unsigned pairs = (unsigned)(tiles < max_pairs ? tiles : max_pairs);
    kern<<<2 * pairs, kThreads, S::kTotal, st>>>(tmA, tmAhi, tmW, tmY, scales, sums,
                                                   reinterpret_cast<const float*>(blob + L.delta_offset),
                                                   reinterpret_cast<const int32_t*>(blob + L.zc_offset),
                                                   static_cast<const __nv_bfloat16*>(bias), acc_out, ldacc, (int)M, (int)N, (int)K,
                                                   act, spr);
    return cuda_status(cudaGetLastError());
}

// The weight operand as one int8 per code, where the handle has one (dvdq_widen_weights); the int32
// output keeps to the 4-bit codes.
template <int ABITS, bool RAW, int EW>
static dvdq_status launch_qgemm_ss_t(const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                     const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy,
                                     int32_t* acc_out, int64_t ldacc, cudaStream_t st) {
    if constexpr (!RAW) {
        if (w.operand != nullptr)
            return launch_qgemm_ss_w<ABITS, RAW, EW, true>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st);
    }
    return launch_qgemm_ss_w<ABITS, RAW, EW, false>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st);
}

// Codes in bytes: eight epilogue warps where the epilogue would otherwise set the pace: a tile's
// mainloop is K / 128 k-blocks long, its epilogue always 256 columns, and a GELU about doubles the
// epilogue's work.
template <bool RAW>
static dvdq_status launch_qgemm_ss(const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                   const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy,
                                   int32_t* acc_out, int64_t ldacc, cudaStream_t st) {
    const bool wide_epilogue = w.K <= 2048 || (act != 0 && w.K <= 6144);
    return wide_epilogue ? launch_qgemm_ss_t<8, RAW, 8>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st)
                         : launch_qgemm_ss_t<8, RAW, 4>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st);
}

// Packed 4- or 6-bit codes, widened into the shared-memory operand stages by warps.
template <bool RAW>
static dvdq_status launch_qgemm_ps(int bits, const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                   const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy,
                                   int32_t* acc_out, int64_t ldacc, cudaStream_t st) {
    const bool wide_epilogue = w.K <= 2048 || (act != 0 && w.K <= 6144);  // as for codes in bytes
    if (bits == 4)
        return wide_epilogue ? launch_qgemm_ss_t<4, RAW, 8>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st)
                             : launch_qgemm_ss_t<4, RAW, 4>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st);
    return wide_epilogue ? launch_qgemm_ss_t<6, RAW, 8>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st)
                         : launch_qgemm_ss_t<6, RAW, 4>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, acc_out, ldacc, st);
}

}  // namespace dvdq
