// The GEMM for block-wise activation scales with the codes kept one int8 each (Sec. 3.2, last
// paragraph: one scale per token and per group of 128, 256 or 1024 rotated channels):
//
//   y_in = bf16( Delta_n * ( sum_g s_ig * acc_ing  -  (z_n - 8) * T_i ) + bias_n ),
//   acc_ing = sum_{k in group g} c_ik (u_nk - 8)   exact int32,    T_i = sum_g s_ig * S_ig.
//
// Same mainloop as qgemm_ss_kernel (a CTA pair owns 256 tokens x 256 channels, both operands of
// tcgen05.mma.cta_group::2.kind::i8 in shared memory, two 256-column int32 accumulators that
// alternate between scale groups).  What a short group changes is the epilogue's share: every
// group's accumulator has to be read, converted and added into an fp32 running sum, two
// instructions per output element and group against the tensor core's G multiply-adds.  Tensor
// memory is full with the two accumulators, so the running sum lives in REGISTERS: eight epilogue
// warps, one row and 128 columns per thread, with the register file re-divided between the roles
// (setmaxnreg: the loaders and the widening warps give registers up, the epilogue warps take them).
// Roles are aligned to groups of four warps, as that instruction requires:
//   warps 0-3    TMA producer of activation tiles | MMA issuer (leader CTA) | idle | TMA producer of
//                weight rows
//   warps 4-11   widen weight codes into the operand stages (two groups, alternate k-blocks)
//   warps 12-19  epilogue: warp w reads tensor-memory lanes 32 * (w % 4).., columns 128 * ((w - 12) / 4)..
// Every wait is bounded, as in qgemm.cuh.
//
// The same skeleton carries the FUSED variant (kFatFuse): a layer with per-token input scales whose
// epilogue does not write bf16 but applies the NEXT layer's activation transform (Eq. 10 for the
// layer that consumes this output): rotate by H_256, one absmax scale per token and 256 channels,
// round to codes, one int8 each.  A 256-wide tile holds whole rotation blocks and whole scale
// groups of its rows, so nothing leaves the tile: a thread owns one row and 128 columns, does the
// butterflies of seven index bits in registers, and meets the thread that owns the row's other
// 128 columns through the (already drained) accumulator columns in tensor memory for the eighth.
#pragma once

#include "qgemm_ss.cuh"

namespace dvdq {

constexpr int kFatThreads = 20 * 32;
constexpr int kFatFirstWWarp = 4, kFatFirstEpilogueWarp = 12;
// setmaxnreg moves registers between the warps of ONE CTA: what the epilogue warps take must have
// been given up by the others, out of the CTA's allocation at launch (threads x the kernel's
// register count), or the taking warps wait for ever.  The host checks the sum against the compiled
// register count before every first launch (fat_kernel_registers_fit) and refuses to launch otherwise.
constexpr int kFatRegsLoader = 40, kFatRegsWiden = 48, kFatRegsEpilogue = 168;
constexpr int kFatRegsTotal = 128 * kFatRegsLoader + 256 * kFatRegsWiden + 256 * kFatRegsEpilogue;
static_assert(kFatRegsTotal <= kFatThreads * 96, "the CTA's register allocation at 96 registers per thread");

template <int N>
__device__ __forceinline__ void regs_take() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void regs_give() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

constexpr int kFatBlk = 0, kFatFuse = 1;

// What the fused epilogue writes: the next layer's codes (one int8 each, row pitch N bytes),
// scales and code sums [M, N / 256], and, if y_dbg is not null, the bf16 layer output it never
// needs itself (for tests).
struct FusedOut {
    uint8_t* codes;
    float* scales;
    int32_t* sums;
    __nv_bfloat16* y_dbg;
    int64_t ldy;
    int bits;
};

template <int MODE, int ABITS, bool WOP>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kFatThreads, 1)
qgemm_fat_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmAhi, const __grid_constant__ CUtensorMap tmW,
                 const __grid_constant__ CUtensorMap tmY, const float* __restrict__ scales,
                 const int32_t* __restrict__ sums, const float* __restrict__ delta, const int32_t* __restrict__ zc,
                 const __nv_bfloat16* __restrict__ bias, int M, int N, int K, int act, int spr, const FusedOut fo) {
    using S = SsSmem<ABITS, WOP>;  // WOP: the weight operand is in global memory already and comes by TMA (see qgemm_ss.cuh)
    constexpr int BN = S::BN, BNh = S::BNh;
    constexpr bool kPackedA = S::kPackedA;  // packed activation codes: the widening warps widen both operands
    constexpr int AST = S::kAStages, APS = S::kAPackedStages, WST = S::kWStages, WPB = S::kWpBars;
    // both operands by TMA into rings of the same depth: one "full" and one "empty" barrier per stage
    // serve both, and the copies of both CTAs count their bytes on the leader's (see qgemm_ss.cuh)
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
    const int KB = K / kBK;   // even: K is a multiple of 256
    const int NG = spr;       // scale groups per token
    const int KBG = KB / NG;  // k-blocks per group: 1, 2 or 8

    const uint32_t bar0 = sbase + S::kBarOff;
    auto a_full = [&](int s) { return bar0 + 8u * s; };  // a slot kept for the layout's sake: copies count on a_ready
    auto a_ready = [&](int s) { return bar0 + 8u * (AST + s); };
    auto a_empty = [&](int s) { return bar0 + 8u * (2 * AST + s); };
    const uint32_t barw = bar0 + 8u * (3 * AST);
    auto ops_full = [&](int s) { return barw + 8u * s; };
    auto ops_empty = [&](int s) { return barw + 8u * (WST + s); };
    auto acc_full = [&](int s) { return barw + 8u * (2 * WST + s); };
    auto acc_empty = [&](int s) { return barw + 8u * (2 * WST + 2 + s); };
    const uint32_t drain_bar = barw + 8u * (2 * WST + 4);
    auto wp_full = [&](int s) { return drain_bar + 8u * (1 + s); };
    auto wp_empty = [&](int s) { return drain_bar + 8u * (1 + WPB + s); };
    auto apk_full = [&](int s) { return drain_bar + 8u * (1 + 2 * WPB + s); };
    auto apk_empty = [&](int s) { return drain_bar + 8u * (1 + 2 * WPB + APS + s); };
    volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + S::kMiscOff);  // [0] tmem base, [1] abort
    volatile uint32_t* abort_flag = misc + 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < AST; ++s) {
            mbar_init(a_full(s), 1);
            mbar_init(a_ready(s), kPackedA ? 2 * (kSsWWarps / kUnpackGroups) : kOneRing ? 2 : 1);
            mbar_init(a_empty(s), 1);
        }
        for (int s = 0; s < APS; ++s) { mbar_init(apk_full(s), 1); mbar_init(apk_empty(s), kSsWWarps / kUnpackGroups); }
        for (int s = 0; s < WST; ++s) { mbar_init(ops_full(s), WOP ? 1 : 2 * (kSsWWarps / kUnpackGroups)); mbar_init(ops_empty(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full(s), 1); mbar_init(acc_empty(s), 2 * 8); }
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

    if (warp < kFatFirstWWarp) {
        regs_give<kFatRegsLoader>();
        if (warp == 0) {
            // ------------------------------------------------------------ TMA producer, activation rows
            if (lane == 0) {
                tma_prefetch_desc(&tmA);
                if (ABITS == 6) tma_prefetch_desc(&tmAhi);
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
                    // giving up (some wait ran out after seconds): copies issued before that have long landed;
                    // a short bounded pause covers the last ones, whose barrier is not this CTA's to poll
                    for (int it = 0; it < 64; ++it) __nanosleep(1000);
                } else if (!ok) {  // giving up: let copies already in flight land before the CTA exits (bounded)
                    const uint32_t n_out = issued < (uint32_t)kRing ? issued : (uint32_t)kRing;
                    for (uint32_t i = 0; i < n_out; ++i) {
                        const uint32_t s = (st + kRing - 1 - i) % kRing;
                        const uint32_t p = (s < st) ? ph : (ph ^ 1u);
                        for (int it = 0; it < (1 << 16) && !mbar_try_wait(ring_full(s), p); ++it) {}
                    }
                }
            }
            __syncwarp();
        } else if (warp == 3) {
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
                            // count their bytes on the leader's "full" barrier of the stage
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
            // An accumulator is acquired only when its first k-block is due.  Groups of two or more
            // k-blocks go two k-blocks per trip (every cycle between two issues is a bubble in the MMA
            // stream, and pairing halves the waits and votes); groups of one go a k-block at a time,
            // so that the epilogue of a group overlaps the next group's MMAs.
            if (rank == 0) {
                constexpr uint32_t idesc = umma_idesc_s8s8s32(2 * kBM, BN);
                uint32_t st = 0, ph = 0, sa = 0, pa = 0, lt = 0, acc = 0;
                bool ok = true;
                const int step = KBG >= 2 ? 2 : 1;
                for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
                    int kin = 0;
                    for (int kb = 0; ok && kb < KB; kb += step) {
                        const bool first = kin == 0;
                        if (first) {
                            acc = lt & 1u;
                            if (!mbar_wait_warp(acc_empty(acc), ((lt >> 1) & 1u) ^ 1u, abort_flag, kWaitAccEmpty)) { ok = false; break; }
                            ++lt;
                        }
                        kin += step;
                        const bool last = kin == KBG;
                        if (last) kin = 0;
                        const uint32_t sa1 = sa + 1 == AST ? 0u : sa + 1, pa1 = sa + 1 == AST ? pa ^ 1u : pa;
                        if (!mbar_wait_warp(a_ready(sa), pa, abort_flag, kWaitPackedFull)) { ok = false; break; }
                        if (!kOneRing && !mbar_wait_warp(ops_full(st), ph, abort_flag, kWaitWideFull)) { ok = false; break; }
                        if (step == 2) {
                            if (!mbar_wait_warp(a_ready(sa1), pa1, abort_flag, kWaitPackedFull)) { ok = false; break; }
                            if (!kOneRing && !mbar_wait_warp(ops_full(st + 1), ph, abort_flag, kWaitWideFull)) { ok = false; break; }
                        }
                        tc_fence_after();
                        if (elect_one()) {
                            const uint32_t d_tmem = tmem_base + acc * BN;
                            for (int h = 0; h < step; ++h) {
                                const uint32_t sah = h ? sa1 : sa;
                                const uint64_t adesc = umma_desc_sw128_kmajor(sbase + S::kAOff + sah * S::kA);
                                const uint64_t bdesc = umma_desc_sw128_kmajor(sbase + S::kWOff + (st + h) * S::kW);
#pragma unroll
                                for (int k = 0; k < kBK / 32; ++k)
                                    tc_mma_i8_ss_pair(d_tmem, adesc + 2u * k, bdesc + 2u * k, idesc, (first && h == 0 && k == 0) ? 0u : 1u);
                                if (!kOneRing) tc_commit_pair(ops_empty(st + h), 3);
                                tc_commit_pair(a_empty(sah), 3);
                            }
                            if (last) tc_commit_pair(acc_full(acc), 3);
                        }
                        __syncwarp();
                        st += step;
                        if (st == WST) { st = 0; ph ^= 1u; }
                        if (step == 2) { sa = sa1; pa = pa1; }
                        if (++sa == AST) { sa = 0; pa ^= 1u; }
                    }
                }
                if (elect_one()) tc_commit_pair(drain_bar, 1);
                __syncwarp();
                mbar_wait(drain_bar, 0u, abort_flag, kWaitDrain);
            }
            __syncwarp();
        } else {
            // idle: TMA copies into operand stages count their bytes on the leader's barrier themselves,
            // and widening warps arrive there
        }
    } else if (warp < kFatFirstEpilogueWarp) {
        regs_give<kFatRegsWiden>();
        if constexpr (WOP && !kPackedA) {
            // the weight operand comes by TMA and the activation codes are bytes: nothing to widen
        } else {
            // ------------------------------------------------------------ widen weight codes -> shared memory
            const uint32_t grp = (uint32_t)(warp - kFatFirstWWarp) >> 2;
            const int u = (threadIdx.x - kFatFirstWWarp * 32) & 127;  // thread of its group of four warps
            uint32_t j = 0;
            bool ok = true;
            const uint32_t rt_zero = runtime_zero();
            for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
                for (int kb = 0; kb < KB; ++kb) {
                    const uint32_t jj = j++;
                    if (jj % kUnpackGroups != grp) continue;
                    if constexpr (kPackedA) {
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
                        // BNh rows x 4 chunks of 32 nibbles, stored as (u - 8): the packed rows go into registers
                        // before the operand stage is known to be free, and are widened on their way out
                        constexpr int kPieces = (BNh * 4) / 128;
                        uint4 p[kPieces];
                        uint32_t loaded = 0u;
#pragma unroll
                        for (int it = 0; it < kPieces; ++it) {
                            const int qi = it * 128 + u, row = qi >> 2, ck = qi & 3;
                            p[it] = lds128(pw + row * (kBK / 2) + ck * 16);
                            loaded ^= p[it].w;
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
                            sts128(drow + (((2 * ck) ^ (row & 7)) << 4), (p[it].x << 4) & 0xF0F0F0F0u, p[it].x & 0xF0F0F0F0u,
                                   (p[it].y << 4) & 0xF0F0F0F0u, p[it].y & 0xF0F0F0F0u);
                            sts128(drow + (((2 * ck + 1) ^ (row & 7)) << 4), (p[it].z << 4) & 0xF0F0F0F0u, p[it].z & 0xF0F0F0F0u,
                                   (p[it].w << 4) & 0xF0F0F0F0u, p[it].w & 0xF0F0F0F0u);
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(map_to_cta(ops_full(wst), 0));
                    }
                }
            }
        }
    } else {
        regs_take<kFatRegsEpilogue>();
        if constexpr (MODE == kFatBlk) {
        // ------------------------------------------------------------ epilogue: running sum over groups in registers
        const int q = warp & 3;                                   // tensor-memory lane quarter this warp may read
        const int half = (warp - kFatFirstEpilogueWarp) >> 2;     // which 128 of the tile's 256 columns
        const int ew = 4 * half + q;
        constexpr int CW = BN / 2;                                 // columns per thread
        const uint32_t c_delta = sbase + S::kConstOff + ew * (3 * CW * 4);
        const uint32_t c_zc = c_delta + CW * 4;                    // (z_n - 8) as a float: exact, |.| <= 8
        const uint32_t c_bias = c_zc + CW * 4;
        const uint32_t stg0 = sbase + S::kStageOutOff + ew * (32 * 64);  // 32 rows x 32 bf16
        constexpr int kShift = ABITS == 4 ? 8 : ABITS == 6 ? 6 : 4;  // log2 of (A factor 16 / 4 / 1) x (W factor 16)
        if (lane == 0) tma_prefetch_desc(&tmY);
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        uint32_t lt = 0;
        bool ok = true;
        for (int tile = pair; ok && tile < num_tiles; tile += num_pairs) {
            const int m0 = (tile / num_n) * (2 * kBM) + (int)rank * kBM, n0 = (tile % num_n) * BN + half * CW;
            __syncwarp();
#pragma unroll
            for (int i = 0; i < CW / 32; ++i) {
                const int c = lane + 32 * i, n = n0 + c;
                const bool okn = n < N;
                sts32f(c_delta + 4 * c, okn ? __ldg(delta + n) : 0.f);
                sts32f(c_zc + 4 * c, okn ? (float)__ldg(zc + n) : 0.f);
                sts32f(c_bias + 4 * c, (okn && bias != nullptr) ? __bfloat162float(bias[n]) : 0.f);
            }
            __syncwarp();
            const int row = m0 + q * 32 + lane;
            const bool row_ok = row < M;
            const float* srow = scales + (int64_t)(row_ok ? row : 0) * NG;
            const int32_t* Srow = sums + (int64_t)(row_ok ? row : 0) * NG;
            // the zero-point term T_i = sum_g s_ig S_ig (each S_ig is exact in fp32) is added up group by
            // group, from loads issued a group ahead
            float T = 0.f;
            uint64_t run[CW / 2];  // fp32 pairs: columns 2i and 2i + 1
#pragma unroll
            for (int t = 0; t < CW / 2; ++t) run[t] = f2_pack(0.f, 0.f);
            float s_next = row_ok ? __ldg(srow) : 0.f;
            float S_next = row_ok ? (float)__ldg(Srow) : 0.f;
            for (int g = 0; g < NG; ++g, ++lt) {
                const uint32_t a = lt & 1u, aph = (lt >> 1) & 1u;
                const float s_k = s_next * (1.0f / (float)(1 << kShift));
                const uint64_t s2 = f2_pack(s_k, s_k);
                T = fmaf(s_next, S_next, T);
                if (g + 1 < NG) {  // the next group's scale and code sum: their latency hides behind this group
                    s_next = row_ok ? __ldg(srow + g + 1) : 0.f;
                    S_next = row_ok ? (float)__ldg(Srow + g + 1) : 0.f;
                }
                if (!mbar_wait(acc_full(a), aph, abort_flag, kWaitAccFull)) { ok = false; break; }
                tc_fence_after();
                // 16 columns at a time, the next load in flight while these are added up
                const uint32_t col0 = tmem_base + a * BN + half * CW + lane_addr;
                uint32_t ra[16], rb[16];
                tmem_ld_32x16(col0, ra);
#pragma unroll
                for (int c = 0; c < CW / 16; c += 2) {
                    tmem_ld_wait();
                    tmem_ld_32x16(col0 + (c + 1) * 16, rb);
#pragma unroll
                    for (int t = 0; t < 16; t += 2)
                        run[c * 8 + t / 2] = f2_fma(f2_pack((float)(int32_t)ra[t], (float)(int32_t)ra[t + 1]), s2, run[c * 8 + t / 2]);
                    tmem_ld_wait();
                    if (c + 2 < CW / 16) tmem_ld_32x16(col0 + (c + 2) * 16, ra);
#pragma unroll
                    for (int t = 0; t < 16; t += 2)
                        run[(c + 1) * 8 + t / 2] = f2_fma(f2_pack((float)(int32_t)rb[t], (float)(int32_t)rb[t + 1]), s2, run[(c + 1) * 8 + t / 2]);
                }
                // the accumulator is in registers: the MMA warp may have it back
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty(a), 0));
            }
            if (!ok) break;
            // ---- after the last group: dequantize, round, stage 32 columns per TMA store
#pragma unroll
            for (int c = 0; c < CW / 32; ++c) {
                if (lane == 0) tma_store_wait_read<0>();
                __syncwarp();
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                    const float4 d0 = lds128f(c_delta + 4 * (c * 32 + j)), d1 = lds128f(c_delta + 4 * (c * 32 + j + 4));
                    const float4 z0 = lds128f(c_zc + 4 * (c * 32 + j)), z1 = lds128f(c_zc + 4 * (c * 32 + j + 4));
                    const float4 b0 = lds128f(c_bias + 4 * (c * 32 + j)), b1 = lds128f(c_bias + 4 * (c * 32 + j + 4));
                    const float dl[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
                    const float zz[8] = {z0.x, z0.y, z0.z, z0.w, z1.x, z1.y, z1.z, z1.w};
                    const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                    uint32_t pk[4];
#pragma unroll
                    for (int t = 0; t < 8; t += 2) {
                        float r0, r1;
                        f2_unpack(run[(c * 32 + j + t) / 2], r0, r1);
                        float y0 = fmaf(fmaf(-zz[t], T, r0), dl[t], bb[t]);
                        float y1 = fmaf(fmaf(-zz[t + 1], T, r1), dl[t + 1], bb[t + 1]);
                        if (act == 1) {
                            y0 = gelu_tanh_f32(__bfloat162float(__float2bfloat16_rn(y0)));
                            y1 = gelu_tanh_f32(__bfloat162float(__float2bfloat16_rn(y1)));
                        }
                        __nv_bfloat162 b2 = __floats2bfloat162_rn(y0, y1);
                        pk[t >> 1] = *reinterpret_cast<uint32_t*>(&b2);
                    }
                    // 64-byte rows, 16-byte chunk index XORed with (row / 2) % 4: the layout a 64B-swizzled TMA store reads
                    const int ch = (j >> 3) ^ ((lane >> 1) & 3);
                    sts128(stg0 + lane * 64 + ch * 16, pk[0], pk[1], pk[2], pk[3]);
                }
                fence_proxy_async_smem();
                __syncwarp();
                const int nb = n0 + c * 32;
                if (lane == 0 && nb < N && m0 + q * 32 < M) {
                    tma_store_2d(&tmY, stg0, nb, m0 + q * 32);
                    tma_store_commit();
                }
            }
        }
        if (lane == 0) tma_store_wait_all();
        __syncwarp();
    
        } else {
        // ------------------------------------------------------------ epilogue: the next layer's rotate-quantize
        const int q = warp & 3;
        const int half = (warp - kFatFirstEpilogueWarp) >> 2;
        const int ew = 4 * half + q;
        constexpr int CW = BN / 2;
        const uint32_t c_delta = sbase + S::kConstOff + ew * (3 * CW * 4);
        const uint32_t c_zc = c_delta + CW * 4;
        const uint32_t c_bias = c_zc + CW * 4;
        // exchange slots of the thread pairs (the staging buffers of the bf16 path are not used here)
        float* x_max = reinterpret_cast<float*>(smem + S::kStageOutOff) + ew * 32;
        int* x_sum = reinterpret_cast<int*>(smem + S::kStageOutOff + 8 * 32 * 4) + ew * 32;
        const int pw = (ew ^ 4) - ew;  // the partner's slots are pw * 32 entries away
        constexpr int kShift = ABITS == 4 ? 8 : ABITS == 6 ? 6 : 4;
        constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23
        const float qmax = (float)((1 << (fo.bits - 1)) - 1);
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        const int gpr = N / BN;  // scale groups per token in the output
        uint32_t lt = 0;
        for (int tile = pair; tile < num_tiles; tile += num_pairs, ++lt) {
            const uint32_t a = lt & 1u, aph = (lt >> 1) & 1u;
            const int m0 = (tile / num_n) * (2 * kBM) + (int)rank * kBM, nt = tile % num_n, n0 = nt * BN + half * CW;
            __syncwarp();
#pragma unroll
            for (int i = 0; i < CW / 32; ++i) {
                const int c = lane + 32 * i, n = n0 + c;
                sts32f(c_delta + 4 * c, __ldg(delta + n));
                sts32f(c_zc + 4 * c, (float)__ldg(zc + n));
                sts32f(c_bias + 4 * c, bias != nullptr ? __bfloat162float(bias[n]) : 0.f);
            }
            __syncwarp();
            const int row = m0 + q * 32 + lane;
            const bool row_ok = row < M;
            const float s_i = row_ok ? scales[row] : 0.f;
            const float S_f = row_ok ? (float)sums[row] : 0.f;
            const float s_k = s_i * (1.0f / (float)(1 << kShift)), nS_k = -S_f * (float)(1 << kShift);
            if (!mbar_wait(acc_full(a), aph, abort_flag, kWaitAccFull)) break;
            tc_fence_after();
            const uint32_t own = tmem_base + a * BN + half * CW + lane_addr, theirs = tmem_base + a * BN + (half ^ 1) * CW + lane_addr;
            // ---- this layer's output, as the bf16 values the next layer is defined on; the butterfly
            // of index bit 0 on the way into the pairs (2i, 2i + 1)
            uint64_t v[CW / 2];
#pragma unroll
            for (int c = 0; c < CW / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(own + c * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const float4 dl = lds128f(c_delta + 4 * (c * 32 + j)), zz = lds128f(c_zc + 4 * (c * 32 + j)), bb = lds128f(c_bias + 4 * (c * 32 + j));
                    const float d4[4] = {dl.x, dl.y, dl.z, dl.w}, z4[4] = {zz.x, zz.y, zz.z, zz.w}, b4[4] = {bb.x, bb.y, bb.z, bb.w};
                    float y[4];
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        y[t] = fmaf(fmaf(z4[t], nS_k, (float)(int32_t)r[j + t]), d4[t] * s_k, b4[t]);
                        y[t] = __bfloat162float(__float2bfloat16_rn(y[t]));
                        if (act == 1) y[t] = __bfloat162float(__float2bfloat16_rn(gelu_tanh_f32(y[t])));
                    }
                    if (fo.y_dbg != nullptr && row_ok) {
                        __nv_bfloat162 p0 = __floats2bfloat162_rn(y[0], y[1]), p1 = __floats2bfloat162_rn(y[2], y[3]);
                        *reinterpret_cast<uint2*>(fo.y_dbg + (int64_t)row * fo.ldy + n0 + c * 32 + j) =
                            make_uint2(*reinterpret_cast<uint32_t*>(&p0), *reinterpret_cast<uint32_t*>(&p1));
                    }
                    v[(c * 32 + j) / 2] = f2_pack(y[0] + y[1], y[0] - y[1]);
                    v[(c * 32 + j) / 2 + 1] = f2_pack(y[2] + y[3], y[2] - y[3]);
                }
            }
            // ---- index bits 1..6: butterflies between register pairs
#pragma unroll
            for (int st = 1; st < CW / 2; st <<= 1)
#pragma unroll
                for (int i = 0; i < CW / 2; ++i)
                    if ((i & st) == 0) f2_butterfly(v[i], v[i + st]);
            // ---- index bit 7: the two threads of a row swap their halves through the accumulator's
            // columns (every value of it is in registers by now) and take sum or difference
#pragma unroll
            for (int c = 0; c < CW / 32; ++c) {
                uint32_t r[32];
#pragma unroll
                for (int t = 0; t < 16; ++t) {
                    float lo, hi;
                    f2_unpack(v[c * 16 + t], lo, hi);
                    r[2 * t] = __float_as_uint(lo);
                    r[2 * t + 1] = __float_as_uint(hi);
                }
                tmem_st_32x32(own + c * 32, r);
            }
            tmem_st_wait();
            tc_fence_before();
            asm volatile("bar.sync %0, 64;" ::"r"(1 + q) : "memory");  // the two warps of this lane quarter
            tc_fence_after();
            const uint64_t sgn = half ? f2_pack(-1.f, -1.f) : f2_pack(1.f, 1.f);
#pragma unroll
            for (int c = 0; c < CW / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(theirs + c * 32, r);
                tmem_ld_wait();
#pragma unroll
                for (int t = 0; t < 16; ++t)  // half 0: own + theirs; half 1: theirs - own
                    v[c * 16 + t] = f2_fma(v[c * 16 + t], sgn, f2_pack(__uint_as_float(r[2 * t]), __uint_as_float(r[2 * t + 1])));
            }
            // both halves are read: the MMA warp may have the accumulator back
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty(a), 0));
            // ---- absmax of the 256 rotated channels (of the un-normalised transform)
            float amax = 0.f;
#pragma unroll
            for (int i = 0; i < CW / 2; ++i) {
                float lo, hi;
                f2_unpack(v[i], lo, hi);
                amax = fmaxf(amax, fmaxf(fabsf(lo), fabsf(hi)));
            }
            x_max[lane] = amax;
            asm volatile("bar.sync %0, 64;" ::"r"(1 + q) : "memory");
            amax = fmaxf(amax, x_max[pw * 32 + lane]);
            const float inv = amax > 0.f ? qmax / amax : 0.f;
            const uint64_t inv2 = f2_pack(inv, inv), magic2 = f2_pack(kMagic, kMagic);
            // ---- quantize and store: per 8 channels the four even ones, then the four odd ones
            uint8_t* crow = fo.codes + (int64_t)row * N + n0;
            int lsum = 0;
#pragma unroll
            for (int k16 = 0; k16 < CW / 16; ++k16) {
                uint32_t w[4];
#pragma unroll
                for (int k8 = 0; k8 < 2; ++k8) {
                    uint32_t b[8];
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        float lo, hi;
                        f2_unpack(f2_fma(v[k16 * 8 + k8 * 4 + t], inv2, magic2), lo, hi);
                        b[2 * t] = __float_as_uint(lo);
                        b[2 * t + 1] = __float_as_uint(hi);
                    }
                    const uint32_t E = __byte_perm(__byte_perm(b[0], b[2], 0x0040), __byte_perm(b[4], b[6], 0x0040), 0x5410);
                    const uint32_t O = __byte_perm(__byte_perm(b[1], b[3], 0x0040), __byte_perm(b[5], b[7], 0x0040), 0x5410);
                    lsum = __dp4a((int)E, 0x01010101, lsum);
                    lsum = __dp4a((int)O, 0x01010101, lsum);
                    w[2 * k8] = E;
                    w[2 * k8 + 1] = O;
                }
                if (row_ok) *reinterpret_cast<uint4*>(crow + k16 * 16) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            x_sum[lane] = lsum;
            asm volatile("bar.sync %0, 64;" ::"r"(1 + q) : "memory");
            if (half == 0 && row_ok) {
                fo.scales[(int64_t)row * gpr + nt] = (amax * (1.0f / 16.0f)) / qmax;  // s = (absmax / sqrt(256)) / qmax
                fo.sums[(int64_t)row * gpr + nt] = lsum + x_sum[pw * 32 + lane];
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

// True if the registers the kernel's roles ask for fit into what the CTA is given at launch.
template <typename Kern>
static bool fat_kernel_registers_fit(Kern kern) {
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess) return false;
    return kFatRegsTotal <= kFatThreads * fa.numRegs && fa.numRegs >= kFatRegsWiden && fa.numRegs <= kFatRegsEpilogue;
}

template <int MODE, int ABITS, bool WOP>
static dvdq_status launch_qgemm_fat_w(const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                      const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy, const FusedOut& fo,
                                      cudaStream_t st) {
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
    if (MODE == kFatFuse) {
        tmY = tmA;  // unused: the fused epilogue stores codes, scales and sums itself
    } else if (!make_out_map32(&tmY, Y, (uint64_t)N, (uint64_t)M, (uint64_t)ldy)) {
        return DVDQ_ERR_CUDA;
    }
    auto kern = qgemm_fat_kernel<MODE, ABITS, WOP>;
    if (!fat_kernel_registers_fit(kern)) return DVDQ_ERR_CUDA;
    static PerDevice<int> cache;
    const int max_pairs = resident_pairs(cache, kern, kFatThreads, S::kTotal);
    if (max_pairs == 0) return DVDQ_ERR_CUDA;
    const int64_t tiles = ((M + 2 * kBM - 1) / (2 * kBM)) * ((N + S::BN - 1) / S::BN);
    const unsigned pairs = (unsigned)(tiles < max_pairs ? tiles : max_pairs);
    kern<<<2 * pairs, kFatThreads, S::kTotal, st>>>(tmA, tmAhi, tmW, tmY, scales, sums, reinterpret_cast<const float*>(blob + L.delta_offset),
                                                    reinterpret_cast<const int32_t*>(blob + L.zc_offset),
                                                    static_cast<const __nv_bfloat16*>(bias), (int)M, (int)N, (int)K, act, spr, fo);
    return cuda_status(cudaGetLastError());
}

template <int MODE, int ABITS>
static dvdq_status launch_qgemm_fat_t(const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                      const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy, const FusedOut& fo,
                                      cudaStream_t st) {
    return w.operand != nullptr ? launch_qgemm_fat_w<MODE, ABITS, true>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, fo, st)
                                : launch_qgemm_fat_w<MODE, ABITS, false>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, fo, st);
}

// Block-wise activation scales, bf16 output; sb = bits a code is stored in (4, 6 or 8).
static dvdq_status launch_qgemm_blk(int sb, const void* codes, const float* scales, const int32_t* sums, int spr, int64_t M,
                                    const dvdq_weights& w, const void* bias, int act, void* Y, int64_t ldy, cudaStream_t st) {
    if (sb == 4) return launch_qgemm_fat_t<kFatBlk, 4>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, FusedOut{}, st);
    if (sb == 6) return launch_qgemm_fat_t<kFatBlk, 6>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, FusedOut{}, st);
    return launch_qgemm_fat_t<kFatBlk, 8>(codes, scales, sums, spr, M, w, bias, act, Y, ldy, FusedOut{}, st);
}

// The layer (per-token input scales) whose epilogue writes the next layer's codes, scales and code
// sums for rot_block = scale_group = 256 instead of bf16.
static dvdq_status launch_qgemm_fused(int sb, const void* codes, const float* scales, const int32_t* sums, int64_t M,
                                      const dvdq_weights& w, const void* bias, int act, const FusedOut& fo, cudaStream_t st) {
    if (sb == 4) return launch_qgemm_fat_t<kFatFuse, 4>(codes, scales, sums, 1, M, w, bias, act, nullptr, 0, fo, st);
    if (sb == 6) return launch_qgemm_fat_t<kFatFuse, 6>(codes, scales, sums, 1, M, w, bias, act, nullptr, 0, fo, st);
    return launch_qgemm_fat_t<kFatFuse, 8>(codes, scales, sums, 1, M, w, bias, act, nullptr, 0, fo, st);
}

}  // namespace dvdq
