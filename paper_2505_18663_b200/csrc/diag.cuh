// Two small kernels that are not on the path: the ceiling of the int8 tensor pipe (an issue loop
// of tcgen05.mma.kind::i8 on operands that stay in shared memory, for the benchmark's roofline)
// and a wait that is made to run out (so that the bounded-wait error path can be exercised
// without harming the device).
#pragma once

#include "qgemm_ss.cuh"

namespace dvdq {

// ------------------------------------------------------------------ int8 tensor-pipe ceiling
// Every CTA pair issues `iters` k-blocks of four 256 x 256 x 32 MMAs (the instruction shape of
// qgemm_ss_kernel) on one resident activation tile and one resident weight half-tile per CTA: no
// loads, no widening, no epilogue.  The operands are filled with a byte pattern (not zeros, so
// that the data paths toggle as they do on real codes).  Work per launch:
// pairs * iters * 4 * 2 * 256 * 256 * 32 integer operations.
constexpr int kCeilThreads = 64;
constexpr int kCeilSmem = 2 * kBM * kBK + 64 + 1024;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kCeilThreads, 1)
int8_ceiling_kernel(int iters) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t a_off = 0, b_off = kBM * kBK, bar = sbase + 2 * kBM * kBK, misc_off = 2 * kBM * kBK + 16;
    volatile uint32_t* misc = reinterpret_cast<volatile uint32_t*>(smem + misc_off);  // [0] tmem base, [1] abort
    const int warp = threadIdx.x >> 5;
    const uint32_t rank = cluster_ctarank();
    for (int i = threadIdx.x; i < 2 * kBM * kBK / 4; i += kCeilThreads)
        reinterpret_cast<uint32_t*>(smem)[i] = 0x9E3779B9u * (uint32_t)(i + 1) + blockIdx.x;
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        misc[1] = 0u;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(sbase + misc_off, kTmemCols);
        tmem_relinquish();
    }
    fence_proxy_async_smem();
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = misc[0];
    if (warp == 0 && rank == 0) {
        constexpr uint32_t idesc = umma_idesc_s8s8s32(2 * kBM, kSsBN);
        const uint64_t adesc = umma_desc_sw128_kmajor(sbase + a_off), bdesc = umma_desc_sw128_kmajor(sbase + b_off);
        if (elect_one()) {
            for (int it = 0; it < iters; ++it) {
                const uint32_t d = tmem_base + (uint32_t)(it & 1) * kSsBN;
#pragma unroll
                for (int k = 0; k < kBK / 32; ++k) tc_mma_i8_ss_pair(d, adesc + 2u * k, bdesc + 2u * k, idesc, (it > 1 || k > 0) ? 1u : 0u);
            }
            tc_commit_pair(bar, 1);
        }
        __syncwarp();
        mbar_wait(bar, 0u, misc + 1, kWaitDrain);
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// ------------------------------------------------------------------ a wait that runs out
// One warp waits on an mbarrier that nobody ever arrives on, with the given limit: the wait gives
// up, records DVDQ_ERR_DEVICE_TIMEOUT with its wait id in the status word and the kernel returns
// normally.  The context stays usable.
__global__ void wait_timeout_kernel(uint64_t limit_ns) {
    __shared__ uint64_t s_bar;
    __shared__ uint32_t s_abort;
    const uint32_t bar = smem_u32(&s_bar);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        s_abort = 0u;
        fence_mbar_init();
    }
    __syncthreads();
    mbar_wait_limit(bar, 0u, &s_abort, kWaitDebug, limit_ns);
}

}  // namespace dvdq
