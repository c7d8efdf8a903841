// Shared declarations of the CUDA sources: packed-format constants, the device status
// word, and thin wrappers around the sm_100a PTX the kernels use (mbarrier, TMA,
// tcgen05).  Nothing here is shared with the CPU oracle.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/dvdq.h"

namespace dvdq {

// ------------------------------------------------------------------ formats

constexpr uint32_t kBlobMagic = 0x51445644u;  // "DVDQ" little endian
constexpr uint32_t kBlobVersion = 1u;
constexpr int64_t kBlobHeaderBytes = 256;     // header padded so that the codes stay 256-byte aligned
constexpr int32_t kLibVersion = 1;

// Storage order of the K axis, shared by activation codes and weight codes.  The integer
// GEMM is a dot product over k, so any permutation applied to both operands gives the same
// accumulators.
constexpr int32_t kKLayoutNatural = 0;        // position p holds logical channel p

__host__ __device__ inline int64_t align_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

// Device copy of the blob header (the host handle dvdq_weights mirrors it).
struct BlobHeader {
    uint32_t magic, version;
    int64_t N, K;
    int32_t rot_block, k_layout;
    int64_t codes_offset, delta_offset, zc_offset;
};

struct BlobLayout {
    int64_t codes_offset, delta_offset, zc_offset, total;
};

__host__ __device__ inline BlobLayout blob_layout(int64_t N, int64_t K) {
    BlobLayout L;
    L.codes_offset = kBlobHeaderBytes;
    L.delta_offset = L.codes_offset + align_up(N * (K / 2), 256);
    L.zc_offset = L.delta_offset + align_up(N * 4, 256);
    L.total = L.zc_offset + align_up(N * 4, 256);
    return L;
}

// Activation code rows: A4 = K/2 bytes (two's-complement nibbles, position 2t in the low
// nibble of byte t).  A6 = a low plane in exactly the A4 format holding the low 4 bits of
// each code, followed by a high plane of K/4 bytes with bits 5:4.  In the high plane one
// 32-bit word covers 16 consecutive positions p = 16m + 8a + i (a in {0,1}, i in 0..7):
// the 2-bit field sits at bit 2*(4*(i>>1) + 2*a + (i&1)).  That order makes the GEMM's
// widening of 16 codes into four int8 words a shift and a mask per word.  A8 = K bytes: int8 codes,
// each group of 8 channels as its four even channels followed by its four odd ones.
__host__ __device__ inline int64_t act_row_bytes(int64_t K, int bits) { return K * bits / 8; }
// bits per stored code: the container's, or the code width when the codes are packed
inline int storage_bits(const dvdq_act_quant& q) { return q.container_bits ? q.container_bits : q.bits; }
__host__ __device__ inline int hi_field_shift(int a, int i) { return 2 * (4 * (i >> 1) + 2 * a + (i & 1)); }

// ------------------------------------------------------------------ device status word

// [0] = status (0 ok, else dvdq_status), [1] = detail of the first failure.  The library is a
// single translation unit, so this is the one copy.
__device__ uint32_t g_device_status[2] = {0u, 0u};

enum WaitId : uint32_t {
    kWaitPackedEmpty = 1, kWaitPackedFull = 2, kWaitWideEmpty = 3, kWaitWideFull = 4,
    kWaitAccEmpty = 5, kWaitAccFull = 6, kWaitDrain = 7, kWaitDebug = 8
};

__device__ __forceinline__ void report_timeout(uint32_t detail) {
    if (atomicCAS(&g_device_status[0], 0u, (uint32_t)DVDQ_ERR_DEVICE_TIMEOUT) == 0u) g_device_status[1] = detail;
}

// ------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Explicit shared-space 16-byte accesses by 32-bit shared address (a generic-pointer access to
// shared memory compiles to the slower generic load/store path).
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ float4 lds128f(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts32f(uint32_t addr, float v) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}

__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// Every wait in the kernels is bounded: it gives up when another role has already given up
// (abort flag in shared memory) or after kWaitLimitNs, records which wait it was, raises the
// abort flag and returns false.  The caller then leaves its loop and walks to the common exit.
constexpr uint64_t kWaitLimitNs = 4000000000ull;  // 4 s

__device__ __forceinline__ bool mbar_wait_limit(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t wait_id,
                                                uint64_t limit_ns) {
    // Reading %globaltimer costs hundreds of cycles, so the clock is consulted only every 1024
    // failed polls (each poll already suspends the thread for a while in hardware).
    uint64_t t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 0x3FFu) == 0u) {
            if (*abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            if (now - t0 > limit_ns) {
                *abort_flag = 1u;
                report_timeout(wait_id);
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t wait_id) {
    return mbar_wait_limit(bar, parity, abort_flag, wait_id, kWaitLimitNs);
}

// mbar_wait by a fully converged warp with one answer for all lanes (a wait that gives up in some
// lanes only must not split the warp before an elect.sync / __syncwarp).
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t wait_id) {
    const bool ok = mbar_wait(bar, parity, abort_flag, wait_id);
    return __all_sync(0xFFFFFFFFu, ok);
}

// Before a buffer that this thread has READ is handed back to whoever overwrites it (a TMA copy
// armed by the arrive that follows), the loads must have DELIVERED.  An mbarrier arrive is not an
// access of the load pipeline, and the instructions that consume the loaded registers may be
// scheduled after it: the refill then lands before a straggling load has read the stage (seen as a
// warp's worth of stale operand rows in one k-block, at full size only, and far more often when
// the epilogue keeps the schedulers busy).  A CTA-scope fence before the arrive made that rare but
// not impossible.  What closes it is a data dependency: the arrive's address is formed from a word of
// every load (ANDed with a zero the compiler cannot see through, so the address does not change),
// and an instruction cannot issue before its operands have been delivered.
__device__ __forceinline__ uint32_t runtime_zero() {
    uint32_t v;
    asm volatile("mov.u32 %0, %%nctaid.y;" : "=r"(v));  // the grids here are one-dimensional: nctaid.y == 1
    return v - 1u;
}
__device__ __forceinline__ void mbar_arrive_after_loads(uint32_t bar, uint32_t loaded_words_masked) {
    mbar_arrive(bar + loaded_words_masked);
}

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(m)) : "memory");
}
// 2-D tiled TMA load global -> shared, completion counted in bytes on an mbarrier.
// x is the innermost coordinate; x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* m, uint32_t bar, int32_t x, int32_t y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(bar), "r"(x), "r"(y)
        : "memory");
}

// The same for a CTA pair: the copy lands in THIS CTA's shared memory and counts its bytes on an
// mbarrier that may be the peer's (a shared::cluster address from map_to_cta), so that one barrier in
// the leader CTA collects the tiles of both CTAs of a stage.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* m, uint32_t cluster_bar, int32_t x, int32_t y) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(cluster_bar), "r"(x), "r"(y)
        : "memory");
}

// Asks L2 for the tile a later tma_load_2d with the same coordinates will copy.
__device__ __forceinline__ void tma_prefetch_l2_2d(const CUtensorMap* m, int32_t x, int32_t y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global [%0, {%1, %2}];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(x), "r"(y)
                 : "memory");
}

// 2-D tiled TMA store shared -> global (bulk async-group completion); elements outside the
// tensor are clipped.  The coordinates must not be negative.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* m, uint32_t src, int32_t x, int32_t y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(m)), "r"(src), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until at most N of this thread's store groups still have to READ their shared memory.
template <int N>
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// True in exactly one lane of a fully converged warp.  Unlike `lane == 0`, the compiler knows the
// enclosing control flow is warp-uniform, so descriptors and addresses stay in uniform registers.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xFFFFFFFF;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

// ---- packed fp32 pairs (sm_100 add/sub/mul/fma.f32x2 on 64-bit registers)
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t f2_sub(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
// (a, b) -> (a + b, a - b) on packed pairs
__device__ __forceinline__ void f2_butterfly(uint64_t& a, uint64_t& b) {
    const uint64_t s = f2_add(a, b), d = f2_sub(a, b);
    a = s;
    b = d;
}

__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// ---- thread-block clusters (CTA pairs)
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
// Arrive on an mbarrier that may live in another CTA of the cluster (address from map_to_cta).
// Default semantics (release at CTA scope), as for a local arrive: the data handed over with
// these arrivals is consumed by the tensor core (async proxy, after fence.proxy.async) or lives in
// tensor memory (after tcgen05.wait::st), never read through the generic proxy of the other CTA.
// A cluster-scope release here costs a device-wide memory barrier per arrival.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

// ---- tensor memory and tcgen05
__device__ __forceinline__ void tmem_alloc(uint32_t smem_slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[tmem] * B[smem]^T, int8 operands, int32 accumulators, for a CTA pair (issued by
// ONE thread of the leader CTA): D is 256 x N, rows 0-127 in the
// leader's tensor memory and rows 128-255 in the peer's; A comes from tensor memory (each CTA holds
// its own 128 rows at the same address), B from shared memory (each CTA holds half of the N rows at
// the same offset).
__device__ __forceinline__ void tc_mma_i8_ts_pair(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::i8 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives once on the mbarrier at this shared-memory offset in EVERY CTA of cta_mask when all
// tcgen05.mma issued so far by this thread have finished (a signal, not a data copy).
__device__ __forceinline__ void tc_commit_pair(uint32_t bar, uint16_t cta_mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(cta_mask) : "memory");
}
// Thread t of the warp writes 32 registers to 32 consecutive 32-bit columns of lane (base_lane + t).
__device__ __forceinline__ void tmem_st_32x32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp receives lane (base_lane + t).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
// The same for 16 columns (half the registers, for code that holds two operands at once).
__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major int8 tile whose rows are 128 bytes wide and
// stored with the 128-byte swizzle: 8-row groups are 1024 bytes apart (stride byte offset),
// the leading byte offset is unused for this layout (set to 16 bytes), descriptor version 1.
__device__ __forceinline__ uint64_t umma_desc_sw128_kmajor(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
    d |= (uint64_t)1u << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= (uint64_t)1u << 46;
    d |= (uint64_t)2u << 61;
    return d;
}
// Instruction descriptor for kind::i8: signed int8 A and B, both K-major, int32 accumulator.
__host__ __device__ constexpr uint32_t umma_idesc_s8s8s32(int m, int n) {
    return (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ------------------------------------------------------------------ host helpers (dvdq_lib.cu)

// Launch-time set-up that CUDA keeps per device (the opt-in to large dynamic shared memory, the
// SM count, occupancy) is cached per device ordinal: one slot per device, filled with that
// device current, under a lock so that host threads may share the library.
constexpr int kMaxDevices = 64;

template <typename T>
struct PerDevice {
    T slot[kMaxDevices] = {};
    bool ready[kMaxDevices] = {};
    std::mutex lock;
    // Returns the current device's slot, calling init(slot, device) the first time; nullptr if
    // the device cannot be queried or init reports failure.
    template <typename Init>
    T* get(Init init) {
        int dev = -1;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
        std::lock_guard<std::mutex> g(lock);
        if (!ready[dev]) {
            if (!init(slot[dev], dev)) return nullptr;
            ready[dev] = true;
        }
        return &slot[dev];
    }
};

dvdq_status check_device_arch();
dvdq_status validate_act_quant(const dvdq_act_quant* q, int64_t K);
dvdq_status validate_weights(const dvdq_weights* w);
dvdq_status cuda_status(cudaError_t e);

}  // namespace dvdq
