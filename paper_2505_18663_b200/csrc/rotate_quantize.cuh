// Online activation transform (Sec. 3.2, Eq. 10): rotate -> auto-scale -> quantize -> pack,
// one kernel, bound by HBM traffic (2K bytes read, K*b/8 + 8 bytes written per token).
//
// A warp owns a span of 1024 consecutive channels of one token (index bits 0..9 below are the
// bits of the channel index inside the span).  The Walsh-Hadamard transform over those bits is
// split so that no butterfly ever needs a warp shuffle:
//
//   load     lane L reads four 16-byte chunks, channels c*256 + 8L + e: bits 0-2 in the chunk,
//            bits 3-7 = lane, bits 8-9 = chunk number.
//   stage A  bits {0,1,3,4}: the raw bf16 words are the B operand of mma.sync.m16n8k16 and the
//            A operand is the +-1 matrix H_16, so D = H_16 * B holds the four butterflies.
//            bf16 inputs and +-1 factors make every product exact; the sums accumulate in fp32.
//            The MMA also moves data: afterwards a lane holds bits {1,2,5,8,9} in registers.
//   stage B  bit 2 through the accumulator input of further MMAs (H*B0 +- H*B1), bits {8,9} as
//            packed f32x2 adds/subs on register pairs, bit 5 as scalar add/sub.
//   turn     one conflict-free transposition through shared memory (8 x 16-byte stores and loads
//            per lane) brings bits {6,7} and {0,1,2} into registers.
//   stage C  bits {6,7} as packed f32x2 adds/subs.
//
// After stage C a lane holds, for each j = bits 7:6, eight channels that are consecutive in
// memory, i.e. exactly one 32-bit word of packed 4-bit codes (or of the low plane of 6-bit
// codes), so the packed layout stays in natural channel order.  Blocks smaller than 1024 skip
// the stages of the upper bits; no rotation (B = 0) runs the same data path with the identity
// in place of H_16.  The 1/sqrt(B) normalisation is folded into the scale.
//
// Blocks of 2048 or 4096 channels span two or four warps: after stage C the warps of a block
// exchange their spans through shared memory once and each forms its own signed sum of the two
// or four spans (the butterflies of index bits 10 and 11).
//
// Scale granularity: one scale per token (the token's warps meet once for the absmax), per
// 1024-channel span (the warp's own absmax), or per 256 / 128 channels (SUB: the absmax of the
// eight lanes that hold the group, for one or for each half of their registers).
//
// Rounding: c = rne(x~ * (qmax / absmax)) as one fused multiply-add onto 1.5 * 2^23, which
// leaves the two's-complement code in the low mantissa bits.  (B = 0 divides instead.)
#pragma once

#include "dvdq_common.cuh"

namespace dvdq {

constexpr int kRqSpan = 1024;
constexpr int kRqMaxWarps = 16;

// D = A * B + C with A 16x16 (row major), B 16x8 (column major), bf16 inputs, fp32 C and D.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1,
                                               const float (&c)[4]) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%10, %11, %12, %13};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}

// Entry (m, s) of the stage-A matrix as bf16 bits: the Sylvester sign (-1)^popcount(m & s), or the
// identity when there is no rotation.
template <bool ROTATE>
__device__ __forceinline__ uint32_t stage_a_entry(int m, int s) {
    if (ROTATE) return (__popc(m & s) & 1) ? 0xBF80u : 0x3F80u;
    return m == s ? 0x3F80u : 0u;
}

// One warp-span of work per loop iteration; CTAs are persistent and walk over groups of
// tokens_per_cta tokens.  FULL = every span is complete (K a multiple of 1024): no per-chunk
// predicates.  Per iteration the warps of a token meet once (a named barrier) for the token's
// absmax, which they combine with a shared-memory atomic max; their code sums are added up the
// same way and written out after the next iteration's barrier.  The slots rotate over three sets:
// a warp's whole iteration is a chain of dependent steps, so the exchange is kept as short as
// it can be (an atomic, the barrier, one broadcast load).
// MODE: the reach of a scale.  kRqToken: one per token, the token's warps meet (more than one span
// per token).  kRqSpan1024: one per warp span (a token of one span, or scale groups of 1024).
// kRqSub: groups of 256 or 128 channels inside the span.
constexpr int kRqToken = 0, kRqSpan1024 = 1, kRqSub = 2;

template <int LOG2B, int BITS, bool FULL, int MODE>
__global__ void __maxnreg__(80)  // two CTAs of 12 warps per SM
rq_kernel(const __nv_bfloat16* __restrict__ X, int M, int K, int ldx,
          uint8_t* __restrict__ codes, float* __restrict__ scales, int32_t* __restrict__ sums,
          int spans, int tokens_per_cta, int num_groups, int scale_group, int code_bits) {
    extern __shared__ __align__(128) float4 s_turn[];  // 256 float4 per warp
    __shared__ unsigned s_max[3][kRqMaxWarps];  // [slot set][token of the CTA]: bits of the token absmax
    __shared__ int s_sum[3][kRqMaxWarps];       // sum of the token's codes
    constexpr bool kRot = LOG2B > 0;
    constexpr int kLog2Span = LOG2B > 10 ? 10 : LOG2B;  // butterflies a warp does on its own span
    constexpr int kCross = 1 << (LOG2B > 10 ? LOG2B - 10 : 0);  // spans per rotation block
    constexpr bool SUB = MODE == kRqSub;
    constexpr bool team = MODE == kRqToken;  // the token's warps exchange absmax and code sums
    // BITS is the width a code is STORED in; the quantizer's own width may be smaller (codes kept in bytes)
    const float qmax = (float)((1 << (code_bits - 1)) - 1);
    constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23: ulp 1, so the fma rounds to an integer
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int tl = warp / spans, sp = warp - tl * spans;
    const int g = lane >> 2, t = lane & 3;
    if (team) {
        if (threadIdx.x < 3 * kRqMaxWarps) {
            (&s_max[0][0])[threadIdx.x] = 0u;
            (&s_sum[0][0])[threadIdx.x] = 0;
        }
        __syncthreads();
    }

    // ---- loop invariants
    // stage-A matrix fragment (H_16, or the identity without a rotation)
    uint32_t afrag[4];
    afrag[0] = stage_a_entry<kRot>(g, 2 * t) | (stage_a_entry<kRot>(g, 2 * t + 1) << 16);
    afrag[1] = stage_a_entry<kRot>(g + 8, 2 * t) | (stage_a_entry<kRot>(g + 8, 2 * t + 1) << 16);
    afrag[2] = stage_a_entry<kRot>(g, 2 * t + 8) | (stage_a_entry<kRot>(g, 2 * t + 9) << 16);
    afrag[3] = stage_a_entry<kRot>(g + 8, 2 * t + 8) | (stage_a_entry<kRot>(g + 8, 2 * t + 9) << 16);
    uint32_t afrag_neg[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) afrag_neg[i] = afrag[i] ^ 0x80008000u;
    // a zero accumulator the compiler cannot fold, so that it stays in four registers
    float zero4[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) asm volatile("mov.f32 %0, 0f00000000;" : "=f"(zero4[i]));
    // channel of the lane's first load chunk and of its first output word
    const int ld_e0 = sp * kRqSpan + lane * 8;                                   // + c * 256
    const int st_e0 = sp * kRqSpan + ((lane >> 3) * 32 + (lane & 7)) * 8;        // + j * 64
    uint32_t ld_ok = 0xFu, st_ok = 0xFu;
    if (!FULL) {
        ld_ok = st_ok = 0u;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (ld_e0 + c * 256 < K) ld_ok |= 1u << c;
            if (st_e0 + c * 64 < K) st_ok |= 1u << c;
        }
    }
    // turn addresses (float4 units): write = wr[r0] + 64 c, read = rd ^ (j | i0 << 2)
    float4* turn = s_turn + warp * 256;
    int wr[2];
    {
        const int b34 = lane >> 3, b0 = (lane >> 2) & 1, b67 = lane & 3;
        const int low = (b67 | (b0 << 2)) ^ b34;
        wr[0] = b34 * 8 + low;
        wr[1] = (b34 + 4) * 8 + (low ^ 4);
    }
    const int rd = lane * 8 + (lane & 7);
    // the same as 32-bit shared addresses: the buffer is 128-byte aligned, so the XOR of the read
    // index is an XOR of the address, and every access is base + immediate or base ^ immediate
    const uint32_t turn_a = smem_u32(turn);
    const uint32_t wr_a[2] = {turn_a + 16u * wr[0], turn_a + 16u * wr[1]};
    const uint32_t rd_a = turn_a + 16u * rd;
    const int row_bytes = (int)act_row_bytes(K, BITS);
    // byte offsets of the lane's first output word (+ 32 j, or + 64 j for 8-bit codes) and of its
    // first high-plane word (+ 16 j): everything else in the loop is one 32 x 32 -> 64 bit multiply-add
    const int st_b0 = BITS == 8 ? st_e0 : st_e0 >> 1;
    const int st_h0 = (K >> 1) + ((st_e0 >> 4) << 2);
    // s = (absmax / sqrt(B)) / qmax as one multiplication by a constant (at most an ulp from the quotient)
    const float rs = ((LOG2B & 1) ? rsqrtf((float)(1 << LOG2B)) : 1.0f / (float)(1 << (LOG2B / 2))) / qmax;

    auto load_span = [&](uint4 (&raw)[4], int group) {
        int token = group * tokens_per_cta + tl;
        if (token >= M) token = M - 1;  // a clamped duplicate
        const uint4* src = reinterpret_cast<const uint4*>(X + ((int64_t)token * ldx + ld_e0));
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            raw[c] = make_uint4(0u, 0u, 0u, 0u);
            if (FULL || (ld_ok >> c & 1u)) raw[c] = __ldg(src + c * 32);
        }
    };

    uint4 raw[4];
    int group = blockIdx.x;
    if (group < num_groups) load_span(raw, group);
    int prev_token = -1;
    float prev_amax = 0.f;
    int cur = 0, nxt = 1, prv = 2;  // slot sets of this iteration, the next one and the previous one
    for (; group < num_groups; group += gridDim.x) {
        // the next iteration's slots start from zero; their last readers passed the previous barrier
        if (team && sp == 0 && lane == 0) {
            s_max[nxt][tl] = 0u;
            s_sum[nxt][tl] = 0;
        }
        // A token past the end is a clamped duplicate of the last one: it computes and stores
        // the same bytes to the same places, which needs no predicate.
        int token = group * tokens_per_cta + tl;
        if (token >= M) token = M - 1;

        // ---- stage A: D = H_16 * B on index bits {0, 3, 4, 1} (k-slot bit 0 = half of a word,
        // bits 1-2 = lane & 3, bit 3 = which of the two words).  Word pair p = bit 2.
        // acc[c][p][r]: c = bits 9:8, p = bit 2, r & 1 = bit 5, r >> 1 = bit 1.
        // The lane now stands for bits 7:6 (lane & 3), bit 0 (lane >> 2 & 1), bits 4:3 (lane >> 3).
        // With a rotation the butterfly on bit 2 rides on the accumulator input:
        // acc[c][0] = H*B0 + H*B1, acc[c][1] = H*B0 - H*B1 (three MMAs instead of two MMAs and adds).
        float acc[4][2][4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (kRot) {
                float m0[4];
                mma_bf16_16816(m0, afrag, raw[c].x, raw[c].y, zero4);
                mma_bf16_16816(acc[c][0], afrag, raw[c].z, raw[c].w, m0);
                mma_bf16_16816(acc[c][1], afrag_neg, raw[c].z, raw[c].w, m0);
            } else {
                mma_bf16_16816(acc[c][0], afrag, raw[c].x, raw[c].y, zero4);
                mma_bf16_16816(acc[c][1], afrag, raw[c].z, raw[c].w, zero4);
            }
        }
        // the next group's loads fly while this one is transformed
        if (group + (int)gridDim.x < num_groups) load_span(raw, group + gridDim.x);

        // ---- stage B: bits 8, 9 on packed pairs (the pair is bit 5), then bit 5 itself
        uint64_t P[4][2][2];
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int p = 0; p < 2; ++p)
#pragma unroll
                for (int h = 0; h < 2; ++h) P[c][p][h] = f2_pack(acc[c][p][2 * h], acc[c][p][2 * h + 1]);
        if (kLog2Span > 8) {
#pragma unroll
            for (int c = 0; c < 4; c += 2)
#pragma unroll
                for (int p = 0; p < 2; ++p)
#pragma unroll
                    for (int h = 0; h < 2; ++h) f2_butterfly(P[c][p][h], P[c + 1][p][h]);
        }
        if (kLog2Span > 9) {
#pragma unroll
            for (int c = 0; c < 2; ++c)
#pragma unroll
                for (int p = 0; p < 2; ++p)
#pragma unroll
                    for (int h = 0; h < 2; ++h) f2_butterfly(P[c][p][h], P[c + 2][p][h]);
        }

        // ---- turn: float4 = bits (1, 2) varying; address = [bits 9 8 5 4 3 | (bits 0 7 6) ^ (bits 5 4 3)]
        __syncwarp();  // the previous iteration's reads of this warp's turn buffer are done
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float v[2][2][2];  // [p][h][r0]
#pragma unroll
            for (int p = 0; p < 2; ++p)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    float lo, hi;
                    f2_unpack(P[c][p][h], lo, hi);
                    v[p][h][0] = kRot ? lo + hi : lo;
                    v[p][h][1] = kRot ? lo - hi : hi;
                }
#pragma unroll
            for (int r0 = 0; r0 < 2; ++r0)
                sts128(wr_a[r0] + 1024u * c, __float_as_uint(v[0][0][r0]), __float_as_uint(v[0][1][r0]), __float_as_uint(v[1][0][r0]),
                       __float_as_uint(v[1][1][r0]));
        }
        __syncwarp();
        // The lane now stands for bits 5:3 (lane & 7) and bits 9:8 (lane >> 3);
        // W[j][i0][h]: j = bits 7:6, i0 = bit 0, h = bit 2, the pair is bit 1.
        uint64_t W[4][2][2];
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int i0 = 0; i0 < 2; ++i0) {
                const float4 f = lds128f(rd_a ^ (16u * (j | (i0 << 2))));
                W[j][i0][0] = f2_pack(f.x, f.y);
                W[j][i0][1] = f2_pack(f.z, f.w);
            }

        // ---- stage C: bits 6 and 7
        if (kLog2Span > 6) {
#pragma unroll
            for (int j = 0; j < 4; j += 2)
#pragma unroll
                for (int i0 = 0; i0 < 2; ++i0)
#pragma unroll
                    for (int h = 0; h < 2; ++h) f2_butterfly(W[j][i0][h], W[j + 1][i0][h]);
        }
        if (kLog2Span > 7) {
#pragma unroll
            for (int j = 0; j < 2; ++j)
#pragma unroll
                for (int i0 = 0; i0 < 2; ++i0)
#pragma unroll
                    for (int h = 0; h < 2; ++h) f2_butterfly(W[j][i0][h], W[j + 2][i0][h]);
        }

        // ---- index bits 10 (and 11): the kCross warps of a rotation block park their spans in
        // their turn buffers, meet, and each takes its signed sum over the block's spans
        if (kCross > 1) {
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int i0 = 0; i0 < 2; ++i0) {
                    float a, b, c, d;
                    f2_unpack(W[j][i0][0], a, b);
                    f2_unpack(W[j][i0][1], c, d);
                    turn[(2 * j + i0) * 32 + lane] = make_float4(a, b, c, d);
                    W[j][i0][0] = W[j][i0][1] = f2_pack(0.f, 0.f);
                }
            asm volatile("bar.sync %0, %1;" ::"r"(1 + tl), "r"(spans * 32) : "memory");
            const int me = sp & (kCross - 1);
#pragma unroll
            for (int o = 0; o < kCross; ++o) {
                const float sg = (__popc(me & o) & 1) ? -1.f : 1.f;  // entry (me, o) of H_2 or H_4
                const uint64_t sg2 = f2_pack(sg, sg);
                const float4* theirs = s_turn + (warp - me + o) * 256;
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int i0 = 0; i0 < 2; ++i0) {
                        const float4 f = theirs[(2 * j + i0) * 32 + lane];
                        W[j][i0][0] = f2_fma(f2_pack(f.x, f.y), sg2, W[j][i0][0]);
                        W[j][i0][1] = f2_fma(f2_pack(f.z, f.w), sg2, W[j][i0][1]);
                    }
            }
            // without the absmax rendezvous below nothing else keeps a fast warp from refilling its
            // turn buffer while a partner still reads it
            if (!team) asm volatile("bar.sync %0, %1;" ::"r"(1 + tl), "r"(spans * 32) : "memory");
        }

        // W[j][i0][h] = channels e and e + 2 of word j, e = i0 + 4 * h; the word covers channels
        // (lane >> 3) * 256 + j * 64 + (lane & 7) * 8 + 0..7 of the span
        // ---- absmax (of the un-normalised transform) of the scale's reach: am[jh] covers this
        // lane's words j = 2 jh, 2 jh + 1
        float am[2] = {0.f, 0.f};
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int i0 = 0; i0 < 2; ++i0)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    float lo, hi;
                    f2_unpack(W[j][i0][h], lo, hi);
                    am[j >> 1] = fmaxf(am[j >> 1], fmaxf(fabsf(lo), fabsf(hi)));
                }
        const unsigned octet = 0xFFu << (lane & 24);  // the eight lanes that hold one 256-channel group
        if (SUB) {
            // non-negative floats order like their bit patterns: one REDUX instead of shuffles
            if (scale_group == 256) am[0] = am[1] = fmaxf(am[0], am[1]);
            am[0] = __uint_as_float(__reduce_max_sync(octet, __float_as_uint(am[0])));
            am[1] = scale_group == 256 ? am[0] : __uint_as_float(__reduce_max_sync(octet, __float_as_uint(am[1])));
        } else {
            float amax = __uint_as_float(__reduce_max_sync(0xFFFFFFFFu, __float_as_uint(fmaxf(am[0], am[1]))));
            // One scale per 1024-channel span: the warp's own absmax is the scale's, nothing is shared
            // between warps.  Per-token scale: the token's warps meet.
            if (team) {
                if (lane == 0) atomicMax(&s_max[cur][tl], __float_as_uint(amax));
                // only the warps of this token meet: named barrier 1 + tl, spans * 32 threads
                asm volatile("bar.sync %0, %1;" ::"r"(1 + tl), "r"(spans * 32) : "memory");
                amax = __uint_as_float(s_max[cur][tl]);
            }
            am[0] = am[1] = amax;
        }
        const float amax = am[0];
        const float inv0 = am[0] > 0.f ? qmax / am[0] : 0.f, inv1 = am[1] > 0.f ? qmax / am[1] : 0.f;
        const uint64_t invs[2] = {f2_pack(inv0, inv0), f2_pack(inv1, inv1)};
        const uint64_t magic2 = f2_pack(kMagic, kMagic);

        // ---- quantize, sum, pack, store
        uint8_t* crow = codes + (int64_t)token * row_bytes;
        int lsum = 0, lsum_lo = 0;  // SUB: lsum_lo keeps the words j = 0, 1
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t b[8];
#pragma unroll
            for (int i0 = 0; i0 < 2; ++i0)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    float lo, hi;
                    if (kRot) {
                        f2_unpack(f2_fma(W[j][i0][h], invs[SUB ? (j >> 1) : 0], magic2), lo, hi);
                    } else {
                        // Without a rotation x~ is a bf16 value, x~ * qmax is exact and exact half-way
                        // quotients are common: take the correctly rounded quotient so that they survive.
                        f2_unpack(W[j][i0][h], lo, hi);
                        const float aj = am[SUB ? (j >> 1) : 0];
                        lo = (aj > 0.f ? __fdiv_rn(lo * qmax, aj) : 0.f) + kMagic;
                        hi = (aj > 0.f ? __fdiv_rn(hi * qmax, aj) : 0.f) + kMagic;
                    }
                    b[i0 + 4 * h] = __float_as_uint(lo);
                    b[i0 + 4 * h + 2] = __float_as_uint(hi);
                }
            // low bytes (= the codes as int8) of the even and of the odd channels
            const uint32_t E = __byte_perm(__byte_perm(b[0], b[2], 0x0040), __byte_perm(b[4], b[6], 0x0040), 0x5410);
            const uint32_t O = __byte_perm(__byte_perm(b[1], b[3], 0x0040), __byte_perm(b[5], b[7], 0x0040), 0x5410);
            lsum = __dp4a((int)E, 0x01010101, lsum);
            lsum = __dp4a((int)O, 0x01010101, lsum);
            if (SUB && j == 1) {
                lsum_lo = lsum;
                lsum = 0;
            }
            const bool ok = FULL || (st_ok >> j & 1u);
            if (BITS == 8) {
                // 8-bit codes: each group of 8 channels is stored as the word of its even channels
                // followed by the word of its odd channels, the order the GEMM consumes
                if (ok) *reinterpret_cast<uint2*>(crow + st_b0 + 64 * j) = make_uint2(E, O);
                continue;
            }
            const uint32_t lo = (E & 0x0F0F0F0Fu) | ((O << 4) & 0xF0F0F0F0u);
            if (ok) *reinterpret_cast<uint32_t*>(crow + st_b0 + 32 * j) = lo;
            if (BITS == 6) {
                // bits 5:4 of 16 consecutive channels share one word of the high plane; the two
                // halves sit in neighbouring lanes
                uint32_t hi = ((E >> 4) & 0x03030303u) | ((O >> 2) & 0x0C0C0C0Cu);
                hi <<= 4 * (lane & 1);
                hi |= __shfl_xor_sync(0xFFFFFFFFu, hi, 1);
                if (ok && ((j ^ lane) & 1) == 0) *reinterpret_cast<uint32_t*>(crow + st_h0 + 16 * j) = hi;
            }
        }
        if (SUB) {
            // groups of 256 channels = this octet's 32 words; groups of 128 = its words j = 0, 1 and j = 2, 3
            const int per_span = kRqSpan / scale_group;  // 4 or 8
            const int gps = K / scale_group;
            int s0 = scale_group == 256 ? lsum_lo + lsum : lsum_lo, s1 = lsum;
            s0 = __reduce_add_sync(octet, s0);
            if (scale_group != 256) s1 = __reduce_add_sync(octet, s1);
            if ((lane & 7) == 0) {
                const int g0 = sp * per_span + (lane >> 3) * (per_span >> 2);
                if (FULL || g0 < gps) {
                    scales[(int64_t)token * gps + g0] = am[0] * rs;
                    sums[(int64_t)token * gps + g0] = s0;
                }
                if (scale_group != 256 && (FULL || g0 + 1 < gps)) {
                    scales[(int64_t)token * gps + g0 + 1] = am[1] * rs;
                    sums[(int64_t)token * gps + g0 + 1] = s1;
                }
            }
            continue;
        }
        lsum = __reduce_add_sync(0xFFFFFFFFu, lsum);
        if (!team) {  // the span's own scale: a token of one span, or one scale per 1024 channels
            if (lane == 0) {
                scales[(int64_t)token * spans + sp] = amax * rs;
                sums[(int64_t)token * spans + sp] = lsum;
            }
            continue;
        }
        if (lane == 0) {
            atomicAdd(&s_sum[cur][tl], lsum);
            // the previous iteration's token: its warps added their code sums before this iteration's barrier
            if (sp == 0 && prev_token >= 0) {
                scales[prev_token] = prev_amax * rs;  // s_i = (absmax / sqrt(B)) / qmax
                sums[prev_token] = s_sum[prv][tl];
            }
        }
        prev_token = token;
        prev_amax = amax;
        const int r = prv;
        prv = cur;
        cur = nxt;
        nxt = r;
    }
    if (!team) return;
    asm volatile("bar.sync %0, %1;" ::"r"(1 + tl), "r"(spans * 32) : "memory");
    if (sp == 0 && lane == 0 && prev_token >= 0) {
        scales[prev_token] = prev_amax * rs;
        sums[prev_token] = s_sum[prv][tl];  // the last iteration's slots
    }
}

template <int LOG2B, int BITS, bool FULL, int MODE>
static dvdq_status launch_rq_kernel(const void* X, int64_t M, int64_t K, int64_t ldx, void* codes, float* scales,
                                    int32_t* sums, int scale_group, int code_bits, cudaStream_t st) {
    const int spans = (int)((K + kRqSpan - 1) / kRqSpan);
    if (spans > kRqMaxWarps) return DVDQ_ERR_SHAPE;
    int tpc = 12 / spans;  // at most 12 tokens per CTA: named barriers 1..12
    if (tpc < 1) tpc = 1;
    constexpr int kCross = LOG2B > 10 ? (1 << (LOG2B > 10 ? LOG2B - 10 : 0)) : 1;  // spans per rotation block
    if (spans % kCross != 0) return DVDQ_ERR_ROT_BLOCK;
    const int warps = spans * tpc;
    const int threads = warps * 32;
    const size_t smem = (size_t)warps * 256 * sizeof(float4);
    const int64_t groups = (M + tpc - 1) / tpc;
    if (M > 0x7FFFFF00ll || ldx > 0x7FFFFFFFll || groups * tpc > 0x7FFFFFFFll) return DVDQ_ERR_SHAPE;
    auto kern = rq_kernel<LOG2B, BITS, FULL, MODE>;
    struct Setup {
        int sm_count;
        int blocks_per_sm[kRqMaxWarps + 1];
    };
    static PerDevice<Setup> cache;
    Setup* su = cache.get([&](Setup& s, int dev) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 kRqMaxWarps * 256 * (int)sizeof(float4)) != cudaSuccess)
            return false;
        return cudaDeviceGetAttribute(&s.sm_count, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess;
    });
    if (!su) return DVDQ_ERR_CUDA;
    if (su->blocks_per_sm[warps] == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kern, threads, smem) != cudaSuccess || n < 1) return DVDQ_ERR_CUDA;
        su->blocks_per_sm[warps] = n;
    }
    const int64_t resident = (int64_t)su->sm_count * su->blocks_per_sm[warps];
    const unsigned grid = (unsigned)(groups < resident ? groups : resident);
    kern<<<grid, threads, smem, st>>>((const __nv_bfloat16*)X, (int)M, (int)K, (int)ldx, (uint8_t*)codes, scales, sums, spans, tpc,
                                      (int)groups, scale_group, code_bits);
    return cuda_status(cudaGetLastError());
}

template <int BITS, int MODE>
static dvdq_status launch_rq_bits(const void* X, int64_t M, int64_t K, int64_t ldx, int rot_block, void* codes,
                                  float* scales, int32_t* sums, int scale_group, int code_bits, cudaStream_t st) {
    int log2b = 0;
    while ((1 << log2b) < rot_block) ++log2b;
    const bool full = K % kRqSpan == 0;
#define DVDQ_RQ_CASE(L)                                                                              \
    case L:                                                                                          \
        return full ? launch_rq_kernel<L, BITS, true, MODE>(X, M, K, ldx, codes, scales, sums, scale_group, code_bits, st)  \
                    : launch_rq_kernel<L, BITS, false, MODE>(X, M, K, ldx, codes, scales, sums, scale_group, code_bits, st);
    switch (log2b) {
        DVDQ_RQ_CASE(0)
        DVDQ_RQ_CASE(6)
        DVDQ_RQ_CASE(7)
        DVDQ_RQ_CASE(8)
        DVDQ_RQ_CASE(9)
        DVDQ_RQ_CASE(10)
        case 11:  // blocks of 2048 and 4096 channels are whole spans: K is a multiple of 1024
            return full ? launch_rq_kernel<11, BITS, true, MODE>(X, M, K, ldx, codes, scales, sums, scale_group, code_bits, st) : DVDQ_ERR_ROT_BLOCK;
        case 12:
            return full ? launch_rq_kernel<12, BITS, true, MODE>(X, M, K, ldx, codes, scales, sums, scale_group, code_bits, st) : DVDQ_ERR_ROT_BLOCK;
        default:
            return DVDQ_ERR_ROT_BLOCK;
    }
#undef DVDQ_RQ_CASE
}

inline dvdq_status launch_rotate_quantize(const void* X, int64_t M, int64_t K, int64_t ldx, const dvdq_act_quant& q,
                                          void* codes, float* scales, int32_t* sums, cudaStream_t st) {
    if (M == 0) return DVDQ_OK;
    const int sb = storage_bits(q);
    const int mode = (q.scale_group != 0 && q.scale_group < kRqSpan) ? kRqSub : (q.scale_group == 0 && K > kRqSpan) ? kRqToken : kRqSpan1024;
#define DVDQ_RQ_BITS(B)                                                                                                       \
    if (sb == B) {                                                                                                            \
        if (mode == kRqSub) return launch_rq_bits<B, kRqSub>(X, M, K, ldx, q.rot_block, codes, scales, sums, q.scale_group, q.bits, st);        \
        if (mode == kRqToken) return launch_rq_bits<B, kRqToken>(X, M, K, ldx, q.rot_block, codes, scales, sums, q.scale_group, q.bits, st);    \
        return launch_rq_bits<B, kRqSpan1024>(X, M, K, ldx, q.rot_block, codes, scales, sums, q.scale_group, q.bits, st);                       \
    }
    DVDQ_RQ_BITS(4)
    DVDQ_RQ_BITS(6)
    DVDQ_RQ_BITS(8)
#undef DVDQ_RQ_BITS
    return DVDQ_ERR_BITS;
}

}  // namespace dvdq
