// Gradient statistics, quantizer and clipping-factor update (arXiv 2407.12637, Sec. 3.1 and 3.3).
// All three are HBM-bound streaming kernels or single-thread bookkeeping; no tensor cores here.
#include <algorithm>
#include <mutex>

#include "lbt_common.cuh"

namespace lbt {

constexpr int kStreamThreads = 256;
constexpr int kBlocksPerSM = 8;  // 8 x 256 threads = the SM's 2048-thread capacity
constexpr uint64_t kGridBarrierLimitNs = 2000000000ull;   // the one-launch quantizer's grid barrier gives up after 2 s

// ------------------------------------------------------------------------------------------
// abs-max over the finite elements + non-finite count (g_max of Sec. 3.1).
// |x| as an unsigned integer orders exactly like |x| as a float, so the reduction is an
// integer max and the result is independent of the order of evaluation.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void absmax_accumulate(float v, uint32_t& m, uint32_t& bad) {
    const uint32_t a = __float_as_uint(v) & 0x7FFFFFFFu;
    if (a >= 0x7F800000u) ++bad; else m = max(m, a);
}

__device__ __forceinline__ void absmax_accumulate4(const float4& v, uint32_t& m, uint32_t& bad) {
    absmax_accumulate(v.x, m, bad); absmax_accumulate(v.y, m, bad);
    absmax_accumulate(v.z, m, bad); absmax_accumulate(v.w, m, bad);
}

__global__ void __launch_bounds__(kStreamThreads, kBlocksPerSM)
absmax_kernel(const float* __restrict__ dY, uint64_t n, lbt_grad_stats_t* __restrict__ out) {
    const uint64_t nvec = n >> 2;
    const float4* __restrict__ v4 = reinterpret_cast<const float4*>(dY);
    uint32_t m = 0, bad = 0;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    // four independent 128-bit loads in flight per thread
    for (; i + 3 * stride < nvec; i += 4 * stride) {
        const float4 a = __ldg(v4 + i), b = __ldg(v4 + i + stride);
        const float4 c = __ldg(v4 + i + 2 * stride), d = __ldg(v4 + i + 3 * stride);
        absmax_accumulate4(a, m, bad); absmax_accumulate4(b, m, bad);
        absmax_accumulate4(c, m, bad); absmax_accumulate4(d, m, bad);
    }
    for (; i < nvec; i += stride) absmax_accumulate4(__ldg(v4 + i), m, bad);
    if (blockIdx.x == 0 && threadIdx.x < (n & 3)) absmax_accumulate(dY[(nvec << 2) + threadIdx.x], m, bad);

    m = __reduce_max_sync(0xFFFFFFFFu, m);
    bad = __reduce_add_sync(0xFFFFFFFFu, bad);
    __shared__ uint32_t s_m[kStreamThreads / 32], s_bad[kStreamThreads / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { s_m[warp] = m; s_bad[warp] = bad; }
    __syncthreads();
    if (warp == 0) {
        m = lane < kStreamThreads / 32 ? s_m[lane] : 0u;
        bad = lane < kStreamThreads / 32 ? s_bad[lane] : 0u;
        m = __reduce_max_sync(0xFFFFFFFFu, m);
        bad = __reduce_add_sync(0xFFFFFFFFu, bad);
        if (lane == 0) {
            if (m) atomicMax(reinterpret_cast<uint32_t*>(&out->g_max), m);
            if (bad) atomicAdd(reinterpret_cast<unsigned long long*>(&out->n_nonfinite), (unsigned long long)bad);
            if (blockIdx.x == 0) out->n = n;
        }
    }
}

// ------------------------------------------------------------------------------------------
// Quantizer (Eq. 1, 2, 4) fused with the clip-out count (Sec. 3.3).  One thread owns the eight
// consecutive elements served by one Philox block and emits 4 bytes (nibbles) or 8 bytes (int8).
// Groups are walked from the end of the tensor backwards: the statistics pass has just streamed
// dY front to back, so its tail is what the L2 still holds.
//
// The kernel is bound by instruction issue as much as by HBM, so the common case takes a fast
// path that produces the same bits as the plain formulas with fewer instructions:
//   * x = RN(g / s) by two Newton corrections around the correctly rounded reciprocal of s
//     (q <- q + (g - s q) y twice, fused multiply-adds; Markstein's theorem makes the second
//     correction of a faithful quotient the correctly rounded one), valid while no intermediate
//     under- or overflows: s in [2^-60, 2^60]; the rare gradient so small that its residual
//     would underflow has |x| < 2^-40, where every outcome below depends on the sign of x only;
// Rounding is done in integer / fixed-point form (round_clipped), exact for the clipped |x| <= 127.
// Anything outside those ranges takes the literal path.
// ------------------------------------------------------------------------------------------
struct QuantParams {
    float c, s, y, qmaxf;  // clipping value, scale, RN(1 / s), qmax as float
    int qmax;
    bool zero;             // s == 0 or non-finite input: every code is 0
    bool fast;
};

// Rounding of the clipped, normalised value x (|x| <= qmax <= 127), shared by both paths; returns
// the code plus `bias` (the packing below wants non-negative digits).
//   nearest:    rint(x), ties to even (Eq. 4): the low bits of x + 1.5 * 2^23;
//   stochastic: floor(x) + [u < trunc(frac(x) * 2^16)] with frac(x) = x - floor(x) taken exactly
//               ==  floor((floor(x * 2^16) + 65535 - u) / 2^16): x * 2^16 is exact and fits int32,
//               the arithmetic shift is a floor division.  `k16` is 65535 - u.
template <bool kStochastic>
__device__ __forceinline__ int round_clipped(float x, uint32_t k16, int bias) {
    if (kStochastic) {
        const int fixed = __float2int_rd(__fmul_rn(x, 65536.0f));
        return (fixed + (int)k16 + (bias << 16)) >> 16;
    }
    return __float_as_int(__fadd_rn(x, 12582912.0f)) - (0x4B400000 - bias);
}

template <bool kStochastic>
__device__ __forceinline__ int quantize_one_literal(float g, const QuantParams& p, uint32_t k16, int bias) {
    float x = __fdiv_rn(g, p.s);                         // Eq. (1)
    x = fminf(fmaxf(x, -p.qmaxf), p.qmaxf);              // Eq. (2)
    return round_clipped<kStochastic>(x, k16, bias);
}

template <bool kStochastic>
__device__ __forceinline__ int quantize_one_fast(float g, const QuantParams& p, uint32_t k16, int bias) {
    float x = __fmul_rn(g, p.y);
    float r = __fmaf_rn(-p.s, x, g);
    x = __fmaf_rn(r, p.y, x);
    r = __fmaf_rn(-p.s, x, g);
    x = __fmaf_rn(r, p.y, x);                            // x = RN(g / s), Eq. (1)
    x = fminf(fmaxf(x, -p.qmaxf), p.qmaxf);              // Eq. (2): clip
    return round_clipped<kStochastic>(x, k16, bias);
}

// max(a, b, c) as one three-input instruction (sm_100); a NaN operand is ignored, as by fmaxf.
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float m;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(m) : "f"(a), "f"(b), "f"(c));
    return m;
}

// Codes are packed as digits of a base-16 (or base-256) number built by multiply-adds: with the
// bias 8 (128) every digit is non-negative, and flipping each digit's top bit afterwards turns
// digit = code + bias into the code's two's-complement field.

// Careful path for one group of eight: exact clip-out count, clip of x, every special case.
template <bool kPacked, bool kStochastic, bool kFastDiv>
__device__ __forceinline__ void careful_group(const float (&g)[8], const uint32_t (&r)[4], const QuantParams& p,
                                              bool nonfinite, uint32_t& n_out, uint32_t& lo, uint32_t& hi) {
    constexpr int kBias = kPacked ? 8 : 128;
    constexpr uint32_t kRadix = kPacked ? 16u : 256u;
    lo = 0; hi = 0;
#pragma unroll
    for (int e = 7; e >= 0; --e) {
        // the zeros that pad a ragged last group never exceed c >= 0: they add nothing to n_out
        n_out += (!nonfinite && fabsf(g[e]) > p.c) ? 1u : 0u;
        uint32_t digit = (uint32_t)kBias;
        if (!p.zero) {
            const uint32_t nr = ~r[e >> 1];
            const uint32_t k16 = (e & 1) ? (nr >> 16) : (nr & 0xFFFFu);   // 65535 - u
            digit = (uint32_t)(kFastDiv ? quantize_one_fast<kStochastic>(g[e], p, k16, kBias)
                                        : quantize_one_literal<kStochastic>(g[e], p, k16, kBias));
        }
        if (kPacked || e < 4) lo = lo * kRadix + digit;
        else hi = hi * kRadix + digit;
    }
    lo ^= kPacked ? 0x88888888u : 0x80808080u;
    hi ^= 0x80808080u;
}

// Streaming path for a group in which every |g| <= c (1 - 2^-20): nothing is clipped (so nothing
// is counted and x needs no clip: |x| < qmax), s is in the fast-division range, codes fit.
//   kMode 0: nibbles (b <= 4); 1: bytes, b = 5, 6; 2: bytes, b = 7, 8.
// Modes 0 and 1 round stochastically with ONE fused multiply-add in round-down mode:
//   RD(x * 2^16 + (1.5 * 2^23 + 65535 - u)) = 1.5 * 2^23 + floor(x * 2^16 + 65535 - u), whose bit
//   pattern shifted right by 16 is 0x4B40 + code (the sum stays inside [2^23, 2^24) for qmax <= 31).
// The constant offsets (0x4B40 or 0x4B400000 per digit) are removed once per word after packing.
template <int kMode, bool kStochastic>
__device__ __forceinline__ void stream_group(const float (&g)[8], const uint32_t (&r)[4], const QuantParams& p,
                                             uint32_t& lo, uint32_t& hi) {
    constexpr bool kPacked = kMode == 0;
    constexpr uint32_t kBias = kPacked ? 8u : 128u;
    constexpr uint32_t kRadix = kPacked ? 16u : 256u;
    constexpr uint32_t kOnes = kPacked ? 0x11111111u : 0x01010101u;      // sum of radix^e over a word's digits
    constexpr bool kFmaRound = kStochastic && kMode != 2;
    constexpr uint32_t kDigitOffset = kFmaRound ? 0x4B40u : (kStochastic ? 0u : 0x4B400000u);
    lo = 0; hi = 0;
#pragma unroll
    for (int e = 7; e >= 0; --e) {
        float x = __fmul_rn(g[e], p.y);
        float res = __fmaf_rn(-p.s, x, g[e]);
        x = __fmaf_rn(res, p.y, x);
        res = __fmaf_rn(-p.s, x, g[e]);
        x = __fmaf_rn(res, p.y, x);                      // x = RN(g / s), Eq. (1)
        uint32_t digit;
        if (kFmaRound) {
            const uint32_t kf = __byte_perm(~r[e >> 1], 0x4B400000u, (e & 1) ? 0x7632 : 0x7610);
            digit = __float_as_uint(__fmaf_rd(x, 65536.0f, __uint_as_float(kf))) >> 16;
        } else if (kStochastic) {
            const uint32_t nr = ~r[e >> 1];
            const uint32_t k16 = (e & 1) ? (nr >> 16) : (nr & 0xFFFFu);
            digit = (uint32_t)((__float2int_rd(__fmul_rn(x, 65536.0f)) + (int)k16 + (int)(kBias << 16)) >> 16);
        } else {
            digit = __float_as_uint(__fadd_rn(x, 12582912.0f));           // 0x4B400000 + rint(x), Eq. (4)
        }
        if (kPacked || e < 4) lo = lo * kRadix + digit;
        else hi = hi * kRadix + digit;
    }
    constexpr uint32_t kFix = (kStochastic && kMode == 2) ? 0u : (kDigitOffset - kBias) * kOnes;
    constexpr uint32_t kFlip = kPacked ? 0x88888888u : 0x80808080u;
    lo = (lo - kFix) ^ kFlip;
    hi = (hi - kFix) ^ kFlip;
}

// One pass of a thread over its groups t, t + stride, ... below t_end.  kFromCache: the Philox words
// of these groups were written by the same thread earlier in the kernel as
// cache[slot * blockDim.x + threadIdx.x], slot counting from 0 at the first group of the pass.  (A
// separate loop rather than a branch per group: the compiler turned the branch into predicated code
// that still issued every instruction of the generator.)
// Idx: the type of the group counters -- 32-bit whenever the group count plus one stride fits (every
// realistic tensor), which turns each address into one wide multiply-add; 64-bit otherwise.
template <int kMode, bool kStochastic, bool kFast, bool kFromCache, typename Idx>
__device__ __forceinline__ void
quantize_group_loop(Idx& t, Idx t_end, Idx stride, const float* __restrict__ dY, uint64_t n,
                    const QuantParams& p, bool nonfinite, const uint32_t* __restrict__ round_keys, uint32_t it0,
                    uint32_t it1, uint64_t grp_offset, uint8_t* __restrict__ q_out, uint8_t* __restrict__ q8_out,
                    const uint4* cache, uint32_t& n_out) {
    constexpr bool kPacked = kMode == 0;
    const Idx last_group = (Idx)(((n + 7) >> 3) - 1), whole_groups = (Idx)(n >> 3);
    const float c_safe = __fmul_rn(p.c, 0.99999905f);   // c (1 - 2^-20)
    const bool want_rand = kStochastic && !p.zero;

    auto load_group = [&](Idx grp, bool full, float (&g)[8]) {
        if (full) {
            const float4* src = reinterpret_cast<const float4*>(dY) + 2 * (size_t)grp;
            const float4 a = __ldg(src);
            const float4 b = __ldg(src + 1);
            g[0] = a.x; g[1] = a.y; g[2] = a.z; g[3] = a.w;
            g[4] = b.x; g[5] = b.y; g[6] = b.z; g[7] = b.w;
        } else {
            const uint64_t base = (uint64_t)grp << 3;
#pragma unroll
            for (int e = 0; e < 8; ++e) g[e] = base + e < n ? dY[base + e] : 0.0f;
        }
    };
    auto rand_group = [&](Idx grp, uint32_t slot, uint32_t (&r)[4]) {
        r[0] = r[1] = r[2] = r[3] = 0u;
        if (!want_rand) return;
        if (kFromCache) {
            const uint4 w = cache[slot * kStreamThreads + threadIdx.x];
            r[0] = w.x; r[1] = w.y; r[2] = w.z; r[3] = w.w;
        } else {
            const uint64_t blk = (uint64_t)grp + grp_offset;   // the block's index in the whole (possibly sharded) tensor
            philox4x32_10_keyed((uint32_t)blk, (uint32_t)(blk >> 32), it0, it1, round_keys, r);
        }
    };
    // the largest magnitude of the group decides: anything near the clipping value sends the whole group to
    // the careful path
    auto streamable = [&](const float (&g)[8]) {
        const float m012 = fmax3(fabsf(g[0]), fabsf(g[1]), fabsf(g[2]));
        const float m345 = fmax3(fabsf(g[3]), fabsf(g[4]), fabsf(g[5]));
        return kFast && fmax3(m012, m345, fmaxf(fabsf(g[6]), fabsf(g[7]))) <= c_safe;
    };
    // lo / hi: packed: lo holds all eight nibbles; bytes: lo = codes 0-3, hi = codes 4-7
    auto store_group = [&](Idx grp, bool full, uint32_t lo, uint32_t hi) {
        const uint64_t base = (uint64_t)grp << 3;
        if (kPacked && q8_out != nullptr) {
            // second copy, one sign-extended byte per code: nibbles 0,2,4,6 and 1,3,5,7, then interleave
            uint32_t ev = lo & 0x0F0F0F0Fu, od = (lo >> 4) & 0x0F0F0F0Fu;
            // (n ^ 8) + 0x78 stays inside its byte; flipping that byte's top bit leaves the nibble's value as int8
            ev = ((ev ^ 0x08080808u) + 0x78787878u) ^ 0x80808080u;
            od = ((od ^ 0x08080808u) + 0x78787878u) ^ 0x80808080u;
            const uint32_t b03 = __byte_perm(ev, od, 0x5140), b47 = __byte_perm(ev, od, 0x7362);
            if (full) {
                reinterpret_cast<uint2*>(q8_out)[grp] = make_uint2(b03, b47);
            } else {
                for (int e = 0; e < 8 && base + e < n; ++e)
                    q8_out[base + e] = (uint8_t)((e < 4 ? b03 >> (8 * e) : b47 >> (8 * (e - 4))) & 0xFFu);
            }
        }
        if (kPacked) {
            if (full) {
                reinterpret_cast<uint32_t*>(q_out)[grp] = lo;
            } else {
                const uint64_t nbytes = (n + 1) >> 1;
                for (uint64_t byte = base >> 1; byte < nbytes; ++byte)
                    q_out[byte] = (uint8_t)(lo >> (8 * (byte - (base >> 1))));
            }
        } else {
            if (full) {
                reinterpret_cast<uint2*>(q_out)[grp] = make_uint2(lo, hi);
            } else {
                for (int e = 0; e < 8 && base + e < n; ++e)
                    q_out[base + e] = (uint8_t)((e < 4 ? lo >> (8 * e) : hi >> (8 * (e - 4))) & 0xFFu);
            }
        }
    };
    auto one_group = [&](Idx grp, bool full, const float (&g)[8], const uint32_t (&r)[4]) {
        uint32_t lo, hi;
        if (streamable(g)) stream_group<kMode, kStochastic>(g, r, p, lo, hi);
        else careful_group<kPacked, kStochastic, kFast>(g, r, p, nonfinite, n_out, lo, hi);
        store_group(grp, full, lo, hi);
    };

    uint32_t slot = 0;
    if (kFast) {
        // Two groups per step: their loads, their Philox chains (ten dependent rounds each) and their division chains
        // sit in one basic block, so the scheduler interleaves them and the fixed latencies of one hide behind the other.
        for (; t + stride < t_end; t += 2 * stride, slot += 2) {
            const Idx grp_a = last_group - t, grp_b = grp_a - stride;
            const bool full_a = grp_a < whole_groups;   // (grp_b < grp_a is then whole too)
            float ga[8], gb[8];
            load_group(grp_a, full_a, ga);
            load_group(grp_b, true, gb);
            uint32_t ra[4], rb[4];
            rand_group(grp_a, slot, ra);
            rand_group(grp_b, slot + 1, rb);
            if (full_a && streamable(ga) && streamable(gb)) {
                uint32_t lo_a, hi_a, lo_b, hi_b;
                stream_group<kMode, kStochastic>(ga, ra, p, lo_a, hi_a);
                stream_group<kMode, kStochastic>(gb, rb, p, lo_b, hi_b);
                store_group(grp_a, true, lo_a, hi_a);
                store_group(grp_b, true, lo_b, hi_b);
            } else {
                one_group(grp_a, full_a, ga, ra);
                one_group(grp_b, true, gb, rb);
            }
        }
    }
    for (; t < t_end; t += stride, ++slot) {
        const Idx grp = last_group - t;
        const bool full = grp < whole_groups;
        float g[8];
        load_group(grp, full, g);
        uint32_t r[4];
        rand_group(grp, slot, r);
        one_group(grp, full, g, r);
    }
}

// All groups of this thread, walked from the end of the tensor backwards.  kCached: the Philox words of
// the thread's first `nslots` groups come from `cache`; later groups are generated here.
template <int kMode, bool kStochastic, bool kFast, bool kCached = false>
__device__ __forceinline__ uint32_t
quantize_groups(const float* __restrict__ dY, uint64_t n, const QuantParams& p, bool nonfinite,
                const uint32_t* __restrict__ round_keys, uint32_t it0, uint32_t it1, uint64_t grp_offset,
                uint8_t* __restrict__ q_out, uint8_t* __restrict__ q8_out, const uint4* cache = nullptr,
                uint32_t nslots = 0) {
    const uint64_t ngroups = (n + 7) >> 3;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    const uint64_t t0 = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool cached = kCached && kStochastic && !p.zero;
    const uint64_t cached_end = cached ? (t0 + (uint64_t)nslots * stride < ngroups ? t0 + (uint64_t)nslots * stride : ngroups) : 0;
    uint32_t n_out = 0;
    if (ngroups + stride <= 0xFFFFFFFFull) {             // no counter passes 2^32, not even after the last step
        uint32_t t = (uint32_t)t0;
        if (cached)
            quantize_group_loop<kMode, kStochastic, kFast, true, uint32_t>(t, (uint32_t)cached_end, (uint32_t)stride, dY, n, p,
                                                                           nonfinite, round_keys, it0, it1, grp_offset,
                                                                           q_out, q8_out, cache, n_out);
        quantize_group_loop<kMode, kStochastic, kFast, false, uint32_t>(t, (uint32_t)ngroups, (uint32_t)stride, dY, n, p,
                                                                        nonfinite, round_keys, it0, it1, grp_offset, q_out,
                                                                        q8_out, cache, n_out);
    } else {
        uint64_t t = t0;
        if (cached)
            quantize_group_loop<kMode, kStochastic, kFast, true, uint64_t>(t, cached_end, stride, dY, n, p, nonfinite,
                                                                           round_keys, it0, it1, grp_offset, q_out, q8_out,
                                                                           cache, n_out);
        quantize_group_loop<kMode, kStochastic, kFast, false, uint64_t>(t, ngroups, stride, dY, n, p, nonfinite, round_keys,
                                                                        it0, it1, grp_offset, q_out, q8_out, cache, n_out);
    }
    return n_out;
}

// Bit-width and rounding mode live in the device-side state, so the specialisation is chosen
// on the device (a block-uniform branch) and the host never has to read the state back.
__global__ void __launch_bounds__(kStreamThreads, 4)
quantize_kernel(const float* __restrict__ dY, uint64_t n, const lbt_interval_state* __restrict__ st,
                lbt_grad_stats_t* __restrict__ stats, uint8_t* __restrict__ q_out, uint8_t* __restrict__ q8_out,
                uint64_t grp_offset, int expect_bits) {
    // the layout of q_out is the one the host sized it for; a state that disagrees gets zero codes
    const int state_bits = min(max(st->bits, 2), 8);
    const int bits = expect_bits != 0 ? expect_bits : state_bits;
    const bool mismatch = bits != state_bits;
    const bool sr = st->rounding == LBT_ROUND_STOCHASTIC;
    QuantParams p;
    const float gamma = st->gamma;
    p.qmax = (1 << (bits - 1)) - 1;
    p.qmaxf = (float)p.qmax;
    p.c = __fmul_rn(gamma, stats->g_max);                // c_g = gamma * g_max (Sec. 3.1)
    p.s = __fdiv_rn(p.c, p.qmaxf);                       // Eq. (2)
    const bool nonfinite = stats->n_nonfinite != 0;
    p.zero = nonfinite || mismatch || !(p.s > 0.0f);
    p.y = p.zero ? 0.0f : __frcp_rn(p.s);
    p.fast = !p.zero && p.s >= 8.673617379884035e-19f && p.s <= 1.152921504606847e18f;    // 2^-60 .. 2^60
    const uint32_t it0 = (uint32_t)st->iter, it1 = (uint32_t)(st->iter >> 32);
    if (mismatch && blockIdx.x == 0 && threadIdx.x == 0)   // (the status word is the one writable field here)
        atomicCAS(const_cast<int32_t*>(&st->dev_status), (int32_t)LBT_OK, (int32_t)LBT_ERR_BITS_MISMATCH);
    __shared__ __align__(16) uint32_t round_keys[20];    // Philox key schedule: key + round * Weyl increments
    if (threadIdx.x < 10) {
        round_keys[2 * threadIdx.x] = (uint32_t)st->seed + threadIdx.x * 0x9E3779B9u;
        round_keys[2 * threadIdx.x + 1] = (uint32_t)(st->seed >> 32) + threadIdx.x * 0xBB67AE85u;
    }
    __syncthreads();

    uint32_t n_out;
#define LBT_QUANT_CASE(MODE, SR, FAST) \
    n_out = quantize_groups<MODE, SR, FAST>(dY, n, p, nonfinite, round_keys, it0, it1, grp_offset, q_out, q8_out)
    const int mode = bits <= 4 ? 0 : (bits <= 6 ? 1 : 2);
    if (p.fast) {
        if (mode == 0)      { if (sr) LBT_QUANT_CASE(0, true, true); else LBT_QUANT_CASE(0, false, true); }
        else if (mode == 1) { if (sr) LBT_QUANT_CASE(1, true, true); else LBT_QUANT_CASE(1, false, true); }
        else                { if (sr) LBT_QUANT_CASE(2, true, true); else LBT_QUANT_CASE(2, false, true); }
    } else {
        if (mode == 0) { if (sr) LBT_QUANT_CASE(0, true, false); else LBT_QUANT_CASE(0, false, false); }
        else           { if (sr) LBT_QUANT_CASE(2, true, false); else LBT_QUANT_CASE(2, false, false); }
    }
#undef LBT_QUANT_CASE

    n_out = __reduce_add_sync(0xFFFFFFFFu, n_out);
    __shared__ uint32_t s_cnt[kStreamThreads / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) s_cnt[warp] = n_out;
    __syncthreads();
    if (warp == 0) {
        n_out = lane < kStreamThreads / 32 ? s_cnt[lane] : 0u;
        n_out = __reduce_add_sync(0xFFFFFFFFu, n_out);
        if (lane == 0) {
            if (n_out) atomicAdd(reinterpret_cast<unsigned long long*>(&stats->n_out), (unsigned long long)n_out);
            if (blockIdx.x == 0) { stats->c = p.c; stats->scale = p.s; }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Clipping-factor update, Eq. (15), (16) / Algorithm 1.  One thread.
// ------------------------------------------------------------------------------------------
__global__ void update_interval_kernel(lbt_interval_state* __restrict__ st,
                                       const lbt_grad_stats_t* __restrict__ stats) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    if (stats->n_nonfinite != 0) {
        if (st->dev_status == LBT_OK) st->dev_status = LBT_ERR_NONFINITE;
    } else if (st->dev_status == LBT_ERR_BITS_MISMATCH) {
        // the quantizer wrote zero codes for a bit-width the host did not expect: gamma stays
    } else {
        const int bits = min(max(st->bits, 2), 8);
        const double levels = (double)((1 << bits) - 1);
        const double lhs = __dmul_rn((double)stats->n_out, levels);
        const double rhs = __dmul_rn((double)st->alpha, (double)stats->n);
        const int sgn = (lhs > rhs) - (lhs < rhs);
        float g = __fadd_rn(st->gamma, __fmul_rn(st->beta, (float)sgn));
        g = fminf(fmaxf(g, st->gamma_min), st->gamma_max);
        st->gamma = g;
    }
    st->iter += 1;
}

// ------------------------------------------------------------------------------------------
// Statistics, quantization and the clipping-factor update in ONE cooperative launch (Sec. 3.1, 3.3,
// Eq. 1, 2, 4, 15, 16), for gradient tensors small enough that their second reading is served by L2.
// Phase 1: abs-max / non-finite count of this block's share, atomics into the statistics.  The phase
// waits on HBM with its issue slots idle, so with stochastic rounding every thread also generates the
// Philox words of its first `nslots` phase-2 groups there (they depend on the element index only, not
// on g_max) and parks them in dynamic shared memory (nslots * blockDim.x * 16 bytes per block): phase 2,
// which is bound by instruction issue, then skips the generator for those groups.
// Grid barrier: every block adds 1 to stats->reserved and waits (bounded) until all have.
// Phase 2: the quantizer exactly as quantize_kernel runs it, now with the global g_max.
// The block that finishes last (second count on the same word) applies Eq. (15), (16) and clears the
// word.  Results are bit-identical to the three separate launches.  The launch is cooperative, so all
// blocks are resident and the barrier cannot wait on a block that has not started.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kStreamThreads, 4)
fused_quantize_kernel(const float* __restrict__ dY, uint64_t n, lbt_interval_state* st, lbt_grad_stats_t* stats,
                      uint8_t* __restrict__ q_out, uint8_t* __restrict__ q8_out, uint64_t grp_offset,
                      uint32_t nslots, int expect_bits) {
    __shared__ uint32_t s_m[kStreamThreads / 32], s_bad[kStreamThreads / 32];
    __shared__ __align__(16) uint32_t round_keys[20];
    extern __shared__ uint4 rnd_cache[];                 // [nslots][kStreamThreads]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // a launch chained behind this one (the expansion of the fused layer call) may be scheduled as blocks
    // here retire; the part of it that reads this kernel's output waits for this grid on the device
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // seed, iteration and rounding mode are not written before every block has left phase 2
    const bool sr = st->rounding == LBT_ROUND_STOCHASTIC;
    const uint64_t iter = st->iter;
    const uint32_t it0 = (uint32_t)iter, it1 = (uint32_t)(iter >> 32);
    if (threadIdx.x < 10) {
        round_keys[2 * threadIdx.x] = (uint32_t)st->seed + threadIdx.x * 0x9E3779B9u;
        round_keys[2 * threadIdx.x + 1] = (uint32_t)(st->seed >> 32) + threadIdx.x * 0xBB67AE85u;
    }
    __syncthreads();
    if (!sr) nslots = 0;
    {   // ---- phase 1
        const uint64_t nvec = n >> 2;
        const float4* __restrict__ v4 = reinterpret_cast<const float4*>(dY);
        uint32_t m = 0, bad = 0;
        const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
        uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
        const uint64_t ngroups = (n + 7) >> 3;
        uint64_t fill_t = i;                             // phase-2 group counter of the slot filled next
        uint32_t fill_slot = 0;
        auto fill_one = [&]() {
            if (fill_slot < nslots) {
                if (fill_t < ngroups) {
                    const uint64_t blk = ngroups - 1 - fill_t + grp_offset;
                    uint32_t r[4];
                    philox4x32_10_keyed((uint32_t)blk, (uint32_t)(blk >> 32), it0, it1, round_keys, r);
                    rnd_cache[fill_slot * kStreamThreads + threadIdx.x] = make_uint4(r[0], r[1], r[2], r[3]);
                }
                ++fill_slot;
                fill_t += stride;
            }
        };
        for (; i + 3 * stride < nvec; i += 4 * stride) {
            const float4 a = __ldg(v4 + i), b = __ldg(v4 + i + stride);
            const float4 c = __ldg(v4 + i + 2 * stride), d = __ldg(v4 + i + 3 * stride);
            fill_one(); fill_one();                      // 16 elements loaded = two groups' worth
            absmax_accumulate4(a, m, bad); absmax_accumulate4(b, m, bad);
            absmax_accumulate4(c, m, bad); absmax_accumulate4(d, m, bad);
        }
        for (; i < nvec; i += stride) absmax_accumulate4(__ldg(v4 + i), m, bad);
        while (fill_slot < nslots) fill_one();
        if (blockIdx.x == 0 && threadIdx.x < (n & 3)) absmax_accumulate(dY[(nvec << 2) + threadIdx.x], m, bad);
        m = __reduce_max_sync(0xFFFFFFFFu, m);
        bad = __reduce_add_sync(0xFFFFFFFFu, bad);
        if (lane == 0) { s_m[warp] = m; s_bad[warp] = bad; }
        __syncthreads();
        if (warp == 0) {
            m = lane < kStreamThreads / 32 ? s_m[lane] : 0u;
            bad = lane < kStreamThreads / 32 ? s_bad[lane] : 0u;
            m = __reduce_max_sync(0xFFFFFFFFu, m);
            bad = __reduce_add_sync(0xFFFFFFFFu, bad);
            if (lane == 0) {
                if (m) atomicMax(reinterpret_cast<uint32_t*>(&stats->g_max), m);
                if (bad) atomicAdd(reinterpret_cast<unsigned long long*>(&stats->n_nonfinite), (unsigned long long)bad);
                if (blockIdx.x == 0) stats->n = n;
                // ---- grid barrier (bounded: 2 s)
                __threadfence();
                atomicAdd(&stats->reserved, 1u);
                if (!counter_wait_bounded(&stats->reserved, gridDim.x, kGridBarrierLimitNs))
                    atomicCAS(&st->dev_status, (int32_t)LBT_OK, (int32_t)LBT_ERR_TIMEOUT);
                __threadfence();
            }
        }
        __syncthreads();
    }
    // ---- phase 2 (the body of quantize_kernel)
    const int state_bits = min(max(st->bits, 2), 8);
    const int bits = expect_bits != 0 ? expect_bits : state_bits;
    const bool mismatch = bits != state_bits;
    QuantParams p;
    const float gamma = *reinterpret_cast<volatile float*>(&st->gamma);
    p.qmax = (1 << (bits - 1)) - 1;
    p.qmaxf = (float)p.qmax;
    p.c = __fmul_rn(gamma, *reinterpret_cast<volatile float*>(&stats->g_max));   // c_g = gamma * g_max (Sec. 3.1)
    p.s = __fdiv_rn(p.c, p.qmaxf);                                               // Eq. (2)
    const bool nonfinite = *reinterpret_cast<volatile unsigned long long*>(&stats->n_nonfinite) != 0;
    p.zero = nonfinite || mismatch || !(p.s > 0.0f);
    p.y = p.zero ? 0.0f : __frcp_rn(p.s);
    p.fast = !p.zero && p.s >= 8.673617379884035e-19f && p.s <= 1.152921504606847e18f;    // 2^-60 .. 2^60
    uint32_t n_out;
#define LBT_QUANT_CASE(MODE, SR, FAST)                                                                          \
    n_out = quantize_groups<MODE, SR, FAST, SR>(dY, n, p, nonfinite, round_keys, it0, it1, grp_offset, q_out, \
                                                q8_out, rnd_cache, nslots)
    const int mode = bits <= 4 ? 0 : (bits <= 6 ? 1 : 2);
    if (p.fast) {
        if (mode == 0)      { if (sr) LBT_QUANT_CASE(0, true, true); else LBT_QUANT_CASE(0, false, true); }
        else if (mode == 1) { if (sr) LBT_QUANT_CASE(1, true, true); else LBT_QUANT_CASE(1, false, true); }
        else                { if (sr) LBT_QUANT_CASE(2, true, true); else LBT_QUANT_CASE(2, false, true); }
    } else {
        if (mode == 0) { if (sr) LBT_QUANT_CASE(0, true, false); else LBT_QUANT_CASE(0, false, false); }
        else           { if (sr) LBT_QUANT_CASE(2, true, false); else LBT_QUANT_CASE(2, false, false); }
    }
#undef LBT_QUANT_CASE
    n_out = __reduce_add_sync(0xFFFFFFFFu, n_out);
    if (lane == 0) s_m[warp] = n_out;
    __syncthreads();
    if (warp == 0) {
        n_out = lane < kStreamThreads / 32 ? s_m[lane] : 0u;
        n_out = __reduce_add_sync(0xFFFFFFFFu, n_out);
        if (lane == 0) {
            if (n_out) atomicAdd(reinterpret_cast<unsigned long long*>(&stats->n_out), (unsigned long long)n_out);
            if (blockIdx.x == 0) { stats->c = p.c; stats->scale = p.s; }
            // ---- the last block to get here updates the clipping factor (Eq. 15, 16 / Algorithm 1)
            __threadfence();
            if (atomicAdd(&stats->reserved, 1u) == 2u * gridDim.x - 1u) {
                __threadfence();
                const unsigned long long total_out = *reinterpret_cast<volatile unsigned long long*>(&stats->n_out);
                if (nonfinite) {
                    if (st->dev_status == LBT_OK) st->dev_status = LBT_ERR_NONFINITE;
                } else if (mismatch) {
                    if (st->dev_status == LBT_OK) st->dev_status = LBT_ERR_BITS_MISMATCH;
                } else {
                    const double levels = (double)((1 << bits) - 1);
                    const double lhs = __dmul_rn((double)total_out, levels);
                    const double rhs = __dmul_rn((double)st->alpha, (double)n);
                    const int sgn = (lhs > rhs) - (lhs < rhs);
                    float g = __fadd_rn(gamma, __fmul_rn(st->beta, (float)sgn));
                    g = fminf(fmaxf(g, st->gamma_min), st->gamma_max);
                    st->gamma = g;
                }
                st->iter = iter + 1;
                stats->reserved = 0u;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Forward-side quantizers (Eq. 1-4): clipping value from the caller, rounding to nearest (ties to
// even).  kSigned: weights, Eq. (2), codes in [-qmax, qmax]; otherwise activations, Eq. (3), codes in
// [0, 2^b - 1].  One pass; a thread owns eight consecutive elements (4 or 8 output bytes).
// The quotient clip(x, c) / s is the correctly rounded one: two Newton corrections around RN(1 / s)
// while s is in [2^-60, 2^60] (|clip(x, c)| <= c keeps every intermediate in range; a value so small
// that its residual underflows rounds to code 0 either way), the division routine otherwise.
// ------------------------------------------------------------------------------------------
struct FwdParams {
    float c, lo, s, y;
    int levels, code_lo;
};

// Eight clipped, normalised, rounded codes (Eq. 1-4) packed as nibbles (w0) or bytes (w0, w1).
template <bool kPacked, bool kFast>
__device__ __forceinline__ void fwd_group(const float (&g)[8], const FwdParams& p, uint32_t& w0, uint32_t& w1) {
    w0 = 0; w1 = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const float v = fminf(fmaxf(g[e], p.lo), p.c);                   // clip(x, c), Eq. (2) / Eq. (3)
        float q;
        if (kFast) {
            q = __fmul_rn(v, p.y);
            float r = __fmaf_rn(-p.s, q, v);
            q = __fmaf_rn(r, p.y, q);
            r = __fmaf_rn(-p.s, q, v);
            q = __fmaf_rn(r, p.y, q);                                    // RN(v / s), Eq. (1)
        } else {
            q = __fdiv_rn(v, p.s);
        }
        const int code = min(max(__float2int_rn(q), p.code_lo), p.levels);   // Eq. (4): nearest, ties to even
        if (kPacked) w0 |= ((uint32_t)code & 0xFu) << (4 * e);
        else if (e < 4) w0 |= ((uint32_t)code & 0xFFu) << (8 * e);
        else w1 |= ((uint32_t)code & 0xFFu) << (8 * (e - 4));
    }
}

template <bool kPacked>
__device__ __forceinline__ void fwd_store(uint8_t* __restrict__ q_out, uint64_t grp, uint64_t n, uint32_t w0, uint32_t w1) {
    const uint64_t base = grp << 3;
    if (base + 8 <= n) {
        if (kPacked) reinterpret_cast<uint32_t*>(q_out)[grp] = w0;
        else reinterpret_cast<uint2*>(q_out)[grp] = make_uint2(w0, w1);
    } else if (kPacked) {
        const uint64_t nbytes = (n + 1) >> 1;
        for (uint64_t byte = base >> 1; byte < nbytes; ++byte) q_out[byte] = (uint8_t)(w0 >> (8 * (byte - (base >> 1))));
    } else {
        for (int e = 0; e < 8 && base + e < n; ++e)
            q_out[base + e] = (uint8_t)((e < 4 ? w0 >> (8 * e) : w1 >> (8 * (e - 4))) & 0xFFu);
    }
}

__device__ __forceinline__ void fwd_load(const float* __restrict__ x, uint64_t grp, uint64_t n, float (&g)[8]) {
    const uint64_t base = grp << 3;
    if (base + 8 <= n) {
        const float4 a = __ldcs(reinterpret_cast<const float4*>(x + base));
        const float4 b = __ldcs(reinterpret_cast<const float4*>(x + base) + 1);
        g[0] = a.x; g[1] = a.y; g[2] = a.z; g[3] = a.w;
        g[4] = b.x; g[5] = b.y; g[6] = b.z; g[7] = b.w;
    } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) g[e] = base + e < n ? x[base + e] : 0.0f;
    }
}

// Two groups per thread and step, both loaded before either is worked on, to keep more bytes in flight.
template <bool kPacked, bool kFast>
__device__ __forceinline__ void fwd_stream(const float* __restrict__ x, uint64_t n, const FwdParams& p,
                                           uint8_t* __restrict__ q_out) {
    const uint64_t ngroups = (n + 7) >> 3;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    for (; grp + stride < ngroups; grp += 2 * stride) {
        float g0[8], g1[8];
        fwd_load(x, grp, n, g0);
        fwd_load(x, grp + stride, n, g1);
        uint32_t w0, w1;
        fwd_group<kPacked, kFast>(g0, p, w0, w1);
        fwd_store<kPacked>(q_out, grp, n, w0, w1);
        fwd_group<kPacked, kFast>(g1, p, w0, w1);
        fwd_store<kPacked>(q_out, grp + stride, n, w0, w1);
    }
    if (grp < ngroups) {
        float g0[8];
        fwd_load(x, grp, n, g0);
        uint32_t w0, w1;
        fwd_group<kPacked, kFast>(g0, p, w0, w1);
        fwd_store<kPacked>(q_out, grp, n, w0, w1);
    }
}

template <bool kSigned>
__global__ void __launch_bounds__(kStreamThreads, 4)
quantize_fwd_kernel(const float* __restrict__ x, uint64_t n, const float* __restrict__ clip, int bits,
                    uint8_t* __restrict__ q_out, float* __restrict__ scale_out) {
    FwdParams p;
    p.c = *clip;
    p.levels = kSigned ? (1 << (bits - 1)) - 1 : (1 << bits) - 1;
    p.s = __fdiv_rn(p.c, (float)p.levels);                                // Eq. (2) / Eq. (3)
    const bool zero = !(p.s > 0.0f) || isinf(p.s);
    const bool fast = !zero && p.s >= 8.673617379884035e-19f && p.s <= 1.152921504606847e18f;   // 2^-60 .. 2^60
    p.y = fast ? __frcp_rn(p.s) : 0.0f;
    p.lo = kSigned ? -p.c : 0.0f;
    p.code_lo = kSigned ? -p.levels : 0;
    const bool packed = bits <= 4;
    if (blockIdx.x == 0 && threadIdx.x == 0) *scale_out = zero ? 0.0f : p.s;
    if (zero) {
        // no positive finite scale: every code is 0
        const uint64_t ngroups = (n + 7) >> 3;
        for (uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < ngroups;
             grp += (uint64_t)gridDim.x * blockDim.x) {
            if (packed) fwd_store<true>(q_out, grp, n, 0u, 0u);
            else fwd_store<false>(q_out, grp, n, 0u, 0u);
        }
    } else if (packed) {
        if (fast) fwd_stream<true, true>(x, n, p, q_out); else fwd_stream<true, false>(x, n, p, q_out);
    } else {
        if (fast) fwd_stream<false, true>(x, n, p, q_out); else fwd_stream<false, false>(x, n, p, q_out);
    }
}

// One block arrives at a counter barrier that expects two arrivals: the wait of the one-launch
// quantizer's grid barrier, run on a count that is never reached.
__global__ void selftest_barrier_kernel(int32_t* status, uint64_t limit_ns) {
    __shared__ uint32_t arrivals;
    if (threadIdx.x != 0) return;
    arrivals = 0u;
    atomicAdd(&arrivals, 1u);
    if (!counter_wait_bounded(&arrivals, 2u, limit_ns)) atomicCAS(status, (int32_t)LBT_OK, (int32_t)LBT_ERR_TIMEOUT);
}

static int stream_grid(uint64_t work_items) {
    const uint64_t blocks = (work_items + kStreamThreads - 1) / kStreamThreads;
    const uint64_t cap = (uint64_t)kNumSMs * kBlocksPerSM;
    return (int)(blocks < 1 ? 1 : (blocks < cap ? blocks : cap));
}

}  // namespace lbt

using namespace lbt;

extern "C" lbt_status lbt_selftest_barrier_timeout(int32_t* dev_status, uint32_t limit_us, void* cuda_stream) {
    if (dev_status == nullptr || limit_us == 0 || limit_us > 1000000u) return LBT_ERR_INVALID_ARG;
    selftest_barrier_kernel<<<1, 32, 0, as_stream(cuda_stream)>>>(dev_status, (uint64_t)limit_us * 1000ull);
    return launch_status();
}

extern "C" lbt_status lbt_grad_stats(const float* dY, uint64_t n, const lbt_interval_state* st,
                                     lbt_grad_stats_t* out, void* ws, size_t ws_bytes, void* cuda_stream) {
    (void)st; (void)ws; (void)ws_bytes;
    if (out == nullptr || (n != 0 && dY == nullptr)) return LBT_ERR_INVALID_ARG;
    if (!aligned16(dY) || (reinterpret_cast<uintptr_t>(out) & 7u)) return LBT_ERR_ALIGNMENT;
    cudaStream_t stream = as_stream(cuda_stream);
    LBT_CUDA_TRY(cudaMemsetAsync(out, 0, sizeof(lbt_grad_stats_t), stream));
    timing_begin(LBT_TIME_STATS, stream);
    absmax_kernel<<<stream_grid((n >> 2) / 4 + 1), kStreamThreads, 0, stream>>>(dY, n, out);
    timing_end(LBT_TIME_STATS, stream);
    return launch_status();
}

lbt_status lbt::launch_quantize(const float* dY, uint64_t n, const lbt_interval_state* st, lbt_grad_stats_t* stats,
                                uint8_t* q_out, uint8_t* q8_out, bool clear_n_out, cudaStream_t stream,
                                uint64_t index_offset, int expect_bits) {
    if (clear_n_out) LBT_CUDA_TRY(cudaMemsetAsync(&stats->n_out, 0, sizeof(uint64_t), stream));
    timing_begin(LBT_TIME_QUANTIZE, stream);
    quantize_kernel<<<stream_grid((n + 7) >> 3), kStreamThreads, 0, stream>>>(dY, n, st, stats, q_out, q8_out,
                                                                                 index_offset >> 3, expect_bits);
    timing_end(LBT_TIME_QUANTIZE, stream);
    return launch_status();
}

extern "C" lbt_status lbt_quantize_grad(const float* dY, uint64_t n, const lbt_interval_state* st,
                                        lbt_grad_stats_t* stats, void* q_out, void* ws, size_t ws_bytes,
                                        void* cuda_stream) {
    (void)ws; (void)ws_bytes;
    if (st == nullptr || stats == nullptr || (n != 0 && (dY == nullptr || q_out == nullptr)))
        return LBT_ERR_INVALID_ARG;
    if (!aligned16(dY) || !aligned16(q_out) || (reinterpret_cast<uintptr_t>(stats) & 7u) ||
        (reinterpret_cast<uintptr_t>(st) & 7u))
        return LBT_ERR_ALIGNMENT;
    return launch_quantize(dY, n, st, stats, static_cast<uint8_t*>(q_out), nullptr, true, as_stream(cuda_stream));
}

extern "C" lbt_status lbt_update_interval(lbt_interval_state* st, const lbt_grad_stats_t* stats,
                                          void* cuda_stream) {
    if (st == nullptr || stats == nullptr) return LBT_ERR_INVALID_ARG;
    update_interval_kernel<<<1, 32, 0, as_stream(cuda_stream)>>>(st, stats);
    return launch_status();
}

template <bool kSigned>
static lbt_status quantize_fwd(const float* x, uint64_t n, const float* d_clip, int bits, void* q_out,
                               float* d_scale_out, void* cuda_stream) {
    if (d_clip == nullptr || d_scale_out == nullptr || (n != 0 && (x == nullptr || q_out == nullptr)))
        return LBT_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8) return LBT_ERR_UNSUPPORTED_BITS;
    if (!aligned16(x) || !aligned16(q_out) || (reinterpret_cast<uintptr_t>(d_clip) & 3u) ||
        (reinterpret_cast<uintptr_t>(d_scale_out) & 3u))
        return LBT_ERR_ALIGNMENT;
    cudaStream_t stream = as_stream(cuda_stream);
    timing_begin(LBT_TIME_FWD_QUANT, stream);
    quantize_fwd_kernel<kSigned><<<stream_grid((n + 7) >> 3), kStreamThreads, 0, stream>>>(
        x, n, d_clip, bits, static_cast<uint8_t*>(q_out), d_scale_out);
    timing_end(LBT_TIME_FWD_QUANT, stream);
    return launch_status();
}

extern "C" lbt_status lbt_quantize_weight(const float* w, uint64_t n, const float* d_clip, int bits, void* q_out,
                                          float* d_scale_out, void* cuda_stream) {
    return quantize_fwd<true>(w, n, d_clip, bits, q_out, d_scale_out, cuda_stream);
}

extern "C" lbt_status lbt_quantize_act(const float* x, uint64_t n, const float* d_clip, int bits, void* q_out,
                                       float* d_scale_out, void* cuda_stream) {
    return quantize_fwd<false>(x, n, d_clip, bits, q_out, d_scale_out, cuda_stream);
}

extern "C" lbt_status lbt_quantize_grad_shard(const float* dY, uint64_t n, uint64_t index_offset,
                                              const lbt_interval_state* st, lbt_grad_stats_t* stats, void* q_out,
                                              void* cuda_stream) {
    if (st == nullptr || stats == nullptr || (n != 0 && (dY == nullptr || q_out == nullptr)))
        return LBT_ERR_INVALID_ARG;
    if ((index_offset & 7u) != 0 || index_offset + n < index_offset) return LBT_ERR_INVALID_ARG;
    if (!aligned16(dY) || !aligned16(q_out) || (reinterpret_cast<uintptr_t>(stats) & 7u) ||
        (reinterpret_cast<uintptr_t>(st) & 7u))
        return LBT_ERR_ALIGNMENT;
    return launch_quantize(dY, n, st, stats, static_cast<uint8_t*>(q_out), nullptr, true, as_stream(cuda_stream),
                           index_offset);
}

namespace lbt {

// Philox words parked in shared memory by fused_quantize_kernel: at most 9 groups per thread
// (9 x 256 x 16 bytes = 36 KB per block, four blocks per multiprocessor; more would take the L1 that
// the abs-max phase needs for its loads in flight).
constexpr uint32_t kFusedCacheSlots = 9;
constexpr int kFusedCacheBytes = (int)(kFusedCacheSlots * kStreamThreads * sizeof(uint4));

// Blocks of fused_quantize_kernel that can be resident at once on the current device (0: cooperative
// launches unsupported), looked up once per device.
static int fused_max_blocks() {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static int cached[kMaxDevices];
    static bool known[kMaxDevices];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
    std::lock_guard<std::mutex> lock(mu);
    if (!known[dev]) {
        int coop = 0, sms = 0, per_sm = 0;
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        // sized for the largest cache of Philox words a launch may ask for, so that every launch fits
        if (coop && (cudaFuncSetAttribute(fused_quantize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          kFusedCacheBytes) != cudaSuccess ||
                     cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fused_quantize_kernel, kStreamThreads,
                                                                   kFusedCacheBytes) != cudaSuccess))
            per_sm = 0;
        cached[dev] = coop ? sms * per_sm : 0;
        known[dev] = true;
    }
    return cached[dev];
}

lbt_status launch_fused_quantize(const float* dY, uint64_t n, lbt_interval_state* st, lbt_grad_stats_t* stats,
                                 uint8_t* q_out, uint8_t* q8_out, cudaStream_t stream, bool* launched,
                                 int expect_bits) {
    *launched = false;
    const int most = fused_max_blocks();
    if (most <= 0) return LBT_OK;   // the caller takes the three-launch path
    LBT_CUDA_TRY(cudaMemsetAsync(stats, 0, sizeof(lbt_grad_stats_t), stream));
    const int grid = std::min(stream_grid((n + 7) >> 3), most);
    uint64_t grp_offset = 0;
    const uint64_t ngroups = (n + 7) >> 3, threads = (uint64_t)grid * kStreamThreads;
    uint32_t nslots = (uint32_t)std::min<uint64_t>((ngroups + threads - 1) / threads, kFusedCacheSlots);
    const size_t cache_bytes = (size_t)nslots * kStreamThreads * sizeof(uint4);
    void* args[] = {&dY, &n, &st, &stats, &q_out, &q8_out, &grp_offset, &nslots, &expect_bits};
    timing_begin(LBT_TIME_STATS, stream);   // (one launch: the statistics tap brackets nothing)
    timing_end(LBT_TIME_STATS, stream);
    timing_begin(LBT_TIME_QUANTIZE, stream);
    const cudaError_t err = cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(fused_quantize_kernel), dim3(grid),
                                                        dim3(kStreamThreads), args, cache_bytes, stream);
    timing_end(LBT_TIME_QUANTIZE, stream);
    if (err != cudaSuccess) return LBT_ERR_CUDA;
    *launched = true;
    return LBT_OK;
}

}  // namespace lbt

extern "C" lbt_status lbt_quantize_grad_fused(const float* dY, uint64_t n, lbt_interval_state* st,
                                              lbt_grad_stats_t* stats, void* q_out, void* cuda_stream) {
    if (st == nullptr || stats == nullptr || (n != 0 && (dY == nullptr || q_out == nullptr)))
        return LBT_ERR_INVALID_ARG;
    if (!aligned16(dY) || !aligned16(q_out) || (reinterpret_cast<uintptr_t>(stats) & 7u) ||
        (reinterpret_cast<uintptr_t>(st) & 7u))
        return LBT_ERR_ALIGNMENT;
    bool launched = false;
    lbt_status rc = launch_fused_quantize(dY, n, st, stats, static_cast<uint8_t*>(q_out), nullptr,
                                          as_stream(cuda_stream), &launched);
    if (rc != LBT_OK || launched) return rc;
    // no cooperative launch on this device: the same three steps as separate launches
    rc = lbt_grad_stats(dY, n, st, stats, nullptr, 0, cuda_stream);
    if (rc != LBT_OK) return rc;
    rc = launch_quantize(dY, n, st, stats, static_cast<uint8_t*>(q_out), nullptr, false, as_stream(cuda_stream));
    if (rc != LBT_OK) return rc;
    return lbt_update_interval(st, stats, cuda_stream);
}
