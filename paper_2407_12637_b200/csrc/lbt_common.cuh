// Shared host/device helpers of the CUDA library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "lbt.h"

#define LBT_CUDA_TRY(expr)                                   \
    do {                                                     \
        cudaError_t lbt_err__ = (expr);                      \
        if (lbt_err__ != cudaSuccess) return LBT_ERR_CUDA;   \
    } while (0)

namespace lbt {

constexpr int kNumSMs = 148;  // B200: 2 dies x 74 SMs; grids are sized in multiples of this

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

static inline lbt_status launch_status() {
    return cudaGetLastError() == cudaSuccess ? LBT_OK : LBT_ERR_CUDA;
}

// The quantizer launch behind lbt_quantize_grad.  `q8_out` (optional) additionally receives the codes
// as one int8 per element, which is the layout the contraction kernels read when the layer needs no
// padding; `clear_n_out` = false when the caller has just cleared the statistics.  `index_offset` (a
// multiple of 8) is the position of dY[0] in the whole tensor when dY is one shard of it: the random
// bits of element i are those of element index_offset + i.  `expect_bits` (0 = none): the bit-width the
// host sized q_out and the integer pipeline for; if the device-side state holds another one the codes
// are written as zeros in the layout of `expect_bits` and dev_status becomes LBT_ERR_BITS_MISMATCH.
lbt_status launch_quantize(const float* dY, uint64_t n, const lbt_interval_state* st, lbt_grad_stats_t* stats,
                           uint8_t* q_out, uint8_t* q8_out, bool clear_n_out, cudaStream_t stream,
                           uint64_t index_offset = 0, int expect_bits = 0);

// Statistics + quantize + clipping-factor update as ONE cooperative launch.  *launched = false (and LBT_OK)
// when the device cannot launch cooperatively: the caller then runs the three separate launches.
lbt_status launch_fused_quantize(const float* dY, uint64_t n, lbt_interval_state* st, lbt_grad_stats_t* stats,
                                 uint8_t* q_out, uint8_t* q8_out, cudaStream_t stream, bool* launched,
                                 int expect_bits = 0);

// Optional timing taps (lbt_set_timing_events): record the caller's events around a launch.
void timing_begin(int kernel_class, cudaStream_t stream);
void timing_end(int kernel_class, cudaStream_t stream);
bool timing_armed(int kernel_class);

__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait on a counter in global (or shared) memory that other blocks add to: true once it has
// reached `target`, false when `limit_ns` ran out first (the caller records LBT_ERR_TIMEOUT and goes on).
__device__ __forceinline__ bool counter_wait_bounded(const uint32_t* counter, uint32_t target, uint64_t limit_ns) {
    const volatile uint32_t* c = counter;
    if (*c >= target) return true;
    const uint64_t t0 = global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int spin = 0; spin < 64; ++spin)
            if (*c >= target) return true;
        if (global_timer_ns() - t0 > limit_ns) return false;
    }
}

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).  One 128-bit block per call.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t (&out)[4]) {
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        const uint32_t n0 = hi1 ^ c1 ^ k0;
        const uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The same generator with the ten round keys precomputed (keys[2 r], keys[2 r + 1] = key + r * Weyl
// increments; 16-byte aligned, e.g. in shared memory): saves the key additions per block.
__device__ __forceinline__ void philox4x32_10_keyed(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                    const uint32_t* __restrict__ keys, uint32_t (&out)[4]) {
#pragma unroll
    for (int pair = 0; pair < 5; ++pair) {
        const uint4 k = *reinterpret_cast<const uint4*>(keys + 4 * pair);  // two rounds' keys
        {
            const uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;   // one wide multiply each
            const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
            const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
            const uint32_t n0 = hi1 ^ c1 ^ k.x, n2 = hi0 ^ c3 ^ k.y;
            c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        }
        {
            const uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;   // one wide multiply each
            const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
            const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
            const uint32_t n0 = hi1 ^ c1 ^ k.z, n2 = hi0 ^ c3 ^ k.w;
            c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        }
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

}  // namespace lbt
