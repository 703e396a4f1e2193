// Diagnostics of Sec. 3.2-3.3 on the device: the quantization error of all gradients E(G) (Eq. 5), of the
// large gradients E(G_L) (Eq. 6, 7), its upper bound U(G_L) (Eq. 8) and the clip-in / clip-out ratios
// (Eq. 9).  G_L is the top alpha fraction by magnitude, found by a radix select over the bit pattern of
// |g| (which orders like |g| itself); among equal magnitudes the earlier elements enter G_L first, which
// needs one in-order pass.  Not part of a training step: a handful of streaming passes over dY.
#include <algorithm>

#include "lbt_common.cuh"

namespace lbt {

constexpr int kDiagThreads = 256;
constexpr int kDiagBuckets = 2048;

struct DiagWork {              // workspace layout (device)
    uint32_t hist[kDiagBuckets];
    uint32_t prefix;           // bits of the threshold's pattern found so far
    uint32_t prefix_mask;
    uint64_t k_remaining;      // rank still to resolve inside the selected bucket
    uint64_t need;             // elements equal to the threshold that belong to G_L
    uint32_t threshold_bits;
    uint32_t pad;
    uint64_t block_ties[1];    // [grid] ties per block, then their exclusive prefix (in place)
};

__device__ __forceinline__ uint32_t abs_bits(float v) { return __float_as_uint(v) & 0x7FFFFFFFu; }

__device__ __forceinline__ int diag_shift(int pass) { return pass == 0 ? 20 : (pass == 1 ? 10 : 0); }
__device__ __forceinline__ uint32_t diag_field(int pass) { return pass == 0 ? 0x7FFu : 0x3FFu; }

__global__ void __launch_bounds__(kDiagThreads)
diag_init_kernel(DiagWork* w, lbt_grad_diag_t* out, uint64_t n, float alpha) {
    for (int i = threadIdx.x; i < kDiagBuckets; i += blockDim.x) w->hist[i] = 0u;
    if (threadIdx.x == 0) {
        const uint64_t n_large = (uint64_t)__double2ll_rn(__dmul_rn((double)alpha, (double)n));   // alpha N, halves to even
        w->prefix = 0u; w->prefix_mask = 0u; w->k_remaining = n_large; w->need = 0; w->threshold_bits = 0x7FFFFFFFu;
        out->n = n; out->n_large = n_large; out->n_in = 0; out->n_out = 0;
        out->sum_all = 0.0; out->sum_large_in = 0.0; out->sum_large_out = 0.0;
        out->e_all = 0.0; out->e_large = 0.0; out->u_large = 0.0; out->threshold = 0.0f; out->reserved = 0u;
    }
}

// Histogram of one field of |g|'s bit pattern over the elements that match the prefix found so far.
__global__ void __launch_bounds__(kDiagThreads)
diag_hist_kernel(const float* __restrict__ g, uint64_t n, int pass, DiagWork* w) {
    __shared__ uint32_t h[kDiagBuckets];
    for (int i = threadIdx.x; i < kDiagBuckets; i += blockDim.x) h[i] = 0u;
    __syncthreads();
    const uint32_t prefix = w->prefix, mask = w->prefix_mask;
    const int shift = diag_shift(pass);
    const uint32_t field = diag_field(pass);
    if (w->k_remaining != 0)
        for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
            const uint32_t a = abs_bits(__ldg(g + i));
            if ((a & mask) == prefix) atomicAdd(&h[(a >> shift) & field], 1u);
        }
    __syncthreads();
    for (int i = threadIdx.x; i < kDiagBuckets; i += blockDim.x)
        if (h[i]) atomicAdd(&w->hist[i], h[i]);
}

// Walk the buckets from the largest magnitude down to the one that holds the k-th largest element.
__global__ void diag_select_kernel(int pass, DiagWork* w) {
    if (threadIdx.x != 0) return;
    const int shift = diag_shift(pass);
    const uint32_t field = diag_field(pass);
    uint64_t k = w->k_remaining;
    if (k != 0) {
        uint64_t seen = 0;
        for (int b = (int)field; b >= 0; --b) {
            const uint64_t c = w->hist[b];
            if (seen + c >= k) {
                w->prefix |= (uint32_t)b << shift;
                w->prefix_mask |= field << shift;
                k -= seen;
                break;
            }
            seen += c;
        }
        w->k_remaining = k;
        if (pass == 2) { w->threshold_bits = w->prefix; w->need = k; }
    }
    for (int i = 0; i < kDiagBuckets; ++i) w->hist[i] = 0u;
}

// Every block owns a contiguous range of groups of eight elements, so that "earlier in memory" is
// (block, step, thread, element) order.
__device__ __forceinline__ void diag_block_range(uint64_t ngroups, uint64_t& lo, uint64_t& hi) {
    const uint64_t per = (ngroups + gridDim.x - 1) / gridDim.x;
    lo = min((uint64_t)blockIdx.x * per, ngroups);
    hi = min(lo + per, ngroups);
}

__global__ void __launch_bounds__(kDiagThreads)
diag_ties_kernel(const float* __restrict__ g, uint64_t n, DiagWork* w) {
    uint64_t lo, hi;
    diag_block_range((n + 7) >> 3, lo, hi);
    const uint32_t t_bits = w->threshold_bits;
    uint32_t ties = 0;
    for (uint64_t grp = lo + threadIdx.x; grp < hi; grp += blockDim.x)
        for (int e = 0; e < 8; ++e) {
            const uint64_t i = (grp << 3) + e;
            if (i < n && abs_bits(__ldg(g + i)) == t_bits) ++ties;
        }
    ties = __reduce_add_sync(0xFFFFFFFFu, ties);
    __shared__ uint32_t s[kDiagThreads / 32];
    if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = ties;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint64_t total = 0;
        for (int i = 0; i < kDiagThreads / 32; ++i) total += s[i];
        w->block_ties[blockIdx.x] = total;
    }
}

__global__ void diag_scan_kernel(DiagWork* w, int blocks) {
    if (threadIdx.x != 0) return;
    uint64_t run = 0;
    for (int b = 0; b < blocks; ++b) { const uint64_t c = w->block_ties[b]; w->block_ties[b] = run; run += c; }
}

__device__ __forceinline__ int diag_code(const uint8_t* __restrict__ q, uint64_t i, bool packed) {
    if (!packed) return (int)(int8_t)q[i];
    const int v = (q[i >> 1] >> (4 * (i & 1))) & 0xF;
    return v >= 8 ? v - 16 : v;
}

__global__ void __launch_bounds__(kDiagThreads)
diag_sums_kernel(const float* __restrict__ g, uint64_t n, const uint8_t* __restrict__ q, int bits,
                 const lbt_grad_stats_t* __restrict__ stats, DiagWork* w, lbt_grad_diag_t* out) {
    uint64_t lo, hi;
    diag_block_range((n + 7) >> 3, lo, hi);
    const uint32_t t_bits = w->threshold_bits;
    const uint64_t need = w->need;
    const bool any_large = out->n_large != 0;
    const float c = stats->c;
    const double s = (double)stats->scale;
    const bool packed = bits <= 4;
    uint64_t tie_base = w->block_ties[blockIdx.x];       // ties in earlier blocks
    __shared__ uint32_t warp_ties[kDiagThreads / 32];
    double sum_all = 0.0, sum_in = 0.0, sum_out = 0.0;
    uint32_t n_in = 0, n_out = 0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (uint64_t base = lo; base < hi; base += blockDim.x) {
        const uint64_t grp = base + threadIdx.x;
        float v[8];
        uint32_t mine = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint64_t i = (grp << 3) + e;
            v[e] = (grp < hi && i < n) ? __ldg(g + i) : 0.0f;
            if (grp < hi && i < n && abs_bits(v[e]) == t_bits) ++mine;
        }
        // ties before this thread's group within the step: warp scan + block scan
        uint32_t incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += up;
        }
        if (lane == 31) warp_ties[warp] = incl;
        __syncthreads();
        uint32_t before = incl - mine, step_total = 0;
        for (int wi = 0; wi < kDiagThreads / 32; ++wi) {
            if (wi < warp) before += warp_ties[wi];
            step_total += warp_ties[wi];
        }
        uint64_t rank = tie_base + before;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const uint64_t i = (grp << 3) + e;
            if (!(grp < hi && i < n)) continue;
            const uint32_t a = abs_bits(v[e]);
            const double err = fabs((double)v[e] - s * (double)diag_code(q, i, packed));
            sum_all += err;
            bool large = any_large && a > t_bits;
            if (any_large && a == t_bits) { large = rank < need; ++rank; }
            if (large) {
                if (fabsf(v[e]) > c) { sum_out += err; ++n_out; } else { sum_in += err; ++n_in; }
            }
        }
        tie_base += step_total;
        __syncthreads();
    }
    // block reduction, then one atomic per block and quantity
    __shared__ double sd[3][kDiagThreads / 32];
    __shared__ uint32_t sc[2][kDiagThreads / 32];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        sum_all += __shfl_xor_sync(0xFFFFFFFFu, sum_all, d);
        sum_in += __shfl_xor_sync(0xFFFFFFFFu, sum_in, d);
        sum_out += __shfl_xor_sync(0xFFFFFFFFu, sum_out, d);
        n_in += __shfl_xor_sync(0xFFFFFFFFu, n_in, d);
        n_out += __shfl_xor_sync(0xFFFFFFFFu, n_out, d);
    }
    if (lane == 0) { sd[0][warp] = sum_all; sd[1][warp] = sum_in; sd[2][warp] = sum_out; sc[0][warp] = n_in; sc[1][warp] = n_out; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0, b = 0, d = 0;
        unsigned long long ci = 0, co = 0;
        for (int i = 0; i < kDiagThreads / 32; ++i) { a += sd[0][i]; b += sd[1][i]; d += sd[2][i]; ci += sc[0][i]; co += sc[1][i]; }
        atomicAdd(&out->sum_all, a); atomicAdd(&out->sum_large_in, b); atomicAdd(&out->sum_large_out, d);
        atomicAdd(reinterpret_cast<unsigned long long*>(&out->n_in), ci);
        atomicAdd(reinterpret_cast<unsigned long long*>(&out->n_out), co);
    }
}

__global__ void diag_final_kernel(const lbt_grad_stats_t* __restrict__ stats, int bits, const DiagWork* w,
                                  lbt_grad_diag_t* out) {
    if (threadIdx.x != 0) return;
    const double g_max = (double)stats->g_max, n = (double)out->n, nl = (double)out->n_large;
    out->threshold = out->n_large ? __uint_as_float(w->threshold_bits) : 0.0f;
    if (!(g_max > 0.0) || out->n == 0) return;
    out->e_all = out->sum_all / (n * g_max);                                              // Eq. (5)
    if (out->n_large == 0) return;
    out->e_large = (out->sum_large_in + out->sum_large_out) / (nl * g_max);               // Eq. (6), (7)
    const double gamma = (double)stats->c / g_max;                                        // the factor in effect
    const double r_in = (double)out->n_in / n, r_out = (double)out->n_out / n;            // Eq. (9)
    out->u_large = ((gamma / (double)((1 << bits) - 2)) * r_in + (1.0 - gamma) * r_out) / (r_in + r_out);   // Eq. (8), (10)
}

static int diag_grid(uint64_t n) {
    const uint64_t blocks = (((n + 7) >> 3) + kDiagThreads - 1) / kDiagThreads;
    return (int)std::max<uint64_t>(1, std::min<uint64_t>(blocks, (uint64_t)kNumSMs * 8));
}

}  // namespace lbt

using namespace lbt;

extern "C" size_t lbt_diagnostics_workspace_bytes(void) {
    return sizeof(DiagWork) + sizeof(uint64_t) * (size_t)kNumSMs * 8 + 256;
}

extern "C" lbt_status lbt_grad_diagnostics(const float* dY, uint64_t n, const void* q_codes, int bits, float alpha,
                                           const lbt_grad_stats_t* stats, lbt_grad_diag_t* out, void* ws,
                                           size_t ws_bytes, void* cuda_stream) {
    if (dY == nullptr || q_codes == nullptr || stats == nullptr || out == nullptr || n == 0) return LBT_ERR_INVALID_ARG;
    if (!(alpha >= 0.0f && alpha <= 1.0f)) return LBT_ERR_INVALID_ARG;
    if (bits < 2 || bits > 8) return LBT_ERR_UNSUPPORTED_BITS;
    if (!aligned16(dY) || (reinterpret_cast<uintptr_t>(out) & 7u) || (reinterpret_cast<uintptr_t>(stats) & 7u))
        return LBT_ERR_ALIGNMENT;
    if (ws == nullptr || ws_bytes < lbt_diagnostics_workspace_bytes()) return LBT_ERR_WORKSPACE;
    DiagWork* w = reinterpret_cast<DiagWork*>((reinterpret_cast<uintptr_t>(ws) + 255) & ~(uintptr_t)255);
    cudaStream_t stream = as_stream(cuda_stream);
    const int grid = diag_grid(n);
    diag_init_kernel<<<1, kDiagThreads, 0, stream>>>(w, out, n, alpha);
    for (int pass = 0; pass < 3; ++pass) {
        diag_hist_kernel<<<grid, kDiagThreads, 0, stream>>>(dY, n, pass, w);
        diag_select_kernel<<<1, 32, 0, stream>>>(pass, w);
    }
    diag_ties_kernel<<<grid, kDiagThreads, 0, stream>>>(dY, n, w);
    diag_scan_kernel<<<1, 32, 0, stream>>>(w, grid);
    diag_sums_kernel<<<grid, kDiagThreads, 0, stream>>>(dY, n, static_cast<const uint8_t*>(q_codes), bits, stats, w, out);
    diag_final_kernel<<<1, 32, 0, stream>>>(stats, bits, w, out);
    return launch_status();
}
