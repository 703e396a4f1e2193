// Integer backward contractions dX = Q(dY) Q(W), dW = Q(dY)^T Q(X) on the tcgen05 tensor cores
// (arXiv 2407.12637 motivates integer arithmetic for the backward pass in Sec. 1; the kernel
// design is this library's).
//
// Data flow of one call:
//   1. "expand" kernels turn the stored codes (nibbles or bytes) into int8 tensors laid out on a
//      zero-padded pixel grid: per image Hg x Wg cells, a cell being one pixel's channel vector.
//      Because every image row is followed by zero cells and every image by zero rows, a filter
//      tap (r, s) becomes a CONSTANT offset in the flat cell index, so both convolution
//      contractions become GEMMs whose operands are plain 2-D row windows -- implicit GEMM with
//      nothing but 2-D TMA tiles.  A linear layer is the 1x1 grid.  For stride 2 the input (dgrad:
//      output) pixels are split into the four parity classes, each a stride-1 problem.
//   2. one TMA + tcgen05 kernel (kind::i8, int32 accumulators in TMEM) computes either
//      contraction; warp 0 issues TMA loads, warp 1 issues MMAs, warps 2-5 drain TMEM and apply
//      the dequantising scale.
//   3. wgrad splits its long reduction over CTAs; partial sums are integers, so their order does
//      not matter and the result is bit-exact.
#include <cuda.h>

#include <algorithm>
#include <cstddef>
#include <mutex>

#include "lbt_common.cuh"
#include "lbt_sm100.cuh"

namespace lbt {

using namespace sm100;

constexpr int kTile = 128;               // rows / bytes per TMA box and MMA M
constexpr int kTileBytes = kTile * 128;  // one 128 x 128-byte operand tile
constexpr int kStages = 4;
constexpr int kStageBytes = 3 * kTileBytes;  // A + up to two B boxes
constexpr int kPairStages = 6;               // CTA-pair kernel: A + one B box per CTA and stage
constexpr int kPairStageBytes = 2 * kTileBytes;
static_assert(kPairStages * kPairStageBytes == kStages * kStageBytes, "both kernels use the same operand ring");
constexpr int kMaxBStages = 8;               // CTA-pair kernel, window mode: B ring of one-box stages beside the two A windows
constexpr int kGemmThreads = 320;               // TMA warp, MMA warp, 8 epilogue warps
constexpr int kEpiWarps = 8;
constexpr int kShortMainLoop = 40;  // reduction steps (128 deep) per tile up to which 8 epilogue warps are used
constexpr int kTmemCols = 512;                    // two accumulator buffers of 256 columns
constexpr int kMaxTaps = 64;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // every on-chip wait gives up after 2 s
constexpr uint64_t kFusedQuantizeBytes = 112ull << 20;  // gradient tensors up to this size take the one-launch quantizer

// ------------------------------------------------------------------------------------------
// Geometry of the padded cell grid (host).
// ------------------------------------------------------------------------------------------
struct Geometry {
    int N, C, H, W, K, R, S, st, pad, P, Q;
    int Hg, Wg;      // cells per image column / row
    int64_t rows;    // N * Hg * Wg cells
    int Kp, Cp;      // channel counts rounded up to 16 (TMA row pitch)
    int ncls;        // st * st parity classes
};

static inline int floordiv(int a, int b) { return (a >= 0) ? a / b : -((-a + b - 1) / b); }
static inline int posmod(int a, int b) { return a - floordiv(a, b) * b; }
static inline int round_up(int a, int b) { return (a + b - 1) / b * b; }

static lbt_status make_geometry(const lbt_conv_desc* d, Geometry* g) {
    if (d == nullptr) return LBT_ERR_INVALID_ARG;
    if (d->N <= 0 || d->C <= 0 || d->H <= 0 || d->W <= 0 || d->K <= 0 || d->R <= 0 || d->S <= 0 ||
        d->stride <= 0 || d->pad < 0)
        return LBT_ERR_INVALID_ARG;
    if (d->stride > 2 || d->R * d->S > kMaxTaps) return LBT_ERR_UNSUPPORTED;
    if (d->H + 2 * d->pad < d->R || d->W + 2 * d->pad < d->S) return LBT_ERR_INVALID_ARG;
    g->N = d->N; g->C = d->C; g->H = d->H; g->W = d->W; g->K = d->K; g->R = d->R; g->S = d->S;
    g->st = d->stride; g->pad = d->pad;
    g->P = (d->H + 2 * d->pad - d->R) / d->stride + 1;
    g->Q = (d->W + 2 * d->pad - d->S) / d->stride + 1;
    // vertical / horizontal reach of the taps in cells, for dgrad and wgrad together
    auto halo = [&](int taps) {
        int lo = 0, hi = 0;
        for (int r = 0; r < taps; ++r) {
            const int dw = floordiv(r - g->pad, g->st);                   // wgrad offset of tap r
            lo = std::min(lo, dw); hi = std::max(hi, dw);
            for (int ph = 0; ph < g->st; ++ph)
                if (posmod(ph + g->pad - r, g->st) == 0) {                // dgrad offset of tap r
                    const int dd = (ph + g->pad - r) / g->st;
                    lo = std::min(lo, dd); hi = std::max(hi, dd);
                }
        }
        return std::max(-lo, hi);
    };
    const int Hc = (g->H + g->st - 1) / g->st, Wc = (g->W + g->st - 1) / g->st;
    g->Hg = std::max(g->P, Hc) + halo(g->R);
    g->Wg = std::max(g->Q, Wc) + halo(g->S);
    g->rows = (int64_t)g->N * g->Hg * g->Wg;
    // cell and pixel indices are 32-bit in the kernels (TMA coordinates, epilogue row slots)
    if (g->rows >= (int64_t)1 << 31 || (int64_t)g->N * g->H * g->W >= (int64_t)1 << 31 ||
        (int64_t)g->K * g->R * g->S >= (int64_t)1 << 31)
        return LBT_ERR_UNSUPPORTED;
    g->Kp = round_up(g->K, 16);
    g->Cp = round_up(g->C, 16);
    g->ncls = g->st * g->st;
    return LBT_OK;
}

struct Workspace {
    size_t off_dy, off_wt, off_x, off_status, off_part;
    size_t total_nowgrad;   // everything dgrad and the forward product need
    size_t total;           // plus the partial sums of a split wgrad reduction
};

// How wgrad spreads its long reduction: output tiles x `splits` slices of the reduction, one work
// unit per CTA (pair): a single round measured as fast as or faster than two or more shorter ones
// and needs half the slabs.  Every slice writes its int32 partial tile to its own slab of
// the workspace; a second kernel adds the slabs (integer sums: exact in any order).
struct WgradPlan {
    bool pair;
    int bn, n_ctile, tile_rows, units, m_tiles, tiles, kb_total, splits, kb_per_split;
    int n_groups;   // > 0: multi-tap tiles (see WgradGroups)
};

// wgrad taps in the order the kernel walks them, and their grouping for multi-tap tiles: the taps of a
// group read the same parity class of X at row offsets no more than 128 apart, so ONE 256-row window of
// X per reduction step serves them all, each tap accumulating into its own TMEM columns.
struct WgradGroups {
    int n_taps, n_groups, acc_cols;
    int shift[kMaxTaps];               // absolute flat-cell offset of the tap
    short cls[kMaxTaps], rs[kMaxTaps]; // parity class of X; r * S + s
    short first[kMaxTaps], count[kMaxTaps];
    int min_shift[kMaxTaps];           // per group
};

static void wgrad_taps(const Geometry& g, WgradGroups* w) {
    w->n_taps = g.R * g.S;
    for (int r = 0; r < g.R; ++r)
        for (int s = 0; s < g.S; ++s) {
            const int t = r * g.S + s;
            w->shift[t] = floordiv(r - g.pad, g.st) * g.Wg + floordiv(s - g.pad, g.st);
            w->cls[t] = (short)(posmod(r - g.pad, g.st) * g.st + posmod(s - g.pad, g.st));
            w->rs[t] = (short)t;
        }
    w->n_groups = 0;
    w->acc_cols = 0;
}

// Multi-tap grouping for the single-CTA kernel with one 128-byte box of X channels per row.
static void wgrad_group(const Geometry& g, WgradGroups* w) {
    wgrad_taps(g, w);
    if (g.Cp > 128 || g.Kp > 128 || w->n_taps < 2) return;
    // order by (class, offset)
    for (int i = 1; i < w->n_taps; ++i)
        for (int j = i; j > 0; --j) {
            const bool before = w->cls[j] < w->cls[j - 1] || (w->cls[j] == w->cls[j - 1] && w->shift[j] < w->shift[j - 1]);
            if (!before) break;
            std::swap(w->shift[j], w->shift[j - 1]); std::swap(w->cls[j], w->cls[j - 1]); std::swap(w->rs[j], w->rs[j - 1]);
        }
    w->acc_cols = (g.Cp + 31) / 32 * 32;
    const int most = std::min(512 / w->acc_cols, 16);
    int ng = 0, cap = most, run_end = 0;
    for (int t = 0; t < w->n_taps;) {
        if (t >= run_end) {   // a new parity class: spread its taps evenly over as few groups as possible
            run_end = t + 1;
            while (run_end < w->n_taps && w->cls[run_end] == w->cls[t]) ++run_end;
            const int len = run_end - t, groups = (len + most - 1) / most;
            cap = (len + groups - 1) / groups;
        }
        int e = t + 1;
        while (e < run_end && e - t < cap && w->shift[e] - w->shift[t] <= 128) ++e;
        w->first[ng] = (short)t; w->count[ng] = (short)(e - t); w->min_shift[ng] = w->shift[t];
        ++ng;
        t = e;
    }
    // groups of unequal size make tiles of unequal cost; with too much imbalance one tile per tap is better
    int largest = 0;
    for (int i = 0; i < ng; ++i) largest = std::max(largest, (int)w->count[i]);
    w->n_groups = 10 * w->n_taps >= 7 * largest * ng ? ng : 0;
}

static WgradPlan plan_wgrad(const Geometry& g, int sms) {
    WgradPlan p;
    p.bn = g.Cp <= 128 ? 128 : 256;
    p.n_ctile = (g.Cp + p.bn - 1) / p.bn;
    p.kb_total = (int)((g.rows + 127) / 128);
    // CTA pairs when both tile dimensions exceed 128 (dY channels and X channels)
    p.pair = p.bn == 256 && g.Kp > 128 && sms >= 2;
    p.tile_rows = p.pair ? 256 : 128;
    p.units = p.pair ? sms / 2 : sms;   // tiles in flight at once
    p.m_tiles = (g.Kp + p.tile_rows - 1) / p.tile_rows;
    WgradGroups grp;
    wgrad_group(g, &grp);
    p.n_groups = p.pair ? 0 : grp.n_groups;
    p.tiles = p.m_tiles * (p.n_groups > 0 ? p.n_groups : g.R * g.S) * p.n_ctile;
    int splits = std::max(1, std::min(p.kb_total, p.units / std::max(p.tiles, 1)));
    p.kb_per_split = (p.kb_total + splits - 1) / splits;
    p.splits = (p.kb_total + p.kb_per_split - 1) / p.kb_per_split;
    return p;
}

static inline int64_t part_stride(const Geometry& g) {   // elements per slab, a multiple of 8 (slabs stay 32-byte aligned)
    return (((int64_t)g.K * g.R * g.S * g.C) + 7) & ~(int64_t)7;
}

static inline bool aligned32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }


static Workspace carve(const Geometry& g) {
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    Workspace w;
    size_t o = 256;  // slack to align the caller's pointer
    w.off_dy = o; o += up((size_t)g.rows * g.Kp);
    w.off_wt = o; o += up((size_t)g.R * g.S * g.K * g.Cp);
    w.off_x = o; o += up((size_t)g.ncls * g.rows * g.Cp);
    w.off_status = o; o += 256;
    w.total_nowgrad = o;
    // sized for the full SM count; fewer SMs mean fewer slices
    const WgradPlan p = plan_wgrad(g, kNumSMs);
    w.off_part = o; o += p.splits > 1 ? up((size_t)p.splits * part_stride(g) * sizeof(int32_t)) : 0;
    w.total = o;
    return w;
}

// ------------------------------------------------------------------------------------------
// Expand: stored codes -> int8 on the padded cell grid.  One thread per 16 output bytes.
// ------------------------------------------------------------------------------------------
// Division of a 32-bit dividend by a fixed divisor as multiply-high + shift (Granlund-Montgomery
// round-up method, exact for every dividend below 2^31); the host prepares it once per launch.
struct FastDiv {
    uint32_t mul, shift, div;
};

static FastDiv make_fastdiv(uint32_t d) {
    FastDiv f;
    f.div = d;
    f.mul = 0;
    f.shift = 0;
    if (d <= 1) return f;
    uint32_t l = 0;
    while ((1ull << l) < d) ++l;                           // l = ceil(log2 d) >= 1
    // m = ceil(2^(31+l) / d) < 2^32 because d > 2^(l-1);  n / d = (n * m) >> (31 + l) for every n < 2^31
    f.mul = (uint32_t)(((1ull << (31 + l)) + d - 1) / d);
    f.shift = l - 1;                                       // after taking the high 32 bits of n * m
    return f;
}

__device__ __forceinline__ uint32_t fast_div(uint32_t n, const FastDiv& f) {
    return f.div <= 1 ? n : (__umulhi(n, f.mul) >> f.shift);
}

struct ExpandArgs {
    const uint8_t* src;
    uint8_t* dst;
    int mode;        // 0: dY -> grid; 1: W[k][r][s][c] -> tap-major [r*S+s][k][c]; 2: X -> parity classes
    int packed;      // 1: two 4-bit codes per byte; 0: one byte per code
    int is_signed;
    int identity;    // destination vector v holds source codes [16 v, 16 v + 16): no padding, no reorder
    int wait_prev;   // 1: the source is written by the kernel this launch is chained behind: wait for that grid first
    int Cs;          // channels per source pixel
    int chunks;      // 16-byte chunks per destination row
    int rows_per_block;
    int64_t rows_total;
    int64_t rows_per_cls;
    int Hg, Wg, Hs, Ws, st, RS, K;
    FastDiv by_chunks, by_cells, by_wg, by_k;
};

__device__ __forceinline__ uint32_t nibbles_to_bytes(uint32_t w, bool is_signed, uint32_t& hi_out) {
    uint32_t e = w & 0x0F0F0F0Fu, o = (w >> 4) & 0x0F0F0F0Fu;  // even / odd elements
    if (is_signed) {
        // sign extension of each nibble without a per-byte subtract: (n ^ 8) + 0x78 stays inside its byte, and
        // flipping that byte's top bit leaves (n ^ 8) - 8 as a two's-complement byte
        e = ((e ^ 0x08080808u) + 0x78787878u) ^ 0x80808080u;
        o = ((o ^ 0x08080808u) + 0x78787878u) ^ 0x80808080u;
    }
    hi_out = __byte_perm(e, o, 0x7362);  // elements 4..7
    return __byte_perm(e, o, 0x5140);    // elements 0..3
}

__device__ __forceinline__ uint32_t load_code(const uint8_t* src, int64_t e, bool packed, bool is_signed) {
    if (!packed) return src[e];
    uint32_t v = (src[e >> 1] >> (4 * (e & 1))) & 0xFu;
    if (is_signed && v >= 8u) v |= 0xF0u;
    return v;
}

// One block handles `rows_per_block` consecutive destination rows; thread t takes the 16-byte chunks
// t, t + 256, ... of that block.  Everything below the block's first row is 32-bit arithmetic: the
// destination vector of chunk `local` is simply (first vector of the block) + local, rows and pixels
// count below 2^31, and only the final byte offsets are 64-bit.
struct ExpandBlock {
    uint32_t j0;        // image-relative (class-relative) index of the block's first row
    uint32_t to_next;   // rows from the block's first row to the start of the next parity class
    int ph0, pw0, ph1, pw1;   // pixel parities (h, w) of the class the block starts in and of the next one
    uint32_t row0, rows_left; // mode 1: first row; all modes: rows that exist from the block's first row on
};

// Source element of the chunk `local` of a block (-1: the chunk is zeros); false past the last row.
__device__ __forceinline__ bool expand_locate(const ExpandArgs& a, const ExpandBlock& eb, uint32_t local, int64_t* src_elem) {
    const uint32_t r_local = fast_div(local, a.by_chunks);
    const uint32_t chunk = local - r_local * (uint32_t)a.chunks;
    if (r_local >= eb.rows_left) return false;
    int32_t pixel = -1;
    if (a.mode == 1) {
        const uint32_t row = eb.row0 + r_local;
        const uint32_t tap = fast_div(row, a.by_k), k = row - tap * (uint32_t)a.K;
        pixel = (int32_t)(k * (uint32_t)a.RS + tap);
    } else {
        const bool next = r_local >= eb.to_next;                 // a block spans less than one class
        const uint32_t j = next ? r_local - eb.to_next : eb.j0 + r_local;
        const uint32_t n = fast_div(j, a.by_cells);
        const uint32_t cell = j - n * (uint32_t)(a.Hg * a.Wg);
        const uint32_t ca = fast_div(cell, a.by_wg), cb = cell - ca * (uint32_t)a.Wg;
        int h = (int)ca, w = (int)cb;
        if (a.mode == 2) {
            h = a.st * h + (next ? eb.ph1 : eb.ph0);
            w = a.st * w + (next ? eb.pw1 : eb.pw0);
        }
        if (h < a.Hs && w < a.Ws) pixel = (int32_t)((n * (uint32_t)a.Hs + (uint32_t)h) * (uint32_t)a.Ws + (uint32_t)w);
    }
    const uint32_t c0 = chunk * 16u;
    *src_elem = (pixel >= 0 && c0 < (uint32_t)a.Cs) ? (int64_t)pixel * a.Cs + c0 : -1;
    return true;
}

__device__ __forceinline__ void expand_body(const ExpandArgs& a, int block, int blocks) {
    const uint32_t per_block = (uint32_t)a.rows_per_block * (uint32_t)a.chunks;
    constexpr int kInFlight = 4;   // chunks a thread has in flight
    for (int64_t blk = block; blk * a.rows_per_block < a.rows_total; blk += blocks) {
        const int64_t row0 = blk * a.rows_per_block;
        ExpandBlock eb;
        {
            // the parity class and class-relative position of the block's first row
            int cls0 = 0;
            int64_t j0 = row0;
            while (a.mode == 2 && j0 >= a.rows_per_cls) { j0 -= a.rows_per_cls; ++cls0; }
            eb.j0 = (uint32_t)j0;
            eb.to_next = a.mode == 2 ? (uint32_t)(a.rows_per_cls - j0) : 0xFFFFFFFFu;
            eb.ph0 = cls0 / a.st; eb.pw0 = cls0 % a.st;
            eb.ph1 = (cls0 + 1) / a.st; eb.pw1 = (cls0 + 1) % a.st;
            eb.row0 = (uint32_t)row0;
            eb.rows_left = (uint32_t)min((int64_t)a.rows_per_block, a.rows_total - row0);
        }
        uint4* __restrict__ dst = reinterpret_cast<uint4*>(a.dst) + row0 * a.chunks;
        if ((a.Cs & 15) == 0) {
            // whole chunks: all loads of a step are issued before the first store
            for (uint32_t local = threadIdx.x; local < per_block; local += 256 * kInFlight) {
                bool live[kInFlight];
                uint4 v[kInFlight];
#pragma unroll
                for (int u = 0; u < kInFlight; ++u) {
                    int64_t e0 = -1;
                    v[u] = make_uint4(0, 0, 0, 0);
                    const uint32_t l = local + 256u * u;
                    live[u] = l < per_block && expand_locate(a, eb, l, &e0);
                    if (e0 >= 0) {
                        if (a.packed) {
                            const uint2 w = __ldg(reinterpret_cast<const uint2*>(a.src + (e0 >> 1)));
                            v[u].x = w.x; v[u].y = w.y;
                        } else {
                            v[u] = __ldg(reinterpret_cast<const uint4*>(a.src + e0));
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < kInFlight; ++u) {
                    if (!live[u]) continue;
                    uint4 out = v[u];
                    if (a.packed) {   // zeros stay zeros
                        const uint32_t w0 = v[u].x, w1 = v[u].y;
                        out.x = nibbles_to_bytes(w0, a.is_signed, out.y);
                        out.z = nibbles_to_bytes(w1, a.is_signed, out.w);
                    }
                    dst[local + 256u * u] = out;
                }
            }
            continue;
        }
        for (uint32_t local = threadIdx.x; local < per_block; local += 256) {
            int64_t e0;
            if (!expand_locate(a, eb, local, &e0)) break;
            uint4 out = make_uint4(0, 0, 0, 0);
            if (e0 >= 0) {
                const int c0 = (int)(local - fast_div(local, a.by_chunks) * (uint32_t)a.chunks) * 16;
                uint32_t b[16];
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    b[i] = (c0 + i < a.Cs) ? (load_code(a.src, e0 + i, a.packed, a.is_signed) & 0xFFu) : 0u;
                out.x = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
                out.y = b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24);
                out.z = b[8] | (b[9] << 8) | (b[10] << 16) | (b[11] << 24);
                out.w = b[12] | (b[13] << 8) | (b[14] << 16) | (b[15] << 24);
            }
            dst[local] = out;
        }
    }
}

// No padding and no reordering (linear layers, 1x1 stride-1 convolutions with channel counts that are
// multiples of 16): a straight stream, 32 codes per thread and step.
__device__ __forceinline__ void expand_identity_body(const ExpandArgs& a, int block, int blocks) {
    const int64_t total = a.rows_total * a.chunks;   // 16-byte destination vectors
    const int64_t pairs = total >> 1;
    const int64_t stride = (int64_t)blocks * blockDim.x;
    int64_t p = (int64_t)block * blockDim.x + threadIdx.x;
    if (a.packed) {
        // four 16-byte loads of a thread in flight before the first store
        for (; p + 3 * stride < pairs; p += 4 * stride) {
            uint4 w[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) w[u] = __ldg(reinterpret_cast<const uint4*>(a.src) + p + u * stride);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                uint4 lo, hi;
                lo.x = nibbles_to_bytes(w[u].x, a.is_signed, lo.y);
                lo.z = nibbles_to_bytes(w[u].y, a.is_signed, lo.w);
                hi.x = nibbles_to_bytes(w[u].z, a.is_signed, hi.y);
                hi.z = nibbles_to_bytes(w[u].w, a.is_signed, hi.w);
                const uint32_t w8[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
                st_global_v8(reinterpret_cast<uint4*>(a.dst) + 2 * (p + u * stride), w8);   // one 32-byte sector
            }
        }
    }
    for (; p < pairs; p += stride) {
        uint4 lo, hi;
        if (a.packed) {
            const uint4 w = __ldg(reinterpret_cast<const uint4*>(a.src) + p);
            lo.x = nibbles_to_bytes(w.x, a.is_signed, lo.y);
            lo.z = nibbles_to_bytes(w.y, a.is_signed, lo.w);
            hi.x = nibbles_to_bytes(w.z, a.is_signed, hi.y);
            hi.z = nibbles_to_bytes(w.w, a.is_signed, hi.w);
        } else {
            lo = __ldg(reinterpret_cast<const uint4*>(a.src) + 2 * p);
            hi = __ldg(reinterpret_cast<const uint4*>(a.src) + 2 * p + 1);
        }
        reinterpret_cast<uint4*>(a.dst)[2 * p] = lo;
        reinterpret_cast<uint4*>(a.dst)[2 * p + 1] = hi;
    }
    if ((total & 1) && block == 0 && threadIdx.x == 0) {   // odd tail vector
        const int64_t v = total - 1;
        uint4 out;
        if (a.packed) {
            const uint2 w = __ldg(reinterpret_cast<const uint2*>(a.src) + v);
            out.x = nibbles_to_bytes(w.x, a.is_signed, out.y);
            out.z = nibbles_to_bytes(w.y, a.is_signed, out.w);
        } else {
            out = __ldg(reinterpret_cast<const uint4*>(a.src) + v);
        }
        reinterpret_cast<uint4*>(a.dst)[v] = out;
    }
}

// Up to three expansions (dY, W, X of one layer) in ONE launch: consecutive block ranges, one per job.
struct ExpandJobs {
    ExpandArgs job[3];
    int first_block[4];   // job i owns blocks [first_block[i], first_block[i + 1])
    int n;
    int chained;          // launched programmatically behind the kernel that writes one job's source
};

__global__ void __launch_bounds__(256) expand_batch_kernel(const __grid_constant__ ExpandJobs jobs) {
    griddep_launch_dependents();   // the contraction behind it may set up early; it waits for this grid before loading
    int j = 0;
    while (j + 1 < jobs.n && (int)blockIdx.x >= jobs.first_block[j + 1]) ++j;
    const int block = (int)blockIdx.x - jobs.first_block[j], blocks = jobs.first_block[j + 1] - jobs.first_block[j];
    // Chained behind the quantizer (jobs.chained): only the job that reads its codes waits for it before
    // working; block 0 waits before it ends, so that this grid never completes before the quantizer has.
    if (jobs.job[j].wait_prev) griddep_wait();
    // one copy of the body per job slot: the job's fields are then read as kernel-parameter operands
    // instead of through an index computed at run time
#define LBT_EXPAND_JOB(J) \
    { if (jobs.job[J].identity) expand_identity_body(jobs.job[J], block, blocks); else expand_body(jobs.job[J], block, blocks); }
    if (j == 0) LBT_EXPAND_JOB(0) else if (j == 1) LBT_EXPAND_JOB(1) else LBT_EXPAND_JOB(2)
#undef LBT_EXPAND_JOB
    if (jobs.chained && blockIdx.x == 0) griddep_wait();
}

// Very few input channels (a network's first layer: C = 3): a cell of 16 channel bytes would be mostly
// padding and every tap a separate, nearly empty operand tile.  Instead the patches are written out
// explicitly -- row (n, p, q) holds X[n, p st + r - pad, q st + s - pad, c] for all (r, s, c), zero outside
// the image, padded to a multiple of 16 bytes -- and the convolution becomes a linear layer with
// I = R S C inputs (forward and wgrad; dW[k][r][s][c] is that layer's [O][I] weight gradient as it stands).
struct Im2colArgs {
    const uint8_t* src;
    uint8_t* dst;
    int packed;
    int C, H, W, S, st, pad, P, Q;
    int cols;      // R * S * C
    int chunks;    // 16-byte chunks per row
    int64_t total; // rows * chunks
    FastDiv by_chunks, by_pq, by_q, by_sc, by_c;
};

__global__ void __launch_bounds__(256) im2col_kernel(const Im2colArgs a) {
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < a.total; idx += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t row = fast_div((uint32_t)idx, a.by_chunks), chunk = (uint32_t)idx - row * (uint32_t)a.chunks;
        const uint32_t n = fast_div(row, a.by_pq), rem = row - n * (uint32_t)(a.P * a.Q);
        const uint32_t p = fast_div(rem, a.by_q), q = rem - p * (uint32_t)a.Q;
        uint32_t b[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t col = chunk * 16u + (uint32_t)i;
            uint32_t v = 0u;
            if (col < (uint32_t)a.cols) {
                const uint32_t r = fast_div(col, a.by_sc), rem2 = col - r * (uint32_t)(a.S * a.C);
                const uint32_t s = fast_div(rem2, a.by_c), c = rem2 - s * (uint32_t)a.C;
                const int h = (int)p * a.st + (int)r - a.pad, w = (int)q * a.st + (int)s - a.pad;
                if (h >= 0 && h < a.H && w >= 0 && w < a.W)
                    v = load_code(a.src, (((int64_t)n * a.H + h) * a.W + w) * a.C + c, a.packed != 0, false) & 0xFFu;
            }
            b[i] = v;
        }
        uint4 out;
        out.x = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
        out.y = b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24);
        out.z = b[8] | (b[9] << 8) | (b[10] << 16) | (b[11] << 24);
        out.w = b[12] | (b[13] << 8) | (b[14] << 16) | (b[15] << 24);
        reinterpret_cast<uint4*>(a.dst)[idx] = out;
    }
}

// ------------------------------------------------------------------------------------------
// The contraction kernel.
// ------------------------------------------------------------------------------------------
struct GemmArgs {
    int mode;          // 0 dgrad: A = dY grid (K-major), B = tap-major W (MN-major)
                       // 1 wgrad: A = dY grid (MN-major), B = X class grid (MN-major)
                       // 2 forward: A = X class grid (K-major, the kernels' tmB0..3), B = W as [K][taps * Cp]
                       //            (K-major, the kernels' tmA); output rows are the cells of the Y grid
    int bn;            // MMA N: 128 or 256
    int b_boxes;       // 128-byte-wide B boxes per stage (bn / 128)
    int n_ctile;       // channel tiles of the output
    int m_tiles;       // 128-row tiles of the output
    int ny;            // dgrad: n_ctile; wgrad: taps * n_ctile
    int band;          // row tiles per band of the tile walk (>= 1)
    int mma_n;         // single-CTA kernel: MMA N actually issued (<= bn, multiple of 16): output columns in use
    int k_last;        // dgrad: valid reduction bytes in the last 128-byte chunk of a tap (32..128, multiple of 16)
    int total_tiles;   // m_tiles * ny * (dgrad: parity classes; wgrad: splits), plus the extra units of split tiles
    int split_n;       // CTA-pair kernel, dgrad / forward: > 1 = the tiles from index split_from on (those of a last, nearly
    int split_from;    //   empty round) are cut into split_n column slices, one unit each, so that all pairs share them
    int kc_per_tap;    // dgrad: 128-byte chunks of the reduction per tap
    int K;             // channels of dY
    int C;             // channels of X / dX
    int RS;            // taps of the filter
    int kb_total;      // wgrad: 128-row blocks of the reduction
    int kb_per_split;  // wgrad
    int direct;        // 1: epilogue writes fp32 (and int32) results; 2: writes the int32 partial sums of its
                       //    reduction slice to slab `slice` of `acc` (slabs are part_stride elements apart)
    int64_t part_stride;
    int epi_warps;     // 4 or 8 epilogue warps at work: 8 drain a tile in half the time, which pays when the
                       // main loop of a tile is short; with long main loops the extra traffic only disturbs it
    int multi;         // wgrad, single-CTA kernel: 1 = a tile covers a GROUP of taps (see WgradGroups); the B part of a
                       // stage is one 256-row window of X, every tap has its own accumulator of acc_cols columns
    int acc_cols;
    int row_direct;    // 1: the epilogue stores each row's 32 columns straight from registers as four 32-byte stores
                       // (rows of the output are 32-byte aligned: C a multiple of 8, 32-byte aligned buffers)
    int tma_store;     // 1: output rows are the tile rows themselves (no halo, no tap interleave), so the epilogue hands
                       // each staged 32 x 32 block to a TMA store instead of reading it back and storing it
    // Programmatic dependent launches (all 0 when a timing tap is armed: an event record between two launches
    // serialises them anyway).
    int wait_prev;     // 1: launched early behind the kernel that writes its operands: wait for that grid after set-up
    int overlap_next;  // 1: let the next launch in the stream be scheduled once every CTA here is past its set-up (and
                       // its wait): that launch either waits for this grid itself or does not depend on it
    int overlap_prev;  // 1: launched behind a grid it does not depend on: this grid does not END before that one has,
                       // so whatever follows in the stream still finds both complete
    int epi_alt;       // single-CTA kernel with 8 epilogue warps: 1 = warps 2-5 drain the tiles of accumulator
                       // buffer 0 and warps 6-9 those of buffer 1 (two tiles drain at once, each warp all the
                       // columns of its rows) instead of all eight sharing every tile
    int a_signed, b_signed;
    int tap_cols;      // forward: columns of W per tap (channels of X rounded up to 16)
    int window;        // dgrad, stride 1, single-CTA kernel: the taps of a tile read overlapping row windows of
                       // dY, so one window of 128 + (largest - smallest tap offset) rows is loaded per
                       // reduction chunk and every tap's A operand is a row offset into it
    int win_boxes;     // 128-row boxes per window
    int win_min_shift; // smallest tap offset
    int n_bstages;     // B ring stages beside the windows
    int n_win;         // A windows: 2 (double-buffered), or 1 in the single-CTA kernel when the resident filter leaves
                       // room for only one
    int w_boxes;       // window mode with small filters: > 0 = all of the tap-major W (this many 128-row boxes per
                       // 128 output channels) is loaded once per CTA and stays in shared memory
    int Hg, Wg, H, W, st;
    int64_t rows;
    const float* scale_a;
    const float* scale_b;
    float* out;
    int32_t* acc;
    int32_t* status;
    FastDiv by_mtiles, by_cells, by_wg;   // divisions by m_tiles, Hg * Wg and Wg as multiply-shift (set by finish_args)
    lbt_grad_stats_t* dx_stats;  // dgrad, optional: receives max |dX|, the non-finite count and the element count of dX
    uint64_t dx_n;               // elements of dX
    int cls_begin[5];          // dgrad: taps of parity class c are [cls_begin[c], cls_begin[c+1])
    int tap_shift[kMaxTaps];   // flat-cell offset of the tap (dgrad: into A; wgrad: into B)
    short tap_aux[kMaxTaps];   // dgrad: r*S+s (slab of W); wgrad: parity class of X
    short tap_rs[kMaxTaps];    // wgrad: r*S+s (where the tap lands in dW)
    short grp_first[kMaxTaps]; // multi-tap wgrad: the taps of group i are [grp_first[i], grp_first[i] + grp_count[i]);
    short grp_count[kMaxTaps]; //   tap_shift then holds the tap's row offset inside its group's window and
    int grp_min_shift[kMaxTaps]; // grp_min_shift the flat-cell offset of the window's first row
};

// Staging rows are 32 words; 16-byte chunk c of row r sits at chunk position c ^ (r & 7), which keeps
// both the row-wise writes and the row-segment reads free of bank conflicts without padding.
struct alignas(16) GemmShared {
    alignas(16) uint32_t stage[kEpiWarps][32 * 32];  // per epilogue warp: 32 rows x 32 columns in transit
    int32_t row_slot[kEpiWarps][32];                 // per epilogue warp: output pixel / filter-tap slot of each
                                                     // row (times C = element offset), -1 = skip
    uint64_t full[kMaxBStages];
    uint64_t empty[kMaxBStages];
    uint64_t a_full[2];      // window mode: the two A windows
    uint64_t a_empty[2];
    uint2 tap_off[kMaxTaps]; // window mode, per tap, in 16-byte units as the descriptors count: x = offset of the
                             // tap's rows in the A window, y = offset of its reduction rows in the resident filter
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    volatile uint32_t abort;
};
constexpr int kGemmSmemBytes = kStages * kStageBytes + 1024 + (int)sizeof(GemmShared);
static_assert(kGemmSmemBytes <= 232448, "exceeds the 227 KB of shared memory a CTA may use");

struct TileInfo {
    int m0, c0, cls, tapi, tap_lo, kb_lo, num_iters;
    int width;   // output columns of this unit: bn, or bn / split_n for a column slice of a left-over tile
};

__device__ __forceinline__ TileInfo decode_tile(const GemmArgs& g, int t, int tile_rows = kTile) {
    TileInfo ti;
    int slice = 0;
    ti.width = g.bn;
    if (g.split_n > 1 && t >= g.split_from) {
        const int u = t - g.split_from;
        t = g.split_from + u / g.split_n;
        slice = u - (u / g.split_n) * g.split_n;
        ti.width = g.bn / g.split_n;
    }
    if (g.mode != 1 && g.total_tiles == g.m_tiles) {
        // one column tile, one class, nothing split: tile t is row tile t (no divisions on the one thread that issues the MMAs)
        ti.m0 = t * tile_rows; ti.c0 = 0;
        ti.cls = 0; ti.tapi = 0; ti.tap_lo = 0; ti.kb_lo = 0;
        ti.num_iters = g.cls_begin[1] * g.kc_per_tap;
        return ti;
    }
    if (g.mode != 1 && g.ny == 1 && g.split_n <= 1) {
        // one column tile per class: class z = t / m_tiles, row tile t % m_tiles
        const int z = (int)fast_div((uint32_t)t, g.by_mtiles);
        ti.m0 = (t - z * g.m_tiles) * tile_rows; ti.c0 = 0;
        ti.cls = z; ti.tapi = 0; ti.kb_lo = 0;
        ti.tap_lo = g.cls_begin[z];
        ti.num_iters = (g.cls_begin[z + 1] - ti.tap_lo) * g.kc_per_tap;
        return ti;
    }
    // Tiles are walked band by band: `band` row tiles x all column tiles, rows fastest.  The CTAs at
    // work at any moment then share a few row strips of A and a few column strips of B that fit in
    // L2 together, instead of sweeping all of A for every column strip.
    const int slab = g.m_tiles * g.ny;
    const int z = t / slab, idx = t - z * slab;
    const int per_band = g.band * g.ny;
    const int band_i = idx / per_band, within = idx - band_i * per_band;
    const int band_rows = min(g.band, g.m_tiles - band_i * g.band);
    const int y = within / band_rows;
    const int m = band_i * g.band + (within - y * band_rows);
    ti.m0 = m * tile_rows;
    ti.cls = 0; ti.tapi = 0; ti.tap_lo = 0; ti.kb_lo = 0;
    if (g.mode != 1) {
        ti.c0 = y * g.bn + slice * ti.width;
        ti.cls = z;
        ti.tap_lo = g.cls_begin[z];
        ti.num_iters = (g.cls_begin[z + 1] - ti.tap_lo) * g.kc_per_tap;
    } else {
        ti.tapi = y / g.n_ctile;
        ti.c0 = (y - ti.tapi * g.n_ctile) * g.bn;
        ti.cls = z;   // the reduction slice, which is also the slab its partial sums go to
        ti.kb_lo = z * g.kb_per_split;
        ti.num_iters = max(min(ti.kb_lo + g.kb_per_split, g.kb_total) - ti.kb_lo, 0);
    }
    return ti;
}

__device__ __forceinline__ void report_timeout(GemmShared* sh, int32_t* status) {
    sh->abort = 1u;
    if (status != nullptr) atomicCAS(status, (int32_t)LBT_OK, (int32_t)LBT_ERR_TIMEOUT);
}

__device__ __forceinline__ bool wait_or_abort(GemmShared* sh, uint64_t* bar, uint32_t parity, int32_t* status) {
    if (sh->abort) return false;
    if (mbar_wait_bounded(bar, parity, kWaitLimitNs)) return true;
    report_timeout(sh, status);
    return false;
}

// for the epilogue warps, which wait a whole main loop for their accumulator
__device__ __forceinline__ bool wait_or_abort_relaxed(GemmShared* sh, uint64_t* bar, uint32_t parity, int32_t* status) {
    if (sh->abort) return false;
    if (mbar_wait_bounded_relaxed(bar, parity, kWaitLimitNs)) return true;
    report_timeout(sh, status);
    return false;
}

// Epilogue of one 128-row accumulator for one warp (32 TMEM lanes): TMEM -> registers -> scale ->
// shared-memory transpose -> row-contiguous global stores (fp32 results, or the int32 partial sums of one
// slice of a split reduction).
// `first_row` is the tile-grid row of lane 0; `tmem_acc` addresses this warp's lanes, column 0 of the
// accumulator; with have_acc == false zeros are written instead (an output class without taps).
// Running statistics of the fp32 outputs one epilogue warp has written (dgrad with GemmArgs.dx_stats): the
// abs-max of the next layer's gradient (Sec. 3.1: g_max = max |G|) comes out of the epilogue for free.
// (float)acc -> (float)acc * scale is monotone in |acc|, so the largest |output| is fl32(max |(float)acc| * scale):
// the warp tracks max |(float)acc| and multiplies once at the end.  Only when the scale is so large (or not
// finite) that a product can overflow -- |scale| > FLT_MAX / 2^31 -- are the outputs themselves examined.
struct OutStats {
    float max_abs = 0.0f;    // max |(float)acc| over the chunks tracked before the multiply
    float max_out = 0.0f;    // max |output| over the finite outputs of the chunks examined one by one
    uint32_t bad = 0;        // non-finite outputs (only a scale beyond FLT_MAX / 2^31 can make one)
    bool on = false, risky = false;
};

__device__ __forceinline__ float fmax3_abs(float a, float b, float c) {
    float m;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(m) : "f"(a), "f"(fabsf(b)), "f"(fabsf(c)));
    return m;
}

template <bool kTrack>
__device__ __forceinline__ void drain_accumulator(const GemmArgs& g, const TileInfo& ti, int64_t first_row,
                                                  uint32_t tmem_acc, bool have_acc, uint32_t* stage,
                                                  int32_t* row_slot, float scale, bool vec_ok, int lane,
                                                  int chunk_lo, int chunk_hi, const CUtensorMap* tm_out,
                                                  OutStats& os) {
    // which output pixel (dgrad) or filter-tap slot (wgrad) this lane's row is; other lanes look it
    // up when they store parts of this row
    bool row_written = false;   // this lane's row is an element of the output (not halo, not past the end)
    int32_t my_slot = -1;
    {
        const int64_t row = first_row + lane;
        int32_t slot = -1;
        if (g.mode != 1) {
            // (cell and pixel counts are below 2^31: 32-bit divisions)
            const uint32_t cells = (uint32_t)(g.Hg * g.Wg), row32 = (uint32_t)row;
            const uint32_t n = fast_div(row32, g.by_cells), cell = row32 - n * cells;
            const uint32_t ca = fast_div(cell, g.by_wg), cb = cell - ca * (uint32_t)g.Wg;
            const int h = g.st * (int)ca + ti.cls / g.st, w = g.st * (int)cb + ti.cls % g.st;
            if (row < g.rows && h < g.H && w < g.W) slot = (int32_t)((n * (uint32_t)g.H + (uint32_t)h) * (uint32_t)g.W + (uint32_t)w);
        } else if (row < g.K) {
            slot = (int32_t)(row * g.RS + g.tap_rs[ti.tapi]);
        }
        __syncwarp();
        row_slot[lane] = slot;
        __syncwarp();
        row_written = slot >= 0;
        my_slot = slot;
    }
    for (int chunk = chunk_lo; chunk < chunk_hi; ++chunk) {
        uint32_t v[32];
        if (have_acc) {
            tmem_ld_32x32(tmem_acc + (uint32_t)(chunk * 32), v);
            tmem_ld_wait();
        } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = 0u;
        }
        const int cbase = ti.c0 + chunk * 32;
        if (cbase >= g.C) continue;  // warp-uniform
        const int passes = g.direct == 1 && g.acc != nullptr ? 2 : 1;
        for (int pass = 0; pass < passes; ++pass) {
            const bool as_float = g.direct == 1 && pass == 0;
            if (g.row_direct) {
                // Every lane holds 32 consecutive columns of one output row: they leave as four 32-byte stores
                // (one full sector each) straight from the registers -- no staging in shared memory, whose
                // bandwidth the operand fetch of the MMAs and the TMA fill already use up.
                uint32_t* dst = as_float ? reinterpret_cast<uint32_t*>(g.out)
                                         : reinterpret_cast<uint32_t*>(g.acc) + (g.direct == 2 ? ti.cls * g.part_stride : 0);
                uint32_t* row_dst = dst + (int64_t)my_slot * g.C + cbase;
                const bool track = kTrack && as_float;
                const int ncols = g.C - cbase;       // a multiple of 8 in this mode
                float cmax = 0.0f, omax = 0.0f;
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                    uint32_t w[8];
                    if (as_float) {
                        float f[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            f[e] = __int2float_rn((int)v[j + e]);
                            w[e] = __float_as_uint(__fmul_rn(f[e], scale));
                        }
                        if (kTrack && track && j < ncols) {
                            if (!os.risky) {
                                cmax = fmax3_abs(cmax, f[0], f[1]); cmax = fmax3_abs(cmax, f[2], f[3]);
                                cmax = fmax3_abs(cmax, f[4], f[5]); cmax = fmax3_abs(cmax, f[6], f[7]);
                            } else {
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    const float o = fabsf(__uint_as_float(w[e]));
                                    if (o <= 3.402823466e38f) omax = fmaxf(omax, o);
                                    else if (row_written) ++os.bad;
                                }
                            }
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < 8; ++e) w[e] = v[j + e];
                    }
                    if (row_written && j < ncols) st_global_cs_v8(row_dst + j, w);
                }
                if (kTrack && track && row_written) { os.max_abs = fmaxf(os.max_abs, cmax); os.max_out = fmaxf(os.max_out, omax); }
                continue;
            }
            if (tm_out != nullptr) {
                // the TMA store of the previous block (this chunk loop's, or the previous tile's) must have read it
                if (lane == 0) tma_store_wait_read();
                __syncwarp();
            }
            // lane = row: park the 32 columns of this row in shared memory
            uint4* srow = reinterpret_cast<uint4*>(stage + lane * 32);
            const bool track = kTrack && as_float;
            const int ncols = g.C - cbase;           // columns of this chunk that exist in the output (warp-uniform)
            const bool track_fast = track && !os.risky && ncols >= 32;
            float cmax = 0.0f;
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
                uint4 w;
                if (as_float) {
                    const float f0 = __int2float_rn((int)v[j]), f1 = __int2float_rn((int)v[j + 1]);
                    const float f2 = __int2float_rn((int)v[j + 2]), f3 = __int2float_rn((int)v[j + 3]);
                    w.x = __float_as_uint(__fmul_rn(f0, scale));
                    w.y = __float_as_uint(__fmul_rn(f1, scale));
                    w.z = __float_as_uint(__fmul_rn(f2, scale));
                    w.w = __float_as_uint(__fmul_rn(f3, scale));
                    if (kTrack && track_fast) {
                        cmax = fmax3_abs(cmax, f0, f1);
                        cmax = fmax3_abs(cmax, f2, f3);
                    }
                } else {
                    w = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                }
                srow[(j >> 2) ^ (lane & 7)] = w;
            }
            if (kTrack && track && !track_fast) {
                // ragged last chunk (columns past C hold no output) or a scale that can overflow: the outputs
                // themselves, read back from this lane's staging row, one by one
                float omax = 0.0f;
#pragma unroll 1
                for (int q = 0; q < 8; ++q) {
                    const uint4 w = srow[q ^ (lane & 7)];
                    const uint32_t o4[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float o = fabsf(__uint_as_float(o4[e]));
                        if (4 * q + e >= ncols) continue;
                        if (o <= 3.402823466e38f) omax = fmaxf(omax, o);
                        else if (row_written) ++os.bad;
                    }
                }
                if (row_written) os.max_out = fmaxf(os.max_out, omax);
            }
            if (kTrack && track && row_written) os.max_abs = fmaxf(os.max_abs, cmax);
            if (tm_out != nullptr) {
                // the staging block is laid out as a 128-byte-swizzled 32 x 32 box: TMA writes it out
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0 && first_row < (g.mode == 1 ? (int64_t)g.K : g.rows)) {   // (a block wholly outside is skipped)
                    tma_store_2d(tm_out, stage, cbase, (int32_t)first_row);
                    tma_store_commit();
                }
                continue;
            }
            __syncwarp();
            uint32_t* dst = as_float ? reinterpret_cast<uint32_t*>(g.out)
                                     : reinterpret_cast<uint32_t*>(g.acc) + (g.direct == 2 ? ti.cls * g.part_stride : 0);
            if (vec_ok) {
                // 8 lanes cover the 128 bytes of one row: 4 rows per instruction, whole sectors
                const int sub = lane >> 3, c4 = (lane & 7) * 4;
#pragma unroll
                for (int r4 = 0; r4 < 32; r4 += 4) {
                    const int r = r4 + sub;
                    const int64_t base = (int64_t)row_slot[r] * g.C;
                    const uint4 w = *reinterpret_cast<const uint4*>(stage + r * 32 + (((lane & 7) ^ (r & 7)) << 2));
                    if (base >= 0 && cbase + c4 < g.C) __stcs(reinterpret_cast<uint4*>(dst + base + cbase + c4), w);
                }
            } else {
                for (int r = 0; r < 32; ++r) {
                    const int64_t base = (int64_t)row_slot[r] * g.C;
                    const uint32_t w = stage[r * 32 + ((((lane >> 2) ^ (r & 7)) << 2) | (lane & 3))];
                    if (base >= 0 && cbase + lane < g.C) dst[base + cbase + lane] = w;
                }
            }
            __syncwarp();
        }
    }
}

// End of an epilogue warp's work: its share of the output statistics goes to the caller's struct.
__device__ __forceinline__ void publish_out_stats(const GemmArgs& g, const OutStats& os, float scale, int lane) {
    if (!os.on) return;
    // (max_abs stays 0 when the scale can overflow: every chunk is then examined one by one)
    const float mine = fmaxf(fabsf(__fmul_rn(os.max_abs, scale)), os.max_out);
    const uint32_t m = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(mine));   // non-negative floats order as integers
    const uint32_t bad = __reduce_add_sync(0xFFFFFFFFu, os.bad);
    if (lane != 0) return;
    const float gm = __uint_as_float(m);
    if (gm > 0.0f) atomicMax(reinterpret_cast<uint32_t*>(&g.dx_stats->g_max), __float_as_uint(gm));
    if (bad) atomicAdd(reinterpret_cast<unsigned long long*>(&g.dx_stats->n_nonfinite), (unsigned long long)bad);
}

__device__ __forceinline__ OutStats make_out_stats(const GemmArgs& g, float scale) {
    OutStats os;
    os.on = g.mode == 0 && g.direct == 1 && g.dx_stats != nullptr;
    os.risky = !(fabsf(scale) <= 1.5845632e29f);    // FLT_MAX / 2^31 rounded down: below it no product overflows
    return os;
}

// The MMAs of one tap: kSteps steps of 32 reduction bytes.  Descriptor start addresses count 16 bytes:
// +2 = 32 bytes along a K-major row, +256 = 32 rows of an MN-major tile.
template <int kSteps>
__device__ __forceinline__ void issue_tap(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          int b_kstep, uint32_t& accumulate) {
#pragma unroll
    for (int k = 0; k < kSteps; ++k) {
        mma_i8_ss(d_tmem, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * b_kstep), idesc, accumulate);
        accumulate = 1u;
    }
}

// All taps of one reduction chunk when window and filter are both resident: nothing to wait for, so
// the one issuing thread only adds the next tap's offsets (fetched one tap ahead) and issues.
template <int kSteps>
__device__ __forceinline__ void issue_resident_taps(uint32_t d_tmem, uint64_t a_desc0, uint64_t b_desc0,
                                                    uint32_t idesc, int b_kstep, const uint2* tap_off, int ntaps,
                                                    uint32_t& accumulate) {
    uint2 next = tap_off[0];
    for (int tq = 0; tq < ntaps; ++tq) {
        const uint2 off = next;
        if (tq + 1 < ntaps) next = tap_off[tq + 1];
        issue_tap<kSteps>(d_tmem, a_desc0 + off.x, b_desc0 + off.y, idesc, b_kstep, accumulate);
    }
}

// Persistent kernel: CTA b works on tiles b, b + gridDim.x, ...  Two TMEM accumulator buffers let
// the epilogue of one tile run under the main loop of the next; the TMA ring keeps running across
// tile boundaries.
__global__ void __launch_bounds__(kGemmThreads, 1)
i8_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
               const __grid_constant__ CUtensorMap tmB3, const __grid_constant__ CUtensorMap tmOut,
               const __grid_constant__ GemmArgs g) {
    // the swizzled operand tiles need 1024-byte alignment; aligning at run time (1 KB of slack) also
    // measured 3 % faster on long main loops than declaring the array 1024-byte aligned
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    GemmShared* sh = reinterpret_cast<GemmShared*>(tiles + kStages * kStageBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 32) {   // the descriptors are on their way while the barriers and TMEM are set up
        prefetch_tensormap(&tmA); prefetch_tensormap(&tmB0);
        if (g.tma_store) prefetch_tensormap(&tmOut);
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sh->tmem_full[b], 1); mbar_init(&sh->tmem_empty[b], g.epi_alt ? 4 : g.epi_warps);
            mbar_init(&sh->a_full[b], 1); mbar_init(&sh->a_empty[b], 1);
        }
        sh->abort = 0u;
        fence_mbar_init();
    }
    if ((g.window || g.multi) && threadIdx.x >= 64 && threadIdx.x < 64 + kMaxTaps) {
        const int t = threadIdx.x - 64;
        // forward: the tap's channels start at column t * tap_cols of W, i.e. in 128-byte column box col / 128
        // (the boxes of a column are b_boxes * 16 KB apart) at byte col % 128 of its rows
        const uint32_t col = (uint32_t)(t * g.tap_cols);
        const uint32_t w_off = g.mode == 2 ? (col >> 7) * (uint32_t)g.b_boxes * (kTileBytes >> 4) + ((col & 127u) >> 4)
                                           : (uint32_t)((int)g.tap_aux[t] * g.K) * 8u;
        sh->tap_off[t] = make_uint2((uint32_t)(g.tap_shift[t] - g.win_min_shift) * 8u, w_off);   // 128 bytes per row
    }
    if (warp == 1) { tmem_alloc(&sh->tmem_base, kTmemCols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // set-up done; from here on the kernel reads what the launch before it wrote
    if (g.wait_prev) griddep_wait();
    if (g.overlap_next) griddep_launch_dependents();
    const uint32_t tmem = sh->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one()) {
            const uint32_t stage_tx = (uint32_t)(1 + (g.multi ? 2 : g.b_boxes)) * kTileBytes;
            uint32_t it_global = 0;
            bool ok = true;
            if (g.window) {
                const uint32_t win_bytes = (uint32_t)g.win_boxes * kTileBytes;
                uint8_t* b_ring = tiles + (uint32_t)g.n_win * win_bytes;   // the resident filter
                uint32_t a_i = 0;
                if ((int)blockIdx.x < g.total_tiles) {
                    // the whole filter, once: box (cb, j) = rows [128 j, 128 j + 128) of output channels [128 cb, ...)
                    mbar_arrive_expect_tx(&sh->full[0], (uint32_t)(g.w_boxes * g.b_boxes) * kTileBytes);
                    for (int cb = 0; cb < g.b_boxes; ++cb)
                        for (int j = 0; j < g.w_boxes; ++j) {
                            if (g.mode == 2)   // W[k][taps * Cp]: column box j of filter rows [128 cb, 128 cb + 128)
                                tma_load_2d(b_ring + (j * g.b_boxes + cb) * kTileBytes, &tmA, &sh->full[0], j * kTile, cb * kTile);
                            else
                                tma_load_2d(b_ring + (cb * g.w_boxes + j) * kTileBytes, &tmB0, &sh->full[0], cb * kTile, j * kTile);
                        }
                }
                for (int t = blockIdx.x; t < g.total_tiles && ok; t += gridDim.x) {
                    const TileInfo ti = decode_tile(g, t);
                    const int ntaps = ti.num_iters / g.kc_per_tap;
                    for (int kc = 0; kc < g.kc_per_tap && ok && ntaps > 0; ++kc, ++a_i) {
                        const uint32_t sa = g.n_win == 2 ? (a_i & 1u) : 0u;
                        ok = wait_or_abort(sh, &sh->a_empty[sa], ((g.n_win == 2 ? a_i >> 1 : a_i) & 1u) ^ 1u, g.status);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&sh->a_full[sa], win_bytes);
                        for (int b = 0; b < g.win_boxes; ++b)
                            tma_load_2d(tiles + sa * win_bytes + b * kTileBytes, g.mode == 2 ? &tmB0 : &tmA, &sh->a_full[sa],
                                        kc * kTile, ti.m0 + g.win_min_shift + b * kTile);
                    }
                }
            }
            // ring of 48 KB stages (A + two B boxes) or, with one B box, of six 32 KB stages
            const int n_stages = g.b_boxes == 1 && !g.multi ? kPairStages : kStages;
            const int stage_bytes = g.b_boxes == 1 && !g.multi ? kPairStageBytes : kStageBytes;
            int s = 0;
            uint32_t ph = 0;
            for (int t = blockIdx.x; !g.window && t < g.total_tiles && ok; t += gridDim.x) {
                const TileInfo ti = decode_tile(g, t);
                for (int it = 0; it < ti.num_iters; ++it, ++it_global, ph ^= (s + 1 == n_stages), s = s + 1 == n_stages ? 0 : s + 1) {
                    ok = wait_or_abort(sh, &sh->empty[s], ph ^ 1u, g.status);
                    if (!ok) break;
                    uint8_t* a_dst = tiles + s * stage_bytes;
                    uint8_t* b_dst = a_dst + kTileBytes;
                    mbar_arrive_expect_tx(&sh->full[s], stage_tx);
                    if (g.mode == 0) {
                        const int tq = it / g.kc_per_tap;
                        const int tap = ti.tap_lo + tq;
                        const int kc = it - tq * g.kc_per_tap;
                        tma_load_2d(a_dst, &tmA, &sh->full[s], kc * kTile, ti.m0 + g.tap_shift[tap]);
                        const int brow = (int)g.tap_aux[tap] * g.K + kc * kTile;
                        for (int b = 0; b < g.b_boxes; ++b)
                            tma_load_2d(b_dst + b * kTileBytes, &tmB0, &sh->full[s], ti.c0 + b * kTile, brow);
                    } else if (g.mode == 2) {
                        const int tap = it / g.kc_per_tap;
                        const int kc = it - tap * g.kc_per_tap;
                        const int xcls = g.tap_aux[tap];
                        const CUtensorMap* ta = xcls == 0 ? &tmB0 : xcls == 1 ? &tmB1 : xcls == 2 ? &tmB2 : &tmB3;
                        tma_load_2d(a_dst, ta, &sh->full[s], kc * kTile, ti.m0 + g.tap_shift[tap]);
                        for (int b = 0; b < g.b_boxes; ++b)
                            tma_load_2d(b_dst + b * kTileBytes, &tmA, &sh->full[s], tap * g.tap_cols + kc * kTile,
                                        ti.c0 + b * kTile);
                    } else {
                        const int row = (ti.kb_lo + it) * kTile;
                        tma_load_2d(a_dst, &tmA, &sh->full[s], ti.m0, row);
                        const int xcls = g.tap_aux[g.multi ? (int)g.grp_first[ti.tapi] : ti.tapi];
                        const CUtensorMap* tb = xcls == 0 ? &tmB0 : xcls == 1 ? &tmB1 : xcls == 2 ? &tmB2 : &tmB3;
                        if (g.multi) {   // the group's 256-row window of X
                            for (int b = 0; b < 2; ++b)
                                tma_load_2d(b_dst + b * kTileBytes, tb, &sh->full[s], ti.c0,
                                            row + g.grp_min_shift[ti.tapi] + b * kTile);
                        } else {
                            for (int b = 0; b < g.b_boxes; ++b)
                                tma_load_2d(b_dst + b * kTileBytes, tb, &sh->full[s], ti.c0 + b * kTile,
                                            row + g.tap_shift[ti.tapi]);
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            // narrow outputs: no MMA work on columns that only hold zero fill
            const uint32_t idesc = idesc_i8(kTile, g.mma_n, g.a_signed != 0, g.b_signed != 0, g.mode == 1, g.mode != 2);
            // stage 0's operands; K-major: 32 bytes (2 units) further along each row per MMA, MN-major: 32 rows (256)
            const uint32_t tiles_u32 = smem_u32(tiles);
            const uint64_t a_desc0 = g.mode != 1 ? smem_desc_sw128(tiles_u32, 16, 1024) : smem_desc_sw128(tiles_u32, kTileBytes, 1024);
            const uint64_t b_desc0 = g.mode == 2 ? smem_desc_sw128(tiles_u32 + kTileBytes, 16, 1024)
                                                 : smem_desc_sw128(tiles_u32 + kTileBytes, kTileBytes, 1024);
            const int a_kstep = g.mode != 1 ? 2 : 256, b_kstep = g.mode == 2 ? 2 : 256;
            const int last_steps = (g.k_last + 31) / 32;
            const int n_stages = g.b_boxes == 1 && !g.multi ? kPairStages : kStages;
            const int stage_bytes = g.b_boxes == 1 && !g.multi ? kPairStageBytes : kStageBytes;
            int s = 0;          // ring position and phase of the generic (non-window) main loop
            uint32_t ph = 0;
            uint32_t it_global = 0, acc_i = 0, win_i = 0;
            bool ok = true, w_ready = false;
            for (int t = blockIdx.x; t < g.total_tiles && ok; t += gridDim.x) {
                const TileInfo ti = decode_tile(g, t);
                if (ti.num_iters == 0) continue;
                // multi-tap tiles use all of TMEM for their accumulators: one buffer, no overlap of tiles
                const uint32_t buf = g.multi ? 0u : (acc_i & 1u);
                ok = wait_or_abort(sh, &sh->tmem_empty[buf], (g.multi ? (acc_i & 1u) : ((acc_i >> 1) & 1u)) ^ 1u, g.status);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem + buf * 256u;
                if (g.window) {
                    // (single-CTA kernel: window mode always comes with the filter resident behind the windows)
                    const uint32_t win_bytes = (uint32_t)g.win_boxes * kTileBytes;
                    const uint32_t b_ring = smem_u32(tiles + (uint32_t)g.n_win * win_bytes);
                    const int ntaps = ti.num_iters / g.kc_per_tap;
                    uint32_t accumulate = 0u;
                    if (!w_ready) {
                        ok = wait_or_abort(sh, &sh->full[0], 0u, g.status);
                        if (!ok) break;
                        tc_fence_after_sync();
                        w_ready = true;
                    }
                    for (int kc = 0; kc < g.kc_per_tap && ok; ++kc, ++win_i) {
                        const uint32_t sa = g.n_win == 2 ? (win_i & 1u) : 0u;
                        ok = wait_or_abort(sh, &sh->a_full[sa], (g.n_win == 2 ? win_i >> 1 : win_i) & 1u, g.status);
                        if (!ok) break;
                        tc_fence_after_sync();
                        const int k_steps = kc == g.kc_per_tap - 1 ? (g.k_last + 31) / 32 : kTile / 32;
                        // Descriptors differ from tap to tap only in their start address (the low field, in
                        // 16-byte units, never carries out of it): one add per operand and MMA keeps this
                        // one-thread loop ahead of the short MMAs of narrow layers.
                        // (The 128-byte swizzle is a function of the shared-memory address bits, so a start
                        // address at any 128-byte row of the window addresses the rows as TMA wrote them.)
                        const uint64_t a_desc0 = smem_desc_sw128(smem_u32(tiles + sa * win_bytes), 16, 1024);
                        // dgrad: B is MN-major (reduction rows continue 16 KB per chunk, the next 128 output channels
                        // w_boxes tiles on); forward: B is K-major (the next chunk is the next column box)
                        const uint64_t b_desc0 =
                            g.mode == 2 ? smem_desc_sw128(b_ring + (uint32_t)(kc * g.b_boxes) * (uint32_t)kTileBytes, 16, 1024)
                                        : smem_desc_sw128(b_ring + (uint32_t)kc * (uint32_t)kTileBytes, (uint32_t)g.w_boxes * kTileBytes, 1024);
                        {
                            const uint2* offs = sh->tap_off + ti.tap_lo;
                            switch (k_steps) {
                                case 1: issue_resident_taps<1>(d_tmem, a_desc0, b_desc0, idesc, b_kstep, offs, ntaps, accumulate); break;
                                case 2: issue_resident_taps<2>(d_tmem, a_desc0, b_desc0, idesc, b_kstep, offs, ntaps, accumulate); break;
                                case 3: issue_resident_taps<3>(d_tmem, a_desc0, b_desc0, idesc, b_kstep, offs, ntaps, accumulate); break;
                                default: issue_resident_taps<4>(d_tmem, a_desc0, b_desc0, idesc, b_kstep, offs, ntaps, accumulate); break;
                            }
                        }
                        if (ok) mma_commit(&sh->a_empty[sa]);
                    }
                    if (ok) mma_commit(&sh->tmem_full[buf]);
                    ++acc_i;
                    continue;
                }
                // The descriptors of a stage differ from those of stage 0 only in the start address field
                // (16-byte units): a few adds per MMA keep this one-thread loop ahead of short MMAs.
                uint32_t accumulate = 0u;
                int kc = 0;   // position inside the tap's reduction (dgrad, forward)
                for (int it = 0; it < ti.num_iters; ++it, ++it_global, ph ^= (s + 1 == n_stages), s = s + 1 == n_stages ? 0 : s + 1) {
                    ok = wait_or_abort(sh, &sh->full[s], ph, g.status);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint64_t a_desc = a_desc0 + (uint64_t)(s * (stage_bytes >> 4));
                    const uint64_t b_desc = b_desc0 + (uint64_t)(s * (stage_bytes >> 4));
                    // dgrad, forward: the last chunk of a tap may hold fewer than 128 channels; the rest is zero fill
                    int k_steps = kTile / 32;
                    if (g.mode != 1 && ++kc == g.kc_per_tap) { kc = 0; k_steps = last_steps; }
                    if (g.multi) {
                        // every tap of the group: same A tile, B = the window from the tap's row offset on
                        const int first = g.grp_first[ti.tapi], cnt = g.grp_count[ti.tapi];
                        uint32_t next = sh->tap_off[first].x;
                        for (int tq = 0; tq < cnt; ++tq) {
                            const uint64_t bt = b_desc + next;
                            if (tq + 1 < cnt) next = sh->tap_off[first + tq + 1].x;
                            const uint32_t dt = d_tmem + (uint32_t)(tq * g.acc_cols);
#pragma unroll
                            for (int k = 0; k < kTile / 32; ++k)
                                mma_i8_ss(dt, a_desc + (uint64_t)(k * 256), bt + (uint64_t)(k * 256), idesc, k > 0 ? 1u : accumulate);
                        }
                        accumulate = 1u;   // from the second reduction step on every accumulator holds a sum
                        mma_commit(&sh->empty[s]);
                        continue;
                    }
#pragma unroll
                    for (int k = 0; k < kTile / 32; ++k) {
                        if (k >= k_steps) break;
                        mma_i8_ss(d_tmem, a_desc + (uint64_t)(k * a_kstep), b_desc + (uint64_t)(k * b_kstep), idesc, accumulate);
                        accumulate = 1u;
                    }
                    mma_commit(&sh->empty[s]);
                }
                if (ok) mma_commit(&sh->tmem_full[buf]);
                ++acc_i;
            }
        }
    } else if (warp - 2 < g.epi_warps) {
        // ------------------------------------------------------------------ epilogue (warps 2..5 or 2..9)
        const int quarter = warp & 3;            // the TMEM lane quarter this warp may read
        const int col_half = (warp - 2) >> 2;    // two warps share a quarter: each takes half of the columns
        uint32_t* stage = sh->stage[warp - 2];
        int32_t* row_slot = sh->row_slot[warp - 2];
        const float scale = __fmul_rn(*g.scale_a, *g.scale_b);
        const bool vec_ok = (g.C & 3) == 0;
        OutStats os = make_out_stats(g, scale);
        if (os.on && blockIdx.x == 0 && warp == 2 && lane == 0) g.dx_stats->n = g.dx_n;
        uint32_t acc_i = 0, seq = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < g.total_tiles && ok; t += gridDim.x, ++seq) {
            const TileInfo ti = decode_tile(g, t);
            const bool have_acc = ti.num_iters > 0;
            const uint32_t buf = g.multi ? 0u : (acc_i & 1u);
            if (g.epi_alt && ((have_acc ? buf : (seq & 1u)) != (uint32_t)col_half)) {
                if (have_acc) ++acc_i;   // the other warp group's tile
                continue;
            }
            if (have_acc) {
                ok = wait_or_abort_relaxed(sh, &sh->tmem_full[buf], g.multi ? (acc_i & 1u) : ((acc_i >> 1) & 1u), g.status);
                ok = __all_sync(0xFFFFFFFFu, ok) != 0;  // TMEM loads need the whole warp
                if (!ok) break;
                tc_fence_after_sync();
            }
            const int chunks = (g.mma_n + 31) / 32;                                   // 32-column chunks in use
            const int chunks_half = (g.epi_warps == 8 && !g.epi_alt) ? (chunks + 1) / 2 : chunks;   // chunks per warp
            const int chunk_lo = g.epi_alt ? 0 : col_half * chunks_half;
            if (g.multi) {
                // one accumulator per tap of the group, acc_cols TMEM columns apart
                const int first = g.grp_first[ti.tapi], cnt = g.grp_count[ti.tapi];
                for (int tq = 0; tq < cnt; ++tq) {
                    TileInfo tj = ti;
                    tj.tapi = first + tq;
                    drain_accumulator<false>(g, tj, (int64_t)ti.m0 + quarter * 32,
                                             tmem + (uint32_t)(tq * g.acc_cols) + ((uint32_t)(quarter * 32) << 16), have_acc,
                                             stage, row_slot, scale, vec_ok, lane, chunk_lo,
                                             min(chunk_lo + chunks_half, chunks), nullptr, os);
                }
            } else if (os.on) {
                drain_accumulator<true>(g, ti, (int64_t)ti.m0 + quarter * 32, tmem + buf * 256u + ((uint32_t)(quarter * 32) << 16),
                                        have_acc, stage, row_slot, scale, vec_ok, lane, chunk_lo,
                                        min(chunk_lo + chunks_half, chunks), g.tma_store ? &tmOut : nullptr, os);
            } else {
                drain_accumulator<false>(g, ti, (int64_t)ti.m0 + quarter * 32, tmem + buf * 256u + ((uint32_t)(quarter * 32) << 16),
                                         have_acc, stage, row_slot, scale, vec_ok, lane, chunk_lo,
                                         min(chunk_lo + chunks_half, chunks), g.tma_store ? &tmOut : nullptr, os);
            }
            if (have_acc) {
                // this warp is done with the accumulator buffer: hand it back to the MMA issuer
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh->tmem_empty[buf]);
                ++acc_i;
            }
        }
        publish_out_stats(g, os, scale, lane);
        if (g.tma_store && lane == 0) tma_store_wait_all();   // this thread's stores have landed before the CTA exits
    }

    tc_fence_before_sync();
    __syncthreads();
    if (sh->abort && threadIdx.x == 0) {
        // a wait ran out: give loads that may still be in flight time to land before the shared
        // memory they target is released
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 20000000ull) __nanosleep(1000);
    }
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
    if (g.overlap_prev && threadIdx.x == 0) griddep_wait();
}

// The same contraction on CTA pairs (tcgen05 cta_group::2): the two CTAs of a cluster compute one
// 256 x 256 tile.  Each CTA loads its 128 rows of A and its 128 columns of B, so one MMA reads a
// third less shared memory per SM than the single-CTA form -- the limit of that kernel -- and the
// pair's 12 ring stages hold the same reduction depth in half the bytes per SM.  Rank 0 issues the
// MMAs; loads of both CTAs complete on rank 0's `full` barriers; `tcgen05.commit` signals the `empty`
// and `tmem_full` barriers of both CTAs; the epilogue warps of both CTAs arrive on rank 0's
// `tmem_empty`.  Pair p works on tiles p, p + pairs, ...
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kGemmThreads, 1)
i8_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                    const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
                    const __grid_constant__ CUtensorMap tmB3, const __grid_constant__ CUtensorMap tmOut,
                    const __grid_constant__ GemmArgs g) {
    // the swizzled operand tiles need 1024-byte alignment; aligning at run time (1 KB of slack) also
    // measured 3 % faster on long main loops than declaring the array 1024-byte aligned
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    GemmShared* sh = reinterpret_cast<GemmShared*>(tiles + kPairStages * kPairStageBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1, pairs = gridDim.x >> 1;

    if (threadIdx.x == 32) {   // the descriptors are on their way while the barriers and TMEM are set up
        prefetch_tensormap(&tmA); prefetch_tensormap(&tmB0);
        if (g.tma_store) prefetch_tensormap(&tmOut);
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < kMaxBStages; ++s) { mbar_init(&sh->full[s], 1); mbar_init(&sh->empty[s], 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sh->tmem_full[b], 1); mbar_init(&sh->tmem_empty[b], 2 * g.epi_warps);
            mbar_init(&sh->a_full[b], 1); mbar_init(&sh->a_empty[b], 1);
        }
        sh->abort = 0u;
        fence_mbar_init();
    }
    if (g.window && threadIdx.x >= 64 && threadIdx.x < 64 + kMaxTaps) {
        const int t = threadIdx.x - 64;   // offsets of a tap's rows in the A window, 16-byte units
        sh->tap_off[t] = make_uint2((uint32_t)(g.tap_shift[t] - g.win_min_shift) * 8u, 0u);
    }
    if (warp == 1) { tmem_alloc_pair(&sh->tmem_base, kTmemCols); tmem_relinquish_pair(); }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();   // the peer's barriers exist before anything signals them
    tc_fence_after_sync();
    // set-up done; from here on the kernel reads what the launch before it wrote
    if (g.wait_prev) griddep_wait();
    if (g.overlap_next) griddep_launch_dependents();
    const uint32_t tmem = sh->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (elect_one()) {
            uint32_t it_global = 0;
            bool ok = true;
            if (g.window) {
                // dgrad / forward, stride 1: one row window per CTA and reduction chunk serves all taps (see the
                // single-CTA kernel); each CTA still loads its half of every tap's B tile through a ring
                const uint32_t win_bytes = (uint32_t)g.win_boxes * kTileBytes;
                uint8_t* b_ring = tiles + 2 * win_bytes;
                const CUtensorMap* ta = g.mode == 2 ? &tmB0 : &tmA;
                uint32_t a_i = 0, b_i = 0;
                for (int t = pair; t < g.total_tiles && ok; t += pairs) {
                    const TileInfo ti = decode_tile(g, t, 2 * kTile);
                    const int m_half = ti.m0 + (int)rank * kTile, c_half = ti.c0 + (int)rank * (ti.width >> 1);
                    const int ntaps = ti.num_iters / g.kc_per_tap;
                    for (int kc = 0; kc < g.kc_per_tap && ok && ntaps > 0; ++kc, ++a_i) {
                        const uint32_t sa = a_i & 1u;
                        ok = wait_or_abort(sh, &sh->a_empty[sa], ((a_i >> 1) & 1u) ^ 1u, g.status);
                        if (!ok) break;
                        if (rank == 0) mbar_arrive_expect_tx(&sh->a_full[sa], 2u * win_bytes);   // both CTAs' windows
                        const uint32_t a_full0 = map_to_cta(smem_u32(&sh->a_full[sa]), 0);
                        for (int b = 0; b < g.win_boxes; ++b)
                            tma_load_2d_pair(tiles + sa * win_bytes + b * kTileBytes, ta, a_full0, kc * kTile,
                                             m_half + g.win_min_shift + b * kTile);
                        for (int tq = 0; tq < ntaps; ++tq, ++b_i) {
                            const int tap = ti.tap_lo + tq;
                            const uint32_t sb = b_i % (uint32_t)g.n_bstages;
                            ok = wait_or_abort(sh, &sh->empty[sb], ((b_i / (uint32_t)g.n_bstages) & 1u) ^ 1u, g.status);
                            if (!ok) break;
                            if (rank == 0) mbar_arrive_expect_tx(&sh->full[sb], 2u * kTileBytes);
                            const uint32_t full0 = map_to_cta(smem_u32(&sh->full[sb]), 0);
                            if (g.mode == 2)
                                tma_load_2d_pair(b_ring + sb * kTileBytes, &tmA, full0, tap * g.tap_cols + kc * kTile, c_half);
                            else
                                tma_load_2d_pair(b_ring + sb * kTileBytes, &tmB0, full0, c_half, (int)g.tap_aux[tap] * g.K + kc * kTile);
                        }
                    }
                }
            }
            for (int t = pair; !g.window && t < g.total_tiles && ok; t += pairs) {
                const TileInfo ti = decode_tile(g, t, 2 * kTile);
                const int m_half = ti.m0 + (int)rank * kTile;   // this CTA's rows of the tile
                const int c_half = ti.c0 + (int)rank * (ti.width >> 1);   // this CTA's columns of B (a 128-byte box
                                                                          // whose first width / 2 bytes the MMA reads)
                for (int it = 0; it < ti.num_iters; ++it, ++it_global) {
                    const int s = it_global % kPairStages;
                    const uint32_t ph = (it_global / kPairStages) & 1u;
                    ok = wait_or_abort(sh, &sh->empty[s], ph ^ 1u, g.status);
                    if (!ok) break;
                    uint8_t* a_dst = tiles + s * kPairStageBytes;
                    uint8_t* b_dst = a_dst + kTileBytes;
                    // rank 0's barrier counts the bytes of both CTAs
                    if (rank == 0) mbar_arrive_expect_tx(&sh->full[s], 4u * kTileBytes);
                    const uint32_t full0 = map_to_cta(smem_u32(&sh->full[s]), 0);
                    if (g.mode == 0) {
                        const int tq = it / g.kc_per_tap;
                        const int tap = ti.tap_lo + tq;
                        const int kc = it - tq * g.kc_per_tap;
                        tma_load_2d_pair(a_dst, &tmA, full0, kc * kTile, m_half + g.tap_shift[tap]);
                        tma_load_2d_pair(b_dst, &tmB0, full0, c_half, (int)g.tap_aux[tap] * g.K + kc * kTile);
                    } else if (g.mode == 2) {
                        const int tap = it / g.kc_per_tap;
                        const int kc = it - tap * g.kc_per_tap;
                        const int xcls = g.tap_aux[tap];
                        const CUtensorMap* ta = xcls == 0 ? &tmB0 : xcls == 1 ? &tmB1 : xcls == 2 ? &tmB2 : &tmB3;
                        tma_load_2d_pair(a_dst, ta, full0, kc * kTile, m_half + g.tap_shift[tap]);
                        tma_load_2d_pair(b_dst, &tmA, full0, tap * g.tap_cols + kc * kTile, c_half);
                    } else {
                        const int row = (ti.kb_lo + it) * kTile;
                        tma_load_2d_pair(a_dst, &tmA, full0, m_half, row);
                        const int xcls = g.tap_aux[ti.tapi];
                        const CUtensorMap* tb = xcls == 0 ? &tmB0 : xcls == 1 ? &tmB1 : xcls == 2 ? &tmB2 : &tmB3;
                        tma_load_2d_pair(b_dst, tb, full0, c_half, row + g.tap_shift[ti.tapi]);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (rank 0 only)
        if (rank == 0 && elect_one()) {
            const uint32_t idesc_full = idesc_i8(2 * kTile, 2 * kTile, g.a_signed != 0, g.b_signed != 0, g.mode == 1, g.mode != 2);
            const uint32_t idesc_slice = idesc_i8(2 * kTile, g.bn / max(g.split_n, 1), g.a_signed != 0, g.b_signed != 0, g.mode == 1,
                                                  g.mode != 2);
            uint32_t it_global = 0, acc_i = 0, win_i = 0;
            bool ok = true;
            for (int t = pair; t < g.total_tiles && ok; t += pairs) {
                const TileInfo ti = decode_tile(g, t, 2 * kTile);
                if (ti.num_iters == 0) continue;
                const uint32_t idesc = ti.width == g.bn ? idesc_full : idesc_slice;
                const uint32_t buf = acc_i & 1u;
                ok = wait_or_abort(sh, &sh->tmem_empty[buf], ((acc_i >> 1) & 1u) ^ 1u, g.status);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem + buf * 256u;
                if (g.window) {
                    const uint32_t win_bytes = (uint32_t)g.win_boxes * kTileBytes;
                    const uint32_t b_ring = smem_u32(tiles + 2 * win_bytes);
                    const uint64_t b_desc0 = g.mode == 2 ? smem_desc_sw128(b_ring, 16, 1024) : smem_desc_sw128(b_ring, kTileBytes, 1024);
                    const int b_kstep = g.mode == 2 ? 2 : 256;
                    const int ntaps = ti.num_iters / g.kc_per_tap;
                    uint32_t accumulate = 0u;
                    for (int kc = 0; kc < g.kc_per_tap && ok; ++kc, ++win_i) {
                        const uint32_t sa = win_i & 1u;
                        ok = wait_or_abort(sh, &sh->a_full[sa], (win_i >> 1) & 1u, g.status);
                        if (!ok) break;
                        tc_fence_after_sync();
                        const uint64_t a_desc0 = smem_desc_sw128(smem_u32(tiles + sa * win_bytes), 16, 1024);
                        for (int tq = 0; tq < ntaps; ++tq, ++it_global) {
                            const uint32_t sb = it_global % (uint32_t)g.n_bstages;
                            ok = wait_or_abort(sh, &sh->full[sb], (it_global / (uint32_t)g.n_bstages) & 1u, g.status);
                            if (!ok) break;
                            tc_fence_after_sync();
                            const uint64_t a_desc = a_desc0 + sh->tap_off[ti.tap_lo + tq].x;
                            const uint64_t b_desc = b_desc0 + (uint64_t)(sb * (kTileBytes >> 4));
#pragma unroll
                            for (int k = 0; k < kTile / 32; ++k) {
                                mma_i8_ss_pair(d_tmem, a_desc + (uint64_t)(k * 2), b_desc + (uint64_t)(k * b_kstep), idesc, accumulate);
                                accumulate = 1u;
                            }
                            mma_commit_pair(&sh->empty[sb]);
                        }
                        if (ok) mma_commit_pair(&sh->a_empty[sa]);
                    }
                    if (ok) mma_commit_pair(&sh->tmem_full[buf]);
                    ++acc_i;
                    continue;
                }
                for (int it = 0; it < ti.num_iters; ++it, ++it_global) {
                    const int s = it_global % kPairStages;
                    const uint32_t ph = (it_global / kPairStages) & 1u;
                    ok = wait_or_abort(sh, &sh->full[s], ph, g.status);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t a_base = smem_u32(tiles + s * kPairStageBytes);
                    const uint32_t b_base = a_base + kTileBytes;
#pragma unroll
                    for (int k = 0; k < kTile / 32; ++k) {
                        const uint64_t a_desc = g.mode != 1 ? smem_desc_sw128(a_base + k * 32, 16, 1024)
                                                            : smem_desc_sw128(a_base + k * 4096, kTileBytes, 1024);
                        const uint64_t b_desc = g.mode == 2 ? smem_desc_sw128(b_base + k * 32, 16, 1024)
                                                            : smem_desc_sw128(b_base + k * 4096, kTileBytes, 1024);
                        mma_i8_ss_pair(d_tmem, a_desc, b_desc, idesc, (it > 0 || k > 0) ? 1u : 0u);
                    }
                    mma_commit_pair(&sh->empty[s]);
                }
                if (ok) mma_commit_pair(&sh->tmem_full[buf]);
                ++acc_i;
            }
        }
    } else if (warp - 2 < g.epi_warps) {
        // ------------------------------------------------------------------ epilogue (warps 2..5 or 2..9, both CTAs)
        const int quarter = warp & 3;
        const int col_half = (warp - 2) >> 2;
        uint32_t* stage = sh->stage[warp - 2];
        int32_t* row_slot = sh->row_slot[warp - 2];
        const float scale = __fmul_rn(*g.scale_a, *g.scale_b);
        const bool vec_ok = (g.C & 3) == 0;
        OutStats os = make_out_stats(g, scale);
        if (os.on && blockIdx.x == 0 && warp == 2 && lane == 0) g.dx_stats->n = g.dx_n;
        uint32_t acc_i = 0;
        bool ok = true;
        for (int t = pair; t < g.total_tiles && ok; t += pairs) {
            const TileInfo ti = decode_tile(g, t, 2 * kTile);
            const bool have_acc = ti.num_iters > 0;
            const uint32_t buf = acc_i & 1u;
            if (have_acc) {
                ok = wait_or_abort_relaxed(sh, &sh->tmem_full[buf], (acc_i >> 1) & 1u, g.status);
                ok = __all_sync(0xFFFFFFFFu, ok) != 0;
                if (!ok) break;
                tc_fence_after_sync();
            }
            const int chunks_half = g.epi_warps == 8 ? max(ti.width / 64, 1) : ti.width / 32;   // chunks per warp
            if (os.on)
                drain_accumulator<true>(g, ti, (int64_t)ti.m0 + (int64_t)rank * kTile + quarter * 32,
                                        tmem + buf * 256u + ((uint32_t)(quarter * 32) << 16), have_acc, stage, row_slot, scale,
                                        vec_ok, lane, col_half * chunks_half, (col_half + 1) * chunks_half,
                                        g.tma_store ? &tmOut : nullptr, os);
            else
                drain_accumulator<false>(g, ti, (int64_t)ti.m0 + (int64_t)rank * kTile + quarter * 32,
                                         tmem + buf * 256u + ((uint32_t)(quarter * 32) << 16), have_acc, stage, row_slot, scale,
                                         vec_ok, lane, col_half * chunks_half, (col_half + 1) * chunks_half,
                                         g.tma_store ? &tmOut : nullptr, os);
            if (have_acc) {
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster_relaxed(map_to_cta(smem_u32(&sh->tmem_empty[buf]), 0));
                ++acc_i;
            }
        }
        publish_out_stats(g, os, scale, lane);
        if (g.tma_store && lane == 0) tma_store_wait_all();   // this thread's stores have landed before the CTA exits
    }

    tc_fence_before_sync();
    __syncthreads();
    if (sh->abort && threadIdx.x == 0) {
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 20000000ull) __nanosleep(1000);
    }
    cluster_sync_all();   // neither CTA leaves while its peer may still touch its barriers or TMEM
    if (warp == 1) tmem_dealloc_pair(tmem, kTmemCols);
    if (g.overlap_prev && threadIdx.x == 0) griddep_wait();
}

// One thread waits, with the kernels' bounded wait, on a barrier that never completes.
__global__ void selftest_wait_kernel(int32_t* status, uint64_t limit_ns) {
    __shared__ uint64_t never;
    if (threadIdx.x != 0) return;
    mbar_init(&never, 1);
    fence_mbar_init();
    if (!mbar_wait_bounded(&never, 0u, limit_ns)) atomicCAS(status, (int32_t)LBT_OK, (int32_t)LBT_ERR_TIMEOUT);
}

// split-reduction finish: acc = sum over the slabs of partial sums; dW = (float)acc * fl32(s_g * s_x)
__global__ void __launch_bounds__(256)
finalize_partials_kernel(const int32_t* __restrict__ part, int splits, int64_t stride, int64_t n,
                         float* __restrict__ out, int32_t* __restrict__ acc_out,
                         const float* __restrict__ scale_a, const float* __restrict__ scale_b) {
    griddep_wait();   // may have been launched before the contraction that writes the slabs has ended
    const float scale = __fmul_rn(*scale_a, *scale_b);
    const int64_t nvec = n >> 2;
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += step) {
        int4 sum = make_int4(0, 0, 0, 0);
#pragma unroll 8
        for (int z = 0; z < splits; ++z) {
            const int4 p = __ldcs(reinterpret_cast<const int4*>(part + z * stride) + v);
            sum.x += p.x; sum.y += p.y; sum.z += p.z; sum.w += p.w;
        }
        reinterpret_cast<float4*>(out)[v] = make_float4(__fmul_rn(__int2float_rn(sum.x), scale), __fmul_rn(__int2float_rn(sum.y), scale),
                                                        __fmul_rn(__int2float_rn(sum.z), scale), __fmul_rn(__int2float_rn(sum.w), scale));
        if (acc_out != nullptr) reinterpret_cast<int4*>(acc_out)[v] = sum;
    }
    if (blockIdx.x == 0 && threadIdx.x < (n & 3)) {   // ragged tail
        const int64_t i = (nvec << 2) + threadIdx.x;
        int sum = 0;
        for (int z = 0; z < splits; ++z) sum += part[z * stride + i];
        out[i] = __fmul_rn(__int2float_rn(sum), scale);
        if (acc_out != nullptr) acc_out[i] = sum;
    }
}

// dW = (float)acc * fl32(s_a * s_b) on finished accumulators
__global__ void __launch_bounds__(256)
finalize_kernel(const int32_t* __restrict__ acc, float* __restrict__ out, int64_t n,
                const float* __restrict__ scale_a, const float* __restrict__ scale_b) {
    const float scale = __fmul_rn(*scale_a, *scale_b);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = __fmul_rn(__int2float_rn(acc[i]), scale);
}

// ------------------------------------------------------------------------------------------
// Host side.
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// 2-D uint8 tensor [rows][pitch bytes], boxes of 128 rows x 128 bytes, 128-byte swizzle, zero fill
// outside the tensor.
static bool make_map(CUtensorMap* tm, const void* base, uint64_t inner, uint64_t rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {inner, rows};
    const cuuint64_t strides[1] = {inner};
    const cuuint32_t box[2] = {128, 128};
    const cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 2-D fp32 output [rows][cols] for the epilogue's TMA stores: boxes of 32 rows x 32 columns (128 bytes),
// 128-byte swizzle (the layout of the epilogue's staging block).
static bool make_out_map(CUtensorMap* tm, const float* base, uint64_t cols, uint64_t rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * sizeof(float)};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Launch, optionally with the programmatic-serialization attribute (the kernel may then be scheduled before the
// launch ahead of it in the stream has ended, and waits for it on the device where it has to).
template <typename... Params, typename... Args>
static cudaError_t launch_kernel(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 bool programmatic, Args&&... args) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = programmatic ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

static bool any_tap_armed() {
    for (int c = 0; c < LBT_TIME_CLASSES; ++c)
        if (timing_armed(c)) return true;
    return false;
}

// Collects the expansions of one call and launches them together.
struct ExpandBatch {
    ExpandJobs jobs{};
    int blocks = 0;
    void add(ExpandArgs e) {
        int64_t want;
        if (e.identity) {
            const int64_t vecs = e.rows_total * e.chunks;
            want = std::max<int64_t>(1, std::min<int64_t>((vecs / 2 + 255) / 256, (int64_t)kNumSMs * 8));
        } else {
            // about 2048 chunks per block, whole rows; never longer than one parity class, so that a block
            // crosses at most one class boundary (the kernel handles exactly one)
            // (fewer rows per block when that is needed to give every SM a few blocks)
            e.rows_per_block = (int)std::max<int64_t>(1, std::min<int64_t>(2048 / e.chunks, e.rows_per_cls));
            e.rows_per_block = (int)std::max<int64_t>(1, std::min<int64_t>(e.rows_per_block, e.rows_total / (4 * kNumSMs)));
            e.by_chunks = make_fastdiv((uint32_t)e.chunks);
            e.by_cells = make_fastdiv((uint32_t)(e.Hg * e.Wg));
            e.by_wg = make_fastdiv((uint32_t)e.Wg);
            e.by_k = make_fastdiv((uint32_t)std::max(e.K, 1));
            const int64_t blocks_needed = (e.rows_total + e.rows_per_block - 1) / e.rows_per_block;
            want = std::max<int64_t>(1, std::min<int64_t>(blocks_needed, (int64_t)kNumSMs * 16));
        }
        jobs.job[jobs.n] = e;
        jobs.first_block[jobs.n] = blocks;
        blocks += (int)want;
        jobs.first_block[++jobs.n] = blocks;
    }
    // `chained`: the launch ahead in the stream is the quantizer whose output the jobs marked `wait_prev` read
    cudaError_t launch(cudaStream_t stream, bool chained = false) {
        if (jobs.n == 0) return cudaSuccess;
        jobs.chained = chained ? 1 : 0;
        return launch_kernel(expand_batch_kernel, dim3((unsigned)blocks), dim3(256), 0, stream, chained, jobs);
    }
};

static int expand_grid(int64_t vecs) {
    const int64_t blocks = (vecs + 255) / 256;
    return (int)std::max<int64_t>(1, std::min<int64_t>(blocks, (int64_t)kNumSMs * 8));
}

static bool bits_ok(int b) { return b >= 2 && b <= 8; }

// Row tiles per band of the tile walk: about the square root of the tiles in flight, so that the
// strips of A and B in use at one time are equally many and few.
static int tile_band(int m_tiles, int ny, int units) {
    if (ny <= 1 || m_tiles <= 1) return std::max(m_tiles, 1);
    int band = 1;
    while ((band + 1) * (band + 1) <= units) ++band;
    return std::max(1, std::min(band, m_tiles));
}

static void finish_args(GemmArgs* a) {
    a->by_mtiles = make_fastdiv((uint32_t)std::max(a->m_tiles, 1));
    a->by_cells = make_fastdiv((uint32_t)std::max(a->Hg * a->Wg, 1));
    a->by_wg = make_fastdiv((uint32_t)std::max(a->Wg, 1));
}

// CTA-pair kernel, dgrad / forward: when the tile count leaves a last round that is at most a quarter full, its tiles
// are cut into 4 column slices (MMA N = 64: each CTA then feeds the first 32 bytes of its 128-byte B rows), so that
// more pairs share the tail.  (A slice takes about as long per step as a whole tile -- the step is bound by the operand
// feed, not by the MMAs -- so the cut pays only where few tiles are left: 3 left-over tiles -3 %; cutting 34 left-over
// tiles in two measured 7 % slower and is not done.)  Returns the unit count.
static int64_t split_last_round(GemmArgs* a, int64_t tiles, int pairs) {
    a->split_n = 0;
    a->split_from = 0;
    const int64_t left = tiles % pairs, full = tiles - left;
    if (full == 0 || left == 0) return tiles;
    const int slices = 4 * left <= pairs ? 4 : 1;
    if (slices == 1 || a->bn != 256) return tiles;
    a->split_n = slices;
    a->split_from = (int)full;
    return full + left * slices;
}

// SMs of the current device: the persistent kernel launches one CTA per SM.
static int sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        return kNumSMs;
    return n;
}

// The contraction kernels use more dynamic shared memory than a launch gets by default; the attribute
// that allows it belongs to the device that is current when it is set, so it is set once per device.
static lbt_status ensure_smem_attr() {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static bool known[kMaxDevices];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LBT_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!known[dev]) {
        if (cudaFuncSetAttribute(i8_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemBytes) != cudaSuccess ||
            cudaFuncSetAttribute(i8_gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemBytes) != cudaSuccess)
            return LBT_ERR_CUDA;
        known[dev] = true;
    }
    return LBT_OK;
}

// The explicit-patch (im2col) lowering of a layer with very few input channels, see im2col_kernel.
static bool im2col_applies(const Geometry& g) {
    const int64_t chunks = ((int64_t)g.R * g.S * g.C + 15) / 16;
    return g.C < 8 && g.R * g.S > 1 && g.R * g.S * g.C <= 1024 && (int64_t)g.N * g.P * g.Q * chunks < ((int64_t)1 << 31);
}

static bool im2col_geometry(const Geometry& g, lbt_conv_desc* lin, Geometry* g2) {
    if (!im2col_applies(g)) return false;
    lin->N = g.N * g.P * g.Q; lin->C = g.R * g.S * g.C; lin->H = 1; lin->W = 1; lin->K = g.K; lin->R = 1; lin->S = 1;
    lin->stride = 1; lin->pad = 0;
    return make_geometry(lin, g2) == LBT_OK;
}

static void launch_im2col(const Geometry& g, const Geometry& g2, const void* q_X, int bits_x, uint8_t* dst, cudaStream_t stream) {
    Im2colArgs a{};
    a.src = static_cast<const uint8_t*>(q_X); a.dst = dst; a.packed = bits_x <= 4;
    a.C = g.C; a.H = g.H; a.W = g.W; a.S = g.S; a.st = g.st; a.pad = g.pad; a.P = g.P; a.Q = g.Q;
    a.cols = g.R * g.S * g.C; a.chunks = g2.Cp / 16; a.total = (int64_t)g.N * g.P * g.Q * a.chunks;
    a.by_chunks = make_fastdiv((uint32_t)a.chunks); a.by_pq = make_fastdiv((uint32_t)(g.P * g.Q));
    a.by_q = make_fastdiv((uint32_t)g.Q); a.by_sc = make_fastdiv((uint32_t)(g.S * g.C)); a.by_c = make_fastdiv((uint32_t)g.C);
    im2col_kernel<<<expand_grid(a.total), 256, 0, stream>>>(a);
}

// Workspace a convolution needs: its own, or that of the linear layer it is lowered to.
static size_t conv_workspace(const Geometry& g, bool wgrad) {
    const Workspace w = carve(g);
    size_t need = wgrad ? w.total : w.total_nowgrad;
    lbt_conv_desc lin;
    Geometry g2;
    if (im2col_geometry(g, &lin, &g2)) {
        const Workspace w2 = carve(g2);
        need = std::max(need, wgrad ? w2.total : w2.total_nowgrad);
    }
    return need;
}

static lbt_status conv_backward_impl(const lbt_conv_desc* d, const void* q_dY, const void* q_W, const void* q_X,
                                     const float* s_g, const float* s_w, const float* s_x, float* dX, float* dW,
                                     int32_t* accX, int32_t* accW, int bits_g, int bits_w, int bits_x,
                                     int32_t* dev_status, void* ws, size_t ws_bytes, cudaStream_t stream,
                                     const uint8_t* dy_int8 = nullptr, const uint8_t* x_int8 = nullptr,
                                     bool behind_quantizer = false, lbt_grad_stats_t* dx_stats = nullptr) {
    // dx_stats: optional, cleared by the caller earlier in the stream: the dgrad epilogue leaves the abs-max,
    // the non-finite count and the element count of dX there.
    // dy_int8: the gradient codes already as one int8 per element in the cell-grid layout (only
    // possible when the grid needs no padding); the expansion of q_dY is then skipped.
    // x_int8: likewise X already in the (class-) grid layout of this geometry.
    // behind_quantizer: the launch ahead in the stream is the one-launch quantizer that writes q_dY / dy_int8.
    Geometry g;
    lbt_status rc = make_geometry(d, &g);
    if (rc != LBT_OK) return rc;
    const bool do_dgrad = dX != nullptr, do_wgrad = dW != nullptr;
    if (q_dY == nullptr || s_g == nullptr || (!do_dgrad && !do_wgrad)) return LBT_ERR_INVALID_ARG;
    if (do_dgrad && (q_W == nullptr || s_w == nullptr)) return LBT_ERR_INVALID_ARG;
    if (do_wgrad && (q_X == nullptr || s_x == nullptr)) return LBT_ERR_INVALID_ARG;
    if (!bits_ok(bits_g) || (do_dgrad && !bits_ok(bits_w)) || (do_wgrad && !bits_ok(bits_x)))
        return LBT_ERR_UNSUPPORTED_BITS;
    if (!aligned16(q_dY) || !aligned16(q_W) || !aligned16(q_X) || !aligned16(dX) || !aligned16(dW) ||
        !aligned16(accX) || !aligned16(accW))
        return LBT_ERR_ALIGNMENT;
    // worst-case accumulator magnitude must fit int32
    const double mag_g = (double)(1 << (bits_g - 1));
    if (do_dgrad && (double)g.K * g.R * g.S * mag_g * (double)(1 << (bits_w - 1)) >= 2147483648.0)
        return LBT_ERR_ACC_RANGE;
    if (do_wgrad && (double)g.N * g.P * g.Q * mag_g * (double)((1 << bits_x) - 1) >= 2147483648.0)
        return LBT_ERR_ACC_RANGE;
    const Workspace w = carve(g);
    if (ws == nullptr || ws_bytes < (x_int8 != nullptr ? w.total : conv_workspace(g, do_wgrad))) return LBT_ERR_WORKSPACE;
    rc = ensure_smem_attr();
    if (rc != LBT_OK) return rc;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(ws) + 255) & ~(uintptr_t)255) - 256;
    // `base + off` with off >= 256 stays inside [ws, ws + total)
    {
        // very few input channels: wgrad as the linear layer over explicit patches (dgrad keeps the grid)
        lbt_conv_desc lin;
        Geometry g2;
        if (do_wgrad && x_int8 == nullptr && im2col_geometry(g, &lin, &g2)) {
            if (do_dgrad) {
                rc = conv_backward_impl(d, q_dY, q_W, nullptr, s_g, s_w, nullptr, dX, nullptr, accX, nullptr, bits_g, bits_w,
                                        bits_x, dev_status, ws, ws_bytes, stream, dy_int8, nullptr, behind_quantizer, dx_stats);
                if (rc != LBT_OK) return rc;
            }
            uint8_t* patches = base + carve(g2).off_x;
            launch_im2col(g, g2, q_X, bits_x, patches, stream);
            if (cudaGetLastError() != cudaSuccess) return LBT_ERR_CUDA;
            return conv_backward_impl(&lin, q_dY, nullptr, q_X, s_g, nullptr, s_x, nullptr, dW, nullptr, accW, bits_g, bits_w,
                                      bits_x, dev_status, ws, ws_bytes, stream, nullptr, patches);
        }
    }
    const uint8_t* dyg = dy_int8 != nullptr ? dy_int8 : base + w.off_dy;
    uint8_t* wt = base + w.off_wt;
    const uint8_t* xg = x_int8 != nullptr ? x_int8 : base + w.off_x;
    int32_t* part_ws = reinterpret_cast<int32_t*>(base + w.off_part);
    int32_t* status = dev_status != nullptr ? dev_status : reinterpret_cast<int32_t*>(base + w.off_status);
    if (dev_status == nullptr) LBT_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), stream));

    // ---- expand the operands onto the cell grid
    timing_begin(LBT_TIME_EXPAND, stream);
    ExpandArgs e{};
    e.Hg = g.Hg; e.Wg = g.Wg; e.st = g.st; e.RS = g.R * g.S; e.K = g.K;
    e.src = static_cast<const uint8_t*>(q_dY); e.dst = base + w.off_dy; e.mode = 0; e.packed = bits_g <= 4; e.is_signed = 1;
    e.Cs = g.K; e.chunks = g.Kp / 16; e.rows_total = g.rows; e.rows_per_cls = g.rows; e.Hs = g.P; e.Ws = g.Q;
    const bool flat = g.st == 1 && g.Hg == g.H && g.Wg == g.W && g.P == g.H && g.Q == g.W;   // grid == image, no halo
    e.identity = flat && g.K == g.Kp;
    // chained behind the quantizer (no timing tap armed): W and X expand while its last blocks drain; the
    // job that reads its codes comes last in block order, so blocks that have to wait do not hold back the others
    const bool chained = behind_quantizer && !any_tap_armed();
    const ExpandArgs e_dy = e;
    ExpandBatch batch;
    if (do_dgrad) {
        e.src = static_cast<const uint8_t*>(q_W); e.dst = wt; e.mode = 1; e.packed = bits_w <= 4; e.is_signed = 1;
        e.Cs = g.C; e.chunks = g.Cp / 16; e.rows_total = (int64_t)g.R * g.S * g.K; e.rows_per_cls = e.rows_total;
        e.identity = g.R * g.S == 1 && g.C == g.Cp;
        batch.add(e);
    }
    if (do_wgrad && x_int8 == nullptr) {
        e.src = static_cast<const uint8_t*>(q_X); e.dst = base + w.off_x; e.mode = 2; e.packed = bits_x <= 4; e.is_signed = 0;
        e.Cs = g.C; e.chunks = g.Cp / 16; e.rows_total = g.rows * g.ncls; e.rows_per_cls = g.rows;
        e.Hs = g.H; e.Ws = g.W;
        e.identity = flat && g.C == g.Cp;
        batch.add(e);
    }
    if (dy_int8 == nullptr) {
        e = e_dy;
        e.wait_prev = chained ? 1 : 0;
        batch.add(e);
    }
    const cudaError_t expand_err = batch.launch(stream, chained);
    timing_end(LBT_TIME_EXPAND, stream);
    if (expand_err != cudaSuccess || cudaGetLastError() != cudaSuccess) return LBT_ERR_CUDA;

    CUtensorMap tmA, tmB[4];
    if (!make_map(&tmA, dyg, (uint64_t)g.Kp, (uint64_t)g.rows)) return LBT_ERR_CUDA;
    const size_t smem = kGemmSmemBytes;
    const int bn = g.Cp <= 128 ? 128 : 256;

    GemmArgs a{};
    a.bn = bn; a.b_boxes = bn / 128; a.n_ctile = (g.Cp + bn - 1) / bn;
    a.mma_n = g.Cp < bn ? g.Cp : bn;          // Cp is a multiple of 16
    a.k_last = g.Kp - (((g.Kp + kTile - 1) / kTile) - 1) * kTile;
    a.K = g.K; a.C = g.C; a.RS = g.R * g.S;
    a.Hg = g.Hg; a.Wg = g.Wg; a.H = g.H; a.W = g.W; a.st = g.st; a.rows = g.rows;
    a.scale_a = s_g; a.status = status; a.a_signed = 1;

    // no timing tap armed: consecutive launches are chained programmatically
    const bool chain = !any_tap_armed();
    const bool behind_expand = chain && batch.jobs.n > 0;   // the launch right before the first contraction is the expansion
    bool overlap = false;
    if (do_dgrad) {
        if (!make_map(&tmB[0], wt, (uint64_t)g.Cp, (uint64_t)g.R * g.S * g.K)) return LBT_ERR_CUDA;
        a.mode = 0; a.kc_per_tap = (g.Kp + kTile - 1) / kTile; a.direct = 1; a.b_signed = 1;
        a.scale_b = s_w; a.out = dX; a.acc = accX;
        a.dx_stats = dx_stats; a.dx_n = (uint64_t)g.N * g.H * g.W * g.C;
        int nt = 0;
        for (int cls = 0; cls < g.ncls; ++cls) {
            a.cls_begin[cls] = nt;
            const int ph = cls / g.st, pw = cls % g.st;
            for (int r = 0; r < g.R; ++r) {
                if (posmod(ph + g.pad - r, g.st) != 0) continue;
                for (int s = 0; s < g.S; ++s) {
                    if (posmod(pw + g.pad - s, g.st) != 0) continue;
                    a.tap_shift[nt] = (ph + g.pad - r) / g.st * g.Wg + (pw + g.pad - s) / g.st;
                    a.tap_aux[nt] = (short)(r * g.S + s);
                    ++nt;
                }
            }
        }
        for (int cls = g.ncls; cls <= 4; ++cls) a.cls_begin[cls] = nt;
        {
            int most_taps = 0;
            for (int cls = 0; cls < g.ncls; ++cls) most_taps = std::max(most_taps, a.cls_begin[cls + 1] - a.cls_begin[cls]);
            a.epi_warps = most_taps * a.kc_per_tap <= kShortMainLoop ? 8 : 4;
        }
        // CTA pairs (256 x 256 tiles) when the output is wide enough and the pairs finish in no more
        // rounds (weighted by their faster main loop) than single CTAs with 128 x 256 tiles would
        const int sms = sm_count();
        const int64_t n128 = ((g.rows + kTile - 1) / kTile) * a.n_ctile * g.ncls;
        const int64_t n256 = ((g.rows + 2 * kTile - 1) / (2 * kTile)) * a.n_ctile * g.ncls;
        const int64_t rounds1 = (n128 + sms - 1) / sms, rounds2 = (n256 + sms / 2 - 1) / (sms / 2);
        const bool pair = bn == 256 && sms >= 2 && 3 * rounds2 <= 4 * rounds1;
        const int tile_rows = pair ? 2 * kTile : kTile;
        a.m_tiles = (int)((g.rows + tile_rows - 1) / tile_rows);
        a.ny = a.n_ctile;
        a.band = tile_band(a.m_tiles, a.ny, pair ? sms / 2 : sms);
        int64_t total = (int64_t)a.m_tiles * a.ny * g.ncls;
        if (total >= ((int64_t)1 << 30)) return LBT_ERR_UNSUPPORTED;
        if (pair) total = split_last_round(&a, total, sms / 2);
        a.total_tiles = (int)total;
        a.epi_alt = (!pair && a.epi_warps == 8) ? 1 : 0;
        // output rows == tile rows (no halo, one class) and nothing but fp32 to write: TMA-store epilogue
        CUtensorMap tmOut = tmA;
        a.tma_store = 0;
        // (where both apply the TMA store measured faster: 1x1 dgrad 50 against 60 us)
        a.row_direct = (g.C & 7) == 0 && aligned32(dX) && aligned32(accX);
        if (flat && accX == nullptr && (g.C & 3) == 0) {
            if (!make_out_map(&tmOut, dX, (uint64_t)g.C, (uint64_t)g.rows)) return LBT_ERR_CUDA;
            a.tma_store = 1;
            a.row_direct = 0;
        }
        // Register-direct stores leave through the port that also carries the read requests of the TMA loads: spread
        // over four warps instead of eight they disturb the main loop of the next tile less (3x3 256-channel dgrad:
        // 723 -> 629 clocks per step, 39.4 -> 36.8 us); with very short main loops (the stride-2 layers: at most 16 steps) the
        // eight warps stay, there the epilogue itself is what a tile waits for
        if (pair && a.row_direct && a.epi_warps == 8) {
            int most_taps = 0;
            for (int cls = 0; cls < g.ncls; ++cls) most_taps = std::max(most_taps, a.cls_begin[cls + 1] - a.cls_begin[cls]);
            if (most_taps * a.kc_per_tap > 16) a.epi_warps = 4;
        }
        if (g.st == 1 && nt > 1) {
            int lo = a.tap_shift[0], hi = a.tap_shift[0];
            for (int t = 1; t < nt; ++t) { lo = std::min(lo, a.tap_shift[t]); hi = std::max(hi, a.tap_shift[t]); }
            const int win_boxes = (kTile + (hi - lo) + kTile - 1) / kTile;
            const int ring_bytes = kStages * kStageBytes - 2 * win_boxes * kTileBytes;
            const int n_b = std::min(pair ? kMaxBStages : kPairStages, ring_bytes / ((pair ? 1 : a.b_boxes) * kTileBytes));   // a pair CTA loads one B box
            if (pair) {
                if (win_boxes <= 3 && n_b >= 4) { a.window = 1; a.win_boxes = win_boxes; a.win_min_shift = lo; a.n_bstages = n_b; a.n_win = 2; a.w_boxes = 0; }
            } else if (win_boxes <= 4) {
                // single-CTA kernel: only with the whole tap-major filter resident beside the window(s) -- loaded
                // once per CTA -- does the window pay (with a B ring it measured slower than one box per tap)
                const int w_bytes = (g.R * g.S * g.K + kTile - 1) / kTile * a.b_boxes * kTileBytes;
                const int all = kStages * kStageBytes;
                const int n_win = w_bytes + 2 * win_boxes * kTileBytes <= all ? 2 : (w_bytes + win_boxes * kTileBytes <= all ? 1 : 0);
                if (a.n_ctile == 1 && n_win > 0) {
                    a.window = 1; a.win_boxes = win_boxes; a.win_min_shift = lo; a.n_bstages = 1; a.n_win = n_win;
                    a.w_boxes = w_bytes / (a.b_boxes * kTileBytes);
                }
            }
        }
        // wgrad reads nothing dgrad writes: launched right behind it (no event record in between), its CTAs
        // may take over the SMs as dgrad's CTAs finish, instead of waiting for the last tile of the last round
        overlap = do_wgrad && chain;
        a.overlap_next = overlap ? 1 : 0;
        a.wait_prev = behind_expand ? 1 : 0;   // set up while the expansion drains, then wait for it
        finish_args(&a);
        timing_begin(LBT_TIME_DGRAD, stream);
        cudaError_t err;
        if (pair) {
            const dim3 grid(2u * (unsigned)std::min<int64_t>(total, sms / 2));
            err = launch_kernel(i8_gemm_pair_kernel, grid, dim3(kGemmThreads), smem, stream, behind_expand, tmA, tmB[0], tmB[0],
                                tmB[0], tmB[0], tmOut, a);
        } else {
            const dim3 grid((unsigned)std::min<int64_t>(total, sms));
            err = launch_kernel(i8_gemm_kernel, grid, dim3(kGemmThreads), smem, stream, behind_expand, tmA, tmB[0], tmB[0],
                                tmB[0], tmB[0], tmOut, a);
        }
        timing_end(LBT_TIME_DGRAD, stream);
        if (err != cudaSuccess || cudaGetLastError() != cudaSuccess) return LBT_ERR_CUDA;
    }
    if (do_wgrad) {
        for (int cls = 0; cls < 4; ++cls) {
            const int c = cls < g.ncls ? cls : 0;
            if (!make_map(&tmB[cls], xg + (size_t)c * g.rows * g.Cp, (uint64_t)g.Cp, (uint64_t)g.rows))
                return LBT_ERR_CUDA;
        }
        const int64_t out_elems = (int64_t)g.K * g.R * g.S * g.C;
        a.mode = 1; a.b_signed = 0; a.scale_b = s_x; a.out = dW; a.window = 0; a.w_boxes = 0; a.dx_stats = nullptr; a.split_n = 0;
        // the plan the workspace was sized for, with at most that many SMs
        const WgradPlan wp = plan_wgrad(g, std::min(sm_count(), kNumSMs));
        const bool pair = wp.pair;
        const int units = wp.units, m_tiles = wp.m_tiles, splits = wp.splits;
        a.kb_total = wp.kb_total;
        a.kb_per_split = wp.kb_per_split;
        a.direct = splits == 1 ? 1 : 2;
        a.part_stride = part_stride(g);
        // eight epilogue warps when the main loop is short -- or when no CTA has a second tile whose main loop the
        // extra traffic could disturb
        a.epi_warps = (a.kb_per_split <= kShortMainLoop || m_tiles * (wp.n_groups > 0 ? wp.n_groups : g.R * g.S) * a.n_ctile * splits <= units) ? 8 : 4;
        a.epi_alt = (!pair && a.epi_warps == 8) ? 1 : 0;
        a.acc = splits == 1 ? accW : part_ws;
        WgradGroups grp;
        wgrad_group(g, &grp);
        a.multi = wp.n_groups > 0 ? 1 : 0;
        a.acc_cols = grp.acc_cols;
        a.win_min_shift = 0;
        for (int t = 0; t < grp.n_taps; ++t) {
            a.tap_shift[t] = grp.shift[t];
            a.tap_aux[t] = grp.cls[t];
            a.tap_rs[t] = grp.rs[t];
        }
        if (a.multi) {
            a.epi_alt = 0;
            for (int i = 0; i < grp.n_groups; ++i) {
                a.grp_first[i] = grp.first[i]; a.grp_count[i] = grp.count[i]; a.grp_min_shift[i] = grp.min_shift[i];
                for (int t = grp.first[i]; t < grp.first[i] + grp.count[i]; ++t) a.tap_shift[t] = grp.shift[t] - grp.min_shift[i];
            }
        }
        // an unsplit reduction of a one-tap filter writes rows of dW as they come: TMA-store epilogue
        CUtensorMap tmOut = tmA;
        a.tma_store = 0;
        a.row_direct = (g.C & 7) == 0 && (splits > 1 ? aligned32(part_ws) : (aligned32(dW) && aligned32(accW)));
        if (splits == 1 && g.R * g.S == 1 && accW == nullptr && (g.C & 3) == 0) {
            if (!make_out_map(&tmOut, dW, (uint64_t)g.C, (uint64_t)g.K)) return LBT_ERR_CUDA;
            a.tma_store = 1;
            a.row_direct = 0;
        }
        a.m_tiles = m_tiles;
        a.ny = (a.multi ? wp.n_groups : g.R * g.S) * a.n_ctile;
        a.band = tile_band(a.m_tiles, a.ny, units);
        a.total_tiles = m_tiles * a.ny * splits;
        // behind dgrad: no wait at the start (dgrad's CTAs release this launch only after their own wait for the
        // expansion) but one at the end; straight behind the expansion: set up early, then wait for it
        a.overlap_prev = overlap ? 1 : 0;
        a.wait_prev = (!do_dgrad && behind_expand) ? 1 : 0;
        a.overlap_next = (chain && splits > 1) ? 1 : 0;   // the reduction of the slabs follows and waits for this grid
        const bool programmatic = overlap || a.wait_prev != 0;
        finish_args(&a);
        timing_begin(LBT_TIME_WGRAD, stream);
        cudaError_t err;
        if (pair) {
            const dim3 grid(2u * (unsigned)std::min(a.total_tiles, units));
            err = launch_kernel(i8_gemm_pair_kernel, grid, dim3(kGemmThreads), smem, stream, programmatic, tmA, tmB[0], tmB[1],
                                tmB[2], tmB[3], tmOut, a);
        } else {
            const dim3 grid((unsigned)std::min(a.total_tiles, units));
            err = launch_kernel(i8_gemm_kernel, grid, dim3(kGemmThreads), smem, stream, programmatic, tmA, tmB[0], tmB[1],
                                tmB[2], tmB[3], tmOut, a);
        }
        timing_end(LBT_TIME_WGRAD, stream);
        if (err != cudaSuccess) return LBT_ERR_CUDA;
        if (cudaGetLastError() != cudaSuccess) return LBT_ERR_CUDA;
        if (splits > 1) {
            if (launch_kernel(finalize_partials_kernel, dim3(expand_grid((out_elems + 3) / 4)), dim3(256), 0, stream, chain,
                              (const int32_t*)part_ws, splits, a.part_stride, out_elems, dW, accW, s_g, s_x) != cudaSuccess ||
                cudaGetLastError() != cudaSuccess)
                return LBT_ERR_CUDA;
        }
    }
    return LBT_OK;
}

// Forward product Y = Q(X) * Q(W) on the same kernels (mode 2): the rows of the output are the cells
// of the Y grid, the reduction runs over taps x channels, X is read from its parity-class grids with
// the tap offsets wgrad uses, W is read as [K][taps * Cp] with the channels of a tap contiguous.
static lbt_status conv_forward_impl(const lbt_conv_desc* d, const void* q_X, const void* q_W, const float* s_x,
                                    const float* s_w, float* Y, int32_t* accY, int bits_x, int bits_w,
                                    int32_t* dev_status, void* ws, size_t ws_bytes, cudaStream_t stream,
                                    const uint8_t* x_int8 = nullptr) {
    // x_int8: X already as int8 in the grid layout of this geometry (the patches of the im2col lowering)
    Geometry g;
    lbt_status rc = make_geometry(d, &g);
    if (rc != LBT_OK) return rc;
    if (q_X == nullptr || q_W == nullptr || s_x == nullptr || s_w == nullptr || Y == nullptr) return LBT_ERR_INVALID_ARG;
    if (!bits_ok(bits_x) || !bits_ok(bits_w)) return LBT_ERR_UNSUPPORTED_BITS;
    if (!aligned16(q_X) || !aligned16(q_W) || !aligned16(Y) || !aligned16(accY)) return LBT_ERR_ALIGNMENT;
    if ((double)g.C * g.R * g.S * (double)((1 << bits_x) - 1) * (double)(1 << (bits_w - 1)) >= 2147483648.0)
        return LBT_ERR_ACC_RANGE;
    if ((int64_t)g.N * g.P * g.Q >= (int64_t)1 << 31 || (int64_t)g.R * g.S * g.Cp >= (int64_t)1 << 31)
        return LBT_ERR_UNSUPPORTED;
    const Workspace w = carve(g);
    if (ws == nullptr || ws_bytes < (x_int8 != nullptr ? w.total_nowgrad : conv_workspace(g, false))) return LBT_ERR_WORKSPACE;
    rc = ensure_smem_attr();
    if (rc != LBT_OK) return rc;
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(ws) + 255) & ~(uintptr_t)255) - 256;
    {
        // very few input channels: the linear layer over explicit patches (W[k][r][s][c] is its [O][I] weight)
        lbt_conv_desc lin;
        Geometry g2;
        if (x_int8 == nullptr && im2col_geometry(g, &lin, &g2)) {
            uint8_t* patches = base + carve(g2).off_x;
            launch_im2col(g, g2, q_X, bits_x, patches, stream);
            if (cudaGetLastError() != cudaSuccess) return LBT_ERR_CUDA;
            return conv_forward_impl(&lin, q_X, q_W, s_x, s_w, Y, accY, bits_x, bits_w, dev_status, ws, ws_bytes, stream, patches);
        }
    }
    uint8_t* wk = base + w.off_wt;     // K x (taps * Cp) int8
    const uint8_t* xg = x_int8 != nullptr ? x_int8 : base + w.off_x;      // parity classes of X on the cell grid
    int32_t* status = dev_status != nullptr ? dev_status : reinterpret_cast<int32_t*>(base + w.off_status);
    if (dev_status == nullptr) LBT_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), stream));

    timing_begin(LBT_TIME_EXPAND, stream);
    const bool flat = g.st == 1 && g.Hg == g.H && g.Wg == g.W && g.P == g.H && g.Q == g.W;
    ExpandArgs e{};
    e.Hg = g.Hg; e.Wg = g.Wg; e.st = g.st; e.RS = g.R * g.S; e.K = g.K;
    e.src = static_cast<const uint8_t*>(q_X); e.dst = base + w.off_x; e.mode = 2; e.packed = bits_x <= 4; e.is_signed = 0;
    e.Cs = g.C; e.chunks = g.Cp / 16; e.rows_total = g.rows * g.ncls; e.rows_per_cls = g.rows;
    e.Hs = g.H; e.Ws = g.W;
    e.identity = flat && g.C == g.Cp;
    ExpandBatch batch;
    if (x_int8 == nullptr) batch.add(e);
    // W[k][r][s][c] is K * R * S "pixels" of C channels: padding the channels to Cp is all it needs
    e.src = static_cast<const uint8_t*>(q_W); e.dst = wk; e.mode = 0; e.packed = bits_w <= 4; e.is_signed = 1;
    e.Hg = 1; e.Wg = 1; e.Hs = 1; e.Ws = 1; e.st = 1;
    e.rows_total = (int64_t)g.K * g.R * g.S; e.rows_per_cls = e.rows_total;
    e.identity = g.C == g.Cp;
    batch.add(e);
    const cudaError_t expand_err = batch.launch(stream);
    timing_end(LBT_TIME_EXPAND, stream);
    if (expand_err != cudaSuccess || cudaGetLastError() != cudaSuccess) return LBT_ERR_CUDA;

    CUtensorMap tmW, tmX[4];
    if (!make_map(&tmW, wk, (uint64_t)g.R * g.S * g.Cp, (uint64_t)g.K)) return LBT_ERR_CUDA;
    for (int cls = 0; cls < 4; ++cls) {
        const int c = cls < g.ncls ? cls : 0;
        if (!make_map(&tmX[cls], xg + (size_t)c * g.rows * g.Cp, (uint64_t)g.Cp, (uint64_t)g.rows)) return LBT_ERR_CUDA;
    }
    const int bn = g.Kp <= 128 ? 128 : 256;
    GemmArgs a{};
    a.mode = 2; a.bn = bn; a.b_boxes = bn / 128; a.n_ctile = (g.Kp + bn - 1) / bn;
    a.mma_n = g.Kp < bn ? g.Kp : bn;
    a.kc_per_tap = (g.Cp + kTile - 1) / kTile;
    a.k_last = g.Cp - (a.kc_per_tap - 1) * kTile;
    a.tap_cols = g.Cp;
    a.K = g.K; a.C = g.K; a.RS = g.R * g.S;              // the epilogue's column count is the number of filters
    a.Hg = g.Hg; a.Wg = g.Wg; a.H = g.P; a.W = g.Q; a.st = 1; a.rows = g.rows;
    a.scale_a = s_x; a.scale_b = s_w; a.a_signed = 0; a.b_signed = 1;
    a.out = Y; a.acc = accY; a.status = status; a.direct = 1;
    for (int r = 0; r < g.R; ++r)
        for (int sx = 0; sx < g.S; ++sx) {
            const int t = r * g.S + sx;
            a.tap_shift[t] = floordiv(r - g.pad, g.st) * g.Wg + floordiv(sx - g.pad, g.st);
            a.tap_aux[t] = (short)(posmod(r - g.pad, g.st) * g.st + posmod(sx - g.pad, g.st));
            a.tap_rs[t] = (short)t;
        }
    a.cls_begin[0] = 0;
    for (int cls = 1; cls <= 4; ++cls) a.cls_begin[cls] = g.R * g.S;
    a.epi_warps = g.R * g.S * a.kc_per_tap <= kShortMainLoop ? 8 : 4;
    const int sms = sm_count();
    const int64_t n128 = ((g.rows + kTile - 1) / kTile) * a.n_ctile;
    const int64_t n256 = ((g.rows + 2 * kTile - 1) / (2 * kTile)) * a.n_ctile;
    const int64_t rounds1 = (n128 + sms - 1) / sms, rounds2 = (n256 + sms / 2 - 1) / (sms / 2);
    const bool pair = bn == 256 && sms >= 2 && 3 * rounds2 <= 4 * rounds1;
    const int tile_rows = pair ? 2 * kTile : kTile;
    a.epi_alt = (!pair && a.epi_warps == 8) ? 1 : 0;
    if (g.st == 1 && g.R * g.S > 1) {
        // one row window of X per reduction chunk serves all taps; a small filter stays resident (see dgrad)
        int lo = a.tap_shift[0], hi = a.tap_shift[0];
        for (int t = 1; t < g.R * g.S; ++t) { lo = std::min(lo, a.tap_shift[t]); hi = std::max(hi, a.tap_shift[t]); }
        const int win_boxes = (kTile + (hi - lo) + kTile - 1) / kTile;
        const int ring_bytes = kStages * kStageBytes - 2 * win_boxes * kTileBytes;
        const int n_b = std::min(pair ? kMaxBStages : kPairStages, ring_bytes / ((pair ? 1 : a.b_boxes) * kTileBytes));
        if (pair) {
            if (win_boxes <= 3 && n_b >= 4) { a.window = 1; a.win_boxes = win_boxes; a.win_min_shift = lo; a.n_bstages = n_b; a.n_win = 2; a.w_boxes = 0; }
        } else if (win_boxes <= 4) {
            const int w_bytes = (g.R * g.S * g.Cp + kTile - 1) / kTile * a.b_boxes * kTileBytes;   // 128-byte column boxes of W
            const bool cols_ok = kTile % g.Cp == 0 || g.Cp % kTile == 0;                              // a tap's chunk never straddles a box
            const int all = kStages * kStageBytes;
            const int n_win = w_bytes + 2 * win_boxes * kTileBytes <= all ? 2 : (w_bytes + win_boxes * kTileBytes <= all ? 1 : 0);
            if (a.n_ctile == 1 && cols_ok && n_win > 0) {
                a.window = 1; a.win_boxes = win_boxes; a.win_min_shift = lo; a.n_bstages = 1; a.n_win = n_win;
                a.w_boxes = w_bytes / (a.b_boxes * kTileBytes);
            }
        }
    }
    // output rows == tile rows (the Y grid has no halo) and nothing but fp32 to write: TMA-store epilogue
    CUtensorMap tmOut = tmW;
    a.tma_store = 0;
    a.row_direct = (g.K & 7) == 0 && aligned32(Y) && aligned32(accY);
    if (g.Hg == g.P && g.Wg == g.Q && accY == nullptr && (g.K & 3) == 0) {
        if (!make_out_map(&tmOut, Y, (uint64_t)g.K, (uint64_t)g.rows)) return LBT_ERR_CUDA;
        a.tma_store = 1;
        a.row_direct = 0;
    }
    if (pair && a.row_direct && g.R * g.S * a.kc_per_tap > 16) a.epi_warps = 4;   // (see the dgrad launch)
    a.m_tiles = (int)((g.rows + tile_rows - 1) / tile_rows);
    a.ny = a.n_ctile;
    a.band = tile_band(a.m_tiles, a.ny, pair ? sms / 2 : sms);
    int64_t total = (int64_t)a.m_tiles * a.ny;
    if (total >= ((int64_t)1 << 30)) return LBT_ERR_UNSUPPORTED;
    if (pair) total = split_last_round(&a, total, sms / 2);
    a.total_tiles = (int)total;
    const size_t smem = kGemmSmemBytes;
    // no timing tap armed and the expansion is the launch right before: set up while it drains, then wait for it
    const bool behind_expand = !any_tap_armed() && batch.jobs.n > 0;
    a.wait_prev = behind_expand ? 1 : 0;
    finish_args(&a);
    timing_begin(LBT_TIME_FORWARD, stream);
    cudaError_t err;
    if (pair) {
        const dim3 grid(2u * (unsigned)std::min<int64_t>(total, sms / 2));
        err = launch_kernel(i8_gemm_pair_kernel, grid, dim3(kGemmThreads), smem, stream, behind_expand, tmW, tmX[0], tmX[1],
                            tmX[2], tmX[3], tmOut, a);
    } else {
        const dim3 grid((unsigned)std::min<int64_t>(total, sms));
        err = launch_kernel(i8_gemm_kernel, grid, dim3(kGemmThreads), smem, stream, behind_expand, tmW, tmX[0], tmX[1],
                            tmX[2], tmX[3], tmOut, a);
    }
    timing_end(LBT_TIME_FORWARD, stream);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? LBT_OK : LBT_ERR_CUDA;
}

static bool gemm_as_conv(int64_t M, int64_t O, int64_t I, lbt_conv_desc* d) {
    if (M <= 0 || O <= 0 || I <= 0 || M >= ((int64_t)1 << 31) || O >= (1 << 30) || I >= (1 << 30)) return false;
    d->N = (int32_t)M; d->C = (int32_t)I; d->H = 1; d->W = 1; d->K = (int32_t)O; d->R = 1; d->S = 1;
    d->stride = 1; d->pad = 0;
    return true;
}

// ------------------------------------------------------------------------------------------
// Built-in scratch for lbt_qgemm_dgrad_static: callers that may not allocate device memory get
// the workspace from this array, which is part of the library's device image on every GPU.
// In host code the array's name is only a handle for the runtime, not a device address; the
// address a kernel (or a tensor map) can use comes from cudaGetSymbolAddress, looked up once per
// device with that device current.
// ------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[LBT_STATIC_SCRATCH_BYTES];

static lbt_status static_scratch_address(void** out) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static void* address[kMaxDevices];
    static bool known[kMaxDevices];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LBT_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!known[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return LBT_ERR_CUDA;
        address[dev] = p;
        known[dev] = true;
    }
    *out = address[dev];
    return LBT_OK;
}

}  // namespace lbt

using namespace lbt;

extern "C" lbt_status lbt_selftest_wait_timeout(int32_t* dev_status, uint32_t limit_us, void* cuda_stream) {
    if (dev_status == nullptr || limit_us == 0 || limit_us > 1000000u) return LBT_ERR_INVALID_ARG;
    selftest_wait_kernel<<<1, 32, 0, as_stream(cuda_stream)>>>(dev_status, (uint64_t)limit_us * 1000ull);
    return launch_status();
}

extern "C" size_t lbt_workspace_bytes(int op, const void* desc) {
    lbt_conv_desc d;
    if (op == LBT_OP_GEMM_DGRAD || op == LBT_OP_GEMM_WGRAD || op == LBT_OP_GEMM_FORWARD) {
        if (desc == nullptr) return 0;
        const lbt_gemm_desc* gd = static_cast<const lbt_gemm_desc*>(desc);
        if (!gemm_as_conv(gd->M, gd->O, gd->I, &d)) return 0;
    } else if (op == LBT_OP_CONV_BACKWARD || op == LBT_OP_CONV_FORWARD) {
        if (desc == nullptr) return 0;
        d = *static_cast<const lbt_conv_desc*>(desc);
    } else {
        return 0;
    }
    Geometry g;
    if (make_geometry(&d, &g) != LBT_OK) return 0;
    return conv_workspace(g, op == LBT_OP_GEMM_WGRAD || op == LBT_OP_CONV_BACKWARD);
}

extern "C" lbt_status lbt_qgemm_dgrad(const void* q_dY, const void* q_W, const float* d_scale_g,
                                      const float* d_scale_w, float* dX, int32_t* acc_out, int64_t M, int64_t O,
                                      int64_t I, int bits_g, int bits_w, int32_t* dev_status, void* ws,
                                      size_t ws_bytes, void* cuda_stream) {
    lbt_conv_desc d;
    if (!gemm_as_conv(M, O, I, &d) || dX == nullptr) return LBT_ERR_INVALID_ARG;
    return conv_backward_impl(&d, q_dY, q_W, nullptr, d_scale_g, d_scale_w, nullptr, dX, nullptr, acc_out, nullptr,
                              bits_g, bits_w, 4, dev_status, ws, ws_bytes, as_stream(cuda_stream));
}

extern "C" lbt_status lbt_qgemm_dgrad_static(const void* q_dY, const void* q_W, const float* d_scale_g,
                                             const float* d_scale_w, float* dX, int32_t* acc_out, int64_t M,
                                             int64_t O, int64_t I, int bits_g, int bits_w, int32_t* dev_status,
                                             void* cuda_stream) {
    lbt_conv_desc d;
    if (!gemm_as_conv(M, O, I, &d) || dX == nullptr) return LBT_ERR_INVALID_ARG;
    Geometry g;
    const lbt_status rc = make_geometry(&d, &g);
    if (rc != LBT_OK) return rc;
    if (carve(g).total_nowgrad > (size_t)LBT_STATIC_SCRATCH_BYTES) return LBT_ERR_SCRATCH_LIMIT;
    void* scratch = nullptr;
    const lbt_status rs = static_scratch_address(&scratch);
    if (rs != LBT_OK) return rs;
    // Every byte of the scratch that the kernels read (int8 operand copies, the status word when the
    // caller passes none) is rewritten by this call first, so stale contents never matter.
    return conv_backward_impl(&d, q_dY, q_W, nullptr, d_scale_g, d_scale_w, nullptr, dX, nullptr, acc_out, nullptr,
                              bits_g, bits_w, 4, dev_status, scratch, (size_t)LBT_STATIC_SCRATCH_BYTES,
                              as_stream(cuda_stream));
}

extern "C" lbt_status lbt_qgemm_wgrad(const void* q_dY, const void* q_X, const float* d_scale_g,
                                      const float* d_scale_x, float* dW, int32_t* acc_out, int64_t M, int64_t O,
                                      int64_t I, int bits_g, int bits_x, int32_t* dev_status, void* ws,
                                      size_t ws_bytes, void* cuda_stream) {
    lbt_conv_desc d;
    if (!gemm_as_conv(M, O, I, &d) || dW == nullptr) return LBT_ERR_INVALID_ARG;
    return conv_backward_impl(&d, q_dY, nullptr, q_X, d_scale_g, nullptr, d_scale_x, nullptr, dW, nullptr, acc_out,
                              bits_g, 4, bits_x, dev_status, ws, ws_bytes, as_stream(cuda_stream));
}

extern "C" lbt_status lbt_qconv_dgrad_wgrad(const lbt_conv_desc* d, const void* q_dY, const void* q_W,
                                            const void* q_X, const float* d_scale_g, const float* d_scale_w,
                                            const float* d_scale_x, float* dX, float* dW, int32_t* accX,
                                            int32_t* accW, int bits_g, int bits_w, int bits_x, int32_t* dev_status,
                                            void* ws, size_t ws_bytes, void* cuda_stream) {
    return conv_backward_impl(d, q_dY, q_W, q_X, d_scale_g, d_scale_w, d_scale_x, dX, dW, accX, accW, bits_g,
                              bits_w, bits_x, dev_status, ws, ws_bytes, as_stream(cuda_stream));
}

static lbt_status qconv_backward_impl(const lbt_conv_desc* d, const float* dY, const void* q_W, const void* q_X,
                                      const float* d_scale_w, const float* d_scale_x, lbt_interval_state* st,
                                      lbt_grad_stats_t* stats, void* q_dY_out, float* dX, float* dW, int32_t* accX,
                                      int32_t* accW, int bits_g, void* ws, size_t ws_bytes, bool stats_ready,
                                      lbt_grad_stats_t* dx_stats, void* cuda_stream) {
    Geometry g;
    lbt_status rc = make_geometry(d, &g);
    if (rc != LBT_OK) return rc;
    if (dY == nullptr || st == nullptr || stats == nullptr || q_dY_out == nullptr) return LBT_ERR_INVALID_ARG;
    if (dx_stats != nullptr && (dX == nullptr || dx_stats == stats)) return LBT_ERR_INVALID_ARG;
    if (!bits_ok(bits_g)) return LBT_ERR_UNSUPPORTED_BITS;
    if (ws == nullptr || ws_bytes < conv_workspace(g, true)) return LBT_ERR_WORKSPACE;
    const uint64_t n = (uint64_t)g.N * g.P * g.Q * g.K;
    if (!aligned16(dY) || !aligned16(q_dY_out) || (reinterpret_cast<uintptr_t>(dx_stats) & 7u)) return LBT_ERR_ALIGNMENT;
    // the statistics of dX start from zero; cleared first so that no memset sits between the chained launches
    if (dx_stats != nullptr) LBT_CUDA_TRY(cudaMemsetAsync(dx_stats, 0, sizeof(lbt_grad_stats_t), as_stream(cuda_stream)));
    // When the cell grid is the tensor itself (no halo, one class, channels a multiple of 16) the
    // quantizer writes the int8 operand of the contractions directly (4-bit codes: a second output;
    // wider codes: q_dY_out already is that operand) and no expansion pass over dY is needed.
    const bool flat = g.st == 1 && g.Hg == g.H && g.Wg == g.W && g.P == g.H && g.Q == g.W && g.K == g.Kp;
    const bool contract = dX != nullptr || dW != nullptr;
    uint8_t* grid_dy = nullptr;
    if (flat && contract) {
        uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(ws) + 255) & ~(uintptr_t)255) - 256;
        grid_dy = bits_g <= 4 ? base + carve(g).off_dy : static_cast<uint8_t*>(q_dY_out);
    }
    uint8_t* q8 = bits_g <= 4 ? grid_dy : nullptr;
    // A gradient tensor that L2 can hold goes through one cooperative launch (statistics, grid barrier,
    // quantizer, update): its second reading comes from L2 and two launches are saved.  Larger tensors
    // keep the three streaming launches.  With the statistics already in place (stats_ready: the dgrad
    // epilogue of the layer behind wrote them) the abs-max pass is skipped: dY is read once.
    bool fused = false;
    if (!stats_ready && n * sizeof(float) <= kFusedQuantizeBytes) {
        rc = launch_fused_quantize(dY, n, st, stats, static_cast<uint8_t*>(q_dY_out), q8, as_stream(cuda_stream), &fused,
                                   bits_g);
        if (rc != LBT_OK) return rc;
    }
    if (!fused) {
        if (!stats_ready) {
            rc = lbt_grad_stats(dY, n, st, stats, nullptr, 0, cuda_stream);
            if (rc != LBT_OK) return rc;
        }
        rc = launch_quantize(dY, n, st, stats, static_cast<uint8_t*>(q_dY_out), q8,
                             /*clear_n_out=*/stats_ready, as_stream(cuda_stream), 0, bits_g);   // lbt_grad_stats clears n_out itself
        if (rc != LBT_OK) return rc;
        rc = lbt_update_interval(st, stats, cuda_stream);
        if (rc != LBT_OK) return rc;
    }
    if (!contract) return LBT_OK;
    return conv_backward_impl(d, q_dY_out, q_W, q_X, &stats->scale, d_scale_w, d_scale_x, dX, dW, accX, accW, bits_g,
                              4, 4, &st->dev_status, ws, ws_bytes, as_stream(cuda_stream), grid_dy, nullptr,
                              /*behind_quantizer=*/fused, dx_stats);
}

extern "C" lbt_status lbt_qconv_backward(const lbt_conv_desc* d, const float* dY, const void* q_W, const void* q_X,
                                         const float* d_scale_w, const float* d_scale_x, lbt_interval_state* st,
                                         lbt_grad_stats_t* stats, void* q_dY_out, float* dX, float* dW,
                                         int32_t* accX, int32_t* accW, int bits_g, void* ws, size_t ws_bytes,
                                         void* cuda_stream) {
    return qconv_backward_impl(d, dY, q_W, q_X, d_scale_w, d_scale_x, st, stats, q_dY_out, dX, dW, accX, accW, bits_g, ws,
                               ws_bytes, false, nullptr, cuda_stream);
}

extern "C" lbt_status lbt_qconv_backward_ex(const lbt_conv_desc* d, const float* dY, const void* q_W, const void* q_X,
                                            const float* d_scale_w, const float* d_scale_x, lbt_interval_state* st,
                                            lbt_grad_stats_t* stats, void* q_dY_out, float* dX, float* dW,
                                            int32_t* accX, int32_t* accW, int bits_g, void* ws, size_t ws_bytes,
                                            int dy_stats_ready, lbt_grad_stats_t* dx_stats, void* cuda_stream) {
    return qconv_backward_impl(d, dY, q_W, q_X, d_scale_w, d_scale_x, st, stats, q_dY_out, dX, dW, accX, accW, bits_g, ws,
                               ws_bytes, dy_stats_ready != 0, dx_stats, cuda_stream);
}

extern "C" lbt_status lbt_qgemm_forward(const void* q_X, const void* q_W, const float* d_scale_x,
                                        const float* d_scale_w, float* Y, int32_t* acc_out, int64_t M, int64_t O,
                                        int64_t I, int bits_x, int bits_w, int32_t* dev_status, void* ws,
                                        size_t ws_bytes, void* cuda_stream) {
    lbt_conv_desc d;
    if (!gemm_as_conv(M, O, I, &d)) return LBT_ERR_INVALID_ARG;
    return conv_forward_impl(&d, q_X, q_W, d_scale_x, d_scale_w, Y, acc_out, bits_x, bits_w, dev_status, ws, ws_bytes,
                             as_stream(cuda_stream));
}

extern "C" lbt_status lbt_qconv_forward(const lbt_conv_desc* d, const void* q_X, const void* q_W,
                                        const float* d_scale_x, const float* d_scale_w, float* Y, int32_t* acc_out,
                                        int bits_x, int bits_w, int32_t* dev_status, void* ws, size_t ws_bytes,
                                        void* cuda_stream) {
    return conv_forward_impl(d, q_X, q_W, d_scale_x, d_scale_w, Y, acc_out, bits_x, bits_w, dev_status, ws, ws_bytes,
                             as_stream(cuda_stream));
}

extern "C" lbt_status lbt_dequantize_acc(const int32_t* acc, uint64_t n, const float* d_scale_a,
                                         const float* d_scale_b, float* out, void* cuda_stream) {
    if (d_scale_a == nullptr || d_scale_b == nullptr || (n != 0 && (acc == nullptr || out == nullptr)))
        return LBT_ERR_INVALID_ARG;
    if (n >= ((uint64_t)1 << 62)) return LBT_ERR_INVALID_ARG;
    if (!aligned16(acc) || !aligned16(out)) return LBT_ERR_ALIGNMENT;
    if (n == 0) return LBT_OK;
    finalize_kernel<<<expand_grid((int64_t)n), 256, 0, as_stream(cuda_stream)>>>(acc, out, (int64_t)n, d_scale_a,
                                                                               d_scale_b);
    return launch_status();
}
