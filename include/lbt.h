/*
 * lbt.h -- C ABI of the B200 (sm_100a) library for the quantized backward pass of
 * arXiv 2407.12637, "Toward INT4 Fixed-Point Training via Exploring Quantization
 * Error for Gradients".
 *
 * One layer, one training iteration:
 *   1. statistics of the full-precision output gradient dY (abs-max; clip-out count),
 *   2. the clipping-factor ("interval") update of Sec. 3.3,
 *   3. b-bit fixed-point quantization of dY (Sec. 3.1),
 *   4. the integer backward contractions dX = Q(dY) Q(W) and dW = Q(dY)^T Q(X), with a
 *      dequantising fp32 epilogue.
 *
 * Conventions, valid for every entry point unless it says otherwise
 *   - Every tensor / struct pointer is a DEVICE pointer owned by the caller and 16-byte aligned.
 *     Only `lbt_conv_desc` / `lbt_gemm_desc` arguments are HOST pointers (read during the call).
 *   - The library allocates no device memory and never synchronises the device: each call
 *     enqueues kernels on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     and returns.  Scratch memory is passed in as `ws` / `ws_bytes`; its size comes from
 *     lbt_workspace_bytes().  Workspace contents are undefined between calls.
 *   - Errors the host can see (bad arguments, unsupported sizes, launch failures) are returned
 *     and nothing is enqueued.  Conditions only the device can see (non-finite gradients, a
 *     bounded wait that ran out) are recorded in a device status word (sticky: the first
 *     non-zero value stays until the caller clears it) and outputs stay defined.
 *   - Layouts: linear layers are row-major, Y[M,O] = X[M,I] W[O,I]^T.  Convolutions use NHWC
 *     activations / gradients and KRSC weights,
 *         Y[n,p,q,k] = sum_{r,s,c} X[n, p*stride + r - pad, q*stride + s - pad, c] W[k,r,s,c].
 *   - Code storage: bit-widths <= 4 are packed two per byte as 4-bit fields, element 2j in bits
 *     0-3 and element 2j+1 in bits 4-7 of byte j (two's complement for signed codes), an odd
 *     tail padded with 0; bit-widths 5..8 take one byte per element.  "Element index" is the
 *     linear index in the buffer as given.
 */
#ifndef LBT_H_
#define LBT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t lbt_status;
enum {
    LBT_OK                   = 0,
    LBT_ERR_INVALID_ARG      = -1,  /* null pointer, non-positive size, inconsistent description */
    LBT_ERR_ALIGNMENT        = -2,  /* a pointer is not 16-byte aligned                            */
    LBT_ERR_UNSUPPORTED_BITS = -3,  /* bit-width outside 2..8                                      */
    LBT_ERR_ACC_RANGE        = -4,  /* the worst-case accumulator does not fit int32              */
    LBT_ERR_WORKSPACE        = -5,  /* ws is null or smaller than lbt_workspace_bytes()           */
    LBT_ERR_CUDA             = -6,  /* a CUDA runtime / driver call failed                        */
    LBT_ERR_NONFINITE        = -7,  /* device-reported: dY holds NaN or Inf                       */
    LBT_ERR_TIMEOUT          = -8,  /* device-reported: a bounded on-chip wait ran out            */
    LBT_ERR_UNSUPPORTED      = -9,  /* a shape this build does not cover (e.g. stride > 2)        */
    LBT_ERR_SCRATCH_LIMIT    = -10, /* the problem needs more than the library's built-in scratch */
    LBT_ERR_BITS_MISMATCH    = -11  /* device-reported: bits_g of lbt_qconv_backward differs from st->bits */
};

enum { LBT_ROUND_NEAREST = 0, LBT_ROUND_STOCHASTIC = 1 };

/*
 * Per-layer interval state (Algorithm 1: hyperparameters b, alpha, beta; input gamma_{i-1};
 * output gamma_i).  Lives in device memory; a plain copy is a checkpoint.
 */
typedef struct lbt_interval_state {
    float    gamma;       /* clipping factor, c_g = gamma * g_max (Sec. 3.1); start at 1.0        */
    float    alpha;       /* ratio of large gradients N(G_L)/N(G) (Sec. 3.2); paper's best 1e-3   */
    float    beta;        /* step of the update, Eq. (15); the paper fixes 1e-3                   */
    float    gamma_min;   /* gamma is clamped to [gamma_min, gamma_max]; the paper keeps gamma in */
    float    gamma_max;   /*   (0, 1]; gamma_max = +inf reproduces the unclamped rule             */
    int32_t  bits;        /* gradient bit-width b, 2..8                                           */
    uint32_t rounding;    /* LBT_ROUND_NEAREST (ties to even) or LBT_ROUND_STOCHASTIC             */
    uint32_t reserved;    /* keeps `seed` 8-byte aligned; write 0                                  */
    uint64_t seed;        /* Philox key                                                           */
    uint64_t iter;        /* Philox stream of the next quantization; ++ in lbt_update_interval    */
    int32_t  dev_status;  /* sticky device-side status word (LBT_OK, LBT_ERR_NONFINITE, ...)      */
    int32_t  reserved2;
} lbt_interval_state;     /* 56 bytes */

/* Per-call statistics of one gradient tensor (device memory). */
typedef struct lbt_grad_stats_t {
    float    g_max;        /* max |dY_i| over the finite elements (Sec. 3.1)                      */
    float    c;            /* clipping value c_g = gamma * g_max                                  */
    float    scale;        /* s = c_g / (2^(b-1) - 1), Eq. (2)                                    */
    uint32_t reserved;     /* scratch of the one-launch quantizer (block counter); 0 between calls   */
    uint64_t n;            /* N(G)                                                                */
    uint64_t n_out;        /* #{ |dY_i| > c_g }, numerator of R(G_out, gamma), Eq. (9)            */
    uint64_t n_nonfinite;  /* #{ dY_i is NaN or Inf }                                             */
} lbt_grad_stats_t;        /* 40 bytes */

/* Linear layer: dY[M,O], W[O,I], X[M,I].  (HOST struct.) */
typedef struct lbt_gemm_desc {
    int64_t M, O, I;
} lbt_gemm_desc;

/* Convolution: X[N,H,W,C], W[K,R,S,C], dY[N,P,Q,K], P = (H + 2 pad - R)/stride + 1.  (HOST struct.) */
typedef struct lbt_conv_desc {
    int32_t N, C, H, W, K, R, S, stride, pad;
} lbt_conv_desc;

enum {
    LBT_OP_GRAD_STATS    = 0,  /* desc ignored                        */
    LBT_OP_QUANTIZE      = 1,  /* desc ignored                        */
    LBT_OP_GEMM_DGRAD    = 2,  /* desc: const lbt_gemm_desc*          */
    LBT_OP_GEMM_WGRAD    = 3,  /* desc: const lbt_gemm_desc*          */
    LBT_OP_CONV_BACKWARD = 4,  /* desc: const lbt_conv_desc*          */
    LBT_OP_GEMM_FORWARD  = 5,  /* desc: const lbt_gemm_desc*          */
    LBT_OP_CONV_FORWARD  = 6   /* desc: const lbt_conv_desc*          */
};

/* Bytes of workspace the operation needs for this description (0 when none; also 0 for an
 * invalid description, which the operation itself then rejects).  Host-only, no CUDA call.
 * The sizes differ by operation: the wgrad contraction (LBT_OP_GEMM_WGRAD, and LBT_OP_CONV_BACKWARD,
 * which covers lbt_qconv_dgrad_wgrad and lbt_qconv_backward) adds room for the int32 partial sums of
 * its split reduction (at most ~20 MB) to what dgrad and the forward product need. */
size_t lbt_workspace_bytes(int op, const void *desc);

/*
 * Statistics, first half (Sec. 3.1: g_max = max(|G|) of one layer).
 * Writes out->g_max, out->n = n, out->n_nonfinite, and clears out->n_out, out->c, out->scale.
 * `st` is not read by this call (it is part of the signature so that the three calls of one
 * iteration take the same arguments); it may be NULL.  n = 0 is valid and gives g_max = 0.
 */
lbt_status lbt_grad_stats(const float *dY, uint64_t n, const lbt_interval_state *st,
                          lbt_grad_stats_t *out, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Quantizer, Eq. (1), (2), (4) with c_g = gamma * g_max, fused with the clip-out count of
 * Sec. 3.3 / Algorithm 1 (the gradients that this very quantization clips):
 *   c = fl32(gamma * g_max); s = fl32(c / qmax), qmax = 2^(b-1) - 1;
 *   x = clamp(fl32(dY_i / s), -qmax, qmax);
 *   nearest:    q = rint(x) (ties to even);
 *   stochastic: q = floor(x) + [u < t], t = trunc(frac(x) * 2^16) with frac(x) = x - floor(x)
 *               taken exactly (no rounding), u = the 16-bit field of
 *               Philox4x32-10(key = seed, counter = (i >> 3, iter)) that belongs to i & 7
 *               (low half of word 0 first);
 *   q_out[i] = clamp(q, -qmax, qmax), packed as the header describes.
 * In:  stats->g_max, stats->n_nonfinite (from lbt_grad_stats on the same dY); st->gamma, bits,
 *      rounding, seed, iter (all read on the device; bits outside 2..8 are clamped into it).
 * Out: stats->c, stats->scale, stats->n_out; q_out (ceil(n/2) bytes for b <= 4, else n bytes).
 * If s == 0 (an all-zero gradient) or n_nonfinite != 0 every code is 0.
 */
lbt_status lbt_quantize_grad(const float *dY, uint64_t n, const lbt_interval_state *st,
                             lbt_grad_stats_t *stats, void *q_out, void *ws, size_t ws_bytes,
                             void *cuda_stream);

/*
 * lbt_grad_stats + lbt_quantize_grad + lbt_update_interval as ONE cooperative launch (Sec. 3.1, 3.3,
 * Eq. 1, 2, 4, 15, 16): every block reduces its share of |dY|, the blocks meet at a bounded grid barrier,
 * quantize with the global g_max and count the clipped elements, and the block that finishes last applies
 * the update.  Same arguments, results (bit for bit) and device-reported conditions as the three calls in
 * sequence; dev_status also becomes LBT_ERR_TIMEOUT if the barrier's 2 s bound runs out.  Meant for
 * gradient tensors that fit L2 (the second reading of dY is then served on-chip and two launches are
 * saved); correct at any size.  With stochastic rounding the random words of each thread's first groups
 * are generated while the first phase waits on memory and kept in up to 36 KB of dynamic shared memory
 * per block.  On a device without cooperative launch it runs the three launches.
 * lbt_qconv_backward takes this path by itself for tensors of at most 112 MiB.
 */
lbt_status lbt_quantize_grad_fused(const float *dY, uint64_t n, lbt_interval_state *st,
                                   lbt_grad_stats_t *stats, void *q_out, void *cuda_stream);

/*
 * Clipping-factor update, Eq. (15), (16) / Algorithm 1:
 *   gamma <- clamp(gamma + beta * sign(n_out / n - alpha / (2^b - 1)), gamma_min, gamma_max),
 * the sign decided on n_out * (2^b - 1) versus alpha * n in binary64, sign(0) = 0; iter <- iter + 1.
 * With stats->n_nonfinite != 0, gamma is left alone and dev_status becomes LBT_ERR_NONFINITE.
 * One thread on the device; no host round trip.
 */
lbt_status lbt_update_interval(lbt_interval_state *st, const lbt_grad_stats_t *stats,
                               void *cuda_stream);

/*
 * Linear-layer backward contractions on the integer tensor cores (the paper motivates integer
 * arithmetic for the backward pass in Sec. 1 and specifies no kernel):
 *   dgrad: dX[m,i] = fl32(s_g * s_w) * sum_o q_dY[m,o] q_W[o,i]
 *   wgrad: dW[o,i] = fl32(s_g * s_x) * sum_m q_dY[m,o] q_X[m,i]
 * q_dY: signed codes of bits_g bits ([M,O]); q_W: signed codes of bits_w bits ([O,I]); q_X:
 * UNSIGNED codes of bits_x bits ([M,I]); storage as the header describes.  d_scale_*: device
 * pointers to one float each.  dX / dW: fp32 outputs.  acc_out (optional, may be NULL): the raw
 * int32 accumulators, same shape as the fp32 output.  dev_status (optional device int32, may be
 * NULL) receives LBT_ERR_TIMEOUT if a bounded wait inside a kernel ran out.
 * LBT_ERR_ACC_RANGE if (reduction length) * max|code_a| * max|code_b| >= 2^31.
 */
lbt_status lbt_qgemm_dgrad(const void *q_dY, const void *q_W, const float *d_scale_g,
                           const float *d_scale_w, float *dX, int32_t *acc_out,
                           int64_t M, int64_t O, int64_t I, int bits_g, int bits_w,
                           int32_t *dev_status, void *ws, size_t ws_bytes, void *cuda_stream);

lbt_status lbt_qgemm_wgrad(const void *q_dY, const void *q_X, const float *d_scale_g,
                           const float *d_scale_x, float *dW, int32_t *acc_out,
                           int64_t M, int64_t O, int64_t I, int bits_g, int bits_x,
                           int32_t *dev_status, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * lbt_qgemm_dgrad for callers that cannot hand over a workspace (the paper has no counterpart;
 * this is a convenience of the library).  Who needs it: code that must not allocate device memory
 * where it calls the library -- a layer hosted inside a framework whose own allocator owns every
 * byte of HBM, a latency-critical loop in which cudaMalloc / cudaFree would stall the device, a
 * process whose memory was reserved in full at start-up so that a later allocation would fail.
 * Same arguments, results and error codes as lbt_qgemm_dgrad, minus `ws` / `ws_bytes`: the scratch
 * is a fixed LBT_STATIC_SCRATCH_BYTES array inside the library's device image (so every GPU that
 * loads the library gives up that much memory until the process exits).
 *   - Returns LBT_ERR_SCRATCH_LIMIT, enqueuing nothing, when
 *     lbt_workspace_bytes(LBT_OP_GEMM_DGRAD, {M,O,I}) exceeds LBT_STATIC_SCRATCH_BYTES
 *     (for instance M = O = I = 1024 fits, 2048 does not).
 *   - It calls no cudaMalloc, cudaFree or other allocating routine.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call before starting any stream capture.
 *   - All calls on a device share the one array.  Each call rewrites every part of it that it later
 *     reads, so nothing needs clearing by the caller and a previous call's leftovers are harmless;
 *     but two calls that overlap on the GPU (different streams, or threads) race on it: keep calls
 *     to this entry point ordered on one stream per device.
 */
#define LBT_STATIC_SCRATCH_BYTES (8u << 20)
lbt_status lbt_qgemm_dgrad_static(const void *q_dY, const void *q_W, const float *d_scale_g,
                                  const float *d_scale_w, float *dX, int32_t *acc_out,
                                  int64_t M, int64_t O, int64_t I, int bits_g, int bits_w,
                                  int32_t *dev_status, void *cuda_stream);

/*
 * Convolution backward contractions alone (codes already quantized), implicit GEMM:
 *   dgrad: dX[n,h,w,c] = fl32(s_g*s_w) * sum_{k,r,s} q_dY[n,p,q,k] q_W[k,r,s,c],
 *          p = (h + pad - r)/stride, q = (w + pad - s)/stride where integral and in range;
 *   wgrad: dW[k,r,s,c] = fl32(s_g*s_x) * sum_{n,p,q} q_dY[n,p,q,k] q_X[n, p*stride + r - pad,
 *          q*stride + s - pad, c], taps outside the image contributing 0.
 * Either output (with its operand) may be NULL to skip that contraction.  stride 1 or 2.
 */
lbt_status lbt_qconv_dgrad_wgrad(const lbt_conv_desc *d, const void *q_dY, const void *q_W,
                                 const void *q_X, const float *d_scale_g, const float *d_scale_w,
                                 const float *d_scale_x, float *dX, float *dW, int32_t *accX,
                                 int32_t *accW, int bits_g, int bits_w, int bits_x,
                                 int32_t *dev_status, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The whole hot path for one convolution layer and one iteration, in stream order:
 *   lbt_grad_stats(dY) -> lbt_quantize_grad (with gamma_{i-1}; counts what it clips)
 *   -> lbt_update_interval (gamma_i for the next iteration) -> dgrad -> wgrad.
 * dY is fp32 [N,P,Q,K]; q_W / q_X are 4-bit codes (signed / unsigned); q_dY_out receives the
 * gradient codes; dX / dW (and their operands) may be NULL to skip a contraction.
 * bits_g must equal st->bits (the host needs it to size q_dY_out and the integer pipeline; the state
 * itself stays on the device).  If the device finds another st->bits, dev_status becomes
 * LBT_ERR_BITS_MISMATCH, the codes are written as zeros in the layout of bits_g (so dX and dW are zero and
 * nothing is written out of bounds) and gamma is left alone.
 * A linear layer is the case H = W = R = S = 1, N = M, C = I, K = O.
 */
lbt_status lbt_qconv_backward(const lbt_conv_desc *d, const float *dY, const void *q_W,
                              const void *q_X, const float *d_scale_w, const float *d_scale_x,
                              lbt_interval_state *st, lbt_grad_stats_t *stats, void *q_dY_out,
                              float *dX, float *dW, int32_t *accX, int32_t *accW, int bits_g,
                              void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * lbt_qconv_backward with the statistics of the NEXT gradient taken where they cost nothing (Sec. 3.1: the
 * quantizer of every layer needs g_max = max |G| over the layer's whole gradient tensor before it can
 * quantize one element, which is a second reading of that tensor).  The gradient a layer receives is the dX
 * the layer behind it has just produced -- directly, where no element-wise operation sits between the two
 * layers -- and the dgrad epilogue holds every element of dX in registers:
 *   dx_stats (device, optional, 8-byte aligned, not the same struct as `stats`): receives g_max = max |dX_i| over
 *     the finite elements, n = the element count of dX and n_nonfinite, exactly as lbt_grad_stats(dX, ...) would
 *     write them (n_out, c, scale cleared); needs dX != NULL.
 *   dy_stats_ready != 0: `stats` already holds g_max, n and n_nonfinite of THIS call's dY (an earlier call's
 *     dx_stats): the abs-max pass over dY is skipped, so dY is read once (4 B + codes per element instead of 8 B).
 *     The caller vouches that they belong to dY; everything else is as in lbt_qconv_backward.
 */
lbt_status lbt_qconv_backward_ex(const lbt_conv_desc *d, const float *dY, const void *q_W,
                                 const void *q_X, const float *d_scale_w, const float *d_scale_x,
                                 lbt_interval_state *st, lbt_grad_stats_t *stats, void *q_dY_out,
                                 float *dX, float *dW, int32_t *accX, int32_t *accW, int bits_g,
                                 void *ws, size_t ws_bytes, int dy_stats_ready,
                                 lbt_grad_stats_t *dx_stats, void *cuda_stream);

/*
 * Forward side of the same layer (Sec. 3.1, Eq. 1-4): the weight and activation quantizers with a
 * clipping value the caller owns (the paper learns it per layer), rounding to nearest (ties to
 * even), and the integer forward product on the same tensor-core kernels.
 *
 * lbt_quantize_weight: zero-centred input, Eq. (2): clip to [-c, c], s = c / (2^(b-1) - 1),
 *   signed codes in [-qmax, qmax].
 * lbt_quantize_act: input after a ReLU, Eq. (3): clip to [0, c], s = c / (2^b - 1), UNSIGNED codes in
 *   [0, 2^b - 1].
 * x: device, n fp32 elements, 16-byte aligned.  d_clip: device pointer to c (one float).  bits: 2..8.
 * q_out: device, 16-byte aligned, the header's storage format (bits <= 4: two codes per byte,
 * (n + 1) / 2 bytes; else n bytes) -- exactly what the q_W / q_X arguments of the contractions take.
 * d_scale_out: device pointer that receives s.  If s is not a positive finite number (c <= 0,
 * infinite or not a number) every code is 0 and s is reported as 0.  min / max drop a NaN operand, so
 * a NaN input takes the lower end of the interval; +-Inf saturate.  One pass: 4 bytes read and 0.5 or
 * 1 byte written per element.
 */
lbt_status lbt_quantize_weight(const float *w, uint64_t n, const float *d_clip, int bits,
                               void *q_out, float *d_scale_out, void *cuda_stream);
lbt_status lbt_quantize_act(const float *x, uint64_t n, const float *d_clip, int bits,
                            void *q_out, float *d_scale_out, void *cuda_stream);

/*
 * Forward product on codes:
 *   linear: Y[m,o]     = fl32(s_x * s_w) * sum_i q_X[m,i] q_W[o,i]
 *   conv:   Y[n,p,q,k] = fl32(s_x * s_w) * sum_{r,s,c} q_X[n, p*st + r - pad, q*st + s - pad, c] q_W[k,r,s,c]
 *           (taps outside the image contribute 0; NHWC / KRSC / NPQK as for the backward calls).
 * q_X: UNSIGNED codes of bits_x bits; q_W: signed codes of bits_w bits.  Y: fp32 output; acc_out
 * (optional): the raw int32 accumulators, same shape.  Workspace: lbt_workspace_bytes with
 * LBT_OP_GEMM_FORWARD / LBT_OP_CONV_FORWARD.  Errors as for the backward contractions
 * (LBT_ERR_ACC_RANGE if C*R*S * (2^bits_x - 1) * 2^(bits_w - 1) >= 2^31).
 */
lbt_status lbt_qgemm_forward(const void *q_X, const void *q_W, const float *d_scale_x,
                             const float *d_scale_w, float *Y, int32_t *acc_out,
                             int64_t M, int64_t O, int64_t I, int bits_x, int bits_w,
                             int32_t *dev_status, void *ws, size_t ws_bytes, void *cuda_stream);
lbt_status lbt_qconv_forward(const lbt_conv_desc *d, const void *q_X, const void *q_W,
                             const float *d_scale_x, const float *d_scale_w, float *Y,
                             int32_t *acc_out, int bits_x, int bits_w, int32_t *dev_status,
                             void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Pieces for batch-sharded (data-parallel) layers that must reproduce the one-GPU result bit for bit.
 * Sec. 3.1 defines g_max, and Sec. 3.3 / Eq. (9) the clip-out ratio, over ALL gradients of a layer, so
 * a layer whose batch is split over ranks reduces them over the ranks (max of g_max, sums of n,
 * n_nonfinite and n_out: plain collectives on the fields of lbt_grad_stats_t, done by the caller between
 * these calls) and sums the integer wgrad accumulators before the dequantising multiply:
 *
 * lbt_quantize_grad_shard: lbt_quantize_grad for a shard whose first element is element
 *   `index_offset` (a multiple of 8, else LBT_ERR_INVALID_ARG) of the whole tensor: the stochastic-
 *   rounding bits of dY[i] are those of element index_offset + i, so the codes equal the matching
 *   slice of the unsharded quantization.  stats->g_max and stats->n_nonfinite must already hold the
 *   reduced values; stats->n_out receives this shard's count.
 * lbt_dequantize_acc: out[i] = (float)acc[i] * fl32(*d_scale_a * *d_scale_b) for n int32 accumulators
 *   (the epilogue of the contractions, applied after the accumulators of all shards have been summed).
 *   acc, out: device, 16-byte aligned.
 */
lbt_status lbt_quantize_grad_shard(const float *dY, uint64_t n, uint64_t index_offset,
                                   const lbt_interval_state *st, lbt_grad_stats_t *stats,
                                   void *q_out, void *cuda_stream);
lbt_status lbt_dequantize_acc(const int32_t *acc, uint64_t n, const float *d_scale_a,
                              const float *d_scale_b, float *out, void *cuda_stream);

/*
 * Diagnostics of Sec. 3.2-3.3 for one quantized gradient tensor (not part of a training step):
 *   E(G)   = sum |g - Q(g)| / (N(G) g_max)                                   Eq. (5)
 *   E(G_L) = the same over the large gradients G_L, split into clip-in / clip-out   Eq. (6), (7)
 *   U(G_L) = (gamma / (2^b - 2) R_in + (1 - gamma) R_out) / (R_in + R_out)    Eq. (8)-(10)
 * G_L is the N(G_L) = alpha N (rounded to nearest, halves to even) gradients of largest magnitude; among
 * equal magnitudes the earlier elements (memory order) belong to it first.  Q(g) = scale * code with the
 * codes and the scale of the quantization being examined; a large gradient is clip-out when |g| > c;
 * gamma is taken as c / g_max.  dY: device, n >= 1 fp32 values (all finite), 16-byte aligned; q_codes:
 * the packed codes lbt_quantize_grad wrote for dY with `bits`; stats: that call's statistics (g_max, c,
 * scale); alpha: host value in [0, 1]; out: device struct; ws: at least lbt_diagnostics_workspace_bytes().
 * Sums are accumulated in binary64 (their last bits depend on the order of accumulation).
 */
typedef struct lbt_grad_diag_t {
    uint64_t n, n_large, n_in, n_out;               /* N(G), N(G_L), N(G_in), N(G_out)              */
    double   sum_all, sum_large_in, sum_large_out;  /* sums of |g - Q(g)|                           */
    double   e_all, e_large, u_large;               /* Eq. (5), Eq. (6) = (7), Eq. (8)              */
    float    threshold;                             /* smallest magnitude in G_L (0 if G_L is empty) */
    uint32_t reserved;
} lbt_grad_diag_t;                                  /* 88 bytes */
size_t lbt_diagnostics_workspace_bytes(void);
lbt_status lbt_grad_diagnostics(const float *dY, uint64_t n, const void *q_codes, int bits, float alpha,
                                const lbt_grad_stats_t *stats, lbt_grad_diag_t *out, void *ws,
                                size_t ws_bytes, void *cuda_stream);

/*
 * Measurement taps (no counterpart in the paper).  After this call the library records the two
 * events (cudaEvent_t passed as void*, created by the caller) on the call's stream immediately
 * before and after every launch of the named kernel class, so that a benchmark can time one
 * kernel inside a fused call with cudaEventElapsedTime.  Passing NULL for both removes the tap.
 * Process-wide and not thread-safe: meant for a benchmark's single thread.
 */
enum {
    LBT_TIME_STATS = 0,     /* abs-max reduction                   */
    LBT_TIME_QUANTIZE = 1,  /* quantize + clip-out count           */
    LBT_TIME_EXPAND = 2,    /* code expansion (all three operands) */
    LBT_TIME_DGRAD = 3,     /* tensor-core contraction for dX      */
    LBT_TIME_WGRAD = 4,     /* tensor-core contraction for dW      */
    LBT_TIME_FORWARD = 5,   /* tensor-core contraction for Y       */
    LBT_TIME_FWD_QUANT = 6, /* weight / activation quantizer       */
    LBT_TIME_CLASSES = 7
};
lbt_status lbt_set_timing_events(int kernel_class, void *ev_start, void *ev_stop);

/*
 * Self-test of the bounded on-chip waits (no counterpart in the paper).  Every wait inside the
 * contraction kernels gives up after a time limit, records LBT_ERR_TIMEOUT and lets the kernel end
 * in an orderly way.  This call runs that very wait routine in a one-thread kernel on a barrier
 * that nothing signals, with a limit of `limit_us` microseconds (1 .. 1 000 000), and stores
 * LBT_ERR_TIMEOUT in *dev_status (device int32, sticky like the other status words) when it
 * expires -- so a deployment can check that a lost signal ends in an error code and a usable
 * context, not in a hang.  Nothing faults and nothing is left running.
 */
lbt_status lbt_selftest_wait_timeout(int32_t *dev_status, uint32_t limit_us, void *cuda_stream);

/*
 * The same self-test for the other kind of bounded wait in the library: the grid barrier of the one-launch
 * quantizer (lbt_quantize_grad_fused), a counter in memory that every block adds to and then polls.  One
 * block arrives at a barrier that expects two, with a limit of `limit_us` microseconds (1 .. 1 000 000);
 * *dev_status becomes LBT_ERR_TIMEOUT when the wait gives up.  Nothing faults and nothing is left running.
 */
lbt_status lbt_selftest_barrier_timeout(int32_t *dev_status, uint32_t limit_us, void *cuda_stream);

/* Static, NUL-terminated name of a status code. */
const char *lbt_status_string(lbt_status status);

#ifdef __cplusplus
}
#endif
#endif /* LBT_H_ */
