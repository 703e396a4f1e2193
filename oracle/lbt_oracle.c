/*
 * lbt_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, single-threaded CPU statement of the quantized backward pass
 * of arXiv 2407.12637 ("Toward INT4 Fixed-Point Training via Exploring
 * Quantization Error for Gradients"): per-layer gradient statistics, the
 * clipping-factor (interval) update, the b-bit gradient quantizer, the two
 * integer backward contractions, and the forward side of the same layer (the
 * weight and activation quantizers of Eq. 2, 3 and the integer forward product).  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it.  It shares no code, header, table
 * or constant with the CUDA library.
 *
 * Arithmetic: `float` is IEEE binary32; build with
 *     gcc -O2 -ffp-contract=off -fno-fast-math
 * so that no multiply-add is fused and every fp32 operation rounds once.
 * Integer contractions accumulate in int64.
 *
 * Pins (see tests/test_oracle_*.py): Philox known answers and a library
 * Philox; closed forms and the half-step / clip-out bounds of Sec. 3.3;
 * power-of-two scale invariance; E(G_L) <= U(G_L) (Eq. 7 vs Eq. 8); the
 * fixed point of Eq. 14; library convolution gradients; adjointness; for the
 * forward side grid points, half-step and saturation bounds, oddness,
 * monotonicity, agreement with the pinned gradient quantizer, a library
 * convolution and matrix product.
 * Parity unpinned: nothing here is checked against the paper's accuracy
 * tables (they need datasets and training).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): counter-based generator  */
/* used for stochastic rounding (Sec. 4.1 names stochastic rounding; the      */
/* generator is this implementation's reading).                                */
/* ------------------------------------------------------------------------- */
void ref_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;   /* Weyl sequence: the key is bumped between rounds */
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* 16 uniform random bits for element i of the call (seed, iter).             */
/* key = seed, counter = (i >> 3, iter); the 128 output bits are eight 16-bit */
/* fields, low half of word 0 first, serving elements 8*blk .. 8*blk+7.       */
uint32_t ref_rand16(uint64_t seed, uint64_t iter, uint64_t i)
{
    uint64_t blk = i >> 3;
    uint32_t ctr[4] = { (uint32_t)blk, (uint32_t)(blk >> 32), (uint32_t)iter, (uint32_t)(iter >> 32) };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    ref_philox4x32_10(ctr, key, out);
    unsigned e = (unsigned)(i & 7u);
    return (out[e >> 1] >> (16u * (e & 1u))) & 0xFFFFu;
}

/* ------------------------------------------------------------------------- */
/* Statistics: g_max = max |g| over the layer (Sec. 3.1), computed over the   */
/* finite elements; non-finite elements are counted.                          */
/* ------------------------------------------------------------------------- */
void ref_grad_stats(const float *dY, uint64_t n, float *g_max, uint64_t *n_nonfinite)
{
    float m = 0.0f;
    uint64_t bad = 0;
    for (uint64_t i = 0; i < n; ++i) {
        float a = fabsf(dY[i]);
        if (!isfinite(a)) { ++bad; continue; }
        if (a > m) m = a;
    }
    *g_max = m;
    *n_nonfinite = bad;
}

/* Clip-out count: #{ i : |g_i| > c } with a strict inequality (Sec. 3.3,     */
/* definition of G_out; Algorithm 1, clip-out ratio numerator).               */
uint64_t ref_clip_count(const float *dY, uint64_t n, float c)
{
    uint64_t cnt = 0;
    for (uint64_t i = 0; i < n; ++i)
        if (fabsf(dY[i]) > c) ++cnt;
    return cnt;
}

/* ------------------------------------------------------------------------- */
/* Gradient quantizer, Eq. (1), (2), (4) with c_g = gamma * g_max (Sec. 3.1). */
/* rounding: 0 = nearest (ties to even), 1 = stochastic (floor + Bernoulli of */
/* the fractional part, 16 random bits per element).                          */
/* Outputs: codes[i] in [-qmax, qmax]; *c_out = c_g; *scale_out = s;          */
/* *n_out = clip-out count of this very quantization.                         */
/* If n_nonfinite != 0 the codes are all 0 and n_out = 0.                     */
/* ------------------------------------------------------------------------- */
void ref_quantize_grad(const float *dY, uint64_t n, float gamma, float g_max,
                       int bits, int rounding, uint64_t seed, uint64_t iter,
                       uint64_t n_nonfinite,
                       int8_t *codes, float *c_out, float *scale_out, uint64_t *n_out)
{
    const int qmax = (1 << (bits - 1)) - 1;          /* 2^(b-1) - 1, Eq. (2)   */
    const float c = gamma * g_max;                   /* clipping value c_g     */
    const float s = c / (float)qmax;                 /* scale factor, Eq. (2)  */
    *c_out = c;
    *scale_out = s;
    if (n_nonfinite != 0) {
        memset(codes, 0, (size_t)n);
        *n_out = 0;
        return;
    }
    uint64_t cnt = 0;
    for (uint64_t i = 0; i < n; ++i) {
        float g = dY[i];
        if (fabsf(g) > c) ++cnt;
        int q = 0;
        if (s > 0.0f) {
            float x = g / s;                                  /* Eq. (1), normalise */
            x = fminf(fmaxf(x, -(float)qmax), (float)qmax);   /* Eq. (2), clip      */
            if (rounding == 0) {
                q = (int)rintf(x);                            /* Eq. (4), rounding  */
            } else {
                float f = floorf(x);
                /* frac(x) = x - floor(x) taken exactly: binary64 holds the difference and  */
                /* its scaling by 2^16 without rounding (|x| <= 127, 24-bit significand)    */
                /* unless -2^-29 < x < 0, where the truncation below is 65535 either way;   */
                /* a binary32 subtraction would round it for small negative x               */
                double frac = (double)x - (double)f;
                uint32_t t = (uint32_t)(frac * 65536.0);      /* exact scale, trunc */
                /* frac < 1 exactly, so trunc(frac 2^16) <= 65535; binary64 rounds 1 - |x| up to  */
                /* 1.0 for negative x closer to zero than 2^-54, which the bound undoes           */
                if (t > 65535u) t = 65535u;
                uint32_t u = ref_rand16(seed, iter, i);
                q = (int)f + (u < t ? 1 : 0);
            }
            if (q > qmax) q = qmax;
            if (q < -qmax) q = -qmax;
        }
        codes[i] = (int8_t)q;
    }
    *n_out = cnt;
}

/* Dequantised value Q(g) = s * code, Eq. (4). */
void ref_dequantize(const int8_t *codes, uint64_t n, float s, float *out)
{
    for (uint64_t i = 0; i < n; ++i) out[i] = s * (float)codes[i];
}

/* ------------------------------------------------------------------------- */
/* Forward-side quantizers, Eq. (1)-(4), with a clipping value c given by the  */
/* caller (Sec. 3.1: learned per layer) and rounding to nearest, ties to even. */
/* Taken in the order the equations give: clip, divide by s, round.            */
/*   weights (zero-centred, Eq. 2):  clip to [-c, c], s = c / (2^(b-1) - 1),   */
/*                                   codes in [-qmax, qmax];                   */
/*   activations (after a ReLU, Eq. 3): clip to [0, c], s = c / (2^b - 1),     */
/*                                   codes in [0, 2^b - 1].                    */
/* If s is not a positive finite number (c <= 0, infinite or not a number)     */
/* every code is 0 and the reported scale is 0.  min/max drop a NaN operand, so a NaN input    */
/* takes the lower end of the interval.                                        */
/* ------------------------------------------------------------------------- */
void ref_quantize_weight(const float *w, uint64_t n, float c, int bits, int8_t *codes, float *scale_out)
{
    const int qmax = (1 << (bits - 1)) - 1;
    const float s = c / (float)qmax;                     /* Eq. (2) */
    if (!(s > 0.0f) || isinf(s)) {
        for (uint64_t i = 0; i < n; ++i) codes[i] = 0;
        *scale_out = 0.0f;
        return;
    }
    for (uint64_t i = 0; i < n; ++i) {
        const float clipped = fminf(fmaxf(w[i], -c), c); /* Eq. (2) */
        const float xn = clipped / s;                    /* Eq. (1) */
        int q = (int)rintf(xn);                          /* Eq. (4) */
        if (q > qmax) q = qmax;
        if (q < -qmax) q = -qmax;
        codes[i] = (int8_t)q;
    }
    *scale_out = s;
}

void ref_quantize_act(const float *x, uint64_t n, float c, int bits, uint8_t *codes, float *scale_out)
{
    const int levels = (1 << bits) - 1;
    const float s = c / (float)levels;                   /* Eq. (3) */
    if (!(s > 0.0f) || isinf(s)) {
        for (uint64_t i = 0; i < n; ++i) codes[i] = 0;
        *scale_out = 0.0f;
        return;
    }
    for (uint64_t i = 0; i < n; ++i) {
        const float clipped = fminf(fmaxf(x[i], 0.0f), c); /* Eq. (3) */
        const float xn = clipped / s;                      /* Eq. (1) */
        int q = (int)rintf(xn);                            /* Eq. (4) */
        if (q > levels) q = levels;
        if (q < 0) q = 0;
        codes[i] = (uint8_t)q;
    }
    *scale_out = s;
}

/* Storage format (this implementation's choice; the paper fixes none):       */
/* bits <= 4: two's-complement nibbles, element 2j in bits 0-3 and 2j+1 in    */
/* bits 4-7 of byte j, an odd tail padded with 0; bits >= 5: one int8 each.   */
void ref_pack(const int8_t *codes, uint64_t n, int bits, uint8_t *out)
{
    if (bits > 4) { memcpy(out, codes, (size_t)n); return; }
    uint64_t nb = (n + 1) / 2;
    for (uint64_t j = 0; j < nb; ++j) {
        uint8_t lo = (uint8_t)codes[2 * j] & 0xFu;
        uint8_t hi = (2 * j + 1 < n) ? ((uint8_t)codes[2 * j + 1] & 0xFu) : 0u;
        out[j] = (uint8_t)(lo | (hi << 4));
    }
}

/* Inverse of ref_pack for nibble data; is_signed selects sign- or zero-extension. */
void ref_unpack4(const uint8_t *packed, uint64_t n, int is_signed, int16_t *out)
{
    for (uint64_t i = 0; i < n; ++i) {
        unsigned v = (packed[i >> 1] >> (4u * (unsigned)(i & 1u))) & 0xFu;
        out[i] = (int16_t)((is_signed && v >= 8u) ? (int)v - 16 : (int)v);
    }
}

/* ------------------------------------------------------------------------- */
/* Clipping-factor update, Eq. (15), (16) / Algorithm 1:                      */
/*   gamma_i = gamma_{i-1} + beta * sign(R_out - alpha / (2^b - 1)),          */
/* R_out = n_out / N.  The comparison is made on n_out * (2^b - 1) versus     */
/* alpha * N in binary64 (both sides of Eq. 16 multiplied by N (2^b - 1)), so */
/* that the sign, including the tie, is decided without a division.           */
/* sign(0) = 0 leaves gamma unchanged.  gamma is clamped to                   */
/* [gamma_min, gamma_max].  With non-finite gradients gamma is unchanged.     */
/* ------------------------------------------------------------------------- */
int ref_update_sign(int bits, float alpha, uint64_t n, uint64_t n_out)
{
    double levels = (double)((1 << bits) - 1);
    double lhs = (double)n_out * levels;
    double rhs = (double)alpha * (double)n;
    return (lhs > rhs) - (lhs < rhs);
}

float ref_update_interval(float gamma, float alpha, float beta, float gamma_min, float gamma_max,
                          int bits, uint64_t n, uint64_t n_out, uint64_t n_nonfinite)
{
    if (n_nonfinite != 0) return gamma;
    int sgn = ref_update_sign(bits, alpha, n, n_out);
    float step = beta * (float)sgn;
    float g = gamma + step;
    g = fminf(fmaxf(g, gamma_min), gamma_max);
    return g;
}

/* ------------------------------------------------------------------------- */
/* Backward contractions as their definitions, int64 sums.                    */
/* Linear layer Y[M,O] = X[M,I] W[O,I]^T:                                      */
/*   dgrad  accX[m,i] = sum_o qdY[m,o] qW[o,i]                                 */
/*   wgrad  accW[o,i] = sum_m qdY[m,o] qX[m,i]                                 */
/* Operand codes are int16 so that signed (dY, W) and unsigned (X) 8-bit       */
/* codes share one routine.                                                   */
/* ------------------------------------------------------------------------- */
int64_t ref_gemm_dgrad_at(const int16_t *qdY, const int16_t *qW, int64_t M, int64_t O, int64_t I,
                          int64_t m, int64_t i)
{
    (void)M;
    int64_t acc = 0;
    for (int64_t o = 0; o < O; ++o)
        acc += (int64_t)qdY[m * O + o] * (int64_t)qW[o * I + i];
    return acc;
}

int64_t ref_gemm_wgrad_at(const int16_t *qdY, const int16_t *qX, int64_t M, int64_t O, int64_t I,
                          int64_t o, int64_t i)
{
    int64_t acc = 0;
    for (int64_t m = 0; m < M; ++m)
        acc += (int64_t)qdY[m * O + o] * (int64_t)qX[m * I + i];
    return acc;
}

/* forward  accY[m,o] = sum_i qX[m,i] qW[o,i]  (the layer itself, on codes) */
int64_t ref_gemm_forward_at(const int16_t *qX, const int16_t *qW, int64_t M, int64_t O, int64_t I,
                            int64_t m, int64_t o)
{
    (void)M; (void)O;
    int64_t acc = 0;
    for (int64_t i = 0; i < I; ++i)
        acc += (int64_t)qX[m * I + i] * (int64_t)qW[o * I + i];
    return acc;
}

/* flat output indices [begin, end) of accY (row-major [M, O]) */
void ref_gemm_forward_range(const int16_t *qX, const int16_t *qW, int64_t M, int64_t O, int64_t I,
                            int64_t begin, int64_t end, int64_t *acc)
{
    for (int64_t idx = begin; idx < end; ++idx)
        acc[idx - begin] = ref_gemm_forward_at(qX, qW, M, O, I, idx / O, idx % O);
}

void ref_gemm_forward_list(const int16_t *qX, const int16_t *qW, int64_t M, int64_t O, int64_t I,
                           const int64_t *idx, int64_t cnt, int64_t *acc)
{
    for (int64_t t = 0; t < cnt; ++t)
        acc[t] = ref_gemm_forward_at(qX, qW, M, O, I, idx[t] / O, idx[t] % O);
}

/* flat output indices [begin, end) of accX (row-major [M, I]) */
void ref_gemm_dgrad_range(const int16_t *qdY, const int16_t *qW, int64_t M, int64_t O, int64_t I,
                          int64_t begin, int64_t end, int64_t *acc)
{
    for (int64_t idx = begin; idx < end; ++idx)
        acc[idx - begin] = ref_gemm_dgrad_at(qdY, qW, M, O, I, idx / I, idx % I);
}

/* flat output indices [begin, end) of accW (row-major [O, I]) */
void ref_gemm_wgrad_range(const int16_t *qdY, const int16_t *qX, int64_t M, int64_t O, int64_t I,
                          int64_t begin, int64_t end, int64_t *acc)
{
    for (int64_t idx = begin; idx < end; ++idx)
        acc[idx - begin] = ref_gemm_wgrad_at(qdY, qX, M, O, I, idx / I, idx % I);
}

void ref_gemm_dgrad_list(const int16_t *qdY, const int16_t *qW, int64_t M, int64_t O, int64_t I,
                         const int64_t *idx, int64_t cnt, int64_t *acc)
{
    for (int64_t t = 0; t < cnt; ++t)
        acc[t] = ref_gemm_dgrad_at(qdY, qW, M, O, I, idx[t] / I, idx[t] % I);
}

void ref_gemm_wgrad_list(const int16_t *qdY, const int16_t *qX, int64_t M, int64_t O, int64_t I,
                         const int64_t *idx, int64_t cnt, int64_t *acc)
{
    for (int64_t t = 0; t < cnt; ++t)
        acc[t] = ref_gemm_wgrad_at(qdY, qX, M, O, I, idx[t] / I, idx[t] % I);
}

/* Convolution, NHWC activations / gradients, KRSC weights:                    */
/*   Y[n,p,q,k] = sum_{r,s,c} X[n, p*st + r - pad, q*st + s - pad, c] W[k,r,s,c] */
/*   P = (H + 2 pad - R)/st + 1, Q likewise.                                   */
typedef struct {
    int64_t N, C, H, W, K, R, S, stride, pad, P, Q;
} ref_conv_shape;

/* dgrad: accX[n,h,w,c] = sum_{k,r,s} qdY[n,p,q,k] qW[k,r,s,c] over the (r,s)   */
/* for which p = (h + pad - r)/st and q = (w + pad - s)/st are integers in range */
int64_t ref_conv_dgrad_at(const ref_conv_shape *d, const int16_t *qdY, const int16_t *qW,
                          int64_t n, int64_t h, int64_t w, int64_t c)
{
    int64_t acc = 0;
    for (int64_t r = 0; r < d->R; ++r) {
        int64_t ph = h + d->pad - r;
        if (ph < 0 || ph % d->stride != 0) continue;
        int64_t p = ph / d->stride;
        if (p >= d->P) continue;
        for (int64_t s = 0; s < d->S; ++s) {
            int64_t qw = w + d->pad - s;
            if (qw < 0 || qw % d->stride != 0) continue;
            int64_t q = qw / d->stride;
            if (q >= d->Q) continue;
            const int16_t *gy = qdY + ((n * d->P + p) * d->Q + q) * d->K;
            for (int64_t k = 0; k < d->K; ++k)
                acc += (int64_t)gy[k] * (int64_t)qW[((k * d->R + r) * d->S + s) * d->C + c];
        }
    }
    return acc;
}

/* wgrad: accW[k,r,s,c] = sum_{n,p,q} qdY[n,p,q,k] qX[n, p*st + r - pad, q*st + s - pad, c], */
/* taps that fall outside the image contribute 0                                              */
int64_t ref_conv_wgrad_at(const ref_conv_shape *d, const int16_t *qdY, const int16_t *qX,
                          int64_t k, int64_t r, int64_t s, int64_t c)
{
    int64_t acc = 0;
    for (int64_t n = 0; n < d->N; ++n)
        for (int64_t p = 0; p < d->P; ++p) {
            int64_t h = p * d->stride + r - d->pad;
            if (h < 0 || h >= d->H) continue;
            for (int64_t q = 0; q < d->Q; ++q) {
                int64_t w = q * d->stride + s - d->pad;
                if (w < 0 || w >= d->W) continue;
                acc += (int64_t)qdY[((n * d->P + p) * d->Q + q) * d->K + k] *
                       (int64_t)qX[((n * d->H + h) * d->W + w) * d->C + c];
            }
        }
    return acc;
}

/* forward: accY[n,p,q,k] = sum_{r,s,c} qX[n, p*st + r - pad, q*st + s - pad, c] qW[k,r,s,c], */
/* taps that fall outside the image contribute 0                                               */
int64_t ref_conv_forward_at(const ref_conv_shape *d, const int16_t *qX, const int16_t *qW,
                            int64_t n, int64_t p, int64_t q, int64_t k)
{
    int64_t acc = 0;
    for (int64_t r = 0; r < d->R; ++r) {
        int64_t h = p * d->stride + r - d->pad;
        if (h < 0 || h >= d->H) continue;
        for (int64_t s = 0; s < d->S; ++s) {
            int64_t w = q * d->stride + s - d->pad;
            if (w < 0 || w >= d->W) continue;
            for (int64_t c = 0; c < d->C; ++c)
                acc += (int64_t)qX[((n * d->H + h) * d->W + w) * d->C + c] *
                       (int64_t)qW[((k * d->R + r) * d->S + s) * d->C + c];
        }
    }
    return acc;
}

static void conv_split_y(const ref_conv_shape *d, int64_t idx, int64_t *n, int64_t *p, int64_t *q, int64_t *k)
{
    *k = idx % d->K; idx /= d->K;
    *q = idx % d->Q; idx /= d->Q;
    *p = idx % d->P; idx /= d->P;
    *n = idx;
}

/* flat output indices of accY in NPQK order */
void ref_conv_forward_range(const ref_conv_shape *d, const int16_t *qX, const int16_t *qW,
                            int64_t begin, int64_t end, int64_t *acc)
{
    for (int64_t idx = begin; idx < end; ++idx) {
        int64_t n, p, q, k;
        conv_split_y(d, idx, &n, &p, &q, &k);
        acc[idx - begin] = ref_conv_forward_at(d, qX, qW, n, p, q, k);
    }
}

void ref_conv_forward_list(const ref_conv_shape *d, const int16_t *qX, const int16_t *qW,
                           const int64_t *idx, int64_t cnt, int64_t *acc)
{
    for (int64_t t = 0; t < cnt; ++t) {
        int64_t n, p, q, k;
        conv_split_y(d, idx[t], &n, &p, &q, &k);
        acc[t] = ref_conv_forward_at(d, qX, qW, n, p, q, k);
    }
}

static void conv_split_x(const ref_conv_shape *d, int64_t idx, int64_t *n, int64_t *h, int64_t *w, int64_t *c)
{
    *c = idx % d->C; idx /= d->C;
    *w = idx % d->W; idx /= d->W;
    *h = idx % d->H; idx /= d->H;
    *n = idx;
}

static void conv_split_w(const ref_conv_shape *d, int64_t idx, int64_t *k, int64_t *r, int64_t *s, int64_t *c)
{
    *c = idx % d->C; idx /= d->C;
    *s = idx % d->S; idx /= d->S;
    *r = idx % d->R; idx /= d->R;
    *k = idx;
}

/* flat output indices of accX in NHWC order */
void ref_conv_dgrad_range(const ref_conv_shape *d, const int16_t *qdY, const int16_t *qW,
                          int64_t begin, int64_t end, int64_t *acc)
{
    for (int64_t idx = begin; idx < end; ++idx) {
        int64_t n, h, w, c;
        conv_split_x(d, idx, &n, &h, &w, &c);
        acc[idx - begin] = ref_conv_dgrad_at(d, qdY, qW, n, h, w, c);
    }
}

/* flat output indices of accW in KRSC order */
void ref_conv_wgrad_range(const ref_conv_shape *d, const int16_t *qdY, const int16_t *qX,
                          int64_t begin, int64_t end, int64_t *acc)
{
    for (int64_t idx = begin; idx < end; ++idx) {
        int64_t k, r, s, c;
        conv_split_w(d, idx, &k, &r, &s, &c);
        acc[idx - begin] = ref_conv_wgrad_at(d, qdY, qX, k, r, s, c);
    }
}

void ref_conv_dgrad_list(const ref_conv_shape *d, const int16_t *qdY, const int16_t *qW,
                         const int64_t *idx, int64_t cnt, int64_t *acc)
{
    for (int64_t t = 0; t < cnt; ++t) {
        int64_t n, h, w, c;
        conv_split_x(d, idx[t], &n, &h, &w, &c);
        acc[t] = ref_conv_dgrad_at(d, qdY, qW, n, h, w, c);
    }
}

void ref_conv_wgrad_list(const ref_conv_shape *d, const int16_t *qdY, const int16_t *qX,
                         const int64_t *idx, int64_t cnt, int64_t *acc)
{
    for (int64_t t = 0; t < cnt; ++t) {
        int64_t k, r, s, c;
        conv_split_w(d, idx[t], &k, &r, &s, &c);
        acc[t] = ref_conv_wgrad_at(d, qdY, qX, k, r, s, c);
    }
}

/* Dequantising epilogue: out = (float)acc * fl32(s_a * s_b); the product of   */
/* the two scales is formed first, in binary32.  Returns the number of        */
/* accumulators whose magnitude does not fit int32.                           */
int64_t ref_epilogue(const int64_t *acc, int64_t cnt, float s_a, float s_b, float *out)
{
    float s = s_a * s_b;
    int64_t overflow = 0;
    for (int64_t t = 0; t < cnt; ++t) {
        if (acc[t] > (int64_t)INT32_MAX || acc[t] < (int64_t)INT32_MIN) ++overflow;
        out[t] = (float)acc[t] * s;
    }
    return overflow;
}
