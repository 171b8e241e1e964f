/*
 * mqg_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, scalar CPU statement of what the MQGrad data-parallel hot path
 * computes: the worker-side Quantize(g, K) and the server-side De-quantize /
 * sum / update of Algorithm 1 (functions WorkerIterate and ReceiveQGThenSendQG,
 * Section 3.2).  The paper delegates the codec to an external page and prints no
 * formula for it, so every concrete step below follows the reading R1..R14 that
 * this repository fixes for it (symmetric affine grid on [-s,+s] with 2^K levels,
 * max-abs scale per bucket, unbiased stochastic rounding driven by Philox4x32-10,
 * LSB-first bit packing).  Each function names the step it implements.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call this
 * file.  It shares no code, header, table or constant with the CUDA library.
 *
 * Arithmetic: IEEE binary32, round-to-nearest-even, one rounding per named
 * operation, no contraction (build with -ffp-contract=off), fmaf from libm.
 *
 * Pins (tests marked "not gpu"): packing against Python big integers; code range;
 * exactness on dyadic grids; exhaustive enumeration of the 65,536 rounding draws;
 * statistical unbiasedness; exact-rational brute force on <= 16 elements; Philox
 * against an independent library implementation; scale against numpy max.
 * The (min, max) nearest-rounding variant at the end of the file (readings M1..M4) is
 * pinned by exact rational arithmetic, dyadic closed forms, the half-step error bound,
 * monotonicity, end points and saturation.
 * The L2-norm scale variant (readings N1..N3, after the (min, max) variant) is pinned by
 * closed forms where every sum is exact, by inputs built so that another summation order or
 * an unfused square gives another float, by exact rational arithmetic with one rounding per
 * named operation, and by the error bound of its sum against the norm in double precision.
 * The 1-bit error-feedback variant (readings E1..E5, last in the file) is pinned by hand-
 * computed small cases, by the conservation law sent + residual = gradient + old residual on
 * exactly representable data, by numpy means on integer data, by order-sensitive inputs and
 * by the separately pinned (min, max) de-quantizer as its receiver.
 * Parity unpinned: both codecs as a whole against the paper -- the paper prints no
 * worked example, error bound or sample output of Quantize / De-quantize.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as
 * easy as 1, 2, 3", SC'11): ten rounds; each round multiplies counter words 0 and
 * 2 by two fixed odd constants, keeps the 64-bit products, and mixes the high
 * halves with the other two counter words and the round key; the key grows by
 * two Weyl constants between rounds. ------------------------------------------ */
void mqo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* R7: the 16 random bits of element i.  g = elem_offset + i is the element's
 * position in the flat model; one Philox block serves eight consecutive g:
 * counter = (lo32(g>>3), hi32(g>>3), worker, step), key = (lo32(seed), hi32(seed));
 * element g uses half (g&1) of output word ((g&7)>>1). */
void mqo_draw_h(uint64_t seed, uint32_t worker, uint32_t step, uint64_t elem_offset,
                uint64_t n, uint16_t *h)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    for (uint64_t i = 0; i < n; ++i) {
        uint64_t g = elem_offset + i;
        uint64_t blk = g >> 3;
        uint32_t ctr[4] = { (uint32_t)blk, (uint32_t)(blk >> 32), worker, step };
        uint32_t y[4];
        mqo_philox4x32_10(ctr, key, y);
        unsigned e = (unsigned)(g & 7u);
        h[i] = (uint16_t)((y[e >> 1] >> (16u * (e & 1u))) & 0xFFFFu);
    }
}

/* R1: bf16 -> fp32 is exact: the 16 stored bits become the high half. */
void mqo_widen_bf16(const uint16_t *in, uint64_t n, float *out)
{
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t bits = (uint32_t)in[i] << 16;
        memcpy(&out[i], &bits, 4);
    }
}

/* R2 + R3: one scale per bucket of `bucket` consecutive elements (the last bucket
 * may be shorter): s_k = max |x_i|; scales below 2^-96 are flushed to zero. */
void mqo_bucket_scales(const float *x, uint64_t n, uint64_t bucket, float *scales)
{
    const float tiny = ldexpf(1.0f, -96);
    uint64_t nb = (n + bucket - 1) / bucket;
    for (uint64_t k = 0; k < nb; ++k) {
        uint64_t lo = k * bucket, hi = lo + bucket;
        if (hi > n) hi = n;
        float s = 0.0f;
        for (uint64_t i = lo; i < hi; ++i) {
            float a = fabsf(x[i]);
            if (a > s) s = a;
        }
        scales[k] = (s < tiny) ? 0.0f : s;
    }
}

/* R4..R8: stochastic-rounding encode of x to the K-bit grid of its bucket.
 * L = 2^K - 1 levels above zero; t = x * (L / 2s) + L/2 lies in [0, L];
 * the code is floor(t), plus one when the uniform draw u = (h + 1/2) / 2^16
 * falls below the fractional part of t. */
void mqo_encode(const float *x, uint64_t n, int bits, uint64_t bucket,
                const float *scales, const uint16_t *h, uint8_t *q)
{
    const float Lf = (float)((1 << bits) - 1);
    const float halfL = 0.5f * Lf;                       /* exact */
    for (uint64_t i = 0; i < n; ++i) {
        float s = scales[i / bucket];
        if (s == 0.0f) { q[i] = 0; continue; }            /* R3 */
        float two_s = 2.0f * s;
        float inv = Lf / two_s;                           /* R4, one rounding */
        float t = fmaf(x[i], inv, halfL);                 /* R5, one rounding */
        if (t < 0.0f) t = 0.0f;
        if (t > Lf) t = Lf;
        float f = floorf(t);                              /* R6 */
        float r = t - f;                                  /* exact */
        float u = ((float)h[i] + 0.5f) * (1.0f / 65536.0f); /* R7, exact */
        int code = (int)f + ((u < r) ? 1 : 0);            /* R8 */
        q[i] = (uint8_t)code;
    }
}

/* R9: code i occupies bits [i*K, i*K+K) of a little-endian bit stream; bit j of
 * the stream is bit (j mod 32) of 32-bit word floor(j/32).  Written one bit at a
 * time on purpose.  `words` must hold ceil(n*K/32) words; pad bits are zero. */
void mqo_pack(const uint8_t *q, uint64_t n, int bits, uint32_t *words)
{
    uint64_t nwords = (n * (uint64_t)bits + 31) / 32;
    for (uint64_t w = 0; w < nwords; ++w) words[w] = 0;
    for (uint64_t i = 0; i < n; ++i) {
        for (int j = 0; j < bits; ++j) {
            if ((q[i] >> j) & 1u) {
                uint64_t pos = i * (uint64_t)bits + (uint64_t)j;
                words[pos >> 5] |= (uint32_t)1u << (pos & 31u);
            }
        }
    }
}

void mqo_unpack(const uint32_t *words, uint64_t n, int bits, uint8_t *q)
{
    for (uint64_t i = 0; i < n; ++i) {
        unsigned code = 0;
        for (int j = 0; j < bits; ++j) {
            uint64_t pos = i * (uint64_t)bits + (uint64_t)j;
            unsigned bit = (words[pos >> 5] >> (pos & 31u)) & 1u;
            code |= bit << j;
        }
        q[i] = (uint8_t)code;
    }
}

/* R10: x^ = (2q - L) * (s / L); a flushed (zero-scale) bucket decodes to +0. */
void mqo_dequantize(const uint8_t *q, uint64_t n, int bits, uint64_t bucket,
                    const float *scales, float *xhat)
{
    const int L = (1 << bits) - 1;
    const float Lf = (float)L;
    for (uint64_t i = 0; i < n; ++i) {
        float s = scales[i / bucket];
        if (s == 0.0f) { xhat[i] = 0.0f; continue; }
        float hstep = s / Lf;                             /* one rounding */
        float level = (float)(2 * (int)q[i] - L);         /* exact */
        xhat[i] = level * hstep;                          /* one rounding */
    }
}

/* R12: w <- w - lr * g as one fused multiply-add per element (Algorithm 1,
 * WorkerIterate's update; the caller passes lr = eta / P to get the mean). */
void mqo_apply(float *params, const float *acc, float lr, uint64_t n)
{
    for (uint64_t i = 0; i < n; ++i)
        params[i] = fmaf(-lr, acc[i], params[i]);
}

/* ---- compositions with the library's calling shapes ---------------------- */

/* Quantize(g, K): R1..R9 for one worker buffer.  dtype 0 = fp32, 1 = bf16. */
int mqo_quantize(const void *grad, uint64_t n, int bits, uint64_t bucket, uint64_t seed,
                 uint32_t *codes, float *scales, int dtype, uint32_t worker,
                 uint32_t step, uint64_t elem_offset)
{
    if (bits < 1 || bits > 8 || bucket == 0) return -1;
    if (n == 0) return 0;
    float *x = (float *)malloc(n * sizeof(float));
    uint16_t *h = (uint16_t *)malloc(n * sizeof(uint16_t));
    uint8_t *q = (uint8_t *)malloc(n);
    if (!x || !h || !q) { free(x); free(h); free(q); return -2; }
    if (dtype == 1) mqo_widen_bf16((const uint16_t *)grad, n, x);
    else memcpy(x, grad, n * sizeof(float));
    mqo_bucket_scales(x, n, bucket, scales);
    mqo_draw_h(seed, worker, step, elem_offset, n, h);
    mqo_encode(x, n, bits, bucket, scales, h, q);
    mqo_pack(q, n, bits, codes);
    free(x); free(h); free(q);
    return 0;
}

/* ReceiveQGThenSendQG up to the sum: R9^-1, R10, R11 in worker order 0..W-1. */
int mqo_dequant_accumulate(const uint32_t *const *codes, const float *const *scales, int W,
                           int bits, uint64_t n, float *acc, uint64_t bucket, int add_into_acc)
{
    if (bits < 1 || bits > 8 || bucket == 0 || W < 1) return -1;
    if (n == 0) return 0;
    uint8_t *q = (uint8_t *)malloc(n);
    float *xhat = (float *)malloc(n * sizeof(float));
    if (!q || !xhat) { free(q); free(xhat); return -2; }
    for (int w = 0; w < W; ++w) {
        mqo_unpack(codes[w], n, bits, q);
        mqo_dequantize(q, n, bits, bucket, scales[w], xhat);
        if (w == 0 && !add_into_acc) {
            for (uint64_t i = 0; i < n; ++i) acc[i] = xhat[i];
        } else {
            for (uint64_t i = 0; i < n; ++i) acc[i] = acc[i] + xhat[i];
        }
    }
    free(q); free(xhat);
    return 0;
}

/* R13: the server's whole step = R10..R12; acc_out may be NULL. */
int mqo_server_step(const uint32_t *const *codes, const float *const *scales, int W, int bits,
                    uint64_t n, uint64_t bucket, float *params, float lr, float *acc_out)
{
    if (n == 0) return 0;
    float *acc = (float *)malloc(n * sizeof(float));
    if (!acc) return -2;
    int rc = mqo_dequant_accumulate(codes, scales, W, bits, n, acc, bucket, 0);
    if (rc == 0) {
        mqo_apply(params, acc, lr, n);
        if (acc_out) memcpy(acc_out, acc, n * sizeof(float));
    }
    free(acc);
    return rc;
}

/* Downlink of the server (ReceiveQGThenSendQG, lines 3-5): the mean of the de-quantized worker
 * gradients, g = (sum_p g_p) * mean_scale with one rounding for the product, is quantized again
 * with the same K and bucket size (elem_offset 0) for the broadcast. */
int mqo_server_requantize(const uint32_t *const *codes, const float *const *scales, int W, int bits,
                          uint64_t n, uint64_t bucket, float mean_scale, uint64_t seed,
                          uint32_t *codes_out, float *scales_out, uint32_t worker, uint32_t step)
{
    if (n == 0) return 0;
    float *g = (float *)malloc(n * sizeof(float));
    if (!g) return -2;
    int rc = mqo_dequant_accumulate(codes, scales, W, bits, n, g, bucket, 0);
    if (rc == 0) {
        for (uint64_t i = 0; i < n; ++i) g[i] = g[i] * mean_scale;
        rc = mqo_quantize(g, n, bits, bucket, seed, codes_out, scales_out, 0, worker, step, 0);
    }
    free(g);
    return rc;
}

/* Per-layer scale: segment j covers elements [seg_off[j], seg_off[j+1]) of the
 * flat gradient, is one bucket, and its bit stream starts at word code_off[j].
 * Element i of segment j draws with g = elem_offset + seg_off[j] + i. */
int mqo_quantize_segments(const void *grad, int nseg, const uint64_t *seg_off,
                          const uint64_t *code_off, int bits, uint64_t seed,
                          uint32_t *codes, float *scales, int dtype, uint32_t worker,
                          uint32_t step, uint64_t elem_offset)
{
    for (int j = 0; j < nseg; ++j) {
        uint64_t len = seg_off[j + 1] - seg_off[j];
        const char *base = (const char *)grad + seg_off[j] * (dtype == 1 ? 2u : 4u);
        if (len == 0) { scales[j] = 0.0f; continue; }
        int rc = mqo_quantize(base, len, bits, len, seed, codes + code_off[j], &scales[j],
                              dtype, worker, step, elem_offset + seg_off[j]);
        if (rc) return rc;
    }
    return 0;
}

int mqo_server_step_segments(const uint32_t *const *codes, const float *const *scales, int W,
                             int bits, int nseg, const uint64_t *seg_off,
                             const uint64_t *code_off, float *params, float lr, float *acc_out)
{
    const uint32_t **cw = (const uint32_t **)malloc(sizeof(*cw) * (size_t)W);
    const float **sw = (const float **)malloc(sizeof(*sw) * (size_t)W);
    if (!cw || !sw) { free(cw); free(sw); return -2; }
    int rc = 0;
    for (int j = 0; j < nseg && rc == 0; ++j) {
        uint64_t len = seg_off[j + 1] - seg_off[j];
        if (len == 0) continue;
        for (int w = 0; w < W; ++w) {
            cw[w] = codes[w] + code_off[j];
            sw[w] = scales[w] + j;
        }
        rc = mqo_server_step(cw, sw, W, bits, len, len, params + seg_off[j], lr,
                             acc_out ? acc_out + seg_off[j] : NULL);
    }
    free(cw); free(sw);
    return rc;
}

/* ---- codec variant: (min, max) range with nearest rounding ------------------
 * The paper prints no codec; the footnote of Section 3.2 refers to a scheme that
 * maps the range [min, max] of a tensor linearly onto the 2^K codes and rounds to
 * the nearest one.  The readings this repository fixes for it (M1..M4):
 *   M1  per bucket lo = min x_i, hi = max x_i (a zero of either sign is stored as +0);
 *       both are sent: two floats per bucket, ranges[2k] = lo, ranges[2k+1] = hi.
 *   M2  r = fl(hi - lo); a bucket with r < 2^-96 is constant: every code is 0.
 *   M3  code = min(L, floor(fma(fl(x - lo), fl(L / r), 1/2))), L = 2^K - 1
 *       (round half up on the scaled offset; deterministic, no random draws).
 *   M4  x^ = fma(q, fl(r / L), lo); a constant bucket decodes to lo.
 * Sum, update and packing are R9, R11, R12 unchanged.
 */
void mqo_bucket_ranges(const float *x, uint64_t n, uint64_t bucket, float *ranges)
{
    uint64_t nb = (n + bucket - 1) / bucket;
    for (uint64_t k = 0; k < nb; ++k) {
        uint64_t b0 = k * bucket, b1 = b0 + bucket;
        if (b1 > n) b1 = n;
        float lo = x[b0], hi = x[b0];
        for (uint64_t i = b0 + 1; i < b1; ++i) {
            if (x[i] < lo) lo = x[i];
            if (x[i] > hi) hi = x[i];
        }
        ranges[2 * k] = lo + 0.0f;                        /* M1: -0 -> +0 */
        ranges[2 * k + 1] = hi + 0.0f;
    }
}

void mqo_encode_minmax(const float *x, uint64_t n, int bits, uint64_t bucket,
                       const float *ranges, uint8_t *q)
{
    const int L = (1 << bits) - 1;
    const float Lf = (float)L;
    const float tiny = ldexpf(1.0f, -96);
    for (uint64_t i = 0; i < n; ++i) {
        float lo = ranges[2 * (i / bucket)], hi = ranges[2 * (i / bucket) + 1];
        float r = hi - lo;                                /* M2, one rounding */
        if (r < tiny) { q[i] = 0; continue; }
        float inv = Lf / r;                               /* one rounding */
        float d = x[i] - lo;                              /* one rounding */
        float t = fmaf(d, inv, 0.5f);                     /* M3, one rounding */
        int code = (int)floorf(t);
        if (code > L) code = L;
        if (code < 0) code = 0;
        q[i] = (uint8_t)code;
    }
}

void mqo_dequantize_minmax(const uint8_t *q, uint64_t n, int bits, uint64_t bucket,
                           const float *ranges, float *xhat)
{
    const float Lf = (float)((1 << bits) - 1);
    const float tiny = ldexpf(1.0f, -96);
    for (uint64_t i = 0; i < n; ++i) {
        float lo = ranges[2 * (i / bucket)], hi = ranges[2 * (i / bucket) + 1];
        float r = hi - lo;
        if (r < tiny) { xhat[i] = lo; continue; }         /* M4, constant bucket */
        float step = r / Lf;                              /* one rounding */
        xhat[i] = fmaf((float)q[i], step, lo);            /* one rounding */
    }
}

int mqo_quantize_minmax(const void *grad, uint64_t n, int bits, uint64_t bucket,
                        uint32_t *codes, float *ranges, int dtype)
{
    if (bits < 1 || bits > 8 || bucket == 0) return -1;
    if (n == 0) return 0;
    float *x = (float *)malloc(n * sizeof(float));
    uint8_t *q = (uint8_t *)malloc(n);
    if (!x || !q) { free(x); free(q); return -2; }
    if (dtype == 1) mqo_widen_bf16((const uint16_t *)grad, n, x);
    else memcpy(x, grad, n * sizeof(float));
    mqo_bucket_ranges(x, n, bucket, ranges);
    mqo_encode_minmax(x, n, bits, bucket, ranges, q);
    mqo_pack(q, n, bits, codes);
    free(x); free(q);
    return 0;
}

int mqo_dequant_accumulate_minmax(const uint32_t *const *codes, const float *const *ranges, int W,
                                  int bits, uint64_t n, float *acc, uint64_t bucket, int add_into_acc)
{
    if (bits < 1 || bits > 8 || bucket == 0 || W < 1) return -1;
    if (n == 0) return 0;
    uint8_t *q = (uint8_t *)malloc(n);
    float *xhat = (float *)malloc(n * sizeof(float));
    if (!q || !xhat) { free(q); free(xhat); return -2; }
    for (int w = 0; w < W; ++w) {
        mqo_unpack(codes[w], n, bits, q);
        mqo_dequantize_minmax(q, n, bits, bucket, ranges[w], xhat);
        if (w == 0 && !add_into_acc) {
            for (uint64_t i = 0; i < n; ++i) acc[i] = xhat[i];
        } else {
            for (uint64_t i = 0; i < n; ++i) acc[i] = acc[i] + xhat[i];
        }
    }
    free(q); free(xhat);
    return 0;
}

int mqo_server_step_minmax(const uint32_t *const *codes, const float *const *ranges, int W, int bits,
                           uint64_t n, uint64_t bucket, float *params, float lr, float *acc_out)
{
    if (n == 0) return 0;
    float *acc = (float *)malloc(n * sizeof(float));
    if (!acc) return -2;
    int rc = mqo_dequant_accumulate_minmax(codes, ranges, W, bits, n, acc, bucket, 0);
    if (rc == 0) {
        mqo_apply(params, acc, lr, n);
        if (acc_out) memcpy(acc_out, acc, n * sizeof(float));
    }
    free(acc);
    return rc;
}

/* ---- codec variant: L2-norm scale --------------------------------------------
 * The paper's related-work section cites quantizers that scale by the Euclidean
 * norm of the vector instead of its largest magnitude.  Only the scale differs
 * from the main codec; the encode, the draws, the packing and the whole server
 * side (R4..R14) are unchanged.  A sum of floats depends on its order, so the
 * order is part of the definition (readings N1..N3):
 *   N1  the bucket is cut into rows of 32 consecutive elements from its first
 *       element (the last row may be shorter).  A row's sum of squares is the
 *       left-to-right chain a <- fma(x_j, x_j, a), starting from a = 0.
 *   N2  the row sums are the leaves of a balanced binary tree of adjacent pairs
 *       (the leaf count padded with zeros to a power of two); each node is the
 *       fp32 sum of its two children.  S = the root.
 *   N3  S < 2^-96 flushes the bucket (scale 0, every code 0); otherwise the scale
 *       is s = fl(sqrt(S)).  With that threshold every |x_i| <= s: a square that
 *       is a normal number has an exact root, and smaller elements are below 2^-48.
 * Inputs whose sum of squares overflows are outside the definition.
 */
float mqo_sumsq_tree(const float *x, uint64_t len)
{
    if (len == 0) return 0.0f;
    uint64_t rows = (len + 31) / 32;
    uint64_t padded = 1;
    while (padded < rows) padded *= 2;
    float *node = (float *)calloc(padded, sizeof(float));
    if (!node) return NAN;
    for (uint64_t r = 0; r < rows; ++r) {                 /* N1 */
        uint64_t j0 = 32 * r, j1 = j0 + 32;
        if (j1 > len) j1 = len;
        float a = 0.0f;
        for (uint64_t j = j0; j < j1; ++j) a = fmaf(x[j], x[j], a);
        node[r] = a;
    }
    for (uint64_t width = padded; width > 1; width /= 2)  /* N2: one tree level per pass */
        for (uint64_t j = 0; j < width / 2; ++j)
            node[j] = node[2 * j] + node[2 * j + 1];
    float S = node[0];
    free(node);
    return S;
}

void mqo_bucket_norms(const float *x, uint64_t n, uint64_t bucket, float *scales)
{
    const float tiny = ldexpf(1.0f, -96);
    uint64_t nb = (n + bucket - 1) / bucket;
    for (uint64_t k = 0; k < nb; ++k) {
        uint64_t b0 = k * bucket, b1 = b0 + bucket;
        if (b1 > n) b1 = n;
        float S = mqo_sumsq_tree(x + b0, b1 - b0);
        scales[k] = (S < tiny) ? 0.0f : sqrtf(S);         /* N3 */
    }
}

/* Quantize(g, K) with the L2-norm scale: mqo_quantize with N1..N3 in place of R2/R3. */
int mqo_quantize_l2(const void *grad, uint64_t n, int bits, uint64_t bucket, uint64_t seed,
                    uint32_t *codes, float *scales, int dtype, uint32_t worker,
                    uint32_t step, uint64_t elem_offset)
{
    if (bits < 1 || bits > 8 || bucket == 0) return -1;
    if (n == 0) return 0;
    float *x = (float *)malloc(n * sizeof(float));
    uint16_t *h = (uint16_t *)malloc(n * sizeof(uint16_t));
    uint8_t *q = (uint8_t *)malloc(n);
    if (!x || !h || !q) { free(x); free(h); free(q); return -2; }
    if (dtype == 1) mqo_widen_bf16((const uint16_t *)grad, n, x);
    else memcpy(x, grad, n * sizeof(float));
    mqo_bucket_norms(x, n, bucket, scales);
    mqo_draw_h(seed, worker, step, elem_offset, n, h);
    mqo_encode(x, n, bits, bucket, scales, h, q);
    mqo_pack(q, n, bits, codes);
    free(x); free(h); free(q);
    return 0;
}

/* Per-layer L2-norm scale: the segment conventions of mqo_quantize_segments. */
int mqo_quantize_segments_l2(const void *grad, int nseg, const uint64_t *seg_off,
                             const uint64_t *code_off, int bits, uint64_t seed,
                             uint32_t *codes, float *scales, int dtype, uint32_t worker,
                             uint32_t step, uint64_t elem_offset)
{
    for (int j = 0; j < nseg; ++j) {
        uint64_t len = seg_off[j + 1] - seg_off[j];
        const char *base = (const char *)grad + seg_off[j] * (dtype == 1 ? 2u : 4u);
        if (len == 0) { scales[j] = 0.0f; continue; }
        int rc = mqo_quantize_l2(base, len, bits, len, seed, codes + code_off[j], &scales[j],
                                 dtype, worker, step, elem_offset + seg_off[j]);
        if (rc) return rc;
    }
    return 0;
}

/* ---- codec variant: one bit per element with error feedback ---------------------
 * Section 2 (Related work) cites the 1-bit scheme in which every gradient value travels
 * as one bit and the quantization error is carried forward into the next mini-batch.
 * The paper gives no formula for it; the readings this repository fixes (E1..E5):
 *   E1  v_i = fl(g_i + e_i), e = the worker's residual of the previous iteration (fp32,
 *       zero before the first one).
 *   E2  q_i = 1 if v_i >= 0 (a zero of either sign included), else 0.
 *   E3  per bucket two reconstruction values, the means of the two classes:
 *       neg = fl(S0 / c0), pos = fl(S1 / c1) (0 for an empty class; a zero of either sign
 *       stored as +0).  c = the class's element count; S = its sum in fixed order: rows
 *       of 32 elements from the bucket's first element, inside a row the chain
 *       a <- fl(a + v_j) over the row's members of the class from a = 0, left to right,
 *       and the row sums combined by the balanced tree of adjacent pairs (as N2).
 *       They are sent as ranges[2k] = neg, ranges[2k + 1] = pos, so that the wire format
 *       is the (min, max) variant's with K = 1 and the receiver needs nothing new.
 *   E4  the value the receiver will reconstruct (M4 with K = 1): r = fl(pos - neg);
 *       x^_i = fma(q_i, r, neg); a bucket with r < 2^-96 is constant: codes 0, x^ = neg.
 *   E5  e_i <- fl(v_i - x^_i): the residual is taken against E4's value, not against the
 *       ideal mean, so nothing the receiver loses is forgotten.
 */
static float mqo_class_sum_tree(const float *v, uint64_t len, int cls)
{
    uint64_t rows = (len + 31) / 32;
    uint64_t padded = 1;
    while (padded < rows) padded *= 2;
    float *node = (float *)calloc(padded, sizeof(float));
    if (!node) return NAN;
    for (uint64_t r = 0; r < rows; ++r) {
        uint64_t j0 = 32 * r, j1 = j0 + 32;
        if (j1 > len) j1 = len;
        float a = 0.0f;
        for (uint64_t j = j0; j < j1; ++j)
            if ((v[j] >= 0.0f ? 1 : 0) == cls) a = a + v[j];
        node[r] = a;
    }
    for (uint64_t width = padded; width > 1; width /= 2)
        for (uint64_t j = 0; j < width / 2; ++j)
            node[j] = node[2 * j] + node[2 * j + 1];
    float S = node[0];
    free(node);
    return S;
}

/* E1..E5 for one worker buffer; residual is read and overwritten.  dtype as mqo_quantize. */
int mqo_quantize_1bit_ef(const void *grad, float *residual, uint64_t n, uint64_t bucket,
                         uint32_t *codes, float *ranges, int dtype)
{
    if (bucket == 0) return -1;
    if (n == 0) return 0;
    const float tiny = ldexpf(1.0f, -96);
    float *v = (float *)malloc(n * sizeof(float));
    uint8_t *q = (uint8_t *)malloc(n);
    if (!v || !q) { free(v); free(q); return -2; }
    if (dtype == 1) mqo_widen_bf16((const uint16_t *)grad, n, v);
    else memcpy(v, grad, n * sizeof(float));
    for (uint64_t i = 0; i < n; ++i) v[i] = v[i] + residual[i];            /* E1 */
    uint64_t nb = (n + bucket - 1) / bucket;
    for (uint64_t k = 0; k < nb; ++k) {
        uint64_t b0 = k * bucket, b1 = b0 + bucket;
        if (b1 > n) b1 = n;
        uint64_t c1 = 0;
        for (uint64_t i = b0; i < b1; ++i) {                               /* E2 */
            q[i] = (v[i] >= 0.0f) ? 1 : 0;
            c1 += q[i];
        }
        uint64_t c0 = (b1 - b0) - c1;
        float S0 = mqo_class_sum_tree(v + b0, b1 - b0, 0);
        float S1 = mqo_class_sum_tree(v + b0, b1 - b0, 1);
        float neg = c0 ? S0 / (float)c0 : 0.0f;                            /* E3 */
        float pos = c1 ? S1 / (float)c1 : 0.0f;
        neg = neg + 0.0f;
        pos = pos + 0.0f;
        ranges[2 * k] = neg;
        ranges[2 * k + 1] = pos;
        float r = pos - neg;                                               /* E4 */
        for (uint64_t i = b0; i < b1; ++i) {
            if (r < tiny) q[i] = 0;
            float xhat = (r < tiny) ? neg : fmaf((float)q[i], r, neg);
            residual[i] = v[i] - xhat;                                     /* E5 */
        }
    }
    mqo_pack(q, n, 1, codes);
    free(v); free(q);
    return 0;
}
