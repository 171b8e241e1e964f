// Device-side building blocks shared by the libmqgrad kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace mqg {

// One thread owns one "row": 32 consecutive elements.  For every bit width K a row packs
// into exactly K 32-bit words, so all shifts are compile-time constants and no code
// straddles a thread boundary.
constexpr int kRowElems = 32;
constexpr int kMaxTileRows = 256;                 // rows per CTA tile = threads per CTA
constexpr int kMaxFusedBucket = kRowElems * kMaxTileRows;   // largest bucket of the one-pass kernel

// Scales below this are flushed to zero (2^-96).
__device__ __forceinline__ float flush_limit() { return __uint_as_float(0x0F800000u); }

// ---------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11).  Counter (c0..c3), key (k0,k1) -> four words.
// The ten round keys depend only on the seed, so they are computed once per thread
// (RoundKeys) and stay in registers across all blocks.
// ---------------------------------------------------------------------------------
struct DrawKey {
    uint32_t seed_lo, seed_hi, worker, step;
};

struct RoundKeys {
    uint32_t k0[10], k1[10];
    uint32_t worker, step;
};

__device__ __forceinline__ RoundKeys make_round_keys(const DrawKey& key)
{
    RoundKeys rk;
    uint32_t a = key.seed_lo, b = key.seed_hi;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        rk.k0[r] = a; rk.k1[r] = b;
        a += 0x9E3779B9u; b += 0xBB67AE85u;
    }
    rk.worker = key.worker; rk.step = key.step;
    return rk;
}

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              const RoundKeys& rk, uint32_t (&y)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk.k1[r];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    y[0] = c0; y[1] = c1; y[2] = c2; y[3] = c3;
}

// The part of a Philox block that is the same for every block of a launch whose counter words c1
// (high half of the block index), c2 (worker) and the key do not change: in round 1 the product of
// c2 and with it the new c0 and c1, in round 2 the product of that c0.  Computed once on the host
// (philox_head), so a block costs two multiplications and one xor less.
struct PhiloxHead {
    uint32_t c1_r1;      // c1 after round 1: lo(M1 * worker)
    uint32_t c0_r1;      // c0 after round 1: hi(M1 * worker) ^ c1 ^ k0[0]
    uint32_t p0hi_r2;    // hi(M0 * c0_r1)
    uint32_t p0lo_r2;    // lo(M0 * c0_r1) = c3 after round 2
};

__host__ __device__ inline PhiloxHead philox_head(uint32_t blk_hi, uint32_t worker, uint32_t key0)
{
    PhiloxHead h;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * worker;
    h.c1_r1 = (uint32_t)p1;
    h.c0_r1 = (uint32_t)(p1 >> 32) ^ blk_hi ^ key0;
    const uint64_t p0 = (uint64_t)0xD2511F53u * h.c0_r1;
    h.p0hi_r2 = (uint32_t)(p0 >> 32);
    h.p0lo_r2 = (uint32_t)p0;
    return h;
}

// philox4x32_10(c0, blk_hi, worker, step) with the launch-wide part taken from `hd`.
__device__ __forceinline__ void philox4x32_10_head(uint32_t c0, const PhiloxHead& hd, const RoundKeys& rk,
                                                   uint32_t (&y)[4])
{
    // round 1: only the product of c0 depends on the block
    const uint64_t q0 = (uint64_t)0xD2511F53u * c0;
    uint32_t c2 = (uint32_t)(q0 >> 32) ^ rk.step ^ rk.k1[0];
    uint32_t c3 = (uint32_t)q0;
    // round 2: the product of c0 (= hd.c0_r1) is known
    const uint64_t q1 = (uint64_t)0xCD9E8D57u * c2;
    c0 = (uint32_t)(q1 >> 32) ^ hd.c1_r1 ^ rk.k0[1];
    c2 = hd.p0hi_r2 ^ c3 ^ rk.k1[1];
    uint32_t c1 = (uint32_t)q1;
    c3 = hd.p0lo_r2;
#pragma unroll
    for (int r = 2; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk.k1[r];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    y[0] = c0; y[1] = c1; y[2] = c2; y[3] = c3;
}

// The draws of a row whose four blocks are blk_lo .. blk_lo + 3 without a carry into the high half.
__device__ __forceinline__ void draw_row_blocks_head(uint32_t blk_lo, const PhiloxHead& hd, const RoundKeys& rk,
                                                     uint32_t (&h)[16])
{
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        uint32_t y[4];
        philox4x32_10_head(blk_lo + b, hd, rk, y);
#pragma unroll
        for (int k = 0; k < 4; ++k) h[4 * b + k] = y[k];
    }
}

// The 16-bit draws of the 32 elements at flat positions g0 .. g0+31, g0 % 8 == 0:
// four Philox blocks, block index g >> 3; element g takes half (g & 1) of word (g & 7) >> 1.
// h[j] holds the two draws of elements 2j (low half) and 2j+1 (high half).
// (blk_lo, blk_hi) = 64-bit block index of the row's first element.
// `worker` is passed beside the keys so one set of round keys can serve several workers.
__device__ __forceinline__ void draw_row_blocks(uint32_t blk_lo, uint32_t blk_hi, uint32_t worker,
                                                const RoundKeys& rk, uint32_t (&h)[16])
{
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        uint32_t y[4];
        const uint32_t lo = blk_lo + b;
        philox4x32_10(lo, blk_hi + (lo < blk_lo ? 1u : 0u), worker, rk.step, rk, y);
#pragma unroll
        for (int k = 0; k < 4; ++k) h[4 * b + k] = y[k];
    }
}

__device__ __forceinline__ void draw_row_blocks(uint32_t blk_lo, uint32_t blk_hi, const RoundKeys& rk,
                                                uint32_t (&h)[16])
{
    draw_row_blocks(blk_lo, blk_hi, rk.worker, rk, h);
}

__device__ __forceinline__ void draw_row_aligned(uint64_t g0, const RoundKeys& rk, uint32_t (&h)[16])
{
    const uint64_t blk0 = g0 >> 3;
    draw_row_blocks((uint32_t)blk0, (uint32_t)(blk0 >> 32), rk, h);
}

// Same for any g0 (slow path: up to five blocks, run-time selection).
static __device__ __noinline__ void draw_row_unaligned(uint64_t g0, const DrawKey& key, uint32_t (&h)[16])
{
    const RoundKeys rk = make_round_keys(key);
    uint32_t y[20];
    const uint64_t blk0 = g0 >> 3;
    for (int b = 0; b < 5; ++b) {
        const uint64_t blk = blk0 + b;
        uint32_t t[4];
        philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), rk.worker, rk.step, rk, t);
        for (int k = 0; k < 4; ++k) y[4 * b + k] = t[k];
    }
    const unsigned shift = (unsigned)(g0 & 7u);       // first element's field in the 40-field run
    for (int j = 0; j < 16; ++j) {
        const unsigned f0 = shift + 2u * j, f1 = f0 + 1u;
        const uint32_t lo = (y[f0 >> 1] >> (16u * (f0 & 1u))) & 0xFFFFu;
        const uint32_t hi = (y[f1 >> 1] >> (16u * (f1 & 1u))) & 0xFFFFu;
        h[j] = lo | (hi << 16);
    }
}

// max(m, |a|, |b|) in one three-input instruction.
__device__ __forceinline__ float max3_abs(float m, float a, float b)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(m), "f"(fabsf(a)), "f"(fabsf(b)));
    return r;
}

__device__ __forceinline__ float row_abs_max(const float (&x)[32])
{
    float mx = 0.0f;
#pragma unroll
    for (int j = 0; j < 32; j += 2) mx = max3_abs(mx, x[j], x[j + 1]);
    return mx;
}

// L2-norm scale variant: a row's sum of squares is the left-to-right chain a <- fma(x_j, x_j, a)
// from a = 0 (the order is part of the variant's definition).
__device__ __forceinline__ float row_sum_squares(const float (&x)[32])
{
    float a = 0.0f;
#pragma unroll
    for (int j = 0; j < 32; ++j) a = __fmaf_rn(x[j], x[j], a);
    return a;
}

// Per-bucket encode constants, pre-scaled by 2^16: T = fma(x, inv16, half_l16) = 2^16 * t with
// t = fl(x * fl(L / 2s) + L/2) -- scaling both constants by a power of two leaves the single
// rounding of the fma unchanged.  A flushed bucket uses (0, 0): every x gives T = 0, code 0.
struct EncodeScale {
    float inv16, half_l16;
};

template <int BITS>
__device__ __forceinline__ EncodeScale encode_scale(float s)
{
    constexpr float Lf = (float)((1 << BITS) - 1);
    EncodeScale e;
    if (s == 0.0f) { e.inv16 = 0.0f; e.half_l16 = 0.0f; }
    else {
        e.inv16 = __fmul_rn(__fdiv_rn(Lf, __fmul_rn(2.0f, s)), 65536.0f);
        e.half_l16 = 32768.0f * Lf;
    }
    return e;
}

// Stochastic-rounding code of one element, as the bit pattern of the float 1.5 * 2^23 + q.
// `hf` is the float 2^23 + h (h = the element's 16-bit draw, merged into the mantissa).
//   code = floor(t) + [u < t - floor(t)],  u = (h + 1/2) / 2^16
//        = ceil(t - u) = ceil((T - (h + 1/2)) / 2^16).
// |T| stands for the clamp to [0, L]: t <= L always holds for |x| <= s, and a t rounded
// slightly below zero has |t| < 2^-17 <= u, which gives code 0 like the clamp.
// Rounding the difference up cannot cross a multiple of 2^16 (those are floats), and adding
// 1.5 * 2^23 with rounding up leaves the ceiling in the low mantissa bits.
__device__ __forceinline__ uint32_t encode_bits(float x, const EncodeScale& e, float hf)
{
    const float T = __fmaf_rn(x, e.inv16, e.half_l16);
    const float hh = __fsub_rn(hf, 8388607.5f);                 // h + 1/2, exact
    const float d = __fadd_ru(fabsf(T), -hh);
    const float w = __fmaf_ru(d, 1.0f / 65536.0f, 12582912.0f);
    return __float_as_uint(w);
}
constexpr uint32_t kCodeBias = 0x4B400000u;      // bit pattern of 1.5 * 2^23

// 2^23 + h for the low / high 16-bit half of a Philox word.
__device__ __forceinline__ float draw_lo(uint32_t y) { return __uint_as_float(__byte_perm(y, 0x4B000000u, 0x7610)); }
__device__ __forceinline__ float draw_hi(uint32_t y) { return __uint_as_float(__byte_perm(y, 0x4B000000u, 0x7632)); }

// Sum (mod 2^32) of the kCodeBias contributions that land in word k of a packed row.
template <int BITS>
__host__ __device__ constexpr uint32_t pack_bias(int k)
{
    uint32_t b = 0;
    for (int j = 0; j < 32; ++j) {
        const int o = j * BITS, wi = o >> 5, sh = o & 31;
        if (wi == k) b += kCodeBias << sh;
        if (sh + BITS > 32 && wi + 1 == k) b += kCodeBias >> (32 - sh);
    }
    return b;
}

// Encode the 32 values of a row and pack them, code j at bits [j*BITS, j*BITS+BITS), into BITS
// words.  The biased patterns kCodeBias + q are accumulated with shift-adds; the first
// contribution to a word also removes that word's total bias (a compile-time constant).
template <int BITS>
__device__ __forceinline__ void encode_pack_row(const float (&x)[32], const EncodeScale& e,
                                                const uint32_t (&h)[16], uint32_t (&w)[BITS])
{
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const float hf = (j & 1) ? draw_hi(h[j >> 1]) : draw_lo(h[j >> 1]);
        const uint32_t c = encode_bits(x[j], e, hf);
        const int o = j * BITS, wi = o >> 5, sh = o & 31;
        if (sh == 0) w[wi] = c - pack_bias<BITS>(wi);
        else w[wi] = w[wi] + (c << sh);
        if (sh + BITS > 32)                                     // the bias has 22 zero low bits:
            w[wi + 1] = (c >> (32 - sh)) - pack_bias<BITS>(wi + 1);   // no carry mixes in
    }
}

// The same with the packed fp32x2 instructions of sm_100: two elements per instruction, each lane rounded
// exactly as the scalar instruction would.  |T| is not taken: a T rounded slightly below zero gives a
// negative difference in (-2^16, 0) either way, and the ceiling of that is code 0.
template <int BITS>
__device__ __forceinline__ void encode_pack_row_packed(const float (&x)[32], const EncodeScale& e,
                                                       const uint32_t (&h)[16], uint32_t (&w)[BITS])
{
    const float2 inv = make_float2(e.inv16, e.inv16), half = make_float2(e.half_l16, e.half_l16);
    const float2 neg1 = make_float2(-1.0f, -1.0f), c = make_float2(8388607.5f, 8388607.5f);
    const float2 r16 = make_float2(1.0f / 65536.0f, 1.0f / 65536.0f), magic = make_float2(12582912.0f, 12582912.0f);
#pragma unroll
    for (int p = 0; p < 16; ++p) {
        const float2 hf = make_float2(draw_lo(h[p]), draw_hi(h[p]));
        const float2 T = __ffma2_rn(make_float2(x[2 * p], x[2 * p + 1]), inv, half);
        const float2 nhh = __ffma2_rn(hf, neg1, c);             // -(h + 1/2), exact
        const float2 d = __fadd2_ru(T, nhh);
        const float2 ww = __ffma2_ru(d, r16, magic);
        const uint32_t cc[2] = {__float_as_uint(ww.x), __float_as_uint(ww.y)};
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int j = 2 * p + q;
            const int o = j * BITS, wi = o >> 5, sh = o & 31;
            if (sh == 0) w[wi] = cc[q] - pack_bias<BITS>(wi);
            else w[wi] = w[wi] + (cc[q] << sh);
            if (sh + BITS > 32) w[wi + 1] = (cc[q] >> (32 - sh)) - pack_bias<BITS>(wi + 1);
        }
    }
}

// ---------------------------------------------------------------------------------
// Codec variant: (min, max) range with nearest rounding.  Per bucket lo = min x, hi = max x
// (a zero of either sign stored as +0), r = fl(hi - lo); code = min(L, floor(fma(fl(x - lo),
// fl(L / r), 1/2))); x^ = fma(q, fl(r / L), lo); a bucket with r < 2^-96 is constant: every code
// is 0 and every x^ is lo.
// ---------------------------------------------------------------------------------

// Order-preserving map of a float's bit pattern to an unsigned integer (-0 sorts just below +0),
// so that integer min / max reductions and atomics serve float min / max.
__device__ __forceinline__ uint32_t ordered_bits(float f)
{
    const uint32_t b = __float_as_uint(f);
    return b ^ ((b >> 31) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t u)
{
    return __uint_as_float(u ^ ((u >> 31) ? 0x80000000u : 0xFFFFFFFFu));
}
constexpr uint32_t kOrderedMinIdentity = 0xFFFFFFFFu;   // above every float
constexpr uint32_t kOrderedMaxIdentity = 0x00000000u;   // below every float

__device__ __forceinline__ void row_min_max(const float (&x)[32], float& lo, float& hi)
{
    lo = x[0]; hi = x[0];
#pragma unroll
    for (int j = 1; j < 32; ++j) { lo = fminf(lo, x[j]); hi = fmaxf(hi, x[j]); }
}

struct RangeEncodeScale {
    float lo, inv;               // inv = fl(L / r), or 0 for a constant bucket (then t = 1/2, code 0)
};

template <int BITS>
__device__ __forceinline__ RangeEncodeScale range_encode_scale(float lo, float hi)
{
    constexpr float Lf = (float)((1 << BITS) - 1);
    RangeEncodeScale e;
    e.lo = lo;
    const float r = __fsub_rn(hi, lo);
    e.inv = r < flush_limit() ? 0.0f : __fdiv_rn(Lf, r);
    return e;
}

// Nearest-rounding code of one element as the bit pattern of the float 1.5 * 2^23 + q:
// t = fma(x - lo, inv, 1/2) >= 1/2 is rounded once, then adding 1.5 * 2^23 with rounding towards
// minus infinity leaves floor(t) in the low mantissa bits.  For lo <= x <= hi, t < L + 1, so the
// clamp to L needs no instruction.
__device__ __forceinline__ uint32_t range_encode_bits(float x, const RangeEncodeScale& e)
{
    const float d = __fsub_rn(x, e.lo);
    const float t = __fmaf_rn(d, e.inv, 0.5f);
    return __float_as_uint(__fadd_rd(t, 12582912.0f));
}

template <int BITS>
__device__ __forceinline__ void range_encode_pack_row(const float (&x)[32], const RangeEncodeScale& e,
                                                      uint32_t (&w)[BITS])
{
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const uint32_t c = range_encode_bits(x[j], e);
        const int o = j * BITS, wi = o >> 5, sh = o & 31;
        if (sh == 0) w[wi] = c - pack_bias<BITS>(wi);
        else w[wi] = w[wi] + (c << sh);
        if (sh + BITS > 32)
            w[wi + 1] = (c >> (32 - sh)) - pack_bias<BITS>(wi + 1);
    }
}

// Code j of a row from its BITS words.
template <int BITS>
__device__ __forceinline__ uint32_t unpack_one(const uint32_t (&w)[BITS], int j)
{
    const int o = j * BITS, wi = o >> 5, sh = o & 31;
    uint32_t v = w[wi] >> sh;
    if (sh + BITS > 32) v |= w[wi + 1] << (32 - sh);
    return v & ((1u << BITS) - 1u);
}

// Zero the bits of a row's words at and beyond `valid_bits` (ragged last row).
template <int BITS>
__device__ __forceinline__ void mask_row_words(uint32_t (&w)[BITS], int valid_bits)
{
#pragma unroll
    for (int k = 0; k < BITS; ++k) {
        const int rem = valid_bits - 32 * k;
        if (rem <= 0) w[k] = 0u;
        else if (rem < 32) w[k] &= (1u << rem) - 1u;
    }
}

// Store / load the BITS words of a row at word index `word0` (a multiple of BITS), using the
// widest access the alignment of every row allows.  `nwords_limit` guards a ragged last row.
template <int BITS>
__device__ __forceinline__ void store_row_words(uint32_t* __restrict__ codes, uint64_t word0,
                                                const uint32_t (&w)[BITS])
{
    if constexpr (BITS % 4 == 0) {
        uint4* p = reinterpret_cast<uint4*>(codes + word0);
#pragma unroll
        for (int k = 0; k < BITS / 4; ++k) p[k] = make_uint4(w[4 * k], w[4 * k + 1], w[4 * k + 2], w[4 * k + 3]);
    } else if constexpr (BITS % 2 == 0) {
        uint2* p = reinterpret_cast<uint2*>(codes + word0);
#pragma unroll
        for (int k = 0; k < BITS / 2; ++k) p[k] = make_uint2(w[2 * k], w[2 * k + 1]);
    } else {
#pragma unroll
        for (int k = 0; k < BITS; ++k) codes[word0 + k] = w[k];
    }
}

template <int BITS>
__device__ __forceinline__ void load_row_words(const uint32_t* __restrict__ codes, uint64_t word0,
                                               uint32_t (&w)[BITS])
{
    if constexpr (BITS % 4 == 0) {
        const uint4* p = reinterpret_cast<const uint4*>(codes + word0);
#pragma unroll
        for (int k = 0; k < BITS / 4; ++k) {
            const uint4 v = __ldg(p + k);
            w[4 * k] = v.x; w[4 * k + 1] = v.y; w[4 * k + 2] = v.z; w[4 * k + 3] = v.w;
        }
    } else if constexpr (BITS % 2 == 0) {
        const uint2* p = reinterpret_cast<const uint2*>(codes + word0);
#pragma unroll
        for (int k = 0; k < BITS / 2; ++k) {
            const uint2 v = __ldg(p + k);
            w[2 * k] = v.x; w[2 * k + 1] = v.y;
        }
    } else {
#pragma unroll
        for (int k = 0; k < BITS; ++k) w[k] = __ldg(codes + word0 + k);
    }
}

// Shared-memory tile of rows x 32 floats with the 128-byte swizzle: the 16-byte chunk c of
// row r lives at chunk position c ^ (r & 7), so that eight threads reading the same chunk
// index of eight consecutive rows touch all 32 banks.
__device__ __forceinline__ int swz(int row, int chunk) { return row * 8 + (chunk ^ (row & 7)); }

__device__ __forceinline__ void read_row(const float4* tile, int row, float (&x)[32])
{
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const float4 v = tile[swz(row, c)];
        x[4 * c] = v.x; x[4 * c + 1] = v.y; x[4 * c + 2] = v.z; x[4 * c + 3] = v.w;
    }
}

__device__ __forceinline__ void write_row(float4* tile, int row, const float (&x)[32])
{
#pragma unroll
    for (int c = 0; c < 8; ++c)
        tile[swz(row, c)] = make_float4(x[4 * c], x[4 * c + 1], x[4 * c + 2], x[4 * c + 3]);
}

// 16-byte asynchronous copy global -> shared: no register staging, so a thread can have all its
// chunks of a tile in flight at once; cp_async_wait_all() (then a barrier) before the data is read.
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;"
                 ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Cooperative, coalesced copy of a tile of `rows` rows into / out of a swizzled tile.  `src`
// points at the tile's first element and `valid` is the number of elements that exist from
// there on (elements at or beyond it read as zero and are never written).  128-bit accesses
// when the tile's first element is 16-byte aligned, 32-bit (16-bit for bf16) otherwise.
// The aligned fp32 path copies asynchronously; with WAIT = false the caller overlaps other work
// with the copies and calls cp_async_wait_all() itself before the barrier that precedes the reads.
template <int THREADS, bool WAIT = true>
__device__ __forceinline__ void load_tile_f32(float4* tile, const float* __restrict__ src,
                                              uint64_t valid, int rows)
{
    if ((reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
        const int chunks = rows * 8;
        for (int idx = threadIdx.x; idx < chunks; idx += THREADS) {
            const uint64_t e = 4ull * idx;
            float4* dst = &tile[swz(idx >> 3, idx & 7)];
            if (e + 4 <= valid) cp_async16(dst, src + e);
            else {
                float4 v;
                v.x = (e + 0 < valid) ? src[e + 0] : 0.0f;
                v.y = (e + 1 < valid) ? src[e + 1] : 0.0f;
                v.z = (e + 2 < valid) ? src[e + 2] : 0.0f;
                v.w = 0.0f;
                *dst = v;
            }
        }
        if (WAIT) cp_async_wait_all();
    } else {
        float* tf = reinterpret_cast<float*>(tile);
        const int elems = rows * 32;
        for (int k = threadIdx.x; k < elems; k += THREADS) {
            const float v = ((uint64_t)k < valid) ? __ldcs(src + k) : 0.0f;
            tf[swz(k >> 5, (k >> 2) & 7) * 4 + (k & 3)] = v;
        }
    }
}

__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

template <int THREADS>
__device__ __forceinline__ void load_tile_bf16(float4* tile, const uint16_t* __restrict__ src,
                                               uint64_t valid, int rows)
{
    if ((reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
        const int groups = rows * 4;                    // 8 bf16 (16 bytes) per group
        for (int idx = threadIdx.x; idx < groups; idx += THREADS) {
            const uint64_t e = 8ull * idx;
            uint32_t u[4];
            if (e + 8 <= valid) {
                const uint4 v = __ldcs(reinterpret_cast<const uint4*>(src + e));
                u[0] = v.x; u[1] = v.y; u[2] = v.z; u[3] = v.w;
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t lo = (e + 2 * k < valid) ? src[e + 2 * k] : 0u;
                    const uint32_t hi = (e + 2 * k + 1 < valid) ? src[e + 2 * k + 1] : 0u;
                    u[k] = lo | (hi << 16);
                }
            }
            const int row = idx >> 2, c = (idx & 3) * 2;
            tile[swz(row, c)] = make_float4(bf16_lo(u[0]), bf16_hi(u[0]), bf16_lo(u[1]), bf16_hi(u[1]));
            tile[swz(row, c + 1)] = make_float4(bf16_lo(u[2]), bf16_hi(u[2]), bf16_lo(u[3]), bf16_hi(u[3]));
        }
    } else {
        float* tf = reinterpret_cast<float*>(tile);
        const int elems = rows * 32;
        for (int k = threadIdx.x; k < elems; k += THREADS) {
            const uint32_t b = ((uint64_t)k < valid) ? (uint32_t)src[k] : 0u;
            tf[swz(k >> 5, (k >> 2) & 7) * 4 + (k & 3)] = bf16_lo(b);
        }
    }
}

template <int THREADS>
__device__ __forceinline__ void store_tile_f32(const float4* tile, float* __restrict__ dst,
                                               uint64_t valid, int rows)
{
    if ((reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
        const int chunks = rows * 8;
        for (int idx = threadIdx.x; idx < chunks; idx += THREADS) {
            const uint64_t e = 4ull * idx;
            if (e >= valid) continue;
            const float4 v = tile[swz(idx >> 3, idx & 7)];
            if (e + 4 <= valid) *reinterpret_cast<float4*>(dst + e) = v;
            else {
                dst[e] = v.x;
                if (e + 1 < valid) dst[e + 1] = v.y;
                if (e + 2 < valid) dst[e + 2] = v.z;
            }
        }
    } else {
        const float* tf = reinterpret_cast<const float*>(tile);
        const int elems = rows * 32;
        for (int k = threadIdx.x; k < elems; k += THREADS)
            if ((uint64_t)k < valid) dst[k] = tf[swz(k >> 5, (k >> 2) & 7) * 4 + (k & 3)];
    }
}

// ---------------------------------------------------------------------------------
// De-quantization.  Constants of one (worker, bucket): x^ = fma(q - (L-1)/2, 2h, -h) with
// h = fl(s / L).  The product (q - (L-1)/2) * 2h and the subtraction of h are exact inside
// the fma, so its single rounding is the rounding of (2q - L) * h.  A zero scale gives +0.
// ---------------------------------------------------------------------------------
struct DecodeScale {
    float two_h, minus_h;
};

// The same constants duplicated for the two lanes of the packed instructions.
struct DecodeScale2 {
    float2 two_h, minus_h;
};
__device__ __forceinline__ DecodeScale2 widen(const DecodeScale& d)
{
    DecodeScale2 r;
    r.two_h = make_float2(d.two_h, d.two_h);
    r.minus_h = make_float2(d.minus_h, d.minus_h);
    return r;
}

template <int BITS>
__device__ __forceinline__ DecodeScale decode_scale(float s)
{
    constexpr float Lf = (float)((1 << BITS) - 1);
    DecodeScale d;
    if (s == 0.0f) { d.two_h = 0.0f; d.minus_h = 0.0f; }
    else {
        const float h = __fdiv_rn(s, Lf);
        d.two_h = __fmul_rn(2.0f, h);
        d.minus_h = -h;
    }
    return d;
}

// (min, max) variant: (two_h, minus_h) := (step, lo), step = fl(r / L), 0 for a constant bucket.
template <int BITS>
__device__ __forceinline__ DecodeScale range_decode_scale(float lo, float hi)
{
    constexpr float Lf = (float)((1 << BITS) - 1);
    DecodeScale d;
    const float r = __fsub_rn(hi, lo);
    d.two_h = r < flush_limit() ? 0.0f : __fdiv_rn(r, Lf);
    d.minus_h = lo;
    return d;
}

// ---------------------------------------------------------------------------------
// Packed fp32x2 arithmetic of sm_100 (__fadd2_rn, __ffma2_rn on float2): one instruction rounds
// two independent fp32 lanes, each exactly as the scalar instruction would.  It halves the
// issue slots of the decode arithmetic.
// ---------------------------------------------------------------------------------

// Two codes at once.  m = the floats 2^23 + q (code merged into the mantissa of 2^23);
// returns v + x^ for both lanes, each x^ rounded once, then the sum rounded once.
// RANGE: the (min, max) variant, x^ = fma(q, step, lo): the same two instructions with
// (two_h, minus_h) := (step, lo) and the offset 2^23 alone.
template <int BITS, bool RANGE = false>
__device__ __forceinline__ float2 accumulate2(float2 v, float2 m, float2 two_h, float2 minus_h)
{
    constexpr float kNegOff = RANGE ? -8388608.0f
                                    : -(8388608.0f + (float)(((1 << BITS) - 2) / 2));   // -(2^23 + (L - 1) / 2)
    const float2 qi = __fadd2_rn(m, make_float2(kNegOff, kNegOff));             // q - (L - 1) / 2, exact
    return __fadd2_rn(v, __ffma2_rn(qi, two_h, minus_h));
}

// `bias` is the bit pattern of 2^23 (0x4B000000).  Callers pass it from a kernel argument so that
// it is a constant-bank operand of the byte permute instead of a register that has to be
// re-materialised when registers are short.
__device__ __forceinline__ float byte_to_biased(uint32_t v, int byte, uint32_t bias)
{
    return __uint_as_float(__byte_perm(v, bias, 0x7650 + byte));
}

// v2[] <- v2[] + de-quantized row; v2[p] holds the running sums of elements 2p and 2p+1 (+0
// before the first worker: 0 + x^ is exact, and turns the -0 of a zero-scale bucket into +0).
template <int BITS, bool RANGE = false>
__device__ __forceinline__ void add_decoded_row(const uint32_t (&w)[BITS], const DecodeScale2& d,
                                                float2 (&v2)[16], uint32_t bias = 0x4B000000u)
{
    if constexpr (BITS == 1 && !RANGE) {
        // x^ = +-s (s = h for one bit): set the sign where the code bit is 0
        const uint32_t sbits = __float_as_uint(-d.minus_h.x);
#pragma unroll
        for (int p = 0; p < 16; ++p) {
            const uint32_t s0 = (~(w[0] << (31 - 2 * p))) & 0x80000000u;
            const uint32_t s1 = (~(w[0] << (30 - 2 * p))) & 0x80000000u;
            v2[p] = __fadd2_rn(v2[p], make_float2(__uint_as_float(sbits | s0), __uint_as_float(sbits | s1)));
        }
    } else {
        const float2 th = d.two_h, mh = d.minus_h;
        if constexpr (BITS == 8) {
#pragma unroll
            for (int p = 0; p < 16; ++p)
                v2[p] = accumulate2<8, RANGE>(v2[p], make_float2(byte_to_biased(w[p >> 1], (2 * p) & 3, bias),
                                                          byte_to_biased(w[p >> 1], (2 * p + 1) & 3, bias)), th, mh);
        } else if constexpr (BITS == 2) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                uint32_t t[4];
#pragma unroll
                for (int r = 0; r < 4; ++r) t[r] = (w[k] >> (2 * r)) & 0x03030303u;
#pragma unroll
                for (int b = 0; b < 4; ++b) {    // element 16k + 4b + r lives in byte b of t[r]
                    v2[8 * k + 2 * b] = accumulate2<2, RANGE>(v2[8 * k + 2 * b],
                                                       make_float2(byte_to_biased(t[0], b, bias), byte_to_biased(t[1], b, bias)), th, mh);
                    v2[8 * k + 2 * b + 1] = accumulate2<2, RANGE>(v2[8 * k + 2 * b + 1],
                                                           make_float2(byte_to_biased(t[2], b, bias), byte_to_biased(t[3], b, bias)), th, mh);
                }
            }
        } else {
            // Widths 3 to 7 (and width 1 of the range variant).  A group of G consecutive codes is
            // brought to bit 0 with one (funnel) shift; code g of the group is then masked IN PLACE
            // into the mantissa of 2^23, which gives the float 2^23 + q * 2^(g K) (g K + K <= 23), and
            // one packed fma with compile-time constants turns two of these into q - off exactly:
            //     fma(2^23 + q 2^s, 2^-s, -(2^(23 - s) + off)) = q - off      (every term is exact).
            // One shift per group and one logic operation per code instead of a shift and a logic
            // operation per code.  off = (L - 1) / 2 for the main codec, 0 for the range variant.
            // Width 4 measured 54.6 us per launch this way against 56.5 us with nibble masks and byte
            // permutes (n = 25 M, W = 8), width 3 51.9 against 55.0 us; widths 1 and 2 measured slower
            // (47.7 against 45.0 us, 47.9 against 47.0 us) and keep their own paths.
            constexpr int G = 4 * BITS <= 23 ? 4 : 2;
            constexpr uint32_t kMask = (1u << BITS) - 1u;
            constexpr float kOff = RANGE ? 0.0f : (float)(((1 << BITS) - 2) / 2);
#pragma unroll
            for (int grp = 0; grp < 32 / G; ++grp) {
                const int o = grp * G * BITS, wi = o >> 5, sh = o & 31;
                uint32_t win;
                if (sh == 0) win = w[wi];
                else if (sh + G * BITS <= 32) win = w[wi] >> sh;
                else win = __funnelshift_r(w[wi], w[wi + 1], sh);
#pragma unroll
                for (int h = 0; h < G / 2; ++h) {
                    constexpr float kTwo23 = 8388608.0f;
                    const int s0 = 2 * h * BITS, s1 = s0 + BITS;            // bit positions inside the group
                    const float2 m = make_float2(__uint_as_float((win & (kMask << s0)) | bias),
                                                 __uint_as_float((win & (kMask << s1)) | bias));
                    const float2 scale = make_float2(1.0f / (float)(1u << s0), 1.0f / (float)(1u << s1));
                    const float2 shift = make_float2(-(kTwo23 / (float)(1u << s0) + kOff),
                                                     -(kTwo23 / (float)(1u << s1) + kOff));
                    const float2 qi = __ffma2_rn(m, scale, shift);          // (q - off) for both lanes, exact
                    const int p = grp * (G / 2) + h;
                    v2[p] = __fadd2_rn(v2[p], __ffma2_rn(qi, th, mh));
                }
            }
        }
    }
}

// v[] (32 floats) <-> v2[] (16 pairs)
__device__ __forceinline__ void pairs_from_floats(const float (&v)[32], float2 (&v2)[16])
{
#pragma unroll
    for (int p = 0; p < 16; ++p) v2[p] = make_float2(v[2 * p], v[2 * p + 1]);
}
__device__ __forceinline__ void floats_from_pairs(const float2 (&v2)[16], float (&v)[32])
{
#pragma unroll
    for (int p = 0; p < 16; ++p) { v[2 * p] = v2[p].x; v[2 * p + 1] = v2[p].y; }
}

}  // namespace mqg
