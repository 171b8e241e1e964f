// The tile code of the TMA-fed quantize kernels (one tile of whole buckets per CTA turn: scale,
// draws, encode, pack), shared by the kernels of mqg_quantize.cu and mqg_segments_workers.cu.
#pragma once

#include "mqg_common.cuh"
#include "mqg_internal.h"
#include "mqg_tma.cuh"

namespace mqg {

struct QuantizeArgs {
    const void* grad;
    uint32_t* codes;
    float* scales;
    uint64_t n;             // elements
    uint64_t nrows;         // ceil(n / 32)
    uint64_t nbuckets;      // ceil(n / bucket)
    uint64_t ncode_words;   // ceil(n * bits / 32)
    uint64_t elem_offset;
    uint32_t rows_per_bucket;   // bucket / 32 (a single ragged bucket counts as "all rows")
    uint32_t tile_rows;         // rows per tile: a multiple of rows_per_bucket, <= 256
    uint32_t buckets_per_tile;
    uint64_t nrows_full;    // floor(n / 32): rows the tensor map covers
    uint32_t ntiles;
    DrawKey key;
    uint32_t poll_limit;        // polls of one barrier wait before the CTA gives up (TMA kernels)
    uint32_t arm_only;          // test hook: 1 = arm the barriers but issue no copy
};


// ---------------------------------------------------------------------------------------
// The same computation fed by TMA: a persistent CTA walks tiles blockIdx.x, +gridDim.x, ...;
// one elected thread keeps STAGES tiled bulk copies (cp.async.bulk.tensor, 128- or 64-byte
// swizzle) in flight into a shared-memory ring, each completing on its own mbarrier, so the
// compute warps never issue a global load and never wait for DRAM latency in steady state.
// One __syncthreads per tile publishes the bucket maxima and releases the stage for refill.
// ---------------------------------------------------------------------------------------
template <int DTYPE>
__device__ __forceinline__ void read_row_swizzled(const uint8_t* stage, int row, float (&x)[32])
{
    if constexpr (DTYPE == 0) {
        read_row(reinterpret_cast<const float4*>(stage), row, x);
    } else {
        const uint4* t = reinterpret_cast<const uint4*>(stage);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint4 v = t[row * 4 + (c ^ ((row >> 1) & 3))];
            const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                x[8 * c + 2 * k] = bf16_lo(u[k]);
                x[8 * c + 2 * k + 1] = bf16_hi(u[k]);
            }
        }
    }
}

// The one row of the gradient that is shorter than 32 elements is not covered by the tensor
// map: its owner copies it (zero-padded) into its own row of the stage with plain loads and
// then reads it back like any other row.
template <int DTYPE>
__device__ __noinline__ void stage_ragged_row(uint8_t* stage, int row, const void* grad, uint64_t e0,
                                              uint64_t n)
{
    for (int j = 0; j < 32; ++j) {
        const bool in = e0 + j < n;
        if constexpr (DTYPE == 0) {
            float* tf = reinterpret_cast<float*>(stage);
            tf[swz(row, j >> 2) * 4 + (j & 3)] = in ? static_cast<const float*>(grad)[e0 + j] : 0.0f;
        } else {
            uint16_t* th = reinterpret_cast<uint16_t*>(stage);
            const int chunk = (j >> 3) ^ ((row >> 1) & 3);
            th[(row * 4 + chunk) * 8 + (j & 7)] = in ? static_cast<const uint16_t*>(grad)[e0 + j] : (uint16_t)0;
        }
    }
}

template <int DTYPE, int THREADS>
struct TmaQuantizeShared {
    static constexpr int kRowBytes = DTYPE == 0 ? 128 : 64;
    // depth of the shared-memory ring: two stages where they fit in 32 KB, else one (the refill
    // of a single stage still hides behind the tile's arithmetic)
    static constexpr int kStages = 2 * THREADS * kRowBytes <= 32768 ? 2 : 1;
    alignas(1024) uint8_t stage[kStages][THREADS * kRowBytes];
    uint32_t slots[3][THREADS / 32];       // bucket maxima, rotating so no reset races a use
    uint32_t slots_lo[3][THREADS / 32];    // bucket minima of the (min, max) variant, as ordered bits
    alignas(8) uint64_t bar[kStages];
};

// Kernel-constant inputs of the TMA kernel beyond QuantizeArgs: the ten Philox round keys are
// computed on the host so the kernel reads them as constant operands.
struct TmaQuantizeConsts {
    RoundKeys rk;
    uint32_t full_tiles;         // leading tiles whose rows are all complete and in range
    uint32_t blk0_lo, blk0_hi;   // Philox block index of element 0: elem_offset / 8; the launch's blocks
                                 // all have the high half blk0_hi (tma_path_applies)
    PhiloxHead head;             // launch-wide part of the blocks of worker rk.worker
};

// What a tile needs to know about the worker it belongs to.  The one-worker kernel builds it
// from its kernel parameters (so every member stays a constant operand), the batched kernel from
// its table.
struct WorkerView {
    const CUtensorMap* map;
    const void* grad;
    uint32_t* codes;
    float* scales;
    PhiloxHead head;             // launch-wide part of this worker's Philox blocks
    uint32_t blk0_lo;            // low half of the Philox block index of the gradient's element 0
};

// One tile, the k-th of this CTA, tile `tile` of worker `wv`.  FULL: every thread owns a complete
// row (no bounds checks).  SHUFFLE: a bucket is an aligned power-of-two group of at most 32 rows
// (lane shuffles); otherwise a whole number of warps (one shared-memory atomic per warp).  After
// the tile's rows are in registers thread 0 calls `refill(stage, bar)` to start the copy that
// uses the stage next.  Returns false if the tile's copy never landed.
// GIVEN: the scale is not computed here: every tile belongs to one bucket whose scale already stands
// at wv.scales[0] (per-layer quantization after its max or norm pass, which also applies the flush);
// no reduction, no scale written.
template <int BITS, int DTYPE, int THREADS, bool FULL, bool SHUFFLE, bool NORM = false, bool GIVEN = false,
          typename Refill>
__device__ __forceinline__ bool quantize_tile(TmaQuantizeShared<DTYPE, THREADS>& sh, const WorkerView wv,
                                              const QuantizeArgs& a, const TmaQuantizeConsts& c,
                                              uint32_t k, uint32_t rot, uint32_t tile, Refill&& refill,
                                              uint32_t local_bucket, bool scale_writer)
{
    constexpr int kQuantStages = TmaQuantizeShared<DTYPE, THREADS>::kStages;
    const uint32_t t = threadIdx.x;
    const uint32_t row = tile * a.tile_rows + t;
    const bool active = FULL || (t < a.tile_rows && row < (uint32_t)a.nrows);
    const uint32_t stg = k % kQuantStages, parity = (k / kQuantStages) & 1;
    const uint32_t bar = smem_u32(&sh.bar[stg]);
    uint8_t* stage = sh.stage[stg];

    // The row's draws depend on nothing but its number.  From three bits on they are computed before the
    // tile's data is waited for: 16 more live registers (four CTAs per SM instead of five) against the
    // overlap of the Philox rounds with the wait.  Measured per 100 MB gradient in the batched launch with the
    // SM clock at its maximum: 17.0 against 18.0 us at K = 4, 18.3 against 18.6 us at K = 6, 19.7 against
    // 20.0 us at K = 8; no difference at one and two bits, which keep the fifth CTA.  (In a long run the power
    // limit sets the clock and both forms take the same time: the instruction count decides there.)
    // bf16 input (half the bytes per tile, no wait to cover) keeps the draws after the wait at every width:
    // 32.3 / 32.1 / 32.7 / 32.4 us per 50 M elements at K = 3 / 4 / 6 / 8 against 33.2 / 32.8 / 33.6 / 32.8 us.
    constexpr bool kEarlyDraw = !NORM && !GIVEN && DTYPE == 0 && BITS >= 3;
    uint32_t h[16];
    if (kEarlyDraw && active) draw_row_blocks_head(wv.blk0_lo + 4u * row, wv.head, c.rk, h);
    bool ok = mbar_try_wait(bar, parity);
    if (!ok) ok = mbar_wait(bar, parity, a.poll_limit);

    float x[32];
    if (active) {
        const bool ragged = !FULL && row >= (uint32_t)a.nrows_full;
        if (ragged) stage_ragged_row<DTYPE>(stage, (int)t, wv.grad, (uint64_t)row * 32, a.n);
        read_row_swizzled<DTYPE>(stage, (int)t, x);
        if (ragged) fence_proxy_async();     // orders those stores before the bulk copy that refills the stage
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) x[j] = 0.0f;
    }
    uint32_t m;
    uint32_t* slot = sh.slots[rot];          // rot = k % 3
    if constexpr (GIVEN) {
        m = 0u;
    } else if constexpr (NORM) {
        // L2-norm scale: the fixed tree over the rows' sums of squares - partner distance 1, 2, 4, ...
        // inside the warp, then (buckets of whole warps) the warp sums, one slot per warp.
        // The row's draws depend on nothing but its number: they are computed here, before the chain of
        // 32 dependent fused multiply-adds, so that the Philox rounds fill the chain's latency gaps.
        // (one launch per worker at n = 25 M: 22.3 / 22.5 / 23.0 us at K = 1 / 4 / 8 against 22.6 / 22.6 / 24.9 us)
        if (active) draw_row_blocks_head(wv.blk0_lo + 4u * row, wv.head, c.rk, h);
        float ss = row_sum_squares(x);
        const uint32_t lanes = SHUFFLE ? a.rows_per_bucket : 32u;
        for (uint32_t d = 1; d < lanes; d <<= 1) ss = __fadd_rn(ss, __shfl_xor_sync(0xFFFFFFFFu, ss, d));
        if (!SHUFFLE && (t & 31) == 0) slot[t >> 5] = __float_as_uint(ss);
        m = __float_as_uint(ss);
    } else {
        m = __float_as_uint(row_abs_max(x));
        if (SHUFFLE) {
            for (uint32_t d = a.rows_per_bucket >> 1; d > 0; d >>= 1)
                m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
        } else {
            m = __reduce_max_sync(0xFFFFFFFFu, m);
            if ((t & 31) == 0) atomicMax(&slot[local_bucket], m);
        }
    }
    if (__syncthreads_or(!ok)) return false;
    if (t == 0) refill(smem_u32(stage), bar);                    // every thread has read the stage
    if (!SHUFFLE && !GIVEN) {
        if constexpr (NORM) {
            // tree over the bucket's warp sums, zero leaves up to four (plain stores: nothing to reset;
            // the slot array is written again two barriers from here)
            static_assert(THREADS / 32 == 4, "the warp-sum tree is written for four warps");
            const uint32_t wpb = a.rows_per_bucket >> 5, first = local_bucket * wpb;
            float v[4];
#pragma unroll
            for (uint32_t i = 0; i < 4; ++i)
                v[i] = (i < wpb && first + i < 4u) ? __uint_as_float(slot[first + i]) : 0.0f;
            m = __float_as_uint(__fadd_rn(__fadd_rn(v[0], v[1]), __fadd_rn(v[2], v[3])));
        } else {
            m = slot[local_bucket];
            if (t < THREADS / 32) sh.slots[rot == 0 ? 2 : rot - 1][t] = 0u; // next used by this CTA's tile k + 2
        }
    }
    if (!active) return true;

    float sc = __uint_as_float(m);
    if constexpr (GIVEN) {
        sc = __ldg(wv.scales);           // final: the scale pass has applied the flush
    } else {
        if constexpr (NORM) sc = sc < flush_limit() ? 0.0f : __fsqrt_rn(sc);     // flush decided on the sum
        else if (sc < flush_limit()) sc = 0.0f;
        const uint32_t bucket = tile * a.buckets_per_tile + local_bucket;
        if (scale_writer && (FULL || bucket < a.nbuckets)) wv.scales[bucket] = sc;
    }

    const EncodeScale es = encode_scale<BITS>(sc);
    // Philox blocks of the row: elem_offset / 8 + 4 * row + 0 .. 3, all in the launch's high half
    if constexpr (!NORM && !kEarlyDraw)
        draw_row_blocks_head(wv.blk0_lo + 4u * row, wv.head, c.rk, h);
    uint32_t w[BITS];
    // The encode's arithmetic runs in packed fp32x2 instructions at every width: 14.3 instead of 17.0 - 17.6
    // executed instructions per element.  With the SM clock at its maximum this gains only at one and two bits
    // (16.6 against 17.2 us per 100 MB gradient at K = 1; from K = 4 on the constant pairs compete with the
    // early draws for registers), but a launch that runs for more than a few tens of milliseconds is held at
    // the board's power limit, where the clock falls until the power fits and fewer instructions per element
    // mean less time: 19.6 against 20.5 us at K = 3, 19.4 against 20.4 us at K = 4, 20.5 against 21.2 us at
    // K = 5, 20.6 against 21.6 us at K = 8 (batched launch, 0.3 s of launches back to back, 1650 - 1720 MHz).
    encode_pack_row_packed<BITS>(x, es, h, w);
    const uint64_t word0 = (uint64_t)row * BITS;
    if (FULL || (uint64_t)row * 32 + 32 <= a.n) {
        store_row_words<BITS>(wv.codes, word0, w);
    } else {
        mask_row_words<BITS>(w, (int)(a.n - (uint64_t)row * 32) * BITS);
#pragma unroll
        for (int j = 0; j < BITS; ++j)
            if (word0 + j < a.ncode_words) wv.codes[word0 + j] = w[j];
    }
    return true;
}

}  // namespace mqg
