// Worker side: per-bucket max-abs scale, stochastic-rounding encode and bit packing in one
// pass over the gradient (Quantize(g, K) of Algorithm 1, WorkerIterate).
//
// Work decomposition: the gradient is cut into rows of 32 elements; a CTA takes a tile of
// up to 256 rows that holds whole buckets, stages it in shared memory with coalesced 128-bit
// loads, and each thread then owns one row: it reads its 32 values from shared memory,
// takes part in the bucket's max reduction, draws its 32 sixteen-bit random numbers from
// four Philox blocks, encodes, packs into K words and stores them.  The gradient is read
// from HBM exactly once.
#include <string.h>

#include <atomic>

#include "mqg_quantize_tile.cuh"

namespace mqg {

// Max over the rows of each bucket of the tile.  `m` is this thread's row max (bit pattern of
// a non-negative float, so unsigned order = float order).  Returns the bucket's max.
__device__ __forceinline__ uint32_t bucket_max(uint32_t m, uint32_t rpb, uint32_t local_bucket,
                                               bool active, uint32_t* s_bucket)
{
    if ((rpb & (rpb - 1)) == 0 && rpb <= 32) {
        // a bucket is an aligned group of rpb lanes: butterfly inside the group
        for (uint32_t d = rpb >> 1; d > 0; d >>= 1)
            m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
        return m;
    }
    if (rpb % 32 == 0) {
        // a warp lies inside one bucket: one shared-memory atomic per warp
        m = __reduce_max_sync(0xFFFFFFFFu, m);
        if ((threadIdx.x & 31) == 0 && active) atomicMax(&s_bucket[local_bucket], m);
    } else if (active) {
        atomicMax(&s_bucket[local_bucket], m);
    }
    __syncthreads();
    return active ? s_bucket[local_bucket] : 0u;
}

template <int BITS, int DTYPE, bool ALIGNED_DRAWS>
__global__ void __launch_bounds__(kMaxTileRows)
quantize_pack_kernel(const QuantizeArgs a)
{
    __shared__ __align__(1024) float4 tile[kMaxTileRows * 8];
    __shared__ uint32_t s_bucket[kMaxTileRows];

    const uint32_t t = threadIdx.x;
    const uint64_t row0 = (uint64_t)blockIdx.x * a.tile_rows;
    const uint64_t rows_left = a.nrows - row0;
    const int rows = (int)(rows_left < a.tile_rows ? rows_left : a.tile_rows);

    if (t < a.buckets_per_tile) s_bucket[t] = 0u;
    if constexpr (DTYPE == 0)
        load_tile_f32<kMaxTileRows>(tile, static_cast<const float*>(a.grad) + row0 * 32,
                                    a.n - row0 * 32, rows);
    else
        load_tile_bf16<kMaxTileRows>(tile, static_cast<const uint16_t*>(a.grad) + row0 * 32,
                                     a.n - row0 * 32, rows);
    __syncthreads();

    const bool active = t < (uint32_t)rows;
    float x[32];
    if (active) read_row(tile, (int)t, x);
    else {
#pragma unroll
        for (int j = 0; j < 32; ++j) x[j] = 0.0f;
    }

    const float mx = row_abs_max(x);

    const uint32_t local_bucket = t / a.rows_per_bucket;
    const uint32_t mbits = bucket_max(__float_as_uint(mx), a.rows_per_bucket, local_bucket, active,
                                      s_bucket);
    if (!active) return;

    float s = __uint_as_float(mbits);
    if (s < flush_limit()) s = 0.0f;
    const uint64_t bucket = (uint64_t)blockIdx.x * a.buckets_per_tile + local_bucket;
    if (t % a.rows_per_bucket == 0 && bucket < a.nbuckets) a.scales[bucket] = s;

    const EncodeScale es = encode_scale<BITS>(s);
    const uint64_t row = row0 + t;
    uint32_t h[16];
    if constexpr (ALIGNED_DRAWS) draw_row_aligned(a.elem_offset + row * 32, make_round_keys(a.key), h);
    else draw_row_unaligned(a.elem_offset + row * 32, a.key, h);

    uint32_t w[BITS];
    encode_pack_row<BITS>(x, es, h, w);

    const uint64_t word0 = row * BITS;
    const uint64_t e0 = row * 32;
    if (e0 + 32 <= a.n) {
        store_row_words<BITS>(a.codes, word0, w);
    } else {
        // ragged last row: pad bits are zero, words beyond the stream are not written
        mask_row_words<BITS>(w, (int)(a.n - e0) * BITS);
#pragma unroll
        for (int k = 0; k < BITS; ++k)
            if (word0 + k < a.ncode_words) a.codes[word0 + k] = w[k];
    }
}



// The same tile for the (min, max) nearest-rounding variant: two reductions instead of one, two
// floats per bucket (ranges[2b] = lo, ranges[2b + 1] = hi), no random draws.  Padding must not
// take part in the range: the elements a ragged row lacks repeat its first element, and threads
// without a row contribute the identities.  sh.slots holds maxima, sh.slots_lo minima, both as
// ordered bits; the kernel initialises them to the identities.
template <int BITS, int DTYPE, int THREADS, bool FULL, bool SHUFFLE, typename Refill>
__device__ __forceinline__ bool range_quantize_tile(TmaQuantizeShared<DTYPE, THREADS>& sh, const WorkerView wv,
                                                    const QuantizeArgs& a, uint32_t k, uint32_t rot, uint32_t tile,
                                                    Refill&& refill, uint32_t local_bucket, bool scale_writer)
{
    constexpr int kQuantStages = TmaQuantizeShared<DTYPE, THREADS>::kStages;
    const uint32_t t = threadIdx.x;
    const uint32_t row = tile * a.tile_rows + t;
    const bool active = FULL || (t < a.tile_rows && row < (uint32_t)a.nrows);
    const uint32_t stg = k % kQuantStages, parity = (k / kQuantStages) & 1;
    const uint32_t bar = smem_u32(&sh.bar[stg]);
    uint8_t* stage = sh.stage[stg];

    bool ok = mbar_try_wait(bar, parity);
    if (!ok) ok = mbar_wait(bar, parity, a.poll_limit);

    float x[32];
    uint32_t mlo = kOrderedMinIdentity, mhi = kOrderedMaxIdentity;
    if (active) {
        const bool ragged = !FULL && row >= (uint32_t)a.nrows_full;
        if (ragged) stage_ragged_row<DTYPE>(stage, (int)t, wv.grad, (uint64_t)row * 32, a.n);
        read_row_swizzled<DTYPE>(stage, (int)t, x);
        if (ragged) fence_proxy_async();     // orders those stores before the bulk copy that refills the stage
        if (!FULL) {
            const uint64_t left = a.n - (uint64_t)row * 32;      // >= 1
#pragma unroll
            for (int j = 1; j < 32; ++j) x[j] = ((uint64_t)j < left) ? x[j] : x[0];
        }
        float lo, hi;
        row_min_max(x, lo, hi);
        mlo = ordered_bits(lo); mhi = ordered_bits(hi);
    }
    uint32_t* slot_hi = sh.slots[rot];       // rot = k % 3
    uint32_t* slot_lo = sh.slots_lo[rot];
    if (SHUFFLE) {
        for (uint32_t d = a.rows_per_bucket >> 1; d > 0; d >>= 1) {
            mlo = min(mlo, __shfl_xor_sync(0xFFFFFFFFu, mlo, d));
            mhi = max(mhi, __shfl_xor_sync(0xFFFFFFFFu, mhi, d));
        }
    } else {
        mlo = __reduce_min_sync(0xFFFFFFFFu, mlo);
        mhi = __reduce_max_sync(0xFFFFFFFFu, mhi);
        if ((t & 31) == 0) { atomicMin(&slot_lo[local_bucket], mlo); atomicMax(&slot_hi[local_bucket], mhi); }
    }
    if (__syncthreads_or(!ok)) return false;
    if (t == 0) refill(smem_u32(stage), bar);                    // every thread has read the stage
    if (!SHUFFLE) {
        mlo = slot_lo[local_bucket]; mhi = slot_hi[local_bucket];
        if (t < THREADS / 32) {                                  // next used by this CTA's tile k + 2
            sh.slots[rot == 0 ? 2 : rot - 1][t] = kOrderedMaxIdentity;
            sh.slots_lo[rot == 0 ? 2 : rot - 1][t] = kOrderedMinIdentity;
        }
    }
    if (!active) return true;

    // a zero of either sign is stored as +0
    const float lo = __fadd_rn(from_ordered_bits(mlo), 0.0f), hi = __fadd_rn(from_ordered_bits(mhi), 0.0f);
    const uint32_t bucket = tile * a.buckets_per_tile + local_bucket;
    if (scale_writer && (FULL || bucket < a.nbuckets))
        reinterpret_cast<float2*>(wv.scales)[bucket] = make_float2(lo, hi);

    const RangeEncodeScale es = range_encode_scale<BITS>(lo, hi);
    uint32_t w[BITS];
    range_encode_pack_row<BITS>(x, es, w);
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

// MODE: kMaxAbs = the main codec, kRange = the (min, max) variant, kNorm = the L2-norm scale variant,
// kGiven = encode against a scale computed by an earlier pass (long segments of the per-layer quantizers).
enum : int { kMaxAbs = 0, kRange = 1, kNorm = 2, kGiven = 3 };

template <int BITS, int DTYPE, int THREADS, bool SHUFFLE, int MODE = kMaxAbs>
__global__ void __launch_bounds__(THREADS, 512 / THREADS)
quantize_tma_kernel(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ QuantizeArgs a,
                    const __grid_constant__ TmaQuantizeConsts c, unsigned int* __restrict__ timeouts)
{
    using Shared = TmaQuantizeShared<DTYPE, THREADS>;
    constexpr int kQuantStages = Shared::kStages;
    __shared__ Shared sh;

    const uint32_t t = threadIdx.x;
    const uint32_t stride = gridDim.x;
    const uint32_t box_bytes = a.tile_rows * Shared::kRowBytes;
    if (t == 0) {
        for (int s = 0; s < kQuantStages; ++s) mbar_init(smem_u32(&sh.bar[s]), 1);
        fence_barrier_init();
    }
    if (t < 3 * (THREADS / 32)) {
        (&sh.slots[0][0])[t] = 0u;     // = kOrderedMaxIdentity
        (&sh.slots_lo[0][0])[t] = kOrderedMinIdentity;
    }
    if (t == 0) prefetch_tensormap(&tmap);
    grid_dependency_release();
    __syncthreads();
    grid_dependency_wait();            // nothing above touches global memory
    uint32_t tile = blockIdx.x;
    if (t == 0) {
        for (uint32_t s = 0; s < (uint32_t)kQuantStages && tile + s * stride < a.ntiles; ++s) {
            mbar_expect_tx(smem_u32(&sh.bar[s]), box_bytes);
            if (!a.arm_only)
                tma_load_2d(smem_u32(sh.stage[s]), &tmap, 0, (int)((tile + s * stride) * a.tile_rows),
                            smem_u32(&sh.bar[s]));
        }
    }
    const uint32_t local_bucket = t / a.rows_per_bucket;
    const bool scale_writer = (t % a.rows_per_bucket) == 0;
    const uint32_t ahead = kQuantStages * stride;       // distance to the tile that refills a stage
    const WorkerView wv = {&tmap, a.grad, a.codes, a.scales, c.head, c.blk0_lo};

    uint32_t k = 0, rot = 0;
    bool ok = true;
#pragma unroll 1
    for (; ok && tile < a.ntiles; tile += stride, ++k, rot = (rot == 2 ? 0 : rot + 1)) {
        auto refill = [&](uint32_t stage, uint32_t bar) {
            const uint32_t next_tile = tile + ahead;
            if (next_tile < a.ntiles) {
                mbar_expect_tx(bar, box_bytes);
                if (!a.arm_only) tma_load_2d(stage, &tmap, 0, (int)(next_tile * a.tile_rows), bar);
            }
        };
        if constexpr (MODE == kRange) {
            if (tile < c.full_tiles)
                ok = range_quantize_tile<BITS, DTYPE, THREADS, true, SHUFFLE>(sh, wv, a, k, rot, tile, refill,
                                                                               local_bucket, scale_writer);
            else
                ok = range_quantize_tile<BITS, DTYPE, THREADS, false, SHUFFLE>(sh, wv, a, k, rot, tile, refill,
                                                                                local_bucket, scale_writer);
        } else {
            constexpr bool NORM = MODE == kNorm, GIVEN = MODE == kGiven;
            if (tile < c.full_tiles)
                ok = quantize_tile<BITS, DTYPE, THREADS, true, SHUFFLE, NORM, GIVEN>(sh, wv, a, c, k, rot, tile, refill,
                                                                                      local_bucket, scale_writer);
            else
                ok = quantize_tile<BITS, DTYPE, THREADS, false, SHUFFLE, NORM, GIVEN>(sh, wv, a, c, k, rot, tile, refill,
                                                                                       local_bucket, scale_writer);
        }
    }
    if (!ok) {
        // A copy never landed: record it, then give the copies still in flight (the one that was
        // being waited for and those issued after it) a last bounded chance to finish before the
        // CTA's shared memory can be handed to another CTA.  The loop's update ran once after the
        // failing tile, so that tile is k - 1 / tile - stride.
        if (t == 0) {
            atomicAdd(timeouts, 1u);
            uint32_t j = k - 1, tl = tile - stride;
            for (int s = 0; s < kQuantStages && tl < a.ntiles; ++s, ++j, tl += stride)
                mbar_wait(smem_u32(&sh.bar[j % kQuantStages]), (j / kQuantStages) & 1, a.poll_limit);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------
// Several workers' gradients in ONE launch (the server-side simulation of P workers, or a host
// with several model replicas on one device).  The launch's fixed costs - scheduling the grid,
// the first tiles' DRAM latency, the last tiles' drain - are paid once instead of once per
// worker.  The tiles of all workers form one sequence v = worker * ntiles + tile, walked exactly
// like the one-worker kernel walks its tiles; every tile is encoded by the same code, so worker
// w's outputs are bit-identical to a one-worker launch with worker id first_worker + w.
// ---------------------------------------------------------------------------------------
struct WorkerTable {
    CUtensorMap map[kMaxWorkers];
    const void* grad[kMaxWorkers];
    uint32_t* codes[kMaxWorkers];
    float* scales[kMaxWorkers];
    PhiloxHead head[kMaxWorkers];
};

template <int BITS, int DTYPE, bool SHUFFLE, int MODE>
__global__ void __launch_bounds__(128, 4)
quantize_workers_kernel(const __grid_constant__ WorkerTable tab, const __grid_constant__ QuantizeArgs a,
                        const __grid_constant__ TmaQuantizeConsts c, uint32_t total_tiles,
                        unsigned int* __restrict__ timeouts)
{
    constexpr int THREADS = 128;
    using Shared = TmaQuantizeShared<DTYPE, THREADS>;
    constexpr int kQuantStages = Shared::kStages;
    __shared__ Shared sh;

    const uint32_t t = threadIdx.x;
    const uint32_t stride = gridDim.x;
    const uint32_t box_bytes = a.tile_rows * Shared::kRowBytes;
    if (t == 0) {
        for (int s = 0; s < kQuantStages; ++s) mbar_init(smem_u32(&sh.bar[s]), 1);
        fence_barrier_init();
    }
    if (t < 3 * (THREADS / 32)) {
        (&sh.slots[0][0])[t] = 0u;     // = kOrderedMaxIdentity
        (&sh.slots_lo[0][0])[t] = kOrderedMinIdentity;
    }
    grid_dependency_release();
    __syncthreads();
    grid_dependency_wait();            // nothing above touches global memory

    // Position in the sequence of all workers' tiles, as (worker, tile of the worker), advanced by
    // `stride` tiles at a time without a division.
    struct Pos { uint32_t w, tile; };
    auto advance = [&](Pos& p, uint32_t by) {
        p.tile += by;
        while (p.tile >= a.ntiles) { p.tile -= a.ntiles; ++p.w; }
    };
    auto load_tile = [&](const Pos& p, uint32_t stage, uint32_t bar) {     // thread 0 only
        mbar_expect_tx(bar, box_bytes);
        if (!a.arm_only) tma_load_2d(stage, &tab.map[p.w], 0, (int)(p.tile * a.tile_rows), bar);
    };
    uint32_t v = blockIdx.x;
    Pos cur = {0u, 0u}, fill = {0u, 0u};   // the tile in work and the one kQuantStages turns ahead of it
    advance(cur, v);
    advance(fill, v);
    uint32_t vfill = v;
    for (uint32_t s = 0; s < (uint32_t)kQuantStages; ++s) {
        if (t == 0 && vfill < total_tiles) load_tile(fill, smem_u32(sh.stage[s]), smem_u32(&sh.bar[s]));
        vfill += stride;
        if (vfill < total_tiles) advance(fill, stride);
    }
    const uint32_t local_bucket = t / a.rows_per_bucket;
    const bool scale_writer = (t % a.rows_per_bucket) == 0;

    uint32_t k = 0, rot = 0;
    bool ok = true;
    uint32_t w = cur.w, tile = cur.tile;
    // Outer loop: the workers this CTA's walk passes through; inner loop: its tiles of that worker.  The
    // worker's table entries (pointers, Philox head) are fetched once per worker, not once per tile:
    // indexed loads from the kernel's parameter block are long-latency loads the tile would wait for.
#pragma unroll 1
    while (ok && v < total_tiles) {
        const WorkerView wv = {&tab.map[w], tab.grad[w], tab.codes[w], tab.scales[w], tab.head[w], c.blk0_lo};
#pragma unroll 1
        for (; ok && tile < a.ntiles && v < total_tiles;
             tile += stride, v += stride, ++k, rot = (rot == 2 ? 0 : rot + 1)) {
            auto refill = [&](uint32_t stage, uint32_t bar) {
                if (vfill < total_tiles) load_tile(fill, stage, bar);
            };
            if constexpr (MODE == kRange) {
                if (tile < c.full_tiles)
                    ok = range_quantize_tile<BITS, DTYPE, THREADS, true, SHUFFLE>(sh, wv, a, k, rot, tile, refill,
                                                                                   local_bucket, scale_writer);
                else
                    ok = range_quantize_tile<BITS, DTYPE, THREADS, false, SHUFFLE>(sh, wv, a, k, rot, tile, refill,
                                                                                    local_bucket, scale_writer);
            } else {
                constexpr bool NORM = MODE == kNorm;
                if (tile < c.full_tiles)
                    ok = quantize_tile<BITS, DTYPE, THREADS, true, SHUFFLE, NORM>(sh, wv, a, c, k, rot, tile, refill,
                                                                                   local_bucket, scale_writer);
                else
                    ok = quantize_tile<BITS, DTYPE, THREADS, false, SHUFFLE, NORM>(sh, wv, a, c, k, rot, tile, refill,
                                                                                    local_bucket, scale_writer);
            }
            vfill += stride;
            if (vfill < total_tiles) advance(fill, stride);
        }
        while (tile >= a.ntiles) { tile -= a.ntiles; ++w; }     // into the next worker (if the walk goes on)
    }
    if (!ok) {                         // as in the one-worker kernel
        if (t == 0) {
            atomicAdd(timeouts, 1u);
            uint32_t j = k - 1, vl = v - stride;
            for (int s = 0; s < kQuantStages && vl < total_tiles; ++s, ++j, vl += stride)
                mbar_wait(smem_u32(&sh.bar[j % kQuantStages]), (j / kQuantStages) & 1, a.poll_limit);
        }
        __syncthreads();
    }
}

template <int BITS>
static cudaError_t launch_bits(const QuantizeArgs& a, int dtype, bool aligned, unsigned grid,
                               cudaStream_t stream)
{
    const dim3 g(grid), b(kMaxTileRows);
    if (dtype == 0) {
        if (aligned) quantize_pack_kernel<BITS, 0, true><<<g, b, 0, stream>>>(a);
        else quantize_pack_kernel<BITS, 0, false><<<g, b, 0, stream>>>(a);
    } else {
        if (aligned) quantize_pack_kernel<BITS, 1, true><<<g, b, 0, stream>>>(a);
        else quantize_pack_kernel<BITS, 1, false><<<g, b, 0, stream>>>(a);
    }
    return cudaGetLastError();
}

template <int BITS, int DTYPE, int THREADS, bool SHUFFLE, int MODE = kMaxAbs>
static cudaError_t launch_tma_inst(const CUtensorMap& map, const QuantizeArgs& a,
                                   const TmaQuantizeConsts& c, unsigned int* timeouts,
                                   cudaStream_t stream)
{
    auto kernel = quantize_tma_kernel<BITS, DTYPE, THREADS, SHUFFLE, MODE>;
    static std::atomic<int> grid_cap[64];                  // per device; 0 = not yet queried (zero-initialised)
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int cap = grid_cap[dev].load(std::memory_order_relaxed);
    if (cap == 0) {
        int occ = 0, sms = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, THREADS, 0);
        if (err != cudaSuccess) return err;
        err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (err != cudaSuccess) return err;
        cap = sms * (occ > 0 ? occ : 1);
        grid_cap[dev].store(cap, std::memory_order_relaxed);   // every thread computes the same value
    }
    unsigned grid = (unsigned)cap;
    if (grid > a.ntiles) grid = a.ntiles;
    return launch_pdl(kernel, grid, THREADS, stream, map, a, c, timeouts);
}

template <int BITS>
static cudaError_t launch_tma_bits(const CUtensorMap& map, const QuantizeArgs& a,
                                   const TmaQuantizeConsts& c, int dtype, int threads, bool shuffle,
                                   unsigned int* timeouts, cudaStream_t stream)
{
#define MQG_TMA_CASE(D, T, S) return launch_tma_inst<BITS, D, T, S>(map, a, c, timeouts, stream)
    if (dtype == 0) {
        if (threads == 128) { if (shuffle) MQG_TMA_CASE(0, 128, true); else MQG_TMA_CASE(0, 128, false); }
        MQG_TMA_CASE(0, 256, false);
    }
    if (threads == 128) { if (shuffle) MQG_TMA_CASE(1, 128, true); else MQG_TMA_CASE(1, 128, false); }
    MQG_TMA_CASE(1, 256, false);
#undef MQG_TMA_CASE
}

// The Philox blocks of the launch (four per row, from block elem_offset / 8 on) all have the same
// high half of the 64-bit block index, so that the part of a block that depends on it is a launch
// constant (PhiloxHead) and a row's block numbers need no carry.  Fails only for a gradient that
// straddles a multiple of 2^35 elements of the flat model; that one takes the general kernels.
static bool blocks_share_high_half(uint64_t n, uint64_t elem_offset)
{
    const uint64_t first = elem_offset >> 3, last = first + 4 * ((n + 31) / 32) - 1;
    return (first >> 32) == (last >> 32);
}

// TMA path: whole rows exist, draws are block-aligned, and a bucket is either an aligned
// power-of-two group of at most 32 rows or a whole number of warps.
static bool tma_path_applies(uint64_t n, uint64_t rpb, uint64_t elem_offset)
{
    if (n < 32 * 64 || (elem_offset & 7u) != 0 || rpb == 0 || rpb > (uint64_t)kMaxTileRows) return false;
    if (n / 32 > 0x7FFFFFFFull) return false;
    if (!blocks_share_high_half(n, elem_offset)) return false;
    return ((rpb & (rpb - 1)) == 0 && rpb <= 32) || rpb % 32 == 0;
}

// Fills the arguments every fused kernel shares.  Returns rows per bucket.
static uint64_t fill_args(QuantizeArgs& a, const void* grad, uint64_t n, int bits, uint64_t bucket,
                          uint64_t seed, uint32_t* codes, float* scales, uint32_t worker, uint32_t step,
                          uint64_t elem_offset)
{
    a.grad = grad; a.codes = codes; a.scales = scales;
    a.n = n;
    a.nrows = (n + 31) / 32;
    a.nbuckets = (n + bucket - 1) / bucket;
    a.ncode_words = (n * (uint64_t)bits + 31) / 32;
    a.elem_offset = elem_offset;
    // bucket % 32 == 0 and bucket <= 8192, or a single bucket of at most 8192 elements
    const uint64_t rpb = (bucket >= n) ? a.nrows : bucket / 32;
    a.rows_per_bucket = (uint32_t)rpb;
    a.buckets_per_tile = (uint32_t)(kMaxTileRows / rpb);
    a.tile_rows = a.buckets_per_tile * a.rows_per_bucket;
    a.key.seed_lo = (uint32_t)seed; a.key.seed_hi = (uint32_t)(seed >> 32);
    a.key.worker = worker; a.key.step = step;
    a.nrows_full = n / 32;
    const WaitPolicy policy = wait_policy();
    a.poll_limit = policy.poll_limit;
    a.arm_only = policy.arm_only;
    return rpb;
}

// Tile shape and constants of the TMA kernels (tma_path_applies() holds).  Returns the CTA size,
// or 0 if the tile count does not fit.
static int fill_tma_args(QuantizeArgs& a, TmaQuantizeConsts& c, uint64_t rpb)
{
    const int threads = rpb <= 128 ? 128 : 256;
    a.buckets_per_tile = (uint32_t)(threads / rpb);
    a.tile_rows = a.buckets_per_tile * a.rows_per_bucket;
    const uint64_t nt = (a.nrows + a.tile_rows - 1) / a.tile_rows;
    if (nt > 0x7FFFFFFFull) return 0;
    a.ntiles = (uint32_t)nt;
    uint32_t k0 = a.key.seed_lo, k1 = a.key.seed_hi;
    for (int r = 0; r < 10; ++r) {
        c.rk.k0[r] = k0; c.rk.k1[r] = k1;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    c.rk.worker = a.key.worker; c.rk.step = a.key.step;
    c.full_tiles = a.tile_rows == (uint32_t)threads ? (uint32_t)(a.nrows_full / a.tile_rows) : 0u;
    c.blk0_lo = (uint32_t)(a.elem_offset >> 3); c.blk0_hi = (uint32_t)(a.elem_offset >> 35);
    c.head = philox_head(c.blk0_hi, c.rk.worker, c.rk.k0[0]);
    return threads;
}

cudaError_t launch_quantize_fused(const void* grad, uint64_t n, int bits, uint64_t bucket,
                                  uint64_t seed, uint32_t* codes, float* scales, int dtype,
                                  uint32_t worker, uint32_t step, uint64_t elem_offset,
                                  cudaStream_t stream)
{
    QuantizeArgs a;
    const uint64_t rpb = fill_args(a, grad, n, bits, bucket, seed, codes, scales, worker, step, elem_offset);
    if (tma_path_applies(n, rpb, elem_offset)) {
        TmaQuantizeConsts c;
        const int threads = fill_tma_args(a, c, rpb);
        if (threads == 0) return cudaErrorInvalidValue;
        CUtensorMap map;
        const char* why = nullptr;
        unsigned int* timeouts = wait_timeout_counter();
        if (timeouts != nullptr &&
            encode_rows_map(&map, grad, a.nrows_full, dtype == 0 ? 4 : 2, 32, a.tile_rows, &why)) {
            const bool shuffle = rpb <= 32;
            switch (bits) {
                case 1: return launch_tma_bits<1>(map, a, c, dtype, threads, shuffle, timeouts, stream);
                case 2: return launch_tma_bits<2>(map, a, c, dtype, threads, shuffle, timeouts, stream);
                case 3: return launch_tma_bits<3>(map, a, c, dtype, threads, shuffle, timeouts, stream);
                case 4: return launch_tma_bits<4>(map, a, c, dtype, threads, shuffle, timeouts, stream);
                case 5: return launch_tma_bits<5>(map, a, c, dtype, threads, shuffle, timeouts, stream);
                case 6: return launch_tma_bits<6>(map, a, c, dtype, threads, shuffle, timeouts, stream);
                case 7: return launch_tma_bits<7>(map, a, c, dtype, threads, shuffle, timeouts, stream);
                case 8: return launch_tma_bits<8>(map, a, c, dtype, threads, shuffle, timeouts, stream);
            }
            return cudaErrorInvalidValue;
        }
        return cudaErrorNotSupported;        // the driver cannot encode a tensor map: no silent detour
    }
    a.buckets_per_tile = (uint32_t)(kMaxTileRows / rpb);
    a.tile_rows = a.buckets_per_tile * a.rows_per_bucket;
    const uint64_t ntiles = (a.nrows + a.tile_rows - 1) / a.tile_rows;
    if (ntiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    a.ntiles = (uint32_t)ntiles;
    const bool aligned = (elem_offset & 7u) == 0;
    switch (bits) {
        case 1: return launch_bits<1>(a, dtype, aligned, (unsigned)ntiles, stream);
        case 2: return launch_bits<2>(a, dtype, aligned, (unsigned)ntiles, stream);
        case 3: return launch_bits<3>(a, dtype, aligned, (unsigned)ntiles, stream);
        case 4: return launch_bits<4>(a, dtype, aligned, (unsigned)ntiles, stream);
        case 5: return launch_bits<5>(a, dtype, aligned, (unsigned)ntiles, stream);
        case 6: return launch_bits<6>(a, dtype, aligned, (unsigned)ntiles, stream);
        case 7: return launch_bits<7>(a, dtype, aligned, (unsigned)ntiles, stream);
        case 8: return launch_bits<8>(a, dtype, aligned, (unsigned)ntiles, stream);
    }
    return cudaErrorInvalidValue;
}

template <int BITS, int DTYPE, bool SHUFFLE, int MODE>
static cudaError_t launch_workers_inst(const WorkerTable& tab, const QuantizeArgs& a,
                                       const TmaQuantizeConsts& c, uint32_t total_tiles,
                                       unsigned int* timeouts, cudaStream_t stream)
{
    auto kernel = quantize_workers_kernel<BITS, DTYPE, SHUFFLE, MODE>;
    static std::atomic<int> grid_cap[64];                  // per device; 0 = not yet queried (zero-initialised)
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int cap = grid_cap[dev].load(std::memory_order_relaxed);
    if (cap == 0) {
        int occ = 0, sms = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, 128, 0);
        if (err != cudaSuccess) return err;
        err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (err != cudaSuccess) return err;
        cap = sms * (occ > 0 ? occ : 1);
        grid_cap[dev].store(cap, std::memory_order_relaxed);   // every thread computes the same value
    }
    unsigned grid = (unsigned)cap;
    if (grid > total_tiles) grid = total_tiles;
    return launch_pdl(kernel, grid, 128, stream, tab, a, c, total_tiles, timeouts);
}

template <int BITS, int MODE>
static cudaError_t launch_workers_bits(const WorkerTable& tab, const QuantizeArgs& a,
                                       const TmaQuantizeConsts& c, uint32_t total_tiles, int dtype,
                                       bool shuffle, unsigned int* timeouts, cudaStream_t stream)
{
    if (dtype == 0)
        return shuffle ? launch_workers_inst<BITS, 0, true, MODE>(tab, a, c, total_tiles, timeouts, stream)
                       : launch_workers_inst<BITS, 0, false, MODE>(tab, a, c, total_tiles, timeouts, stream);
    return shuffle ? launch_workers_inst<BITS, 1, true, MODE>(tab, a, c, total_tiles, timeouts, stream)
                   : launch_workers_inst<BITS, 1, false, MODE>(tab, a, c, total_tiles, timeouts, stream);
}

bool quantize_workers_applies(int W, uint64_t n, uint64_t bucket, uint64_t elem_offset)
{
    if (W < 2 || W > kMaxWorkers || n == 0) return false;
    const uint64_t nrows = (n + 31) / 32;
    const uint64_t rpb = (bucket >= n) ? nrows : bucket / 32;
    if ((bucket < n ? bucket : n) > (uint64_t)kMaxFusedBucket) return false;
    if (!tma_path_applies(n, rpb, elem_offset) || rpb > 128) return false;
    const uint64_t tile_rows = (128 / rpb) * rpb;
    const uint64_t nt = (nrows + tile_rows - 1) / tile_rows;
    return nt * (uint64_t)W <= 0x7FFFFFFFull;
}

cudaError_t launch_quantize_workers(const void* const* grads, int W, uint64_t n, int bits,
                                    uint64_t bucket, uint64_t seed, uint32_t* const* codes,
                                    float* const* scales, int dtype, uint32_t first_worker,
                                    uint32_t step, uint64_t elem_offset, int mode, cudaStream_t stream)
{
    QuantizeArgs a;
    const uint64_t rpb = fill_args(a, grads[0], n, bits, bucket, seed, codes[0], scales[0], first_worker,
                                   step, elem_offset);
    TmaQuantizeConsts c;
    if (fill_tma_args(a, c, rpb) != 128) return cudaErrorInvalidValue;
    unsigned int* timeouts = wait_timeout_counter();
    if (timeouts == nullptr) return cudaErrorNotSupported;
    WorkerTable tab;
    memset(&tab, 0, sizeof(tab));
    for (int w = 0; w < W; ++w) {
        const char* why = nullptr;
        if (!encode_rows_map(&tab.map[w], grads[w], a.nrows_full, dtype == 0 ? 4 : 2, 32, a.tile_rows, &why))
            return cudaErrorNotSupported;
        tab.grad[w] = grads[w]; tab.codes[w] = codes[w]; tab.scales[w] = scales[w];
        tab.head[w] = philox_head(c.blk0_hi, first_worker + (uint32_t)w, c.rk.k0[0]);
    }
    const uint32_t total_tiles = a.ntiles * (uint32_t)W;
    const bool shuffle = rpb <= 32;
    switch (bits) {
#define MQG_WORKERS_CASE(B) \
        case B: return mode == kNorm ? launch_workers_bits<B, kNorm>(tab, a, c, total_tiles, dtype, shuffle, timeouts, stream) \
                     : mode == kRange ? launch_workers_bits<B, kRange>(tab, a, c, total_tiles, dtype, shuffle, timeouts, stream) \
                     : launch_workers_bits<B, kMaxAbs>(tab, a, c, total_tiles, dtype, shuffle, timeouts, stream)
        MQG_WORKERS_CASE(1); MQG_WORKERS_CASE(2); MQG_WORKERS_CASE(3); MQG_WORKERS_CASE(4);
        MQG_WORKERS_CASE(5); MQG_WORKERS_CASE(6); MQG_WORKERS_CASE(7); MQG_WORKERS_CASE(8);
#undef MQG_WORKERS_CASE
    }
    return cudaErrorInvalidValue;
}

// ---- (min, max) nearest-rounding variant on the TMA kernel (buckets of at most 128 rows) ----
template <int BITS>
static cudaError_t launch_range_bits(const CUtensorMap& map, const QuantizeArgs& a, const TmaQuantizeConsts& c,
                                     int dtype, bool shuffle, unsigned int* timeouts, cudaStream_t stream)
{
    if (dtype == 0)
        return shuffle ? launch_tma_inst<BITS, 0, 128, true, kRange>(map, a, c, timeouts, stream)
                       : launch_tma_inst<BITS, 0, 128, false, kRange>(map, a, c, timeouts, stream);
    return shuffle ? launch_tma_inst<BITS, 1, 128, true, kRange>(map, a, c, timeouts, stream)
                   : launch_tma_inst<BITS, 1, 128, false, kRange>(map, a, c, timeouts, stream);
}

bool quantize_range_fused_applies(uint64_t n, uint64_t bucket)
{
    if (n == 0) return false;
    const uint64_t nrows = (n + 31) / 32;
    const uint64_t rpb = (bucket >= n) ? nrows : bucket / 32;
    return tma_path_applies(n, rpb, 0) && rpb <= 128;
}

cudaError_t launch_quantize_range_fused(const void* grad, uint64_t n, int bits, uint64_t bucket,
                                        uint32_t* codes, float* ranges, int dtype, cudaStream_t stream)
{
    QuantizeArgs a;
    const uint64_t rpb = fill_args(a, grad, n, bits, bucket, 0, codes, ranges, 0, 0, 0);
    TmaQuantizeConsts c;
    if (fill_tma_args(a, c, rpb) != 128) return cudaErrorInvalidValue;
    unsigned int* timeouts = wait_timeout_counter();
    if (timeouts == nullptr) return cudaErrorNotSupported;
    CUtensorMap map;
    const char* why = nullptr;
    if (!encode_rows_map(&map, grad, a.nrows_full, dtype == 0 ? 4 : 2, 32, a.tile_rows, &why))
        return cudaErrorNotSupported;
    const bool shuffle = rpb <= 32;
    switch (bits) {
        case 1: return launch_range_bits<1>(map, a, c, dtype, shuffle, timeouts, stream);
        case 2: return launch_range_bits<2>(map, a, c, dtype, shuffle, timeouts, stream);
        case 3: return launch_range_bits<3>(map, a, c, dtype, shuffle, timeouts, stream);
        case 4: return launch_range_bits<4>(map, a, c, dtype, shuffle, timeouts, stream);
        case 5: return launch_range_bits<5>(map, a, c, dtype, shuffle, timeouts, stream);
        case 6: return launch_range_bits<6>(map, a, c, dtype, shuffle, timeouts, stream);
        case 7: return launch_range_bits<7>(map, a, c, dtype, shuffle, timeouts, stream);
        case 8: return launch_range_bits<8>(map, a, c, dtype, shuffle, timeouts, stream);
    }
    return cudaErrorInvalidValue;
}

// ---- L2-norm scale variant on the TMA kernel (buckets of at most 128 rows, block-aligned draws) ----
template <int BITS>
static cudaError_t launch_norm_bits(const CUtensorMap& map, const QuantizeArgs& a, const TmaQuantizeConsts& c,
                                    int dtype, bool shuffle, unsigned int* timeouts, cudaStream_t stream)
{
    if (dtype == 0)
        return shuffle ? launch_tma_inst<BITS, 0, 128, true, kNorm>(map, a, c, timeouts, stream)
                       : launch_tma_inst<BITS, 0, 128, false, kNorm>(map, a, c, timeouts, stream);
    return shuffle ? launch_tma_inst<BITS, 1, 128, true, kNorm>(map, a, c, timeouts, stream)
                   : launch_tma_inst<BITS, 1, 128, false, kNorm>(map, a, c, timeouts, stream);
}

bool quantize_norm_fused_applies(uint64_t n, uint64_t bucket, uint64_t elem_offset)
{
    if (n == 0) return false;
    const uint64_t nrows = (n + 31) / 32;
    const uint64_t rpb = (bucket >= n) ? nrows : bucket / 32;
    return tma_path_applies(n, rpb, elem_offset) && rpb <= 128;
}

cudaError_t launch_quantize_norm_fused(const void* grad, uint64_t n, int bits, uint64_t bucket, uint64_t seed,
                                       uint32_t* codes, float* scales, int dtype, uint32_t worker,
                                       uint32_t step, uint64_t elem_offset, cudaStream_t stream)
{
    QuantizeArgs a;
    const uint64_t rpb = fill_args(a, grad, n, bits, bucket, seed, codes, scales, worker, step, elem_offset);
    TmaQuantizeConsts c;
    if (fill_tma_args(a, c, rpb) != 128) return cudaErrorInvalidValue;
    unsigned int* timeouts = wait_timeout_counter();
    if (timeouts == nullptr) return cudaErrorNotSupported;
    CUtensorMap map;
    const char* why = nullptr;
    if (!encode_rows_map(&map, grad, a.nrows_full, dtype == 0 ? 4 : 2, 32, a.tile_rows, &why))
        return cudaErrorNotSupported;
    const bool shuffle = rpb <= 32;
    switch (bits) {
        case 1: return launch_norm_bits<1>(map, a, c, dtype, shuffle, timeouts, stream);
        case 2: return launch_norm_bits<2>(map, a, c, dtype, shuffle, timeouts, stream);
        case 3: return launch_norm_bits<3>(map, a, c, dtype, shuffle, timeouts, stream);
        case 4: return launch_norm_bits<4>(map, a, c, dtype, shuffle, timeouts, stream);
        case 5: return launch_norm_bits<5>(map, a, c, dtype, shuffle, timeouts, stream);
        case 6: return launch_norm_bits<6>(map, a, c, dtype, shuffle, timeouts, stream);
        case 7: return launch_norm_bits<7>(map, a, c, dtype, shuffle, timeouts, stream);
        case 8: return launch_norm_bits<8>(map, a, c, dtype, shuffle, timeouts, stream);
    }
    return cudaErrorInvalidValue;
}

// ---- encode against a given scale on the TMA kernel: one long segment (= one bucket) per launch ----
bool quantize_given_scale_applies(const void* grad, uint64_t n, const uint32_t* codes, uint64_t elem_offset,
                                  uint64_t min_elems)
{
    return n >= min_elems && n / 32 <= 0x7FFFFFFFull && (elem_offset & 7u) == 0 &&
           blocks_share_high_half(n, elem_offset) &&
           (reinterpret_cast<uintptr_t>(grad) & 15u) == 0 && (reinterpret_cast<uintptr_t>(codes) & 15u) == 0;
}

cudaError_t launch_quantize_given_scale(const void* grad, uint64_t n, int bits, uint64_t seed, uint32_t* codes,
                                        float* scale, int dtype, uint32_t worker, uint32_t step,
                                        uint64_t elem_offset, cudaStream_t stream)
{
    QuantizeArgs a;
    fill_args(a, grad, n, bits, 128 * 32, seed, codes, scale, worker, step, elem_offset);   // tiles of 128 rows
    a.nbuckets = 1;
    TmaQuantizeConsts c;
    if (fill_tma_args(a, c, 128) != 128) return cudaErrorInvalidValue;
    unsigned int* timeouts = wait_timeout_counter();
    if (timeouts == nullptr) return cudaErrorNotSupported;
    CUtensorMap map;
    const char* why = nullptr;
    if (!encode_rows_map(&map, grad, a.nrows_full, dtype == 0 ? 4 : 2, 32, a.tile_rows, &why))
        return cudaErrorNotSupported;
#define MQG_GIVEN_CASE(B) \
    case B: return dtype == 0 ? launch_tma_inst<B, 0, 128, false, kGiven>(map, a, c, timeouts, stream) \
                              : launch_tma_inst<B, 1, 128, false, kGiven>(map, a, c, timeouts, stream)
    switch (bits) {
        MQG_GIVEN_CASE(1); MQG_GIVEN_CASE(2); MQG_GIVEN_CASE(3); MQG_GIVEN_CASE(4);
        MQG_GIVEN_CASE(5); MQG_GIVEN_CASE(6); MQG_GIVEN_CASE(7); MQG_GIVEN_CASE(8);
    }
#undef MQG_GIVEN_CASE
    return cudaErrorInvalidValue;
}

}  // namespace mqg
