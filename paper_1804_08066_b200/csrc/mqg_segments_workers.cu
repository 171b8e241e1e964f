// Per-layer quantization (one scale per segment) of SEVERAL workers' gradients in three launches
// instead of five per worker (Section 4.1 quantizes whole layers; Algorithm 1, WorkerIterate line 3,
// for every worker of the simulation):
//   1. zero_scales_kernel   - the scale arrays start at zero (they are the max pass's accumulators);
//   2. absmax_workers_kernel - the max pass over every (worker, segment, tile), blockIdx.y = worker;
//   3. encode_workers_kernel - the encode pass.  Every (worker, long segment) pair is an "entry"
//      with a tensor map of its own; the persistent CTAs first walk the 128-row tiles of all entries
//      as one sequence, fed by tiled bulk copies exactly like quantize_workers_kernel (tile code of
//      mqg_quantize_tile.cuh, given-scale mode), and then share the tiles of the short segments of
//      all workers, staged with 16-byte asynchronous copies.
// Worker w's outputs are bit-identical to mqg_quantize_segments with worker id first_worker + w.
#include <string.h>

#include <atomic>

#include "mqg_quantize_tile.cuh"
#include "mqg_segments.cuh"

namespace mqg {

constexpr int kMaxSegEntries = kMaxSegEntriesPerLaunch;        // (worker, long segment) pairs per launch

struct SegEntry {
    const void* grad;        // the segment's first element (for its ragged last row)
    uint32_t* codes;         // the segment's first code word
    float* scale;            // its scale, final when the encode pass starts
    uint64_t n;              // elements
    uint32_t ntiles;         // tiles of 128 rows
    uint32_t full_tiles;     // leading tiles whose 128 rows are all complete
    uint32_t blk0_lo;        // low half of the Philox block index of the segment's first element
    PhiloxHead head;         // launch-wide part of its blocks (worker, high half of the block index)
};

struct SegEntryTable {
    CUtensorMap map[kMaxSegEntries];
    SegEntry e[kMaxSegEntries];
    int nent;
};

// The segments that are not entries: the table lists their 256-row tiles; every worker has the same.
struct ShortSegments {
    SegmentTable tab;
    const void* grad[kMaxWorkers];
    uint32_t* codes[kMaxWorkers];
    float* scales[kMaxWorkers];          // scale of the table's first segment
    uint64_t elem_offset;
    uint32_t first_worker;
    int W;
};

struct ScalePtrs {
    float* scales[kMaxWorkers];
    const void* grad[kMaxWorkers];
};

__global__ void zero_scales_kernel(const ScalePtrs p, int nseg)
{
    float* s = p.scales[blockIdx.x];
    for (int j = threadIdx.x; j < nseg; j += blockDim.x) s[j] = 0.0f;
}

// The max pass of mqg_segments.cu with the worker in blockIdx.y.
template <int DTYPE>
__global__ void __launch_bounds__(kMaxTileRows)
absmax_workers_kernel(const ScalePtrs p, const SegmentTable tab)
{
    __shared__ uint32_t s_warp[kMaxTileRows / 32];
    const TileGeom g = locate_tile<1>(tab, blockIdx.x);
    const uint64_t count = g.valid < (uint64_t)(kMaxTileRows * 32) ? g.valid : (uint64_t)(kMaxTileRows * 32);
    float mx = 0.0f;
    if constexpr (DTYPE == 0) {
        const float* src = static_cast<const float*>(p.grad[blockIdx.y]) + g.elem0;
        if ((reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
            const uint64_t n4 = count / 4;
            for (uint64_t i = threadIdx.x; i < n4; i += kMaxTileRows) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(src) + i);
                mx = fmaxf(fmaxf(mx, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
            }
            for (uint64_t i = n4 * 4 + threadIdx.x; i < count; i += kMaxTileRows)
                mx = fmaxf(mx, fabsf(__ldg(src + i)));
        } else {
            for (uint64_t i = threadIdx.x; i < count; i += kMaxTileRows)
                mx = fmaxf(mx, fabsf(__ldg(src + i)));
        }
    } else {
        const uint16_t* src = static_cast<const uint16_t*>(p.grad[blockIdx.y]) + g.elem0;
        if ((reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
            const uint64_t n8 = count / 8;
            for (uint64_t i = threadIdx.x; i < n8; i += kMaxTileRows) {
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(src) + i);
                const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    mx = fmaxf(mx, fmaxf(fabsf(bf16_lo(u[k])), fabsf(bf16_hi(u[k]))));
            }
            for (uint64_t i = n8 * 8 + threadIdx.x; i < count; i += kMaxTileRows)
                mx = fmaxf(mx, fabsf(bf16_lo(__ldg(src + i))));
        } else {
            for (uint64_t i = threadIdx.x; i < count; i += kMaxTileRows)
                mx = fmaxf(mx, fabsf(bf16_lo(__ldg(src + i))));
        }
    }
    uint32_t m = __reduce_max_sync(0xFFFFFFFFu, __float_as_uint(mx));
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
        m = threadIdx.x < kMaxTileRows / 32 ? s_warp[threadIdx.x] : 0u;
        m = __reduce_max_sync(0xFFFFFFFFu, m);
        // a tile's maximum below the flush limit does not count, so the scale left by the pass is final
        if (threadIdx.x == 0 && m >= __float_as_uint(flush_limit()))
            atomicMax(reinterpret_cast<unsigned int*>(p.scales[blockIdx.y]) + g.seg, m);
    }
}

// The encode pass (see the head of the file).  total_tiles = tiles of all entries; short_units =
// W x (tiles of ss.tab) x 2: a 256-row tile of the table is encoded as two halves of 128 rows.
template <int BITS, int DTYPE>
__global__ void __launch_bounds__(128, 5)
encode_workers_kernel(const __grid_constant__ SegEntryTable ent, const __grid_constant__ ShortSegments ss,
                      const __grid_constant__ QuantizeArgs a, const __grid_constant__ TmaQuantizeConsts c,
                      uint32_t total_tiles, uint32_t short_units, unsigned int* __restrict__ timeouts)
{
    constexpr int THREADS = 128;
    using Shared = TmaQuantizeShared<DTYPE, THREADS>;
    constexpr int kQuantStages = Shared::kStages;
    __shared__ Shared sh;

    const uint32_t t = threadIdx.x;
    const uint32_t stride = gridDim.x;
    const uint32_t box_bytes = THREADS * Shared::kRowBytes;
    if (t == 0) {
        for (int s = 0; s < kQuantStages; ++s) mbar_init(smem_u32(&sh.bar[s]), 1);
        fence_barrier_init();
    }
    grid_dependency_release();
    __syncthreads();
    grid_dependency_wait();            // nothing above touches global memory

    // ---- the tiles of the entries, one sequence walked like quantize_workers_kernel walks its workers
    struct Pos { uint32_t e, tile; };
    auto advance = [&](Pos& p, uint32_t by) {
        p.tile += by;
        while (p.tile >= ent.e[p.e].ntiles) { p.tile -= ent.e[p.e].ntiles; ++p.e; }
    };
    auto load_tile = [&](const Pos& p, uint32_t stage, uint32_t bar) {     // thread 0 only
        mbar_expect_tx(bar, box_bytes);
        if (!a.arm_only) tma_load_2d(stage, &ent.map[p.e], 0, (int)(p.tile * THREADS), bar);
    };
    uint32_t v = blockIdx.x;
    Pos cur = {0u, 0u}, fill = {0u, 0u};
    if (v < total_tiles) { advance(cur, v); advance(fill, v); }
    uint32_t vfill = v;
    for (uint32_t s = 0; s < (uint32_t)kQuantStages; ++s) {
        if (t == 0 && vfill < total_tiles) load_tile(fill, smem_u32(sh.stage[s]), smem_u32(&sh.bar[s]));
        vfill += stride;
        if (vfill < total_tiles) advance(fill, stride);
    }

    uint32_t k = 0, rot = 0;
    bool ok = true;
#pragma unroll 1
    for (; ok && v < total_tiles; v += stride, ++k, rot = (rot == 2 ? 0 : rot + 1)) {
        const SegEntry& e = ent.e[cur.e];
        const uint32_t tile = cur.tile;
        const WorkerView wv = {&ent.map[cur.e], e.grad, e.codes, e.scale, e.head, e.blk0_lo};
        auto refill = [&](uint32_t stage, uint32_t bar) {
            if (vfill < total_tiles) load_tile(fill, stage, bar);
        };
        if (tile < e.full_tiles) {
            ok = quantize_tile<BITS, DTYPE, THREADS, true, false, false, true>(sh, wv, a, c, k, rot, tile, refill,
                                                                                0u, false);
        } else {
            QuantizeArgs ae = a;           // the bounds of this entry, needed by its last tile only
            ae.n = e.n;
            ae.nrows = (e.n + 31) / 32;
            ae.nrows_full = e.n / 32;
            ae.ncode_words = (e.n * BITS + 31) / 32;
            ok = quantize_tile<BITS, DTYPE, THREADS, false, false, false, true>(sh, wv, ae, c, k, rot, tile, refill,
                                                                                 0u, false);
        }
        if (v + stride < total_tiles) advance(cur, stride);
        vfill += stride;
        if (vfill < total_tiles) advance(fill, stride);
    }
    if (!ok) {                         // as in quantize_workers_kernel
        if (t == 0) {
            atomicAdd(timeouts, 1u);
            uint32_t j = k - 1, vl = v - stride;
            for (int s = 0; s < kQuantStages && vl < total_tiles; ++s, ++j, vl += stride)
                mbar_wait(smem_u32(&sh.bar[j % kQuantStages]), (j / kQuantStages) & 1, a.poll_limit);
        }
        __syncthreads();
        return;
    }

    // ---- the short segments of all workers: plain asynchronous copies into the (now idle) stages
    if (short_units == 0) return;
    __syncthreads();
    float4* tilebuf = reinterpret_cast<float4*>(sh.stage[0]);          // 128 rows x 128 bytes
    const uint32_t per_worker = short_units / (uint32_t)ss.W;
#pragma unroll 1
    for (uint32_t s = blockIdx.x; s < short_units; s += stride) {
        const uint32_t w = s / per_worker, rem = s - w * per_worker;
        const TileGeom g = locate_tile<BITS>(ss.tab, rem >> 1);
        const int r0 = (int)(rem & 1u) * THREADS;
        if (r0 >= g.rows) continue;                                    // the same for the whole CTA
        const int rows = min(THREADS, g.rows - r0);
        const uint64_t elem0 = g.elem0 + 32ull * r0, valid = g.valid - 32ull * r0;
        if constexpr (DTYPE == 0)
            load_tile_f32<THREADS>(tilebuf, static_cast<const float*>(ss.grad[w]) + elem0, valid, rows);
        else
            load_tile_bf16<THREADS>(tilebuf, static_cast<const uint16_t*>(ss.grad[w]) + elem0, valid, rows);
        const float sc = ss.scales[w][g.seg];
        __syncthreads();
        if (t < (uint32_t)rows) {
            float x[32];
            read_row(tilebuf, (int)t, x);
            const EncodeScale es = encode_scale<BITS>(sc);
            const uint64_t g0 = ss.elem_offset + elem0 + 32ull * t;
            uint32_t h[16];
            if ((g0 & 7u) == 0) {
                const uint64_t blk = g0 >> 3;
                draw_row_blocks((uint32_t)blk, (uint32_t)(blk >> 32), ss.first_worker + w, c.rk, h);
            } else {
                const DrawKey key = {c.rk.k0[0], c.rk.k1[0], ss.first_worker + w, c.rk.step};
                draw_row_unaligned(g0, key, h);
            }
            uint32_t cw[BITS];
            encode_pack_row<BITS>(x, es, h, cw);
            const uint64_t word0 = g.word0 + (uint64_t)(r0 + (int)t) * BITS;
            const uint64_t left = valid - 32ull * t;       // elements of the segment from this row on
            if (left < 32) mask_row_words<BITS>(cw, (int)left * BITS);
#pragma unroll
            for (int j = 0; j < BITS; ++j)
                if (word0 + j < g.words_end) ss.codes[w][word0 + j] = cw[j];
        }
        __syncthreads();                                               // the buffer is free again
    }
}

// ---- host side --------------------------------------------------------------------------------

cudaError_t launch_zero_scales(float* const* scales, int W, int nseg, cudaStream_t stream)
{
    ScalePtrs p;
    memset(&p, 0, sizeof(p));
    for (int w = 0; w < W; ++w) p.scales[w] = scales[w];
    zero_scales_kernel<<<W, 128, 0, stream>>>(p, nseg);
    return cudaGetLastError();
}

// Max pass over the tiles `tab` lists, for every worker; scales[w] + first is the scale of the
// table's first segment.
cudaError_t launch_absmax_workers(const void* const* grads, float* const* scales, int first, int W,
                                  const SegmentTable& tab, int dtype, cudaStream_t stream)
{
    const uint32_t ntiles = tab.tile_start[tab.nseg];
    if (ntiles == 0) return cudaSuccess;
    ScalePtrs p;
    memset(&p, 0, sizeof(p));
    for (int w = 0; w < W; ++w) { p.scales[w] = scales[w] + first; p.grad[w] = grads[w]; }
    const dim3 grid(ntiles, (unsigned)W);
    if (dtype == 0) absmax_workers_kernel<0><<<grid, kMaxTileRows, 0, stream>>>(p, tab);
    else absmax_workers_kernel<1><<<grid, kMaxTileRows, 0, stream>>>(p, tab);
    return cudaGetLastError();
}

template <int BITS, int DTYPE>
static cudaError_t launch_encode_inst(const SegEntryTable& ent, const ShortSegments& ss, const QuantizeArgs& a,
                                      const TmaQuantizeConsts& c, uint32_t total_tiles, uint32_t short_units,
                                      unsigned int* timeouts, cudaStream_t stream)
{
    auto kernel = encode_workers_kernel<BITS, DTYPE>;
    static std::atomic<int> grid_cap[64];          // per device; 0 = not yet queried (zero-initialised)
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
    const uint64_t work = (uint64_t)total_tiles + short_units;
    unsigned grid = (unsigned)cap;
    if (grid > work) grid = (unsigned)work;
    if (grid == 0) return cudaSuccess;
    return launch_pdl(kernel, grid, 128, stream, ent, ss, a, c, total_tiles, short_units, timeouts);
}

// One encode launch: the entries ent[0 .. nent) (a (worker, long segment) pair each, see
// SegEntryHost) and, if short_tab != nullptr, the tiles of that table for all W workers.
cudaError_t launch_encode_workers(const SegEntryHost* entries, int nent, const SegmentTable* short_tab,
                                  const void* const* grads, uint32_t* const* codes, float* const* scales,
                                  int scale_first, int W, int bits, uint64_t seed, int dtype,
                                  uint32_t first_worker, uint32_t step, uint64_t elem_offset, cudaStream_t stream)
{
    if (nent < 0 || nent > kMaxSegEntries) return cudaErrorInvalidValue;
    unsigned int* timeouts = wait_timeout_counter();
    if (timeouts == nullptr) return cudaErrorNotSupported;
    QuantizeArgs a;
    memset(&a, 0, sizeof(a));
    a.tile_rows = 128; a.rows_per_bucket = 128; a.buckets_per_tile = 1; a.nbuckets = 1;
    a.key.seed_lo = (uint32_t)seed; a.key.seed_hi = (uint32_t)(seed >> 32);
    a.key.worker = first_worker; a.key.step = step;
    const WaitPolicy policy = wait_policy();
    a.poll_limit = policy.poll_limit;
    a.arm_only = policy.arm_only;
    TmaQuantizeConsts c;
    memset(&c, 0, sizeof(c));
    uint32_t k0 = a.key.seed_lo, k1 = a.key.seed_hi;
    for (int r = 0; r < 10; ++r) {
        c.rk.k0[r] = k0; c.rk.k1[r] = k1;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    c.rk.worker = first_worker; c.rk.step = step;

    SegEntryTable ent;
    memset(&ent, 0, sizeof(ent));
    ent.nent = nent;
    uint64_t total = 0;
    for (int i = 0; i < nent; ++i) {
        const SegEntryHost& h = entries[i];
        SegEntry& e = ent.e[i];
        const uint64_t nrows = (h.n + 31) / 32, nrows_full = h.n / 32;
        const char* why = nullptr;
        if (!encode_rows_map(&ent.map[i], h.grad, nrows_full, dtype == 0 ? 4 : 2, 32, 128, &why))
            return cudaErrorNotSupported;
        e.grad = h.grad; e.codes = h.codes; e.scale = h.scale; e.n = h.n;
        e.ntiles = (uint32_t)((nrows + 127) / 128);
        e.full_tiles = (uint32_t)(nrows_full / 128);
        const uint64_t blk0 = h.elem_offset >> 3;
        e.blk0_lo = (uint32_t)blk0;
        e.head = philox_head((uint32_t)(blk0 >> 32), h.worker, c.rk.k0[0]);
        total += e.ntiles;
    }
    if (total > 0x7FFFFFFFull) return cudaErrorInvalidValue;

    ShortSegments ss;
    memset(&ss, 0, sizeof(ss));
    ss.W = W > 0 ? W : 1;
    ss.first_worker = first_worker;
    ss.elem_offset = elem_offset;
    uint64_t short_units = 0;
    if (short_tab != nullptr) {
        ss.tab = *short_tab;
        for (int w = 0; w < W; ++w) { ss.grad[w] = grads[w]; ss.codes[w] = codes[w]; ss.scales[w] = scales[w] + scale_first; }
        short_units = 2ull * short_tab->tile_start[short_tab->nseg] * (uint64_t)W;
        if (short_units > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    }
#define MQG_ENC_CASE(B) \
    case B: return dtype == 0 ? launch_encode_inst<B, 0>(ent, ss, a, c, (uint32_t)total, (uint32_t)short_units, timeouts, stream) \
                              : launch_encode_inst<B, 1>(ent, ss, a, c, (uint32_t)total, (uint32_t)short_units, timeouts, stream)
    switch (bits) {
        MQG_ENC_CASE(1); MQG_ENC_CASE(2); MQG_ENC_CASE(3); MQG_ENC_CASE(4);
        MQG_ENC_CASE(5); MQG_ENC_CASE(6); MQG_ENC_CASE(7); MQG_ENC_CASE(8);
    }
#undef MQG_ENC_CASE
    return cudaErrorInvalidValue;
}

}  // namespace mqg
