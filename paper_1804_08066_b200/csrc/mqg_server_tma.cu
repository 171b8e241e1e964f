// Fused server pass (the fast path of mqg_server_step for uniform buckets of at least 1024 elements,
// of 512, 768, 896, 960 or 992, and - for few workers - of 32 to 256): every WARP is an independent
// pipeline over a contiguous range of 32-row tiles.  Nothing is loaded through registers:
//   * a tile's 32 x 32 parameters arrive by a tiled bulk copy (TMA) into the warp's own swizzled
//     shared-memory stage while the tile's workers are being summed, are updated in place and leave
//     by a tiled bulk store;
//   * the code words of the tile (32 rows x K words per worker, contiguous in each worker's
//     stream) arrive by 16-byte asynchronous copies, one instruction of the warp per worker (two
//     above four bits), into a two-deep ring of code stages, a group of workers per stage, issued
//     two stages ahead of their use.  (One linear bulk copy per worker, completing on an mbarrier,
//     cost about a dozen instructions of the warp per copy - the operands of a bulk copy travel
//     through the uniform datapath - and with eight of them per tile a third of the kernel's
//     instructions were overhead: 40.1 executed instructions per parameter at four bits and eight
//     workers against 31.4 now.)
// A warp therefore never waits for DRAM latency in steady state and there is no CTA-wide barrier
// anywhere.  Per-(worker, bucket) de-quantization constants are computed once per tile into the
// warp's small shared table, one tile ahead.
#include <string.h>

#include <atomic>

#include "mqg_segments.cuh"
#include "mqg_tma.cuh"

namespace mqg {

constexpr int kSrvWarps = 4;                      // warps per CTA, each with its own pipeline
constexpr int kSrvThreads = 32 * kSrvWarps;
constexpr int kSrvTileRows = 32;                  // rows per tile = lanes per warp
constexpr uint32_t kSrvTileBytes = kSrvTileRows * 128;
constexpr int kCodeDepth = 2;                     // code stages per warp

// Workers whose code words share one code stage: at most 4 KB per stage, so that a CTA's shared
// memory (13 KB per warp) lets four CTAs = 16 warps share an SM, and a power of two, so that the
// usual worker counts fill whole stages.
template <int BITS>
struct ServerGroup { static constexpr int value = BITS <= 4 ? 8 : 4; };

// Barrier ID (1 .. 15; 0 is the one of __syncthreads) among `threads` threads of a CTA (a multiple of 32:
// whole warps); every thread that takes part names the same count.
template <int ID>
__device__ __forceinline__ void named_barrier(uint32_t threads)
{
    asm volatile("bar.sync %0, %1;" ::"n"(ID), "r"(threads) : "memory");
}

struct ServerTmaArgs {
    WorkerPtrs ptrs;
    float* params;
    uint64_t n, ncode_words;
    uint32_t nrows;              // ceil(n / 32)
    uint32_t nrows_full;         // floor(n / 32): rows the tensor map and the code copies cover
    uint32_t ntiles;             // ceil(nrows_full / 32)
    uint32_t nbuckets;
    uint32_t rows_per_bucket;    // such that a tile touches at most 1 << nbt_shift buckets
    int rpb_shift;               // log2(rows_per_bucket) if a power of two, else -1
    int nbt_shift;               // log2 of the buckets a tile can touch: 1 (two buckets), or 2..5 for
                                 // buckets of 8, 4, 2, 1 rows; W << nbt_shift <= 2 * kMaxWorkers
    int W;
    float neg_lr;
    uint32_t bias_bits;          // 0x4B000000 (2^23), a run-time constant for the byte permutes
    uint32_t poll_limit;         // polls of one barrier wait before the warp gives up
    uint32_t arm_only;           // test hook: 1 = arm the barriers but issue no parameter copy
};

// SEGS: the launch covers several gradients ("segments" of a per-layer step, each ONE bucket with a
// scale of its own) instead of one gradient with uniform buckets.  The tiles of all segments form
// one sequence that is split over the warps as usual; a tile's segment is found with a cursor that
// only moves forward.
constexpr int kMaxSrvSegs = kMaxServerSegsPerLaunch;
struct ServerSegEntry {
    uint32_t tile_start;     // number of the segment's first tile in the launch's sequence
    uint32_t nrows_full;     // floor(n / 32): rows its tensor map and code copies cover
    uint32_t scale_idx;      // index of its scale in every worker's scale array
    uint32_t ragged;         // n % 32: elements of its last, incomplete row (0 = none)
    uint64_t code_word0;     // word offset of its bit stream in every worker's code buffer
    uint64_t elem0;          // offset of its first element in a.params
};
struct ServerSegTable {
    CUtensorMap map[kMaxSrvSegs];
    ServerSegEntry e[kMaxSrvSegs + 1];     // e[nseg].tile_start = tiles of the launch
    int nseg;
};

// Where a tile lives: the tensor map of its gradient, its first row there, the rows the map covers,
// the word offset of the gradient's bit stream and (SEGS) the index of its scale.
struct TileLoc {
    const CUtensorMap* map;
    uint32_t row0, nrows_full, scale_idx;
    uint64_t code_word0;
};

template <bool SEGS>
__device__ __forceinline__ TileLoc locate_srv_tile(const CUtensorMap* map_full, const ServerTmaArgs& a,
                                                   const ServerSegTable* segs, uint32_t tile, uint32_t& cursor)
{
    TileLoc t;
    if constexpr (SEGS) {
        while (tile >= segs->e[cursor + 1].tile_start) ++cursor;
        const ServerSegEntry& e = segs->e[cursor];
        t.map = &segs->map[cursor];
        t.row0 = (tile - e.tile_start) * kSrvTileRows;
        t.nrows_full = e.nrows_full;
        t.scale_idx = e.scale_idx;
        t.code_word0 = e.code_word0;
    } else {
        t.map = map_full;
        t.row0 = tile * kSrvTileRows;
        t.nrows_full = a.nrows_full;
        t.scale_idx = 0;
        t.code_word0 = 0;
    }
    return t;
}

// Dynamic shared memory of one CTA (base rounded up to 1024 bytes for the 128-byte swizzle).
template <int BITS>
struct ServerSmem {
    alignas(1024) uint8_t stage[kSrvWarps][kSrvTileBytes];      // one parameter tile per warp
    alignas(16) uint32_t code[kSrvWarps][kCodeDepth][ServerGroup<BITS>::value][kSrvTileRows * BITS];
    float4 table[kSrvWarps][2 * kMaxWorkers];     // (2h, 2h, -h, -h) per (worker, bucket of the tile): entry
                                                  // (worker << nbt_shift) + bucket-of-tile
    uint64_t bar[kSrvWarps];                      // parameter tile landed
};

__device__ __forceinline__ uint32_t bucket_of_row(const ServerTmaArgs& a, uint32_t row)
{
    return a.rpb_shift >= 0 ? row >> a.rpb_shift : row / a.rows_per_bucket;
}

// Scales of the (worker, bucket) pairs of the tile that starts at row0: lane l holds pair l and,
// when there are more than 32 pairs (`wide`), pair l + 32 (pair = (worker << nbt_shift) +
// bucket-of-tile).  RANGE: the pair's (lo, hi) instead of its scale (the `scales` pointers then
// address arrays of two floats per bucket).
template <bool RANGE, bool SEGS>
__device__ __forceinline__ void load_tile_scales(const ServerTmaArgs& a, const TileLoc& loc, uint32_t lane,
                                                 bool wide, float2 (&s)[2])
{
    // SEGS: the tile lies in one bucket, the segment's (nbt_shift = 0: pair = worker)
    const uint32_t first = SEGS ? loc.scale_idx : bucket_of_row(a, loc.row0);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        if (h == 1 && !wide) break;
        const uint32_t pair = lane + 32u * h, w = pair >> a.nbt_shift;
        const uint32_t b = first + (pair & ((1u << a.nbt_shift) - 1u));
        const bool have = w < (uint32_t)a.W && (SEGS || b < a.nbuckets);
        if (RANGE) s[h] = have ? __ldg(reinterpret_cast<const float2*>(a.ptrs.scales[w]) + b) : make_float2(0.0f, 0.0f);
        else s[h] = make_float2(have ? __ldg(a.ptrs.scales[w] + b) : 0.0f, 0.0f);
    }
}

template <int BITS, bool RANGE>
__device__ __forceinline__ void store_tile_scales(const ServerTmaArgs& a, float4* table, uint32_t lane,
                                                  bool wide, const float2 (&s)[2])
{
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        if (h == 1 && !wide) break;
        const uint32_t pair = lane + 32u * h, w = pair >> a.nbt_shift;
        if (w < (uint32_t)a.W) {
            const DecodeScale d = RANGE ? range_decode_scale<BITS>(s[h].x, s[h].y) : decode_scale<BITS>(s[h].x);
            table[pair] = make_float4(d.two_h, d.two_h, d.minus_h, d.minus_h);
        }
    }
}

// A lane's K words of one worker from a code stage, with the widest shared-memory access the
// lane's offset (lane * K words) allows.
template <int BITS>
__device__ __forceinline__ void read_stage_words(const uint32_t* __restrict__ stage_row, uint32_t (&w)[BITS])
{
    if constexpr (BITS % 4 == 0) {
        const uint4* p = reinterpret_cast<const uint4*>(stage_row);
#pragma unroll
        for (int k = 0; k < BITS / 4; ++k) {
            const uint4 v = p[k];
            w[4 * k] = v.x; w[4 * k + 1] = v.y; w[4 * k + 2] = v.z; w[4 * k + 3] = v.w;
        }
    } else if constexpr (BITS % 2 == 0) {
        const uint2* p = reinterpret_cast<const uint2*>(stage_row);
#pragma unroll
        for (int k = 0; k < BITS / 2; ++k) {
            const uint2 v = p[k];
            w[2 * k] = v.x; w[2 * k + 1] = v.y;
        }
    } else {
#pragma unroll
        for (int k = 0; k < BITS; ++k) w[k] = stage_row[k];
    }
}

// 16-byte asynchronous copy that reads only the first `src_bytes` bytes of the source and fills the
// rest of the 16 bytes with zeros.
__device__ __forceinline__ void cp_async16_partial(uint32_t smem_dst, const void* gmem_src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_dst), "l"(gmem_src), "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void cp_async16_to(uint32_t smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Starts the copies of one code stage: the words of rows [row0, row0 + 32) (fewer in the last tile
// of the gradient) of workers g0 .. g0 + group - 1 (those that exist).  A worker's words of these
// rows are contiguous in its stream and start on a 16-byte boundary (row0 is a multiple of 32):
// (and so does the bit stream of a segment that takes part in a SEGS launch): the warp copies them in 16-byte pieces, lane l the l-th piece (and the (l + 32)-th for more than
// four bits), asynchronously and without passing through registers.  The piece that holds the end
// of a short last tile is copied up to that end and zero-filled.  `lane_off` = 16 * lane.
template <int BITS>
__device__ __forceinline__ void fill_code_stage(const ServerTmaArgs& a, uint32_t stage, const TileLoc& loc, int g0,
                                                uint32_t lane_off)
{
    constexpr int kGroup = ServerGroup<BITS>::value;
    constexpr uint32_t kWorkerBytes = kSrvTileRows * BITS * 4;
    constexpr int kPieces = (int)((kWorkerBytes / 16 + 31) / 32);       // pieces per lane: 1 or 2
    const uint32_t rows_here = min((uint32_t)kSrvTileRows, loc.nrows_full - loc.row0);
    const uint64_t byte0 = (loc.code_word0 + (uint64_t)loc.row0 * BITS) * 4 + lane_off;
    if (rows_here == (uint32_t)kSrvTileRows && g0 + kGroup <= a.W) {
#pragma unroll
        for (int pc = 0; pc < kPieces; ++pc) {
            if (lane_off + 512u * pc < kWorkerBytes) {
#pragma unroll
                for (int i = 0; i < kGroup; ++i)
                    cp_async16_to(stage + i * kWorkerBytes + lane_off + 512u * pc,
                                  reinterpret_cast<const uint8_t*>(a.ptrs.codes[g0 + i]) + byte0 + 512u * pc);
            }
        }
    } else {
        const uint32_t bytes_here = rows_here * BITS * 4;
        const int nwk = min(kGroup, a.W - g0);
#pragma unroll
        for (int pc = 0; pc < kPieces; ++pc) {
            const uint32_t off = lane_off + 512u * pc;
            if (off < bytes_here) {
                const uint32_t nb = min(16u, bytes_here - off);
                for (int i = 0; i < nwk; ++i)
                    cp_async16_partial(stage + i * kWorkerBytes + off,
                                       reinterpret_cast<const uint8_t*>(a.ptrs.codes[g0 + i]) + byte0 + 512u * pc, nb);
            }
        }
    }
}

// CTAs per SM the register budget is set for (what the shared memory allows at three bits and more;
// five CTAs of 96 registers at one and two bits measured 0.3 us slower per launch than four).
template <int BITS>
constexpr int server_min_ctas() { return 4; }

// MODE 1: dst = params, dst <- fma(-lr, sum, dst).  MODE 0: dst = acc, dst <- sum.
// MODE 2: dst = acc, the sum continues from the value already there.
// RANGE: the (min, max) nearest-rounding variant (x^ = fma(q, step, lo)).
// The one row of a gradient that has fewer than 32 elements (row `row`, the last one): plain loads and
// stores by a single thread.  `params` is the gradient's first parameter, n its length, its bit stream
// the words [code_word0, words_end) of every worker's buffer, `bucket` the index of the row's scale.
template <int BITS, int MODE, bool RANGE>
__device__ __noinline__ void server_ragged_row(const ServerTmaArgs& a, float* params, uint32_t row, uint64_t n,
                                               uint64_t code_word0, uint64_t words_end, uint32_t bucket)
{
    const uint64_t e0 = (uint64_t)row * 32;
    const uint64_t word0 = code_word0 + (uint64_t)row * BITS;
    float2 v2[16];
#pragma unroll
    for (int p = 0; p < 16; ++p) {
        v2[p] = make_float2(0.0f, 0.0f);
        if constexpr (MODE == 2) {
            if (e0 + 2 * p < n) v2[p].x = params[e0 + 2 * p];
            if (e0 + 2 * p + 1 < n) v2[p].y = params[e0 + 2 * p + 1];
        }
    }
    for (int w = 0; w < a.W; ++w) {
        uint32_t cw[BITS];
#pragma unroll
        for (int j = 0; j < BITS; ++j)
            cw[j] = (word0 + j < words_end) ? __ldg(a.ptrs.codes[w] + word0 + j) : 0u;
        const DecodeScale2 d = widen(RANGE ? range_decode_scale<BITS>(__ldg(a.ptrs.scales[w] + 2 * bucket),
                                                                      __ldg(a.ptrs.scales[w] + 2 * bucket + 1))
                                           : decode_scale<BITS>(__ldg(a.ptrs.scales[w] + bucket)));
        add_decoded_row<BITS, RANGE>(cw, d, v2);
    }
    float v[32];
    floats_from_pairs(v2, v);
#pragma unroll
    for (int j = 0; j < 32; ++j)
        if (e0 + j < n) params[e0 + j] = MODE == 1 ? __fmaf_rn(a.neg_lr, v[j], params[e0 + j]) : v[j];
}

template <int BITS, int MODE, bool RANGE, bool SEGS>
__device__ __forceinline__ void server_tma_body(const CUtensorMap* map_full, const ServerTmaArgs& a,
                                                const ServerSegTable* segs, unsigned int* __restrict__ timeouts)
{
    extern __shared__ uint8_t smem_raw[];
    ServerSmem<BITS>& sm = *reinterpret_cast<ServerSmem<BITS>*>(
        smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u));
    constexpr int kGroup = ServerGroup<BITS>::value;
    constexpr uint32_t kWorkerWords = kSrvTileRows * BITS;
    const uint32_t lane = threadIdx.x & 31u;
    // the warp's number, taken from lane 0 so that the compiler knows it is the same in every lane
    const uint32_t wid = __shfl_sync(0xFFFFFFFFu, threadIdx.x >> 5, 0);
    uint8_t* stage = sm.stage[wid];
    float4* table = sm.table[wid];
    const uint32_t bar = smem_u32(&sm.bar[wid]);
    const uint32_t code_base = smem_u32(&sm.code[wid][0][0][0]);
    constexpr uint32_t kCodeStageBytes = kGroup * kWorkerWords * 4;

    if (lane == 0) {
        mbar_init(bar, 1);
        fence_barrier_init();
        if (!SEGS) prefetch_tensormap(map_full);
    }
    __syncwarp();
    grid_dependency_wait();            // nothing above touches global memory

    // This warp's tiles: gwarp, gwarp + nwarps, gwarp + 2 nwarps, ...  At any moment the grid then works
    // on one window of consecutive tiles, and the four warps of a CTA on four consecutive ones: their
    // requests for a worker's code words (32 K bytes per tile) fall into the same DRAM pages at about the
    // same time.  Against a contiguous range of tiles per warp, per launch at eight workers: 37.5 against
    // 39.7 us at one bit, 44.5 against 47.6 at three, 61.0 against 63.0 at eight (n = 25 M); 89 against 94,
    // 115 against 123, 143 against 147 us at n = 61 M.
    const uint32_t gwarp = blockIdx.x * kSrvWarps + wid, nwarps = gridDim.x * kSrvWarps;
    const uint32_t base = a.ntiles / nwarps, extra = a.ntiles % nwarps;
    const uint32_t t_begin = gwarp, t_step = nwarps;
    const uint32_t ntiles = base + (gwarp < extra ? 1u : 0u);
    // Three and four bits: the warps of a CTA start every tile together (a CTA barrier per tile, for the
    // `base` tiles that every warp of the grid has), which keeps those requests together for the whole
    // launch: 106 against 116 us at three bits, 121 against 127 us at four (n = 61 M; 44.3 and 46.9 against
    // 44.3 and 48.0 us at n = 25 M); no gain at one and two bits, a loss of 1 to 2 % from five bits on.
    constexpr bool kCtaSync = BITS == 3 || BITS == 4;
    const uint32_t sync_tiles = base;
    const uint32_t last_row = a.nrows_full - 1;    // nrows_full >= 1 on this path (not used by SEGS)
    uint32_t cur_e = 0, next_e = 0, fill_e = 0;    // SEGS: segment cursors of the tile in work, the next
                                                   // tile (its scales) and the tile whose codes are fetched
    const uint32_t groups = ((uint32_t)a.W + kGroup - 1) / kGroup;      // code stages per tile
    const uint32_t nunits = ntiles * groups;
    const bool wide = ((uint32_t)a.W << a.nbt_shift) > 32u;             // more than 32 table entries
    const uint32_t lane_off = lane * 16u;
    // MODE 1: the tile's parameters are requested before this worker of the tile is summed (see
    // load_params below); measured best of 1 .. 4 at eight workers, per launch of n = 25 M: 55.8 us
    // against 57.7 us at five bits, 65.2 against 68.0 us at eight, no difference up to four bits
    constexpr int kIssueAt = 4;
    const int issue_at = min(kIssueAt, a.W - 1);

    bool failed = false;
    uint32_t k = 0, u = 0;                         // tile and code stage in use
    if (ntiles > 0) {
        float2 s0[2];
        const TileLoc first = locate_srv_tile<SEGS>(map_full, a, segs, t_begin, next_e);
        load_tile_scales<RANGE, SEGS>(a, first, lane, wide, s0);
        store_tile_scales<BITS, RANGE>(a, table, lane, wide, s0);
        if (MODE == 2 && lane == 0) {
            mbar_expect_tx(bar, kSrvTileBytes);
            if (!a.arm_only) tma_load_2d(smem_u32(stage), first.map, 0, (int)first.row0, bar);
        }
        // the first kCodeDepth code stages (u2 = stage number, tile u2 / groups, group u2 % groups);
        // one copy group per stage, empty when there is no such stage
#pragma unroll
        for (uint32_t u2 = 0; u2 < (uint32_t)kCodeDepth; ++u2) {
            if (u2 < nunits)
                fill_code_stage<BITS>(a, code_base + u2 * kCodeStageBytes,
                                      locate_srv_tile<SEGS>(map_full, a, segs, t_begin + (u2 / groups) * t_step, fill_e),
                                      (int)(u2 % groups) * kGroup, lane_off);
            cp_async_commit();
        }
        __syncwarp();
    }
    // position of the code stage kCodeDepth ahead of the one in use, kept incrementally
    uint32_t fill_tile = kCodeDepth / groups, fill_group = kCodeDepth % groups;

#pragma unroll 1
    for (; k < ntiles; ++k) {
        if constexpr (kCtaSync) {
            if (k < sync_tiles) named_barrier<1>(kSrvThreads);
        }
        const uint32_t parity = k & 1;
        const TileLoc loc = locate_srv_tile<SEGS>(map_full, a, segs, t_begin + k * t_step, cur_e);
        const uint32_t row0 = loc.row0;
        const bool have_next = k + 1 < ntiles;
        float2 s_next[2];
        TileLoc loc_next = loc;
        if (have_next) {
            loc_next = locate_srv_tile<SEGS>(map_full, a, segs, t_begin + (k + 1) * t_step, next_e);
            load_tile_scales<RANGE, SEGS>(a, loc_next, lane, wide, s_next);
        }

        // Sum of the W de-quantized rows, in worker order.  Lanes past the end of the gradient
        // (only in the very last tile) decode whatever their slot of the stage holds; they are
        // never stored.
        const uint32_t row = min(row0 + lane, last_row);
        const uint32_t lb = SEGS ? 0u : bucket_of_row(a, row) - bucket_of_row(a, row0);
        const float4* my_table = table + lb;
        float2 v2[16];
        bool ok = true;
        if constexpr (MODE == 2) {
            // the sum continues from the accumulator: its tile is needed before the first worker
            ok = mbar_try_wait(bar, parity);
            if (!ok) ok = mbar_wait(bar, parity, a.poll_limit);
            if (!__all_sync(0xFFFFFFFFu, ok)) { failed = true; break; }
            const float4* tl = reinterpret_cast<const float4*>(stage);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 p = tl[swz((int)lane, c)];
                v2[2 * c] = make_float2(p.x, p.y);
                v2[2 * c + 1] = make_float2(p.z, p.w);
            }
        } else {
#pragma unroll
            for (int p = 0; p < 16; ++p) v2[p] = make_float2(0.0f, 0.0f);
        }

#pragma unroll 1
        for (uint32_t g = 0; g < groups; ++g, ++u) {
            const uint32_t cs = u % kCodeDepth;
            const uint32_t cstage_addr = code_base + cs * kCodeStageBytes;
            const uint32_t* cstage = &sm.code[wid][cs][0][0] + lane * BITS;
            cp_async_wait_group<kCodeDepth - 1>();     // this lane's pieces of the stage have landed
            __syncwarp();                              // ... and so have the other lanes'
            const int g0 = (int)g * kGroup;
            auto decode_worker = [&](int i) {
                uint32_t w[BITS];
                read_stage_words<BITS>(cstage + i * kWorkerWords, w);
                const float4 e = my_table[(uint32_t)(g0 + i) << a.nbt_shift];
                DecodeScale2 d;
                d.two_h = make_float2(e.x, e.y); d.minus_h = make_float2(e.z, e.w);
                add_decoded_row<BITS, RANGE>(w, d, v2, a.bias_bits);
            };
            // MODE 1: the parameter stage held tile k-1, whose store was committed at the end of the last
            // iteration: once that store has read its source the stage takes tile k, which is not
            // needed before the last worker is summed.  The load starts when half of eight workers are
            // summed, by when the store has long read the stage.  The gradient's last tile may be short: the
            // box is clipped by the tensor's bounds and the rows beyond arrive as zeros, still counted
            // in the bytes.
            auto load_params = [&]() {
                if (lane == 0) {
                    bulk_wait_read<0>();
                    mbar_expect_tx(bar, kSrvTileBytes);
                    if (!a.arm_only) tma_load_2d(smem_u32(stage), loc.map, 0, (int)row0, bar);
                }
            };
            static_assert(kIssueAt == 4 && kGroup % 4 == 0, "the parameter load is issued between blocks of four workers");
            if (g0 + kGroup <= a.W) {              // a whole stage: blocks of four workers in straight-line code
#pragma unroll 1
                for (int i0 = 0; i0 < kGroup; i0 += 4) {
                    // (the positions a whole stage can hold issue_at at: worker 4 when W >= 5, else the
                    // stage's last worker when W == group size)
                    if (MODE == 1 && g0 + i0 == issue_at) load_params();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (MODE == 1 && i == 3 && i0 + i == kGroup - 1 && g0 + i0 + i == issue_at) load_params();
                        decode_worker(i0 + i);
                    }
                }
            } else {
#pragma unroll 1
                for (int i = 0; g0 + i < a.W; ++i) {
                    if (MODE == 1 && g0 + i == issue_at) load_params();
                    decode_worker(i);
                }
            }
            __syncwarp();                          // every lane has read the stage: refill it
            if (u + kCodeDepth < nunits)
                fill_code_stage<BITS>(a, cstage_addr,
                                      locate_srv_tile<SEGS>(map_full, a, segs, t_begin + fill_tile * t_step, fill_e),
                                      (int)fill_group * kGroup, lane_off);
            cp_async_commit();
            if (++fill_group == groups) { fill_group = 0; ++fill_tile; }
        }

        if constexpr (MODE == 1) {
            ok = mbar_try_wait(bar, parity);
            if (!ok) ok = mbar_wait(bar, parity, a.poll_limit);
            if (!__all_sync(0xFFFFFFFFu, ok)) { failed = true; break; }
        }
        if constexpr (MODE == 0) {
            // nothing is loaded: the stage is only written by this warp, once the store of the tile
            // before has read it
            if (lane == 0) bulk_wait_read<0>();
            __syncwarp();
        }

        {
            float4* tl = reinterpret_cast<float4*>(stage);
            const float2 nlr = make_float2(a.neg_lr, a.neg_lr);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int idx = swz((int)lane, c);
                float2 lo = v2[2 * c], hi = v2[2 * c + 1];
                if constexpr (MODE == 1) {          // params <- fma(-lr, sum, params), in place
                    const float4 p = tl[idx];
                    lo = __ffma2_rn(nlr, lo, make_float2(p.x, p.y));
                    hi = __ffma2_rn(nlr, hi, make_float2(p.z, p.w));
                }
                tl[idx] = make_float4(lo.x, lo.y, hi.x, hi.y);
            }
        }
        fence_proxy_async();                                   // the bulk store must see these writes
        if (have_next) {
            // constants of the next tile; the table was last read before the group loop's last
            // __syncwarp
            store_tile_scales<BITS, RANGE>(a, table, lane, wide, s_next);
        }
        __syncwarp();
        if (lane == 0) {
            // a short last tile is clipped by the tensor's bounds
            tma_store_2d(loc.map, 0, (int)row0, smem_u32(stage));
            bulk_commit();
            if (MODE == 2 && have_next) {
                bulk_wait_read<0>();
                mbar_expect_tx(bar, kSrvTileBytes);
                if (!a.arm_only) tma_load_2d(smem_u32(stage), loc_next.map, 0, (int)loc_next.row0, bar);
            }
        }
    }
    if constexpr (kCtaSync) {
        if (failed)                     // a warp that gave up still arrives at the barriers the others expect
            for (uint32_t kk = k + 1; kk < sync_tiles; ++kk) named_barrier<1>(kSrvThreads);
    }
    cp_async_wait_group<0>();                                  // no code copy outlives the warp
    if (lane == 0) {
        if (failed) {
            // The tile's copy did not land within the poll limit: count it and give it one more
            // bounded chance before the shared memory can be handed to another CTA.
            atomicAdd(timeouts, 1u);
            mbar_wait(bar, k & 1, a.poll_limit);
        }
        bulk_wait_all<0>();                                    // stores done before the stage goes away
    }

    // A last row of fewer than 32 elements is not covered by the tensor map: one lane of the
    // grid's last CTA handles it (SEGS: one lane per segment that has such a row).
    if (blockIdx.x == gridDim.x - 1) {
        if constexpr (SEGS) {
            for (int j = (int)threadIdx.x; j < segs->nseg; j += kSrvThreads) {
                const ServerSegEntry& e = segs->e[j];
                if (e.ragged == 0) continue;
                const uint64_t n = (uint64_t)e.nrows_full * 32 + e.ragged;
                server_ragged_row<BITS, MODE, RANGE>(a, a.params + e.elem0, e.nrows_full, n, e.code_word0,
                                                     e.code_word0 + (n * BITS + 31) / 32, e.scale_idx);
            }
        } else if (a.nrows > a.nrows_full && threadIdx.x == kSrvThreads - 1) {
            server_ragged_row<BITS, MODE, RANGE>(a, a.params, a.nrows_full, a.n, 0, a.ncode_words,
                                                 bucket_of_row(a, a.nrows_full));
        }
    }
}

// One gradient with uniform buckets.
template <int BITS, int MODE, bool RANGE>
__global__ void __launch_bounds__(kSrvThreads, server_min_ctas<BITS>())
server_tma_kernel(const __grid_constant__ CUtensorMap map_full, const __grid_constant__ ServerTmaArgs a,
                  unsigned int* __restrict__ timeouts)
{
    server_tma_body<BITS, MODE, RANGE, false>(&map_full, a, nullptr, timeouts);
}

// The short segments of a per-layer step (those that are not entries of the segment table): their
// tiles come from the table-driven layout of mqg_segments.cuh, cut into pieces of 32 rows, one per warp
// turn.  A lane owns a row: plain loads of its code words, four workers requested at a time, and of its
// 32 parameters.  A few per cent of a layered gradient; folded into the launch of the long segments so
// that the step is one launch.
struct ServerShortSegs {
    SegmentTable tab;
    int scale_first;             // index of the table's first segment in every worker's scale array
    uint32_t pieces;             // 8 x tiles of the table
};

template <int BITS>
__device__ __noinline__ void server_short_piece(const ServerTmaArgs& a, const ServerShortSegs& ss, uint32_t piece,
                                                uint32_t lane)
{
    const TileGeom g = locate_tile<BITS>(ss.tab, piece >> 3);
    const uint32_t r = (piece & 7u) * 32u + lane;
    if (r >= (uint32_t)g.rows) return;
    const uint64_t e0 = g.elem0 + 32ull * r;
    const uint64_t left = g.valid - 32ull * r;            // elements from this row to the segment's end
    const uint64_t word0 = g.word0 + (uint64_t)r * BITS;
    const uint64_t scale_idx = (uint64_t)ss.scale_first + g.seg;
    float2 v2[16];
#pragma unroll
    for (int p = 0; p < 16; ++p) v2[p] = make_float2(0.0f, 0.0f);
    constexpr int kBatch = 4;
    for (int w0 = 0; w0 < a.W; w0 += kBatch) {
        uint32_t cw[kBatch][BITS];
        float sc[kBatch];
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            const int wk = min(w0 + i, a.W - 1);          // a worker past the last one repeats it (not summed)
#pragma unroll
            for (int k = 0; k < BITS; ++k)
                cw[i][k] = (word0 + k < g.words_end) ? __ldg(a.ptrs.codes[wk] + word0 + k) : 0u;
            sc[i] = __ldg(a.ptrs.scales[wk] + scale_idx);
        }
#pragma unroll
        for (int i = 0; i < kBatch; ++i)
            if (w0 + i < a.W) add_decoded_row<BITS>(cw[i], widen(decode_scale<BITS>(sc[i])), v2);
    }
    float* p = a.params + e0;
    if (left >= 32 && (reinterpret_cast<uintptr_t>(p) & 15u) == 0) {
        const float2 nlr = make_float2(a.neg_lr, a.neg_lr);
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const float4 q = reinterpret_cast<const float4*>(p)[c];
            const float2 lo = __ffma2_rn(nlr, v2[2 * c], make_float2(q.x, q.y));
            const float2 hi = __ffma2_rn(nlr, v2[2 * c + 1], make_float2(q.z, q.w));
            reinterpret_cast<float4*>(p)[c] = make_float4(lo.x, lo.y, hi.x, hi.y);
        }
    } else {
        float v[32];
        floats_from_pairs(v2, v);
#pragma unroll
        for (int j = 0; j < 32; ++j)
            if ((uint64_t)j < left) p[j] = __fmaf_rn(a.neg_lr, v[j], p[j]);
    }
}

// Several long segments of a per-layer step (fused update only), then the step's short segments.
template <int BITS>
__global__ void __launch_bounds__(kSrvThreads, server_min_ctas<BITS>())
server_tma_segments_kernel(const __grid_constant__ ServerSegTable segs, const __grid_constant__ ServerShortSegs ss,
                           const __grid_constant__ ServerTmaArgs a, unsigned int* __restrict__ timeouts)
{
    server_tma_body<BITS, 1, false, true>(nullptr, a, &segs, timeouts);
    const uint32_t wid = __shfl_sync(0xFFFFFFFFu, threadIdx.x >> 5, 0);
    const uint32_t nwarps = gridDim.x * kSrvWarps;
    // the warps that finished their share of the long segments first are the last ones of the grid
    for (uint32_t piece = nwarps - 1 - (blockIdx.x * kSrvWarps + wid); piece < ss.pieces; piece += nwarps)
        server_short_piece<BITS>(a, ss, piece, threadIdx.x & 31u);
}

template <int BITS, int MODE, bool RANGE>
static cudaError_t launch_server_tma_inst(const void* params, ServerTmaArgs& a, unsigned int* timeouts,
                                          cudaStream_t stream)
{
    auto kernel = server_tma_kernel<BITS, MODE, RANGE>;
    constexpr size_t kSmemBytes = sizeof(ServerSmem<BITS>) + 1024;   // + slack to round the base up
    static std::atomic<int> grid_cap[64];                 // per device; 0 = not yet set up (zero-initialised)
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int cap = grid_cap[dev].load(std::memory_order_relaxed);
    if (cap == 0) {
        int occ = 0, sms = 0;
        err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (err != cudaSuccess) return err;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kSrvThreads, kSmemBytes);
        if (err != cudaSuccess) return err;
        err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (err != cudaSuccess) return err;
        cap = sms * (occ > 0 ? occ : 1);
        grid_cap[dev].store(cap, std::memory_order_relaxed);   // every thread computes the same value
    }
    // the tiles are split evenly over the warps of the grid; tiny inputs are not spread too thin
    uint64_t grid = (uint64_t)cap;
    const uint64_t max_warps = (a.ntiles + 3) / 4;
    if (grid * kSrvWarps > max_warps) grid = (max_warps + kSrvWarps - 1) / kSrvWarps;
    CUtensorMap map_full;
    const char* why = nullptr;
    if (!encode_rows_map(&map_full, params, a.nrows_full, 4, 32, kSrvTileRows, &why)) return cudaErrorNotSupported;
    // Launched as a programmatic dependent of the kernel before it, WITHOUT releasing its own dependents
    // early: the launch is set up while that kernel still runs and starts the moment its last CTA has
    // gone (2.2 us per launch at every bit width, eight launches back to back).  Releasing the
    // dependents at the top of the kernel, as the quantize kernels do, loses that again: the next
    // launch's CTAs then take the SMs in the order in which this launch's CTAs retire, and the even
    // split of the tiles over the SMs is gone.
    return launch_pdl_smem(kernel, (unsigned)grid, kSrvThreads, kSmemBytes, stream, map_full, a, timeouts);
}

template <int BITS, bool RANGE>
static cudaError_t launch_server_tma_bits(const void* dst, ServerTmaArgs& a, int mode, unsigned int* timeouts,
                                          cudaStream_t stream)
{
    if (mode == 1) return launch_server_tma_inst<BITS, 1, RANGE>(dst, a, timeouts, stream);
    if (mode == 2) return launch_server_tma_inst<BITS, 2, RANGE>(dst, a, timeouts, stream);
    return launch_server_tma_inst<BITS, 0, RANGE>(dst, a, timeouts, stream);
}

bool server_tma_applies(uint64_t n, uint64_t bucket)
{
    const uint64_t nrows = (n + 31) / 32;
    const uint64_t rpb = bucket >= n ? nrows : bucket / 32;
    if (n / 32 < 4 * (uint64_t)kSrvTileRows || nrows > 0x7FFFFFFFull) return false;
    if (rpb >= (uint64_t)kSrvTileRows) return true;
    // Shorter buckets qualify when no 32-row tile (tiles start at multiples of 32 rows) can hold two
    // bucket boundaries, i.e. touch three buckets: the boundaries' offsets inside a tile are multiples
    // of g = gcd(rows per bucket, 32), so the first one lies at least g rows in and the next one
    // rows-per-bucket further: beyond the tile iff g + rpb >= 32 (buckets of 16, 24, 28, 30, 31 rows).
    if (rpb < 16) return false;
    uint64_t g = rpb, r = 32;
    while (r != 0) { const uint64_t t = g % r; g = r; r = t; }
    return g + rpb >= 32;
}

// log2 of the buckets a tile can touch, or -1 if the kernel does not take the shape: 1 for the shapes
// above; buckets of 8, 4, 2 or 1 rows (256 .. 32 elements) divide a tile into 4 .. 32 buckets, which
// the warp's table of 2 * kMaxWorkers entries holds for up to 16, 8, 4, 2 workers.
static int server_tma_nbt_shift(uint64_t n, uint64_t bucket, int W)
{
    if (server_tma_applies(n, bucket)) return 1;
    const uint64_t nrows = (n + 31) / 32;
    if (n / 32 < 4 * (uint64_t)kSrvTileRows || nrows > 0x7FFFFFFFull || bucket >= n) return -1;
    const uint64_t rpb = bucket / 32;
    for (int sft = 2; sft <= 5; ++sft)
        if (rpb == (32u >> sft)) return ((uint64_t)W << sft) <= 2 * (uint64_t)kMaxWorkers ? sft : -1;
    return -1;
}

bool server_tma_applies(uint64_t n, uint64_t bucket, int W) { return server_tma_nbt_shift(n, bucket, W) >= 0; }

// mode 1: dst = params (update with lr); mode 0: dst = acc (overwrite); mode 2: dst = acc (add into)
template <bool RANGE>
static cudaError_t launch_server_tma_codec(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                                           float* params, float lr, int mode, cudaStream_t stream)
{
    ServerTmaArgs a;
    a.ptrs = ptrs;
    a.params = params;
    a.n = n;
    a.ncode_words = (n * (uint64_t)bits + 31) / 32;
    a.nrows = (uint32_t)((n + 31) / 32);
    a.nrows_full = (uint32_t)(n / 32);
    a.ntiles = (a.nrows_full + kSrvTileRows - 1) / kSrvTileRows;
    a.nbuckets = (uint32_t)((n + bucket - 1) / bucket);
    const uint64_t rpb = bucket >= n ? a.nrows : bucket / 32;
    a.rows_per_bucket = (uint32_t)(rpb > 0xFFFFFFFFull ? 0xFFFFFFFFull : rpb);
    a.rpb_shift = -1;
    for (int sft = 0; sft < 32; ++sft)
        if (((uint64_t)1 << sft) == rpb) a.rpb_shift = sft;
    a.nbt_shift = server_tma_nbt_shift(n, bucket, W);
    if (a.nbt_shift < 0) return cudaErrorInvalidValue;
    a.W = W;
    a.neg_lr = -lr;
    a.bias_bits = 0x4B000000u;
    const WaitPolicy policy = wait_policy();
    a.poll_limit = policy.poll_limit;
    a.arm_only = policy.arm_only;
    unsigned int* timeouts = wait_timeout_counter();
    if (timeouts == nullptr) return cudaErrorNotSupported;
    switch (bits) {
        case 1: return launch_server_tma_bits<1, RANGE>(params, a, mode, timeouts, stream);
        case 2: return launch_server_tma_bits<2, RANGE>(params, a, mode, timeouts, stream);
        case 3: return launch_server_tma_bits<3, RANGE>(params, a, mode, timeouts, stream);
        case 4: return launch_server_tma_bits<4, RANGE>(params, a, mode, timeouts, stream);
        case 5: return launch_server_tma_bits<5, RANGE>(params, a, mode, timeouts, stream);
        case 6: return launch_server_tma_bits<6, RANGE>(params, a, mode, timeouts, stream);
        case 7: return launch_server_tma_bits<7, RANGE>(params, a, mode, timeouts, stream);
        case 8: return launch_server_tma_bits<8, RANGE>(params, a, mode, timeouts, stream);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_server_tma(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                              float* params, float lr, int mode, cudaStream_t stream)
{
    return launch_server_tma_codec<false>(ptrs, W, bits, n, bucket, params, lr, mode, stream);
}

cudaError_t launch_server_range_tma(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                                    float* params, float lr, int mode, cudaStream_t stream)
{
    return launch_server_tma_codec<true>(ptrs, W, bits, n, bucket, params, lr, mode, stream);
}

// ---- downlink: de-quantize, sum, scale to the mean and quantize again -------------------------------
// (ReceiveQGThenSendQG of Algorithm 1, lines 1-5; steps 6-8 of Fig. 3.)  The decode half is the server
// kernel's: every warp stages the code words of its 32-row tiles by asynchronous copies, two stages
// ahead, and sums the W workers in registers.  The encode half is the quantize kernels' row code.  In
// between stands the bucket maximum: a CTA takes 128 consecutive rows at a time, one 32-row tile per
// warp, so a bucket of 32 rows or fewer is reduced by lane shuffles and a bucket of 64 or 128 rows by
// the two or four warps that hold it, through shared memory and a named barrier of just those warps.
// Persistent CTAs, no CTA-wide barrier, no global load through registers.
struct RequantWarpArgs {
    ServerTmaArgs s;             // decode side: ptrs, nrows_full (= all rows), buckets, W, bias
    uint32_t* codes_out;
    float* scales_out;
    float mean_scale;
    uint32_t nct;                // CTA tiles of 128 rows
    uint32_t warps_per_bucket;   // 1 (buckets of at most 32 rows), 2 or 4
    RoundKeys rk;                // Philox round keys of the re-quantization's draws
    PhiloxHead head;             // and the launch-wide part of its blocks
};

template <int BITS>
struct RequantSmem {
    alignas(16) uint32_t code[kSrvWarps][kCodeDepth][ServerGroup<BITS>::value][kSrvTileRows * BITS];
    float4 table[kSrvWarps][2 * kMaxWorkers];
    uint32_t bmax[2][kSrvWarps];                  // tile maxima, double-buffered by the parity of the turn
};

template <int BITS>
__global__ void __launch_bounds__(kSrvThreads, 4)
requantize_warp_kernel(const __grid_constant__ RequantWarpArgs ra)
{
    extern __shared__ uint8_t smem_raw[];
    RequantSmem<BITS>& sm = *reinterpret_cast<RequantSmem<BITS>*>(
        smem_raw + ((16u - (smem_u32(smem_raw) & 15u)) & 15u));
    const ServerTmaArgs& a = ra.s;
    constexpr int kGroup = ServerGroup<BITS>::value;
    constexpr uint32_t kWorkerWords = kSrvTileRows * BITS;
    constexpr uint32_t kCodeStageBytes = kGroup * kWorkerWords * 4;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t wid = __shfl_sync(0xFFFFFFFFu, threadIdx.x >> 5, 0);
    float4* table = sm.table[wid];
    const uint32_t code_base = smem_u32(&sm.code[wid][0][0][0]);
    grid_dependency_wait();            // nothing above touches global memory

    // this CTA's tiles of 128 rows: blockIdx.x, blockIdx.x + gridDim.x, ... (the grid works on one window of
    // consecutive tiles at a time, as in the server kernel); warp w takes rows 32 w .. 32 w + 31 of each
    const uint32_t base = ra.nct / gridDim.x, extra = ra.nct % gridDim.x;
    const uint32_t nct = base + (blockIdx.x < extra ? 1u : 0u);
    const uint32_t groups = ((uint32_t)a.W + kGroup - 1) / kGroup;      // code stages per tile
    const uint32_t nunits = nct * groups;
    const bool wide = ((uint32_t)a.W << a.nbt_shift) > 32u;
    const uint32_t lane_off = lane * 16u;
    const uint32_t last_row = a.nrows_full - 1;
    const uint32_t G = ra.warps_per_bucket;
    auto tile_loc = [&](uint32_t kk) {
        TileLoc t;
        t.map = nullptr;
        t.row0 = ((blockIdx.x + kk * gridDim.x) * kSrvWarps + wid) * kSrvTileRows;
        t.nrows_full = a.nrows_full;
        t.scale_idx = 0;
        t.code_word0 = 0;
        return t;
    };
    auto fill = [&](uint32_t stage, uint32_t kk, int g0) {           // a tile beyond the last row has no codes
        const TileLoc t = tile_loc(kk);
        if (t.row0 < a.nrows_full) fill_code_stage<BITS>(a, stage, t, g0, lane_off);
    };

    uint32_t u = 0;
    if (nct > 0) {
        float2 s0[2];
        load_tile_scales<false, false>(a, tile_loc(0), lane, wide, s0);
        store_tile_scales<BITS, false>(a, table, lane, wide, s0);
#pragma unroll
        for (uint32_t u2 = 0; u2 < (uint32_t)kCodeDepth; ++u2) {
            if (u2 < nunits) fill(code_base + u2 * kCodeStageBytes, u2 / groups, (int)(u2 % groups) * kGroup);
            cp_async_commit();
        }
        __syncwarp();
    }
    uint32_t fill_tile = kCodeDepth / groups, fill_group = kCodeDepth % groups;

#pragma unroll 1
    for (uint32_t k = 0; k < nct; ++k) {
        const TileLoc loc = tile_loc(k);
        const uint32_t row0 = loc.row0;
        const bool have_next = k + 1 < nct;
        float2 s_next[2];
        if (have_next) load_tile_scales<false, false>(a, tile_loc(k + 1), lane, wide, s_next);
        const uint32_t row_c = min(row0 + lane, last_row);
        const uint32_t lb = bucket_of_row(a, row_c) - bucket_of_row(a, min(row0, last_row));
        const float4* my_table = table + lb;
        float2 v2[16];
#pragma unroll
        for (int p = 0; p < 16; ++p) v2[p] = make_float2(0.0f, 0.0f);

#pragma unroll 1
        for (uint32_t g = 0; g < groups; ++g, ++u) {
            const uint32_t cs = u % kCodeDepth;
            const uint32_t* cstage = &sm.code[wid][cs][0][0] + lane * BITS;
            cp_async_wait_group<kCodeDepth - 1>();
            __syncwarp();
            const int g0 = (int)g * kGroup;
            auto decode_worker = [&](int i) {
                uint32_t w[BITS];
                read_stage_words<BITS>(cstage + i * kWorkerWords, w);
                const float4 e = my_table[(uint32_t)(g0 + i) << a.nbt_shift];
                DecodeScale2 d;
                d.two_h = make_float2(e.x, e.y); d.minus_h = make_float2(e.z, e.w);
                add_decoded_row<BITS, false>(w, d, v2, a.bias_bits);
            };
            if (g0 + kGroup <= a.W) {
#pragma unroll
                for (int i = 0; i < kGroup; ++i) decode_worker(i);
            } else {
#pragma unroll 1
                for (int i = 0; g0 + i < a.W; ++i) decode_worker(i);
            }
            __syncwarp();                          // every lane has read the stage: refill it
            if (u + kCodeDepth < nunits) fill(code_base + cs * kCodeStageBytes, fill_tile, (int)fill_group * kGroup);
            cp_async_commit();
            if (++fill_group == groups) { fill_group = 0; ++fill_tile; }
        }

        // the mean, and the bucket maximum of its magnitudes
        const uint32_t row = row0 + lane;
        const bool active = row < a.nrows_full;
        float x[32];
        {
            const float2 ms = make_float2(ra.mean_scale, ra.mean_scale);
#pragma unroll
            for (int p = 0; p < 16; ++p) {
                const float2 y = __fmul2_rn(v2[p], ms);
                x[2 * p] = y.x;
                x[2 * p + 1] = y.y;
            }
            if (row0 + kSrvTileRows > a.nrows_full && !active) {     // only in the gradient's last tiles:
#pragma unroll
                for (int j = 0; j < 32; ++j) x[j] = 0.0f;            // lanes past the end decode what their slot holds
            }
        }
        uint32_t m = __float_as_uint(row_abs_max(x));
        if (G == 1) {
            const uint32_t rpb = min(a.rows_per_bucket, (uint32_t)kSrvTileRows);
            for (uint32_t d = rpb >> 1; d > 0; d >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
        } else {
            m = __reduce_max_sync(0xFFFFFFFFu, m);
            uint32_t* slot = sm.bmax[k & 1];
            if (lane == 0) slot[wid] = m;
            const uint32_t first = wid & ~(G - 1);
            if (G == 4 || first == 0) named_barrier<1>(32 * G);   // the warps that hold this bucket
            else named_barrier<2>(32 * G);
            m = max(slot[first], slot[first + 1]);
            if (G == 4) m = max(m, max(slot[first + 2], slot[first + 3]));
        }
        float sc = __uint_as_float(m);
        if (sc < flush_limit()) sc = 0.0f;
        if (active) {
            const bool writer = G == 1 ? (row & (a.rows_per_bucket - 1)) == 0 : ((wid & (G - 1)) == 0 && lane == 0);
            if (writer) ra.scales_out[row >> a.rpb_shift] = sc;
            const EncodeScale es = encode_scale<BITS>(sc);
            // (spreading the four Philox blocks over the decode of the workers, to fill its gaps, measured
            // 3 to 5 us slower per launch: the kernel then needs all 128 registers)
            uint32_t h[16];
            draw_row_blocks_head(4u * row, ra.head, ra.rk, h);     // the downlink draws from position 0
            uint32_t w[BITS];
            // (the encode's arithmetic in packed fp32x2 instructions: 0.5 to 1 us per launch at every width;
            // a fifth resident CTA, which 95 registers would allow, changes nothing: the kernel waits on
            // its arithmetic pipes, not on latency)
            encode_pack_row_packed<BITS>(x, es, h, w);
            store_row_words<BITS>(ra.codes_out, (uint64_t)row * BITS, w);
        }
        if (have_next) store_tile_scales<BITS, false>(a, table, lane, wide, s_next);
        __syncwarp();
    }
    cp_async_wait_group<0>();                                  // no code copy outlives the warp
}

template <int BITS>
static cudaError_t launch_requantize_warp_inst(const RequantWarpArgs& ra, cudaStream_t stream)
{
    auto kernel = requantize_warp_kernel<BITS>;
    constexpr size_t kSmemBytes = sizeof(RequantSmem<BITS>) + 16;
    static std::atomic<int> grid_cap[64];                 // per device; 0 = not yet set up (zero-initialised)
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int cap = grid_cap[dev].load(std::memory_order_relaxed);
    if (cap == 0) {
        int occ = 0, sms = 0;
        err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (err != cudaSuccess) return err;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kSrvThreads, kSmemBytes);
        if (err != cudaSuccess) return err;
        err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (err != cudaSuccess) return err;
        cap = sms * (occ > 0 ? occ : 1);
        grid_cap[dev].store(cap, std::memory_order_relaxed);   // every thread computes the same value
    }
    unsigned grid = (unsigned)cap;
    if (grid > ra.nct) grid = ra.nct;
    return launch_pdl_smem(kernel, grid, kSrvThreads, kSmemBytes, stream, ra);
}

// Whole rows, at least 512 of them, fewer than 2^30 (so the draws' block numbers have no high half),
// and buckets of 2^k rows, k <= 7 (at most 4096 elements), those below 32 rows few enough per tile for
// the warp's table.
bool requantize_warp_applies(uint64_t n, uint64_t bucket, int W)
{
    if (n % 32 != 0 || n / 32 < 512 || n / 32 >= (1ull << 30) || bucket >= n || bucket % 32 != 0) return false;
    const uint64_t rpb = bucket / 32;
    if ((rpb & (rpb - 1)) != 0 || rpb > 128) return false;
    if (rpb >= 32) return true;
    return ((uint64_t)W * (32 / rpb)) <= 2 * (uint64_t)kMaxWorkers;
}

cudaError_t launch_requantize_warp(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                                   float mean_scale, uint64_t seed, uint32_t* codes_out, float* scales_out,
                                   uint32_t worker, uint32_t step, cudaStream_t stream)
{
    RequantWarpArgs ra;
    memset(&ra, 0, sizeof(ra));
    ServerTmaArgs& a = ra.s;
    a.ptrs = ptrs;
    a.n = n;
    a.ncode_words = (n * (uint64_t)bits + 31) / 32;
    a.nrows = a.nrows_full = (uint32_t)(n / 32);
    a.nbuckets = (uint32_t)((n + bucket - 1) / bucket);
    const uint64_t rpb = bucket / 32;
    a.rows_per_bucket = (uint32_t)rpb;
    a.rpb_shift = 0;
    while (((uint64_t)1 << a.rpb_shift) < rpb) ++a.rpb_shift;
    a.nbt_shift = 0;                                     // buckets a tile of 32 rows touches: 32 / rpb
    while (rpb < 32 && (rpb << a.nbt_shift) < 32) ++a.nbt_shift;
    a.W = W;
    a.bias_bits = 0x4B000000u;
    ra.codes_out = codes_out; ra.scales_out = scales_out;
    ra.mean_scale = mean_scale;
    ra.nct = (uint32_t)((n / 32 + kSrvThreads - 1) / kSrvThreads);
    ra.warps_per_bucket = rpb <= 32 ? 1u : (uint32_t)(rpb / 32);
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        ra.rk.k0[r] = k0; ra.rk.k1[r] = k1;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    ra.rk.worker = worker; ra.rk.step = step;
    ra.head = philox_head(0u, worker, ra.rk.k0[0]);
    switch (bits) {
        case 1: return launch_requantize_warp_inst<1>(ra, stream);
        case 2: return launch_requantize_warp_inst<2>(ra, stream);
        case 3: return launch_requantize_warp_inst<3>(ra, stream);
        case 4: return launch_requantize_warp_inst<4>(ra, stream);
        case 5: return launch_requantize_warp_inst<5>(ra, stream);
        case 6: return launch_requantize_warp_inst<6>(ra, stream);
        case 7: return launch_requantize_warp_inst<7>(ra, stream);
        case 8: return launch_requantize_warp_inst<8>(ra, stream);
    }
    return cudaErrorInvalidValue;
}

// ---- several long segments of a per-layer step in one launch --------------------------------------
template <int BITS>
static cudaError_t launch_server_segs_inst(const ServerSegTable& tab, const ServerShortSegs& ss, const ServerTmaArgs& a,
                                           unsigned int* timeouts, cudaStream_t stream)
{
    auto kernel = server_tma_segments_kernel<BITS>;
    constexpr size_t kSmemBytes = sizeof(ServerSmem<BITS>) + 1024;   // + slack to round the base up
    static std::atomic<int> grid_cap[64];                 // per device; 0 = not yet set up (zero-initialised)
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int cap = grid_cap[dev].load(std::memory_order_relaxed);
    if (cap == 0) {
        int occ = 0, sms = 0;
        err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
        if (err != cudaSuccess) return err;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kSrvThreads, kSmemBytes);
        if (err != cudaSuccess) return err;
        err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (err != cudaSuccess) return err;
        cap = sms * (occ > 0 ? occ : 1);
        grid_cap[dev].store(cap, std::memory_order_relaxed);   // every thread computes the same value
    }
    uint64_t grid = (uint64_t)cap;
    const uint64_t max_warps = (a.ntiles + 3) / 4;
    if (grid * kSrvWarps > max_warps) grid = (max_warps + kSrvWarps - 1) / kSrvWarps;
    return launch_pdl_smem(kernel, (unsigned)grid, kSrvThreads, kSmemBytes, stream, tab, ss, a, timeouts);
}

bool server_tma_segment_applies(uint64_t len) { return server_tma_applies(len, len); }

cudaError_t launch_server_tma_segments(const WorkerPtrs& ptrs, int W, int bits, const ServerSegHost* segs, int nseg,
                                       const SegmentTable* short_tab, int short_first, float* params, float lr,
                                       cudaStream_t stream)
{
    if (nseg < 1 || nseg > kMaxSrvSegs) return cudaErrorInvalidValue;
    ServerShortSegs ss;
    memset(&ss, 0, sizeof(ss));
    if (short_tab != nullptr) {
        const uint64_t pieces = 8ull * short_tab->tile_start[short_tab->nseg];
        if (pieces > 0x7FFFFFFFull) return cudaErrorInvalidValue;
        ss.tab = *short_tab;
        ss.scale_first = short_first;
        ss.pieces = (uint32_t)pieces;
    }
    ServerSegTable tab;
    memset(&tab, 0, sizeof(tab));
    tab.nseg = nseg;
    uint64_t tiles = 0;
    for (int j = 0; j < nseg; ++j) {
        const ServerSegHost& h = segs[j];
        ServerSegEntry& e = tab.e[j];
        const uint64_t nrows_full = h.n / 32;
        if (nrows_full == 0 || nrows_full > 0x7FFFFFFFull) return cudaErrorInvalidValue;
        const char* why = nullptr;
        if (!encode_rows_map(&tab.map[j], params + h.elem0, nrows_full, 4, 32, kSrvTileRows, &why))
            return cudaErrorNotSupported;
        e.tile_start = (uint32_t)tiles;
        e.nrows_full = (uint32_t)nrows_full;
        e.scale_idx = h.scale_idx;
        e.ragged = (uint32_t)(h.n % 32);
        e.code_word0 = h.code_word0;
        e.elem0 = h.elem0;
        tiles += (nrows_full + kSrvTileRows - 1) / kSrvTileRows;
        if (tiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    }
    tab.e[nseg].tile_start = (uint32_t)tiles;
    ServerTmaArgs a;
    memset(&a, 0, sizeof(a));
    a.ptrs = ptrs;
    a.params = params;
    a.nrows = a.nrows_full = 1;          // not used by a launch over segments
    a.ntiles = (uint32_t)tiles;
    a.nbuckets = 1;
    a.rows_per_bucket = 1; a.rpb_shift = 0;
    a.nbt_shift = 0;                     // a tile lies in one bucket: table entry = worker
    a.W = W;
    a.neg_lr = -lr;
    a.bias_bits = 0x4B000000u;
    const WaitPolicy policy = wait_policy();
    a.poll_limit = policy.poll_limit;
    a.arm_only = policy.arm_only;
    unsigned int* timeouts = wait_timeout_counter();
    if (timeouts == nullptr) return cudaErrorNotSupported;
    switch (bits) {
        case 1: return launch_server_segs_inst<1>(tab, ss, a, timeouts, stream);
        case 2: return launch_server_segs_inst<2>(tab, ss, a, timeouts, stream);
        case 3: return launch_server_segs_inst<3>(tab, ss, a, timeouts, stream);
        case 4: return launch_server_segs_inst<4>(tab, ss, a, timeouts, stream);
        case 5: return launch_server_segs_inst<5>(tab, ss, a, timeouts, stream);
        case 6: return launch_server_segs_inst<6>(tab, ss, a, timeouts, stream);
        case 7: return launch_server_segs_inst<7>(tab, ss, a, timeouts, stream);
        case 8: return launch_server_segs_inst<8>(tab, ss, a, timeouts, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace mqg
