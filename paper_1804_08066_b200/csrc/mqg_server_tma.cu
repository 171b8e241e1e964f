// Fused server pass fed by TMA (the fast path of mqg_server_step for uniform buckets of at
// least 1024 elements): every WARP is an independent pipeline over a contiguous range of rows.
// It walks its range in tiles of 32 rows; a tile's 32 x 32 parameters arrive by a tiled bulk
// copy into the warp's own swizzled shared-memory stage (two stages, the next tile is always in
// flight), are updated in place and leave by a tiled bulk store, so parameter traffic is always
// full 128-byte lines and never waits on another warp: there is no CTA-wide barrier anywhere.
// All warps get ranges of the same length (to within one row), so the SMs finish together.
// The W code streams are read straight from global memory with 128/64/32-bit loads (a lane's
// row is K consecutive words per worker), a group of workers at a time, the first group one
// tile ahead.  Per-(worker, bucket) de-quantization constants are computed once per tile into
// the warp's small shared table, also one tile ahead.
#include "mqg_common.cuh"
#include "mqg_internal.h"
#include "mqg_tma.cuh"

namespace mqg {

constexpr int kSrvWarps = 4;                      // warps per CTA, each with its own pipeline
constexpr int kSrvThreads = 32 * kSrvWarps;
constexpr int kSrvTileRows = 32;                  // rows per tile = lanes per warp
constexpr uint32_t kSrvTileBytes = kSrvTileRows * 128;

struct ServerTmaArgs {
    WorkerPtrs ptrs;
    float* params;
    uint64_t n, ncode_words;
    uint32_t nrows;              // ceil(n / 32)
    uint32_t nrows_full;         // floor(n / 32): rows the tensor maps cover
    uint32_t range_rows;         // rows per warp: ceil(nrows_full / number of warps in the grid)
    uint32_t nbuckets;
    uint32_t rows_per_bucket;    // >= 32, so a tile touches at most two buckets
    int rpb_shift;               // log2(rows_per_bucket) if a power of two, else -1
    int W;
    float neg_lr;
    uint32_t bias_bits;          // 0x4B000000 (2^23), a run-time constant for the byte permutes
    uint32_t tail_bytes;         // bytes of the short box: (range_rows % 32) * 128
};

struct alignas(1024) ServerWarpShared {
    uint8_t stage[2][kSrvTileBytes];
    float4 table[2][kMaxWorkers][2];      // (2h, 2h, -h, -h) per worker and bucket of the tile
    uint64_t bar[2];
};

__device__ __forceinline__ uint32_t bucket_of_row(const ServerTmaArgs& a, uint32_t row)
{
    return a.rpb_shift >= 0 ? row >> a.rpb_shift : row / a.rows_per_bucket;
}

// Requests the code words of workers g0 .. g0+GROUP-1 (those that exist) for one row.
template <int BITS, int GROUP>
__device__ __forceinline__ void load_group(const ServerTmaArgs& a, int g0, uint64_t word0,
                                           uint32_t (&wbuf)[GROUP][BITS])
{
#pragma unroll
    for (int i = 0; i < GROUP; ++i)
        if (g0 + i < a.W) load_row_words<BITS>(a.ptrs.codes[g0 + i], word0, wbuf[i]);
}

// Scales of the (worker, bucket) pairs of the tile that starts at row0: lane l holds pair l and
// pair l + 32 (pair = 2 * worker + bucket-of-tile).
__device__ __forceinline__ void load_tile_scales(const ServerTmaArgs& a, uint32_t row0, uint32_t lane,
                                                 float (&s)[2])
{
    const uint32_t first = bucket_of_row(a, row0);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t pair = lane + 32u * h, w = pair >> 1, b = first + (pair & 1u);
        s[h] = (w < (uint32_t)a.W && b < a.nbuckets) ? __ldg(a.ptrs.scales[w] + b) : 0.0f;
    }
}

template <int BITS>
__device__ __forceinline__ void store_tile_scales(const ServerTmaArgs& a, float4 (*table)[2], uint32_t lane,
                                                  const float (&s)[2])
{
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t pair = lane + 32u * h, w = pair >> 1;
        if (w < (uint32_t)a.W) {
            const DecodeScale d = decode_scale<BITS>(s[h]);
            table[w][pair & 1u] = make_float4(d.two_h, d.two_h, d.minus_h, d.minus_h);
        }
    }
}

// CTAs per SM the register budget is set for: the decode of the wider codes schedules better
// with up to 128 registers (4 CTAs = 16 warps per SM) than with 5 CTAs and 102 registers.
template <int BITS>
constexpr int server_min_ctas() { return BITS == 1 ? 5 : 4; }

// MODE 1: dst = params, dst <- fma(-lr, sum, dst).  MODE 0: dst = acc, dst <- sum.
// MODE 2: dst = acc, the sum continues from the value already there.
template <int BITS, int MODE>
__global__ void __launch_bounds__(kSrvThreads, server_min_ctas<BITS>())
server_tma_kernel(const __grid_constant__ CUtensorMap map_full, const __grid_constant__ CUtensorMap map_tail,
                  const __grid_constant__ ServerTmaArgs a, unsigned int* __restrict__ timeouts)
{
    __shared__ ServerWarpShared shared[kSrvWarps];
    const uint32_t lane = threadIdx.x & 31u, wid = threadIdx.x >> 5;
    ServerWarpShared& sh = shared[wid];

    if (lane == 0) {
        mbar_init(smem_u32(&sh.bar[0]), 1);
        mbar_init(smem_u32(&sh.bar[1]), 1);
        fence_barrier_init();
        prefetch_tensormap(&map_full);
        prefetch_tensormap(&map_tail);
    }
    grid_dependency_release();
    __syncwarp();
    grid_dependency_wait();                        // nothing above touches global memory

    // this warp's rows: [r_begin, r_end)
    const uint32_t gwarp = blockIdx.x * kSrvWarps + wid;
    const uint64_t begin64 = (uint64_t)gwarp * a.range_rows;
    const uint32_t r_begin = begin64 < a.nrows_full ? (uint32_t)begin64 : a.nrows_full;
    const uint32_t r_end = (begin64 + a.range_rows < a.nrows_full) ? r_begin + a.range_rows : a.nrows_full;
    const uint32_t ntiles = (r_end - r_begin + kSrvTileRows - 1) / kSrvTileRows;
    const uint32_t last_row = a.nrows_full - 1;    // nrows_full >= 1 on this path

    constexpr int kGroup = BITS <= 4 ? 8 : 32 / BITS;        // workers whose words are in flight together
    uint32_t wbuf[kGroup][BITS];
    bool failed = false;
    uint32_t k = 0;
    if (ntiles > 0) {
        float s0[2];
        load_tile_scales(a, r_begin, lane, s0);
        store_tile_scales<BITS>(a, sh.table[0], lane, s0);
        load_group<BITS, kGroup>(a, 0, (uint64_t)min(r_begin + lane, last_row) * BITS, wbuf);
        if (MODE != 0 && lane == 0) {
            mbar_expect_tx(smem_u32(&sh.bar[0]), kSrvTileBytes);
            tma_load_2d(smem_u32(sh.stage[0]), &map_full, 0, (int)r_begin, smem_u32(&sh.bar[0]));
        }
        __syncwarp();
    }

#pragma unroll 1
    for (; k < ntiles; ++k) {
        const uint32_t stg = k & 1, parity = (k >> 1) & 1;
        const uint32_t row0 = r_begin + k * kSrvTileRows;
        const bool have_next = k + 1 < ntiles;
        // The other stage held tile k-1, whose store was committed at the end of the last
        // iteration: once that store has read its source the stage can take tile k+1.
        if (MODE == 0) {
            // nothing is loaded: the stage is only written by this warp, once the store that used
            // it two tiles ago has read it
            if (lane == 0) bulk_wait_read<1>();
            __syncwarp();
        } else if (lane == 0 && have_next) {
            bulk_wait_read<0>();
            const uint32_t bar = smem_u32(&sh.bar[stg ^ 1]);
            const uint32_t next0 = row0 + kSrvTileRows;
            if (r_end - next0 >= (uint32_t)kSrvTileRows || r_end == a.nrows_full) {
                mbar_expect_tx(bar, kSrvTileBytes);
                tma_load_2d(smem_u32(sh.stage[stg ^ 1]), &map_full, 0, (int)next0, bar);
            } else {                               // short last tile of the range: the short box
                mbar_expect_tx(bar, a.tail_bytes);
                tma_load_2d(smem_u32(sh.stage[stg ^ 1]), &map_tail, 0, (int)next0, bar);
            }
        }
        float s_next[2];
        if (have_next) load_tile_scales(a, row0 + kSrvTileRows, lane, s_next);

        // Sum of the W de-quantized rows, in worker order.  Lanes past the end of the gradient
        // (only in the very last tile) decode the last row instead; they are never stored.
        const uint32_t row = min(row0 + lane, last_row);
        const uint32_t lb = bucket_of_row(a, row) - bucket_of_row(a, row0);
        const uint64_t word0 = (uint64_t)row * BITS;
        float2 v2[16];
        bool ok = true;
        if constexpr (MODE == 2) {
            // the sum continues from the accumulator: its tile is needed before the first worker
            ok = mbar_try_wait(smem_u32(&sh.bar[stg]), parity);
            if (!ok) ok = mbar_wait(smem_u32(&sh.bar[stg]), parity);
            const float4* tl = reinterpret_cast<const float4*>(sh.stage[stg]);
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
        const uint64_t word0_next = (uint64_t)min(row0 + kSrvTileRows + lane, last_row) * BITS;
        auto decode_slots = [&](int g0, int lo, int hi) {
#pragma unroll
            for (int i = lo; i < hi; ++i) {
                if (g0 + i < a.W) {
                    const float4 e = sh.table[stg][g0 + i][lb];
                    DecodeScale2 d;
                    d.two_h = make_float2(e.x, e.y); d.minus_h = make_float2(e.z, e.w);
                    add_decoded_row<BITS>(wbuf[i], d, v2, a.bias_bits);
                }
            }
        };
        auto prefetch_slots = [&](int lo, int hi) {      // next tile's first group into freed slots
#pragma unroll
            for (int i = lo; i < hi; ++i)
                if (i < a.W) load_row_words<BITS>(a.ptrs.codes[i], word0_next, wbuf[i]);
        };
        constexpr int kHalf = kGroup / 2;
        if (BITS >= 5 && a.W <= kGroup) {
            // one group of wide codes: the slots of each half are refilled for the next tile as
            // soon as the half has been decoded, so the requests have the rest of the tile's work
            // to land (measured: faster for K >= 5, slower for the narrow loads of K <= 3)
            decode_slots(0, 0, kHalf);
            if (have_next) prefetch_slots(0, kHalf);
            decode_slots(0, kHalf, kGroup);
            if (have_next) prefetch_slots(kHalf, kGroup);
        } else {
#pragma unroll 1
            for (int g0 = 0; g0 < a.W; g0 += kGroup) {
                if (g0 > 0) load_group<BITS, kGroup>(a, g0, word0, wbuf);
                decode_slots(g0, 0, kGroup);
            }
            if (have_next) prefetch_slots(0, kGroup);
        }

        if constexpr (MODE == 1) {
            ok = mbar_try_wait(smem_u32(&sh.bar[stg]), parity);
            if (!ok) ok = mbar_wait(smem_u32(&sh.bar[stg]), parity);
        }
        if (MODE != 0 && !__all_sync(0xFFFFFFFFu, ok)) { failed = true; break; }

        {
            float4* tl = reinterpret_cast<float4*>(sh.stage[stg]);
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
            // constants of the next tile; table[stg ^ 1] was last read in the previous iteration
            store_tile_scales<BITS>(a, sh.table[stg ^ 1], lane, s_next);
        }
        __syncwarp();
        if (lane == 0) {
            // A tile that ends at this warp's range end but before the end of the gradient must
            // not overwrite the next warp's rows: its store uses the map with the shorter box.
            // At the end of the gradient the full box is clipped by the tensor's bounds.
            const uint32_t rows_here = r_end - row0;
            if (rows_here >= (uint32_t)kSrvTileRows || r_end == a.nrows_full)
                tma_store_2d(&map_full, 0, (int)row0, smem_u32(sh.stage[stg]));
            else
                tma_store_2d(&map_tail, 0, (int)row0, smem_u32(sh.stage[stg]));
            bulk_commit();
        }
    }
    if (lane == 0) {
        if (failed) {
            atomicAdd(timeouts, 1u);
            // the copy that was being waited for and the one issued at the top of this iteration
            mbar_wait(smem_u32(&sh.bar[k & 1]), (k >> 1) & 1);
            if (k + 1 < ntiles) mbar_wait(smem_u32(&sh.bar[(k + 1) & 1]), ((k + 1) >> 1) & 1);
        }
        bulk_wait_all<0>();                                    // stores done before the stage goes away
    }

    // A last row of fewer than 32 elements is not covered by the tensor maps: one lane of the
    // grid's last warp handles it with plain loads and stores.
    if (a.nrows > a.nrows_full && blockIdx.x == gridDim.x - 1 && threadIdx.x == kSrvThreads - 1) {
        const uint32_t row = a.nrows_full;
        const uint64_t e0 = (uint64_t)row * 32;
        const uint64_t word0 = (uint64_t)row * BITS;
        const uint32_t bucket = bucket_of_row(a, row);
        float2 v2[16];
#pragma unroll
        for (int p = 0; p < 16; ++p) {
            v2[p] = make_float2(0.0f, 0.0f);
            if constexpr (MODE == 2) {
                if (e0 + 2 * p < a.n) v2[p].x = a.params[e0 + 2 * p];
                if (e0 + 2 * p + 1 < a.n) v2[p].y = a.params[e0 + 2 * p + 1];
            }
        }
        for (int w = 0; w < a.W; ++w) {
            uint32_t cw[BITS];
#pragma unroll
            for (int j = 0; j < BITS; ++j)
                cw[j] = (word0 + j < a.ncode_words) ? __ldg(a.ptrs.codes[w] + word0 + j) : 0u;
            const DecodeScale2 d = widen(decode_scale<BITS>(__ldg(a.ptrs.scales[w] + bucket)));
            add_decoded_row<BITS>(cw, d, v2);
        }
        float v[32];
        floats_from_pairs(v2, v);
#pragma unroll
        for (int j = 0; j < 32; ++j)
            if (e0 + j < a.n) a.params[e0 + j] = MODE == 1 ? __fmaf_rn(a.neg_lr, v[j], a.params[e0 + j]) : v[j];
    }
}

template <int BITS, int MODE>
static cudaError_t launch_server_tma_inst(const void* params, ServerTmaArgs& a, unsigned int* timeouts,
                                          cudaStream_t stream)
{
    auto kernel = server_tma_kernel<BITS, MODE>;
    static int grid_cap[64] = {};
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (grid_cap[dev] == 0) {
        int occ = 0, sms = 0;
        err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kernel, kSrvThreads, 0);
        if (err != cudaSuccess) return err;
        err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (err != cudaSuccess) return err;
        grid_cap[dev] = sms * (occ > 0 ? occ : 1);
    }
    // every warp of the grid gets the same number of rows (the last ones may get fewer)
    uint64_t grid = (uint64_t)grid_cap[dev];
    const uint64_t min_rows = 4 * kSrvTileRows;               // do not spread tiny inputs too thin
    const uint64_t max_warps = (a.nrows_full + min_rows - 1) / min_rows;
    if (grid * kSrvWarps > max_warps) grid = (max_warps + kSrvWarps - 1) / kSrvWarps;
    const uint64_t warps = grid * kSrvWarps;
    a.range_rows = (uint32_t)((a.nrows_full + warps - 1) / warps);
    CUtensorMap map_full, map_tail;
    const char* why = nullptr;
    if (!encode_rows_map(&map_full, params, a.nrows_full, 4, 32, kSrvTileRows, &why)) return cudaErrorNotSupported;
    const uint32_t rem = a.range_rows % kSrvTileRows;
    a.tail_bytes = (rem ? rem : (uint32_t)kSrvTileRows) * 128u;
    if (!encode_rows_map(&map_tail, params, a.nrows_full, 4, 32, rem ? rem : kSrvTileRows, &why))
        return cudaErrorNotSupported;
    return launch_pdl(kernel, (unsigned)grid, kSrvThreads, stream, map_full, map_tail, a, timeouts);
}

template <int BITS>
static cudaError_t launch_server_tma_bits(const void* dst, ServerTmaArgs& a, int mode, unsigned int* timeouts,
                                          cudaStream_t stream)
{
    if (mode == 1) return launch_server_tma_inst<BITS, 1>(dst, a, timeouts, stream);
    if (mode == 2) return launch_server_tma_inst<BITS, 2>(dst, a, timeouts, stream);
    return launch_server_tma_inst<BITS, 0>(dst, a, timeouts, stream);
}

bool server_tma_applies(uint64_t n, uint64_t bucket)
{
    const uint64_t nrows = (n + 31) / 32;
    const uint64_t rpb = bucket >= n ? nrows : bucket / 32;
    return n / 32 >= 4 * (uint64_t)kSrvTileRows && nrows <= 0x7FFFFFFFull && rpb >= (uint64_t)kSrvTileRows;
}

// mode 1: dst = params (update with lr); mode 0: dst = acc (overwrite); mode 2: dst = acc (add into)
cudaError_t launch_server_tma(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                              float* params, float lr, int mode, cudaStream_t stream)
{
    ServerTmaArgs a;
    a.ptrs = ptrs;
    a.params = params;
    a.n = n;
    a.ncode_words = (n * (uint64_t)bits + 31) / 32;
    a.nrows = (uint32_t)((n + 31) / 32);
    a.nrows_full = (uint32_t)(n / 32);
    a.range_rows = 0;
    a.nbuckets = (uint32_t)((n + bucket - 1) / bucket);
    const uint64_t rpb = bucket >= n ? a.nrows : bucket / 32;
    a.rows_per_bucket = (uint32_t)(rpb > 0xFFFFFFFFull ? 0xFFFFFFFFull : rpb);
    a.rpb_shift = -1;
    for (int sft = 0; sft < 32; ++sft)
        if (((uint64_t)1 << sft) == rpb) a.rpb_shift = sft;
    a.W = W;
    a.neg_lr = -lr;
    a.bias_bits = 0x4B000000u;
    unsigned int* timeouts = wait_timeout_counter();
    if (timeouts == nullptr) return cudaErrorNotSupported;
    switch (bits) {
        case 1: return launch_server_tma_bits<1>(params, a, mode, timeouts, stream);
        case 2: return launch_server_tma_bits<2>(params, a, mode, timeouts, stream);
        case 3: return launch_server_tma_bits<3>(params, a, mode, timeouts, stream);
        case 4: return launch_server_tma_bits<4>(params, a, mode, timeouts, stream);
        case 5: return launch_server_tma_bits<5>(params, a, mode, timeouts, stream);
        case 6: return launch_server_tma_bits<6>(params, a, mode, timeouts, stream);
        case 7: return launch_server_tma_bits<7>(params, a, mode, timeouts, stream);
        case 8: return launch_server_tma_bits<8>(params, a, mode, timeouts, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace mqg
