// Fused server pass fed by TMA (the fast path of mqg_server_step for uniform buckets):
// persistent CTAs walk tiles of 128 rows; the tile's 128 x 32 parameters arrive by a tiled bulk
// copy into a swizzled shared-memory stage, are updated in place and leave by a tiled bulk
// store, so parameter traffic never passes through registers of more than one thread and is
// always full 128-byte lines.  The W code streams are read straight from global memory with
// 128/64/32-bit loads (a thread's row is K consecutive words per worker), a group of workers
// at a time, the first group one tile ahead.  Per-(worker, bucket) de-quantization constants are computed once per tile
// into a small shared table, one tile ahead.
#include "mqg_common.cuh"
#include "mqg_internal.h"
#include "mqg_tma.cuh"

namespace mqg {

constexpr int kSrvThreads = 128;        // rows per tile = threads per CTA
constexpr int kSrvMaxBuckets = 10;      // buckets one tile can touch when a bucket has >= 16 rows

struct ServerTmaArgs {
    WorkerPtrs ptrs;
    float* params;
    uint64_t n, ncode_words;
    uint32_t nrows;              // ceil(n / 32)
    uint32_t full_tiles;         // tiles of 128 complete rows
    uint32_t nbuckets;
    uint32_t rows_per_bucket;
    int rpb_shift;               // log2(rows_per_bucket) if a power of two, else -1
    int W;
    float neg_lr;
    uint32_t bias_bits;          // 0x4B000000 (2^23), a run-time constant for the byte permutes
};

struct ServerTmaShared {
    alignas(1024) uint8_t stage[2][kSrvThreads * 128];
    float4 table[2][kMaxWorkers][kSrvMaxBuckets];     // (2h, 2h, -h, -h) per worker and bucket of the tile
    alignas(8) uint64_t bar[2];
};

__device__ __forceinline__ uint32_t bucket_of_row(const ServerTmaArgs& a, uint32_t row)
{
    return a.rpb_shift >= 0 ? row >> a.rpb_shift : row / a.rows_per_bucket;
}

// De-quantization constants of every (worker, bucket) pair the tile touches.
template <int BITS>
__device__ __forceinline__ void fill_scale_table(const ServerTmaArgs& a, float4 (*table)[kSrvMaxBuckets],
                                                 uint32_t tile)
{
    const uint32_t first = bucket_of_row(a, tile * kSrvThreads);
    const uint32_t last = bucket_of_row(a, tile * kSrvThreads + kSrvThreads - 1);
    const uint32_t nb = last - first + 1;                      // <= kSrvMaxBuckets
    for (uint32_t i = threadIdx.x; i < nb * (uint32_t)a.W; i += kSrvThreads) {
        const uint32_t w = i / nb, lb = i - w * nb;
        float s = 0.0f;
        if (first + lb < a.nbuckets) s = __ldg(a.ptrs.scales[w] + first + lb);
        const DecodeScale d = decode_scale<BITS>(s);
        table[w][lb] = make_float4(d.two_h, d.two_h, d.minus_h, d.minus_h);
    }
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

template <int BITS>
__global__ void __launch_bounds__(kSrvThreads, 5)
server_tma_kernel(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ ServerTmaArgs a,
                  unsigned int* __restrict__ timeouts)
{
    __shared__ ServerTmaShared sh;
    const uint32_t t = threadIdx.x;
    const uint32_t stride = gridDim.x;
    constexpr uint32_t kTileBytes = kSrvThreads * 128;

    if (t == 0) {
        mbar_init(smem_u32(&sh.bar[0]), 1);
        mbar_init(smem_u32(&sh.bar[1]), 1);
        fence_barrier_init();
    }
    if (t == 0) prefetch_tensormap(&tmap);
    grid_dependency_release();
    grid_dependency_wait();            // nothing above touches global memory
    uint32_t tile = blockIdx.x;
    if (tile < a.full_tiles) fill_scale_table<BITS>(a, sh.table[0], tile);
    __syncthreads();
    if (t == 0 && tile < a.full_tiles) {
        mbar_expect_tx(smem_u32(&sh.bar[0]), kTileBytes);
        tma_load_2d(smem_u32(sh.stage[0]), &tmap, 0, (int)(tile * kSrvThreads), smem_u32(&sh.bar[0]));
    }

    constexpr int kGroup = BITS <= 4 ? 8 : 32 / BITS;        // workers whose words are in flight together
    uint32_t wbuf[kGroup][BITS];
    if (tile < a.full_tiles)
        load_group<BITS, kGroup>(a, 0, (uint64_t)(tile * kSrvThreads + t) * BITS, wbuf);

    uint32_t k = 0;
    bool failed = false;
#pragma unroll 1
    for (; tile < a.full_tiles; tile += stride, ++k) {
        const uint32_t stg = k & 1, parity = (k >> 1) & 1;
        // The other stage held tile k-1, whose store was committed at the end of the last
        // iteration: once that store has read its source the stage can take tile k+1.
        if (t == 0 && tile + stride < a.full_tiles) {
            bulk_wait_read<0>();
            const uint32_t bar = smem_u32(&sh.bar[stg ^ 1]);
            mbar_expect_tx(bar, kTileBytes);
            tma_load_2d(smem_u32(sh.stage[stg ^ 1]), &tmap, 0, (int)((tile + stride) * kSrvThreads), bar);
        }

        // sum of the W de-quantized rows, in worker order; independent of the parameters, so
        // it overlaps the wait for the parameter tile
        const uint32_t row = tile * kSrvThreads + t;
        const uint32_t lb = bucket_of_row(a, row) - bucket_of_row(a, tile * kSrvThreads);
        const uint64_t word0 = (uint64_t)row * BITS;
        float2 v2[16];
#pragma unroll
        for (int p = 0; p < 16; ++p) v2[p] = make_float2(0.0f, 0.0f);
        // Workers are taken in groups of kGroup whose code words are all requested before any is
        // decoded.  The first group of this tile was requested at the end of the previous
        // iteration (or before the loop), so its latency is already covered.
#pragma unroll 1
        for (int g0 = 0; g0 < a.W; g0 += kGroup) {
            if (g0 > 0) load_group<BITS, kGroup>(a, g0, word0, wbuf);
#pragma unroll
            for (int i = 0; i < kGroup; ++i) {
                if (g0 + i < a.W) {
                    const float4 e = sh.table[stg][g0 + i][lb];
                    DecodeScale2 d;
                    d.two_h = make_float2(e.x, e.y); d.minus_h = make_float2(e.z, e.w);
                    add_decoded_row<BITS>(wbuf[i], d, v2, a.bias_bits);
                }
            }
        }

        bool ok = mbar_try_wait(smem_u32(&sh.bar[stg]), parity);
        if (!ok) ok = mbar_wait(smem_u32(&sh.bar[stg]), parity);

        // params <- fma(-lr, sum, params), in place in the stage
        {
            float4* tl = reinterpret_cast<float4*>(sh.stage[stg]);
            const float2 nlr = make_float2(a.neg_lr, a.neg_lr);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int idx = swz((int)t, c);
                const float4 p = tl[idx];
                const float2 lo = __ffma2_rn(nlr, v2[2 * c], make_float2(p.x, p.y));
                const float2 hi = __ffma2_rn(nlr, v2[2 * c + 1], make_float2(p.z, p.w));
                tl[idx] = make_float4(lo.x, lo.y, hi.x, hi.y);
            }
        }
        fence_proxy_async();                                   // the bulk store must see these writes
        if (tile + stride < a.full_tiles)                      // first worker group of the next tile
            load_group<BITS, kGroup>(a, 0, (uint64_t)((tile + stride) * kSrvThreads + t) * BITS, wbuf);
        // constants of this CTA's next tile; table[stg ^ 1] was last read two barriers ago
        if (tile + stride < a.full_tiles) fill_scale_table<BITS>(a, sh.table[stg ^ 1], tile + stride);
        failed = __syncthreads_or(!ok) != 0;
        if (failed) break;
        if (t == 0) {
            tma_store_2d(&tmap, 0, (int)(tile * kSrvThreads), smem_u32(sh.stage[stg]));
            bulk_commit();
        }
    }
    if (t == 0) {
        if (failed) {
            atomicAdd(timeouts, 1u);
            // the copy that was being waited for and the one issued at the top of this iteration
            mbar_wait(smem_u32(&sh.bar[k & 1]), (k >> 1) & 1);
            if (tile + stride < a.full_tiles) mbar_wait(smem_u32(&sh.bar[(k + 1) & 1]), ((k + 1) >> 1) & 1);
        }
        bulk_wait_all<0>();                                    // stores done before the stage goes away
    }

    // The rows after the last full tile (fewer than 128, the last one possibly ragged) are few:
    // the last CTA handles them with plain loads and stores.
    if (!failed && blockIdx.x == gridDim.x - 1) {
        const uint32_t row = a.full_tiles * kSrvThreads + t;
        if (row < a.nrows) {
            const uint64_t e0 = (uint64_t)row * 32;
            const uint64_t word0 = (uint64_t)row * BITS;
            const uint32_t bucket = bucket_of_row(a, row);
            float2 v2[16];
#pragma unroll
            for (int p = 0; p < 16; ++p) v2[p] = make_float2(0.0f, 0.0f);
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
                if (e0 + j < a.n) a.params[e0 + j] = __fmaf_rn(a.neg_lr, v[j], a.params[e0 + j]);
        }
    }
}

template <int BITS>
static cudaError_t launch_server_tma_bits(const CUtensorMap& map, const ServerTmaArgs& a,
                                          unsigned int* timeouts, cudaStream_t stream)
{
    auto kernel = server_tma_kernel<BITS>;
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
    unsigned grid = (unsigned)grid_cap[dev];
    if (grid > a.full_tiles) grid = a.full_tiles;
    return launch_pdl(kernel, grid, kSrvThreads, stream, map, a, timeouts);
}

bool server_tma_applies(uint64_t n, uint64_t bucket)
{
    const uint64_t nrows = (n + 31) / 32;
    const uint64_t rpb = bucket >= n ? nrows : bucket / 32;
    return n / 32 >= (uint64_t)kSrvThreads && nrows <= 0x7FFFFFFFull && rpb >= 16;
}

cudaError_t launch_server_tma(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                              float* params, float lr, cudaStream_t stream)
{
    ServerTmaArgs a;
    a.ptrs = ptrs;
    a.params = params;
    a.n = n;
    a.ncode_words = (n * (uint64_t)bits + 31) / 32;
    a.nrows = (uint32_t)((n + 31) / 32);
    a.full_tiles = (uint32_t)((n / 32) / kSrvThreads);
    a.nbuckets = (uint32_t)((n + bucket - 1) / bucket);
    const uint64_t rpb = bucket >= n ? a.nrows : bucket / 32;
    a.rows_per_bucket = (uint32_t)(rpb > 0xFFFFFFFFull ? 0xFFFFFFFFull : rpb);
    a.rpb_shift = -1;
    for (int sft = 0; sft < 32; ++sft)
        if (((uint64_t)1 << sft) == rpb) a.rpb_shift = sft;
    a.W = W;
    a.neg_lr = -lr;
    a.bias_bits = 0x4B000000u;
    CUtensorMap map;
    const char* why = nullptr;
    unsigned int* timeouts = wait_timeout_counter();
    if (timeouts == nullptr || !encode_rows_map(&map, params, n / 32, 4, 32, kSrvThreads, &why))
        return cudaErrorNotSupported;
    switch (bits) {
        case 1: return launch_server_tma_bits<1>(map, a, timeouts, stream);
        case 2: return launch_server_tma_bits<2>(map, a, timeouts, stream);
        case 3: return launch_server_tma_bits<3>(map, a, timeouts, stream);
        case 4: return launch_server_tma_bits<4>(map, a, timeouts, stream);
        case 5: return launch_server_tma_bits<5>(map, a, timeouts, stream);
        case 6: return launch_server_tma_bits<6>(map, a, timeouts, stream);
        case 7: return launch_server_tma_bits<7>(map, a, timeouts, stream);
        case 8: return launch_server_tma_bits<8>(map, a, timeouts, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace mqg
