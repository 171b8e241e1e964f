// Downlink half of the server (ReceiveQGThenSendQG of Algorithm 1, steps 6-8 of Fig. 3):
// de-quantize and sum the W workers' buffers, scale the sum to the mean, and quantize the result
// again with the same bit width for the broadcast -- in one pass, so the fp32 global gradient
// never touches HBM.  A thread owns a row of 32 elements; a CTA owns whole buckets: the row sums
// stay in registers while the bucket maximum is found, then are encoded and packed.
#include "mqg_common.cuh"
#include "mqg_internal.h"

namespace mqg {

struct RequantArgs {
    WorkerPtrs ptrs;
    uint32_t* codes_out;
    float* scales_out;
    uint64_t n, nrows, nbuckets, ncode_words;
    uint32_t rows_per_bucket, tile_rows, buckets_per_tile;
    uint32_t full_tiles;         // leading tiles whose 256 rows are all complete
    int W;
    float mean_scale;
    uint32_t bias_bits;          // 0x4B000000 (2^23), a run-time constant for the byte permutes
    RoundKeys rk;                // Philox round keys of the re-quantization's draws
};

// De-quantization constants (2h, -h) per (worker, bucket of the tile), computed once per tile when
// the tile holds at most kTableBuckets buckets; smaller buckets compute them per row.
constexpr int kTableBuckets = 32;

// A row's BITS words from a staged copy of a worker's code words (widest access the offset allows).
template <int BITS>
__device__ __forceinline__ void staged_row_words(const uint32_t* __restrict__ p, uint32_t (&w)[BITS])
{
    if constexpr (BITS % 4 == 0) {
#pragma unroll
        for (int k = 0; k < BITS / 4; ++k) {
            const uint4 v = reinterpret_cast<const uint4*>(p)[k];
            w[4 * k] = v.x; w[4 * k + 1] = v.y; w[4 * k + 2] = v.z; w[4 * k + 3] = v.w;
        }
    } else if constexpr (BITS % 2 == 0) {
#pragma unroll
        for (int k = 0; k < BITS / 2; ++k) {
            const uint2 v = reinterpret_cast<const uint2*>(p)[k];
            w[2 * k] = v.x; w[2 * k + 1] = v.y;
        }
    } else {
#pragma unroll
        for (int k = 0; k < BITS; ++k) w[k] = p[k];
    }
}

// One tile.  FULL: every thread owns a complete row (vector loads, no bounds checks).  TABLE: the
// de-quantization constants come from the shared table.  STAGE (full tiles only): all workers' code
// words of the tile are copied into shared memory by 16-byte asynchronous copies at the start, so
// that no worker's decode waits for a global load.
template <int BITS, bool FULL, bool TABLE, bool STAGE>
__device__ __forceinline__ void requantize_tile(const RequantArgs& a, uint32_t* s_bucket,
                                                float2 (*s_table)[kTableBuckets], uint32_t* s_codes)
{
    const uint32_t t = threadIdx.x;
    const uint64_t row0 = (uint64_t)blockIdx.x * a.tile_rows;
    const uint64_t rows_left = a.nrows - row0;
    const uint32_t rows = FULL ? a.tile_rows : (uint32_t)(rows_left < a.tile_rows ? rows_left : a.tile_rows);
    const bool active = FULL || t < rows;
    const uint64_t row = row0 + t;
    const uint32_t local_bucket = t / a.rows_per_bucket;
    const uint64_t bucket = (uint64_t)blockIdx.x * a.buckets_per_tile + local_bucket;

    constexpr uint32_t kWorkerWords = kMaxTileRows * BITS;      // one worker's words of a full tile
    if constexpr (FULL && STAGE) {
        const uint32_t chunks = (uint32_t)a.W * (kWorkerWords / 4);
        for (uint32_t idx = t; idx < chunks; idx += kMaxTileRows) {
            const uint32_t w = idx / (kWorkerWords / 4), c = idx - w * (kWorkerWords / 4);
            cp_async16(s_codes + w * kWorkerWords + 4 * c, a.ptrs.codes[w] + row0 * BITS + 4 * c);
        }
    }
    if (t < a.buckets_per_tile) s_bucket[t] = 0u;
    if (TABLE) {
        for (uint32_t idx = t; idx < (uint32_t)a.W * a.buckets_per_tile; idx += blockDim.x) {
            const uint32_t w = idx / a.buckets_per_tile, lbk = idx - w * a.buckets_per_tile;
            const uint64_t gb = (uint64_t)blockIdx.x * a.buckets_per_tile + lbk;
            const DecodeScale d = decode_scale<BITS>(gb < a.nbuckets ? __ldg(a.ptrs.scales[w] + gb) : 0.0f);
            s_table[w][lbk] = make_float2(d.two_h, d.minus_h);
        }
    }
    if constexpr (FULL && STAGE) cp_async_wait_all();
    __syncthreads();

    float x[32];
    if (active) {
        const uint64_t word0 = row * BITS;
        float2 v2[16];
#pragma unroll
        for (int p = 0; p < 16; ++p) v2[p] = make_float2(0.0f, 0.0f);
#pragma unroll 4
        for (int w = 0; w < a.W; ++w) {
            uint32_t cw[BITS];
            if constexpr (FULL && STAGE) {
                staged_row_words<BITS>(s_codes + w * kWorkerWords + t * BITS, cw);
            } else if (FULL) {
                load_row_words<BITS>(a.ptrs.codes[w], word0, cw);
            } else {
#pragma unroll
                for (int j = 0; j < BITS; ++j)
                    cw[j] = (word0 + j < a.ncode_words) ? __ldg(a.ptrs.codes[w] + word0 + j) : 0u;
            }
            DecodeScale2 d;
            if (TABLE) {
                const float2 e = s_table[w][local_bucket];
                d.two_h = make_float2(e.x, e.x); d.minus_h = make_float2(e.y, e.y);
            } else {
                d = widen(decode_scale<BITS>(__ldg(a.ptrs.scales[w] + bucket)));
            }
            add_decoded_row<BITS>(cw, d, v2, a.bias_bits);
        }
        const float2 ms = make_float2(a.mean_scale, a.mean_scale);
#pragma unroll
        for (int p = 0; p < 16; ++p) v2[p] = __fmul2_rn(v2[p], ms);
        floats_from_pairs(v2, x);
        if (!FULL) {
            const uint64_t left = a.n - row * 32;          // elements of this row that exist
#pragma unroll
            for (int j = 0; j < 32; ++j) x[j] = ((uint64_t)j < left) ? x[j] : 0.0f;
        }
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) x[j] = 0.0f;
    }

    uint32_t m = __float_as_uint(row_abs_max(x));
    const uint32_t rpb = a.rows_per_bucket;
    if ((rpb & (rpb - 1)) == 0 && rpb <= 32) {
        for (uint32_t d = rpb >> 1; d > 0; d >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
    } else {
        if (active) atomicMax(&s_bucket[local_bucket], m);
        __syncthreads();
        m = active ? s_bucket[local_bucket] : 0u;
    }
    if (!active) return;

    float s = __uint_as_float(m);
    if (s < flush_limit()) s = 0.0f;
    if (t % a.rows_per_bucket == 0 && (FULL || bucket < a.nbuckets)) a.scales_out[bucket] = s;

    const EncodeScale es = encode_scale<BITS>(s);
    uint32_t h[16];
    // Philox block of the row's first element: 4 * row (64-bit; the downlink draws from position 0)
    draw_row_blocks((uint32_t)(row << 2), (uint32_t)(row >> 30), a.rk, h);
    uint32_t w[BITS];
    encode_pack_row<BITS>(x, es, h, w);
    const uint64_t word0 = row * BITS;
    if (FULL || row * 32 + 32 <= a.n) {
        store_row_words<BITS>(a.codes_out, word0, w);
    } else {
        mask_row_words<BITS>(w, (int)(a.n - row * 32) * BITS);
#pragma unroll
        for (int k = 0; k < BITS; ++k)
            if (word0 + k < a.ncode_words) a.codes_out[word0 + k] = w[k];
    }
}

template <int BITS, bool TABLE, bool STAGE>
__global__ void __launch_bounds__(kMaxTileRows)
requantize_kernel(const __grid_constant__ RequantArgs a)
{
    extern __shared__ __align__(16) uint32_t s_codes[];        // STAGE: W x 256 x BITS words
    __shared__ uint32_t s_bucket[kMaxTileRows];
    __shared__ float2 s_table[TABLE ? kMaxWorkers : 1][kTableBuckets];
    if (blockIdx.x < a.full_tiles) requantize_tile<BITS, true, TABLE, STAGE>(a, s_bucket, s_table, s_codes);
    else requantize_tile<BITS, false, TABLE, STAGE>(a, s_bucket, s_table, s_codes);
}

// Code words are staged in shared memory when all workers' words of a tile fit in 64 KB (three CTAs
// per SM at that size; the kernel is bound by arithmetic, not by occupancy).
constexpr size_t kMaxStagedCodeBytes = 64 * 1024;

template <int BITS>
static cudaError_t launch_requantize_bits(const RequantArgs& a, unsigned grid, cudaStream_t stream)
{
    if (a.buckets_per_tile > (uint32_t)kTableBuckets) {
        requantize_kernel<BITS, false, false><<<grid, kMaxTileRows, 0, stream>>>(a);
        return cudaGetLastError();
    }
    // Measured per width at n = 25 M, W = 8 (us per launch, register loads -> staged): 2: 60.6 -> 51.9,
    // 3: 58.4 -> 54.5, 4: 58.6 -> 57.0, 8: 67.9 -> 57.5; 1 unchanged; 5, 6, 7 two microseconds slower
    // (their rows are not 8- or 16-byte multiples, so the staged words are read back one by one).
    constexpr bool kStagePays = BITS == 2 || BITS == 3 || BITS == 4 || BITS == 8;
    const size_t staged = (size_t)a.W * kMaxTileRows * BITS * sizeof(uint32_t);
    if (!kStagePays || a.full_tiles == 0 || staged > kMaxStagedCodeBytes) {
        requantize_kernel<BITS, true, false><<<grid, kMaxTileRows, 0, stream>>>(a);
        return cudaGetLastError();
    }
    static bool configured[64] = {};                           // per device
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        err = cudaFuncSetAttribute(requantize_kernel<BITS, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   (int)kMaxStagedCodeBytes);
        if (err != cudaSuccess) return err;
        configured[dev] = true;
    }
    requantize_kernel<BITS, true, true><<<grid, kMaxTileRows, staged, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_requantize(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                              float mean_scale, uint64_t seed, uint32_t* codes_out, float* scales_out,
                              uint32_t worker, uint32_t step, cudaStream_t stream)
{
    if (requantize_warp_applies(n, bucket, W))
        return launch_requantize_warp(ptrs, W, bits, n, bucket, mean_scale, seed, codes_out, scales_out, worker, step,
                                      stream);
    RequantArgs a;
    a.ptrs = ptrs; a.codes_out = codes_out; a.scales_out = scales_out;
    a.n = n;
    a.nrows = (n + 31) / 32;
    a.nbuckets = (n + bucket - 1) / bucket;
    a.ncode_words = (n * (uint64_t)bits + 31) / 32;
    const uint64_t rpb = (bucket >= n) ? a.nrows : bucket / 32;     // <= 256 (checked by the caller)
    a.rows_per_bucket = (uint32_t)rpb;
    a.buckets_per_tile = (uint32_t)(kMaxTileRows / rpb);
    a.tile_rows = a.buckets_per_tile * a.rows_per_bucket;
    a.W = W; a.mean_scale = mean_scale;
    a.bias_bits = 0x4B000000u;
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        a.rk.k0[r] = k0; a.rk.k1[r] = k1;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    a.rk.worker = worker; a.rk.step = step;
    const uint64_t ntiles = (a.nrows + a.tile_rows - 1) / a.tile_rows;
    if (ntiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    a.full_tiles = a.tile_rows == (uint32_t)kMaxTileRows ? (uint32_t)((n / 32) / a.tile_rows) : 0u;
    const unsigned grid = (unsigned)ntiles;
    switch (bits) {
        case 1: return launch_requantize_bits<1>(a, grid, stream);
        case 2: return launch_requantize_bits<2>(a, grid, stream);
        case 3: return launch_requantize_bits<3>(a, grid, stream);
        case 4: return launch_requantize_bits<4>(a, grid, stream);
        case 5: return launch_requantize_bits<5>(a, grid, stream);
        case 6: return launch_requantize_bits<6>(a, grid, stream);
        case 7: return launch_requantize_bits<7>(a, grid, stream);
        case 8: return launch_requantize_bits<8>(a, grid, stream);
    }
    return cudaErrorInvalidValue;
}

}  // namespace mqg
