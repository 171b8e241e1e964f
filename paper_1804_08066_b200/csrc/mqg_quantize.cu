// Worker side: per-bucket max-abs scale, stochastic-rounding encode and bit packing in one
// pass over the gradient (Quantize(g, K) of Algorithm 1, WorkerIterate).
//
// Work decomposition: the gradient is cut into rows of 32 elements; a CTA takes a tile of
// up to 256 rows that holds whole buckets, stages it in shared memory with coalesced 128-bit
// loads, and each thread then owns one row: it reads its 32 values from shared memory,
// takes part in the bucket's max reduction, draws its 32 sixteen-bit random numbers from
// four Philox blocks, encodes, packs into K words and stores them.  The gradient is read
// from HBM exactly once.
#include "mqg_common.cuh"
#include "mqg_internal.h"

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
    DrawKey key;
};

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

    float mx = 0.0f;
#pragma unroll
    for (int j = 0; j < 32; ++j) mx = fmaxf(mx, fabsf(x[j]));

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
    if constexpr (ALIGNED_DRAWS) draw_row_aligned(a.elem_offset + row * 32, a.key, h);
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

cudaError_t launch_quantize_fused(const void* grad, uint64_t n, int bits, uint64_t bucket,
                                  uint64_t seed, uint32_t* codes, float* scales, int dtype,
                                  uint32_t worker, uint32_t step, uint64_t elem_offset,
                                  cudaStream_t stream)
{
    QuantizeArgs a;
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
    const uint64_t ntiles = (a.nrows + a.tile_rows - 1) / a.tile_rows;
    if (ntiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;
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

}  // namespace mqg
