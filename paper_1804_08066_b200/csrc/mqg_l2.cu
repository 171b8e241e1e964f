// Codec variant: the scale of a bucket is its Euclidean norm instead of its largest magnitude
// (the norm-scaled quantizers of the paper's related-work section); encode, draws, packing and
// the whole server side are those of the main codec.  A float sum depends on its order, so the
// order is part of the definition and every kernel here evaluates exactly this tree:
//   - rows of 32 consecutive elements counted from the bucket's first element; a row's sum of
//     squares is the left-to-right chain a <- fma(x_j, x_j, a) from a = 0 (one thread, registers);
//   - the row sums are the leaves of a balanced binary tree of adjacent pairs, the leaf count
//     padded with zeros to a power of two (lane shuffles with partner distance 1, 2, 4, ...,
//     then the warps of a bucket, then - for segments longer than a tile - the tiles);
//   - S < 2^-96 flushes the bucket, otherwise s = sqrt(S) correctly rounded.
// Adding +0 is exact, so evaluating more (all-zero) leaves or levels than the padded tree has
// does not change the result; that is what lets a fixed 256-row tile serve every bucket shape.
#include "mqg_segments.cuh"
#include "mqg_tree.cuh"

namespace mqg {

namespace {

__device__ __forceinline__ float norm_from_sum(float S)
{
    return S < flush_limit() ? 0.0f : __fsqrt_rn(S);
}

struct L2Args {
    const void* grad;
    uint32_t* codes;
    float* scales;
    uint64_t n, nrows, nbuckets, ncode_words, elem_offset;
    uint32_t rows_per_bucket, tile_rows, buckets_per_tile;
    DrawKey key;
};

// Buckets of at most 8192 elements: a CTA takes a tile of whole buckets (up to 256 rows), so the
// norm and the encode share one pass over the gradient.
template <int BITS, int DTYPE>
__global__ void __launch_bounds__(kMaxTileRows)
l2_quantize_kernel(const L2Args a)
{
    __shared__ __align__(1024) float4 tile[kMaxTileRows * 8];
    __shared__ float s_part[kMaxTileRows];

    const uint32_t t = threadIdx.x;
    const uint64_t row0 = (uint64_t)blockIdx.x * a.tile_rows;
    const uint64_t rows_left = a.nrows - row0;
    const int rows = (int)(rows_left < a.tile_rows ? rows_left : a.tile_rows);

    if constexpr (DTYPE == 0)
        load_tile_f32<kMaxTileRows>(tile, static_cast<const float*>(a.grad) + row0 * 32,
                                    a.n - row0 * 32, rows);
    else
        load_tile_bf16<kMaxTileRows>(tile, static_cast<const uint16_t*>(a.grad) + row0 * 32,
                                     a.n - row0 * 32, rows);
    __syncthreads();

    const bool active = t < (uint32_t)rows;
    float x[32];
    if (active) read_row(tile, (int)t, x);          // elements beyond n were staged as zeros
    else {
#pragma unroll
        for (int j = 0; j < 32; ++j) x[j] = 0.0f;
    }
    const float S = bucket_tree_sum(row_sum_squares(x), a.rows_per_bucket, s_part);
    if (!active) return;

    const float s = norm_from_sum(S);
    const uint32_t local_bucket = t / a.rows_per_bucket;
    const uint64_t bucket = (uint64_t)blockIdx.x * a.buckets_per_tile + local_bucket;
    if (t % a.rows_per_bucket == 0 && bucket < a.nbuckets) a.scales[bucket] = s;

    const EncodeScale es = encode_scale<BITS>(s);   // every |x| <= s: the encode needs no clamp
    const uint64_t row = row0 + t;
    const uint64_t g0 = a.elem_offset + row * 32;
    uint32_t h[16];
    if ((g0 & 7u) == 0) draw_row_aligned(g0, make_round_keys(a.key), h);
    else draw_row_unaligned(g0, a.key, h);

    uint32_t w[BITS];
    encode_pack_row<BITS>(x, es, h, w);

    const uint64_t word0 = row * BITS;
    const uint64_t e0 = row * 32;
    if (e0 + 32 <= a.n) {
        store_row_words<BITS>(a.codes, word0, w);
    } else {
        mask_row_words<BITS>(w, (int)(a.n - e0) * BITS);
#pragma unroll
        for (int k = 0; k < BITS; ++k)
            if (word0 + k < a.ncode_words) a.codes[word0 + k] = w[k];
    }
}

// Segments, pass 1: the tile's sum (an aligned subtree of 256
// rows) goes to partial[blockIdx.x].
template <int DTYPE>
__global__ void __launch_bounds__(kMaxTileRows)
l2_partials_kernel(const void* __restrict__ grad, const SegmentTable tab, float* __restrict__ partial)
{
    __shared__ __align__(1024) float4 tile[kMaxTileRows * 8];
    __shared__ float s_part[kMaxTileRows / 32];
    const uint32_t t = threadIdx.x;
    const TileGeom g = locate_tile<1>(tab, blockIdx.x);
    if constexpr (DTYPE == 0)
        load_tile_f32<kMaxTileRows>(tile, static_cast<const float*>(grad) + g.elem0, g.valid, g.rows);
    else
        load_tile_bf16<kMaxTileRows>(tile, static_cast<const uint16_t*>(grad) + g.elem0, g.valid, g.rows);
    __syncthreads();
    float a = 0.0f;
    if (t < (uint32_t)g.rows) {
        float x[32];
        read_row(tile, (int)t, x);
        a = row_sum_squares(x);
    }
    a = warp_tree(a, 32);
    if ((t & 31) == 0) s_part[t >> 5] = a;
    __syncthreads();
    if (t == 0) partial[blockIdx.x] = tree8(s_part, 0, kMaxTileRows / 32);
}

// Pass 2: one CTA per segment folds the segment's tile sums, in place, one tree level per
// barrier, and writes the segment's scale.
__global__ void __launch_bounds__(256)
l2_finish_kernel(const SegmentTable tab, float* __restrict__ partial, float* __restrict__ scales)
{
    const uint32_t seg = blockIdx.x;
    const uint64_t first = tab.tile_start[seg], count = tab.tile_start[seg + 1] - first;
    float* p = partial + first;
    for (uint64_t d = 1; d < count; d <<= 1) {
        for (uint64_t j = (uint64_t)threadIdx.x * 2 * d; j < count; j += 256ull * 2 * d)
            if (j + d < count) p[j] = __fadd_rn(p[j], p[j + d]);   // a missing partner is a zero leaf
        __syncthreads();
    }
    if (threadIdx.x == 0) scales[seg] = count ? norm_from_sum(p[0]) : 0.0f;
}

template <int BITS>
cudaError_t launch_l2_bits(const L2Args& a, int dtype, unsigned grid, cudaStream_t stream)
{
    if (dtype == 0) l2_quantize_kernel<BITS, 0><<<grid, kMaxTileRows, 0, stream>>>(a);
    else l2_quantize_kernel<BITS, 1><<<grid, kMaxTileRows, 0, stream>>>(a);
    return cudaGetLastError();
}

// partials -> scales for one table; `partial` has room for the table's tiles.
cudaError_t sums_and_scales(const void* grad, const SegmentTable& tab, float* scales, int dtype, float* partial,
                            cudaStream_t stream)
{
    const uint32_t ntiles = tab.tile_start[tab.nseg];
    if (tab.nseg == 0) return cudaSuccess;
    if (ntiles != 0) {
        if (dtype == 0) l2_partials_kernel<0><<<ntiles, kMaxTileRows, 0, stream>>>(grad, tab, partial);
        else l2_partials_kernel<1><<<ntiles, kMaxTileRows, 0, stream>>>(grad, tab, partial);
        const cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
    }
    l2_finish_kernel<<<(unsigned)tab.nseg, 256, 0, stream>>>(tab, partial, scales);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_quantize_l2(const void* grad, uint64_t n, int bits, uint64_t bucket, uint64_t seed,
                               uint32_t* codes, float* scales, int dtype, uint32_t worker, uint32_t step,
                               uint64_t elem_offset, cudaStream_t stream)
{
    if (quantize_norm_fused_applies(n, bucket, elem_offset))        // TMA-fed persistent kernel
        return launch_quantize_norm_fused(grad, n, bits, bucket, seed, codes, scales, dtype, worker, step,
                                          elem_offset, stream);
    L2Args a;
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
    const unsigned grid = (unsigned)ntiles;
    switch (bits) {
        case 1: return launch_l2_bits<1>(a, dtype, grid, stream);
        case 2: return launch_l2_bits<2>(a, dtype, grid, stream);
        case 3: return launch_l2_bits<3>(a, dtype, grid, stream);
        case 4: return launch_l2_bits<4>(a, dtype, grid, stream);
        case 5: return launch_l2_bits<5>(a, dtype, grid, stream);
        case 6: return launch_l2_bits<6>(a, dtype, grid, stream);
        case 7: return launch_l2_bits<7>(a, dtype, grid, stream);
        case 8: return launch_l2_bits<8>(a, dtype, grid, stream);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_segments_l2_scales(const void* grad, const SegmentTable& tab, float* scales_base, int dtype,
                                      float* partial, cudaStream_t stream)
{
    return sums_and_scales(grad, tab, scales_base, dtype, partial, stream);
}

}  // namespace mqg
