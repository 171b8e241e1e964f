// Worker side with one scale per segment (per-layer scale) or with buckets larger than a CTA
// tile: the max and the encode cannot share one pass over on-chip storage, so the gradient
// is read twice -- a max pass that folds every tile's max (if it reaches the flush limit) into
// scales[] with an atomic max on the float's bit pattern, then an encode pass identical to the
// one-pass kernel's.
#include "mqg_segments.cuh"

namespace mqg {

template <int DTYPE>
__global__ void __launch_bounds__(kMaxTileRows)
absmax_segments_kernel(const SegQuantArgs a, const SegmentTable tab)
{
    __shared__ uint32_t s_warp[kMaxTileRows / 32];
    const TileGeom g = locate_tile<1>(tab, blockIdx.x);
    const uint64_t count = g.valid < (uint64_t)(kMaxTileRows * 32) ? g.valid : (uint64_t)(kMaxTileRows * 32);
    float mx = 0.0f;
    if constexpr (DTYPE == 0) {
        const float* src = static_cast<const float*>(a.grad) + g.elem0;
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
        const uint16_t* src = static_cast<const uint16_t*>(a.grad) + g.elem0;
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
        // a tile's maximum below the flush limit does not count: a segment whose every tile stays below
        // it keeps the scale 0 the pass started from, so the scale that stands after the pass is final
        if (threadIdx.x == 0 && m >= __float_as_uint(flush_limit()))
            atomicMax(reinterpret_cast<unsigned int*>(a.scales) + g.seg, m);
    }
}

template <int BITS, int DTYPE>
__global__ void __launch_bounds__(kMaxTileRows)
encode_segments_kernel(const SegQuantArgs a, const SegmentTable tab)
{
    __shared__ __align__(1024) float4 tile[kMaxTileRows * 8];
    const uint32_t t = threadIdx.x;
    const TileGeom g = locate_tile<BITS>(tab, blockIdx.x);

    if constexpr (DTYPE == 0)
        load_tile_f32<kMaxTileRows>(tile, static_cast<const float*>(a.grad) + g.elem0, g.valid, g.rows);
    else
        load_tile_bf16<kMaxTileRows>(tile, static_cast<const uint16_t*>(a.grad) + g.elem0, g.valid, g.rows);

    const float s = a.scales[g.seg];        // final: the max pass has applied the flush
    __syncthreads();
    if (t >= (uint32_t)g.rows) return;

    float x[32];
    read_row(tile, (int)t, x);
    const EncodeScale es = encode_scale<BITS>(s);
    const uint64_t g0 = a.elem_offset + g.elem0 + 32ull * t;
    uint32_t h[16];
    if ((g0 & 7u) == 0) draw_row_aligned(g0, make_round_keys(a.key), h);
    else draw_row_unaligned(g0, a.key, h);

    uint32_t w[BITS];
    encode_pack_row<BITS>(x, es, h, w);

    const uint64_t word0 = g.word0 + (uint64_t)t * BITS;
    const uint64_t left = g.valid - 32ull * t;          // elements of the segment from this row on
    if (left < 32) mask_row_words<BITS>(w, (int)left * BITS);
#pragma unroll
    for (int k = 0; k < BITS; ++k)
        if (word0 + k < g.words_end) a.codes[word0 + k] = w[k];
}

template <int BITS>
static cudaError_t launch_encode_bits(const SegQuantArgs& a, const SegmentTable& tab, int dtype,
                                      unsigned grid, cudaStream_t stream)
{
    if (dtype == 0) encode_segments_kernel<BITS, 0><<<grid, kMaxTileRows, 0, stream>>>(a, tab);
    else encode_segments_kernel<BITS, 1><<<grid, kMaxTileRows, 0, stream>>>(a, tab);
    return cudaGetLastError();
}

cudaError_t launch_encode_segments(const SegQuantArgs& a, const SegmentTable& tab, int bits, int dtype,
                                   unsigned grid, cudaStream_t stream)
{
    switch (bits) {
        case 1: return launch_encode_bits<1>(a, tab, dtype, grid, stream);
        case 2: return launch_encode_bits<2>(a, tab, dtype, grid, stream);
        case 3: return launch_encode_bits<3>(a, tab, dtype, grid, stream);
        case 4: return launch_encode_bits<4>(a, tab, dtype, grid, stream);
        case 5: return launch_encode_bits<5>(a, tab, dtype, grid, stream);
        case 6: return launch_encode_bits<6>(a, tab, dtype, grid, stream);
        case 7: return launch_encode_bits<7>(a, tab, dtype, grid, stream);
        case 8: return launch_encode_bits<8>(a, tab, dtype, grid, stream);
    }
    return cudaErrorInvalidValue;
}

static cudaError_t two_pass(const SegQuantArgs& a, const SegmentTable& tab, uint64_t ntiles,
                            uint64_t nscales, int bits, int dtype, cudaStream_t stream)
{
    cudaError_t err = cudaMemsetAsync(a.scales, 0, nscales * sizeof(float), stream);
    if (err != cudaSuccess) return err;
    if (ntiles == 0) return cudaSuccess;
    if (ntiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    const unsigned grid = (unsigned)ntiles;
    if (dtype == 0) absmax_segments_kernel<0><<<grid, kMaxTileRows, 0, stream>>>(a, tab);
    else absmax_segments_kernel<1><<<grid, kMaxTileRows, 0, stream>>>(a, tab);
    err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    return launch_encode_segments(a, tab, bits, dtype, grid, stream);
}

// The two passes of the per-layer quantizer as separate launches (the caller may give some segments'
// encode to another kernel): the max pass over every segment of `tab`, and the encode pass over the
// tiles `tab` lists.
cudaError_t launch_segments_absmax(const void* grad, const SegmentTable& tab, float* scales_base, int dtype,
                                   cudaStream_t stream)
{
    SegQuantArgs a;
    a.grad = grad; a.codes = nullptr; a.scales = scales_base; a.elem_offset = 0;
    a.key.seed_lo = a.key.seed_hi = a.key.worker = a.key.step = 0;
    cudaError_t err = cudaMemsetAsync(scales_base, 0, (size_t)tab.nseg * sizeof(float), stream);
    if (err != cudaSuccess) return err;
    const uint32_t ntiles = tab.tile_start[tab.nseg];
    if (ntiles == 0) return cudaSuccess;
    if (dtype == 0) absmax_segments_kernel<0><<<ntiles, kMaxTileRows, 0, stream>>>(a, tab);
    else absmax_segments_kernel<1><<<ntiles, kMaxTileRows, 0, stream>>>(a, tab);
    return cudaGetLastError();
}

cudaError_t launch_segments_encode(const void* grad, const SegmentTable& tab, int bits, uint64_t seed,
                                   uint32_t* codes, float* scales_base, int dtype, uint32_t worker,
                                   uint32_t step, uint64_t elem_offset, cudaStream_t stream)
{
    SegQuantArgs a;
    a.grad = grad; a.codes = codes; a.scales = scales_base; a.elem_offset = elem_offset;
    a.key.seed_lo = (uint32_t)seed; a.key.seed_hi = (uint32_t)(seed >> 32);
    a.key.worker = worker; a.key.step = step;
    const uint32_t ntiles = tab.tile_start[tab.nseg];
    if (ntiles == 0) return cudaSuccess;
    return launch_encode_segments(a, tab, bits, dtype, ntiles, stream);
}

cudaError_t launch_quantize_big_buckets(const void* grad, uint64_t n, int bits, uint64_t bucket,
                                        uint64_t seed, uint32_t* codes, float* scales, int dtype,
                                        uint32_t worker, uint32_t step, uint64_t elem_offset,
                                        cudaStream_t stream)
{
    SegQuantArgs a;
    a.grad = grad; a.codes = codes; a.scales = scales; a.elem_offset = elem_offset;
    a.key.seed_lo = (uint32_t)seed; a.key.seed_hi = (uint32_t)(seed >> 32);
    a.key.worker = worker; a.key.step = step;
    SegmentTable tab;
    tab.nseg = 0;
    const uint64_t b = bucket < n ? bucket : n;          // a single bucket is n long
    tab.uniform_bucket = b;
    tab.n_total = n;
    const uint64_t tile_elems = (uint64_t)kMaxTileRows * 32;
    const uint64_t tpb = (b + tile_elems - 1) / tile_elems;
    if (tpb > 0xFFFFFFFFull) return cudaErrorInvalidValue;
    tab.tiles_per_bucket = (uint32_t)tpb;
    const uint64_t nb = (n + b - 1) / b;
    const uint64_t full = n / b;                          // full buckets have tpb tiles each
    uint64_t ntiles = full * tpb;
    if (nb > full) ntiles += ((n - full * b) + tile_elems - 1) / tile_elems;
    // the grid enumerates tiles_per_bucket tiles for every bucket; the last (shorter) bucket
    // has fewer real tiles, so its tail tiles are simply not launched
    return two_pass(a, tab, ntiles, nb, bits, dtype, stream);
}

}  // namespace mqg
