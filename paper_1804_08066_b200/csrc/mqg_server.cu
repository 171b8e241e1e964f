// Server side: unpack + de-quantize the W workers' buffers, sum them in worker order and apply
// the SGD update, in one pass (De-quantize, sum and update of Algorithm 1,
// ReceiveQGThenSendQG / steps 6-7 of Fig. 3).
//
// Same decomposition as the worker kernel: a thread owns a row of 32 elements, i.e. K code
// words per worker (read straight from global memory, vectorised where K allows) and 32
// parameters (moved through a swizzled shared-memory tile so that global accesses stay
// coalesced 128-bit).
#include "mqg_segments.cuh"

namespace mqg {

struct ServerArgs {
    WorkerPtrs ptrs;
    float* params;           // may be null (accumulate only)
    float* acc;              // may be null when params != null
    uint64_t n, nrows, ncode_words;
    uint32_t rows_per_bucket;
    int scale_base;          // segments: index of the table's first segment in scales[]
    int W;
    int add_into;
    float lr;
};

// Sum of the W de-quantized rows in worker order, continuing from v[] when have_init.
// VEC: the row's words may be fetched with the vector width the bit width allows.
template <int BITS, bool VEC>
__device__ __forceinline__ void accumulate_row(const ServerArgs& a, uint64_t scale_idx,
                                               uint64_t word0, uint64_t words_end, bool full_row,
                                               float (&v)[32], bool have_init)
{
    float2 v2[16];
    if (have_init) pairs_from_floats(v, v2);
    else {
#pragma unroll
        for (int p = 0; p < 16; ++p) v2[p] = make_float2(0.0f, 0.0f);
    }
    // four workers at a time: their code words and scales are all requested before the first one is
    // decoded, so that a row waits for global memory once per four workers, not once per worker
    constexpr int kBatch = 4;
    for (int w0 = 0; w0 < a.W; w0 += kBatch) {
        uint32_t w[kBatch][BITS];
        float sc[kBatch];
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            const int wk = min(w0 + i, a.W - 1);            // a worker past the last one repeats it (not summed)
            if (VEC && full_row) load_row_words<BITS>(a.ptrs.codes[wk], word0, w[i]);
            else {
#pragma unroll
                for (int k = 0; k < BITS; ++k)
                    w[i][k] = (word0 + k < words_end) ? __ldg(a.ptrs.codes[wk] + word0 + k) : 0u;
            }
            sc[i] = __ldg(a.ptrs.scales[wk] + scale_idx);
        }
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            if (w0 + i < a.W) {
                const DecodeScale2 d = widen(decode_scale<BITS>(sc[i]));
                add_decoded_row<BITS>(w[i], d, v2);
            }
        }
    }
    floats_from_pairs(v2, v);
}

// MODE 0: acc = sum (optionally continuing from acc).  MODE 1: params update, acc optional.
// SEG: tiles come from a segment table (one scale per segment) instead of uniform buckets.
template <int BITS, int MODE, bool SEG>
__global__ void __launch_bounds__(kMaxTileRows)
server_kernel(const ServerArgs a, const SegmentTable tab)
{
    __shared__ __align__(1024) float4 tile[kMaxTileRows * 8];

    const uint32_t t = threadIdx.x;
    uint64_t elem0, valid, word0, words_end, scale_idx;
    int rows;
    if constexpr (SEG) {
        const TileGeom g = locate_tile<BITS>(tab, blockIdx.x);
        elem0 = g.elem0; valid = g.valid; rows = g.rows;
        word0 = g.word0 + (uint64_t)t * BITS;
        words_end = g.words_end;
        scale_idx = (uint64_t)a.scale_base + g.seg;
    } else {
        const uint64_t row0 = (uint64_t)blockIdx.x * kMaxTileRows;
        const uint64_t rows_left = a.nrows - row0;
        rows = (int)(rows_left < (uint64_t)kMaxTileRows ? rows_left : (uint64_t)kMaxTileRows);
        elem0 = row0 * 32; valid = a.n - elem0;
        word0 = (row0 + t) * BITS;
        words_end = a.ncode_words;
        scale_idx = (row0 + t) / a.rows_per_bucket;
    }
    const bool active = t < (uint32_t)rows;
    const bool full_row = 32ull * t + 32 <= valid;

    float v[32];
    if constexpr (MODE == 0) {
        float* acc = a.acc + elem0;
        if (a.add_into) {
            load_tile_f32<kMaxTileRows>(tile, acc, valid, rows);
            __syncthreads();
            if (active) read_row(tile, (int)t, v);
        }
        if (active) {
            accumulate_row<BITS, !SEG>(a, scale_idx, word0, words_end, full_row, v, a.add_into != 0);
            write_row(tile, (int)t, v);
        }
        __syncthreads();
        store_tile_f32<kMaxTileRows>(tile, acc, valid, rows);
    } else {
        float* params = a.params + elem0;
        load_tile_f32<kMaxTileRows, false>(tile, params, valid, rows);    // in flight during the decode
        if (active) accumulate_row<BITS, !SEG>(a, scale_idx, word0, words_end, full_row, v, false);
        cp_async_wait_all();
        __syncthreads();
        if (active) {
            float p[32];
            read_row(tile, (int)t, p);
            const float nlr = -a.lr;
#pragma unroll
            for (int j = 0; j < 32; ++j) p[j] = __fmaf_rn(nlr, v[j], p[j]);
            write_row(tile, (int)t, p);
        }
        __syncthreads();
        store_tile_f32<kMaxTileRows>(tile, params, valid, rows);
        if (a.acc != nullptr) {
            __syncthreads();
            if (active) write_row(tile, (int)t, v);
            __syncthreads();
            store_tile_f32<kMaxTileRows>(tile, a.acc + elem0, valid, rows);
        }
    }
}

__global__ void __launch_bounds__(256)
apply_kernel(float* __restrict__ params, const float* __restrict__ acc, float lr, uint64_t n)
{
    const float nlr = -lr;
    const uint64_t n4 = n / 4;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        float4 p = reinterpret_cast<float4*>(params)[i];
        const float4 g = __ldcs(reinterpret_cast<const float4*>(acc) + i);
        p.x = __fmaf_rn(nlr, g.x, p.x);
        p.y = __fmaf_rn(nlr, g.y, p.y);
        p.z = __fmaf_rn(nlr, g.z, p.z);
        p.w = __fmaf_rn(nlr, g.w, p.w);
        reinterpret_cast<float4*>(params)[i] = p;
    }
    if (blockIdx.x == 0 && threadIdx.x < (n & 3)) {
        const uint64_t i = n4 * 4 + threadIdx.x;
        params[i] = __fmaf_rn(nlr, acc[i], params[i]);
    }
}

template <int BITS, bool SEG>
static cudaError_t launch_server_bits(const ServerArgs& a, const SegmentTable& tab, unsigned grid,
                                      cudaStream_t stream)
{
    if (a.params == nullptr) server_kernel<BITS, 0, SEG><<<grid, kMaxTileRows, 0, stream>>>(a, tab);
    else server_kernel<BITS, 1, SEG><<<grid, kMaxTileRows, 0, stream>>>(a, tab);
    return cudaGetLastError();
}

template <bool SEG>
static cudaError_t dispatch_bits(int bits, const ServerArgs& a, const SegmentTable& tab,
                                 uint64_t ntiles, cudaStream_t stream)
{
    if (ntiles == 0) return cudaSuccess;
    if (ntiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    const unsigned grid = (unsigned)ntiles;
    switch (bits) {
        case 1: return launch_server_bits<1, SEG>(a, tab, grid, stream);
        case 2: return launch_server_bits<2, SEG>(a, tab, grid, stream);
        case 3: return launch_server_bits<3, SEG>(a, tab, grid, stream);
        case 4: return launch_server_bits<4, SEG>(a, tab, grid, stream);
        case 5: return launch_server_bits<5, SEG>(a, tab, grid, stream);
        case 6: return launch_server_bits<6, SEG>(a, tab, grid, stream);
        case 7: return launch_server_bits<7, SEG>(a, tab, grid, stream);
        case 8: return launch_server_bits<8, SEG>(a, tab, grid, stream);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_server(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                          float* params, float lr, float* acc, int add_into, cudaStream_t stream)
{
    if (server_tma_applies(n, bucket, W)) {
        if (params != nullptr && acc == nullptr)
            return launch_server_tma(ptrs, W, bits, n, bucket, params, lr, 1, stream);
        if (params == nullptr)
            return launch_server_tma(ptrs, W, bits, n, bucket, acc, 0.0f, add_into ? 2 : 0, stream);
    }
    ServerArgs a;
    a.ptrs = ptrs;
    a.params = params; a.acc = acc;
    a.n = n;
    a.nrows = (n + 31) / 32;
    a.ncode_words = (n * (uint64_t)bits + 31) / 32;
    // bucket % 32 == 0, or a single bucket (bucket >= n): every row lies in one bucket
    const uint64_t rpb = (bucket >= n) ? a.nrows : bucket / 32;
    a.rows_per_bucket = (uint32_t)(rpb > 0xFFFFFFFFull ? 0xFFFFFFFFull : rpb);
    a.scale_base = 0;
    a.W = W; a.add_into = add_into; a.lr = lr;
    SegmentTable tab;
    tab.nseg = 0; tab.uniform_bucket = 0; tab.n_total = n; tab.tiles_per_bucket = 0;
    return dispatch_bits<false>(bits, a, tab, (a.nrows + kMaxTileRows - 1) / kMaxTileRows, stream);
}

cudaError_t launch_server_segments(const WorkerPtrs& ptrs, int W, int bits, const SegmentTable& tab,
                                   int scale_base, float* params, float lr, float* acc,
                                   cudaStream_t stream)
{
    ServerArgs a;
    a.ptrs = ptrs;
    a.params = params; a.acc = acc;
    a.n = 0; a.nrows = 0; a.ncode_words = 0; a.rows_per_bucket = 1;
    a.scale_base = scale_base;
    a.W = W; a.add_into = 0; a.lr = lr;
    return dispatch_bits<true>(bits, a, tab, tab.tile_start[tab.nseg], stream);
}

cudaError_t launch_apply(float* params, const float* acc, float lr, uint64_t n, cudaStream_t stream)
{
    const uint64_t n4 = n / 4;
    uint64_t blocks = (n4 + 255) / 256;
    if (blocks < 1) blocks = 1;
    int dev = 0, sms = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err == cudaSuccess) err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (err != cudaSuccess) return err;
    if (blocks > (uint64_t)sms * 16) blocks = (uint64_t)sms * 16;
    apply_kernel<<<(unsigned)blocks, 256, 0, stream>>>(params, acc, lr, n);
    return cudaGetLastError();
}

}  // namespace mqg
