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
    int W;
    float mean_scale;
    DrawKey key;
};

template <int BITS>
__global__ void __launch_bounds__(kMaxTileRows)
requantize_kernel(const RequantArgs a)
{
    __shared__ uint32_t s_bucket[kMaxTileRows];
    const uint32_t t = threadIdx.x;
    const uint64_t row0 = (uint64_t)blockIdx.x * a.tile_rows;
    const uint64_t rows_left = a.nrows - row0;
    const uint32_t rows = (uint32_t)(rows_left < a.tile_rows ? rows_left : a.tile_rows);
    const bool active = t < rows;
    const uint64_t row = row0 + t;
    const uint32_t local_bucket = t / a.rows_per_bucket;
    const uint64_t bucket = (uint64_t)blockIdx.x * a.buckets_per_tile + local_bucket;

    if (t < a.buckets_per_tile) s_bucket[t] = 0u;
    __syncthreads();

    float x[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) x[j] = 0.0f;
    if (active) {
        const uint64_t word0 = row * BITS;
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
        floats_from_pairs(v2, x);
        const uint64_t left = a.n - row * 32;              // elements of this row that exist
#pragma unroll
        for (int j = 0; j < 32; ++j) x[j] = ((uint64_t)j < left) ? __fmul_rn(x[j], a.mean_scale) : 0.0f;
    }

    const uint32_t mbits = [&] {
        uint32_t m = __float_as_uint(row_abs_max(x));
        const uint32_t rpb = a.rows_per_bucket;
        if ((rpb & (rpb - 1)) == 0 && rpb <= 32) {
            for (uint32_t d = rpb >> 1; d > 0; d >>= 1) m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
            return m;
        }
        if (active) atomicMax(&s_bucket[local_bucket], m);
        __syncthreads();
        return active ? s_bucket[local_bucket] : 0u;
    }();
    if (!active) return;

    float s = __uint_as_float(mbits);
    if (s < flush_limit()) s = 0.0f;
    if (t % a.rows_per_bucket == 0 && bucket < a.nbuckets) a.scales_out[bucket] = s;

    const EncodeScale es = encode_scale<BITS>(s);
    uint32_t h[16];
    draw_row_aligned(row * 32, make_round_keys(a.key), h);
    uint32_t w[BITS];
    encode_pack_row<BITS>(x, es, h, w);
    const uint64_t word0 = row * BITS;
    if (row * 32 + 32 <= a.n) {
        store_row_words<BITS>(a.codes_out, word0, w);
    } else {
        mask_row_words<BITS>(w, (int)(a.n - row * 32) * BITS);
#pragma unroll
        for (int k = 0; k < BITS; ++k)
            if (word0 + k < a.ncode_words) a.codes_out[word0 + k] = w[k];
    }
}

cudaError_t launch_requantize(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                              float mean_scale, uint64_t seed, uint32_t* codes_out, float* scales_out,
                              uint32_t worker, uint32_t step, cudaStream_t stream)
{
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
    a.key.seed_lo = (uint32_t)seed; a.key.seed_hi = (uint32_t)(seed >> 32);
    a.key.worker = worker; a.key.step = step;
    const uint64_t ntiles = (a.nrows + a.tile_rows - 1) / a.tile_rows;
    if (ntiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    const unsigned grid = (unsigned)ntiles;
    switch (bits) {
        case 1: requantize_kernel<1><<<grid, kMaxTileRows, 0, stream>>>(a); break;
        case 2: requantize_kernel<2><<<grid, kMaxTileRows, 0, stream>>>(a); break;
        case 3: requantize_kernel<3><<<grid, kMaxTileRows, 0, stream>>>(a); break;
        case 4: requantize_kernel<4><<<grid, kMaxTileRows, 0, stream>>>(a); break;
        case 5: requantize_kernel<5><<<grid, kMaxTileRows, 0, stream>>>(a); break;
        case 6: requantize_kernel<6><<<grid, kMaxTileRows, 0, stream>>>(a); break;
        case 7: requantize_kernel<7><<<grid, kMaxTileRows, 0, stream>>>(a); break;
        case 8: requantize_kernel<8><<<grid, kMaxTileRows, 0, stream>>>(a); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace mqg
