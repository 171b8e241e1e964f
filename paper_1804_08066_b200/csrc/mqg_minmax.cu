// General (any shape) kernels of the (min, max) nearest-rounding codec variant: the scheme the
// footnote of Section 3.2 refers to, a bucket's range [min, max] mapped linearly onto the 2^K
// codes.  The fast paths are the TMA kernels in mqg_quantize.cu (RANGE tile) and
// mqg_server_tma.cu; the kernels here take every other shape: buckets above 4096 elements, tiny
// inputs, small buckets on the server side, an extra accumulator output.  A thread owns a row of
// 32 elements throughout; buckets are whole rows (multiples of 32 elements, or one bucket).
#include "mqg_common.cuh"
#include "mqg_internal.h"

namespace mqg {

constexpr int kRangeThreads = 256;

struct RangeArgs {
    const void* grad;
    uint32_t* codes;
    float* ranges;               // 2 floats per bucket; holds ordered bits between the passes
    uint64_t n, nrows, nbuckets, ncode_words, rows_per_bucket;
    int warp_in_one_bucket;      // every warp's 32 rows lie in one bucket
};

// The valid elements of a row as floats; the elements a ragged last row lacks repeat its first
// element, which is neutral for min / max and never stored.
template <int DTYPE>
__device__ __forceinline__ void load_row(const RangeArgs& a, uint64_t row, float (&x)[32])
{
    const uint64_t e0 = row * 32;
    if (e0 + 32 <= a.n) {
        if constexpr (DTYPE == 0) {
            const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(a.grad) + e0);
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float4 v = __ldg(p + c);
                x[4 * c] = v.x; x[4 * c + 1] = v.y; x[4 * c + 2] = v.z; x[4 * c + 3] = v.w;
            }
        } else {
            const uint4* p = reinterpret_cast<const uint4*>(static_cast<const uint16_t*>(a.grad) + e0);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint4 v = __ldg(p + c);
                const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    x[8 * c + 2 * k] = bf16_lo(u[k]);
                    x[8 * c + 2 * k + 1] = bf16_hi(u[k]);
                }
            }
        }
    } else {
        const uint64_t left = a.n - e0;                  // >= 1
        for (int j = 0; j < 32; ++j) {
            const uint64_t e = e0 + ((uint64_t)j < left ? j : 0);
            if constexpr (DTYPE == 0) x[j] = __ldg(static_cast<const float*>(a.grad) + e);
            else x[j] = __uint_as_float((uint32_t)__ldg(static_cast<const uint16_t*>(a.grad) + e) << 16);
        }
    }
}

__global__ void range_init_kernel(uint32_t* ranges_bits, uint64_t nbuckets)
{
    const uint64_t b = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (b < nbuckets) {
        ranges_bits[2 * b] = kOrderedMinIdentity;
        ranges_bits[2 * b + 1] = kOrderedMaxIdentity;
    }
}

// Pass 1: every row folds its min and max into its bucket's pair of ordered-bit words.
template <int DTYPE>
__global__ void __launch_bounds__(kRangeThreads)
range_reduce_kernel(const RangeArgs a)
{
    const uint64_t row = (uint64_t)blockIdx.x * kRangeThreads + threadIdx.x;
    const bool active = row < a.nrows;
    uint32_t mlo = kOrderedMinIdentity, mhi = kOrderedMaxIdentity;
    uint64_t bucket = 0;
    if (active) {
        float x[32], lo, hi;
        load_row<DTYPE>(a, row, x);
        row_min_max(x, lo, hi);
        mlo = ordered_bits(lo); mhi = ordered_bits(hi);
        bucket = row / a.rows_per_bucket;
    }
    uint32_t* out = reinterpret_cast<uint32_t*>(a.ranges);
    if (a.warp_in_one_bucket) {
        mlo = __reduce_min_sync(0xFFFFFFFFu, mlo);
        mhi = __reduce_max_sync(0xFFFFFFFFu, mhi);
        // lane 0's row is the warp's first row: active whenever any lane is
        if ((threadIdx.x & 31) == 0 && active) {
            atomicMin(out + 2 * bucket, mlo);
            atomicMax(out + 2 * bucket + 1, mhi);
        }
    } else if (active) {
        atomicMin(out + 2 * bucket, mlo);
        atomicMax(out + 2 * bucket + 1, mhi);
    }
}

// Ordered bits -> floats, a zero of either sign stored as +0.
__global__ void range_finalize_kernel(float* ranges, uint64_t nbuckets)
{
    const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < 2 * nbuckets)
        ranges[i] = __fadd_rn(from_ordered_bits(reinterpret_cast<const uint32_t*>(ranges)[i]), 0.0f);
}

// Pass 2: encode and pack against the finished ranges.
template <int BITS, int DTYPE>
__global__ void __launch_bounds__(kRangeThreads)
range_encode_kernel(const RangeArgs a)
{
    const uint64_t row = (uint64_t)blockIdx.x * kRangeThreads + threadIdx.x;
    if (row >= a.nrows) return;
    float x[32];
    load_row<DTYPE>(a, row, x);
    const uint64_t bucket = row / a.rows_per_bucket;
    const RangeEncodeScale es = range_encode_scale<BITS>(__ldg(a.ranges + 2 * bucket), __ldg(a.ranges + 2 * bucket + 1));
    uint32_t w[BITS];
    range_encode_pack_row<BITS>(x, es, w);
    const uint64_t word0 = row * BITS;
    if (row * 32 + 32 <= a.n) {
        store_row_words<BITS>(a.codes, word0, w);
    } else {
        mask_row_words<BITS>(w, (int)(a.n - row * 32) * BITS);
#pragma unroll
        for (int k = 0; k < BITS; ++k)
            if (word0 + k < a.ncode_words) a.codes[word0 + k] = w[k];
    }
}

template <int BITS>
static void launch_encode(const RangeArgs& a, int dtype, unsigned grid, cudaStream_t stream)
{
    if (dtype == 0) range_encode_kernel<BITS, 0><<<grid, kRangeThreads, 0, stream>>>(a);
    else range_encode_kernel<BITS, 1><<<grid, kRangeThreads, 0, stream>>>(a);
}

cudaError_t launch_quantize_range_general(const void* grad, uint64_t n, int bits, uint64_t bucket,
                                          uint32_t* codes, float* ranges, int dtype, cudaStream_t stream)
{
    RangeArgs a;
    a.grad = grad; a.codes = codes; a.ranges = ranges;
    a.n = n;
    a.nrows = (n + 31) / 32;
    a.nbuckets = (n + bucket - 1) / bucket;
    a.ncode_words = (n * (uint64_t)bits + 31) / 32;
    a.rows_per_bucket = bucket >= n ? a.nrows : bucket / 32;
    a.warp_in_one_bucket = (bucket >= n || a.rows_per_bucket % 32 == 0) ? 1 : 0;
    const uint64_t row_blocks = (a.nrows + kRangeThreads - 1) / kRangeThreads;
    const uint64_t pair_blocks = (2 * a.nbuckets + 255) / 256;
    if (row_blocks > 0x7FFFFFFFull || pair_blocks > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    range_init_kernel<<<(unsigned)((a.nbuckets + 255) / 256), 256, 0, stream>>>(reinterpret_cast<uint32_t*>(ranges),
                                                                                a.nbuckets);
    if (dtype == 0) range_reduce_kernel<0><<<(unsigned)row_blocks, kRangeThreads, 0, stream>>>(a);
    else range_reduce_kernel<1><<<(unsigned)row_blocks, kRangeThreads, 0, stream>>>(a);
    range_finalize_kernel<<<(unsigned)pair_blocks, 256, 0, stream>>>(ranges, a.nbuckets);
    const unsigned grid = (unsigned)row_blocks;
    switch (bits) {
        case 1: launch_encode<1>(a, dtype, grid, stream); break;
        case 2: launch_encode<2>(a, dtype, grid, stream); break;
        case 3: launch_encode<3>(a, dtype, grid, stream); break;
        case 4: launch_encode<4>(a, dtype, grid, stream); break;
        case 5: launch_encode<5>(a, dtype, grid, stream); break;
        case 6: launch_encode<6>(a, dtype, grid, stream); break;
        case 7: launch_encode<7>(a, dtype, grid, stream); break;
        case 8: launch_encode<8>(a, dtype, grid, stream); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

// ---- server side, any shape ---------------------------------------------------------------
struct RangeServerArgs {
    WorkerPtrs ptrs;             // scales[w] = worker w's ranges
    float* params;               // may be null
    float* acc;                  // may be null when params is given
    uint64_t n, nrows, ncode_words, rows_per_bucket;
    int W, add_into;
    float neg_lr;
    uint32_t bias_bits;
};

template <int BITS>
__global__ void __launch_bounds__(kRangeThreads)
range_server_kernel(const __grid_constant__ RangeServerArgs a)
{
    const uint64_t row = (uint64_t)blockIdx.x * kRangeThreads + threadIdx.x;
    if (row >= a.nrows) return;
    const uint64_t e0 = row * 32, word0 = row * BITS, bucket = row / a.rows_per_bucket;
    const bool full = e0 + 32 <= a.n;
    float2 v2[16];
#pragma unroll
    for (int p = 0; p < 16; ++p) {
        v2[p] = make_float2(0.0f, 0.0f);
        if (a.add_into) {                                    // the sum continues from the accumulator
            if (e0 + 2 * p < a.n) v2[p].x = a.acc[e0 + 2 * p];
            if (e0 + 2 * p + 1 < a.n) v2[p].y = a.acc[e0 + 2 * p + 1];
        }
    }
    for (int w = 0; w < a.W; ++w) {
        uint32_t cw[BITS];
        if (full) {
            load_row_words<BITS>(a.ptrs.codes[w], word0, cw);
        } else {
#pragma unroll
            for (int j = 0; j < BITS; ++j)
                cw[j] = (word0 + j < a.ncode_words) ? __ldg(a.ptrs.codes[w] + word0 + j) : 0u;
        }
        const DecodeScale2 d = widen(range_decode_scale<BITS>(__ldg(a.ptrs.scales[w] + 2 * bucket),
                                                              __ldg(a.ptrs.scales[w] + 2 * bucket + 1)));
        add_decoded_row<BITS, true>(cw, d, v2, a.bias_bits);
    }
    float v[32];
    floats_from_pairs(v2, v);
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if (e0 + j < a.n) {
            if (a.acc) a.acc[e0 + j] = v[j];
            if (a.params) a.params[e0 + j] = __fmaf_rn(a.neg_lr, v[j], a.params[e0 + j]);
        }
    }
}

cudaError_t launch_server_range(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                                float* params, float lr, float* acc, int add_into, cudaStream_t stream)
{
    if (server_tma_applies(n, bucket, W)) {
        if (params != nullptr && acc == nullptr)
            return launch_server_range_tma(ptrs, W, bits, n, bucket, params, lr, 1, stream);
        if (params == nullptr)
            return launch_server_range_tma(ptrs, W, bits, n, bucket, acc, 0.0f, add_into ? 2 : 0, stream);
    }
    RangeServerArgs a;
    a.ptrs = ptrs; a.params = params; a.acc = acc;
    a.n = n;
    a.nrows = (n + 31) / 32;
    a.ncode_words = (n * (uint64_t)bits + 31) / 32;
    a.rows_per_bucket = bucket >= n ? a.nrows : bucket / 32;
    a.W = W; a.add_into = add_into;
    a.neg_lr = -lr;
    a.bias_bits = 0x4B000000u;
    const uint64_t blocks = (a.nrows + kRangeThreads - 1) / kRangeThreads;
    if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    const unsigned grid = (unsigned)blocks;
    switch (bits) {
        case 1: range_server_kernel<1><<<grid, kRangeThreads, 0, stream>>>(a); break;
        case 2: range_server_kernel<2><<<grid, kRangeThreads, 0, stream>>>(a); break;
        case 3: range_server_kernel<3><<<grid, kRangeThreads, 0, stream>>>(a); break;
        case 4: range_server_kernel<4><<<grid, kRangeThreads, 0, stream>>>(a); break;
        case 5: range_server_kernel<5><<<grid, kRangeThreads, 0, stream>>>(a); break;
        case 6: range_server_kernel<6><<<grid, kRangeThreads, 0, stream>>>(a); break;
        case 7: range_server_kernel<7><<<grid, kRangeThreads, 0, stream>>>(a); break;
        case 8: range_server_kernel<8><<<grid, kRangeThreads, 0, stream>>>(a); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace mqg
