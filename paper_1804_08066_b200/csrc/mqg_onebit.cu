// Codec variant: one bit per element with error feedback (the 1-bit scheme of the paper's
// related-work section).  Per element v = g + e with e the worker's residual of the last
// iteration; the code is the sign of v (a zero counts as non-negative); a bucket's two
// reconstruction values are the means of its two classes, sent as (neg, pos) in the (min, max)
// variant's wire format so that the ordinary K = 1 receiver decodes them; the new residual is
// v minus the value that receiver will reconstruct: neg for code 0, fl(fl(pos - neg) + neg) for
// code 1, and neg for every element of a bucket whose spread fl(pos - neg) is below 2^-96 (its
// codes are cleared).  The class sums have a fixed order - inside a row of 32 elements a
// left-to-right chain over the members of the class, then the balanced tree over the bucket's
// rows - and the counts are exact, so the results are reproducible bit for bit.
//
// One pass: a CTA stages a tile of whole buckets (up to 256 rows) of g and of e in shared memory
// with 16-byte asynchronous copies (the whole tile in flight at once, nothing through registers),
// every thread owns a row, and the new residual leaves through e's tile with coalesced stores.
// 12 + 1/8 bytes per element of traffic for almost no arithmetic.
#include "mqg_internal.h"
#include "mqg_tree.cuh"

namespace mqg {

namespace {

struct OneBitArgs {
    const void* grad;
    float* residual;
    uint32_t* codes;
    float* ranges;
    uint64_t n, nrows, nbuckets, ncode_words, bucket_len;   // bucket_len = min(bucket, n)
    uint32_t rows_per_bucket, tile_rows, buckets_per_tile;
};

template <int DTYPE>
__device__ __forceinline__ float grad_at(const void* grad, uint64_t i)
{
    if constexpr (DTYPE == 0) return __ldcs(static_cast<const float*>(grad) + i);
    else return bf16_lo(__ldcs(static_cast<const uint16_t*>(grad) + i));
}

// tile_g <- g (widened), tile_e <- e for `rows` rows starting at element e0 (a multiple of 32, so
// 16-byte aligned in every buffer); elements at or beyond n are staged as zeros.  Whole 16-byte
// chunks travel as asynchronous copies, so a CTA has its entire tile in flight at once.
template <int DTYPE>
__device__ __forceinline__ void stage_tiles(float4* tile_g, float4* tile_e, const OneBitArgs& a, uint64_t e0, int rows)
{
    const uint64_t valid = a.n - e0;
    const int chunks = rows * 8;
    for (int idx = threadIdx.x; idx < chunks; idx += kMaxTileRows) {
        const uint64_t e = 4ull * idx;
        const int dst = swz(idx >> 3, idx & 7);
        if (e + 4 <= valid) {
            cp_async16(&tile_e[dst], a.residual + e0 + e);
            if constexpr (DTYPE == 0) {
                cp_async16(&tile_g[dst], static_cast<const float*>(a.grad) + e0 + e);
            } else {
                const uint2 gv = __ldcs(reinterpret_cast<const uint2*>(static_cast<const uint16_t*>(a.grad) + e0 + e));
                tile_g[dst] = make_float4(bf16_lo(gv.x), bf16_hi(gv.x), bf16_lo(gv.y), bf16_hi(gv.y));
            }
        } else {
            float g[4], r[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const bool in = e + k < valid;
                g[k] = in ? grad_at<DTYPE>(a.grad, e0 + e + k) : 0.0f;
                r[k] = in ? __ldcs(a.residual + e0 + e + k) : 0.0f;
            }
            tile_g[dst] = make_float4(g[0], g[1], g[2], g[3]);
            tile_e[dst] = make_float4(r[0], r[1], r[2], r[3]);
        }
    }
    cp_async_wait_all();
}

constexpr size_t kOneBitSmemBytes = 2 * kMaxTileRows * 128 + 3 * kMaxTileRows * sizeof(float) + 1024;

template <int DTYPE>
__global__ void __launch_bounds__(kMaxTileRows)
onebit_ef_kernel(const OneBitArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = smem_raw + ((1024u - ((uint32_t)__cvta_generic_to_shared(smem_raw) & 1023u)) & 1023u);
    float4* tile_g = reinterpret_cast<float4*>(base);
    float4* tile = tile_g + kMaxTileRows * 8;            // the residual's tile, rewritten in place
    float (*s_part)[kMaxTileRows] = reinterpret_cast<float (*)[kMaxTileRows]>(tile + kMaxTileRows * 8);

    const uint32_t t = threadIdx.x;
    const uint64_t row0 = (uint64_t)blockIdx.x * a.tile_rows;
    const uint64_t rows_left = a.nrows - row0;
    const int rows = (int)(rows_left < a.tile_rows ? rows_left : a.tile_rows);
    stage_tiles<DTYPE>(tile_g, tile, a, row0 * 32, rows);
    __syncthreads();

    const bool active = t < (uint32_t)rows;
    const uint64_t row = row0 + t;
    float v[32];
    uint32_t mask = 0u;                          // the row's elements that exist
    if (active) {
        float g[32];
        read_row(tile_g, (int)t, g);
        read_row(tile, (int)t, v);
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = __fadd_rn(g[j], v[j]);      // v = g + e, one rounding
        const uint64_t left = a.n - row * 32;
        mask = left >= 32 ? 0xFFFFFFFFu : ((1u << (uint32_t)left) - 1u);
    } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) v[j] = 0.0f;
    }
    // sign bits and the two class sums of the row, left to right (a non-member adds +0: exact)
    uint32_t word = 0u;
    float pos = 0.0f, neg = 0.0f;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const bool nn = v[j] >= 0.0f;
        word |= (nn ? 1u : 0u) << j;
        pos = __fadd_rn(pos, nn ? v[j] : 0.0f);
        neg = __fadd_rn(neg, nn ? 0.0f : v[j]);
    }
    word &= mask;                                // padding is staged as +0, which is no member
    const float S1 = bucket_tree_sum(pos, a.rows_per_bucket, s_part[0]);
    const float S0 = bucket_tree_sum(neg, a.rows_per_bucket, s_part[1]);
    const float c1 = bucket_tree_sum((float)__popc(word), a.rows_per_bucket, s_part[2]);   // exact: <= 8192

    const uint32_t local_bucket = t / a.rows_per_bucket;
    const uint64_t bucket = (uint64_t)blockIdx.x * a.buckets_per_tile + local_bucket;
    float e_new[32];
    if (active) {
        const uint64_t start = bucket * a.bucket_len;
        const uint64_t len = a.n - start < a.bucket_len ? a.n - start : a.bucket_len;
        const float c0 = (float)len - c1;
        const float mean0 = __fadd_rn(c0 > 0.0f ? __fdiv_rn(S0, c0) : 0.0f, 0.0f);   // -0 -> +0
        const float mean1 = __fadd_rn(c1 > 0.0f ? __fdiv_rn(S1, c1) : 0.0f, 0.0f);
        if (t % a.rows_per_bucket == 0)
            reinterpret_cast<float2*>(a.ranges)[bucket] = make_float2(mean0, mean1);
        const float r = __fsub_rn(mean1, mean0);
        const bool constant = r < flush_limit();
        const float top = __fadd_rn(r, mean0);          // what the receiver makes of code 1
        if (constant) word = 0u;
#pragma unroll
        for (int j = 0; j < 32; ++j)
            e_new[j] = __fsub_rn(v[j], ((word >> j) & 1u) ? top : mean0);
        write_row(tile, (int)t, e_new);                 // own row only: no other thread reads it
        if (row < a.ncode_words) a.codes[row] = word;   // one bit per element: one word per row
    }
    __syncthreads();
    store_tile_f32<kMaxTileRows>(tile, a.residual + row0 * 32, a.n - row0 * 32, rows);
}

}  // namespace

cudaError_t launch_quantize_onebit_ef(const void* grad, float* residual, uint64_t n, uint64_t bucket,
                                      uint32_t* codes, float* ranges, int dtype, cudaStream_t stream)
{
    OneBitArgs a;
    a.grad = grad; a.residual = residual; a.codes = codes; a.ranges = ranges;
    a.n = n;
    a.nrows = (n + 31) / 32;
    a.nbuckets = (n + bucket - 1) / bucket;
    a.ncode_words = a.nrows;
    a.bucket_len = bucket < n ? bucket : n;
    // bucket % 32 == 0 and bucket <= 8192, or a single bucket of at most 8192 elements
    const uint64_t rpb = (bucket >= n) ? a.nrows : bucket / 32;
    a.rows_per_bucket = (uint32_t)rpb;
    a.buckets_per_tile = (uint32_t)(kMaxTileRows / rpb);
    a.tile_rows = a.buckets_per_tile * a.rows_per_bucket;
    const uint64_t ntiles = (a.nrows + a.tile_rows - 1) / a.tile_rows;
    if (ntiles > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    static bool configured[2][64] = {};                 // per dtype and device
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dtype != 0][dev]) {
        err = dtype == 0 ? cudaFuncSetAttribute(onebit_ef_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)kOneBitSmemBytes)
                         : cudaFuncSetAttribute(onebit_ef_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)kOneBitSmemBytes);
        if (err != cudaSuccess) return err;
        configured[dtype != 0][dev] = true;
    }
    if (dtype == 0) onebit_ef_kernel<0><<<(unsigned)ntiles, kMaxTileRows, kOneBitSmemBytes, stream>>>(a);
    else onebit_ef_kernel<1><<<(unsigned)ntiles, kMaxTileRows, kOneBitSmemBytes, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace mqg
