// Host-side launchers behind the C ABI (arguments already validated by mqg_api.cu).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace mqg {

// For entry points implemented outside mqg_api.cu: stores the calling thread's message for
// mqg_last_error() and returns `code`.
int report_error(int code, const char* fmt, ...);

constexpr int kMaxWorkers = 32;
constexpr int kMaxSegmentsPerLaunch = 64;

struct WorkerPtrs {
    const uint32_t* codes[kMaxWorkers];
    const float* scales[kMaxWorkers];
};

// Segment table passed by value to the segment kernels (one chunk of <= kMaxSegmentsPerLaunch
// segments per launch).  A tile is 256 rows of 32 elements inside one segment.
// uniform_bucket != 0 selects the arithmetic layout instead of the table: segment j is
// elements [j * uniform_bucket, min((j+1) * uniform_bucket, n_total)), its codes start at word
// j * uniform_bucket * bits / 32, and it has tiles_per_bucket tiles.
struct SegmentTable {
    int nseg;
    uint32_t tile_start[kMaxSegmentsPerLaunch + 1];   // prefix sum of tiles per segment
    uint64_t seg_off[kMaxSegmentsPerLaunch + 1];      // element offsets
    uint64_t code_off[kMaxSegmentsPerLaunch];         // word offsets
    uint64_t uniform_bucket;
    uint64_t n_total;
    uint32_t tiles_per_bucket;
};

cudaError_t launch_quantize_fused(const void* grad, uint64_t n, int bits, uint64_t bucket,
                                  uint64_t seed, uint32_t* codes, float* scales, int dtype,
                                  uint32_t worker, uint32_t step, uint64_t elem_offset,
                                  cudaStream_t stream);

// One launch for W >= 2 workers' gradients of the same shape (host arrays of device pointers);
// worker w draws as worker id first_worker + w.  Only when quantize_workers_applies() holds.
// mode: 0 = the main codec, 1 = the (min, max) variant (`scales[w]` then points at worker w's ranges, two floats
// per bucket; seed, first_worker, step and elem_offset are not used), 2 = the L2-norm scale variant.
bool quantize_workers_applies(int W, uint64_t n, uint64_t bucket, uint64_t elem_offset);
cudaError_t launch_quantize_workers(const void* const* grads, int W, uint64_t n, int bits,
                                    uint64_t bucket, uint64_t seed, uint32_t* const* codes,
                                    float* const* scales, int dtype, uint32_t first_worker,
                                    uint32_t step, uint64_t elem_offset, int mode, cudaStream_t stream);

// (min, max) nearest-rounding variant.  ranges[2b] = lo, ranges[2b + 1] = hi of bucket b.
// Fused one-pass kernel for buckets of at most 4096 elements; otherwise the general launches
// (ranges by atomics on ordered bits, then encode).
bool quantize_range_fused_applies(uint64_t n, uint64_t bucket);
cudaError_t launch_quantize_range_fused(const void* grad, uint64_t n, int bits, uint64_t bucket,
                                        uint32_t* codes, float* ranges, int dtype, cudaStream_t stream);
cudaError_t launch_quantize_range_general(const void* grad, uint64_t n, int bits, uint64_t bucket,
                                          uint32_t* codes, float* ranges, int dtype, cudaStream_t stream);
// Server pass of the variant: `ptrs.scales[w]` points at worker w's ranges.
cudaError_t launch_server_range(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                                float* params, float lr, float* acc, int add_into, cudaStream_t stream);
cudaError_t launch_server_range_tma(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                                    float* dst, float lr, int mode, cudaStream_t stream);

// L2-norm scale variant.  Buckets of at most kMaxFusedBucket elements: one pass.  Segments: tile
// sums into `partial` (one float per tile of the table, in tile order) and a fold per segment give
// the scales (launch_segments_l2_scales); the encode is the ordinary segment encode.
bool quantize_norm_fused_applies(uint64_t n, uint64_t bucket, uint64_t elem_offset);
cudaError_t launch_quantize_norm_fused(const void* grad, uint64_t n, int bits, uint64_t bucket, uint64_t seed,
                                       uint32_t* codes, float* scales, int dtype, uint32_t worker,
                                       uint32_t step, uint64_t elem_offset, cudaStream_t stream);
cudaError_t launch_quantize_l2(const void* grad, uint64_t n, int bits, uint64_t bucket, uint64_t seed,
                               uint32_t* codes, float* scales, int dtype, uint32_t worker, uint32_t step,
                               uint64_t elem_offset, cudaStream_t stream);
cudaError_t launch_segments_l2_scales(const void* grad, const SegmentTable& tab, float* scales_base, int dtype,
                                      float* partial, cudaStream_t stream);

// 1-bit error-feedback variant: sign codes, class means as (neg, pos) ranges, residual updated in
// place.  Buckets of at most kMaxFusedBucket elements.
cudaError_t launch_quantize_onebit_ef(const void* grad, float* residual, uint64_t n, uint64_t bucket,
                                      uint32_t* codes, float* ranges, int dtype, cudaStream_t stream);

// The two passes of the per-layer quantizer (scales_base points at the scale of the table's first
// segment), and the encode of ONE long segment (= one
// bucket whose scale already stands at *scale) on the TMA-fed quantize kernel.
cudaError_t launch_segments_absmax(const void* grad, const SegmentTable& tab, float* scales_base, int dtype,
                                   cudaStream_t stream);
cudaError_t launch_segments_encode(const void* grad, const SegmentTable& tab, int bits, uint64_t seed,
                                   uint32_t* codes, float* scales_base, int dtype, uint32_t worker,
                                   uint32_t step, uint64_t elem_offset, cudaStream_t stream);
// Shortest segment that gets a launch of its own on the bulk-copy kernels (one-worker per-layer calls), and
// shortest segment that becomes one entry of a launch shared by many segments (the all-workers quantizer,
// the per-layer server step): 8 tiles of 128 rows.  Shorter segments go through the table-driven code.
// (Entries from 2^15 instead of 2^20 elements on the AlexNet-shaped gradient, W = 8: the five convolution
// tensors join the three large ones; quantize call 620 against 631 us, server step 137 against 140 us at K = 4.)
constexpr uint64_t kOwnLaunchSegmentElems = 1ull << 20;
constexpr uint64_t kEntrySegmentElems = 1ull << 15;
bool quantize_given_scale_applies(const void* grad, uint64_t n, const uint32_t* codes, uint64_t elem_offset,
                                  uint64_t min_elems = kOwnLaunchSegmentElems);
cudaError_t launch_quantize_given_scale(const void* grad, uint64_t n, int bits, uint64_t seed, uint32_t* codes,
                                        float* scale, int dtype, uint32_t worker, uint32_t step,
                                        uint64_t elem_offset, cudaStream_t stream);

// Per-layer quantization of several workers in three launches (mqg_segments_workers.cu): zero the
// scale arrays, max pass over all (worker, segment) pairs, one encode pass.  A SegEntryHost is one
// (worker, long segment) pair for which quantize_given_scale_applies() holds.
struct SegEntryHost {
    const void* grad;        // the segment's first element
    uint32_t* codes;         // its first code word
    float* scale;            // its scale
    uint64_t n;              // its length
    uint64_t elem_offset;    // flat position of its first element (for the draws)
    uint32_t worker;         // worker id of the draws
};
constexpr int kMaxSegEntriesPerLaunch = 64;
cudaError_t launch_zero_scales(float* const* scales, int W, int nseg, cudaStream_t stream);
cudaError_t launch_absmax_workers(const void* const* grads, float* const* scales, int first, int W,
                                  const SegmentTable& tab, int dtype, cudaStream_t stream);
cudaError_t launch_encode_workers(const SegEntryHost* entries, int nent, const SegmentTable* short_tab,
                                  const void* const* grads, uint32_t* const* codes, float* const* scales,
                                  int scale_first, int W, int bits, uint64_t seed, int dtype,
                                  uint32_t first_worker, uint32_t step, uint64_t elem_offset, cudaStream_t stream);

// Two-pass quantize with uniform large buckets (bucket > kMaxFusedBucket, or a single bucket
// whose length is not a multiple of 32).
cudaError_t launch_quantize_big_buckets(const void* grad, uint64_t n, int bits, uint64_t bucket,
                                        uint64_t seed, uint32_t* codes, float* scales, int dtype,
                                        uint32_t worker, uint32_t step, uint64_t elem_offset,
                                        cudaStream_t stream);

// Server pass over uniform buckets.  params == nullptr: only accumulate (acc required).
// params != nullptr: update params (acc optional output).  add_into only without params.
cudaError_t launch_server(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                          float* params, float lr, float* acc, int add_into, cudaStream_t stream);

// TMA-fed server pass over uniform buckets of >= 32 rows.  mode 1: dst = params, updated with lr;
// mode 0: dst = acc, overwritten with the sum; mode 2: dst = acc, the sum continues from it.
bool server_tma_applies(uint64_t n, uint64_t bucket);          // for any worker count
bool server_tma_applies(uint64_t n, uint64_t bucket, int W);   // also buckets of 32 .. 256 elements for few workers
cudaError_t launch_server_tma(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                              float* dst, float lr, int mode, cudaStream_t stream);

// The fused update of up to kMaxServerSegsPerLaunch long segments of a per-layer step in ONE launch of
// the TMA-fed server kernel (a segment is a gradient with a single bucket).  Every segment must
// satisfy server_tma_segment_applies(n), and params + elem0 and every worker's codes + code_word0
// must be 16-byte aligned.
struct ServerSegHost {
    uint64_t n;              // elements of the segment
    uint64_t elem0;          // offset of its first parameter in `params`
    uint64_t code_word0;     // word offset of its bit stream in every worker's code buffer
    uint32_t scale_idx;      // index of its scale in every worker's scale array
};
constexpr int kMaxServerSegsPerLaunch = 16;
bool server_tma_segment_applies(uint64_t len);
// short_tab (may be null): the table of the step's other segments, updated by the same launch with plain
// loads; short_first = index of the table's first segment in the scale arrays.
cudaError_t launch_server_tma_segments(const WorkerPtrs& ptrs, int W, int bits, const ServerSegHost* segs, int nseg,
                                       const SegmentTable* short_tab, int short_first, float* params, float lr,
                                       cudaStream_t stream);

cudaError_t launch_server_segments(const WorkerPtrs& ptrs, int W, int bits, const SegmentTable& tab,
                                   int scale_base, float* params, float lr, float* acc,
                                   cudaStream_t stream);

// Server downlink: de-quantize + sum + scale to the mean + quantize again (buckets <= 8192).
cudaError_t launch_requantize(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                              float mean_scale, uint64_t seed, uint32_t* codes_out, float* scales_out,
                              uint32_t worker, uint32_t step, cudaStream_t stream);

// The same on the warp-pipelined kernel of mqg_server_tma.cu (whole rows, buckets of 2^k rows up to 128).
bool requantize_warp_applies(uint64_t n, uint64_t bucket, int W);
cudaError_t launch_requantize_warp(const WorkerPtrs& ptrs, int W, int bits, uint64_t n, uint64_t bucket,
                                   float mean_scale, uint64_t seed, uint32_t* codes_out, float* scales_out,
                                   uint32_t worker, uint32_t step, cudaStream_t stream);

cudaError_t launch_apply(float* params, const float* acc, float lr, uint64_t n, cudaStream_t stream);

}  // namespace mqg
