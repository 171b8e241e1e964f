// C ABI of libmqgrad: argument checks, dispatch to the kernel launchers, error reporting.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <utility>
#include <vector>

#include "../../include/mqgrad.h"
#include "mqg_common.cuh"
#include "mqg_internal.h"
#include "mqg_tma.cuh"

namespace {

thread_local char g_err[256] = "";

mqg_status fail(mqg_status code, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

mqg_status cuda_fail(const char* what, cudaError_t err)
{
    return fail(MQG_ERR_CUDA, "%s: %s", what, cudaGetErrorString(err));
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3u) == 0; }
bool aligned8(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 7u) == 0; }

mqg_status check_bits(int bits)
{
    if (bits < 1 || bits > 8) return fail(MQG_ERR_BITS, "bits = %d is outside 1..8", bits);
    return MQG_OK;
}

mqg_status check_bucket(uint64_t n, uint64_t bucket)
{
    if (bucket == 0) return fail(MQG_ERR_INVALID, "bucket must be >= 1");
    if (bucket < n && bucket % 32 != 0)
        return fail(MQG_ERR_INVALID, "bucket = %llu must be a multiple of 32 (or >= n)",
                    (unsigned long long)bucket);
    return MQG_OK;
}

// With `empty` (nothing to process) only W is checked: the buffers may be null.
mqg_status check_workers(const uint32_t* const* codes, const float* const* scales, int W,
                         bool empty, mqg::WorkerPtrs* out)
{
    if (W < 1 || W > MQG_MAX_WORKERS)
        return fail(MQG_ERR_TOO_MANY_WORKERS, "W = %d is outside 1..%d", W, MQG_MAX_WORKERS);
    if (empty) return MQG_OK;
    if (!codes || !scales) return fail(MQG_ERR_INVALID, "codes / scales pointer table is null");
    for (int w = 0; w < W; ++w) {
        if (!codes[w] || !scales[w])
            return fail(MQG_ERR_INVALID, "worker %d: codes or scales buffer is null", w);
        if (!aligned16(codes[w])) return fail(MQG_ERR_ALIGN, "worker %d: codes not 16-byte aligned", w);
        if (!aligned4(scales[w])) return fail(MQG_ERR_ALIGN, "worker %d: scales not 4-byte aligned", w);
        out->codes[w] = codes[w];
        out->scales[w] = scales[w];
    }
    for (int w = W; w < mqg::kMaxWorkers; ++w) { out->codes[w] = nullptr; out->scales[w] = nullptr; }
    return MQG_OK;
}

// Validates a segment table and cuts it into chunks of at most kMaxSegmentsPerLaunch segments;
// calls fn(table, first_segment_index) for each chunk.  Segments for which skip(j) holds get no
// tiles in the tables, exactly like empty segments: another launch takes care of them.  skip is
// only called once the table has been checked.
struct SkipNone { bool operator()(int) const { return false; } };

template <typename Fn, typename Skip = SkipNone>
mqg_status for_each_chunk(int nseg, const uint64_t* seg_off, const uint64_t* code_off, int bits,
                          Fn&& fn, Skip&& skip = Skip())
{
    if (nseg < 0) return fail(MQG_ERR_INVALID, "nseg = %d is negative", nseg);
    if (nseg == 0) return MQG_OK;
    if (!seg_off || !code_off) return fail(MQG_ERR_INVALID, "segment table is null");
    for (int j = 0; j < nseg; ++j) {
        if (seg_off[j + 1] < seg_off[j]) return fail(MQG_ERR_INVALID, "seg_off decreases at %d", j);
        const uint64_t len = seg_off[j + 1] - seg_off[j];
        const uint64_t need = (len * (uint64_t)bits + 31) / 32;
        if (code_off[j + 1] < code_off[j] || code_off[j + 1] - code_off[j] < need)
            return fail(MQG_ERR_INVALID, "code_off leaves segment %d fewer than %llu words", j,
                        (unsigned long long)need);
    }
    const uint64_t tile_elems = (uint64_t)mqg::kMaxTileRows * 32;
    int j = 0;
    while (j < nseg) {
        mqg::SegmentTable tab;
        std::memset(&tab, 0, sizeof(tab));
        int k = 0;
        uint64_t tiles = 0;
        while (j + k < nseg && k < mqg::kMaxSegmentsPerLaunch) {
            const uint64_t len = seg_off[j + k + 1] - seg_off[j + k];
            const uint64_t t = skip(j + k) ? 0 : (len + tile_elems - 1) / tile_elems;
            if (tiles + t > 0x7FFFFFFFull) break;
            tab.tile_start[k] = (uint32_t)tiles;
            tab.seg_off[k] = seg_off[j + k];
            tab.code_off[k] = code_off[j + k];
            tiles += t;
            ++k;
        }
        if (k == 0) return fail(MQG_ERR_INVALID, "segment %d is too large for one launch", j);
        tab.tile_start[k] = (uint32_t)tiles;
        tab.seg_off[k] = seg_off[j + k];
        tab.nseg = k;
        const mqg_status st = fn(tab, j);
        if (st != MQG_OK) return st;
        j += k;
    }
    return MQG_OK;
}

}  // namespace

int mqg::report_error(int code, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

extern "C" {

size_t mqg_code_words(uint64_t n, int bits) { return (size_t)((n * (uint64_t)bits + 31) / 32); }

size_t mqg_num_buckets(uint64_t n, uint64_t bucket)
{
    return bucket ? (size_t)((n + bucket - 1) / bucket) : 0;
}

size_t mqg_wire_bytes(uint64_t n, int bits, uint64_t bucket)
{
    return 4 * mqg_code_words(n, bits) + 4 * mqg_num_buckets(n, bucket);
}

const char* mqg_last_error(void) { return g_err; }

int mqg_version(void) { return 100; }

mqg_status mqg_device_timeouts(unsigned int* count)
{
    if (!count) return fail(MQG_ERR_INVALID, "count is null");
    const cudaError_t err = mqg::read_wait_timeouts(count);
    if (err != cudaSuccess) return cuda_fail("mqg_device_timeouts", err);
    return MQG_OK;
}

mqg_status mqg_check_timeouts(unsigned int* count, int reset)
{
    unsigned int c = 0;
    const cudaError_t err = mqg::read_wait_timeouts(&c, reset != 0);
    if (err != cudaSuccess) return cuda_fail("mqg_check_timeouts", err);
    if (count) *count = c;
    if (c != 0) return fail(MQG_ERR_TIMEOUT, "%u bounded wait(s) of a kernel ran out on this device", c);
    return MQG_OK;
}

mqg_status mqg_test_wait_override(uint32_t poll_limit, int arm_only)
{
    mqg::set_wait_policy(poll_limit, arm_only != 0 ? 1u : 0u);
    return MQG_OK;
}

mqg_status mqg_quantize(const void* grad, uint64_t n, int bits, uint64_t bucket, uint64_t seed,
                        uint32_t* codes, float* scales, mqg_dtype dtype, uint32_t worker,
                        uint32_t step, uint64_t elem_offset, void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (mqg_status st = check_bucket(n, bucket)) return st;
    if (dtype != MQG_F32 && dtype != MQG_BF16) return fail(MQG_ERR_INVALID, "unknown dtype %d", (int)dtype);
    if (n == 0) return MQG_OK;
    if (!grad || !codes || !scales) return fail(MQG_ERR_INVALID, "grad, codes or scales is null");
    if (!aligned16(grad)) return fail(MQG_ERR_ALIGN, "grad not 16-byte aligned");
    if (!aligned16(codes)) return fail(MQG_ERR_ALIGN, "codes not 16-byte aligned");
    if (!aligned4(scales)) return fail(MQG_ERR_ALIGN, "scales not 4-byte aligned");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint64_t eff = bucket < n ? bucket : n;
    cudaError_t err;
    if (eff <= (uint64_t)mqg::kMaxFusedBucket)
        err = mqg::launch_quantize_fused(grad, n, bits, bucket, seed, codes, scales, (int)dtype,
                                         worker, step, elem_offset, stream);
    else
        err = mqg::launch_quantize_big_buckets(grad, n, bits, bucket, seed, codes, scales, (int)dtype,
                                               worker, step, elem_offset, stream);
    if (err != cudaSuccess) return cuda_fail("mqg_quantize", err);
    return MQG_OK;
}

mqg_status mqg_quantize_workers(const void* const* grads, int W, uint64_t n, int bits, uint64_t bucket,
                                uint64_t seed, uint32_t* const* codes, float* const* scales,
                                mqg_dtype dtype, uint32_t first_worker, uint32_t step,
                                uint64_t elem_offset, void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (mqg_status st = check_bucket(n, bucket)) return st;
    if (dtype != MQG_F32 && dtype != MQG_BF16) return fail(MQG_ERR_INVALID, "unknown dtype %d", (int)dtype);
    if (W < 1 || W > MQG_MAX_WORKERS)
        return fail(MQG_ERR_TOO_MANY_WORKERS, "W = %d outside 1..%d", W, MQG_MAX_WORKERS);
    if (n == 0) return MQG_OK;
    if (!grads || !codes || !scales) return fail(MQG_ERR_INVALID, "grads, codes or scales is null");
    for (int w = 0; w < W; ++w) {
        if (!grads[w] || !codes[w] || !scales[w])
            return fail(MQG_ERR_INVALID, "worker %d: grad, codes or scales is null", w);
        if (!aligned16(grads[w])) return fail(MQG_ERR_ALIGN, "worker %d: grad not 16-byte aligned", w);
        if (!aligned16(codes[w])) return fail(MQG_ERR_ALIGN, "worker %d: codes not 16-byte aligned", w);
        if (!aligned4(scales[w])) return fail(MQG_ERR_ALIGN, "worker %d: scales not 4-byte aligned", w);
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (mqg::quantize_workers_applies(W, n, bucket, elem_offset)) {
        const cudaError_t err = mqg::launch_quantize_workers(grads, W, n, bits, bucket, seed, codes, scales,
                                                             (int)dtype, first_worker, step, elem_offset,
                                                             0, stream);
        if (err != cudaSuccess) return cuda_fail("mqg_quantize_workers", err);
        return MQG_OK;
    }
    // shapes the batched kernel does not take: one launch per worker, same results
    for (int w = 0; w < W; ++w) {
        const mqg_status st = mqg_quantize(grads[w], n, bits, bucket, seed, codes[w], scales[w], dtype,
                                           first_worker + (uint32_t)w, step, elem_offset, cuda_stream);
        if (st != MQG_OK) return st;
    }
    return MQG_OK;
}

mqg_status mqg_quantize_minmax(const void* grad, uint64_t n, int bits, uint64_t bucket, uint32_t* codes,
                               float* ranges, mqg_dtype dtype, void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (mqg_status st = check_bucket(n, bucket)) return st;
    if (dtype != MQG_F32 && dtype != MQG_BF16) return fail(MQG_ERR_INVALID, "unknown dtype %d", (int)dtype);
    if (n == 0) return MQG_OK;
    if (!grad || !codes || !ranges) return fail(MQG_ERR_INVALID, "grad, codes or ranges is null");
    if (!aligned16(grad)) return fail(MQG_ERR_ALIGN, "grad not 16-byte aligned");
    if (!aligned16(codes)) return fail(MQG_ERR_ALIGN, "codes not 16-byte aligned");
    if (!aligned8(ranges)) return fail(MQG_ERR_ALIGN, "ranges not 8-byte aligned");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const cudaError_t err = mqg::quantize_range_fused_applies(n, bucket)
        ? mqg::launch_quantize_range_fused(grad, n, bits, bucket, codes, ranges, (int)dtype, stream)
        : mqg::launch_quantize_range_general(grad, n, bits, bucket, codes, ranges, (int)dtype, stream);
    if (err != cudaSuccess) return cuda_fail("mqg_quantize_minmax", err);
    return MQG_OK;
}

mqg_status mqg_quantize_workers_minmax(const void* const* grads, int W, uint64_t n, int bits, uint64_t bucket,
                                       uint32_t* const* codes, float* const* ranges, mqg_dtype dtype,
                                       void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (mqg_status st = check_bucket(n, bucket)) return st;
    if (dtype != MQG_F32 && dtype != MQG_BF16) return fail(MQG_ERR_INVALID, "unknown dtype %d", (int)dtype);
    if (W < 1 || W > MQG_MAX_WORKERS)
        return fail(MQG_ERR_TOO_MANY_WORKERS, "W = %d outside 1..%d", W, MQG_MAX_WORKERS);
    if (n == 0) return MQG_OK;
    if (!grads || !codes || !ranges) return fail(MQG_ERR_INVALID, "grads, codes or ranges is null");
    for (int w = 0; w < W; ++w) {
        if (!grads[w] || !codes[w] || !ranges[w])
            return fail(MQG_ERR_INVALID, "worker %d: grad, codes or ranges is null", w);
        if (!aligned16(grads[w])) return fail(MQG_ERR_ALIGN, "worker %d: grad not 16-byte aligned", w);
        if (!aligned16(codes[w])) return fail(MQG_ERR_ALIGN, "worker %d: codes not 16-byte aligned", w);
        if (!aligned8(ranges[w])) return fail(MQG_ERR_ALIGN, "worker %d: ranges not 8-byte aligned", w);
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (mqg::quantize_workers_applies(W, n, bucket, 0)) {
        const cudaError_t err = mqg::launch_quantize_workers(grads, W, n, bits, bucket, 0, codes, ranges,
                                                             (int)dtype, 0, 0, 0, 1, stream);
        if (err != cudaSuccess) return cuda_fail("mqg_quantize_workers_minmax", err);
        return MQG_OK;
    }
    // shapes the batched kernel does not take: one call per worker, same results
    for (int w = 0; w < W; ++w) {
        const mqg_status st = mqg_quantize_minmax(grads[w], n, bits, bucket, codes[w], ranges[w], dtype, cuda_stream);
        if (st != MQG_OK) return st;
    }
    return MQG_OK;
}

// The variant's worker tables: as check_workers, with the stricter alignment of the range pairs.
static mqg_status check_range_workers(const uint32_t* const* codes, const float* const* ranges, int W,
                                      bool empty, mqg::WorkerPtrs* out)
{
    if (mqg_status st = check_workers(codes, ranges, W, empty, out)) return st;
    if (empty) return MQG_OK;
    for (int w = 0; w < W; ++w)
        if (!aligned8(ranges[w])) return fail(MQG_ERR_ALIGN, "worker %d: ranges not 8-byte aligned", w);
    return MQG_OK;
}

mqg_status mqg_dequant_accumulate_minmax(const uint32_t* const* codes, const float* const* ranges, int W,
                                         int bits, uint64_t n, float* acc, uint64_t bucket,
                                         int add_into_acc, void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (mqg_status st = check_bucket(n, bucket)) return st;
    mqg::WorkerPtrs ptrs;
    if (mqg_status st = check_range_workers(codes, ranges, W, n == 0, &ptrs)) return st;
    if (n == 0) return MQG_OK;
    if (!acc) return fail(MQG_ERR_INVALID, "acc is null");
    if (!aligned16(acc)) return fail(MQG_ERR_ALIGN, "acc not 16-byte aligned");
    const cudaError_t err = mqg::launch_server_range(ptrs, W, bits, n, bucket, nullptr, 0.0f, acc,
                                                     add_into_acc ? 1 : 0,
                                                     static_cast<cudaStream_t>(cuda_stream));
    if (err != cudaSuccess) return cuda_fail("mqg_dequant_accumulate_minmax", err);
    return MQG_OK;
}

mqg_status mqg_server_step_minmax(const uint32_t* const* codes, const float* const* ranges, int W, int bits,
                                  uint64_t n, uint64_t bucket, float* params, float lr, float* acc_out,
                                  void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (mqg_status st = check_bucket(n, bucket)) return st;
    mqg::WorkerPtrs ptrs;
    if (mqg_status st = check_range_workers(codes, ranges, W, n == 0, &ptrs)) return st;
    if (n == 0) return MQG_OK;
    if (!params) return fail(MQG_ERR_INVALID, "params is null");
    if (!aligned16(params)) return fail(MQG_ERR_ALIGN, "params not 16-byte aligned");
    if (acc_out && !aligned16(acc_out)) return fail(MQG_ERR_ALIGN, "acc_out not 16-byte aligned");
    const cudaError_t err = mqg::launch_server_range(ptrs, W, bits, n, bucket, params, lr, acc_out, 0,
                                                     static_cast<cudaStream_t>(cuda_stream));
    if (err != cudaSuccess) return cuda_fail("mqg_server_step_minmax", err);
    return MQG_OK;
}

mqg_status mqg_dequant_accumulate(const uint32_t* const* codes, const float* const* scales, int W,
                                  int bits, uint64_t n, float* acc, uint64_t bucket,
                                  int add_into_acc, void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (mqg_status st = check_bucket(n, bucket)) return st;
    mqg::WorkerPtrs ptrs;
    if (mqg_status st = check_workers(codes, scales, W, n == 0, &ptrs)) return st;
    if (n == 0) return MQG_OK;
    if (!acc) return fail(MQG_ERR_INVALID, "acc is null");
    if (!aligned16(acc)) return fail(MQG_ERR_ALIGN, "acc not 16-byte aligned");
    const cudaError_t err = mqg::launch_server(ptrs, W, bits, n, bucket, nullptr, 0.0f, acc,
                                               add_into_acc ? 1 : 0,
                                               static_cast<cudaStream_t>(cuda_stream));
    if (err != cudaSuccess) return cuda_fail("mqg_dequant_accumulate", err);
    return MQG_OK;
}

mqg_status mqg_apply(float* params, const float* acc, float lr, uint64_t n, void* cuda_stream)
{
    if (n == 0) return MQG_OK;
    if (!params || !acc) return fail(MQG_ERR_INVALID, "params or acc is null");
    if (!aligned16(params) || !aligned16(acc)) return fail(MQG_ERR_ALIGN, "params / acc not 16-byte aligned");
    const cudaError_t err = mqg::launch_apply(params, acc, lr, n, static_cast<cudaStream_t>(cuda_stream));
    if (err != cudaSuccess) return cuda_fail("mqg_apply", err);
    return MQG_OK;
}

mqg_status mqg_server_step(const uint32_t* const* codes, const float* const* scales, int W, int bits,
                           uint64_t n, uint64_t bucket, float* params, float lr, float* acc_out,
                           void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (mqg_status st = check_bucket(n, bucket)) return st;
    mqg::WorkerPtrs ptrs;
    if (mqg_status st = check_workers(codes, scales, W, n == 0, &ptrs)) return st;
    if (n == 0) return MQG_OK;
    if (!params) return fail(MQG_ERR_INVALID, "params is null");
    if (!aligned16(params)) return fail(MQG_ERR_ALIGN, "params not 16-byte aligned");
    if (acc_out && !aligned16(acc_out)) return fail(MQG_ERR_ALIGN, "acc_out not 16-byte aligned");
    const cudaError_t err = mqg::launch_server(ptrs, W, bits, n, bucket, params, lr, acc_out, 0,
                                               static_cast<cudaStream_t>(cuda_stream));
    if (err != cudaSuccess) return cuda_fail("mqg_server_step", err);
    return MQG_OK;
}

mqg_status mqg_server_requantize(const uint32_t* const* codes, const float* const* scales, int W,
                                 int bits, uint64_t n, uint64_t bucket, float mean_scale,
                                 uint64_t seed, uint32_t* codes_out, float* scales_out,
                                 uint32_t worker, uint32_t step, void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (mqg_status st = check_bucket(n, bucket)) return st;
    mqg::WorkerPtrs ptrs;
    if (mqg_status st = check_workers(codes, scales, W, n == 0, &ptrs)) return st;
    if (n == 0) return MQG_OK;
    const uint64_t eff = bucket < n ? bucket : n;
    if (eff > (uint64_t)mqg::kMaxFusedBucket)
        return fail(MQG_ERR_INVALID, "mqg_server_requantize supports buckets of at most %d elements",
                    mqg::kMaxFusedBucket);
    if (!codes_out || !scales_out) return fail(MQG_ERR_INVALID, "codes_out or scales_out is null");
    if (!aligned16(codes_out)) return fail(MQG_ERR_ALIGN, "codes_out not 16-byte aligned");
    if (!aligned4(scales_out)) return fail(MQG_ERR_ALIGN, "scales_out not 4-byte aligned");
    const cudaError_t err = mqg::launch_requantize(ptrs, W, bits, n, bucket, mean_scale, seed, codes_out,
                                                   scales_out, worker, step,
                                                   static_cast<cudaStream_t>(cuda_stream));
    if (err != cudaSuccess) return cuda_fail("mqg_server_requantize", err);
    return MQG_OK;
}

mqg_status mqg_quantize_segments(const void* grad, int nseg, const uint64_t* seg_off,
                                 const uint64_t* code_off, int bits, uint64_t seed,
                                 uint32_t* codes, float* scales, mqg_dtype dtype, uint32_t worker,
                                 uint32_t step, uint64_t elem_offset, void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (dtype != MQG_F32 && dtype != MQG_BF16) return fail(MQG_ERR_INVALID, "unknown dtype %d", (int)dtype);
    if (nseg > 0) {
        if (!grad || !codes || !scales) return fail(MQG_ERR_INVALID, "grad, codes or scales is null");
        if (!aligned16(grad)) return fail(MQG_ERR_ALIGN, "grad not 16-byte aligned");
        if (!aligned16(codes)) return fail(MQG_ERR_ALIGN, "codes not 16-byte aligned");
        if (!aligned4(scales)) return fail(MQG_ERR_ALIGN, "scales not 4-byte aligned");
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // Max pass over every segment; then the encode pass.  A long segment whose buffers are aligned
    // for bulk copies is encoded by the TMA-fed quantize kernel in a launch of its own (its scale is
    // final by then); in the table-driven encode launch it has no tiles.  Same results bit for bit.
    const size_t esz = dtype == MQG_BF16 ? 2 : 4;
    auto own = [&](int j) {
        return mqg::quantize_given_scale_applies(static_cast<const char*>(grad) + seg_off[j] * esz,
                                                 seg_off[j + 1] - seg_off[j], codes + code_off[j],
                                                 elem_offset + seg_off[j]);
    };
    mqg_status st = for_each_chunk(nseg, seg_off, code_off, bits,
        [&](const mqg::SegmentTable& tab, int first) -> mqg_status {
            const cudaError_t err = mqg::launch_segments_absmax(grad, tab, scales + first, (int)dtype, stream);
            if (err != cudaSuccess) return cuda_fail("mqg_quantize_segments", err);
            return MQG_OK;
        });
    if (st != MQG_OK) return st;
    st = for_each_chunk(nseg, seg_off, code_off, bits,
        [&](const mqg::SegmentTable& tab, int first) -> mqg_status {
            const cudaError_t err = mqg::launch_segments_encode(grad, tab, bits, seed, codes, scales + first,
                                                                (int)dtype, worker, step, elem_offset, stream);
            if (err != cudaSuccess) return cuda_fail("mqg_quantize_segments", err);
            return MQG_OK;
        }, own);
    if (st != MQG_OK) return st;
    for (int j = 0; j < nseg; ++j) {
        if (!own(j)) continue;
        const cudaError_t err = mqg::launch_quantize_given_scale(
            static_cast<const char*>(grad) + seg_off[j] * esz, seg_off[j + 1] - seg_off[j], bits, seed,
            codes + code_off[j], scales + j, (int)dtype, worker, step, elem_offset + seg_off[j], stream);
        if (err != cudaSuccess) return cuda_fail("mqg_quantize_segments", err);
    }
    return MQG_OK;
}

mqg_status mqg_quantize_segments_workers(const void* const* grads, int W, int nseg, const uint64_t* seg_off,
                                         const uint64_t* code_off, int bits, uint64_t seed,
                                         uint32_t* const* codes, float* const* scales, mqg_dtype dtype,
                                         uint32_t first_worker, uint32_t step, uint64_t elem_offset,
                                         void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (dtype != MQG_F32 && dtype != MQG_BF16) return fail(MQG_ERR_INVALID, "unknown dtype %d", (int)dtype);
    if (W < 1 || W > MQG_MAX_WORKERS)
        return fail(MQG_ERR_TOO_MANY_WORKERS, "W = %d is outside 1..%d", W, MQG_MAX_WORKERS);
    if (nseg < 0) return fail(MQG_ERR_INVALID, "nseg = %d is negative", nseg);
    if (nseg == 0) return MQG_OK;
    if (!grads || !codes || !scales) return fail(MQG_ERR_INVALID, "grads, codes or scales pointer table is null");
    for (int w = 0; w < W; ++w) {
        if (!grads[w] || !codes[w] || !scales[w])
            return fail(MQG_ERR_INVALID, "worker %d: grad, codes or scales is null", w);
        if (!aligned16(grads[w])) return fail(MQG_ERR_ALIGN, "worker %d: grad not 16-byte aligned", w);
        if (!aligned16(codes[w])) return fail(MQG_ERR_ALIGN, "worker %d: codes not 16-byte aligned", w);
        if (!aligned4(scales[w])) return fail(MQG_ERR_ALIGN, "worker %d: scales not 4-byte aligned", w);
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t esz = dtype == MQG_BF16 ? 2 : 4;
    // a long segment whose buffers are aligned for bulk copies with every worker is an entry of the
    // TMA-fed part of the encode launch; all other segments go through its table-driven part
    auto own = [&](int j) {
        for (int w = 0; w < W; ++w)
            if (!mqg::quantize_given_scale_applies(static_cast<const char*>(grads[w]) + seg_off[j] * esz,
                                                   seg_off[j + 1] - seg_off[j], codes[w] + code_off[j],
                                                   elem_offset + seg_off[j], mqg::kEntrySegmentElems))
                return false;
        return true;
    };
    bool zeroed = false;
    mqg_status st = for_each_chunk(nseg, seg_off, code_off, bits,
        [&](const mqg::SegmentTable& tab, int first) -> mqg_status {
            if (!zeroed) {                 // after the table has been validated
                const cudaError_t err = mqg::launch_zero_scales(scales, W, nseg, stream);
                if (err != cudaSuccess) return cuda_fail("mqg_quantize_segments_workers", err);
                zeroed = true;
            }
            const cudaError_t err = mqg::launch_absmax_workers(grads, scales, first, W, tab, (int)dtype, stream);
            if (err != cudaSuccess) return cuda_fail("mqg_quantize_segments_workers", err);
            return MQG_OK;
        });
    if (st != MQG_OK) return st;

    std::vector<mqg::SegEntryHost> entries;
    for (int j = 0; j < nseg; ++j) {
        if (seg_off[j + 1] == seg_off[j] || !own(j)) continue;
        for (int w = 0; w < W; ++w) {
            mqg::SegEntryHost e;
            e.grad = static_cast<const char*>(grads[w]) + seg_off[j] * esz;
            e.codes = codes[w] + code_off[j];
            e.scale = scales[w] + j;
            e.n = seg_off[j + 1] - seg_off[j];
            e.elem_offset = elem_offset + seg_off[j];
            e.worker = first_worker + (uint32_t)w;
            entries.push_back(e);
        }
    }
    std::vector<std::pair<mqg::SegmentTable, int>> short_tabs;
    st = for_each_chunk(nseg, seg_off, code_off, bits,
        [&](const mqg::SegmentTable& tab, int first) -> mqg_status {
            if (tab.tile_start[tab.nseg] != 0) short_tabs.emplace_back(tab, first);
            return MQG_OK;
        }, own);
    if (st != MQG_OK) return st;
    const size_t per = (size_t)mqg::kMaxSegEntriesPerLaunch;
    const size_t entry_launches = (entries.size() + per - 1) / per;
    const size_t launches = entry_launches > short_tabs.size() ? entry_launches : short_tabs.size();
    for (size_t i = 0; i < launches; ++i) {
        const size_t e0 = i * per;
        const int nent = e0 < entries.size() ? (int)(entries.size() - e0 < per ? entries.size() - e0 : per) : 0;
        const mqg::SegmentTable* tab = i < short_tabs.size() ? &short_tabs[i].first : nullptr;
        const int first = i < short_tabs.size() ? short_tabs[i].second : 0;
        const cudaError_t err = mqg::launch_encode_workers(nent ? entries.data() + e0 : nullptr, nent, tab, grads,
                                                           codes, scales, first, W, bits, seed, (int)dtype,
                                                           first_worker, step, elem_offset, stream);
        if (err != cudaSuccess) return cuda_fail("mqg_quantize_segments_workers", err);
    }
    return MQG_OK;
}

mqg_status mqg_quantize_l2(const void* grad, uint64_t n, int bits, uint64_t bucket, uint64_t seed,
                           uint32_t* codes, float* scales, mqg_dtype dtype, uint32_t worker,
                           uint32_t step, uint64_t elem_offset, void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (mqg_status st = check_bucket(n, bucket)) return st;
    if (dtype != MQG_F32 && dtype != MQG_BF16) return fail(MQG_ERR_INVALID, "unknown dtype %d", (int)dtype);
    if (n == 0) return MQG_OK;
    if ((bucket < n ? bucket : n) > (uint64_t)mqg::kMaxFusedBucket)
        return fail(MQG_ERR_INVALID, "mqg_quantize_l2 supports buckets of at most %d elements; use "
                    "mqg_quantize_segments_l2 for longer ones", mqg::kMaxFusedBucket);
    if (!grad || !codes || !scales) return fail(MQG_ERR_INVALID, "grad, codes or scales is null");
    if (!aligned16(grad)) return fail(MQG_ERR_ALIGN, "grad not 16-byte aligned");
    if (!aligned16(codes)) return fail(MQG_ERR_ALIGN, "codes not 16-byte aligned");
    if (!aligned4(scales)) return fail(MQG_ERR_ALIGN, "scales not 4-byte aligned");
    const cudaError_t err = mqg::launch_quantize_l2(grad, n, bits, bucket, seed, codes, scales, (int)dtype,
                                                    worker, step, elem_offset,
                                                    static_cast<cudaStream_t>(cuda_stream));
    if (err != cudaSuccess) return cuda_fail("mqg_quantize_l2", err);
    return MQG_OK;
}

mqg_status mqg_quantize_workers_l2(const void* const* grads, int W, uint64_t n, int bits, uint64_t bucket,
                                   uint64_t seed, uint32_t* const* codes, float* const* scales,
                                   mqg_dtype dtype, uint32_t first_worker, uint32_t step,
                                   uint64_t elem_offset, void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (mqg_status st = check_bucket(n, bucket)) return st;
    if (dtype != MQG_F32 && dtype != MQG_BF16) return fail(MQG_ERR_INVALID, "unknown dtype %d", (int)dtype);
    if (W < 1 || W > MQG_MAX_WORKERS)
        return fail(MQG_ERR_TOO_MANY_WORKERS, "W = %d outside 1..%d", W, MQG_MAX_WORKERS);
    if (n == 0) return MQG_OK;
    if ((bucket < n ? bucket : n) > (uint64_t)mqg::kMaxFusedBucket)
        return fail(MQG_ERR_INVALID, "mqg_quantize_workers_l2 supports buckets of at most %d elements; use "
                    "mqg_quantize_segments_l2 for longer ones", mqg::kMaxFusedBucket);
    if (!grads || !codes || !scales) return fail(MQG_ERR_INVALID, "grads, codes or scales is null");
    for (int w = 0; w < W; ++w) {
        if (!grads[w] || !codes[w] || !scales[w])
            return fail(MQG_ERR_INVALID, "worker %d: grad, codes or scales is null", w);
        if (!aligned16(grads[w])) return fail(MQG_ERR_ALIGN, "worker %d: grad not 16-byte aligned", w);
        if (!aligned16(codes[w])) return fail(MQG_ERR_ALIGN, "worker %d: codes not 16-byte aligned", w);
        if (!aligned4(scales[w])) return fail(MQG_ERR_ALIGN, "worker %d: scales not 4-byte aligned", w);
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (mqg::quantize_workers_applies(W, n, bucket, elem_offset)) {
        const cudaError_t err = mqg::launch_quantize_workers(grads, W, n, bits, bucket, seed, codes, scales,
                                                             (int)dtype, first_worker, step, elem_offset,
                                                             2, stream);
        if (err != cudaSuccess) return cuda_fail("mqg_quantize_workers_l2", err);
        return MQG_OK;
    }
    // shapes the batched kernel does not take: one launch per worker, same results
    for (int w = 0; w < W; ++w) {
        const mqg_status st = mqg_quantize_l2(grads[w], n, bits, bucket, seed, codes[w], scales[w], dtype,
                                              first_worker + (uint32_t)w, step, elem_offset, cuda_stream);
        if (st != MQG_OK) return st;
    }
    return MQG_OK;
}

mqg_status mqg_quantize_1bit_ef(const void* grad, float* residual, uint64_t n, uint64_t bucket,
                                uint32_t* codes, float* ranges, mqg_dtype dtype, void* cuda_stream)
{
    if (mqg_status st = check_bucket(n, bucket)) return st;
    if (dtype != MQG_F32 && dtype != MQG_BF16) return fail(MQG_ERR_INVALID, "unknown dtype %d", (int)dtype);
    if (n == 0) return MQG_OK;
    if ((bucket < n ? bucket : n) > (uint64_t)mqg::kMaxFusedBucket)
        return fail(MQG_ERR_INVALID, "mqg_quantize_1bit_ef supports buckets of at most %d elements",
                    mqg::kMaxFusedBucket);
    if (!grad || !residual || !codes || !ranges)
        return fail(MQG_ERR_INVALID, "grad, residual, codes or ranges is null");
    if (!aligned16(grad)) return fail(MQG_ERR_ALIGN, "grad not 16-byte aligned");
    if (!aligned16(residual)) return fail(MQG_ERR_ALIGN, "residual not 16-byte aligned");
    if (!aligned16(codes)) return fail(MQG_ERR_ALIGN, "codes not 16-byte aligned");
    if (!aligned8(ranges)) return fail(MQG_ERR_ALIGN, "ranges not 8-byte aligned");
    const cudaError_t err = mqg::launch_quantize_onebit_ef(grad, residual, n, bucket, codes, ranges, (int)dtype,
                                                           static_cast<cudaStream_t>(cuda_stream));
    if (err != cudaSuccess) return cuda_fail("mqg_quantize_1bit_ef", err);
    return MQG_OK;
}

size_t mqg_l2_workspace_floats(int nseg, const uint64_t* seg_off)
{
    if (nseg <= 0 || !seg_off) return 0;
    const uint64_t tile_elems = (uint64_t)mqg::kMaxTileRows * 32;
    uint64_t tiles = 0;
    for (int j = 0; j < nseg; ++j)
        if (seg_off[j + 1] > seg_off[j]) tiles += (seg_off[j + 1] - seg_off[j] + tile_elems - 1) / tile_elems;
    return (size_t)tiles;
}

mqg_status mqg_quantize_segments_l2(const void* grad, int nseg, const uint64_t* seg_off,
                                    const uint64_t* code_off, int bits, uint64_t seed,
                                    uint32_t* codes, float* scales, mqg_dtype dtype, uint32_t worker,
                                    uint32_t step, uint64_t elem_offset, float* workspace,
                                    size_t workspace_floats, void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    if (dtype != MQG_F32 && dtype != MQG_BF16) return fail(MQG_ERR_INVALID, "unknown dtype %d", (int)dtype);
    if (nseg > 0) {
        if (!grad || !codes || !scales) return fail(MQG_ERR_INVALID, "grad, codes or scales is null");
        if (!aligned16(grad)) return fail(MQG_ERR_ALIGN, "grad not 16-byte aligned");
        if (!aligned16(codes)) return fail(MQG_ERR_ALIGN, "codes not 16-byte aligned");
        if (!aligned4(scales)) return fail(MQG_ERR_ALIGN, "scales not 4-byte aligned");
        if (!seg_off || !code_off) return fail(MQG_ERR_INVALID, "segment table is null");
        const size_t need = mqg_l2_workspace_floats(nseg, seg_off);
        if (need > workspace_floats)
            return fail(MQG_ERR_INVALID, "workspace holds %llu floats, %llu needed (mqg_l2_workspace_floats)",
                        (unsigned long long)workspace_floats, (unsigned long long)need);
        if (need != 0 && !workspace) return fail(MQG_ERR_INVALID, "workspace is null");
        if (!aligned4(workspace)) return fail(MQG_ERR_ALIGN, "workspace not 4-byte aligned");
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // Sums and scales of every segment first; then the encode, where a long segment with buffers
    // aligned for bulk copies takes a launch of the TMA-fed quantize kernel of its own.
    const size_t esz = dtype == MQG_BF16 ? 2 : 4;
    auto own = [&](int j) {
        return mqg::quantize_given_scale_applies(static_cast<const char*>(grad) + seg_off[j] * esz,
                                                 seg_off[j + 1] - seg_off[j], codes + code_off[j],
                                                 elem_offset + seg_off[j]);
    };
    size_t used = 0;                      // tiles of the chunks already launched
    mqg_status st = for_each_chunk(nseg, seg_off, code_off, bits,
        [&](const mqg::SegmentTable& tab, int first) -> mqg_status {
            const cudaError_t err = mqg::launch_segments_l2_scales(grad, tab, scales + first, (int)dtype,
                                                                   workspace + used, stream);
            if (err != cudaSuccess) return cuda_fail("mqg_quantize_segments_l2", err);
            used += tab.tile_start[tab.nseg];
            return MQG_OK;
        });
    if (st != MQG_OK) return st;
    st = for_each_chunk(nseg, seg_off, code_off, bits,
        [&](const mqg::SegmentTable& tab, int first) -> mqg_status {
            const cudaError_t err = mqg::launch_segments_encode(grad, tab, bits, seed, codes, scales + first,
                                                                (int)dtype, worker, step, elem_offset, stream);
            if (err != cudaSuccess) return cuda_fail("mqg_quantize_segments_l2", err);
            return MQG_OK;
        }, own);
    if (st != MQG_OK) return st;
    for (int j = 0; j < nseg; ++j) {
        if (!own(j)) continue;
        const cudaError_t err = mqg::launch_quantize_given_scale(
            static_cast<const char*>(grad) + seg_off[j] * esz, seg_off[j + 1] - seg_off[j], bits, seed,
            codes + code_off[j], scales + j, (int)dtype, worker, step, elem_offset + seg_off[j], stream);
        if (err != cudaSuccess) return cuda_fail("mqg_quantize_segments_l2", err);
    }
    return MQG_OK;
}

mqg_status mqg_server_step_segments(const uint32_t* const* codes, const float* const* scales, int W,
                                    int bits, int nseg, const uint64_t* seg_off,
                                    const uint64_t* code_off, float* params, float lr,
                                    float* acc_out, void* cuda_stream)
{
    if (mqg_status st = check_bits(bits)) return st;
    mqg::WorkerPtrs ptrs;
    if (mqg_status st = check_workers(codes, scales, W, nseg <= 0, &ptrs)) return st;
    if (nseg > 0) {
        if (!params) return fail(MQG_ERR_INVALID, "params is null");
        if (!aligned16(params)) return fail(MQG_ERR_ALIGN, "params not 16-byte aligned");
        if (acc_out && !aligned16(acc_out)) return fail(MQG_ERR_ALIGN, "acc_out not 16-byte aligned");
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // A long segment is a gradient with a single bucket: the long segments whose buffers are aligned for
    // bulk copies go to the TMA-fed server kernel together, in one launch; all other segments share
    // the table-driven launch.  The results are the same bit for bit either way.
    constexpr uint64_t kOwnLaunchElems = mqg::kEntrySegmentElems;
    auto own = [&](int j) {
        const uint64_t len = seg_off[j + 1] - seg_off[j];
        if (acc_out || len < kOwnLaunchElems || !mqg::server_tma_applies(len, len)) return false;
        bool aligned = aligned16(params + seg_off[j]);
        for (int w = 0; w < W && aligned; ++w) aligned = aligned16(codes[w] + code_off[j]);
        return aligned;
    };
    // the long segments first (they decide how the short ones are handled)
    std::vector<mqg::ServerSegHost> longs;
    for (int j = 0; nseg > 0 && seg_off && code_off && j < nseg; ++j) {
        if (seg_off[j + 1] < seg_off[j]) break;          // a bad table: for_each_chunk below reports it
        if (!own(j)) continue;
        mqg::ServerSegHost h;
        h.n = seg_off[j + 1] - seg_off[j];
        h.elem0 = seg_off[j];
        h.code_word0 = code_off[j];
        h.scale_idx = (uint32_t)j;
        longs.push_back(h);
    }
    // The other segments: table-driven launches - except that ONE table of short segments rides along
    // with the (first) launch of the long ones, so that a typical layered step is a single launch.
    std::vector<std::pair<mqg::SegmentTable, int>> short_tabs;
    const mqg_status st = for_each_chunk(nseg, seg_off, code_off, bits,
        [&](const mqg::SegmentTable& tab, int first) -> mqg_status {
            if (tab.tile_start[tab.nseg] != 0) short_tabs.emplace_back(tab, first);
            return MQG_OK;
        }, own);
    if (st != MQG_OK) return st;
    const bool fold = !longs.empty() && !short_tabs.empty();
    for (size_t i = fold ? 1 : 0; i < short_tabs.size(); ++i) {
        const cudaError_t err = mqg::launch_server_segments(ptrs, W, bits, short_tabs[i].first, short_tabs[i].second,
                                                            params, lr, acc_out, stream);
        if (err != cudaSuccess) return cuda_fail("mqg_server_step_segments", err);
    }
    for (size_t i = 0; i < longs.size(); i += (size_t)mqg::kMaxServerSegsPerLaunch) {
        const size_t cnt = longs.size() - i < (size_t)mqg::kMaxServerSegsPerLaunch ? longs.size() - i
                                                                                   : (size_t)mqg::kMaxServerSegsPerLaunch;
        const bool with_short = fold && i == 0;
        const cudaError_t err = mqg::launch_server_tma_segments(
            ptrs, W, bits, longs.data() + i, (int)cnt, with_short ? &short_tabs[0].first : nullptr,
            with_short ? short_tabs[0].second : 0, params, lr, stream);
        if (err != cudaSuccess) return cuda_fail("mqg_server_step_segments", err);
    }
    return MQG_OK;
}

}  // extern "C"
