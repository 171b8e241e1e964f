/*
 * mqgrad.h -- C ABI of libmqgrad: the per-iteration gradient codec of MQGrad
 * (arXiv 1804.08066) for one NVIDIA B200 (sm_100a).
 *
 * The paper's data path per training iteration (Algorithm 1, Section 3.2):
 *   worker:  g~ <- Quantize(g, K)                         (WorkerIterate)
 *   server:  g_p <- De-quantize(g~_p) for p = 1..P,
 *            g <- sum_p g_p / P,  w <- w - eta * g        (ReceiveQGThenSendQG, steps 6-7 of Fig. 3)
 * The paper leaves the codec itself to an external page; this library fixes it as:
 * a symmetric K-bit affine grid on [-s, +s] per bucket (s = max |x| of the bucket),
 * unbiased stochastic rounding with 16 random bits per element from Philox4x32-10,
 * and LSB-first packing of the K-bit codes into little-endian 32-bit words.
 *
 * Conventions that hold for every call
 *   - Every data pointer is caller-owned DEVICE memory unless stated otherwise; the
 *     library never allocates, frees or keeps device memory.  Arrays of pointers
 *     (codes[W], scales[W]) and segment tables are HOST arrays, read during the call.
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL = the
 *     default stream) and return without waiting for it.
 *   - Return value: MQG_OK, or a negative mqg_status; nothing is thrown and nothing
 *     aborts.  Arguments are checked on the host before any launch; on an error
 *     nothing has been enqueued.  mqg_last_error() gives the calling thread's message.
 *   - n == 0 is a valid no-op.  Inputs must be finite; results for NaN/Inf are unspecified.
 *   - Output buffers must not overlap inputs, except `params`, updated in place.
 *   - grad, params, acc and codes must be 16-byte aligned; scales 4-byte aligned.
 *   - 1 <= bits <= 8.  L = 2^bits - 1.
 *   - bucket >= 1, and bucket % 32 == 0 unless bucket >= n (one bucket), so that every
 *     bucket's codes start on a word boundary for every bit width.
 */
#ifndef MQGRAD_H_
#define MQGRAD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int mqg_status;
enum {
    MQG_OK = 0,
    MQG_ERR_INVALID = -1,          /* null pointer, bad bucket, bad segment table, overlapping sizes */
    MQG_ERR_BITS = -2,             /* bits outside 1..8 */
    MQG_ERR_ALIGN = -3,            /* a buffer is not aligned as required */
    MQG_ERR_TOO_MANY_WORKERS = -4, /* W outside 1..MQG_MAX_WORKERS */
    MQG_ERR_CUDA = -5,             /* a CUDA runtime call failed; see mqg_last_error() */
    MQG_ERR_TIMEOUT = -6           /* a kernel's bounded wait ran out (mqg_check_timeouts) */
};

typedef enum { MQG_F32 = 0, MQG_BF16 = 1 } mqg_dtype;

#define MQG_MAX_WORKERS 32

/* Number of 32-bit words of one worker's packed stream: ceil(n * bits / 32).  Host-only helper. */
size_t mqg_code_words(uint64_t n, int bits);

/* Number of buckets (= scales) for n elements: ceil(n / bucket).  Host-only helper. */
size_t mqg_num_buckets(uint64_t n, uint64_t bucket);

/* Bytes one worker sends for n elements: 4 * code_words + 4 * num_buckets (reported, never timed). */
size_t mqg_wire_bytes(uint64_t n, int bits, uint64_t bucket);

/*
 * Quantize(g, K) of Algorithm 1 (WorkerIterate), fused with packing.
 *   grad        [in]  n elements of `dtype` (fp32, or bf16 widened exactly to fp32 in the kernel)
 *   codes       [out] mqg_code_words(n, bits) words; code i at bits [i*bits, i*bits+bits) of the
 *                     stream, bit j of the stream = bit (j % 32) of word j / 32; pad bits are zero
 *   scales      [out] mqg_num_buckets(n, bucket) floats; s_k = max |x| of bucket k, flushed to 0
 *                     below 2^-96 (then every code of the bucket is 0)
 *   seed, worker, step, elem_offset
 *                     key the random draws: element i draws from Philox4x32-10 with key = seed and
 *                     counter = ((elem_offset + i) / 8, worker, step), 16 bits per element, so the
 *                     codes are a pure function of the arguments (reproducible, order-free).
 *                     elem_offset is the element's position in the flat model; multiples of 8
 *                     take the fast path.
 * Per element: t = fma(x, L / (2 s), L / 2) in fp32, code = floor(t) + [u < t - floor(t)],
 * u = (h + 1/2) / 65536.
 */
mqg_status mqg_quantize(const void* grad, uint64_t n, int bits, uint64_t bucket, uint64_t seed,
                        uint32_t* codes, float* scales,
                        mqg_dtype dtype, uint32_t worker, uint32_t step, uint64_t elem_offset,
                        void* cuda_stream);

/*
 * Quantize(g_p, K) of Algorithm 1 for W workers whose gradients live on this device (P workers
 * simulated on one GPU, or several replicas per device), in one launch where the shape allows:
 * exactly mqg_quantize(grads[w], ..., codes[w], scales[w], worker = first_worker + w, ...) for
 * w = 0..W-1, bit for bit, without paying the per-launch fixed cost W times.
 *   grads, codes, scales  HOST arrays of W device pointers (read during the call only); each
 *                         buffer as in mqg_quantize; the outputs are what mqg_server_step and
 *                         mqg_dequant_accumulate take as codes[] / scales[]
 * Shapes outside the one-launch kernel (buckets above 4096 elements, fewer than 2048 elements,
 * elem_offset not a multiple of 8, W = 1) run as W launches inside the call.
 * Errors: as mqg_quantize, per worker; MQG_ERR_TOO_MANY_WORKERS for W outside 1..MQG_MAX_WORKERS.
 */
mqg_status mqg_quantize_workers(const void* const* grads, int W, uint64_t n, int bits, uint64_t bucket,
                                uint64_t seed, uint32_t* const* codes, float* const* scales,
                                mqg_dtype dtype, uint32_t first_worker, uint32_t step,
                                uint64_t elem_offset, void* cuda_stream);

/*
 * De-quantize + sum of Algorithm 1 (ReceiveQGThenSendQG, before the division by P):
 *   acc[i] = ((x^_0[i] + x^_1[i]) + ... ) in worker order 0..W-1, fp32,
 *   x^_w[i] = (2 q - L) * (s / L) with one rounding for s / L and one for the product;
 *   a zero-scale bucket decodes to +0.
 *   codes, scales  [in]  HOST arrays of W device pointers, laid out as mqg_quantize writes them
 *   acc            [out] n floats; overwritten, or (add_into_acc != 0) the sum continues from the
 *                        value already there: acc = ((acc + x^_0) + x^_1) + ...
 */
mqg_status mqg_dequant_accumulate(const uint32_t* const* codes, const float* const* scales, int W,
                                  int bits, uint64_t n, float* acc,
                                  uint64_t bucket, int add_into_acc, void* cuda_stream);

/*
 * w <- w - eta * g of Algorithm 1 (WorkerIterate's update), one fused multiply-add per element:
 * params[i] = fma(-lr, acc[i], params[i]).  Pass lr = eta / P to apply the mean of P workers.
 */
mqg_status mqg_apply(float* params, const float* acc, float lr, uint64_t n, void* cuda_stream);

/*
 * The server's whole step in one pass over memory (steps 6-7 of Fig. 3, Section 3.2): unpack,
 * de-quantize and sum W workers' buffers and update the shared parameters, with exactly the
 * roundings of mqg_dequant_accumulate followed by mqg_apply.
 *   params   [in/out] n floats, updated in place
 *   acc_out  [out]    optional (may be NULL): the summed gradient, n floats
 */
mqg_status mqg_server_step(const uint32_t* const* codes, const float* const* scales, int W, int bits,
                           uint64_t n, uint64_t bucket, float* params, float lr, float* acc_out,
                           void* cuda_stream);

/*
 * The server's downlink (ReceiveQGThenSendQG of Algorithm 1, lines 3-5; steps 6-8 of Fig. 3): the
 * global gradient g = (sum_p g_p) * mean_scale, with the sum as in mqg_dequant_accumulate and one
 * rounding for the product (pass mean_scale = 1 / P for the paper's mean), is quantized again with
 * the same bit width and bucket, exactly as mqg_quantize(g, ...) with elem_offset 0 would, without
 * storing g.  Workers then apply it with mqg_server_step(W = 1, lr = eta).
 *   codes_out, scales_out [out] laid out as mqg_quantize writes them
 *   worker, step               key the random draws of this encode (use an id no worker uses)
 * Buckets (or a single bucket n) above 8192 elements are rejected with MQG_ERR_INVALID.
 */
mqg_status mqg_server_requantize(const uint32_t* const* codes, const float* const* scales, int W,
                                 int bits, uint64_t n, uint64_t bucket, float mean_scale,
                                 uint64_t seed, uint32_t* codes_out, float* scales_out,
                                 uint32_t worker, uint32_t step, void* cuda_stream);

/*
 * Codec variant: the (min, max) range scheme the footnote of Section 3.2 refers to, with nearest
 * rounding and no random draws.  Per bucket lo = min x, hi = max x (a zero of either sign stored
 * as +0), r = fl(hi - lo), L = 2^bits - 1:
 *     code = min(L, floor(fma(fl(x - lo), fl(L / r), 1/2)))      x^ = fma(code, fl(r / L), lo)
 * a bucket with r < 2^-96 is constant: every code is 0 and every x^ is lo.
 *   ranges  [out] 2 * mqg_num_buckets(n, bucket) floats, 8-byte aligned: ranges[2b] = lo,
 *                 ranges[2b + 1] = hi of bucket b
 *   codes   [out] as mqg_quantize
 * Buckets of at most 4096 elements take one pass over the gradient; larger ones two.
 * Errors as mqg_quantize; MQG_ERR_ALIGN for a ranges pointer that is not 8-byte aligned.
 */
mqg_status mqg_quantize_minmax(const void* grad, uint64_t n, int bits, uint64_t bucket, uint32_t* codes,
                               float* ranges, mqg_dtype dtype, void* cuda_stream);
/*
 * The (min, max) variant for W workers' gradients of the same shape in ONE launch (the variant's
 * counterpart of mqg_quantize_workers; the scheme the footnote of Section 3.2 points to): worker w's
 * outputs are bit-identical to mqg_quantize_minmax on its gradient.
 *   grads / codes / ranges   HOST arrays of W DEVICE pointers, each as in mqg_quantize_minmax; caller-owned
 * Shapes the batched kernel does not take run as W calls with the same results.
 * Errors as mqg_quantize_minmax, plus MQG_ERR_TOO_MANY_WORKERS for W outside 1..MQG_MAX_WORKERS.
 */
mqg_status mqg_quantize_workers_minmax(const void* const* grads, int W, uint64_t n, int bits, uint64_t bucket,
                                       uint32_t* const* codes, float* const* ranges, mqg_dtype dtype,
                                       void* cuda_stream);


/*
 * Server side of the variant: mqg_dequant_accumulate and mqg_server_step with x^ as above and the
 * same ordered sum and fused update.  `ranges` is a HOST array of W device pointers, each laid out
 * as mqg_quantize_minmax writes it.
 */
mqg_status mqg_dequant_accumulate_minmax(const uint32_t* const* codes, const float* const* ranges, int W,
                                         int bits, uint64_t n, float* acc, uint64_t bucket,
                                         int add_into_acc, void* cuda_stream);
mqg_status mqg_server_step_minmax(const uint32_t* const* codes, const float* const* ranges, int W, int bits,
                                  uint64_t n, uint64_t bucket, float* params, float lr, float* acc_out,
                                  void* cuda_stream);

/*
 * Codec variant: one bit per element with error feedback, the 1-bit scheme that the related-work
 * section (Section 2) cites: the sign of every value is sent and the quantization error is carried
 * into the next mini-batch.  With e the worker's residual (n floats kept by the caller from one
 * iteration to the next, zero before the first):
 *     v = fl(g + e);   code = 1 if v >= 0 (a zero of either sign included) else 0
 *     per bucket: neg = mean of v over the elements with code 0, pos = mean over those with code 1
 *                 (0 for an empty class), written as ranges[2b] = neg, ranges[2b + 1] = pos
 *     x^ = what mqg_server_step_minmax / mqg_dequant_accumulate_minmax with bits = 1 reconstruct from
 *          (code, neg, pos): neg for code 0, fl(fl(pos - neg) + neg) for code 1; a bucket with
 *          fl(pos - neg) < 2^-96 is constant (codes cleared, x^ = neg)
 *     e <- fl(v - x^)
 * The class sums are taken in a fixed order (inside a row of 32 elements from the bucket's start a
 * left-to-right chain over the class's members; the rows' sums by a balanced tree of adjacent
 * pairs, leaf count padded with zeros to a power of two), so the result is reproducible bit for bit.
 *   residual [in/out] n floats, 16-byte aligned, updated in place
 *   codes    [out]    mqg_code_words(n, 1) words;  ranges [out] 2 * mqg_num_buckets(n, bucket) floats,
 *                     8-byte aligned.  The server side is the (min, max) variant's with bits = 1.
 * Buckets (or a single bucket n) above 8192 elements are rejected with MQG_ERR_INVALID.
 */
mqg_status mqg_quantize_1bit_ef(const void* grad, float* residual, uint64_t n, uint64_t bucket,
                                uint32_t* codes, float* ranges, mqg_dtype dtype, void* cuda_stream);

/*
 * Codec variant: the bucket's scale is its Euclidean norm, as in the norm-scaled quantizers the
 * related-work section (Section 2) cites, instead of its largest magnitude.  Everything else is
 * mqg_quantize: same encode against [-s, +s], same draws, same packing, and the outputs are
 * consumed by the ordinary server calls (mqg_server_step, mqg_dequant_accumulate,
 * mqg_server_requantize).  Because a float sum depends on its order, the order is fixed:
 *   - the bucket is cut into rows of 32 consecutive elements from its first element; a row's sum
 *     of squares is the chain a <- fma(x_j, x_j, a), left to right, from a = 0;
 *   - the row sums are combined by a balanced binary tree of adjacent pairs (leaf count padded
 *     with zeros to a power of two); S is the root;
 *   - scales[k] = 0 if S < 2^-96 (every code of the bucket is then 0), else sqrt(S) rounded once.
 * The result is therefore reproducible bit for bit, on any device and launch shape.  Inputs whose
 * sum of squares overflows fp32 give unspecified results.
 * Buckets (or a single bucket n) above 8192 elements are rejected with MQG_ERR_INVALID: use the
 * segment form below for those.  Other arguments and errors as mqg_quantize.
 */
mqg_status mqg_quantize_l2(const void* grad, uint64_t n, int bits, uint64_t bucket, uint64_t seed,
                           uint32_t* codes, float* scales, mqg_dtype dtype, uint32_t worker,
                           uint32_t step, uint64_t elem_offset, void* cuda_stream);

/*
 * The L2-norm variant for W workers' gradients of the same shape in ONE launch (the variant's
 * counterpart of mqg_quantize_workers; related-work codec of Section 2, granularity as Section 4.1):
 * worker w's outputs are bit-identical to mqg_quantize_l2 with worker id first_worker + w.
 *   grads / codes / scales   HOST arrays of W DEVICE pointers, each as in mqg_quantize_l2; caller-owned
 * Shapes the batched kernel does not take run as W launches with the same results.
 * Errors as mqg_quantize_l2, plus MQG_ERR_TOO_MANY_WORKERS for W outside 1..MQG_MAX_WORKERS.
 */
mqg_status mqg_quantize_workers_l2(const void* const* grads, int W, uint64_t n, int bits, uint64_t bucket,
                                   uint64_t seed, uint32_t* const* codes, float* const* scales,
                                   mqg_dtype dtype, uint32_t first_worker, uint32_t step,
                                   uint64_t elem_offset, void* cuda_stream);

/*
 * The same variant with one norm per segment (per-layer scale), segment tables as in
 * mqg_quantize_segments below; the outputs go to mqg_server_step_segments.  The rows and the
 * tree of a segment start at the segment's first element.
 *   workspace        [scratch] DEVICE memory for the partial sums: at least
 *                    mqg_l2_workspace_floats(nseg, seg_off) floats (one per 8192 elements of every
 *                    segment, rounded up per segment), 4-byte aligned.  Contents on entry do not
 *                    matter and are undefined on return; calls that may run concurrently on the
 *                    device need separate workspaces.
 *   workspace_floats its size in floats; MQG_ERR_INVALID when too small.
 * The gradient is read twice (sum pass, encode pass).
 */
size_t mqg_l2_workspace_floats(int nseg, const uint64_t* seg_off);
mqg_status mqg_quantize_segments_l2(const void* grad, int nseg, const uint64_t* seg_off,
                                    const uint64_t* code_off, int bits, uint64_t seed,
                                    uint32_t* codes, float* scales, mqg_dtype dtype, uint32_t worker,
                                    uint32_t step, uint64_t elem_offset, float* workspace,
                                    size_t workspace_floats, void* cuda_stream);

/*
 * mqg_quantize_segments_l2 without the workspace argument, for callers that cannot supply device
 * memory of their own: processes whose device memory has all been handed to one pool at start-up
 * (a later allocation fails), latency-critical paths that must not run into the device-wide
 * synchronisation of an allocation, and plug-ins or callbacks whose host only lets them launch
 * work on the buffers they are given.  (The paper has no counterpart: this is a property of the
 * library's interface, not of the method.)  The partial sums go to an array inside the library
 * image instead; arguments, results and errors are otherwise exactly those of
 * mqg_quantize_segments_l2.
 *   - Limit: mqg_l2_workspace_floats(nseg, seg_off) <= MQG_L2_STATIC_WORKSPACE_FLOATS (65,536 partial
 *     sums, one per started 8192 elements of every segment: about 5 * 10^8 elements); beyond it the
 *     call returns MQG_ERR_INVALID, enqueues nothing, and mqg_last_error() names both numbers.
 *   - Cost: the array (256 KiB) occupies device memory on every GPU that loads the library, from
 *     load until the process exits, also if this function is never called.
 *   - The call allocates and frees nothing, on the host or the device.  The first call on each
 *     device looks up the array's device address (once; later calls reuse it); make that first
 *     call before any stream capture begins.
 *   - All calls on a device share the one array, and it keeps what the last call left in it.
 *     Nothing in it needs to be zero on entry (every element read is written earlier in the same
 *     call), but two calls whose kernels can overlap on the device - different streams, or
 *     different host threads on different streams - race on it and corrupt each other's scales:
 *     order them on one stream or with events.
 */
#define MQG_L2_STATIC_WORKSPACE_FLOATS 65536
mqg_status mqg_quantize_segments_l2_static(const void* grad, int nseg, const uint64_t* seg_off,
                                           const uint64_t* code_off, int bits, uint64_t seed,
                                           uint32_t* codes, float* scales, mqg_dtype dtype,
                                           uint32_t worker, uint32_t step, uint64_t elem_offset,
                                           void* cuda_stream);

/*
 * Per-layer scale (Section 4.1 quantizes the two large fully connected layers, each as a whole): the flat
 * gradient is cut into nseg segments; segment j = elements [seg_off[j], seg_off[j+1]) is ONE bucket
 * with scale scales[j], and its bit stream starts on a word boundary at word code_off[j].
 *   seg_off   [in] HOST array of nseg+1 non-decreasing element offsets (seg_off[0] may be > 0)
 *   code_off  [in] HOST array of nseg+1 word offsets; code_off[j+1] - code_off[j] >=
 *                  mqg_code_words(seg_off[j+1] - seg_off[j], bits)
 *   grad      [in] the whole flat gradient (element 0 of the array is flat index 0)
 *   codes     [out] code_off[nseg] words;  scales [out] nseg floats
 * Element i of segment j draws with position elem_offset + seg_off[j] + i.  Empty segments get
 * scale 0.  The gradient is read twice (max pass, encode pass).
 * Performance note: a segment of 2^20 elements or more (2^15 or more in mqg_quantize_segments_workers
 * and mqg_server_step_segments, where such segments share a launch) is encoded (and, in
 * mqg_server_step_segments, applied) by the bulk-copy kernels when grad + seg_off[j], codes + code_off[j] (every worker's, on
 * the server) and params + seg_off[j] are 16-byte aligned and elem_offset + seg_off[j] is a multiple
 * of 8; otherwise by the table-driven kernels.  The results do not depend on which kernel ran.
 */
mqg_status mqg_quantize_segments(const void* grad, int nseg, const uint64_t* seg_off,
                                 const uint64_t* code_off, int bits, uint64_t seed,
                                 uint32_t* codes, float* scales, mqg_dtype dtype, uint32_t worker,
                                 uint32_t step, uint64_t elem_offset, void* cuda_stream);

/*
 * mqg_quantize_segments for W workers' gradients that share one segment table, in three launches for
 * all of them (zero the scales, max pass, encode pass) instead of five per worker - the per-layer
 * counterpart of mqg_quantize_workers, for a host that plays several workers on one device (all
 * workers run Quantize(g, K) with the same K in an iteration; Algorithm 1, WorkerIterate line 3).
 *   grads/codes/scales [in] HOST arrays of W device pointers; worker w draws with worker id
 *                      first_worker + w; codes[w] takes code_off[nseg] words, scales[w] nseg floats
 * Worker w's outputs are bit-identical to mqg_quantize_segments(grads[w], ..., first_worker + w, ...).
 * Errors as mqg_quantize_segments, per worker; MQG_ERR_TOO_MANY_WORKERS for W outside
 * 1..MQG_MAX_WORKERS.
 */
mqg_status mqg_quantize_segments_workers(const void* const* grads, int W, int nseg, const uint64_t* seg_off,
                                         const uint64_t* code_off, int bits, uint64_t seed,
                                         uint32_t* const* codes, float* const* scales, mqg_dtype dtype,
                                         uint32_t first_worker, uint32_t step, uint64_t elem_offset,
                                         void* cuda_stream);

/* mqg_server_step for buffers written by mqg_quantize_segments (same segment tables). */
mqg_status mqg_server_step_segments(const uint32_t* const* codes, const float* const* scales, int W,
                                    int bits, int nseg, const uint64_t* seg_off,
                                    const uint64_t* code_off, float* params, float lr,
                                    float* acc_out, void* cuda_stream);

/*
 * Kernels stage data through shared memory with asynchronous bulk copies and wait for them on
 * barriers with a bounded number of polls; a wait that runs out makes the kernel record it in a
 * per-device counter, abandon its work and return (its outputs are then incomplete) instead of
 * hanging.  This call synchronises with the current device and stores the number of such events
 * since the library was loaded in *count (0 in a healthy run).  Returns MQG_OK or MQG_ERR_CUDA.
 */
mqg_status mqg_device_timeouts(unsigned int* count);

/*
 * The same counter as a status, for bracketing a step: synchronises with the current device, stores
 * the number of waits that ran out since the library was loaded or since the last call with
 * reset != 0 in *count (count may be NULL), clears the counter if reset != 0, and returns
 * MQG_ERR_TIMEOUT when that number is not zero (the outputs of the calls enqueued on this device
 * since the last clear are then incomplete and the step has to be repeated), else MQG_OK;
 * MQG_ERR_CUDA if the device cannot be read.  The calls themselves are asynchronous and cannot
 * report it: a kernel that gives up has long been enqueued with MQG_OK.  The paper has no
 * counterpart (its transport is a blocking push / pull; Algorithm 1).
 */
mqg_status mqg_check_timeouts(unsigned int* count, int reset);

/*
 * TEST HOOK, process-wide, not for production use: the kernels launched after this call poll a
 * barrier at most poll_limit times (0 restores the default), and with arm_only != 0 they arm their
 * barriers for the bytes of a staging copy but do not issue the copy, so that the wait runs out
 * with nothing in flight, the kernel counts it, drains and returns without writing its outputs.
 * mqg_test_wait_override(0, 0) restores normal operation.  Always returns MQG_OK.
 */
mqg_status mqg_test_wait_override(uint32_t poll_limit, int arm_only);

/* Message of the last error returned to the calling thread ("" if none).  Never NULL. */
const char* mqg_last_error(void);

/* Library version, major * 10000 + minor * 100 + patch. */
int mqg_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MQGRAD_H_ */
