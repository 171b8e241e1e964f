// mqg_quantize_segments_l2_static: the per-layer L2-norm quantizer for callers that have no device
// memory to hand over as a workspace and no way to get any.
//
// Who that is: code that runs after the process has given all of the device's memory to one pool
// (a serving runtime or a framework allocator that reserves everything at start-up, so that a
// later cudaMalloc fails), code on a latency-critical path where the device-wide synchronisation
// an allocation implies is not acceptable, and code that is only allowed to launch work (plug-ins
// and callbacks whose host hands them input and output buffers and forbids anything that changes
// the device's memory map).  Such a caller cannot build the workspace that
// mqg_quantize_segments_l2 asks for.
//
// The partial sums therefore live in an array that is part of the library image: it takes up
// device memory on every GPU the library is used on, from the moment the image is loaded there
// until the process exits, whether or not this entry point is ever called.  Its size is the
// limit of this entry point.
#include <mutex>

#include "../../include/mqgrad.h"
#include "mqg_internal.h"

// One float per tile of 8192 elements: 256 KiB per device, enough for 2^29 elements in full tiles.
static __device__ __align__(256) float g_l2_tile_sums[MQG_L2_STATIC_WORKSPACE_FLOATS];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
float* g_tile_sums_address[kMaxDevices] = {};

// In host code the array's name only stands for the symbol: it is not an address a kernel can
// use.  The address differs per device and has to be asked for with that device current; it is
// looked up on the first call on each device and kept.
cudaError_t tile_sums_address(float** out)
{
    int dev = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err != cudaSuccess) return err;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_tile_sums_address[dev] == nullptr) {
        float* p = nullptr;
        err = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_l2_tile_sums);
        if (err != cudaSuccess) return err;
        g_tile_sums_address[dev] = p;
    }
    *out = g_tile_sums_address[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" mqg_status mqg_quantize_segments_l2_static(const void* grad, int nseg, const uint64_t* seg_off,
                                                      const uint64_t* code_off, int bits, uint64_t seed,
                                                      uint32_t* codes, float* scales, mqg_dtype dtype,
                                                      uint32_t worker, uint32_t step, uint64_t elem_offset,
                                                      void* cuda_stream)
{
    if (nseg > 0 && seg_off != nullptr) {
        for (int j = 0; j < nseg; ++j)       // a decreasing table would make the count meaningless
            if (seg_off[j + 1] < seg_off[j])
                return mqg::report_error(MQG_ERR_INVALID, "seg_off decreases at %d", j);
        const size_t need = mqg_l2_workspace_floats(nseg, seg_off);
        if (need > (size_t)MQG_L2_STATIC_WORKSPACE_FLOATS)
            return mqg::report_error(MQG_ERR_INVALID,
                                     "mqg_quantize_segments_l2_static: the segments need %llu partial sums, the "
                                     "built-in array holds %d; use mqg_quantize_segments_l2 with a workspace",
                                     (unsigned long long)need, MQG_L2_STATIC_WORKSPACE_FLOATS);
    }
    float* tile_sums = nullptr;
    const cudaError_t err = tile_sums_address(&tile_sums);
    if (err != cudaSuccess)
        return mqg::report_error(MQG_ERR_CUDA, "mqg_quantize_segments_l2_static: address of the built-in array: %s",
                                 cudaGetErrorString(err));
    // Nothing in the array has to start at zero: the sum pass writes every element that the fold
    // reads, so whatever an earlier call left there is overwritten before it is looked at.
    return mqg_quantize_segments_l2(grad, nseg, seg_off, code_off, bits, seed, codes, scales, dtype, worker,
                                    step, elem_offset, tile_sums, (size_t)MQG_L2_STATIC_WORKSPACE_FLOATS,
                                    cuda_stream);
}
