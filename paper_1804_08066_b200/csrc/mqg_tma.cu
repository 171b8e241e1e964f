// Host side of the TMA helpers: tensor-map encoding through the driver entry point (so the
// library needs no link-time dependency on libcuda) and the per-device timeout counter.
#include <atomic>
#include <mutex>

#include "mqg_tma.cuh"

namespace mqg {

__device__ unsigned int g_wait_timeouts = 0;

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

constexpr int kMaxDevices = 64;
std::mutex g_counter_mutex;
unsigned int* g_counter_ptr[kMaxDevices] = {};

}  // namespace

bool encode_rows_map(CUtensorMap* map, const void* base, uint64_t rows, int elem_bytes,
                     uint32_t row_elems, uint32_t box_rows, const char** why)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) { *why = "cuTensorMapEncodeTiled entry point not available"; return false; }
    const uint32_t row_bytes = row_elems * (uint32_t)elem_bytes;
    CUtensorMapDataType dt;
    CUtensorMapSwizzle sw;
    if (elem_bytes == 4) dt = CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    else if (elem_bytes == 2) dt = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    else { *why = "unsupported element size"; return false; }
    if (row_bytes == 128) sw = CU_TENSOR_MAP_SWIZZLE_128B;
    else if (row_bytes == 64) sw = CU_TENSOR_MAP_SWIZZLE_64B;
    else { *why = "unsupported row size"; return false; }
    const cuuint64_t dims[2] = {row_elems, rows};
    const cuuint64_t strides[1] = {row_bytes};
    const cuuint32_t box[2] = {row_elems, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { *why = "cuTensorMapEncodeTiled failed"; return false; }
    return true;
}

unsigned int* wait_timeout_counter()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_counter_mutex);
    if (!g_counter_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_wait_timeouts) != cudaSuccess) return nullptr;
        g_counter_ptr[dev] = static_cast<unsigned int*>(p);
    }
    return g_counter_ptr[dev];
}

cudaError_t read_wait_timeouts(unsigned int* count, bool reset)
{
    cudaError_t err = cudaMemcpyFromSymbol(count, g_wait_timeouts, sizeof(unsigned int), 0, cudaMemcpyDeviceToHost);
    if (err == cudaSuccess && reset && *count != 0) {
        const unsigned int zero = 0;
        err = cudaMemcpyToSymbol(g_wait_timeouts, &zero, sizeof(unsigned int), 0, cudaMemcpyHostToDevice);
    }
    return err;
}

namespace {
std::atomic<uint32_t> g_poll_limit{kMaxWaitPolls};
std::atomic<uint32_t> g_arm_only{0};
}  // namespace

WaitPolicy wait_policy()
{
    WaitPolicy p;
    p.poll_limit = g_poll_limit.load(std::memory_order_relaxed);
    p.arm_only = g_arm_only.load(std::memory_order_relaxed);
    return p;
}

void set_wait_policy(uint32_t poll_limit, uint32_t arm_only)
{
    g_poll_limit.store(poll_limit == 0 ? kMaxWaitPolls : poll_limit, std::memory_order_relaxed);
    g_arm_only.store(arm_only ? 1u : 0u, std::memory_order_relaxed);
}

}  // namespace mqg
