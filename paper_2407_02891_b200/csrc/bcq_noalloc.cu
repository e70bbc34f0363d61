// bcq_gemv_noalloc: the batch-1 product for callers that cannot obtain device memory.
//
// The split-K form of the lookup-table kernel needs scratch memory (one 64-bit word per row that
// gathers the K splits' partial sums and counts their arrivals).  Here that scratch is a fixed
// array that is part of the library image, so the call neither takes a workspace nor allocates one.
#include <mutex>

#include "bcq_internal.cuh"

// Lives in the device memory of every GPU that loads this library, from load until exit.
static __device__ __align__(256) unsigned char g_noalloc_scratch[BCQ_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void *g_scratch_addr[kMaxDevices] = {};

// In host code `g_noalloc_scratch` is only a handle for the runtime, not an address a kernel can
// use; the device address has to be asked for, once per device, with that device current.
int scratch_address(void **out)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return bcq::record_cuda_error(e);
    if (dev < 0 || dev >= kMaxDevices) return bcq::record_cuda_error(cudaErrorInvalidDevice);
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return bcq::record_cuda_error(e);
        if (!p) return bcq::record_cuda_error(cudaErrorInvalidSymbol);
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return BCQ_OK;
}

}  // namespace

extern "C" int bcq_gemv_noalloc(const bcq_desc *desc, const void *packed_dev, const uint16_t *alpha_dev,
                                const uint16_t *z_dev, const uint16_t *x_dev, uint16_t *y_dev, void *stream)
{
    bcq_plan plan;
    int rc = bcq_plan_default(desc, 1, 0, &plan);
    if (rc != BCQ_OK) return rc;
    const size_t need = bcq_workspace_bytes(desc, 1, &plan);
    if (need > size_t(BCQ_NOALLOC_SCRATCH_BYTES)) return BCQ_ERR_SCRATCH_LIMIT;
    if (need == 0) return bcq_gemv_plan(desc, &plan, packed_dev, alpha_dev, z_dev, x_dev, y_dev, nullptr, 0, stream);

    void *scratch = nullptr;
    rc = scratch_address(&scratch);
    if (rc != BCQ_OK) return rc;
    // The array keeps whatever the previous call left (a completed product leaves its words zero, one that
    // was cut short need not): the kernel needs every word it uses to start at zero.
    const cudaError_t e = cudaMemsetAsync(scratch, 0, need, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return bcq::record_cuda_error(e);
    return bcq_gemv_plan(desc, &plan, packed_dev, alpha_dev, z_dev, x_dev, y_dev, scratch,
                         size_t(BCQ_NOALLOC_SCRATCH_BYTES), stream);
}
