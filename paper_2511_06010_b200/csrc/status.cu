// The library's one sticky device-side status word.  Kernels that find something wrong while they
// run (a bounded wait of the tensor-core kernel that ran out, routing indices that break the
// grouping's preconditions, an entry outside the batch) lower it with atomicMin to a negative
// moska_status and carry on without touching memory they should not; moska_device_status() hands
// it to the host and clears it.
#include <mutex>

#include "common.cuh"

namespace moska {

static __device__ int g_status = 0;

// `g_status` is a host-side handle in host code; its address on the current device is looked up
// once per device and kept.
int status_word(int** out)
{
    constexpr int kMaxDevices = 64;
    static int* dev_ptr[kMaxDevices] = {nullptr};
    static std::mutex mtx;
    int dev = 0;
    MOSKA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices)
        return fail(MOSKA_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
    std::lock_guard<std::mutex> lock(mtx);
    if (dev_ptr[dev] == nullptr) {
        void* p = nullptr;
        MOSKA_CUDA_TRY(cudaGetSymbolAddress(&p, g_status));
        dev_ptr[dev] = static_cast<int*>(p);
    }
    *out = dev_ptr[dev];
    return MOSKA_OK;
}

int read_status(int* out)
{
    MOSKA_CUDA_TRY(cudaDeviceSynchronize());
    MOSKA_CUDA_TRY(cudaMemcpyFromSymbol(out, g_status, sizeof(int)));
    const int zero = 0;
    MOSKA_CUDA_TRY(cudaMemcpyToSymbol(g_status, &zero, sizeof(int)));
    return MOSKA_OK;
}

}  // namespace moska
