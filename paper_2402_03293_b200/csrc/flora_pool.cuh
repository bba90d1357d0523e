// Stream-ordered scratch memory for the calls that need some for their own duration (job tables and r x r products
// of the transfer, the tables of single-matrix calls).  It comes from a memory pool that the library owns, one per
// device, whose freed blocks stay cached up to 64 MB: with the device's default pool a synchronisation hands freed
// memory back to the driver, and the next call pays milliseconds to get it again.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

namespace flora {

constexpr int POOL_MAX_DEVICES = 64;

inline cudaError_t scratch_alloc(void** out, size_t bytes, cudaStream_t st)
{
    static std::mutex mutex;
    static cudaMemPool_t pools[POOL_MAX_DEVICES] = {};
    static bool tried[POOL_MAX_DEVICES] = {};
    int dev = -1;
    cudaMemPool_t pool = nullptr;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < POOL_MAX_DEVICES) {
        std::lock_guard<std::mutex> lock(mutex);
        if (!tried[dev]) {
            tried[dev] = true;
            cudaMemPoolProps props = {};
            props.allocType = cudaMemAllocationTypePinned;
            props.handleTypes = cudaMemHandleTypeNone;
            props.location.type = cudaMemLocationTypeDevice;
            props.location.id = dev;
            uint64_t keep = 64ull << 20;
            if (cudaMemPoolCreate(&pools[dev], &props) != cudaSuccess ||
                cudaMemPoolSetAttribute(pools[dev], cudaMemPoolAttrReleaseThreshold, &keep) != cudaSuccess) {
                cudaGetLastError();
                pools[dev] = nullptr;                       // the device's default pool serves instead
            }
        }
        pool = pools[dev];
    }
    return pool ? cudaMallocFromPoolAsync(out, bytes, pool, st) : cudaMallocAsync(out, bytes, st);
}

}  // namespace flora
