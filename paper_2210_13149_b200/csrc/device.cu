// Per-device facts the launchers size their grids from.
#include <atomic>

#include "bigcn_internal.cuh"

namespace bigcn {

int sm_count()
{
    constexpr int kMaxDevices = 64;
    static std::atomic<int> cached[kMaxDevices];            // 0 = not yet queried
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 1;
    int v = cached[dev].load(std::memory_order_relaxed);
    if (v > 0) return v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1) return 1;
    cached[dev].store(v, std::memory_order_relaxed);
    return v;
}

}  // namespace bigcn
