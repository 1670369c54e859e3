// Host-side helpers shared by the launch code of several kernels.
#pragma once

#include <cuda_runtime.h>

#include <mutex>
#include <set>
#include <utility>

namespace prom {

// Remembers which (device, key) pairs have been seen.  A kernel's dynamic shared-memory limit
// (cudaFuncAttributeMaxDynamicSharedMemorySize) belongs to the device that was current when it
// was set, so a process that drives several GPUs must raise it once on each of them.
class OncePerDevice {
public:
    // true the first time (dev, key) is asked about, false afterwards
    bool first(int dev, const void *key)
    {
        std::lock_guard<std::mutex> lk(mu_);
        return seen_.insert(std::make_pair(dev, key)).second;
    }
    void forget(int dev, const void *key)
    {
        std::lock_guard<std::mutex> lk(mu_);
        seen_.erase(std::make_pair(dev, key));
    }

private:
    std::mutex mu_;
    std::set<std::pair<int, const void *>> seen_;
};

// Raises `func`'s dynamic shared-memory limit to `bytes` on the current device, once per device.
template <class F>
static cudaError_t raise_smem_limit(F *func, int bytes)
{
    static OncePerDevice table;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const void *key = reinterpret_cast<const void *>(func);
    if (!table.first(dev, key)) return cudaSuccess;
    e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) table.forget(dev, key);       // try again on the next call
    return e;
}

}  // namespace prom
