// Per-device, per-kernel set-up that launchers would otherwise repeat on every call.
#include <map>
#include <mutex>
#include <utility>

#include "common.cuh"

namespace ssm {

// The dynamic shared-memory limit is an attribute of the function in one device's context:
// set it the first time a kernel is launched on a device, remember that it was.
bool set_max_dynamic_smem(const void* kernel, size_t bytes) {
    static std::mutex mu;
    static std::map<std::pair<const void*, int>, size_t> done;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(mu);
    auto it = done.find({kernel, dev});
    if (it != done.end() && it->second >= bytes) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    done[{kernel, dev}] = bytes;
    return true;
}

// Workspace layouts, operand packing order and kernel choices depend on the SM count, so it is
// looked up for the device that is current, once per ordinal.
int device_sm_count() {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static int cache[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        (void)cudaGetLastError();
        return 148;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (!cache[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            return 148;
        }
        cache[dev] = n;
    }
    return cache[dev];
}

}  // namespace ssm
