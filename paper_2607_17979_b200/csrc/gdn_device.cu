// Per-device facts the launchers need on every call, looked up once per device and process:
// the SM count, whether cooperative launches exist, and which kernels already had their dynamic
// shared memory limit raised.  (Each of these is a driver round trip of a microsecond or more,
// which is most of the host cost of a small decode or prefill call.)
#include "gdn_common.cuh"
#include <mutex>

namespace gdn {
namespace {

constexpr int kMaxDevices = 64;
constexpr int kMaxKernels = 64;
std::mutex g_mutex;
DeviceInfo g_info[kMaxDevices];
bool g_have[kMaxDevices] = {};
struct SmemEntry { int dev; const void* kernel; int bytes; };
SmemEntry g_smem[kMaxKernels];
int g_smem_count = 0;

}  // namespace

cudaError_t device_info(DeviceInfo* out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    out->device = dev;
    if (dev >= 0 && dev < kMaxDevices) {
        std::lock_guard<std::mutex> lock(g_mutex);
        if (g_have[dev]) {
            *out = g_info[dev];
            return cudaSuccess;
        }
    }
    int sms = 0, coop = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    if (e != cudaSuccess) return e;
    out->sms = sms;
    out->cooperative = coop;
    if (dev >= 0 && dev < kMaxDevices) {
        std::lock_guard<std::mutex> lock(g_mutex);
        g_info[dev] = *out;
        g_have[dev] = true;
    }
    return cudaSuccess;
}

cudaError_t ensure_dynamic_smem(const void* kernel, int bytes) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    {
        std::lock_guard<std::mutex> lock(g_mutex);
        for (int i = 0; i < g_smem_count; ++i)
            if (g_smem[i].dev == dev && g_smem[i].kernel == kernel && g_smem[i].bytes >= bytes)
                return cudaSuccess;
    }
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_smem_count < kMaxKernels) g_smem[g_smem_count++] = SmemEntry{dev, kernel, bytes};
    return cudaSuccess;
}

}  // namespace gdn
