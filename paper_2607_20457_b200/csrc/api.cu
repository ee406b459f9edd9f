// Status strings, ABI version and the device gate shared by all entry points.
#include <atomic>

#include "common.cuh"

namespace pulsar {

int32_t check_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return PULSAR_ERR_CUDA; }
    static int cached_dev = -1;
    static int32_t cached_rc = PULSAR_ERR_CUDA;
    if (dev == cached_dev) return cached_rc;
    int major = 0, minor = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return PULSAR_ERR_CUDA;
    }
    cached_rc = (major == 10 && minor == 0) ? PULSAR_OK : PULSAR_ERR_UNSUPPORTED_DEVICE;
    cached_dev = dev;
    return cached_rc;
}

int sm_count() {
    static int cached_dev = -1, cached = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        if (cudaDeviceGetAttribute(&cached, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) cached = 148;
        cached_dev = dev;
    }
    return cached;
}

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(static_cast<uint64_t>(n), std::memory_order_relaxed); }

}  // namespace pulsar

extern "C" const char* pulsar_status_string(int32_t status) {
    switch (status) {
        case PULSAR_OK: return "PULSAR_OK";
        case PULSAR_ERR_INVALID_ARG: return "PULSAR_ERR_INVALID_ARG";
        case PULSAR_ERR_SHAPE: return "PULSAR_ERR_SHAPE";
        case PULSAR_ERR_ALIGNMENT: return "PULSAR_ERR_ALIGNMENT";
        case PULSAR_ERR_WORKSPACE: return "PULSAR_ERR_WORKSPACE";
        case PULSAR_ERR_UNSUPPORTED_DEVICE: return "PULSAR_ERR_UNSUPPORTED_DEVICE";
        case PULSAR_ERR_CUDA: return "PULSAR_ERR_CUDA";
        case PULSAR_ERR_TIMEOUT: return "PULSAR_ERR_TIMEOUT";
        case PULSAR_ERR_DEVICE_CHECK: return "PULSAR_ERR_DEVICE_CHECK";
        default: return "PULSAR_ERR_UNKNOWN";
    }
}

extern "C" int32_t pulsar_abi_version(void) { return 1; }

extern "C" uint64_t pulsar_launch_count(void) { return pulsar::g_launches.load(std::memory_order_relaxed); }
