// Status strings, ABI version and the device gate shared by all entry points.
#include <atomic>

#include "common.cuh"

namespace pulsar {

// Per-device facts are cached per host thread (a thread may switch devices between calls).
int32_t check_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return PULSAR_ERR_CUDA; }
    thread_local int cached_dev = -1;
    thread_local int32_t cached_rc = PULSAR_ERR_CUDA;
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
    thread_local int cached_dev = -1, cached = 148;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return 148; }
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            return 148;
        }
        cached = n;
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

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded device wait used by every kernel of the library.
// ---------------------------------------------------------------------------------------------
namespace pulsar {
namespace {
__global__ void wait_selftest_kernel(int32_t* status, unsigned long long limit_ns, int32_t* result) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(&bar, 1);
        mbar_fence_init();
    }
    __syncthreads();
    // Nothing ever arrives on the barrier: the wait must give up after limit_ns, report the
    // time-out and let the kernel finish normally.
    const bool ok = mbar_wait(&bar, 0, &abort_flag, status, limit_ns);
    __syncthreads();
    if (threadIdx.x == 0 && result != nullptr) *result = (ok ? 1 : 0) | (abort_flag ? 2 : 0);
}
}  // namespace
}  // namespace pulsar

extern "C" int32_t pulsar_wait_selftest(int32_t* device_status, uint64_t limit_ns, int32_t* device_result,
                                        void* stream) {
    if (limit_ns == 0 || limit_ns > 1000000000ull) return PULSAR_ERR_INVALID_ARG;     // at most one second
    int32_t rc = pulsar::check_device();
    if (rc != PULSAR_OK) return rc;
    pulsar::wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(device_status, limit_ns,
                                                                                  device_result);
    PULSAR_CUDA_OK(cudaGetLastError());
    pulsar::count_launch();
    return PULSAR_OK;
}
