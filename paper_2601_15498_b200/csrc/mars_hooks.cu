// Storage and C entry point of the test hooks (see mars_hooks.cuh), and the device check.
#include "mars_hooks.cuh"

#include <atomic>

#include <cuda_runtime.h>

#include "mars.h"

namespace mars {

static std::atomic<int> g_hook[kHookCount];

int hook(int which)
{
    return (which >= 0 && which < kHookCount) ? g_hook[which].load(std::memory_order_relaxed) : 0;
}

}  // namespace mars

extern "C" int mars_test_hook(int which, int value)
{
    if (which < 0 || which >= mars::kHookCount || value < 0) return -1;
    return mars::g_hook[which].exchange(value, std::memory_order_relaxed);
}

extern "C" mars_status_t mars_device_check(int *sm_count, int *sm_tuned)
{
    constexpr int kTunedSms = 148;
    if (sm_tuned) *sm_tuned = kTunedSms;
    int dev = -1, sms = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return MARS_ERR_CUDA;
    }
    if (sm_count) *sm_count = sms;
    return (sms == kTunedSms && major == 10) ? MARS_OK : MARS_ERR_UNSUPPORTED;
}
