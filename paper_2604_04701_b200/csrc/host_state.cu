// The library's host-side state: per-device results of one-time set-up, and the test hooks.
#include "kernels.h"

namespace muxq {

namespace {
std::mutex g_mutex;
PerDevice<int> g_sms;
TestHooks g_hooks;
}  // namespace

int current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
    return dev;
}

std::mutex &device_mutex() { return g_mutex; }

int num_sms() {
    const int dev = current_device();
    if (dev < 0) return 0;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_sms.have[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 0;
        g_sms.v[dev] = n;
        g_sms.have[dev] = true;
    }
    return g_sms.v[dev];
}

const TestHooks &test_hooks() { return g_hooks; }
void set_test_hooks(const TestHooks &h) {
    std::lock_guard<std::mutex> lock(g_mutex);
    g_hooks = h;
}

}  // namespace muxq
