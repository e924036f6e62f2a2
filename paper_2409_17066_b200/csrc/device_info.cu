// Per-device facts the launch plans depend on, looked up once per device ordinal.
#include "common.cuh"

#include <atomic>
#include <stdlib.h>
#include <string.h>

namespace vptq {

namespace {
constexpr int kMaxDevices = 64;
std::atomic<int> g_sm_count[kMaxDevices];     // 0 = not looked up yet
std::atomic<unsigned long long> g_wait_limit{0};
}

unsigned long long debug_wait_limit() { return g_wait_limit.load(std::memory_order_relaxed); }
void set_debug_wait_limit(unsigned long long cycles) { g_wait_limit.store(cycles, std::memory_order_relaxed); }

// Streaming multiprocessors of the CURRENT device (every persistent grid and every row split is sized by
// it, so a plan made with one device current must be launched with that device current).  Without a
// usable device (size queries on a machine with no GPU) the answer is that of a B200.
int device_sm_count()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) return 148;
    if (dev < kMaxDevices) {
        const int cached = g_sm_count[dev].load(std::memory_order_relaxed);
        if (cached > 0) return cached;
    }
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) return 148;
    if (dev < kMaxDevices) g_sm_count[dev].store(v, std::memory_order_relaxed);
    return v;
}

bool pdl_enabled(const char *family)
{
    static const char *off = getenv("VPTQ_NO_PDL");          // read once
    if (off == nullptr || off[0] == 0) return true;
    return strstr(off, "all") == nullptr && strstr(off, family) == nullptr;
}

}  // namespace vptq
