// Host-only entry points of the HORA library.
#include <atomic>

#include "hora_common.cuh"

namespace hora {
static std::atomic<unsigned long long> g_launches{0};
void count_launches(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

int sm_count() {
    constexpr int kMaxDev = 64, kFallback = 148;           // B200, should the query fail
    static std::atomic<int> cached[kMaxDev];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return kFallback;
    int n = cached[dev].load(std::memory_order_acquire);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return kFallback;
    cached[dev].store(n, std::memory_order_release);
    return n;
}
}  // namespace hora

#ifdef HORA_CHECKED
namespace hora {
constexpr int kMaxCheckedUnits = 16;
static unsigned (*g_check_fetch[kMaxCheckedUnits])();
static int g_check_units = 0;
void register_check_word(unsigned (*fetch_and_clear)()) {
    if (g_check_units < kMaxCheckedUnits) g_check_fetch[g_check_units++] = fetch_and_clear;
}
}  // namespace hora
#endif

extern "C" int32_t hora_checked_violation(void) {
#ifdef HORA_CHECKED
    if (cudaDeviceSynchronize() != cudaSuccess) return -2;
    int32_t first = 0;
    for (int k = 0; k < hora::g_check_units; ++k) {
        const unsigned v = hora::g_check_fetch[k]();          // reads and clears every unit's word
        if (v != 0u && first == 0) first = (int32_t)v;
    }
    return first;
#else
    return -1;
#endif
}

extern "C" const char *hora_status_string(hora_status_t status) {
    switch (status) {
        case HORA_OK: return "ok";
        case HORA_ERR_INVALID_ARG: return "invalid argument";
        case HORA_ERR_INVALID_VALUE: return "invalid value in device data";
        case HORA_ERR_INFEASIBLE: return "budget exceeds the total cap";
        case HORA_ERR_NOT_INTEGER: return "exact mode needs integer-valued priors";
        case HORA_ERR_EXACT_RANGE: return "exact mode: parameters out of range";
        case HORA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case HORA_ERR_CUDA: return "CUDA runtime error";
        case HORA_ERR_INTERNAL: return "internal consistency check failed";
    }
    return "unknown status";
}

extern "C" int hora_version(void) { return 200; }

extern "C" uint64_t hora_launch_count(void) { return hora::g_launches.load(std::memory_order_relaxed); }
