// Checked build (-DHORA_CHECKED): index checks that record instead of trapping.
//
// HORA_AT(array, index, count) stands for array[index].  In a checked build an index outside [0, count) is
// recorded — the first one wins: (file id << 20) | line — in a word of device memory and the access is redirected
// to a scratch slot, so nothing faults, nothing traps and the kernel runs on; hora_checked_violation() reads the
// word back.  In the normal build the macro is the plain access and costs nothing.  It guards the accesses whose
// index is computed from device DATA (histogram bins taken from key bits, list slots handed out by atomics, row
// positions found by searches, slab positions derived from offsets); loop counters that run to a bound stated
// next to them are left alone.
#pragma once

#include "hora_common.cuh"

namespace hora {

#ifdef HORA_CHECKED
// one word and one scratch slot per translation unit (device code is not linked across files)
static __device__ unsigned int g_check_word = 0u;
static __device__ __align__(16) unsigned long long g_check_sink[4];

template <typename T>
__device__ __forceinline__ T &checked_at(T *arr, long long i, long long n, unsigned site) {
    static_assert(sizeof(T) <= sizeof(g_check_sink), "the scratch slot holds any element type used here");
    if (i < 0 || i >= n) {
        atomicCAS(&g_check_word, 0u, site);
        return *reinterpret_cast<T *>(g_check_sink);
    }
    return arr[i];
}

// host: every checked translation unit registers how to read (and clear) its word
void register_check_word(unsigned (*fetch_and_clear)());

#define HORA_AT(arr, i, n) \
    (::hora::checked_at((arr), (long long)(i), (long long)(n), (unsigned)((HORA_FILE_ID << 20) | __LINE__)))

#define HORA_CHECKED_REGISTER()                                                                  \
    namespace {                                                                                  \
    struct HoraCheckRegistration {                                                               \
        HoraCheckRegistration() {                                                                \
            ::hora::register_check_word([]() -> unsigned {                                       \
                unsigned v = 0u, zero = 0u;                                                      \
                if (cudaMemcpyFromSymbol(&v, ::hora::g_check_word, sizeof v) != cudaSuccess) return 0xFFFFFFFFu; \
                if (v != 0u) cudaMemcpyToSymbol(::hora::g_check_word, &zero, sizeof zero);       \
                return v;                                                                        \
            });                                                                                  \
        }                                                                                        \
    } g_hora_check_registration;                                                                 \
    }
#else
#define HORA_AT(arr, i, n) ((arr)[i])
#define HORA_CHECKED_REGISTER()
#endif

}  // namespace hora
