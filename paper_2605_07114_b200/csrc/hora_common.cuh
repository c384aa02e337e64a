// Shared device/host helpers of the HORA CUDA library (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "hora.h"

namespace hora {

constexpr int kWarp = 32;
constexpr unsigned kFull = 0xFFFFFFFFu;

// First data-dependent error wins; later kernels of the same call see it and stand down.
__device__ __forceinline__ void raise_status(int32_t *status, int32_t code) {
    if (status != nullptr) atomicCAS(status, 0, code);
}

__device__ __forceinline__ int lane_id() { return threadIdx.x & (kWarp - 1); }

__device__ __forceinline__ double shfl_up_f64(double v, int d) { return __shfl_up_sync(kFull, v, d); }
__device__ __forceinline__ double shfl_idx_f64(double v, int l) { return __shfl_sync(kFull, v, l); }

// Posterior parameters of one prompt (Eq. posterior) with the validity checks every kernel repeats.
struct Posterior {
    double a, b;
    int32_t cap;
    bool ok;
};

// The posterior and its checks from a prompt's raw inputs (already in registers).
__device__ __forceinline__ Posterior make_posterior(double al, double be, int32_t ci, int32_t capi, int32_t G0, int32_t ld) {
    Posterior p;
    p.cap = capi;
    p.ok = (al > 0.0) && (be > 0.0) && (al < 1.0e300) && (be < 1.0e300) && (ci >= 0) && (ci <= G0) &&
           (p.cap >= 0) && (p.cap <= ld);
    p.a = al + (double)ci;
    p.b = be + (double)(G0 - ci);
    if (!p.ok) p.cap = 0;
    return p;
}

__device__ __forceinline__ Posterior load_posterior(const double *alpha, const double *beta, double alpha0,
                                                    double beta0, const int32_t *c, int32_t G0,
                                                    const int32_t *cap, int32_t cap_scalar, int32_t ld, int64_t i) {
    const double al = alpha ? __ldg(alpha + i) : alpha0;
    const double be = beta ? __ldg(beta + i) : beta0;
    return make_posterior(al, be, __ldg(c + i), cap ? __ldg(cap + i) : cap_scalar, G0, ld);
}

inline hora_status_t cuda_ok(cudaError_t e) { return e == cudaSuccess ? HORA_OK : HORA_ERR_CUDA; }

// Multiprocessors of the current device (148 on B200), looked up once per device; persistent grids are sized
// in multiples of it.
int sm_count();

inline int clamp_grid(int64_t want, int per_sm) {
    const int64_t cap = (int64_t)sm_count() * per_sm;
    if (want < 1) want = 1;
    return (int)(want < cap ? want : cap);
}

// Programmatic dependent launch.  The kernels of the hot calls are launched with the attribute set below and
// open with pdl_enter(), before which they touch no global memory: it returns once the kernel before it in the
// stream has finished and its writes are visible (hence, by induction, every earlier one).  What this buys: the
// launch of a kernel is set up while the kernel in front still runs, so the gap between the short dependent
// kernels of a call shrinks (hora_allocate: 85 -> 68 us at N = 512, 116 -> 100 us at N = 16384, 0.489 -> 0.478 ms
// at N = 2^20).  No kernel signals early (griddepcontrol.launch_dependents): letting the next kernel's CTAs move
// in beside a running one was measured and made the full-size call slower (0.478 -> 0.51-0.56 ms), whichever
// kernel gave the signal.  After a kernel that does not take part (or a copy, or a memset) the attribute changes
// nothing, and pdl_enter() in a kernel launched without it returns at once.
__device__ __forceinline__ void pdl_enter() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t stream,
                              Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Host-side count of kernels this library has launched in this process (see hora_launch_count).
void count_launches(int n);

// Launchers shared between translation units.
hora_status_t launch_gains(const double *alpha, const double *beta, double alpha0, double beta0,
                           const int32_t *c, int32_t G0, const int32_t *cap, int32_t cap_scalar, int64_t N,
                           int32_t ld, double *gains, int32_t *status_dev, cudaStream_t stream);

}  // namespace hora
