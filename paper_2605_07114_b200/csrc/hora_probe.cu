// Measurement aid (no counterpart in the paper): the fp64 rate of the device, so that kernels bound by plain
// fp64 arithmetic can be held against a measured peak rather than a datasheet figure.
#include "hora_common.cuh"

namespace hora {

constexpr int kProbeThreads = 256;
constexpr int kProbeChains = 8;               // independent dependency chains per thread

// Every thread runs kProbeChains independent chains of `iters` fused multiply-adds; nothing touches memory until
// the one store at the end that keeps the compiler from dropping the work.
__global__ void __launch_bounds__(kProbeThreads)
fp64_probe_kernel(int32_t iters, double seed, double *sink) {
    double x[kProbeChains];
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) x[k] = seed + (double)(threadIdx.x + k);
    const double m = 1.0 - 1.0e-9, a = 1.0e-9;
    for (int32_t i = 0; i < iters; ++i) {
#pragma unroll
        for (int k = 0; k < kProbeChains; ++k) x[k] = fma(x[k], m, a);
    }
    double s = 0.0;
#pragma unroll
    for (int k = 0; k < kProbeChains; ++k) s += x[k];
    if (s == -1.0) sink[0] = s;               // never true: x stays positive
}

}  // namespace hora

extern "C" uint64_t hora_fp64_probe(int32_t iters, double *sink_dev, void *stream) {
    using namespace hora;
    if (iters < 1 || sink_dev == nullptr) return 0;
    const int grid = sm_count() * 8;
    fp64_probe_kernel<<<grid, kProbeThreads, 0, static_cast<cudaStream_t>(stream)>>>(iters, 1.0, sink_dev);
    if (cudaGetLastError() != cudaSuccess) return 0;
    count_launches(1);
    return (uint64_t)grid * kProbeThreads * kProbeChains * (uint64_t)iters;
}
