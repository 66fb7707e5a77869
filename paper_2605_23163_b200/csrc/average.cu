// Equal-weight mean of N rollout trajectories: out[w][c] = (1/N) sum_f traj[f][w][c].
// The sum runs in fp64 so the fp32 result is correctly rounded up to one ulp even when
// rollouts cancel.
#include "fdd_internal.h"
#include "tc_ptx.cuh"

namespace {
__global__ void average_kernel(const float* __restrict__ traj, int n, int elems, float* __restrict__ out) {
    tc::grid_dependency_wait();          // (launched for an early start behind the kernel ahead of it)
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= elems) return;
    double acc = 0.0;
    for (int f = 0; f < n; ++f) acc += static_cast<double>(traj[static_cast<size_t>(f) * elems + e]);
    out[e] = static_cast<float>(acc / static_cast<double>(n));
}
}  // namespace

cudaError_t launch_average(const float* traj, int n, int w, float* out, cudaStream_t st) {
    const int elems = w * 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((elems + 127) / 128);
    cfg.blockDim = dim3(128);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    cfg.numAttrs = overlap_launch_attribute(st, attr);
    cfg.attrs = attr;
    return cudaLaunchKernelEx(&cfg, average_kernel, traj, n, elems, out);
}
