// Equal-weight mean of N rollout trajectories: out[w][c] = (1/N) sum_f traj[f][w][c].
// The sum runs in fp64 so the fp32 result is correctly rounded up to one ulp even when
// rollouts cancel.
#include "fdd_internal.h"

namespace {
__global__ void average_kernel(const float* __restrict__ traj, int n, int elems, float* __restrict__ out) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= elems) return;
    double acc = 0.0;
    for (int f = 0; f < n; ++f) acc += static_cast<double>(traj[static_cast<size_t>(f) * elems + e]);
    out[e] = static_cast<float>(acc / static_cast<double>(n));
}
}  // namespace

cudaError_t launch_average(const float* traj, int n, int w, float* out, cudaStream_t st) {
    const int elems = w * 2;
    average_kernel<<<(elems + 127) / 128, 128, 0, st>>>(traj, n, elems, out);
    return cudaGetLastError();
}
