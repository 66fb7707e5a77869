// Jerk-minimising interpolation of the rollout trajectories, fused with their averaging.
//
// The curve through knots (t_k, x_k), k = 0 .. n, that minimises the integral of the squared jerk
// is the natural quintic spline: a quintic per interval, four continuous derivatives, third and
// fourth derivative zero at both ends.  It is linear in the knot values, so the W_out output
// waypoints are a fixed matrix times the knot values, and the mean of the interpolated rollouts
// is that matrix times the mean of the rollouts.  The host builds the matrix once per
// (W, W_out) by solving the spline conditions directly (fp64, dense elimination, at most 198
// unknowns); the kernel averages the rollouts in fp64 and applies it.
// Knots: the origin of the vehicle frame at t = 0, waypoint k at t = k + 1; outputs at
// t_j = (j + 1) W / W_out.
#include "fdd_internal.h"

#include <cmath>
#include <vector>

namespace {

// coefficient of c_m in the d-th derivative of sum_m c_m s^m at s
double poly_term(int m, int d, double s) {
    if (m < d) return 0.0;
    double f = 1.0;
    for (int i = 0; i < d; ++i) f *= static_cast<double>(m - i);
    return f * std::pow(s, m - d);
}

// Solve A x = B (A: n x n, B: n x r, both row-major, overwritten) with partial pivoting.
bool solve_dense(std::vector<double>& A, std::vector<double>& B, int n, int r) {
    for (int c = 0; c < n; ++c) {
        int p = c;
        for (int i = c + 1; i < n; ++i)
            if (std::fabs(A[static_cast<size_t>(i) * n + c]) > std::fabs(A[static_cast<size_t>(p) * n + c])) p = i;
        if (std::fabs(A[static_cast<size_t>(p) * n + c]) < 1e-300) return false;
        if (p != c) {
            for (int j = 0; j < n; ++j) std::swap(A[static_cast<size_t>(p) * n + j], A[static_cast<size_t>(c) * n + j]);
            for (int j = 0; j < r; ++j) std::swap(B[static_cast<size_t>(p) * r + j], B[static_cast<size_t>(c) * r + j]);
        }
        const double inv = 1.0 / A[static_cast<size_t>(c) * n + c];
        for (int i = c + 1; i < n; ++i) {
            const double f = A[static_cast<size_t>(i) * n + c] * inv;
            if (f == 0.0) continue;
            for (int j = c; j < n; ++j) A[static_cast<size_t>(i) * n + j] -= f * A[static_cast<size_t>(c) * n + j];
            for (int j = 0; j < r; ++j) B[static_cast<size_t>(i) * r + j] -= f * B[static_cast<size_t>(c) * r + j];
        }
    }
    for (int c = n - 1; c >= 0; --c) {
        const double inv = 1.0 / A[static_cast<size_t>(c) * n + c];
        for (int j = 0; j < r; ++j) {
            double v = B[static_cast<size_t>(c) * r + j];
            for (int k = c + 1; k < n; ++k) v -= A[static_cast<size_t>(c) * n + k] * B[static_cast<size_t>(k) * r + j];
            B[static_cast<size_t>(c) * r + j] = v * inv;
        }
    }
    return true;
}

__global__ void average_jmt_kernel(const float* __restrict__ traj, int n, int w, int w_out,
                                   const double* __restrict__ weights, float* __restrict__ out) {
    __shared__ double mean[kJmtMaxWaypoints * 2];
    const int elems = w * 2;
    for (int e = threadIdx.x; e < elems; e += blockDim.x) {
        double acc = 0.0;
        for (int f = 0; f < n; ++f) acc += static_cast<double>(traj[static_cast<size_t>(f) * elems + e]);
        mean[e] = acc / static_cast<double>(n);
    }
    __syncthreads();
    for (int o = threadIdx.x; o < w_out * 2; o += blockDim.x) {
        const int j = o >> 1, c = o & 1;
        double acc = 0.0;
        for (int k = 0; k < w; ++k) acc += weights[static_cast<size_t>(j) * w + k] * mean[k * 2 + c];
        out[o] = static_cast<float>(acc);
    }
}

}  // namespace

// weights[j][k]: what waypoint k (k = 0 .. w - 1, at t = k + 1) contributes to output j; the origin
// knot contributes nothing (its value is zero) but shapes the curve.
bool jmt_weights(int w, int w_out, std::vector<double>* weights) {
    const int n_seg = w;                       // intervals [k, k + 1], k = 0 .. w - 1
    const int n = 6 * n_seg;
    std::vector<double> A(static_cast<size_t>(n) * n, 0.0), B(static_cast<size_t>(n) * w, 0.0);
    int row = 0;
    auto at = [&](int r, int seg, int m) -> double& { return A[static_cast<size_t>(r) * n + seg * 6 + m]; };
    for (int s = 0; s < n_seg; ++s) {
        // the interval's polynomial in its local variable (0 at the left knot, 1 at the right one)
        for (int m = 0; m < 6; ++m) at(row, s, m) = poly_term(m, 0, 0.0);
        if (s > 0) B[static_cast<size_t>(row) * w + (s - 1)] = 1.0;          // left knot: waypoint s - 1 (the origin for s = 0)
        ++row;
        for (int m = 0; m < 6; ++m) at(row, s, m) = poly_term(m, 0, 1.0);
        B[static_cast<size_t>(row) * w + s] = 1.0;                              // right knot: waypoint s
        ++row;
    }
    for (int s = 0; s + 1 < n_seg; ++s)
        for (int d = 1; d <= 4; ++d) {                                          // derivatives 1..4 continuous
            for (int m = 0; m < 6; ++m) {
                at(row, s, m) = poly_term(m, d, 1.0);
                at(row, s + 1, m) = -poly_term(m, d, 0.0);
            }
            ++row;
        }
    for (int d = 3; d <= 4; ++d) {                                              // natural ends
        for (int m = 0; m < 6; ++m) at(row, 0, m) = poly_term(m, d, 0.0);
        ++row;
        for (int m = 0; m < 6; ++m) at(row, n_seg - 1, m) = poly_term(m, d, 1.0);
        ++row;
    }
    if (row != n || !solve_dense(A, B, n, w)) return false;
    weights->assign(static_cast<size_t>(w_out) * w, 0.0);
    for (int j = 0; j < w_out; ++j) {
        const double t = static_cast<double>(j + 1) * w / w_out;
        int seg = static_cast<int>(std::floor(t));
        if (seg >= n_seg) seg = n_seg - 1;
        const double s = t - seg;
        for (int k = 0; k < w; ++k) {
            double v = 0.0;
            for (int m = 0; m < 6; ++m) v += B[static_cast<size_t>(seg * 6 + m) * w + k] * poly_term(m, 0, s);
            (*weights)[static_cast<size_t>(j) * w + k] = v;
        }
    }
    return true;
}

cudaError_t launch_average_jmt(const float* traj, int n, int w, int w_out, const double* d_weights, float* out,
                               cudaStream_t st) {
    average_jmt_kernel<<<1, 128, 0, st>>>(traj, n, w, w_out, d_weights, out);
    return cudaGetLastError();
}
