// Append a finished block's K/V rows to each rollout's private suffix cache.
// Source [N][d][Hkv][D] (token-major, as projected), destination [N][Hkv][cap][D]
// (head-major, so that a key tile of one head is contiguous).  16-byte copies.
#include "fdd_internal.h"

namespace {
__global__ void kv_commit_kernel(const uint4* __restrict__ k_blk, const uint4* __restrict__ v_blk,
                                 uint4* __restrict__ suffix_k, uint4* __restrict__ suffix_v,
                                 int n_forks, int d, int n_kv_heads, int vec_per_row,
                                 int suffix_len, int suffix_capacity) {
    const long long total = static_cast<long long>(n_forks) * d * n_kv_heads * vec_per_row;
    for (long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; idx < total;
         idx += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int c = static_cast<int>(idx % vec_per_row);
        long long t = idx / vec_per_row;
        const int h = static_cast<int>(t % n_kv_heads); t /= n_kv_heads;
        const int i = static_cast<int>(t % d);
        const int f = static_cast<int>(t / d);
        const long long dst = ((static_cast<long long>(f) * n_kv_heads + h) * suffix_capacity + suffix_len + i)
                                  * vec_per_row + c;
        suffix_k[dst] = k_blk[idx];
        suffix_v[dst] = v_blk[idx];
    }
}
}  // namespace

cudaError_t launch_kv_commit(const __nv_bfloat16* k_blk, const __nv_bfloat16* v_blk,
                             __nv_bfloat16* suffix_k, __nv_bfloat16* suffix_v,
                             int n_forks, int d, int n_kv_heads, int head_dim,
                             int suffix_len, int suffix_capacity, cudaStream_t st) {
    const int vec_per_row = head_dim / 8;
    const long long total = static_cast<long long>(n_forks) * d * n_kv_heads * vec_per_row;
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    if (blocks > 148 * 8) blocks = 148 * 8;
    if (blocks < 1) blocks = 1;
    kv_commit_kernel<<<static_cast<unsigned>(blocks), threads, 0, st>>>(
        reinterpret_cast<const uint4*>(k_blk), reinterpret_cast<const uint4*>(v_blk),
        reinterpret_cast<uint4*>(suffix_k), reinterpret_cast<uint4*>(suffix_v),
        n_forks, d, n_kv_heads, vec_per_row, suffix_len, suffix_capacity);
    return cudaGetLastError();
}
