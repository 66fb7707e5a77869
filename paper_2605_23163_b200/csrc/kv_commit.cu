// Append a finished block's K/V rows to a cache: every rollout's private suffix (fdd_kv_commit),
// or the shared prefix itself when the one rollout that decodes the deterministic sections
// commits a block (fdd_prefix_extend).  Source [N][d][Hkv][D] (token-major, as projected);
// destination head-major, so that a key tile of one head is contiguous:
//   private suffix    [N][Hkv][cap][D]
//   contiguous prefix [Hkv][cap][D]
//   paged prefix      [pages][Hkv][64][D], logical page -> physical page through the page table.
// 16-byte copies; all scenes of a call go into one launch.
#include "fdd_internal.h"
#include "tc_ptx.cuh"

namespace {
__global__ void kv_commit_kernel(const __grid_constant__ CommitArgs a) {
    tc::grid_dependency_wait();          // (launched for an early start behind the kernel ahead of it)
    for (long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; idx < a.total;
         idx += static_cast<long long>(gridDim.x) * blockDim.x) {
        int s = 0;
        while (s + 1 < a.n && idx >= a.set[s + 1].vec_begin) ++s;
        const CommitSet& cs = a.set[s];
        const long long local = idx - cs.vec_begin;
        const int c = static_cast<int>(local % a.vec_per_row);
        long long t = local / a.vec_per_row;
        const int h = static_cast<int>(t % a.n_kv_heads); t /= a.n_kv_heads;
        const int i = static_cast<int>(t % cs.d);
        const int f = static_cast<int>(t / cs.d);
        const int tok = cs.len + i;
        long long dst;
        if (cs.mode == kCommitSuffix) {
            dst = ((static_cast<long long>(f) * a.n_kv_heads + h) * cs.cap + tok) * a.vec_per_row + c;
        } else if (cs.mode == kCommitPrefix) {
            dst = (static_cast<long long>(h) * cs.cap + tok) * a.vec_per_row + c;
        } else {
            const long long page = cs.page_table[tok / cs.page_tokens];
            if (page < 0 || page >= cs.cap) {           // a page table entry outside the pool: nothing is written
                atomicCAS(a.status, 0, FDD_ERR_INVALID_ARG);
                continue;
            }
            dst = ((page * a.n_kv_heads + h) * cs.page_tokens + tok % cs.page_tokens) * a.vec_per_row + c;
        }
        reinterpret_cast<uint4*>(cs.k_dst)[dst] = reinterpret_cast<const uint4*>(cs.k_src)[local];
        reinterpret_cast<uint4*>(cs.v_dst)[dst] = reinterpret_cast<const uint4*>(cs.v_src)[local];
    }
}
}  // namespace

cudaError_t launch_kv_commit(const CommitArgs& a, int sm_count, cudaStream_t st) {
    const int threads = 256;
    long long blocks = (a.total + threads - 1) / threads;
    const long long most = static_cast<long long>(sm_count > 0 ? sm_count : 148) * 8;
    if (blocks > most) blocks = most;
    if (blocks < 1) blocks = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(blocks));
    cfg.blockDim = dim3(threads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    cfg.numAttrs = overlap_launch_attribute(st, attr);
    cfg.attrs = attr;
    return cudaLaunchKernelEx(&cfg, kv_commit_kernel, a);
}
