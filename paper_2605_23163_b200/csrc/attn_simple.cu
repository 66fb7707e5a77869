// Block-causal decode attention, CUDA-core version (fp32 math on bf16 inputs).
//
// One CTA handles 32 query rows of one (rollout, KV head): row r = i * G + g covers block
// position i and the g-th query head of the group.  It walks the keys of the shared prefix,
// the rollout's private suffix and the block itself in tiles of 32 with an online soft-max.
// This kernel serves every shape (any block length, head_dim 64/128, paged or contiguous
// prefix, causal-in-block masking); the tensor-core kernel takes over the shapes it supports.
#include "fdd_internal.h"

#include <math_constants.h>

namespace {

constexpr int kRows = 32;      // query rows per CTA
constexpr int kKeys = 32;      // keys per tile
constexpr int kThreadsA = 256; // 8 threads per row

template <int D>
struct SimpleSmem {
    float q[kRows][D + 1];
    float k[kKeys][D + 1];
    float v[kKeys][D];
    float p[kRows][kKeys + 1];
};

__device__ __forceinline__ const __nv_bfloat16* key_row(const AttnProblem& a, const __nv_bfloat16* prefix,
                                                        const __nv_bfloat16* suffix, const __nv_bfloat16* blk,
                                                        int f, int h, int j, int D) {
    if (j < a.prefix_len) {
        if (a.page_tokens == 0)
            return prefix + (static_cast<size_t>(h) * a.prefix_capacity + j) * D;
        const int page = a.page_table[j / a.page_tokens];
        return prefix + ((static_cast<size_t>(page) * a.n_kv_heads + h) * a.page_tokens + j % a.page_tokens) * D;
    }
    j -= a.prefix_len;
    if (j < a.suffix_len)
        return suffix + ((static_cast<size_t>(f) * a.n_kv_heads + h) * a.suffix_capacity + j) * D;
    j -= a.suffix_len;
    return blk + ((static_cast<size_t>(f) * a.d + j) * a.n_kv_heads + h) * D;
}

template <int D>
__global__ void __launch_bounds__(kThreadsA)
attn_simple_kernel(const AttnProblem a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SimpleSmem<D>& sm = *reinterpret_cast<SimpleSmem<D>*>(smem_raw);

    const int G = a.n_q_heads / a.n_kv_heads;
    const int R = a.d * G;
    const int r0 = blockIdx.x * kRows;
    const int h = blockIdx.y;      // KV head
    const int f = blockIdx.z;      // rollout
    if (a.gate != nullptr && a.gate[f] == 0) return;   // the whole CTA: this rollout sits the call out
    const int tid = threadIdx.x;
    const int rr = tid >> 3;       // local row
    const int t8 = tid & 7;
    const int r = r0 + rr;
    const bool row_ok = r < R;
    const int qi = row_ok ? r / G : 0;       // block position of this row
    const int qg = row_ok ? r - qi * G : 0;  // head inside the group
    const float qscale = a.scale * 1.4426950408889634f;

    // stage Q (scaled into the log2 domain)
    for (int e = tid; e < kRows * D; e += kThreadsA) {
        const int lr = e / D, c = e - lr * D;
        const int gr = r0 + lr;
        float val = 0.0f;
        if (gr < R) {
            const int i = gr / G, g = gr - i * G;
            val = __bfloat162float(a.q[((static_cast<size_t>(f) * a.d + i) * a.n_q_heads + h * G + g) * D + c]) * qscale;
        }
        sm.q[lr][c] = val;
    }

    constexpr int DV = D / 8;
    float o[DV];
#pragma unroll
    for (int x = 0; x < DV; ++x) o[x] = 0.0f;
    float m = -CUDART_INF_F, l = 0.0f;

    const int total = a.prefix_len + a.suffix_len + a.d;
    const int block_start = a.prefix_len + a.suffix_len;
    for (int j0 = 0; j0 < total; j0 += kKeys) {
        __syncthreads();   // previous tile fully consumed (also covers the Q staging)
        {   // load K and V tile: thread -> key tid / 8, slice tid % 8
            const int kj = tid >> 3, part = tid & 7;
            const int j = j0 + kj;
            constexpr int EPT = D / 8;   // elements per thread
            if (j < total) {
                const __nv_bfloat16* kp = key_row(a, a.prefix_k, a.suffix_k, a.k_blk, f, h, j, D) + part * EPT;
                const __nv_bfloat16* vp = key_row(a, a.prefix_v, a.suffix_v, a.v_blk, f, h, j, D) + part * EPT;
#pragma unroll
                for (int x = 0; x < EPT; x += 8) {
                    const uint4 kr = *reinterpret_cast<const uint4*>(kp + x);
                    const uint4 vr = *reinterpret_cast<const uint4*>(vp + x);
                    const uint32_t kw[4] = {kr.x, kr.y, kr.z, kr.w};
                    const uint32_t vw[4] = {vr.x, vr.y, vr.z, vr.w};
#pragma unroll
                    for (int y = 0; y < 4; ++y) {
                        sm.k[kj][part * EPT + x + 2 * y] = __uint_as_float(kw[y] << 16);
                        sm.k[kj][part * EPT + x + 2 * y + 1] = __uint_as_float(kw[y] & 0xFFFF0000u);
                        sm.v[kj][part * EPT + x + 2 * y] = __uint_as_float(vw[y] << 16);
                        sm.v[kj][part * EPT + x + 2 * y + 1] = __uint_as_float(vw[y] & 0xFFFF0000u);
                    }
                }
            } else {
#pragma unroll
                for (int x = 0; x < EPT; ++x) { sm.k[kj][part * EPT + x] = 0.0f; sm.v[kj][part * EPT + x] = 0.0f; }
            }
        }
        __syncthreads();

        // scores: this thread owns keys c = t8 * 4 + {0..3} of row rr
        float s[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll 8
        for (int c = 0; c < D; ++c) {
            const float qv = sm.q[rr][c];
#pragma unroll
            for (int y = 0; y < 4; ++y) s[y] = fmaf(qv, sm.k[t8 * 4 + y][c], s[y]);
        }
        float tmax = -CUDART_INF_F;
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const int j = j0 + t8 * 4 + y;
            bool visible = j < total;
            if (a.causal_in_block && j >= block_start && (j - block_start) > qi) visible = false;
            if (!visible) s[y] = -CUDART_INF_F;
            tmax = fmaxf(tmax, s[y]);
        }
#pragma unroll
        for (int off = 1; off < 8; off <<= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xFFFFFFFFu, tmax, off));
        const float m_new = fmaxf(m, tmax);
        float alpha = 1.0f, psum = 0.0f;
        if (m_new > -CUDART_INF_F) {
            alpha = exp2f(m - m_new);
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                const float pv = exp2f(s[y] - m_new);
                sm.p[rr][t8 * 4 + y] = pv;
                psum += pv;
            }
        } else {
#pragma unroll
            for (int y = 0; y < 4; ++y) sm.p[rr][t8 * 4 + y] = 0.0f;
        }
#pragma unroll
        for (int off = 1; off < 8; off <<= 1) psum += __shfl_xor_sync(0xFFFFFFFFu, psum, off);
        l = l * alpha + psum;
        m = m_new;
        __syncwarp();
#pragma unroll
        for (int x = 0; x < DV; ++x) o[x] *= alpha;
        for (int c = 0; c < kKeys; ++c) {
            const float pv = sm.p[rr][c];
#pragma unroll
            for (int x = 0; x < DV; ++x) o[x] = fmaf(pv, sm.v[c][x * 8 + t8], o[x]);
        }
    }

    if (row_ok) {
        const float inv = l > 0.0f ? 1.0f / l : 0.0f;
        __nv_bfloat16* op = a.out + ((static_cast<size_t>(f) * a.d + qi) * a.n_q_heads + h * G + qg) * D;
#pragma unroll
        for (int x = 0; x < DV; ++x) op[x * 8 + t8] = __float2bfloat16_rn(o[x] * inv);
    }
}

}  // namespace

cudaError_t launch_attention_simple(const AttnProblem& p, int head_dim, cudaStream_t st) {
    const int G = p.n_q_heads / p.n_kv_heads;
    const int R = p.d * G;
    const dim3 grid((R + kRows - 1) / kRows, p.n_kv_heads, p.n_forks);
    if (head_dim == 128) {
        const size_t bytes = sizeof(SimpleSmem<128>);
        cudaError_t e = cudaFuncSetAttribute(attn_simple_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (e != cudaSuccess) return e;
        attn_simple_kernel<128><<<grid, kThreadsA, bytes, st>>>(p);
    } else {
        const size_t bytes = sizeof(SimpleSmem<64>);
        cudaError_t e = cudaFuncSetAttribute(attn_simple_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        if (e != cudaSuccess) return e;
        attn_simple_kernel<64><<<grid, kThreadsA, bytes, st>>>(p);
    }
    return cudaGetLastError();
}
