// Confidence-threshold parallel unmasking: vocabulary-wide soft-max statistics and
// (Gumbel-perturbed) arg-max per MASKED row, then the per-rollout commit rule.
//
// Kernel 1 (unmask_partial_kernel): one CTA per (row, chunk).  A CTA streams one chunk of one
// row of logits from HBM exactly once with 16-byte loads, keeps it in registers, and
// reduces it to (max, sum exp, best perturbed score, its vocabulary id and logit).  Rows
// whose position is not MASKED exit at once, so only the rows the method needs are read.
// Kernel 2 (unmask_finalize_kernel): one CTA per rollout merges the chunk records of its
// rows, forms the confidences and applies the threshold / at-least-one rule.
#include "fdd_internal.h"

#include <math_constants.h>

namespace {

constexpr int kThreads = 256;
constexpr int kPerThread = kUnmaskChunk / kThreads;   // 32 vocabulary entries per thread

constexpr uint32_t kPhiloxM0 = 0xD2511F53u, kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u, kPhiloxW1 = 0xBB67AE85u;

// Philox4x32 with 10 rounds (Salmon et al., SC'11), written from the published round function.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        if (r > 0) { k.x += kPhiloxW0; k.y += kPhiloxW1; }
        const uint32_t hi0 = __umulhi(kPhiloxM0, c.x), lo0 = kPhiloxM0 * c.x;
        const uint32_t hi1 = __umulhi(kPhiloxM1, c.z), lo1 = kPhiloxM1 * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    }
    return c;
}

// g = -ln(-ln(u)), u = (k + 0.5) * 2^-23 with k the top 23 bits of the word; u is exact in fp32.
__device__ __forceinline__ float gumbel_from_bits(uint32_t k23) {
    const float u = (static_cast<float>(k23) + 0.5f) * 1.1920928955078125e-07f;
    return -logf(-logf(u));
}

template <typename T> struct LogitVec;
template <> struct LogitVec<__nv_bfloat16> {
    static constexpr int kVec = 8;
    __device__ static void load(const __nv_bfloat16* p, float* out) {
        const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            out[2 * i] = __uint_as_float(w[i] << 16);
            out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};
template <> struct LogitVec<float> {
    static constexpr int kVec = 4;
    __device__ static void load(const float* p, float* out) {
        const float4 raw = __ldcs(reinterpret_cast<const float4*>(p));
        out[0] = raw.x; out[1] = raw.y; out[2] = raw.z; out[3] = raw.w;
    }
    __device__ static float load1(const float* p) { return *p; }
};

struct Best {
    float score, logit;
    int index;
};
__device__ __forceinline__ Best better(const Best& a, const Best& b) {
    // larger score wins; equal scores -> lower vocabulary id
    if (b.score > a.score || (b.score == a.score && b.index < a.index)) return b;
    return a;
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
unmask_partial_kernel(const T* __restrict__ logits, const uint8_t* __restrict__ state,
                      const uint64_t* __restrict__ seeds, UnmaskPartial* __restrict__ partial,
                      int d, int vocab, int n_chunks, float temperature,
                      uint32_t block_idx, uint32_t step, int vec_ok) {
    const int row = blockIdx.x / n_chunks;
    if (state[row] != FDD_MASKED) return;
    const int chunk = blockIdx.x - row * n_chunks;
    const int tid = threadIdx.x;
    constexpr int kVec = LogitVec<T>::kVec;
    constexpr int kIter = kPerThread / kVec;

    __shared__ float g_upper[256];     // upper bound of the Gumbel value per top-8-bit bin
    __shared__ float red_max[kThreads / 32], red_sum[kThreads / 32];
    __shared__ Best red_best[kThreads / 32];

    const bool noisy = temperature != 0.0f;
    if (noisy) {
        const uint32_t k_hi = ((static_cast<uint32_t>(tid) + 1u) << 15) - 1u;
        g_upper[tid] = gumbel_from_bits(k_hi) + 1e-3f;
    }

    const T* row_ptr = logits + static_cast<size_t>(row) * vocab;
    const int chunk_base = chunk * kUnmaskChunk;

    float val[kPerThread];
#pragma unroll
    for (int it = 0; it < kIter; ++it) {
        const int v0 = chunk_base + (it * kThreads + tid) * kVec;
        if (vec_ok && v0 + kVec <= vocab) {
            LogitVec<T>::load(row_ptr + v0, &val[it * kVec]);
        } else {
#pragma unroll
            for (int j = 0; j < kVec; ++j)
                val[it * kVec + j] = (v0 + j < vocab) ? LogitVec<T>::load1(row_ptr + v0 + j) : -CUDART_INF_F;
        }
    }

    float m = -CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < kPerThread; ++i) m = fmaxf(m, val[i]);
    float s = 0.0f;
    if (m > -CUDART_INF_F) {
#pragma unroll
        for (int i = 0; i < kPerThread; ++i) s += __expf(val[i] - m);
    }

    Best best{-CUDART_INF_F, -CUDART_INF_F, 0x7FFFFFFF};
    if (!noisy) {
#pragma unroll
        for (int it = 0; it < kIter; ++it) {
#pragma unroll
            for (int j = 0; j < kVec; ++j) {
                const float l = val[it * kVec + j];
                if (l > best.score) best = Best{l, l, chunk_base + (it * kThreads + tid) * kVec + j};
            }
        }
    } else {
        __syncthreads();                       // g_upper ready
        const int fork = row / d, pos = row - fork * d;
        const uint64_t seed = seeds[fork];
        const uint2 key = make_uint2(static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32));
#pragma unroll
        for (int it = 0; it < kIter; ++it) {
            const int v0 = chunk_base + (it * kThreads + tid) * kVec;
#pragma unroll
            for (int q4 = 0; q4 < kVec / 4; ++q4) {
                const int vq = v0 + q4 * 4;
                if (vq >= vocab) continue;
                const uint4 r = philox4x32_10(make_uint4(static_cast<uint32_t>(vq >> 2), pos, step, block_idx), key);
                const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float l = val[it * kVec + q4 * 4 + j];
                    const uint32_t k23 = w[j] >> 9;
                    // cheap test first: even the largest Gumbel value of this bin cannot reach the best
                    const float bound = fmaf(temperature, g_upper[k23 >> 15], l);
                    if (bound >= best.score && l > -CUDART_INF_F) {
                        const float sc = fmaf(temperature, gumbel_from_bits(k23), l);
                        if (sc > best.score) best = Best{sc, l, vq + j};
                    }
                }
            }
        }
    }

    // block reduction
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float m2 = __shfl_xor_sync(0xFFFFFFFFu, m, off);
        const float s2 = __shfl_xor_sync(0xFFFFFFFFu, s, off);
        const float mn = fmaxf(m, m2);
        if (mn > -CUDART_INF_F) s = s * __expf(m - mn) + s2 * __expf(m2 - mn);
        m = mn;
        Best o;
        o.score = __shfl_xor_sync(0xFFFFFFFFu, best.score, off);
        o.logit = __shfl_xor_sync(0xFFFFFFFFu, best.logit, off);
        o.index = __shfl_xor_sync(0xFFFFFFFFu, best.index, off);
        best = better(best, o);
    }
    const int warp = tid >> 5, lane = tid & 31;
    if (lane == 0) { red_max[warp] = m; red_sum[warp] = s; red_best[warp] = best; }
    __syncthreads();
    if (tid == 0) {
        float M = red_max[0], S = red_sum[0];
        Best B = red_best[0];
        for (int w2 = 1; w2 < kThreads / 32; ++w2) {
            const float mn = fmaxf(M, red_max[w2]);
            if (mn > -CUDART_INF_F) S = S * __expf(M - mn) + red_sum[w2] * __expf(red_max[w2] - mn);
            M = mn;
            B = better(B, red_best[w2]);
        }
        UnmaskPartial out;
        out.row_max = M; out.sum_exp = S; out.best_score = B.score; out.best_logit = B.logit;
        out.best_index = B.index; out.pad[0] = out.pad[1] = out.pad[2] = 0;
        partial[static_cast<size_t>(row) * n_chunks + chunk] = out;
    }
}

__global__ void __launch_bounds__(128)
unmask_finalize_kernel(const UnmaskPartial* __restrict__ partial, int32_t* __restrict__ tokens,
                       uint8_t* __restrict__ state, int32_t* __restrict__ n_committed,
                       int32_t* __restrict__ n_left, float* __restrict__ conf_out,
                       int d, int n_chunks, float threshold) {
    const int fork = blockIdx.x;
    const int i = threadIdx.x;
    __shared__ float s_conf[128];
    __shared__ int s_masked, s_pass;
    if (i == 0) { s_masked = 0; s_pass = 0; }
    __syncthreads();

    const int row = fork * d + i;
    bool masked = false;
    float conf = -1.0f;
    int tok = 0;
    if (i < d) {
        masked = state[row] == FDD_MASKED;
        if (masked) {
            const UnmaskPartial* p = partial + static_cast<size_t>(row) * n_chunks;
            float M = -CUDART_INF_F;
            for (int c = 0; c < n_chunks; ++c) M = fmaxf(M, p[c].row_max);
            float S = 0.0f;
            Best B{-CUDART_INF_F, -CUDART_INF_F, 0x7FFFFFFF};
            for (int c = 0; c < n_chunks; ++c) {
                S += p[c].sum_exp * expf(p[c].row_max - M);
                B = better(B, Best{p[c].best_score, p[c].best_logit, p[c].best_index});
            }
            conf = expf(B.logit - M) / S;
            tok = B.index;
        }
        if (conf_out) conf_out[row] = masked ? conf : CUDART_NAN_F;
    }
    s_conf[i] = masked ? conf : -1.0f;
    const bool pass = masked && conf > threshold;
    if (masked) atomicAdd(&s_masked, 1);
    if (pass) atomicAdd(&s_pass, 1);
    __syncthreads();
    const int n_masked = s_masked, n_pass = s_pass;
    bool commit = pass;
    if (n_masked > 0 && n_pass == 0) {
        // at-least-one rule: the most confident MASKED position, lowest index on ties
        int best_i = -1;
        float best_c = -1.0f;
        for (int j = 0; j < d; ++j) {
            const float c = s_conf[j];
            if (c > best_c) { best_c = c; best_i = j; }
        }
        commit = (i == best_i);
    }
    if (commit && i < d) {
        tokens[row] = tok;
        state[row] = FDD_COMMITTED;
    }
    if (i == 0) {
        const int nc = (n_masked == 0) ? 0 : (n_pass > 0 ? n_pass : 1);
        n_committed[fork] = nc;
        n_left[fork] = n_masked - nc;
    }
}

}  // namespace

cudaError_t launch_unmask(fdd_ctx* ctx, const UnmaskProblem& p, cudaStream_t st, int* n_launches) {
    const int rows = p.n_forks * p.d;
    const int n_chunks = unmask_chunks(p.vocab);
    UnmaskPartial* partial = static_cast<UnmaskPartial*>(ctx->ws_unmask);
    const dim3 grid(static_cast<unsigned>(n_chunks) * static_cast<unsigned>(rows));
    if (p.logits_dtype == FDD_LOGITS_BF16) {
        const int vec_ok = (p.vocab % 8 == 0) && (reinterpret_cast<uintptr_t>(p.logits) % 16 == 0);
        unmask_partial_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(
            static_cast<const __nv_bfloat16*>(p.logits), p.state, p.seeds, partial, p.d, p.vocab,
            n_chunks, p.temperature, p.block_idx, p.step, vec_ok);
    } else {
        const int vec_ok = (p.vocab % 4 == 0) && (reinterpret_cast<uintptr_t>(p.logits) % 16 == 0);
        unmask_partial_kernel<float><<<grid, kThreads, 0, st>>>(
            static_cast<const float*>(p.logits), p.state, p.seeds, partial, p.d, p.vocab,
            n_chunks, p.temperature, p.block_idx, p.step, vec_ok);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    unmask_finalize_kernel<<<p.n_forks, 128, 0, st>>>(partial, p.tokens, p.state, p.n_committed,
                                                     p.n_left, p.conf, p.d, n_chunks, p.threshold);
    *n_launches += 2;
    return cudaGetLastError();
}

// -------------------------------------------------------------------------------------------------
// fdd_unmask_static: the same unmasking step for callers that must not allocate.
//
// Its scratch (the per (row, chunk) records) lives in a fixed device array that is part of the
// loaded library image, so the call needs no context, no fork set and no allocation of any kind.
// -------------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxRecords = FDD_UNMASK_STATIC_MAX_RECORDS;
constexpr int kStaticMaxDevices = 64;

// Held by every GPU that loads the library until the process exits (2 MiB).
static __device__ __align__(256) UnmaskPartial g_static_partials[kStaticMaxRecords];

// Device address of g_static_partials per device ordinal, resolved on first use.  In host code the
// array's name is only a handle for the runtime; the address a kernel can use must be asked for.
UnmaskPartial* g_static_ptr[kStaticMaxDevices];
bool g_static_ready[kStaticMaxDevices];

void put_error(char* err, size_t err_len, const char* text) {
    if (err && err_len) snprintf(err, err_len, "%s", text);
}

}  // namespace

extern "C" fdd_status fdd_unmask_static(const void* logits, int logits_dtype, int n_forks, int block_len,
                                        int vocab, int32_t* tokens, uint8_t* state, const uint64_t* seeds,
                                        float threshold, float temperature, uint32_t block_idx,
                                        uint32_t step, int32_t* n_committed, int32_t* n_left, float* conf,
                                        void* stream, char* err, size_t err_len) {
    if (!logits || !tokens || !state || !seeds || !n_committed || !n_left) {
        put_error(err, err_len, "fdd_unmask_static: a required pointer is NULL");
        return FDD_ERR_INVALID_ARG;
    }
    if (logits_dtype != FDD_LOGITS_F32 && logits_dtype != FDD_LOGITS_BF16) {
        put_error(err, err_len, "fdd_unmask_static: logits_dtype must be FDD_LOGITS_F32 or FDD_LOGITS_BF16");
        return FDD_ERR_INVALID_ARG;
    }
    if (n_forks < 1 || block_len < 1 || vocab < 1 || !(temperature >= 0.0f) || threshold != threshold) {
        put_error(err, err_len, "fdd_unmask_static: sizes must be >= 1, temperature >= 0, threshold not NaN");
        return FDD_ERR_INVALID_ARG;
    }
    if (block_len > 128) {
        put_error(err, err_len, "fdd_unmask_static: block_len above 128 is not supported");
        return FDD_ERR_UNSUPPORTED;
    }
    const long long records = static_cast<long long>(n_forks) * block_len * unmask_chunks(vocab);
    if (records > kStaticMaxRecords) {
        if (err && err_len)
            snprintf(err, err_len,
                     "fdd_unmask_static: n_forks * block_len * ceil(vocab / %d) = %lld exceeds the fixed scratch of %d records",
                     kUnmaskChunk, records, kStaticMaxRecords);
        return FDD_ERR_CAPACITY;
    }
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kStaticMaxDevices) {
        put_error(err, err_len, "fdd_unmask_static: no usable current CUDA device");
        return FDD_ERR_CUDA;
    }
    if (!g_static_ready[dev]) {
        // once per device, with that device current: resolve the array's device address
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_partials);
        if (e != cudaSuccess || !p) {
            if (err && err_len) snprintf(err, err_len, "fdd_unmask_static: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            return FDD_ERR_CUDA;
        }
        g_static_ptr[dev] = static_cast<UnmaskPartial*>(p);
        g_static_ready[dev] = true;
    }
    UnmaskPartial* partial = g_static_ptr[dev];
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int rows = n_forks * block_len;
    const int n_chunks = unmask_chunks(vocab);
    const dim3 grid(static_cast<unsigned>(n_chunks) * static_cast<unsigned>(rows));
    if (logits_dtype == FDD_LOGITS_BF16) {
        const int vec_ok = (vocab % 8 == 0) && (reinterpret_cast<uintptr_t>(logits) % 16 == 0);
        unmask_partial_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(
            static_cast<const __nv_bfloat16*>(logits), state, seeds, partial, block_len, vocab, n_chunks,
            temperature, block_idx, step, vec_ok);
    } else {
        const int vec_ok = (vocab % 4 == 0) && (reinterpret_cast<uintptr_t>(logits) % 16 == 0);
        unmask_partial_kernel<float><<<grid, kThreads, 0, st>>>(
            static_cast<const float*>(logits), state, seeds, partial, block_len, vocab, n_chunks,
            temperature, block_idx, step, vec_ok);
    }
    e = cudaGetLastError();
    if (e == cudaSuccess) {
        unmask_finalize_kernel<<<n_forks, 128, 0, st>>>(partial, tokens, state, n_committed, n_left, conf,
                                                       block_len, n_chunks, threshold);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) {
        if (err && err_len) snprintf(err, err_len, "fdd_unmask_static: launch failed: %s", cudaGetErrorString(e));
        return FDD_ERR_CUDA;
    }
    return FDD_OK;
}
