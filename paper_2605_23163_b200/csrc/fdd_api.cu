// Host side of the C ABI: argument validation, fork-set metadata, kernel dispatch.
#include "fdd_internal.h"

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>


namespace {

fdd_status fail(fdd_ctx* ctx, fdd_status code, const char* fmt, ...) {
    if (ctx) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof(buf), fmt, ap);
        va_end(ap);
        ctx->last_error = buf;
    }
    return code;
}

fdd_status cuda_fail(fdd_ctx* ctx, cudaError_t e, const char* what) {
    return fail(ctx, FDD_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

// Seeds travel to the device as kernel arguments: stream-ordered like everything else, no
// staging buffer, no allocation, no synchronisation.
constexpr size_t kMapPoolEntries = 64;
constexpr int kSeedsPerLaunch = 240;
struct SeedChunk {
    uint64_t value[kSeedsPerLaunch];
    uint64_t* dst[kSeedsPerLaunch];
    int n;
};

__global__ void seed_store_kernel(const __grid_constant__ SeedChunk c) {
    const int i = threadIdx.x;
    if (i < c.n) *c.dst[i] = c.value[i];
}

// Store the seeds of every set of the call that has not been used for sampling yet.
cudaError_t ensure_seeds(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, cudaStream_t st) {
    SeedChunk& chunk = *static_cast<SeedChunk*>(ctx->seed_chunk);   // 4 KB, kept off the stack, one per context
    chunk.n = 0;
    auto flush = [&]() -> cudaError_t {
        if (chunk.n == 0) return cudaSuccess;
        seed_store_kernel<<<1, 256, 0, st>>>(chunk);
        ctx->launches += 1;
        chunk.n = 0;
        return cudaGetLastError();
    };
    for (int s = 0; s < n_sets; ++s) {
        fdd_forkset* fs = sets[s];
        if (fs->seeds_on_device) continue;
        for (int f = 0; f < fs->n_forks; ++f) {
            chunk.value[chunk.n] = fs->h_seeds[f];
            chunk.dst[chunk.n] = fs->d_seeds + f;
            if (++chunk.n == kSeedsPerLaunch) {
                cudaError_t e = flush();
                if (e != cudaSuccess) return e;
            }
        }
        fs->seeds_on_device = true;
    }
    return flush();
}

bool set_alive(const fdd_ctx* ctx, const fdd_forkset* s) {
    return s && std::find(ctx->live_sets.begin(), ctx->live_sets.end(), s) != ctx->live_sets.end();
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Common checks of a batched call; fills total rollouts and per-set row offsets.
fdd_status check_sets(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, const int32_t* block_len,
                      int* total_forks) {
    if (!sets || n_sets < 1 || !block_len) return fail(ctx, FDD_ERR_INVALID_ARG, "sets/block_len missing or n_sets < 1");
    int total = 0;
    for (int s = 0; s < n_sets; ++s) {
        if (!set_alive(ctx, sets[s])) return fail(ctx, FDD_ERR_STATE, "fork set %d is not a live set of this context", s);
        if (block_len[s] < 1 || block_len[s] > ctx->cfg.max_block)
            return fail(ctx, FDD_ERR_CAPACITY, "block_len[%d] = %d outside [1, %d]", s, block_len[s], ctx->cfg.max_block);
        total += sets[s]->n_forks;
    }
    if (total > ctx->cfg.max_forks)
        return fail(ctx, FDD_ERR_CAPACITY, "%d rollouts in one call exceed max_forks = %d", total, ctx->cfg.max_forks);
    *total_forks = total;
    return FDD_OK;
}

}  // namespace

extern "C" {

fdd_status fdd_create(const fdd_config* cfg, fdd_ctx** out) {
    if (!out) return FDD_ERR_INVALID_ARG;
    *out = nullptr;
    if (!cfg) return FDD_ERR_INVALID_ARG;
    if (cfg->n_q_heads < 1 || cfg->n_kv_heads < 1 || cfg->vocab < 1 || cfg->n_layers < 1 ||
        cfg->max_block < 1 || cfg->max_forks < 1 || cfg->page_tokens < 0)
        return FDD_ERR_INVALID_ARG;
    if (cfg->logits_dtype != FDD_LOGITS_F32 && cfg->logits_dtype != FDD_LOGITS_BF16) return FDD_ERR_INVALID_ARG;
    if (cfg->head_dim != 64 && cfg->head_dim != 128) return FDD_ERR_UNSUPPORTED;
    if (cfg->n_q_heads % cfg->n_kv_heads != 0 || cfg->n_q_heads / cfg->n_kv_heads > 16) return FDD_ERR_UNSUPPORTED;
    if (cfg->max_block > 128) return FDD_ERR_UNSUPPORTED;
    if (cfg->page_tokens != 0 && cfg->page_tokens != 64) return FDD_ERR_UNSUPPORTED;

    fdd_ctx* ctx = new (std::nothrow) fdd_ctx();
    if (!ctx) return FDD_ERR_CUDA;
    ctx->cfg = *cfg;
    cudaError_t e = cudaGetDevice(&ctx->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->d_status, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMallocHost(&ctx->h_status, sizeof(int));
    for (int i = 0; i < 2 && e == cudaSuccess; ++i) {
        const size_t bytes = sizeof(int2) * static_cast<size_t>(cfg->max_forks > 0 ? cfg->max_forks : 1);
        e = cudaHostAlloc(&ctx->h_counts[i], bytes, cudaHostAllocMapped);
        if (e == cudaSuccess) {
            memset(ctx->h_counts[i], 0, bytes);
            e = cudaHostGetDevicePointer(&ctx->d_counts[i], ctx->h_counts[i], 0);
        }
    }
    ctx->seed_chunk = new (std::nothrow) SeedChunk();
    if (!ctx->seed_chunk && e == cudaSuccess) e = cudaErrorMemoryAllocation;
    if (e == cudaSuccess) {
        const long long max_rows = static_cast<long long>(cfg->max_forks) * cfg->max_block;
        ctx->ws_unmask_bytes = unmask_workspace_bytes(cfg->vocab, static_cast<int>(std::min<long long>(max_rows, kUnmaskMaxRows)));
        e = cudaMalloc(&ctx->ws_unmask, ctx->ws_unmask_bytes);
    }
    if (e == cudaSuccess) {
        ctx->attn_max_ctas = ctx->sm_count > 0 ? ctx->sm_count : 148;
        ctx->ws_attn_bytes = attention_ptc_workspace_bytes(cfg->head_dim, ctx->attn_max_ctas);
        e = cudaMalloc(&ctx->ws_attn, ctx->ws_attn_bytes);
    }
    if (e == cudaSuccess) {
        // one counter per attention unit: (KV head, pair of 128-row tiles, rollout)
        const int G = cfg->n_q_heads / cfg->n_kv_heads;
        const int row_pairs = (cfg->max_block * G + 255) / 256;
        ctx->attn_max_units = cfg->n_kv_heads * row_pairs * cfg->max_forks;
        // two counters per unit: pieces written, CTAs done with their share of the merge
        e = cudaMalloc(&ctx->attn_unit_count, sizeof(int) * 2 * ctx->attn_max_units);
        if (e == cudaSuccess) e = cudaMemset(ctx->attn_unit_count, 0, sizeof(int) * 2 * ctx->attn_max_units);
    }
    if (e != cudaSuccess) {
        fdd_destroy(ctx);
        return FDD_ERR_CUDA;
    }
    *out = ctx;
    return FDD_OK;
}

void fdd_destroy(fdd_ctx* ctx) {
    if (!ctx) return;
    for (fdd_forkset* s : ctx->live_sets) {
        if (s->d_seeds) cudaFree(s->d_seeds);
        delete s;
    }
    for (const fdd_ctx::SeedBuf& b : ctx->seed_pool) cudaFree(b.ptr);
    for (const fdd_ctx::JmtWeights& j : ctx->jmt_weights) cudaFree(j.d_weights);
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->h_status) cudaFreeHost(ctx->h_status);
    for (int i = 0; i < 2; ++i)
        if (ctx->h_counts[i]) cudaFreeHost(ctx->h_counts[i]);
    if (ctx->ws_unmask) cudaFree(ctx->ws_unmask);
    if (ctx->ws_attn) cudaFree(ctx->ws_attn);
    if (ctx->attn_unit_count) cudaFree(ctx->attn_unit_count);
    delete static_cast<SeedChunk*>(ctx->seed_chunk);
    delete ctx;
}

const char* fdd_last_error(const fdd_ctx* ctx) { return ctx ? ctx->last_error.c_str() : "null context"; }

uint64_t fdd_launch_count(const fdd_ctx* ctx) { return ctx ? ctx->launches : 0; }

fdd_status fdd_fork(fdd_ctx* ctx, const void* const* prefix_k, const void* const* prefix_v,
                    const int32_t* page_table, int prefix_len, int prefix_capacity,
                    int n_forks, const uint64_t* seeds,
                    void* const* suffix_k, void* const* suffix_v, int suffix_capacity,
                    fdd_forkset** out) {
    if (!ctx) return FDD_ERR_INVALID_ARG;
    if (!out) return fail(ctx, FDD_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (!prefix_k || !prefix_v || !seeds || !suffix_k || !suffix_v)
        return fail(ctx, FDD_ERR_INVALID_ARG, "a pointer array is NULL");
    if (prefix_len < 0 || prefix_capacity < 0 || suffix_capacity < 0)
        return fail(ctx, FDD_ERR_INVALID_ARG, "negative length or capacity");
    if (n_forks < 1 || n_forks > ctx->cfg.max_forks)
        return fail(ctx, FDD_ERR_CAPACITY, "n_forks = %d outside [1, %d]", n_forks, ctx->cfg.max_forks);
    const int pt = ctx->cfg.page_tokens;
    if (pt == 0) {
        if (page_table) return fail(ctx, FDD_ERR_INVALID_ARG, "page_table given but the context is configured contiguous");
        if (prefix_len > prefix_capacity)
            return fail(ctx, FDD_ERR_CAPACITY, "prefix_len %d exceeds prefix_capacity %d", prefix_len, prefix_capacity);
    } else {
        if (!page_table && prefix_len > 0) return fail(ctx, FDD_ERR_INVALID_ARG, "paged context needs a page_table");
        if ((prefix_len + pt - 1) / pt > prefix_capacity)
            return fail(ctx, FDD_ERR_CAPACITY, "prefix_len %d needs more than %d pages", prefix_len, prefix_capacity);
    }
    for (int l = 0; l < ctx->cfg.n_layers; ++l) {
        if ((prefix_len > 0 && (!prefix_k[l] || !prefix_v[l])) || (suffix_capacity > 0 && (!suffix_k[l] || !suffix_v[l])))
            return fail(ctx, FDD_ERR_INVALID_ARG, "NULL cache pointer for layer %d", l);
        if (!aligned16(prefix_k[l]) || !aligned16(prefix_v[l]) || !aligned16(suffix_k[l]) || !aligned16(suffix_v[l]))
            return fail(ctx, FDD_ERR_INVALID_ARG, "cache pointer of layer %d is not 16-byte aligned", l);
    }
    fdd_forkset* s = new (std::nothrow) fdd_forkset();
    if (!s) return fail(ctx, FDD_ERR_CUDA, "out of host memory");
    s->ctx = ctx;
    s->n_forks = n_forks;
    s->prefix_len = prefix_len;
    s->prefix_capacity = prefix_capacity;
    s->page_table = page_table;
    s->prefix_k.assign(prefix_k, prefix_k + ctx->cfg.n_layers);
    s->prefix_v.assign(prefix_v, prefix_v + ctx->cfg.n_layers);
    s->suffix_k.assign(suffix_k, suffix_k + ctx->cfg.n_layers);
    s->suffix_v.assign(suffix_v, suffix_v + ctx->cfg.n_layers);
    s->suffix_capacity = suffix_capacity;
    s->suffix_len = 0;
    // the tensor maps of an earlier set over the same caches serve again
    for (size_t i = 0; i < ctx->map_pool.size(); ++i) {
        TcMapPoolEntry& m = ctx->map_pool[i];
        if (m.n_forks == n_forks && m.prefix_len == prefix_len && m.prefix_capacity == prefix_capacity &&
            m.suffix_capacity == suffix_capacity && m.prefix_k == s->prefix_k && m.prefix_v == s->prefix_v &&
            m.suffix_k == s->suffix_k && m.suffix_v == s->suffix_v) {
            s->map_cache = std::move(m.maps);
            ctx->map_pool.erase(ctx->map_pool.begin() + i);
            break;
        }
    }
    s->map_cache.resize(ctx->cfg.n_layers);
    s->h_seeds.assign(seeds, seeds + n_forks);
    // A seed buffer left by a freed set serves again (the smallest that is large enough); only a
    // context that has never held this many rollouts allocates.
    int best = -1;
    for (size_t i = 0; i < ctx->seed_pool.size(); ++i)
        if (ctx->seed_pool[i].cap >= n_forks && (best < 0 || ctx->seed_pool[i].cap < ctx->seed_pool[best].cap))
            best = static_cast<int>(i);
    if (best >= 0) {
        s->d_seeds = ctx->seed_pool[best].ptr;
        s->seed_cap = ctx->seed_pool[best].cap;
        ctx->seed_pool.erase(ctx->seed_pool.begin() + best);
    } else {
        s->seed_cap = std::max(n_forks, 64);
        cudaError_t e = cudaMalloc(&s->d_seeds, sizeof(uint64_t) * s->seed_cap);
        if (e != cudaSuccess) {
            delete s;
            return cuda_fail(ctx, e, "fdd_fork seeds");
        }
    }
    ctx->live_sets.push_back(s);
    *out = s;
    return FDD_OK;
}

fdd_status fdd_forkset_free(fdd_ctx* ctx, fdd_forkset* set) {
    if (!ctx) return FDD_ERR_INVALID_ARG;
    auto it = std::find(ctx->live_sets.begin(), ctx->live_sets.end(), set);
    if (!set || it == ctx->live_sets.end()) return fail(ctx, FDD_ERR_STATE, "fork set is not live (double free?)");
    ctx->live_sets.erase(it);
    // Work of the set may still be in flight: the buffer is not freed (that would wait for the
    // device) but kept; whoever gets it next writes it in stream order, after that work.
    ctx->seed_pool.push_back({set->d_seeds, set->seed_cap});
    if (ctx->map_pool.size() >= kMapPoolEntries) ctx->map_pool.erase(ctx->map_pool.begin());
    ctx->map_pool.push_back({std::move(set->prefix_k), std::move(set->prefix_v), std::move(set->suffix_k),
                             std::move(set->suffix_v), set->n_forks, set->prefix_len, set->prefix_capacity,
                             set->suffix_capacity, std::move(set->map_cache)});
    delete set;
    return FDD_OK;
}

int fdd_forkset_suffix_len(const fdd_forkset* set) { return set ? set->suffix_len : FDD_ERR_INVALID_ARG; }

fdd_status fdd_forkset_reset(fdd_ctx* ctx, fdd_forkset* set) {
    if (!ctx) return FDD_ERR_INVALID_ARG;
    if (!set_alive(ctx, set)) return fail(ctx, FDD_ERR_STATE, "fork set is not live");
    set->suffix_len = 0;
    return FDD_OK;
}

fdd_status fdd_block_attn(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, int layer,
                          const void* q, const void* k_blk, const void* v_blk, void* out,
                          const int32_t* block_len, float scale, int causal_in_block, void* stream) {
    return fdd_block_attn_gated(ctx, sets, n_sets, layer, q, k_blk, v_blk, out, block_len, scale, causal_in_block,
                                nullptr, stream);
}

fdd_status fdd_block_attn_gated(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, int layer,
                                const void* q, const void* k_blk, const void* v_blk, void* out,
                                const int32_t* block_len, float scale, int causal_in_block,
                                const int32_t* gate, void* stream) {
    CallRange range("fdd_block_attn");
    if (!ctx) return FDD_ERR_INVALID_ARG;
    int total = 0;
    fdd_status st = check_sets(ctx, sets, n_sets, block_len, &total);
    if (st != FDD_OK) return st;
    if (!q || !k_blk || !v_blk || !out) return fail(ctx, FDD_ERR_INVALID_ARG, "q/k_blk/v_blk/out is NULL");
    if (!aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) || (reinterpret_cast<uintptr_t>(out) & 31u) != 0)
        return fail(ctx, FDD_ERR_INVALID_ARG, "q/k_blk/v_blk must be 16-byte aligned, out 32-byte aligned");
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, FDD_ERR_SHAPE, "layer %d outside [0, %d)", layer, ctx->cfg.n_layers);
    if (!(scale > 0.0f)) return fail(ctx, FDD_ERR_INVALID_ARG, "scale must be positive");
    if (gate && total > kAttnMaxGatedForks)
        return fail(ctx, FDD_ERR_CAPACITY, "%d rollouts in one gated call exceed %d", total, kAttnMaxGatedForks);
    const fdd_config& c = ctx->cfg;
    cudaStream_t st_ = static_cast<cudaStream_t>(stream);
    size_t q_off = 0, kv_off = 0;
    int fork_off = 0;
    std::vector<AttnProblem> tc_probs;
    std::vector<TcMapCache*> tc_caches;
    for (int s = 0; s < n_sets; ++s) {
        fdd_forkset* fs = sets[s];
        AttnProblem p;
        p.q = static_cast<const __nv_bfloat16*>(q) + q_off;
        p.k_blk = static_cast<const __nv_bfloat16*>(k_blk) + kv_off;
        p.v_blk = static_cast<const __nv_bfloat16*>(v_blk) + kv_off;
        p.out = static_cast<__nv_bfloat16*>(out) + q_off;
        p.prefix_k = static_cast<const __nv_bfloat16*>(fs->prefix_k[layer]);
        p.prefix_v = static_cast<const __nv_bfloat16*>(fs->prefix_v[layer]);
        p.page_table = fs->page_table;
        p.suffix_k = static_cast<const __nv_bfloat16*>(fs->suffix_k[layer]);
        p.suffix_v = static_cast<const __nv_bfloat16*>(fs->suffix_v[layer]);
        p.n_forks = fs->n_forks;
        p.d = block_len[s];
        p.n_q_heads = c.n_q_heads;
        p.n_kv_heads = c.n_kv_heads;
        p.prefix_len = fs->prefix_len;
        p.prefix_capacity = fs->prefix_capacity;
        p.page_tokens = c.page_tokens;
        p.suffix_len = fs->suffix_len;
        p.suffix_capacity = fs->suffix_capacity;
        p.causal_in_block = causal_in_block ? 1 : 0;
        p.scale = scale;
        p.gate = gate ? gate + fork_off : nullptr;
        fork_off += fs->n_forks;
        if (attention_tc_supported(p, c.head_dim)) {
            // the tensor-core kernel takes many scenes per launch
            tc_probs.push_back(p);
            tc_caches.push_back(&fs->map_cache[layer]);
        } else {
            // the CUDA-core kernel covers the remaining shapes (GQA groups that are not a power of two)
            cudaError_t e = launch_attention_simple(p, c.head_dim, st_);
            ctx->launches += 1;
            if (e != cudaSuccess) return cuda_fail(ctx, e, "fdd_block_attn launch");
        }
        q_off += static_cast<size_t>(fs->n_forks) * p.d * c.n_q_heads * c.head_dim;
        kv_off += static_cast<size_t>(fs->n_forks) * p.d * c.n_kv_heads * c.head_dim;
    }
    for (size_t first = 0; first < tc_probs.size(); first += kTcMaxSets) {
        const int n = static_cast<int>(std::min<size_t>(kTcMaxSets, tc_probs.size() - first));
        int n_launches = 0;
        cudaError_t e = launch_attention_ptc(ctx, tc_probs.data() + first, tc_caches.data() + first, n, c.head_dim, st_,
                                             &n_launches);
        ctx->launches += n_launches;
        if (e != cudaSuccess) return cuda_fail(ctx, e, "fdd_block_attn launch");
    }
    return FDD_OK;
}

static fdd_status unmask_like(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, const void* logits,
                              int32_t* tokens, uint8_t* state, const int32_t* block_len,
                              float threshold, float temperature, uint32_t block_idx, uint32_t step,
                              int32_t* n_committed, int32_t* n_left, float* conf, void* stream, int mode,
                              uint32_t* step_counter = nullptr) {
    if (!ctx) return FDD_ERR_INVALID_ARG;
    int total = 0;
    fdd_status st = check_sets(ctx, sets, n_sets, block_len, &total);
    if (st != FDD_OK) return st;
    if (!logits || !tokens || !state || !n_committed || !n_left)
        return fail(ctx, FDD_ERR_INVALID_ARG, "logits/tokens/state/n_committed/n_left is NULL");
    if (!(temperature >= 0.0f)) return fail(ctx, FDD_ERR_INVALID_ARG, "temperature must be >= 0");
    if (threshold != threshold) return fail(ctx, FDD_ERR_INVALID_ARG, "threshold is NaN");
    const fdd_config& c = ctx->cfg;
    const size_t esz = c.logits_dtype == FDD_LOGITS_BF16 ? 2 : 4;
    if (temperature > 0.0f) {
        cudaError_t e = ensure_seeds(ctx, sets, n_sets, static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) return cuda_fail(ctx, e, "seed upload");
    }
    // Sets go to the kernels in groups of at most kUnmaskMaxSets sets and kUnmaskMaxRows rows.
    size_t row_off = 0;
    int fork_off = 0;
    int s = 0;
    while (s < n_sets) {
        UnmaskProblem p;
        p.sets.n_sets = 0;
        p.sets.row_off[0] = 0;
        p.sets.fork_off[0] = 0;
        while (s < n_sets && p.sets.n_sets < kUnmaskMaxSets) {
            const fdd_forkset* fs = sets[s];
            const int rows = fs->n_forks * block_len[s];
            if (rows > kUnmaskMaxRows)
                return fail(ctx, FDD_ERR_CAPACITY, "set %d: %d rollouts x %d positions exceed %d rows per set", s,
                            fs->n_forks, block_len[s], kUnmaskMaxRows);
            const int k = p.sets.n_sets;
            if (p.sets.row_off[k] + rows > kUnmaskMaxRows) break;
            p.sets.d[k] = block_len[s];
            p.sets.seeds[k] = fs->d_seeds;
            p.sets.row_off[k + 1] = p.sets.row_off[k] + rows;
            p.sets.fork_off[k + 1] = p.sets.fork_off[k] + fs->n_forks;
            ++p.sets.n_sets;
            ++s;
        }
        p.logits = static_cast<const char*>(logits) + row_off * c.vocab * esz;
        p.tokens = tokens + row_off;
        p.state = state + row_off;
        p.n_committed = n_committed + fork_off;
        p.n_left = n_left + fork_off;
        p.conf = conf ? conf + row_off : nullptr;
        p.vocab = c.vocab;
        p.logits_dtype = c.logits_dtype;
        p.threshold = threshold;
        p.temperature = temperature;
        p.block_idx = block_idx;
        p.step = step;
        p.step_counter = step_counter;
        p.bump_counter = (step_counter != nullptr && s == n_sets) ? 1 : 0;      // the last group of the call advances it
        p.left_mirror = (mode == 0 && ctx->unmask_left_mirror) ? ctx->unmask_left_mirror + fork_off : nullptr;
        p.mirror_stamp = ctx->unmask_mirror_stamp;
        int n_launches = 0;
        cudaError_t e = launch_unmask(ctx, p, static_cast<cudaStream_t>(stream), &n_launches, mode);
        ctx->launches += n_launches;
        if (e != cudaSuccess) return cuda_fail(ctx, e, "fdd_unmask launch");
        row_off += static_cast<size_t>(p.sets.row_off[p.sets.n_sets]);
        fork_off += p.sets.fork_off[p.sets.n_sets];
    }
    return FDD_OK;
}

fdd_status fdd_unmask(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, const void* logits,
                      int32_t* tokens, uint8_t* state, const int32_t* block_len,
                      float threshold, float temperature, uint32_t block_idx, uint32_t step,
                      int32_t* n_committed, int32_t* n_left, float* conf, void* stream) {
    CallRange range("fdd_unmask");
    return unmask_like(ctx, sets, n_sets, logits, tokens, state, block_len, threshold, temperature, block_idx, step,
                       n_committed, n_left, conf, stream, 0);
}

fdd_status fdd_unmask_counted(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, const void* logits,
                              int32_t* tokens, uint8_t* state, const int32_t* block_len,
                              float threshold, float temperature, uint32_t block_idx, uint32_t* step_counter,
                              int32_t* n_committed, int32_t* n_left, float* conf, void* stream) {
    CallRange range("fdd_unmask_counted");
    if (ctx && !step_counter) return fail(ctx, FDD_ERR_INVALID_ARG, "step_counter is NULL");
    return unmask_like(ctx, sets, n_sets, logits, tokens, state, block_len, threshold, temperature, block_idx, 0u,
                       n_committed, n_left, conf, stream, 0, step_counter);
}

fdd_status fdd_ss_draft(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, const void* logits,
                        int32_t* tokens, uint8_t* state, const int32_t* block_len,
                        float temperature, uint32_t block_idx, uint32_t step,
                        int32_t* n_drafted, int32_t* n_left, void* stream) {
    CallRange range("fdd_ss_draft");
    // every MASKED position passes a threshold below any probability
    return unmask_like(ctx, sets, n_sets, logits, tokens, state, block_len, -1.0f, temperature, block_idx, step,
                       n_drafted, n_left, nullptr, stream, 1);
}

fdd_status fdd_ss_accept(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, const void* ar_logits,
                         int32_t* tokens, uint8_t* state, const int32_t* block_len,
                         float temperature, uint32_t block_idx, uint32_t step,
                         int32_t* n_accepted, int32_t* n_left, void* stream) {
    CallRange range("fdd_ss_accept");
    return unmask_like(ctx, sets, n_sets, ar_logits, tokens, state, block_len, 0.0f, temperature, block_idx, step,
                       n_accepted, n_left, nullptr, stream, 2);
}

// Common body of fdd_kv_commit (to_prefix = false) and fdd_prefix_extend (to_prefix = true).
static fdd_status commit_like(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, int layer,
                              const void* k_blk, const void* v_blk, const int32_t* block_len,
                              int advance, void* stream, bool to_prefix) {
    if (!ctx) return FDD_ERR_INVALID_ARG;
    int total = 0;
    fdd_status st = check_sets(ctx, sets, n_sets, block_len, &total);
    if (st != FDD_OK) return st;
    if (!k_blk || !v_blk) return fail(ctx, FDD_ERR_INVALID_ARG, "k_blk/v_blk is NULL");
    if (!aligned16(k_blk) || !aligned16(v_blk)) return fail(ctx, FDD_ERR_INVALID_ARG, "k_blk/v_blk must be 16-byte aligned");
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, FDD_ERR_SHAPE, "layer %d outside [0, %d)", layer, ctx->cfg.n_layers);
    const fdd_config& c = ctx->cfg;
    for (int s = 0; s < n_sets; ++s) {
        const fdd_forkset* fs = sets[s];
        if (!to_prefix) {
            if (fs->suffix_len + block_len[s] > fs->suffix_capacity)
                return fail(ctx, FDD_ERR_CAPACITY, "set %d: suffix %d + block %d exceeds capacity %d", s,
                            fs->suffix_len, block_len[s], fs->suffix_capacity);
            continue;
        }
        if (fs->n_forks != 1)
            return fail(ctx, FDD_ERR_STATE, "set %d has %d rollouts: only a set of one rollout extends its prefix", s, fs->n_forks);
        if (fs->suffix_len != 0)
            return fail(ctx, FDD_ERR_STATE, "set %d has a private suffix of %d tokens: the prefix must stay in front of it", s, fs->suffix_len);
        const int need = fs->prefix_len + block_len[s];
        const bool fits = c.page_tokens == 0 ? need <= fs->prefix_capacity
                                             : (need + c.page_tokens - 1) / c.page_tokens <= fs->prefix_capacity;
        if (!fits)
            return fail(ctx, FDD_ERR_CAPACITY, "set %d: prefix %d + block %d exceeds the cache (%d %s)", s, fs->prefix_len,
                        block_len[s], fs->prefix_capacity, c.page_tokens ? "pages" : "tokens");
        if (c.page_tokens != 0 && !fs->page_table)
            return fail(ctx, FDD_ERR_INVALID_ARG, "set %d: a paged prefix needs its page table", s);
    }
    size_t kv_off = 0;
    for (int first = 0; first < n_sets; first += kCommitMaxSets) {
        CommitArgs a;
        a.n = std::min(kCommitMaxSets, n_sets - first);
        a.n_kv_heads = c.n_kv_heads;
        a.vec_per_row = c.head_dim / 8;
        a.status = ctx->d_status;
        a.total = 0;
        for (int k = 0; k < a.n; ++k) {
            fdd_forkset* fs = sets[first + k];
            CommitSet& cs = a.set[k];
            cs.k_src = static_cast<const __nv_bfloat16*>(k_blk) + kv_off;
            cs.v_src = static_cast<const __nv_bfloat16*>(v_blk) + kv_off;
            cs.n_forks = fs->n_forks;
            cs.d = block_len[first + k];
            cs.page_table = fs->page_table;
            cs.page_tokens = c.page_tokens > 0 ? c.page_tokens : 1;
            if (to_prefix) {
                // the prefix caches are the caller's and read-only for every other call
                cs.k_dst = const_cast<void*>(fs->prefix_k[layer]);
                cs.v_dst = const_cast<void*>(fs->prefix_v[layer]);
                cs.len = fs->prefix_len;
                cs.cap = fs->prefix_capacity;
                cs.mode = c.page_tokens == 0 ? kCommitPrefix : kCommitPagedPrefix;
            } else {
                cs.k_dst = fs->suffix_k[layer];
                cs.v_dst = fs->suffix_v[layer];
                cs.len = fs->suffix_len;
                cs.cap = fs->suffix_capacity;
                cs.mode = kCommitSuffix;
            }
            cs.vec_begin = a.total;
            const size_t elems = static_cast<size_t>(fs->n_forks) * cs.d * c.n_kv_heads * c.head_dim;
            a.total += static_cast<long long>(elems / 8);
            kv_off += elems;
        }
        cudaError_t e = launch_kv_commit(a, ctx->sm_count, static_cast<cudaStream_t>(stream));
        ctx->launches += 1;
        if (e != cudaSuccess) return cuda_fail(ctx, e, to_prefix ? "fdd_prefix_extend launch" : "fdd_kv_commit launch");
    }
    if (advance)
        for (int s = 0; s < n_sets; ++s) {
            if (to_prefix) sets[s]->prefix_len += block_len[s];
            else sets[s]->suffix_len += block_len[s];
        }
    return FDD_OK;
}

fdd_status fdd_kv_commit(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, int layer,
                         const void* k_blk, const void* v_blk, const int32_t* block_len,
                         int advance, void* stream) {
    CallRange range("fdd_kv_commit");
    return commit_like(ctx, sets, n_sets, layer, k_blk, v_blk, block_len, advance, stream, false);
}

fdd_status fdd_prefix_extend(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, int layer,
                             const void* k_blk, const void* v_blk, const int32_t* block_len,
                             int advance, void* stream) {
    CallRange range("fdd_prefix_extend");
    return commit_like(ctx, sets, n_sets, layer, k_blk, v_blk, block_len, advance, stream, true);
}

int fdd_forkset_prefix_len(const fdd_forkset* set) { return set ? set->prefix_len : FDD_ERR_INVALID_ARG; }

fdd_status fdd_average_rollouts(fdd_ctx* ctx, const float* traj, int n, int w, float* out, void* stream) {
    CallRange range("fdd_average_rollouts");
    if (!ctx) return FDD_ERR_INVALID_ARG;
    if (!traj || !out) return fail(ctx, FDD_ERR_INVALID_ARG, "traj/out is NULL");
    if (n < 1 || w < 1) return fail(ctx, FDD_ERR_INVALID_ARG, "n and w must be >= 1");
    cudaError_t e = launch_average(traj, n, w, out, static_cast<cudaStream_t>(stream));
    ctx->launches += 1;
    if (e != cudaSuccess) return cuda_fail(ctx, e, "fdd_average_rollouts launch");
    return FDD_OK;
}

fdd_status fdd_average_rollouts_jmt(fdd_ctx* ctx, const float* traj, int n, int w, int w_out, float* out,
                                    void* stream) {
    CallRange range("fdd_average_rollouts_jmt");
    if (!ctx) return FDD_ERR_INVALID_ARG;
    if (!traj || !out) return fail(ctx, FDD_ERR_INVALID_ARG, "traj/out is NULL");
    if (n < 1 || w < 1 || w_out < 1) return fail(ctx, FDD_ERR_INVALID_ARG, "n, w and w_out must be >= 1");
    if (w < 2) return fail(ctx, FDD_ERR_UNSUPPORTED, "w = 1: two knots do not fix a jerk-minimising curve");
    if (w > kJmtMaxWaypoints || w_out > kJmtMaxOutputs)
        return fail(ctx, FDD_ERR_CAPACITY, "w = %d / w_out = %d beyond %d / %d", w, w_out, kJmtMaxWaypoints, kJmtMaxOutputs);
    const double* d_weights = nullptr;
    for (const fdd_ctx::JmtWeights& j : ctx->jmt_weights)
        if (j.w == w && j.w_out == w_out) d_weights = j.d_weights;
    if (!d_weights) {
        // first call for this pair of sizes: build the matrix on the host and keep it on the device
        std::vector<double> weights;
        if (!jmt_weights(w, w_out, &weights)) return fail(ctx, FDD_ERR_UNSUPPORTED, "spline system is singular");
        double* d = nullptr;
        cudaError_t e = cudaMalloc(&d, weights.size() * sizeof(double));
        if (e == cudaSuccess) e = cudaMemcpy(d, weights.data(), weights.size() * sizeof(double), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            if (d) cudaFree(d);
            return cuda_fail(ctx, e, "fdd_average_rollouts_jmt weights");
        }
        ctx->jmt_weights.push_back({w, w_out, d});
        d_weights = d;
    }
    cudaError_t e = launch_average_jmt(traj, n, w, w_out, d_weights, out, static_cast<cudaStream_t>(stream));
    ctx->launches += 1;
    if (e != cudaSuccess) return cuda_fail(ctx, e, "fdd_average_rollouts_jmt launch");
    return FDD_OK;
}

fdd_status fdd_upload_masked_rows(fdd_ctx* ctx, const void* host_logits, void* dev_logits,
                                  const uint8_t* host_state, int rows, size_t* bytes_copied, void* stream) {
    CallRange range("fdd_upload_masked_rows");
    if (!ctx) return FDD_ERR_INVALID_ARG;
    if (bytes_copied) *bytes_copied = 0;
    if (!host_logits || !dev_logits || !host_state || rows < 0)
        return fail(ctx, FDD_ERR_INVALID_ARG, "host_logits/dev_logits/host_state is NULL or rows < 0");
    const size_t row_bytes = static_cast<size_t>(ctx->cfg.vocab) * (ctx->cfg.logits_dtype == FDD_LOGITS_BF16 ? 2 : 4);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    size_t total = 0;
    int r = 0;
    while (r < rows) {
        if (host_state[r] != FDD_MASKED) { ++r; continue; }
        int e = r + 1;
        while (e < rows && host_state[e] == FDD_MASKED) ++e;            // one copy per run of MASKED rows
        const size_t off = static_cast<size_t>(r) * row_bytes, len = static_cast<size_t>(e - r) * row_bytes;
        cudaError_t err = cudaMemcpyAsync(static_cast<char*>(dev_logits) + off, static_cast<const char*>(host_logits) + off,
                                          len, cudaMemcpyHostToDevice, st);
        if (err != cudaSuccess) return cuda_fail(ctx, err, "fdd_upload_masked_rows copy");
        total += len;
        r = e;
    }
    if (bytes_copied) *bytes_copied = total;
    return FDD_OK;
}

fdd_status fdd_set_merge_wait_limit(fdd_ctx* ctx, long long sm_clocks) {
    if (!ctx) return FDD_ERR_INVALID_ARG;
    if (sm_clocks < 1) return fail(ctx, FDD_ERR_INVALID_ARG, "the wait limit must be at least one clock");
    ctx->attn_merge_wait_limit = sm_clocks;
    return FDD_OK;
}

fdd_status fdd_poll_status(fdd_ctx* ctx, void* stream) {
    if (!ctx) return FDD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_status, 0, sizeof(int), st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "fdd_poll_status");
    const int code = *ctx->h_status;
    if (code != FDD_OK) {
        // a kernel that gave up may have left piece counters of the attention merge half counted
        cudaMemsetAsync(ctx->attn_unit_count, 0, sizeof(int) * 2 * ctx->attn_max_units, st);
        cudaStreamSynchronize(st);
        return fail(ctx, code, "a kernel recorded device status %d", code);
    }
    return FDD_OK;
}

}  // extern "C"
