// fdd_decode_block: the denoising loop of one block (Sec. 3.3), driven by the library.
//
// Per step: gated attention for every layer and the unmasking step, which also writes the
// per-rollout counts of MASKED positions into host memory.  The host side is the part that matters
// here: on short steps (one scene, a few rollouts) the kernels of a step take a few tens of
// microseconds, less than an interpreter needs to marshal the same calls, so the loop lives in
// native code and runs one step ahead of the counts it reads.
#include "fdd_internal.h"

#include <chrono>

namespace {

// Wait until every rollout's (n_left, stamp) of the step with this stamp has reached the host; their
// sum goes to *left.  The wait is bounded: it ends with an error if the stream reports one, if the
// stream has run empty without the counts arriving, or after kCountWaitSeconds.
constexpr double kCountWaitSeconds = 30.0;

fdd_status wait_for_counts(fdd_ctx* ctx, int buf, int stamp, int forks, cudaStream_t st, int* left) {
    const volatile long long* src = reinterpret_cast<const volatile long long*>(ctx->h_counts[buf]);
    const auto t0 = std::chrono::steady_clock::now();
    int f = 0, sum = 0;
    unsigned spins = 0;
    bool drained = false;
    while (f < forks) {
        const long long v = src[f];                      // one aligned 8-byte load: count in the low half, stamp in the high half
        if (static_cast<int>(v >> 32) == stamp) {
            sum += static_cast<int>(v & 0xFFFFFFFFLL);
            ++f;
            continue;
        }
        if ((++spins & 0x3FFu) == 0) {
            const double waited = std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
            if (waited > 200e-6) {
                // a long wait: make sure the stream is still alive
                if (drained) {
                    ctx->last_error = "fdd_decode_block: the stream ran empty but the counts of a step never arrived";
                    return FDD_ERR_CUDA;
                }
                const cudaError_t q = cudaStreamQuery(st);
                if (q == cudaSuccess) drained = true;    // everything issued has completed: one more look at the counts, then give up
                else if (q != cudaErrorNotReady) {
                    ctx->last_error = std::string("fdd_decode_block: ") + cudaGetErrorString(q);
                    return FDD_ERR_CUDA;
                }
            }
            if (waited > kCountWaitSeconds) {
                ctx->last_error = "fdd_decode_block: timed out waiting for the counts of a step";
                return FDD_ERR_DEVICE_TIMEOUT;
            }
        }
#if defined(__x86_64__) || defined(__i386__)
        __builtin_ia32_pause();
#endif
    }
    *left = sum;
    return FDD_OK;
}

}  // namespace

fdd_status fdd_decode_block(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, int n_layers,
                            int max_steps, int n_inputs,
                            const void* const* q, const void* const* k_blk, const void* const* v_blk,
                            void* const* out, const void* const* logits,
                            int32_t* tokens, uint8_t* state, const int32_t* block_len,
                            float scale, int causal_in_block, float threshold, float temperature,
                            uint32_t block_idx, int commit_kv,
                            int32_t* n_committed, int32_t* n_left,
                            int* steps_taken, int* masked_left,
                            fdd_step_fn before_step, void* user, void* stream) {
    CallRange range("fdd_decode_block");
    if (!ctx) return FDD_ERR_INVALID_ARG;
    if (!q || !k_blk || !v_blk || !out || !logits || !steps_taken || !n_left || !n_committed) {
        ctx->last_error = "fdd_decode_block: a required pointer is NULL";
        return FDD_ERR_INVALID_ARG;
    }
    if (n_layers < 1 || n_layers > ctx->cfg.n_layers || max_steps < 1 || n_inputs < 1 || n_sets < 1 || !sets) {
        ctx->last_error = "fdd_decode_block: n_layers must be in [1, context layers], max_steps, n_inputs and n_sets >= 1";
        return FDD_ERR_INVALID_ARG;
    }
    int forks = 0;
    for (int s = 0; s < n_sets; ++s) {
        if (!sets[s]) {
            ctx->last_error = "fdd_decode_block: a fork set is NULL";
            return FDD_ERR_INVALID_ARG;
        }
        forks += sets[s]->n_forks;
    }
    if (forks > ctx->cfg.max_forks) {
        ctx->last_error = "fdd_decode_block: more rollouts than the context was created for";
        return FDD_ERR_CAPACITY;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    *steps_taken = 0;
    if (masked_left) *masked_left = 0;

    int stamp_of[2] = {0, 0};
    // One denoising step on the stream.  From the second step on, attention skips the rollouts that
    // the step before left without a MASKED position (n_left is written by that step's unmask and
    // read by this step's attention, both on `st`).
    auto enqueue = [&](int t) -> fdd_status {
        if (before_step) before_step(user, t, stream);
        const int in = t % n_inputs;
        for (int layer = 0; layer < n_layers; ++layer) {
            const int i = in * n_layers + layer;
            const fdd_status rc = fdd_block_attn_gated(ctx, sets, n_sets, layer, q[i], k_blk[i], v_blk[i], out[i], block_len,
                                                       scale, causal_in_block, t == 0 ? nullptr : n_left, stream);
            if (rc != FDD_OK) return rc;
        }
        // the unmasking step also writes (n_left, stamp) of every rollout into host memory that the
        // device can address: the host sees the counts the moment they land, without a copy and
        // without an event on the stream (which would sit between this step and the next one's early start)
        if (++ctx->count_stamp <= 0) ctx->count_stamp = 1;
        stamp_of[t & 1] = ctx->count_stamp;
        ctx->unmask_left_mirror = ctx->d_counts[t & 1];
        ctx->unmask_mirror_stamp = ctx->count_stamp;
        const fdd_status rc = fdd_unmask(ctx, sets, n_sets, logits[in], tokens, state, block_len, threshold, temperature,
                                         block_idx, static_cast<uint32_t>(t), n_committed, n_left, nullptr, stream);
        ctx->unmask_left_mirror = nullptr;
        if (rc != FDD_OK) return rc;
        return FDD_OK;
    };

    fdd_status rc = enqueue(0);
    int t = 0, left = 0;
    while (rc == FDD_OK) {
        // step t + 1 goes out before the host knows what step t left: if the block turns out to be
        // complete, its kernels find every rollout gated off and no MASKED row, and return at once
        if (t + 1 < max_steps) rc = enqueue(t + 1);
        if (rc != FDD_OK) break;
        rc = wait_for_counts(ctx, t & 1, stamp_of[t & 1], forks, st, &left);
        if (rc != FDD_OK) break;
        ++t;
        if (left == 0 || t >= max_steps) break;
    }
    if (rc != FDD_OK) return rc;
    *steps_taken = t;
    if (masked_left) *masked_left = left;
    if (commit_kv && left == 0) {
        // the block is complete: its keys and values, as the last step projected them, join every
        // rollout's private cache
        const int in = (t - 1) % n_inputs;
        for (int layer = 0; layer < n_layers; ++layer) {
            rc = fdd_kv_commit(ctx, sets, n_sets, layer, k_blk[in * n_layers + layer], v_blk[in * n_layers + layer], block_len,
                               layer == n_layers - 1 ? 1 : 0, stream);
            if (rc != FDD_OK) return rc;
        }
    }
    return FDD_OK;
}
