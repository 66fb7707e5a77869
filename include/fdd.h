/*
 * fdd.h -- C ABI of the block-diffusion decode hot path for NVIDIA B200 (sm_100a).
 *
 * One denoising step of section-wise block-diffusion decoding with N rollouts
 * forked from a shared prefix KV cache:
 *   fdd_fork             share one prefix cache between N rollouts      (Sec. 3.4, "Shared prefix")
 *   fdd_block_attn       block-causal attention of the current block    (Sec. 3.1, "Block-Causal Diffusion")
 *   fdd_unmask           confidence-threshold parallel unmasking        (Sec. 3.3, "Section Diffusion";
 *                                                                        Sec. 3.2 scaffold; Sec. 3.1 "visible tokens fixed")
 *   fdd_ss_draft/_accept draft and accept scan of Scaffold Speculative Decoding (Sec. 3.3, Algorithm)
 *   fdd_plan_blocks      section-aligned blocks of the output template         (Sec. 3.2)
 *   fdd_kv_commit        append the finished block to each private cache (Sec. 3.3 cache reuse; Sec. 3.4 fork)
 *   fdd_prefix_extend    append a deterministic block to the shared cache before the fork (Sec. 3.4)
 *   fdd_average_rollouts equal-weight mean of N trajectories            (Sec. 3.4, trajectory averaging)
 *   fdd_average_rollouts_jmt  the same after jerk-minimising interpolation  (Sec. 3.4)
 *
 * Conventions
 *   - Every tensor is caller-owned.  "device" pointers are CUDA device memory of the
 *     current device, "host" pointers are ordinary host memory.  The library allocates
 *     only small metadata and its own scratch (at fdd_create / fdd_fork).
 *   - bf16 tensors are raw 16-bit bfloat16.  All tensors are dense, row-major in the
 *     index order written, and must be 16-byte aligned.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = default
 *     stream) and return without synchronising unless stated.  Argument errors are
 *     detected on the host before anything is launched and returned synchronously.
 *   - Every call that enqueues work (and fdd_plan_blocks) is wrapped in an NVTX range that
 *     carries its name, for profilers that follow NVTX; without one attached this costs nothing.
 *   - No call aborts, throws or prints.  A negative fdd_status is an error; the text
 *     is available from fdd_last_error().
 *   - A context and its fork sets must be used from one host thread at a time.  The calls
 *     on one context share its scratch buffers, so the work they enqueue has to execute in
 *     call order: use one stream per context, or order the streams yourself.
 *
 * Position state codes (uint8): 0 = MASKED (to be decoded), 1 = COMMITTED, 2 = SCAFFOLD
 * (frozen structural token, Sec. 3.2), 3 = DRAFT (between fdd_ss_draft and fdd_ss_accept).
 */
#ifndef FDD_H_
#define FDD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int fdd_status;
#define FDD_OK                   0
#define FDD_ERR_INVALID_ARG     (-1)  /* NULL pointer, negative size, bad enum                */
#define FDD_ERR_SHAPE           (-2)  /* sizes inconsistent with the context configuration   */
#define FDD_ERR_CAPACITY        (-3)  /* private cache, fork count or block length exceeded  */
#define FDD_ERR_STATE           (-4)  /* freed / foreign fork set                            */
#define FDD_ERR_CUDA            (-5)  /* a CUDA runtime call failed (text has the reason)    */
#define FDD_ERR_DEVICE_TIMEOUT  (-6)  /* a bounded device-side wait gave up                  */
#define FDD_ERR_UNSUPPORTED     (-7)  /* configuration outside what the kernels implement    */

#define FDD_MASKED    0
#define FDD_COMMITTED 1
#define FDD_SCAFFOLD  2
#define FDD_DRAFT     3   /* drafted, not yet verified (Scaffold Speculative Decoding only) */

#define FDD_LOGITS_F32  0
#define FDD_LOGITS_BF16 1

typedef struct fdd_ctx fdd_ctx;         /* opaque: configuration, scratch, device status word */
typedef struct fdd_forkset fdd_forkset; /* opaque: N rollouts over one shared prefix cache     */

typedef struct fdd_config {
    int n_q_heads;    /* Hq                                                        */
    int n_kv_heads;   /* Hkv, divides Hq; query head h reads KV head h / (Hq/Hkv)  */
    int head_dim;     /* D: 64 or 128                                              */
    int vocab;        /* V                                                         */
    int n_layers;     /* L: number of per-layer caches a fork set carries          */
    int page_tokens;  /* 0: contiguous prefix cache; else tokens per page (64)     */
    int max_block;    /* largest block length d accepted (<= 128)                  */
    int max_forks;    /* largest total number of rollouts in one call              */
    int logits_dtype; /* FDD_LOGITS_F32 or FDD_LOGITS_BF16                         */
} fdd_config;

/* Create / destroy a context on the current CUDA device.  Allocates the device status
 * word and the scratch buffers (partials of attention units cut between CTAs, unmask
 * records), sized from cfg.
 * Returns FDD_ERR_UNSUPPORTED for head_dim not in {64,128}, Hq % Hkv != 0, Hq/Hkv > 16,
 * max_block > 128; FDD_ERR_CUDA if no usable device.  *out is NULL on failure. */
fdd_status fdd_create(const fdd_config* cfg, fdd_ctx** out);
void fdd_destroy(fdd_ctx* ctx);

/* Text of the most recent error on this context ("" if none).  Valid until the next call. */
const char* fdd_last_error(const fdd_ctx* ctx);

/* Number of kernels this context has launched so far (for accounting). */
uint64_t fdd_launch_count(const fdd_ctx* ctx);

/*
 * fdd_fork -- Sec. 3.4 "Shared prefix": the deterministic sections are decoded once and
 * their KV cache is forked N times.  Nothing is copied: the N rollouts read the same
 * prefix memory, and each gets an empty private suffix.
 *
 *   prefix_k, prefix_v  host arrays [L] of device pointers, one cache per layer, bf16.
 *                       contiguous (cfg.page_tokens == 0): [Hkv][prefix_capacity][D]
 *                       paged:                             [prefix_capacity pages][Hkv][page_tokens][D]
 *                       Read-only for the library except for fdd_prefix_extend; must stay valid
 *                       while the fork set lives, and the caller does not write the first
 *                       prefix_len tokens.
 *   page_table          device int32 [ceil(prefix_len / page_tokens)] physical page of each
 *                       logical page (paged layout), NULL for the contiguous layout.  Every
 *                       entry must be in [0, prefix_capacity); entries are read on the device.
 *   prefix_len          valid prefix tokens (>= 0).
 *   prefix_capacity     tokens per head (contiguous) or number of physical pages (paged).
 *   n_forks             N >= 1, <= cfg.max_forks.
 *   seeds               host uint64 [N]: the noise key of each rollout (copied; the first call
 *                       that samples stores them on the device, in stream order).
 *   suffix_k, suffix_v  host arrays [L] of device pointers, bf16 [N][Hkv][suffix_capacity][D],
 *                       caller-owned, written by fdd_kv_commit only.
 *   suffix_capacity     tokens each rollout may append per layer.
 */
fdd_status fdd_fork(fdd_ctx* ctx, const void* const* prefix_k, const void* const* prefix_v,
                    const int32_t* page_table, int prefix_len, int prefix_capacity,
                    int n_forks, const uint64_t* seeds,
                    void* const* suffix_k, void* const* suffix_v, int suffix_capacity,
                    fdd_forkset** out);
/* Neither fdd_fork nor fdd_forkset_free waits for the device; a set may be freed while the
 * work enqueued for it is still running (its caches are the caller's to keep alive). */
fdd_status fdd_forkset_free(fdd_ctx* ctx, fdd_forkset* set);
/* Committed private tokens per rollout (same for every rollout of a set); < 0 on error. */
int fdd_forkset_suffix_len(const fdd_forkset* set);
/* Forget every committed block (suffix length back to 0); the memory is not cleared. */
fdd_status fdd_forkset_reset(fdd_ctx* ctx, fdd_forkset* set);

/*
 * fdd_block_attn -- Sec. 3.1: the tokens of the current block attend bidirectionally to
 * each other and causally to everything before the block.  For rollout f of a set the keys
 * are the shared prefix, f's private suffix and all block_len keys of f's block:
 *   out[f,i,h,:] = sum_j softmax_j(scale * q[f,i,h,:] . k_j[h/G,:]) v_j[h/G,:]
 * computed with bf16 operands, fp32 accumulation, bf16 output.
 *
 *   sets, n_sets   host array of fork sets handled in this call (independent scenes).
 *   layer          which per-layer cache to read, 0 <= layer < L.
 *   q              device bf16, rollouts of all sets packed in set order:
 *                  set s contributes [N_s][d_s][Hq][D]; k_blk, v_blk likewise [N_s][d_s][Hkv][D].
 *   out            device bf16, same packing and shape as q; 32-byte aligned (rows are written in
 *                  32-byte pieces).
 *   block_len      host int32 [n_sets]: d_s, 1 <= d_s <= cfg.max_block.
 *   scale          soft-max scale (1/sqrt(D) by convention), the same for every set of the call.
 * The tensor-core kernel is launched cooperatively (its CTAs wait, with a bound, for one another's
 * partial results): it needs as many free SMs as it has CTAs, and the launch fails with
 * FDD_ERR_CUDA where the device cannot give them (an MPS share of the SMs, for instance).
 * All sets of a call go into one launch (groups of 16 sets).  Rollouts with equal inputs agree
 * up to the rounding of the bf16 output, not bit for bit: where a unit of work is cut between
 * CTAs depends on its place in the call.
 *   causal_in_block 0: bidirectional inside the block (denoising pass);
 *                  1: query i sees block keys 0..i only (the causal verifier pass of
 *                  Scaffold Speculative Decoding, Sec. 3.3 step 3).
 */
fdd_status fdd_block_attn(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, int layer,
                          const void* q, const void* k_blk, const void* v_blk, void* out,
                          const int32_t* block_len, float scale, int causal_in_block,
                          void* stream);

/*
 * fdd_block_attn_gated -- fdd_block_attn for the rollouts that still decode.  Under the
 * confidence threshold of Sec. 3.3 the rollouts of a batch finish their block after different
 * numbers of denoising steps; a rollout whose block is complete needs no further attention.
 *
 *   gate   device int32 [sum N_s], rollouts in set order, read by the kernel when it runs (the
 *          n_left array that fdd_unmask wrote in the step before fits as it is): rollout r takes
 *          part if gate[r] != 0; otherwise its rows of out are left untouched and none of its
 *          keys are read.  NULL: every rollout takes part (fdd_block_attn).
 * The work of the launch is laid out on the device from the gate values, so a caller may enqueue
 * the next step before it has seen the result of this one: once every entry is 0 the launch
 * returns at once.  With a gate a call takes at most 2048 rollouts (FDD_ERR_CAPACITY beyond).  Everything else as fdd_block_attn.
 */
fdd_status fdd_block_attn_gated(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, int layer,
                                const void* q, const void* k_blk, const void* v_blk, void* out,
                                const int32_t* block_len, float scale, int causal_in_block,
                                const int32_t* gate, void* stream);

/*
 * fdd_unmask -- one parallel unmasking step (Sec. 3.3 "iteratively unmasks value
 * positions"; Sec. 3.1: visible tokens stay fixed; Sec. 3.2: scaffold never rewritten).
 * For every rollout f and every position i with state MASKED:
 *   tok  = argmax_v (logit[v] + temperature * g[v])            lowest v on ties
 *   conf = softmax(logit)[tok]                                  noise-free probability
 * where g[v] = -ln(E[v]) and the E[v] are independent Exp(1) variates built as a race over
 * groups of 16 consecutive ids from two Philox4x32-10 streams under key = the rollout's seed
 * (low, high word).  Group j = v / 16 has the word
 *   R = output word j % 4 of counter (j / 4, i, step, block_idx),
 * every id the fine bits
 *   f[v] = top 23 bits of output word v % 4 of counter (v / 4, i + 2^31, step, block_idx).
 * The id 16 j + R % 16 (the group's leader) holds the group's minimum,
 *   E = -ln(U) / 16,  U = ((R >> 4) + (f + 0.5) * 2^-23) / 2^28,
 * every other id of the group E[v] = E_leader - ln((f[v] + 0.5) * 2^-23)
 * (the word of a group bounds its 16 draws, which lets the kernel skip the second stream for almost
 * every v); temperature == 0 uses no noise.  Positions with
 * conf > threshold are committed (token written, state -> COMMITTED); if a rollout has
 * MASKED positions and none passes, its single most confident one (lowest i on ties)
 * is committed.  Nothing else is written; rollouts without MASKED positions are no-ops.
 *
 *   logits        device, packed like q: [N_s][d_s][V], fp32 or bf16 per cfg.logits_dtype.
 *                 Only rows of MASKED positions are read.  N_s * d_s <= 8192 per set
 *                 (FDD_ERR_CAPACITY otherwise); the bulk copies need 16-byte aligned rows
 *                 (V % 8 == 0 for bf16, V % 4 == 0 for fp32, 16-byte aligned base), else a
 *                 slower path runs.
 *   tokens        device int32 [N_s][d_s], in/out.     state: device uint8, in/out.
 *   n_committed   device int32 [sum N_s]: commits of this step per rollout (written).
 *   n_left        device int32 [sum N_s]: MASKED positions remaining per rollout (written).
 *   conf          device fp32 packed [N_s][d_s] or NULL: confidence of every position that
 *                 was MASKED on entry, NaN elsewhere.
 */
fdd_status fdd_unmask(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, const void* logits,
                      int32_t* tokens, uint8_t* state, const int32_t* block_len,
                      float threshold, float temperature, uint32_t block_idx, uint32_t step,
                      int32_t* n_committed, int32_t* n_left, float* conf, void* stream);

/*
 * fdd_unmask_counted -- fdd_unmask with the denoising step counted on the device.  The step
 * index enters the noise, so a caller that records one step as a CUDA graph and replays it
 * (Sec. 4.3 credits part of the deployed speed-up to CUDA graphs) cannot pass it by value.
 *   step_counter  device uint32: read by the kernels when they run (the step index of this call),
 *                 incremented by one when the call's work is done.  Set it to 0 at the start of
 *                 a block (cudaMemsetAsync on the same stream).
 * Everything else as fdd_unmask with step = *step_counter.  The library's calls allocate nothing
 * and never synchronise on the paths a step takes (fdd_block_attn[_gated], fdd_unmask[_counted])
 * once each has run before with the same shapes, so they can be issued while a stream is being
 * captured.
 */
fdd_status fdd_unmask_counted(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, const void* logits,
                              int32_t* tokens, uint8_t* state, const int32_t* block_len,
                              float threshold, float temperature, uint32_t block_idx,
                              uint32_t* step_counter, int32_t* n_committed, int32_t* n_left,
                              float* conf, void* stream);

/*
 * fdd_ss_draft, fdd_ss_accept -- Scaffold Speculative Decoding (Sec. 3.3, Algorithm steps 1-3).
 * Scaffold positions are accepted as they are (step 1: they are never read or written).
 *
 * fdd_ss_draft (step 2): `logits` are the diffusion head's, from one bidirectional pass
 * (fdd_block_attn with causal_in_block = 0).  Every MASKED position gets
 * argmax_v (logit[v] + temperature * g[v]) (noise and packing as in fdd_unmask) and the state
 * FDD_DRAFT.  n_drafted / n_left: device int32 [sum N_s], drafts written / MASKED left (0).
 *
 * fdd_ss_accept (step 3): `ar_logits[f][i]` are the AR head's logits FOR position i from one causal
 * pass over the block (fdd_block_attn with causal_in_block = 1).  Per rollout, over the FDD_DRAFT
 * positions from left to right: the draft is accepted (state -> COMMITTED) while it equals the
 * verifier's token argmax_v (ar_logit[v] + temperature * g[v]) (temperature > 0: the sampled
 * verifier of Sec. 3.4); at the first mismatch the verifier's token replaces the draft and is
 * accepted, and every later FDD_DRAFT position goes back to MASKED for the next draft / verify
 * cycle.  n_accepted: positions that became COMMITTED in this call; n_left: MASKED afterwards.
 * Only rows in state FDD_DRAFT are read.  Limits as for fdd_unmask.
 */
fdd_status fdd_ss_draft(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, const void* logits,
                        int32_t* tokens, uint8_t* state, const int32_t* block_len,
                        float temperature, uint32_t block_idx, uint32_t step,
                        int32_t* n_drafted, int32_t* n_left, void* stream);
fdd_status fdd_ss_accept(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, const void* ar_logits,
                         int32_t* tokens, uint8_t* state, const int32_t* block_len,
                         float temperature, uint32_t block_idx, uint32_t step,
                         int32_t* n_accepted, int32_t* n_left, void* stream);

/*
 * fdd_kv_commit -- Sec. 3.3 / 3.4: a finished block's K/V join the cache of the rollout
 * that produced them and are reused, not recomputed, by later blocks.  Copies rollout f's
 * rows of k_blk / v_blk ([N_s][d_s][Hkv][D], packed like fdd_block_attn) to positions
 * [len, len + d_s) of f's private suffix of `layer`, bit for bit.  With advance != 0 the
 * set's suffix length grows by d_s afterwards (pass it on the last layer).
 * FDD_ERR_CAPACITY if len + d_s > suffix_capacity (nothing is launched).
 */
fdd_status fdd_kv_commit(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, int layer,
                         const void* k_blk, const void* v_blk, const int32_t* block_len,
                         int advance, void* stream);

/*
 * fdd_prefix_extend -- Sec. 3.4 "Shared prefix": the first three sections are deterministic, so
 * they are decoded once, by a fork set of ONE rollout, and the N rollouts of the trajectory section
 * are forked from the cache that holds them.  This call is that set's commit: its block's K/V
 * ([1][d_s][Hkv][D], packed like fdd_block_attn) go to positions [P, P + d_s) of the shared prefix
 * cache of `layer` itself (P = the set's current prefix length), bit for bit, in the cache's own
 * layout (paged: through the page table, whose entries for the touched pages the caller has filled
 * in).  With advance != 0 the set's prefix length grows by d_s afterwards (pass it on the last
 * layer).  A later fdd_fork over the same cache buffers with prefix_len = fdd_forkset_prefix_len(set)
 * gives N rollouts that share everything decoded so far; nothing is copied or re-laid.
 * This is the only call that writes a prefix cache.  It writes beyond the current prefix length
 * only, so fork sets that already read the same buffers with a shorter length are not disturbed.
 * FDD_ERR_STATE if a set has more than one rollout or has committed a private suffix;
 * FDD_ERR_CAPACITY if P + d_s exceeds prefix_capacity (nothing is launched).  A page table entry
 * outside [0, prefix_capacity) is not followed: the rows are dropped and the device status word
 * gets FDD_ERR_INVALID_ARG (see fdd_poll_status).
 */
fdd_status fdd_prefix_extend(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, int layer,
                             const void* k_blk, const void* v_blk, const int32_t* block_len,
                             int advance, void* stream);
/* Tokens of the shared prefix the set currently reads; < 0 on error. */
int fdd_forkset_prefix_len(const fdd_forkset* set);

/*
 * fdd_average_rollouts -- Sec. 3.4: tau_out = (1/N) sum_i tau_i.
 *   traj  device fp32 [n][w][2];  out  device fp32 [w][2];  n >= 1, w >= 1.
 */
fdd_status fdd_average_rollouts(fdd_ctx* ctx, const float* traj, int n, int w, float* out,
                                void* stream);

/*
 * fdd_average_rollouts_jmt -- Sec. 3.4: every rollout's trajectory is interpolated to w_out
 * waypoints by jerk-minimising fitting, then the interpolants are averaged with equal weights.
 * The paper gives no formula; this library's reading: per coordinate, the curve through the
 * origin of the vehicle frame at t = 0 and waypoint k at t = k + 1 that minimises the integral
 * of the squared jerk (the natural quintic spline), sampled at t_j = (j + 1) * w / w_out.
 *   traj  device fp32 [n][w][2];  out  device fp32 [w_out][2];  n >= 1, 2 <= w <= 32,
 *   1 <= w_out <= 256 (FDD_ERR_CAPACITY beyond; w = 1 is FDD_ERR_UNSUPPORTED: every curve of
 *   constant acceleration through two knots has zero jerk, so there is no single minimiser).
 * The first call for a pair (w, w_out) builds the interpolation matrix on the host, allocates
 * w_out * w doubles on the device for it and waits for their upload; later calls only launch.
 */
fdd_status fdd_average_rollouts_jmt(fdd_ctx* ctx, const float* traj, int n, int w, int w_out,
                                    float* out, void* stream);

/*
 * fdd_decode_block -- Sec. 3.3: the denoising loop of one block, run by the library.  "At every
 * step the block attends to the cached context, the model scores the MASKED positions, the
 * confident ones are committed, and the loop ends when no MASK is left; the finished block's
 * K/V are then cached."  Equivalent to the caller doing, for t = 0, 1, ...:
 *     for layer in [0, n_layers): fdd_block_attn_gated(layer, q, k_blk, v_blk -> out; gate = n_left of step t - 1,
 *                                                      every rollout at t = 0)
 *     fdd_unmask(logits, step = t) -> tokens, state, n_committed, n_left
 *     stop when sum(n_left) == 0 (or after max_steps steps)
 * and then, with commit_kv != 0 and the block complete, fdd_kv_commit for every layer with the K/V
 * of the last step (advance on the last layer).  The loop lives here because on short steps (one
 * scene, few rollouts) the kernels take less time than an interpreter needs to issue them: the
 * library issues step t + 1 before it reads the counts of step t, so the GPU never waits for the
 * host; if step t completed the block, the kernels of step t + 1 find every rollout gated off and
 * no MASKED row and return at once (n_committed and n_left then hold that step's zeros).
 *   q, k_blk, v_blk, out   host arrays [n_inputs][n_layers] of device pointers, each laid out as for
 *                          fdd_block_attn; step t uses row t mod n_inputs (a caller whose model
 *                          writes every step into the same buffers passes n_inputs = 1)
 *   logits                 host array [n_inputs] of device pointers, laid out as for fdd_unmask
 *   tokens, state, n_committed, n_left   device, as for fdd_unmask
 *   steps_taken            host out: steps that found a MASKED position on entry
 *   masked_left            host out or NULL: MASKED positions left (0 unless max_steps ran out)
 *   before_step            NULL, or a function the library calls as before_step(user, t, stream)
 *                          before it issues step t: the place where a caller enqueues, on `stream`,
 *                          the model work that produces step t's q / k / v / logits
 * The counts reach the host through pinned host memory that the unmasking step writes itself
 * (count and a per-step stamp in one 8-byte store), which the call polls: no copy and no event sits
 * between two steps on the stream.  The poll is bounded: it ends with FDD_ERR_CUDA if the stream
 * reports an error or runs empty without the counts, and with FDD_ERR_DEVICE_TIMEOUT after 30 s.
 * The call returns when the counts of the last step have reached the host; the commits it issued
 * may still be running.
 * Errors as for the calls it makes; nothing is issued after the first failure.
 */
typedef void (*fdd_step_fn)(void* user, int step, void* stream);
fdd_status fdd_decode_block(fdd_ctx* ctx, fdd_forkset* const* sets, int n_sets, int n_layers,
                            int max_steps, int n_inputs,
                            const void* const* q, const void* const* k_blk, const void* const* v_blk,
                            void* const* out, const void* const* logits,
                            int32_t* tokens, uint8_t* state, const int32_t* block_len,
                            float scale, int causal_in_block, float threshold, float temperature,
                            uint32_t block_idx, int commit_kv,
                            int32_t* n_committed, int32_t* n_left,
                            int* steps_taken, int* masked_left,
                            fdd_step_fn before_step, void* user, void* stream);

/*
 * fdd_unmask_static -- the unmasking step of fdd_unmask for callers that cannot allocate device
 * memory.  (The paper has no counterpart; this is a deployment variant of fdd_unmask.)
 *
 * Who needs it: code that runs after the vehicle stack has finished initialising and is then
 * forbidden to allocate (a real-time planning loop with a fixed memory budget, a plugin that is
 * handed pre-allocated buffers only, a process whose allocator is locked after start-up).
 * cudaMalloc may block on the whole device, take unbounded time or fail late, so fdd_create and
 * fdd_fork (which allocate scratch and seed storage) are not available to such callers.  This
 * call needs neither a context nor a fork set and performs no allocation of any kind: its scratch
 * is a fixed array inside the library image (FDD_UNMASK_STATIC_MAX_RECORDS records of 32 bytes =
 * 2 MiB, resident on every GPU that loads the library until the process exits).
 *
 * It computes exactly what fdd_unmask computes for one set (same kernels, same rule, same noise).
 *   logits        device [n_forks][block_len][vocab], fp32 or bf16 per logits_dtype
 *   tokens, state device, in/out, [n_forks][block_len]
 *   seeds         device uint64 [n_forks] (the caller keeps them on the device)
 *   n_committed, n_left  device int32 [n_forks] (written);  conf: device fp32 [n_forks][block_len] or NULL
 *   err, err_len  optional host buffer that receives the error text (may be NULL / 0)
 * Limits: block_len <= 128, n_forks * block_len <= 8192 rows, and
 * n_forks * block_len * ceil(vocab / 8192) <= FDD_UNMASK_STATIC_MAX_RECORDS; anything larger is
 * rejected with FDD_ERR_CAPACITY before any launch (e.g. vocab 151936 has 19 record slots per row,
 * so up to 3449 rows: 32 rollouts x 64 positions fit).
 * Set-up: the first call on each device (with that device current) asks the runtime for the
 * device address of the array (cudaGetSymbolAddress) and caches it; make that first call before
 * any stream capture begins.  Later calls do no set-up.
 * Sharing: all calls on a device use the same array, which keeps whatever the previous call
 * left in it.  Nothing in it has to start at zero: every record that is read was written earlier
 * in the same call (the first record of a row says how many of its records are valid).  Two calls whose kernels can overlap on the GPU (different streams without
 * ordering) race on it; order them.  The host side is not thread-safe for the first call per device.
 */
#define FDD_UNMASK_STATIC_MAX_RECORDS 65536
fdd_status fdd_unmask_static(const void* logits, int logits_dtype, int n_forks, int block_len,
                             int vocab, int32_t* tokens, uint8_t* state, const uint64_t* seeds,
                             float threshold, float temperature, uint32_t block_idx, uint32_t step,
                             int32_t* n_committed, int32_t* n_left, float* conf, void* stream,
                             char* err, size_t err_len);

/*
 * fdd_plan_blocks -- Sec. 3.2 "Section-Aligned Blocks": block borders follow section borders, and
 * section s with E_s editable (value) positions is cut into ceil(E_s / d) blocks.  Host code only.
 * Inside a section the blocks are filled from the left with d editable positions each (the last
 * takes the rest); a block ends right after its last editable position, the section's last block
 * at the section's end, so scaffold tokens travel with the value tokens that follow them; a
 * section without editable positions is one block that needs no decoding.
 *   editable       host uint8 [length]: 1 = value position, 0 = scaffold
 *   section_end    host int32 [n_sections]: exclusive end of each section, non-decreasing, last == length
 *   block_begin, block_end, block_section   host int32 [capacity], written: block b covers positions
 *                  [block_begin[b], block_end[b]) of section block_section[b]; *n_blocks = their number
 * FDD_ERR_CAPACITY if more than `capacity` blocks are needed, FDD_ERR_INVALID_ARG for bad arguments.
 */
fdd_status fdd_plan_blocks(const uint8_t* editable, const int32_t* section_end, int n_sections,
                           int length, int d, int32_t* block_begin, int32_t* block_end,
                           int32_t* block_section, int capacity, int* n_blocks);

/*
 * fdd_upload_masked_rows -- host-to-device copy of exactly the logits rows the next fdd_unmask
 * will read (Sec. 3.3: only MASKED value positions are decoded; everything else is never read).
 * For callers whose logits live in host memory.
 *   host_logits   host (pinned for an asynchronous copy) [rows][V], dtype per cfg.logits_dtype
 *   dev_logits    device buffer of the same shape; rows that are not copied keep their old bytes
 *   host_state    host uint8 [rows]: the state array as the caller last read it from the device
 *   bytes_copied  optional: bytes enqueued
 * One cudaMemcpyAsync per run of consecutive MASKED rows, on `stream`; returns without waiting.
 */
fdd_status fdd_upload_masked_rows(fdd_ctx* ctx, const void* host_logits, void* dev_logits,
                                  const uint8_t* host_state, int rows, size_t* bytes_copied, void* stream);

/*
 * fdd_pull_masked_rows -- the same rows (Sec. 3.3: only MASKED value positions are decoded), fetched
 * by a kernel that reads the state array on the device and pulls the rows out of host memory
 * itself.  Nothing goes back to the host and nothing is synchronised, so the call can be issued
 * ahead of the counts of the step before, like the other calls of a step.
 *   host_logits   pinned host memory that the device can address (cudaHostAlloc / cudaHostRegister;
 *                 FDD_ERR_INVALID_ARG otherwise) [rows][V], dtype per cfg.logits_dtype
 *   dev_logits    device buffer of the same shape; rows that are not MASKED keep their old bytes
 *   dev_state     device uint8 [rows], read when the kernel runs (stream order)
 *   bytes_pulled  device counter or NULL: the bytes of every pulled row are added to it
 * One launch of 32 CTAs on `stream` (a link of 55 GB/s is filled by 16); rows whose pitch is a
 * multiple of 16 bytes move in 16-byte pieces, others two bytes at a time.
 */
fdd_status fdd_pull_masked_rows(fdd_ctx* ctx, const void* host_logits, void* dev_logits,
                                const uint8_t* dev_state, int rows, unsigned long long* bytes_pulled,
                                void* stream);

/*
 * fdd_set_merge_wait_limit -- how long a CTA of fdd_block_attn waits for the partial results of the
 * other CTAs that share a unit of work with it, in SM clocks (default 4e9, about two seconds).  When
 * the limit runs out the CTA records FDD_ERR_DEVICE_TIMEOUT in the device status word and returns
 * without writing its share of the output; the launch itself always ends.  fdd_poll_status then
 * reports the error and puts the context's counters back in order, and the next call is valid.
 * Meant for deployments that want a tighter bound than the default, and for testing the error path
 */
fdd_status fdd_set_merge_wait_limit(fdd_ctx* ctx, long long sm_clocks);

/* Synchronise `stream` and return the device status word: FDD_OK, or the first error a
 * kernel recorded (FDD_ERR_DEVICE_TIMEOUT, FDD_ERR_INVALID_ARG).  Reading clears it. */
fdd_status fdd_poll_status(fdd_ctx* ctx, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* FDD_H_ */
