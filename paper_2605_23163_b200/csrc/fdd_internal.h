// Internal declarations shared by the host API and the kernel files.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <string>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "fdd.h"

// A named NVTX range around one library call: profilers that follow NVTX show which call a kernel
// belongs to; without one attached the two calls return at once.
struct CallRange {
    explicit CallRange(const char* name) { nvtxRangePushA(name); }
    ~CallRange() { nvtxRangePop(); }
    CallRange(const CallRange&) = delete;
    CallRange& operator=(const CallRange&) = delete;
};

// TMA tensor maps of one scene for the persistent tensor-core attention kernel.
struct TcSetMaps {
    CUtensorMap q;                  // (D, Hq, d, N)
    CUtensorMap bk, bv;             // (D, Hkv, d, N)
    CUtensorMap sk, sv;             // (D, S, Hkv, N)
    CUtensorMap pk, pv;             // contiguous: (D, P, Hkv); paged: (D, 64, Hkv, pages)
    CUtensorMap pk_tail, pv_tail;   // paged only: token dimension cut to the last page's fill
};
constexpr int kTcMaxSets = 16;      // scenes per attention launch

// The maps last built for one (fork set, layer) and what they were built from.
struct TcMapCache {
    bool valid = false;
    const void* q = nullptr;
    const void* k_blk = nullptr;
    const void* v_blk = nullptr;
    int d = 0;
    int suffix_len = -1;
    int prefix_len = -1;
    TcSetMaps maps;
};

// Tensor maps of a freed fork set, kept for a later set over the same caches (a server forks the
// same prefix block after block).
struct TcMapPoolEntry {
    std::vector<const void*> prefix_k, prefix_v;
    std::vector<void*> suffix_k, suffix_v;
    int n_forks, prefix_len, prefix_capacity, suffix_capacity;
    std::vector<TcMapCache> maps;
};

struct fdd_ctx {
    fdd_config cfg;
    int device = 0;
    int sm_count = 0;
    int* d_status = nullptr;          // device status word (first error wins)
    int* h_status = nullptr;          // pinned mirror
    int2* h_counts[2] = {nullptr, nullptr};   // pinned and mapped, [max_forks] each: (n_left, stamp) of the two steps in flight (fdd_decode_block)
    int2* d_counts[2] = {nullptr, nullptr};   // the device's addresses of h_counts
    int2* unmask_left_mirror = nullptr;       // set by fdd_decode_block around its fdd_unmask calls
    int unmask_mirror_stamp = 0;
    int count_stamp = 0;                      // the stamp of the step issued last
    void* ws_unmask = nullptr;        // per (row, tile) partial reductions
    size_t ws_unmask_bytes = 0;
    void* ws_attn = nullptr;          // partial outputs of attention units cut between CTAs
    size_t ws_attn_bytes = 0;
    int* attn_unit_count = nullptr;   // device [2][attn_max_units]: pieces written / merge shares done per unit (self-resetting)
    int attn_max_units = 0;
    int attn_max_ctas = 0;
    std::vector<uint64_t> attn_args;  // host buffer for the attention kernel's argument block (8-byte aligned)
    long long attn_merge_wait_limit = 4000000000LL;   // SM clocks (about two seconds): wait for the pieces of a cut unit
    void* seed_chunk = nullptr;       // host staging of seeds on their way to the device as kernel arguments
    uint64_t launches = 0;
    std::string last_error;
    std::vector<fdd_forkset*> live_sets;
    struct SeedBuf { uint64_t* ptr; int cap; };
    std::vector<SeedBuf> seed_pool;   // device seed buffers of freed fork sets, kept for the next fork
    std::vector<TcMapPoolEntry> map_pool;
    struct JmtWeights { int w, w_out; double* d_weights; };
    std::vector<JmtWeights> jmt_weights;   // interpolation matrices built so far (device, fp64 [w_out][w])
};

struct fdd_forkset {
    fdd_ctx* ctx = nullptr;
    int n_forks = 0;
    int prefix_len = 0;
    int prefix_capacity = 0;
    const int32_t* page_table = nullptr;   // device
    std::vector<const void*> prefix_k, prefix_v;
    std::vector<void*> suffix_k, suffix_v;
    int suffix_capacity = 0;
    int suffix_len = 0;
    uint64_t* d_seeds = nullptr;            // device [seed_cap], from the context's pool
    int seed_cap = 0;
    std::vector<uint64_t> h_seeds;          // the caller's seeds, stored on the device by the first call that needs them
    bool seeds_on_device = false;
    std::vector<TcMapCache> map_cache;      // per layer
};

// One scene's slice of a batched call, as the kernels see it.
struct AttnProblem {
    const __nv_bfloat16* q;        // [N][d][Hq][D]
    const __nv_bfloat16* k_blk;    // [N][d][Hkv][D]
    const __nv_bfloat16* v_blk;
    __nv_bfloat16* out;            // [N][d][Hq][D]
    const __nv_bfloat16* prefix_k; // contiguous [Hkv][cap][D] or paged [pages][Hkv][pt][D]
    const __nv_bfloat16* prefix_v;
    const int32_t* page_table;     // device or nullptr
    const __nv_bfloat16* suffix_k; // [N][Hkv][scap][D]
    const __nv_bfloat16* suffix_v;
    int n_forks, d, n_q_heads, n_kv_heads;
    int prefix_len, prefix_capacity, page_tokens;
    int suffix_len, suffix_capacity;
    int causal_in_block;
    float scale;
    const int32_t* gate;           // device [N], 0 = leave the rollout out; nullptr = all take part
};

constexpr int kJmtMaxWaypoints = 32;        // decoded waypoints per rollout the interpolation takes
constexpr int kJmtMaxOutputs = 256;         // interpolated waypoints
constexpr int kAttnMaxGatedForks = 2048;    // rollouts of one fdd_block_attn_gated call
constexpr int kUnmaskMaxSets = 16;          // scenes per unmask launch

// Several scenes of one unmask call, packed in set order (rows = rollouts x positions).
struct UnmaskSets {
    int n_sets;
    int row_off[kUnmaskMaxSets + 1];        // first row of each set (and the total)
    int fork_off[kUnmaskMaxSets + 1];       // first rollout of each set (and the total)
    int d[kUnmaskMaxSets];                  // block length of each set
    const uint64_t* seeds[kUnmaskMaxSets];  // device [n_forks of the set]
};

struct UnmaskProblem {
    const void* logits;     // [rows][V]
    int32_t* tokens;        // [rows]
    uint8_t* state;         // [rows]
    int32_t* n_committed;   // [forks]
    int32_t* n_left;        // [forks]
    float* conf;            // [rows] or nullptr
    UnmaskSets sets;
    int vocab, logits_dtype;
    float threshold, temperature;
    uint32_t block_idx, step;
    uint32_t* step_counter = nullptr;   // device or nullptr: its value is added to `step` when the kernels run
    int bump_counter = 0;               // increment it once this launch pair is done
    int2* left_mirror = nullptr;        // host memory mapped for the device, [forks], or nullptr: (n_left, mirror_stamp) is written there too
    int mirror_stamp = 0;
};

// Unmask scratch: one record per (row, chunk).
struct UnmaskPartial {
    float row_max;     // max logit of the chunk
    float sum_exp;     // sum exp(logit - row_max)
    float best_score;  // max of logit + T * gumbel
    float best_logit;  // logit at the best score
    int best_index;    // vocabulary id of the best score (lowest on ties)
    int pad[3];
};

static constexpr int kUnmaskTile = 2048;    // vocabulary entries per tile of the streaming kernel (one bulk copy)
static constexpr int kUnmaskChunk = 8192;   // vocabulary entries per record slot of fdd_unmask_static
static constexpr int kUnmaskMaxRows = 8192; // rollouts x positions of one launch (the kernel compacts them in shared memory)
// Record slots per row when tiles_per_item tiles share a slot.
static inline int unmask_items_per_row(int vocab, int tiles_per_item) {
    const int tiles = (vocab + kUnmaskTile - 1) / kUnmaskTile;
    return (tiles + tiles_per_item - 1) / tiles_per_item;
}
size_t unmask_workspace_bytes(int vocab, int max_rows);

cudaError_t launch_attention_simple(const AttnProblem& p, int head_dim, cudaStream_t st);
bool attention_tc_supported(const AttnProblem& a, int head_dim);
size_t attention_ptc_workspace_bytes(int head_dim, int max_ctas);
cudaError_t launch_attention_ptc(fdd_ctx* ctx, const AttnProblem* probs, TcMapCache* const* caches, int n,
                                 int head_dim, cudaStream_t st, int* n_launches);
cudaError_t launch_unmask(fdd_ctx* ctx, const UnmaskProblem& p, cudaStream_t st, int* n_launches, int mode = 0);
// One scene's part of a cache append.
constexpr int kCommitSuffix = 0, kCommitPrefix = 1, kCommitPagedPrefix = 2;
constexpr int kCommitMaxSets = 16;          // scenes per append launch
struct CommitSet {
    const void* k_src;       // this scene's rows of k_blk / v_blk
    const void* v_src;
    void* k_dst;             // the layer's cache
    void* v_dst;
    const int32_t* page_table;
    long long vec_begin;     // first 16-byte vector of this scene in the launch
    int n_forks, d, len, cap, mode, page_tokens;
};
struct CommitArgs {
    CommitSet set[kCommitMaxSets];
    int n;
    long long total;         // 16-byte vectors of all scenes
    int n_kv_heads, vec_per_row;
    int* status;             // device status word
};
// Launch attribute that lets a kernel be made resident while the kernel ahead of it on the stream
// drains (such a kernel waits for that kernel's completion, griddepcontrol.wait, before it reads or
// writes anything).  Not used while the stream is being captured into a graph.  Returns the number
// of attributes written.
inline int overlap_launch_attribute(cudaStream_t st, cudaLaunchAttribute* attr) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return 0;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    return 1;
}
cudaError_t launch_kv_commit(const CommitArgs& a, int sm_count, cudaStream_t st);
cudaError_t launch_average(const float* traj, int n, int w, float* out, cudaStream_t st);
bool jmt_weights(int w, int w_out, std::vector<double>* weights);
cudaError_t launch_average_jmt(const float* traj, int n, int w, int w_out, const double* d_weights, float* out,
                               cudaStream_t st);
