// Confidence-threshold parallel unmasking: vocabulary-wide soft-max statistics and
// (Gumbel-perturbed) arg-max per MASKED row, then the per-rollout commit rule.
//
// Kernel 1 (unmask_stream_kernel): persistent grid, every warp on its own.  The MASKED rows of the
// call, cut into tiles of 2048 ids and laid end to end, are split into equal contiguous ranges, one
// per warp (tail of a row, whole rows, head of the next; one record per (row, warp), merged by the
// second kernel).  A warp streams its tiles from HBM once, through a ring of bulk asynchronous
// copies (cp.async.bulk, completion on an mbarrier, no multicast) into its own part of shared
// memory, three tiles deep; a lane takes 64 consecutive ids of a tile (16-byte reads, chunk order
// rotated by the lane so that the banks do not collide) and keeps running soft-max statistics.
// There is no CTA-wide barrier after the set-up, and nothing but the few logits that can win the
// arg-max is looked at twice.  Rows that are not MASKED are never read.
//
// Noise (temperature > 0).  The Gumbel draws are g = -ln(E) with E an exponential race over groups
// of 16 consecutive ids: group j has the 32-bit word R = word j % 4 of Philox block j / 4 (so the 64
// ids of a lane share one block), which fixes the "leader" 16 j + R % 16 holding the group's
// smallest E = -ln(U) / 16, U = ((R >> 4) + (f + 0.5) 2^-23) / 2^28; every other id of the group has
// E = E_leader - ln((f + 0.5) 2^-23) with 23 fine bits f of its own (second Philox stream, one block
// per 4 ids).  The word alone bounds all 16 draws from above, g < 32 ln 2 - ln(2^28 - 1 - (R >> 4)),
// and the leader's draw from below, which is what makes the kernel cheap.  While a lane's 64 ids
// are in shared memory the streaming pass takes the largest of their four words and forms
//   an upper bound of every score of the block: its largest logit + T * (bound of that word), and
//   a lower bound of one score: the logit of that word's leader + T * (lower bound of its draw);
// the warp keeps the largest lower bound so far, L (also: the largest logit so far with the smallest
// draw there is), and notes the blocks whose upper bound reaches it in a short list in shared
// memory.  After the piece L is a lower bound of the piece's best score, and only the noted blocks
// that still reach it (a handful) are read again, from L2, and scored exactly with the second
// stream, one group of 16 ids per lane.
// Any id left out cannot reach L, so the arg-max (lowest id on ties) is exact.
//
// Kernel 2 (unmask_finalize_kernel): one CTA per rollout merges the records of its rows, forms the
// confidences and applies the threshold / at-least-one rule.
#include "fdd_internal.h"
#include "tc_ptx.cuh"

#include <math_constants.h>

#include <atomic>

namespace {

constexpr int kWarps = 8;                             // per CTA; every warp works alone
constexpr int kThreads = kWarps * 32;
constexpr int kGroup = 16;                            // ids per group of the noise construction
constexpr int kLaneIds = 64;                          // consecutive ids a lane takes per tile: one Philox block of group words
constexpr int kTile = kUnmaskTile;                    // ids per tile (one bulk copy, one warp)
constexpr int kStages = 3;                            // tiles a warp holds in shared memory (two in flight while one is reduced)
constexpr int kMaxRows = kUnmaskMaxRows;              // rows of one launch (32 per thread in the set-up)
constexpr int kPiecePadNoisy = 5, kPiecePadGreedy = 3;   // the per-piece work of a warp, in tiles of streaming
constexpr int kMinPiecesPerRow = 8;                   // rows are cut on their own when each can have this many warps
constexpr int kMaxList = 224;                         // blocks in reach of the running lower bound kept per piece (a few dozen expected)
constexpr long long kCopyWaitLimit = 4000000000LL;    // SM clocks a warp waits for one of its own copies (about two seconds)
static_assert(kTile == 32 * kLaneIds, "a tile is 64 ids for each of 32 lanes");
static_assert(kMaxRows <= kThreads * 32, "the set-up gives every thread at most 32 rows");

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kGumbelMin = -2.95f;                  // no draw is smaller: E <= 36 / 16 + 23 ln 2 + ln 2 < e^2.95

constexpr uint32_t kPhiloxM0 = 0xD2511F53u, kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u, kPhiloxW1 = 0xBB67AE85u;
constexpr uint32_t kFineStream = 0x80000000u;         // added to the position word for the fine bits

// Philox4x32 with 10 rounds (Salmon et al., SC'11), written from the published round function:
// (c0, c1, c2, c3) -> (hi(M1 c2) ^ c1 ^ k0, lo(M1 c2), hi(M0 c0) ^ c3 ^ k1, lo(M0 c0)), the key
// bumped by the Weyl constants between rounds.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        if (r > 0) { k.x += kPhiloxW0; k.y += kPhiloxW1; }
        const uint64_t p0 = static_cast<uint64_t>(kPhiloxM0) * c.x;
        const uint64_t p1 = static_cast<uint64_t>(kPhiloxM1) * c.z;
        c = make_uint4(static_cast<uint32_t>(p1 >> 32) ^ c.y ^ k.x, static_cast<uint32_t>(p1),
                       static_cast<uint32_t>(p0 >> 32) ^ c.w ^ k.y, static_cast<uint32_t>(p0));
    }
    return c;
}
__device__ __forceinline__ uint32_t pick_word(const uint4& r, int k) {
    return k == 0 ? r.x : (k == 1 ? r.y : (k == 2 ? r.z : r.w));
}

// One bulk asynchronous copy global -> shared of this CTA; `bytes` and both addresses are multiples
// of 16.  Completion is counted in bytes on the mbarrier.
// The logits are read once: the copy marks their lines as the first to leave L2, so that a step's
// hundreds of MB do not push out what the attention kernel of the next step reads again (the
// shared prefix and the caches).
__device__ __forceinline__ uint64_t read_once_policy() {
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy)
                 : "memory");
}

// Wait for one of the warp's own copies; false once the time limit has run out.
__device__ __forceinline__ bool wait_copy(uint32_t bar, uint32_t parity) {
    if (tc::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!tc::mbar_try_wait(bar, parity))
        if (clock64() - t0 > kCopyWaitLimit) return false;
    return true;
}
// Position of the (k + 1)-th set bit of mask (k < popc(mask)).
__device__ __forceinline__ int nth_set_bit(uint32_t mask, int k) {
    for (; k > 0; --k) mask &= mask - 1;
    return __ffs(mask) - 1;
}

template <typename T> struct Logit;
template <> struct Logit<__nv_bfloat16> {
    static constexpr int kPerChunk = 8;                  // logits per 16-byte chunk
    __device__ static float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    __device__ static __nv_bfloat16 minus_inf() { return __ushort_as_bfloat16(0xFF80u); }
    __device__ static void widen(const uint4& w, float* out) {
        const uint32_t x[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            out[2 * i] = __uint_as_float(x[i] << 16);
            out[2 * i + 1] = __uint_as_float(x[i] & 0xFFFF0000u);
        }
    }
};
template <> struct Logit<float> {
    static constexpr int kPerChunk = 4;
    __device__ static float load1(const float* p) { return *p; }
    __device__ static float minus_inf() { return -CUDART_INF_F; }
    __device__ static void widen(const uint4& w, float* out) {
        out[0] = __uint_as_float(w.x); out[1] = __uint_as_float(w.y);
        out[2] = __uint_as_float(w.z); out[3] = __uint_as_float(w.w);
    }
};

// 16 logits starting at vocabulary id v0 (a multiple of 16), from global memory; ids >= vocab read as -inf.
template <typename T>
__device__ __forceinline__ void load_group(const T* row_ptr, int v0, int vocab, int vec_ok, float* val) {
    if (vec_ok && v0 + kGroup <= vocab) {
        const uint4* p = reinterpret_cast<const uint4*>(row_ptr + v0);
#pragma unroll
        for (int c = 0; c < kGroup / Logit<T>::kPerChunk; ++c) Logit<T>::widen(p[c], val + c * Logit<T>::kPerChunk);
    } else {
#pragma unroll
        for (int j = 0; j < kGroup; ++j) val[j] = (v0 + j < vocab) ? Logit<T>::load1(row_ptr + v0 + j) : -CUDART_INF_F;
    }
}

struct Best {
    float score, logit;
    int index;
};
__device__ __forceinline__ Best better(const Best& a, const Best& b) {
    // larger score wins; equal scores -> lower vocabulary id
    if (b.score > a.score || (b.score == a.score && b.index < a.index)) return b;
    return a;
}
__device__ __forceinline__ Best warp_best(Best b) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Best o;
        o.score = __shfl_xor_sync(0xFFFFFFFFu, b.score, off);
        o.logit = __shfl_xor_sync(0xFFFFFFFFu, b.logit, off);
        o.index = __shfl_xor_sync(0xFFFFFFFFu, b.index, off);
        b = better(b, o);
    }
    return b;
}

// ---- phase 2 of the noisy step: exact scores of the 16 ids of one group.
struct RowNoise {                                       // what fixes the draws of one row
    uint2 keys;                                         // the rollout's seed
    uint32_t pos, step, block_idx;
};
// Upper bound of every draw of a group from its word alone: U < (h + 1) / 2^28 = 1 - d / 2^28 with
// d = 2^28 - 1 - h, so -ln U > d / 2^28, E > d / 2^32 and g < 32 ln 2 - ln d (no bound for d = 0).
__device__ __forceinline__ float word_gumbel_bound(uint32_t R) {
    const uint32_t d = 0x0FFFFFFFu - (R >> 4);
    return d == 0u ? CUDART_INF_F : 22.18070977791825f - __logf(static_cast<float>(d)) + 1e-3f;
}
// E of a group's leader, -ln(U) / 16 with U = (h + (f + 0.5) 2^-23) / 2^28, h = R >> 4, on the fast
// logarithm (absolute error 4e-7 on [0.5, 2], 3 ulp elsewhere).  In the upper half of the range the
// logarithm goes through y = 1 - U, which fp32 holds almost exactly there: a series below 2^-6, where
// the fast logarithm of a number next to 1 would lose the leading digits of -ln U.
__device__ __forceinline__ float leader_exponential(uint32_t R, uint32_t f23) {
    const uint32_t h = R >> 4;
    const float frac = (static_cast<float>(f23) + 0.5f) * 1.1920928955078125e-07f;
    float nl;                                               // -ln(U)
    if (h >= (1u << 27)) {
        const float y = (static_cast<float>((1u << 28) - h) - frac) * 3.7252902984619140625e-09f;   // 1 - U
        nl = y < 0.015625f ? y * fmaf(y, fmaf(y, fmaf(y, 0.25f, 0.33333334f), 0.5f), 1.0f) : -__logf(1.0f - y);
    } else {
        nl = 19.408121055678468f - __logf(static_cast<float>(h) + frac);                            // 28 ln 2 - ln(2^28 U)
    }
    return nl * 0.0625f;
}
struct ScoreArgs {
    float lb, temperature;
    int vocab, vec_ok;
};
// The best exact score among the 16 ids of group v0 (score -inf if the group cannot reach the lower
// bound a.lb, or has no finite logit).  One Philox block for the group's word and four for the fine
// bits of its ids, all independent of each other and of the load; every id is then scored, without a
// branch: E = E_leader for the leader, E_leader - ln((f + 0.5) 2^-23) for the others, g = -ln E.
template <typename T>
__device__ __noinline__ Best score_group(const T* row_ptr, int v0, ScoreArgs a, RowNoise n) {
    Best best{-CUDART_INF_F, -CUDART_INF_F, 0x7FFFFFFF};
    float val[kGroup];
    load_group(row_ptr, v0, a.vocab, a.vec_ok, val);
    const int j = v0 >> 4;
    const uint32_t R = pick_word(philox4x32_10(make_uint4(static_cast<uint32_t>(j >> 2), n.pos, n.step, n.block_idx), n.keys), j & 3);
    uint32_t f[kGroup];
#pragma unroll
    for (int k = 0; k < kGroup / 4; ++k) {
        const uint4 r = philox4x32_10(make_uint4(static_cast<uint32_t>((v0 >> 2) + k), n.pos | kFineStream, n.step, n.block_idx), n.keys);
        f[4 * k] = r.x >> 9; f[4 * k + 1] = r.y >> 9; f[4 * k + 2] = r.z >> 9; f[4 * k + 3] = r.w >> 9;
    }
    float gmax = val[0];
#pragma unroll
    for (int i = 1; i < kGroup; ++i) gmax = fmaxf(gmax, val[i]);
    if (!(fmaf(a.temperature, word_gumbel_bound(R), gmax) >= a.lb - 1e-3f)) return best;
    const int li = static_cast<int>(R & 15u);
    uint32_t f_lead = f[0];
#pragma unroll
    for (int i = 1; i < kGroup; ++i) if (i == li) f_lead = f[i];
    const float e_lead = leader_exponential(R, f_lead);
#pragma unroll
    for (int i = kGroup - 1; i >= 0; --i) {             // downwards: equal scores keep the lower id
        const float e = i == li ? e_lead : e_lead + (15.942385152878742f - __logf(static_cast<float>(f[i]) + 0.5f));   // 23 ln 2 - ln(f + 0.5)
        const float sc = fmaf(a.temperature, -__logf(e), val[i]);
        if (val[i] > -CUDART_INF_F && sc >= best.score) best = Best{sc, val[i], v0 + i};
    }
    return best;
}

// The ri-th selected row (ascending) from the set-up's per-thread runs: thread t owns rows
// [t * per, (t + 1) * per), s_before[t] selected rows lie before its run, bit k of s_mask[t] says
// that row t * per + k is selected.
__device__ __forceinline__ int nth_selected_row(const int* s_before, const uint32_t* s_mask, int per, int ri) {
    int lo = 0, hi = kThreads - 1;
    while (lo < hi) {                                    // the last thread with s_before <= ri (its run is not empty)
        const int mid = (lo + hi + 1) >> 1;
        if (s_before[mid] <= ri) lo = mid; else hi = mid - 1;
    }
    return lo * per + nth_set_bit(s_mask[lo], ri - s_before[lo]);
}

// Item index of position v on the axis that has `pad` extra items in front of every row's ipr items.
__device__ __forceinline__ long long padded_to_item(long long v, int ipr, int pad) {
    const long long r = v / (ipr + pad);
    const long long off = v - r * (ipr + pad);
    return r * ipr + (off > pad ? off - pad : 0);
}

// A block (the 64 ids of one lane in one tile) whose upper bound reached the running lower bound.
struct Reach {
    float ub;            // upper bound of the block's scores
    uint16_t tile;       // tile inside the piece
    uint16_t lane;
};
static_assert(sizeof(Reach) == 8, "eight bytes per kept block");

// Shared memory of the streaming kernel beyond its static arrays: the rings, the lists of kept blocks, the barriers.
template <typename T>
constexpr int stream_smem_bytes() {
    return kWarps * kStages * kTile * static_cast<int>(sizeof(T)) + kWarps * kMaxList * 8 + kWarps * kStages * 8;
}

template <typename T, bool NOISY>
__global__ void __launch_bounds__(kThreads, sizeof(T) == 2 ? 2 : 1)
unmask_stream_kernel(const T* __restrict__ logits, const uint8_t* __restrict__ state,
                     const __grid_constant__ UnmaskSets sets, UnmaskPartial* __restrict__ partial,
                     int vocab, int tiles_per_item, float temperature,
                     uint32_t block_idx, uint32_t step, int bulk_ok, int select_state,
                     const uint32_t* __restrict__ step_counter, int* __restrict__ status) {
    // The launch may have been made resident before the kernel ahead of it on the stream was done (its
    // set-up then overlaps that kernel's tail); nothing is read before this wait.  The kernel behind
    // this one (the per-rollout step) may come in as soon as every CTA here has started.
    tc::grid_dependency_wait();
    tc::grid_launch_dependents();
    if (step_counter != nullptr) step += *step_counter;    // the denoising step as counted on the device
    const int rows = sets.row_off[sets.n_sets];
    __shared__ int s_before[kThreads];                  // selected rows before the thread's run
    __shared__ uint32_t s_mask[kThreads];               // which rows of the thread's run are selected (MASKED, or DRAFT for the verifier)
    __shared__ int s_warp_count[kWarps];
    __shared__ int s_n_list[kWarps];
    extern __shared__ __align__(128) unsigned char s_dyn[];
    constexpr int kStageBytes = kTile * static_cast<int>(sizeof(T));
    constexpr int kPerChunk = Logit<T>::kPerChunk;
    constexpr int kLaneChunks = kLaneIds / kPerChunk;   // 16-byte chunks of a lane's 64 ids: 8 (bf16) or 16 (fp32)
    constexpr int kLaneGroups = kLaneIds / kGroup;      // groups of a lane's 64 ids

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    unsigned char* ring = s_dyn + warp * (kStages * kStageBytes);
    Reach* list = reinterpret_cast<Reach*>(s_dyn + kWarps * kStages * kStageBytes) + warp * kMaxList;
    uint64_t* bars = reinterpret_cast<uint64_t*>(s_dyn + kWarps * kStages * kStageBytes + kWarps * kMaxList * 8) + warp * kStages;

    // ---- set-up (the only CTA-wide part): which rows are selected.  A thread takes a run of
    // consecutive rows, one block-wide prefix sum places the runs.
    const int per = (rows + kThreads - 1) / kThreads;              // <= 32 (rows <= 8192)
    int n_rows;
    {
        const int r_begin = min(rows, tid * per), r_end = min(rows, r_begin + per);
        uint32_t mine = 0;
        for (int r = r_begin; r < r_end; ++r) mine |= (state[r] == select_state ? 1u : 0u) << (r - r_begin);
        const int cnt = __popc(mine);
        int incl = cnt;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += up;
        }
        if (lane == 31) s_warp_count[warp] = incl;
        if (lane == 0) {
            s_n_list[warp] = 0;
            if (bulk_ok) {
                for (int s = 0; s < kStages; ++s) tc::mbar_init(tc::smem_u32(&bars[s]), 1);
                tc::fence_barrier_init();
            }
        }
        __syncthreads();
        int before = incl - cnt, total = 0;
#pragma unroll
        for (int w2 = 0; w2 < kWarps; ++w2) {
            if (w2 < warp) before += s_warp_count[w2];
            total += s_warp_count[w2];
        }
        s_before[tid] = before;
        s_mask[tid] = mine;
        n_rows = total;
        __syncthreads();
    }
    if (n_rows == 0) return;

    // ---- this warp's range of work items.  An item is tiles_per_item consecutive tiles of a row
    // (the last item of a row may be shorter); a row has items_per_row of them and as many record
    // slots.  Two ways to hand them out:
    //  - few rows (at least kMinPiecesPerRow warps for each): a row is cut into ppr equal pieces, warp c
    //    takes piece c % ppr of row c / ppr.  No warp then works on two rows, which would cost it two
    //    rounds of the per-piece work (reductions, exact re-scoring, a record) while the others wait;
    //  - otherwise the items of all rows, laid end to end, are cut into equal contiguous ranges, warp
    //    c (of the G that get work) owns items [W c / G, W (c + 1) / G): tail of a row, whole rows, head
    //    of the next.
    const int tiles_per_row = (vocab + kTile - 1) / kTile;
    const int ipr = (tiles_per_row + tiles_per_item - 1) / tiles_per_item;
    const long long W = static_cast<long long>(n_rows) * ipr;
    const long long warps_all = static_cast<long long>(gridDim.x) * kWarps;
    const long long gw = static_cast<long long>(warp) * gridDim.x + blockIdx.x;   // warps of a CTA lie a grid apart: few items spread over all SMs
    const int ppr = static_cast<int>(min(static_cast<long long>(ipr), warps_all / n_rows));   // pieces per row if rows are cut on their own
    const bool by_row = ppr == ipr || ppr >= kMinPiecesPerRow;                   // (few pieces per row would leave too many warps without work)
    const long long G = by_row ? static_cast<long long>(n_rows) * ppr : min(warps_all, W);
    if (gw >= G) return;
    // (in items; only where a range is much longer than it)
    const int pad = (W >= 16 * G) ? ((NOISY ? kPiecePadNoisy : kPiecePadGreedy) + tiles_per_item - 1) / tiles_per_item : 0;
    const long long Vp = static_cast<long long>(n_rows) * (ipr + pad);
    long long range_begin, range_end;
    if (by_row) {
        const int ri = static_cast<int>(gw / ppr), pc = static_cast<int>(gw - static_cast<long long>(ri) * ppr);
        range_begin = static_cast<long long>(ri) * ipr + ipr * pc / ppr;
        range_end = static_cast<long long>(ri) * ipr + ipr * (pc + 1) / ppr;
    } else {
        // A warp whose range takes in a row's start works on two rows and pays the per-piece work
        // twice.  That work is counted as `pad` items at the start of every row: the ranges are equal on
        // the axis with those items put in, and are then mapped back (a range that falls inside the
        // padding alone, which needs a range shorter than pad, is empty).
        range_begin = padded_to_item(Vp * gw / G, ipr, pad);
        range_end = padded_to_item(Vp * (gw + 1) / G, ipr, pad);
        if (range_begin >= range_end) return;
    }

    const uint32_t full = 0xFFFFFFFFu;
    const int sw = lane & 7;                            // rotation of the chunk order (bank conflicts)
    bool alive = true;                                  // false once a wait for a copy ran out

    // ---- producer side (lane 0 issues, every lane keeps the same cursor): tile k of the warp's
    // sequence goes to stage k % kStages, which is the stage the consumer has just left
    const uint32_t ring_u32 = tc::smem_u32(ring), bars_u32 = tc::smem_u32(bars);
    long long p_at = range_begin;                       // next item to open
    int p_tile = 0, p_tile_end = 0;
    const T* p_row_ptr = nullptr;
    uint32_t p_k = 0;
    const uint64_t l2_policy = read_once_policy();
    auto produce_one = [&](int stage) {
        if (!bulk_ok) return;
        if (p_tile == p_tile_end) {
            if (p_at >= range_end) return;
            const int ri = static_cast<int>(p_at / ipr);
            const int c0 = static_cast<int>(p_at - static_cast<long long>(ri) * ipr);
            const int c1 = static_cast<int>(min(static_cast<long long>(ipr), c0 + (range_end - p_at)));
            p_at += c1 - c0;
            p_tile = c0 * tiles_per_item;
            p_tile_end = min(tiles_per_row, c1 * tiles_per_item);
            p_row_ptr = logits + static_cast<size_t>(nth_selected_row(s_before, s_mask, per, ri)) * vocab;
        }
        if (lane == 0) {
            const int v0 = p_tile * kTile;
            const uint32_t bytes = static_cast<uint32_t>(min(kTile, vocab - v0)) * sizeof(T);
            const uint32_t bar = bars_u32 + stage * 8;
            tc::mbar_arrive_expect_tx(bar, bytes);
            bulk_load(ring_u32 + stage * kStageBytes, p_row_ptr + v0, bytes, bar, l2_policy);
        }
        ++p_tile;
        ++p_k;
    };
    for (int s = 0; s < kStages; ++s) produce_one(s);

    uint32_t c_k = 0;                                   // tiles consumed so far: the next one sits in stage c_k % kStages
    int stage = 0;
    uint32_t phase = 0;                                 // parity of the stage's current use
    for (long long at = range_begin; at < range_end && alive;) {
        // ---- open the piece: items [at, at + n) of one row
        const int ri = static_cast<int>(at / ipr);
        const int chunk0 = static_cast<int>(at - static_cast<long long>(ri) * ipr);
        const int chunk1 = static_cast<int>(min(static_cast<long long>(ipr), chunk0 + (range_end - at)));
        at += chunk1 - chunk0;
        const int tile0 = chunk0 * tiles_per_item, tile1 = min(tiles_per_row, chunk1 * tiles_per_item);
        const int row = nth_selected_row(s_before, s_mask, per, ri);
        const int seg_end = min(vocab, tile1 * kTile);
        // which of the row's records this is, and how many there are
        int seg, segs;
        if (by_row) {
            seg = static_cast<int>(gw - static_cast<long long>(ri) * ppr);
            segs = ppr;
        } else {
            // the warps that hold the row's first and last item, on the padded axis
            const long long v_first = static_cast<long long>(ri) * (ipr + pad) + pad;
            const int w_first = static_cast<int>(((v_first + 1) * G + Vp - 1) / Vp) - 1;
            const int w_last = static_cast<int>(((v_first + ipr) * G + Vp - 1) / Vp) - 1;
            seg = static_cast<int>(gw) - w_first;
            segs = w_last - w_first + 1;
        }
        const T* row_ptr = logits + static_cast<size_t>(row) * vocab;
        int set = 0;
        while (set + 1 < sets.n_sets && row >= sets.row_off[set + 1]) ++set;
        const int local = row - sets.row_off[set];
        const int fork = local / sets.d[set], pos = local - fork * sets.d[set];   // rollout inside its set
        uint2 keys = make_uint2(0u, 0u);
        if (NOISY) {
            const uint64_t seed = sets.seeds[set][fork];
            // (through a shuffle, which tells the compiler that the key is the same in every lane: the
            // round keys of the Philox blocks then live in uniform registers)
            keys = make_uint2(__shfl_sync(0xFFFFFFFFu, static_cast<uint32_t>(seed), 0),
                              __shfl_sync(0xFFFFFFFFu, static_cast<uint32_t>(seed >> 32), 0));
        }

        // ---- pass 1: stream the piece; per lane the running maximum m and sum exp(l - m).  The greedy
        // step also keeps the first tile t1 that showed m (u1 = m there); the noisy step keeps the warp's
        // running lower bound lb of the piece's best score and lists the blocks that reach it.
        float m = -CUDART_INF_F, s = 0.0f, nml = 0.0f;  // nml = -m log2(e) once m is finite
        float u1 = -CUDART_INF_F, lb = -CUDART_INF_F;
        int t1 = tile0;
        Best best{-CUDART_INF_F, -CUDART_INF_F, 0x7FFFFFFF};
        for (int tile = tile0; tile < tile1; ++tile) {
            unsigned char* buf = ring + stage * kStageBytes;
            const int tile_base = tile * kTile;
            if (bulk_ok) {
                if (!wait_copy(bars_u32 + stage * 8, phase)) alive = false;
                alive = __all_sync(full, alive);
                if (!alive) break;
            } else {
                // rows that bulk copies cannot address (odd vocabulary, unaligned base): the warp fills the stage itself
                T* dst = reinterpret_cast<T*>(buf);
                for (int i = lane; i < kTile; i += 32)
                    dst[i] = (tile_base + i < vocab) ? row_ptr[tile_base + i] : Logit<T>::minus_inf();
                __syncwarp();
            }
            const int vb = tile_base + lane * kLaneIds;  // first id of the lane's 64
            const uint4* sp = reinterpret_cast<const uint4*>(buf) + lane * kLaneChunks;
            const T* lp = reinterpret_cast<const T*>(buf) + lane * kLaneIds;
            float bm64 = -CUDART_INF_F;
            // (per lane: in a row's last tile the lanes whose 64 ids all exist take the fast path too, the
            // lanes beyond the row's end have nothing to do, and at most one lane straddles the end)
            const bool whole = vb + kLaneIds <= seg_end;
            uint4 rq = make_uint4(0u, 0u, 0u, 0u);      // the words of the block's four groups
            if (NOISY) rq = philox4x32_10(make_uint4(static_cast<uint32_t>(vb >> 6), pos, step, block_idx), keys);
            if (whole) {
                // whole tile: two halves of 32 logits, chunk c of the lane read from place c ^ sw (the
                // eight lanes of a quarter warp then touch eight different 16-byte columns of the banks)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    float v[32];
#pragma unroll
                    for (int c = 0; c < kLaneChunks / 2; ++c)
                        Logit<T>::widen(sp[(h * (kLaneChunks / 2) + c) ^ sw], v + c * kPerChunk);
                    float g8[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) g8[u] = tc::max3(v[4 * u], v[4 * u + 1], fmaxf(v[4 * u + 2], v[4 * u + 3]));
                    const float bm = tc::max3(tc::max3(g8[0], g8[1], g8[2]), tc::max3(g8[3], g8[4], g8[5]), fmaxf(g8[6], g8[7]));
                    bm64 = fmaxf(bm64, bm);
                    {
                        // rescale by 2^((m - mn) log2 e): exactly 1 while the maximum stands (the rounded nml
                        // must not enter here).  Without a branch, so that the tile step is one straight run of
                        // instructions and the Philox rounds of the noisy step overlap the exponentials.
                        const float mn = fmaxf(m, bm);
                        s *= tc::ex2(mn == m ? 0.0f : (m - mn) * kLog2e);
                        m = mn;
                        nml = mn > -CUDART_INF_F ? -mn * kLog2e : 0.0f;
                    }
                    // packed fp32x2 arithmetic: one FMA and one add per two logits
                    const uint64_t l2e2 = tc::pack2(kLog2e, kLog2e), nm2 = tc::pack2(nml, nml);
                    uint64_t acc[2] = {tc::pack2(0.f, 0.f), tc::pack2(0.f, 0.f)};
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        float x0, x1;
                        tc::unpack2(tc::fma2(tc::pack2(v[i], v[i + 1]), l2e2, nm2), x0, x1);
                        acc[(i >> 1) & 1] = tc::add2(acc[(i >> 1) & 1], tc::pack2(tc::ex2(x0), tc::ex2(x1)));
                    }
                    float a0, a1;
                    tc::unpack2(tc::add2(acc[0], acc[1]), a0, a1);
                    s += a0 + a1;
                }
            } else if (vb < seg_end) {
                // the lane that straddles the row's end: ids from seg_end on do not exist
                for (int e = 0; e < kLaneIds; ++e)
                    if (vb + e < seg_end) bm64 = fmaxf(bm64, Logit<T>::load1(lp + e));
                if (bm64 > m) {
                    s *= tc::ex2((m - bm64) * kLog2e);
                    m = bm64;
                    nml = -bm64 * kLog2e;
                }
                float add = 0.0f;
                for (int e = 0; e < kLaneIds; ++e)
                    if (vb + e < seg_end) add += tc::ex2(fmaf(Logit<T>::load1(lp + e), kLog2e, nml));
                s += add;
            }
            if (!NOISY) {
                t1 = bm64 > u1 ? tile : t1;             // strictly: t1 is the first tile that holds the lane's maximum
                u1 = fmaxf(u1, bm64);
            } else {
                // The block's four words: the largest one bounds every draw of the block, and its group's
                // leader gives a score that exists.  d = 2^28 - 1 - (R >> 4), cut to 23 bits (d5 = d / 32,
                // rounded down) so that it turns into a float exactly; both bounds stay on the safe side.
                uint32_t rmax;
                int gp;                                 // the group (of the block's four) that holds rmax
                if (whole) {
                    const uint32_t r01 = max(rq.x, rq.y), r23 = max(rq.z, rq.w);
                    rmax = max(r01, r23);
                    gp = rmax == rq.x ? 0 : (rmax == rq.y ? 1 : (rmax == rq.z ? 2 : 3));
                } else {
                    rmax = rq.x;                        // (group 0 exists: the block does)
                    gp = 0;
#pragma unroll
                    for (int g = 1; g < kLaneGroups; ++g)
                        if (vb + g * kGroup < seg_end && pick_word(rq, g) > rmax) { rmax = pick_word(rq, g); gp = g; }
                }
                const uint32_t d5 = (0x0FFFFFFFu - (rmax >> 4)) >> 5;
                const float fd5 = __uint_as_float(0x4B000000u | d5) - 8388608.0f;          // d5 as a float, exactly
                // g < 32 ln 2 - ln d <= 27 ln 2 - ln d5
                const float g_hi = d5 == 0u ? CUDART_INF_F : fmaf(-kLn2, __log2f(fd5), 18.71497388f + 2e-3f);
                const float ub = fmaf(temperature, g_hi, bm64);
                const bool reaches = bm64 > -CUDART_INF_F && ub >= lb - 1e-3f;
                // (no block in reach: no score of this tile step can raise the bound either, since the
                // lower bounds below lie under the blocks' upper bounds)
                if (__any_sync(full, reaches)) {
                    // g_leader >= 32 ln 2 - ln((d + 1) (1 + y)), y = (d + 1) / 2^28 <= 1 / 2; d + 1 <= 32 (d5 + 1)
                    const float y = (fd5 + 1.0f) * 1.1920928955078125e-07f;                 // >= (d + 1) / 2^28
                    const float g_lo = y <= 0.5f ? fmaf(-kLn2, __log2f(fd5 + 1.0f), 18.71497388f - 2e-3f) - y : kGumbelMin;
                    const int li = gp * kGroup + static_cast<int>(rmax & 15u);
                    // a score that exists in this block: that leader's, or the largest logit's with the smallest draw there is
                    float lo = bm64 > -CUDART_INF_F ? fmaf(temperature, kGumbelMin, bm64) : -CUDART_INF_F;
                    if (vb + li < seg_end) lo = fmaxf(lo, fmaf(temperature, g_lo, Logit<T>::load1(lp + li)));
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) lo = fmaxf(lo, __shfl_xor_sync(full, lo, off));
                    lb = fmaxf(lb, lo);
                    if (reaches && ub >= lb - 1e-3f) {
                        const int slot = atomicAdd(&s_n_list[warp], 1);
                        if (slot < kMaxList) list[slot] = Reach{ub, static_cast<uint16_t>(tile - tile0), static_cast<uint16_t>(lane)};
                    }
                }
            }
            __syncwarp();                               // every lane is done with the stage
            produce_one(stage);                         // tile c_k + kStages goes into it
            ++c_k;
            if (++stage == kStages) {
                stage = 0;
                phase ^= 1u;
            }
        }
        if (!alive) break;

        if (NOISY) {
            // ---- pass 2: lb is now a lower bound of the piece's best score.  The listed blocks that still
            // reach it are read again (the piece has just gone through L2) and scored exactly, group by
            // group: a turn deals out eight blocks, one group per lane, so that the loads are in flight
            // together.  (A list that ran over, or a piece of more than 65536 tiles: every block.)
            __syncwarp();
            const RowNoise noise{keys, static_cast<uint32_t>(pos), step, block_idx};
            const ScoreArgs sargs{lb, temperature, vocab, bulk_ok};
            const float cut = lb - 1e-3f;
            const int n_seen = *reinterpret_cast<volatile int*>(&s_n_list[warp]);
            const bool every = n_seen > kMaxList || tile1 - tile0 > 65536;
            int n_blocks = 0;
            if (every) {
                n_blocks = (tile1 - tile0) * 32;
            } else {
                // keep the blocks that reach the final bound, in place
                for (int c0 = 0; c0 < n_seen; c0 += 32) {
                    const int c = c0 + lane;
                    Reach r{-CUDART_INF_F, 0, 0};
                    if (c < n_seen) r = list[c];
                    const bool keep = r.ub >= cut;
                    const uint32_t km = __ballot_sync(full, keep);
                    if (keep) list[n_blocks + __popc(km & ((1u << lane) - 1u))] = r;
                    n_blocks += __popc(km);
                    __syncwarp();
                }
            }
            // Up to eight listed blocks (the usual case): one turn, a group of 16 ids per lane.
            if (n_blocks <= 32 / kLaneGroups) {
                const int blk = lane / kLaneGroups;
                if (blk < n_blocks) {
                    const int tl = every ? blk / 32 : list[blk].tile, fl = every ? blk % 32 : list[blk].lane;
                    const int v0 = (tile0 + tl) * kTile + fl * kLaneIds + (lane % kLaneGroups) * kGroup;
                    if (v0 < seg_end) best = better(best, score_group<T>(row_ptr, v0, sargs, noise));
                }
                __syncwarp();
                n_blocks = 0;
            }
            // More: thirty-two listed blocks at a time, in two stages.  Stage one, a block per lane: the
            // block's four words (one Philox block) and the largest logit of each of its four groups give a
            // bound per group, which is tighter than the block's (about one group in three of a listed
            // block still reaches).  Stage two, a group per lane: the groups that reach are dealt out over
            // the lanes and scored exactly, so that no lane idles behind a group that was ruled out.  The
            // best exact score so far raises the bar for the next thirty-two.
            ScoreArgs turn_args = sargs;
            for (int c0 = 0; c0 < n_blocks; c0 += 32) {
                const int c = c0 + lane;
                int vb0 = seg_end;                              // first id of this lane's block (none: seg_end)
                if (c < n_blocks) {
                    const int tl = every ? c / 32 : list[c].tile, fl = every ? c % 32 : list[c].lane;
                    vb0 = (tile0 + tl) * kTile + fl * kLaneIds;
                }
                uint32_t reach = 0;                             // bit g: group g of the block can reach the bar
                if (vb0 < seg_end) {
                    // (a listed block lies inside the piece as a whole; only the row's end can cut it short,
                    // and ids beyond the vocabulary read as -inf)
                    const uint4 rq4 = philox4x32_10(make_uint4(static_cast<uint32_t>(vb0 >> 6), static_cast<uint32_t>(pos), step, block_idx), keys);
                    float val[kLaneGroups][kGroup];
#pragma unroll
                    for (int g = 0; g < kLaneGroups; ++g) load_group(row_ptr, vb0 + g * kGroup, vocab, bulk_ok, val[g]);
#pragma unroll
                    for (int g = 0; g < kLaneGroups; ++g) {
                        float gmax = val[g][0];
#pragma unroll
                        for (int i = 1; i < kGroup; ++i) gmax = fmaxf(gmax, val[g][i]);
                        if (fmaf(temperature, word_gumbel_bound(pick_word(rq4, g)), gmax) >= turn_args.lb - 1e-3f) reach |= 1u << g;
                    }
                }
                uint32_t mg[kLaneGroups];
                int total = 0;
#pragma unroll
                for (int g = 0; g < kLaneGroups; ++g) {
                    mg[g] = __ballot_sync(full, (reach >> g) & 1u);
                    total += __popc(mg[g]);
                }
                for (int j0 = 0; j0 < total; j0 += 32) {
                    int r = j0 + lane, g = 0, src = 0;
                    const bool act = r < total;
                    if (act) {
                        while (r >= __popc(mg[g])) { r -= __popc(mg[g]); ++g; }
                        src = nth_set_bit(mg[g], r);
                    }
                    const int v_src = __shfl_sync(full, vb0, src);
                    if (act) best = better(best, score_group<T>(row_ptr, v_src + g * kGroup, turn_args, noise));
                    __syncwarp();
                }
                if (c0 + 32 < n_blocks) {
                    float seen = best.score;
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) seen = fmaxf(seen, __shfl_xor_sync(full, seen, off));
                    turn_args.lb = fmaxf(turn_args.lb, seen);
                }
            }
            if (lane == 0) s_n_list[warp] = 0;          // the list is empty again for the next piece
        } else {
            // ---- greedy: the piece's maximum and its first place.  The lanes that hold the maximum look
            // for it in the 64 ids of the first tile that showed it (equal values in later tiles have
            // higher ids).
            float pm = u1;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) pm = fmaxf(pm, __shfl_xor_sync(full, pm, off));
            if (pm > -CUDART_INF_F && u1 == pm) {
                int at_e = 0x7FFFFFFF;
                const int vb = t1 * kTile + lane * kLaneIds;
#pragma unroll
                for (int g = kLaneGroups - 1; g >= 0; --g) {
                    float val[kGroup];
                    load_group(row_ptr, vb + g * kGroup, vocab, bulk_ok, val);
#pragma unroll
                    for (int i = kGroup - 1; i >= 0; --i)
                        if (val[i] == pm) at_e = vb + g * kGroup + i;
                }
                best = Best{pm, pm, at_e};
            }
        }

        // ---- the piece's record
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float mx = __shfl_xor_sync(full, m, off);
            const float sx = __shfl_xor_sync(full, s, off);
            const float mn = fmaxf(m, mx);
            if (mn > -CUDART_INF_F) s = s * __expf(m - mn) + sx * __expf(mx - mn);
            m = mn;
        }
        best = warp_best(best);
        if (lane == 0) {
            UnmaskPartial out;
            out.row_max = m; out.sum_exp = s; out.best_score = best.score; out.best_logit = best.logit;
            out.best_index = best.index;
            out.pad[0] = segs;                          // how many records this row has (read from record 0)
            out.pad[1] = out.pad[2] = 0;
            partial[static_cast<size_t>(row) * ipr + seg] = out;
        }
        __syncwarp();
    }

    if (!alive) {
        // A copy did not arrive in time: say so, then give the copies still in flight one more bounded
        // wait each before the shared memory they write to is handed back.
        if (lane == 0 && status != nullptr) atomicCAS(status, 0, FDD_ERR_DEVICE_TIMEOUT);
        for (uint32_t k = c_k; k < p_k; ++k) {
            const long long t0 = clock64();
            while (!tc::mbar_try_wait(tc::smem_u32(&bars[k % kStages]), (k / kStages) & 1u))
                if (clock64() - t0 > kCopyWaitLimit) break;
        }
    }
}

// Soft-max statistics of a row spread over several records: (m, s) with s = sum exp(l - m).
__device__ __forceinline__ void merge_stats(float& m, float& s, float m2, float s2) {
    const float mn = fmaxf(m, m2);
    if (mn > -CUDART_INF_F) s = s * __expf(m - mn) + s2 * __expf(m2 - mn);
    m = mn;
}

constexpr int kFinalizeThreads = 512;               // the first 128 are the positions of the rollout; all of them merge records

__global__ void __launch_bounds__(kFinalizeThreads)
unmask_finalize_kernel(const UnmaskPartial* __restrict__ partial, int32_t* __restrict__ tokens,
                       uint8_t* __restrict__ state, int32_t* __restrict__ n_committed,
                       int32_t* __restrict__ n_left, float* __restrict__ conf_out,
                       const __grid_constant__ UnmaskSets sets, int items_per_row, float threshold, int commit_state,
                       uint32_t* __restrict__ step_bump, int2* __restrict__ left_mirror, int mirror_stamp) {
    tc::grid_launch_dependents();                       // the next kernel may be made resident; it waits for this one
    tc::grid_dependency_wait();                         // the streaming kernel's records are complete and visible
    // (the streaming kernel of this call has read the counter; the next call sees it advanced)
    if (step_bump != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *step_bump += 1u;
    const int fork = blockIdx.x;                        // rollout index over all sets of the call
    const int i = threadIdx.x, warp = i >> 5, lane = i & 31;
    int set = 0;
    while (set + 1 < sets.n_sets && fork >= sets.fork_off[set + 1]) ++set;
    const int d = sets.d[set];
    const int row0 = sets.row_off[set] + (fork - sets.fork_off[set]) * d;
    __shared__ float s_conf[128];
    __shared__ int s_tok[128], s_nrec[128], s_rows[128];
    __shared__ int s_masked, s_pass, s_max_rec;
    if (i == 0) { s_masked = 0; s_pass = 0; s_max_rec = 1; }
    __syncthreads();

    // ---- the MASKED positions of the rollout and how many records each has (one round trip each)
    const int row = row0 + i;
    const bool masked = i < d && state[row] == FDD_MASKED;     // (d <= 128: threads beyond it only help with the merge)
    if (masked) {
        // records the first kernel wrote for this row (never more than the row has slots)
        const int n_rec = max(1, min(items_per_row, partial[static_cast<size_t>(row) * items_per_row].pad[0]));
        s_nrec[i] = n_rec;
        s_rows[atomicAdd(&s_masked, 1)] = i;
        atomicMax(&s_max_rec, n_rec);
    }
    if (i < 128) s_conf[i] = -1.0f;
    __syncthreads();
    const int n_masked = s_masked;

    // ---- merge the records: a group of w lanes per position (w = the largest record count, rounded up
    // to a power of two, 32 at most), so that all records of 32 / w positions are fetched in one round
    // trip per warp.  Early steps have many positions with two or three records, late steps a few
    // positions with up to a record per tile.
    int w = 1;
    while (w < s_max_rec && w < 32) w <<= 1;
    const int per = 32 / w, sub = lane / w, sl = lane - sub * w;
    for (int base = warp * per; base < n_masked; base += (kFinalizeThreads / 32) * per) {   // (warp-uniform bounds)
        const int k = base + sub;
        const bool valid = k < n_masked;
        const int j = valid ? s_rows[k] : 0;
        const int nr = valid ? s_nrec[j] : 0;
        const UnmaskPartial* p = partial + static_cast<size_t>(row0 + j) * items_per_row;
        float M = -CUDART_INF_F, S = 0.0f;
        Best B{-CUDART_INF_F, -CUDART_INF_F, 0x7FFFFFFF};
        for (int c = sl; c < nr; c += w) {
            const float4 st4 = *reinterpret_cast<const float4*>(&p[c]);     // row_max, sum_exp, best_score, best_logit
            const int idx = p[c].best_index;
            merge_stats(M, S, st4.x, st4.y);
            B = better(B, Best{st4.z, st4.w, idx});
        }
        for (int off = w >> 1; off > 0; off >>= 1) {
            const float m2 = __shfl_xor_sync(0xFFFFFFFFu, M, off), s2 = __shfl_xor_sync(0xFFFFFFFFu, S, off);
            Best o;
            o.score = __shfl_xor_sync(0xFFFFFFFFu, B.score, off);
            o.logit = __shfl_xor_sync(0xFFFFFFFFu, B.logit, off);
            o.index = __shfl_xor_sync(0xFFFFFFFFu, B.index, off);
            merge_stats(M, S, m2, s2);
            B = better(B, o);
        }
        if (valid && sl == 0) {
            s_conf[j] = expf(B.logit - M) / S;
            s_tok[j] = B.index;
        }
    }
    __syncthreads();

    // ---- the commit rule of the rollout
    const float conf = i < 128 ? s_conf[i] : -1.0f;
    if (i < d && conf_out) conf_out[row] = masked ? conf : CUDART_NAN_F;
    const bool pass = masked && conf > threshold;
    if (pass) atomicAdd(&s_pass, 1);
    __syncthreads();
    const int n_pass = s_pass;
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
        tokens[row] = s_tok[i];
        state[row] = static_cast<uint8_t>(commit_state);
    }
    if (i == 0) {
        const int nc = (n_masked == 0) ? 0 : (n_pass > 0 ? n_pass : 1);
        n_committed[fork] = nc;
        n_left[fork] = n_masked - nc;
        // host memory the GPU can write: count and stamp go out as one 8-byte store, so a host that
        // sees the stamp of this call sees its count
        if (left_mirror != nullptr)
            *reinterpret_cast<unsigned long long*>(left_mirror + fork) =
                (static_cast<unsigned long long>(static_cast<uint32_t>(mirror_stamp)) << 32) | static_cast<uint32_t>(n_masked - nc);
    }
}


// Accept scan of Scaffold Speculative Decoding: one CTA per rollout.  The first kernel has left, for
// every DRAFT row, the verifier's token (arg-max of its perturbed logits).  Going left to right, a
// draft is accepted while it equals the verifier's token; at the first mismatch the verifier's token
// replaces it and every later draft goes back to MASKED.
__global__ void __launch_bounds__(128)
ss_accept_kernel(const UnmaskPartial* __restrict__ partial, int32_t* __restrict__ tokens,
                 uint8_t* __restrict__ state, int32_t* __restrict__ n_accepted, int32_t* __restrict__ n_left,
                 const __grid_constant__ UnmaskSets sets, int items_per_row) {
    const int fork = blockIdx.x;
    const int i = threadIdx.x;
    int set = 0;
    while (set + 1 < sets.n_sets && fork >= sets.fork_off[set + 1]) ++set;
    const int d = sets.d[set];
    const int row = sets.row_off[set] + (fork - sets.fork_off[set]) * d + i;
    __shared__ int s_first_mismatch, s_accepted, s_masked;
    if (i == 0) { s_first_mismatch = 0x7FFFFFFF; s_accepted = 0; s_masked = 0; }
    __syncthreads();
    int st = FDD_SCAFFOLD, tok = 0;
    bool draft = false, mismatch = false;
    if (i < d) {
        st = state[row];
        draft = st == FDD_DRAFT;
        if (draft) {
            const UnmaskPartial* p = partial + static_cast<size_t>(row) * items_per_row;
            const int n_rec = p[0].pad[0];
            Best B{-CUDART_INF_F, -CUDART_INF_F, 0x7FFFFFFF};
            for (int c = 0; c < n_rec; ++c) B = better(B, Best{p[c].best_score, p[c].best_logit, p[c].best_index});
            tok = B.index;
            mismatch = tok != tokens[row];
            if (mismatch) atomicMin(&s_first_mismatch, i);
        }
    }
    __syncthreads();
    const int stop = s_first_mismatch;                  // position of the replacement token, if any
    if (draft) {
        if (i <= stop) {
            if (i == stop) tokens[row] = tok;           // the verifier's token, always accepted
            state[row] = FDD_COMMITTED;
            atomicAdd(&s_accepted, 1);
        } else {
            state[row] = FDD_MASKED;                    // discarded draft
            atomicAdd(&s_masked, 1);
        }
    } else if (i < d && st == FDD_MASKED) {
        atomicAdd(&s_masked, 1);
    }
    __syncthreads();
    if (i == 0) {
        n_accepted[fork] = s_accepted;
        n_left[fork] = s_masked;
    }
}

}  // namespace

namespace {

// Per-device set-up of the streaming kernels (they need more dynamic shared memory than a kernel
// gets without asking) and the device's SM count, done by the first launch on each device.
constexpr int kMaxDevices = 64;
std::atomic<int> g_device_ready[kMaxDevices];
int g_device_sms[kMaxDevices];
int g_device_ctas[kMaxDevices][4];          // resident CTAs per SM of each instantiation: [bf16 noisy, bf16 greedy, fp32 noisy, fp32 greedy]

template <typename T, bool NOISY>
cudaError_t setup_one(int* ctas_per_sm) {
    auto kernel = unmask_stream_kernel<T, NOISY>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, stream_smem_bytes<T>());
    // all of the SM's configurable memory as shared memory: two CTAs of the bf16 kernel need 215 KB
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(ctas_per_sm, kernel, kThreads, stream_smem_bytes<T>());
    if (e == cudaSuccess && *ctas_per_sm < 1) e = cudaErrorLaunchOutOfResources;
    return e;
}

cudaError_t device_setup(int dev, int* sm_count, const int** ctas_per_sm) {
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!g_device_ready[dev].load(std::memory_order_acquire)) {
        int* c = g_device_ctas[dev];
        cudaError_t e = setup_one<__nv_bfloat16, true>(c + 0);
        if (e == cudaSuccess) e = setup_one<__nv_bfloat16, false>(c + 1);
        if (e == cudaSuccess) e = setup_one<float, true>(c + 2);
        if (e == cudaSuccess) e = setup_one<float, false>(c + 3);
        int sms = 0;
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        g_device_sms[dev] = sms > 0 ? sms : 148;
        g_device_ready[dev].store(1, std::memory_order_release);
    }
    *sm_count = g_device_sms[dev];
    *ctas_per_sm = g_device_ctas[dev];
    return cudaSuccess;
}

template <typename T, bool NOISY>
void launch_stream(const UnmaskProblem& p, UnmaskPartial* partial, int tiles_per_item, int bulk_ok, int select_state,
                   int* status, int resident_ctas, cudaStream_t st) {
    const int rows = p.sets.row_off[p.sets.n_sets];
    const int tiles_per_row = (p.vocab + kTile - 1) / kTile;
    const long long items = static_cast<long long>(rows) * ((tiles_per_row + tiles_per_item - 1) / tiles_per_item);
    // persistent: as many CTAs as fit on the SMs, fewer when there is not an item for every warp
    const long long fit = resident_ctas;
    const long long need = (items + kWarps - 1) / kWarps;
    const unsigned grid = static_cast<unsigned>(need < fit ? (need < 1 ? 1 : need) : fit);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = stream_smem_bytes<T>();
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    const int n_attr = overlap_launch_attribute(st, attr);
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    cudaLaunchKernelEx(&cfg, unmask_stream_kernel<T, NOISY>, static_cast<const T*>(p.logits), static_cast<const uint8_t*>(p.state),
                       p.sets, partial, p.vocab, tiles_per_item, p.temperature, p.block_idx, p.step, bulk_ok, select_state,
                       static_cast<const uint32_t*>(p.step_counter), status);
}

// Both entry points launch the same two kernels; only the home of the records differs.
// mode 0: unmasking step; 1: draft of Scaffold Speculative Decoding (every MASKED row becomes DRAFT);
// 2: its accept scan (rows in state DRAFT are read, then the scan runs).
// tiles_per_item: how many 2048-id tiles share one record slot (a row has ceil(tiles / tiles_per_item) slots).
cudaError_t launch_unmask_kernels(const UnmaskProblem& p, UnmaskPartial* partial, int tiles_per_item, int dev,
                                  int* status, cudaStream_t st, int mode = 0) {
    const int select_state = mode == 2 ? FDD_DRAFT : FDD_MASKED;
    const int rows = p.sets.row_off[p.sets.n_sets];
    const int forks = p.sets.fork_off[p.sets.n_sets];
    if (rows > kMaxRows) return cudaErrorInvalidValue;
    int sm_count = 0;
    const int* per_sm = nullptr;
    cudaError_t e = device_setup(dev, &sm_count, &per_sm);
    if (e != cudaSuccess) return e;
    const int items_per_row = unmask_items_per_row(p.vocab, tiles_per_item);
    const bool noisy = p.temperature != 0.0f;
    // bulk copies need 16-byte aligned rows: base and row pitch
    if (p.logits_dtype == FDD_LOGITS_BF16) {
        const int bulk_ok = (p.vocab % 8 == 0) && (reinterpret_cast<uintptr_t>(p.logits) % 16 == 0);
        if (noisy) launch_stream<__nv_bfloat16, true>(p, partial, tiles_per_item, bulk_ok, select_state, status, sm_count * per_sm[0], st);
        else launch_stream<__nv_bfloat16, false>(p, partial, tiles_per_item, bulk_ok, select_state, status, sm_count * per_sm[1], st);
    } else {
        const int bulk_ok = (p.vocab % 4 == 0) && (reinterpret_cast<uintptr_t>(p.logits) % 16 == 0);
        if (noisy) launch_stream<float, true>(p, partial, tiles_per_item, bulk_ok, select_state, status, sm_count * per_sm[2], st);
        else launch_stream<float, false>(p, partial, tiles_per_item, bulk_ok, select_state, status, sm_count * per_sm[3], st);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (mode == 2)
        ss_accept_kernel<<<forks, 128, 0, st>>>(partial, p.tokens, p.state, p.n_committed, p.n_left, p.sets, items_per_row);
    else
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(forks);
        cfg.blockDim = dim3(kFinalizeThreads);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        cfg.numAttrs = overlap_launch_attribute(st, attr);
        cfg.attrs = attr;
        cudaLaunchKernelEx(&cfg, unmask_finalize_kernel, static_cast<const UnmaskPartial*>(partial), p.tokens, p.state,
                           p.n_committed, p.n_left, p.conf, p.sets, items_per_row, p.threshold,
                           mode == 1 ? static_cast<int>(FDD_DRAFT) : static_cast<int>(FDD_COMMITTED),
                           p.bump_counter ? p.step_counter : static_cast<uint32_t*>(nullptr), p.left_mirror, p.mirror_stamp);
    }
    return cudaGetLastError();
}

}  // namespace

size_t unmask_workspace_bytes(int vocab, int max_rows) {
    const int rows = max_rows < kMaxRows ? max_rows : kMaxRows;      // a launch takes at most kMaxRows rows
    return static_cast<size_t>(rows) * unmask_items_per_row(vocab, 1) * sizeof(UnmaskPartial);
}

cudaError_t launch_unmask(fdd_ctx* ctx, const UnmaskProblem& p, cudaStream_t st, int* n_launches, int mode) {
    *n_launches += 2;
    return launch_unmask_kernels(p, static_cast<UnmaskPartial*>(ctx->ws_unmask), 1, ctx->device, ctx->d_status, st, mode);
}

// -------------------------------------------------------------------------------------------------
// fdd_unmask_static: the same unmasking step for callers that must not allocate.
//
// Its scratch (the per (row, chunk) records) lives in a fixed device array that is part of the
// loaded library image, so the call needs no context, no fork set and no allocation of any kind.
// -------------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxRecords = FDD_UNMASK_STATIC_MAX_RECORDS;
constexpr int kStaticTilesPerItem = kUnmaskChunk / kUnmaskTile;    // one record slot per 8192 ids

// Held by every GPU that loads the library until the process exits (2 MiB).
static __device__ __align__(256) UnmaskPartial g_static_partials[kStaticMaxRecords];

// Device address of g_static_partials per device ordinal, resolved on first use.  In host code the
// array's name is only a handle for the runtime; the address a kernel can use must be asked for.
UnmaskPartial* g_static_ptr[kMaxDevices];
bool g_static_ready[kMaxDevices];

void put_error(char* err, size_t err_len, const char* text) {
    if (err && err_len) snprintf(err, err_len, "%s", text);
}

}  // namespace

extern "C" fdd_status fdd_unmask_static(const void* logits, int logits_dtype, int n_forks, int block_len,
                                        int vocab, int32_t* tokens, uint8_t* state, const uint64_t* seeds,
                                        float threshold, float temperature, uint32_t block_idx,
                                        uint32_t step, int32_t* n_committed, int32_t* n_left, float* conf,
                                        void* stream, char* err, size_t err_len) {
    CallRange range("fdd_unmask_static");
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
    const long long n_rows = static_cast<long long>(n_forks) * block_len;
    if (n_rows > kUnmaskMaxRows) {
        if (err && err_len)
            snprintf(err, err_len, "fdd_unmask_static: n_forks * block_len = %lld exceeds the %d rows one call takes",
                     n_rows, kUnmaskMaxRows);
        return FDD_ERR_CAPACITY;
    }
    const long long records = n_rows * unmask_items_per_row(vocab, kStaticTilesPerItem);
    if (records > kStaticMaxRecords) {
        if (err && err_len)
            snprintf(err, err_len,
                     "fdd_unmask_static: n_forks * block_len * ceil(vocab / %d) = %lld exceeds the fixed scratch of %d records",
                     kUnmaskChunk, records, kStaticMaxRecords);
        return FDD_ERR_CAPACITY;
    }
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
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
    UnmaskProblem p;
    p.logits = logits; p.tokens = tokens; p.state = state;
    p.n_committed = n_committed; p.n_left = n_left; p.conf = conf;
    p.sets.n_sets = 1;
    p.sets.row_off[0] = 0; p.sets.row_off[1] = n_forks * block_len;
    p.sets.fork_off[0] = 0; p.sets.fork_off[1] = n_forks;
    p.sets.d[0] = block_len; p.sets.seeds[0] = seeds;
    p.vocab = vocab; p.logits_dtype = logits_dtype;
    p.threshold = threshold; p.temperature = temperature; p.block_idx = block_idx; p.step = step;
    e = launch_unmask_kernels(p, g_static_ptr[dev], kStaticTilesPerItem, dev, nullptr, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        if (err && err_len) snprintf(err, err_len, "fdd_unmask_static: launch failed: %s", cudaGetErrorString(e));
        return FDD_ERR_CUDA;
    }
    return FDD_OK;
}
