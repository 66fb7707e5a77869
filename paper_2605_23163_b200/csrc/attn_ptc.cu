// Block-causal decode attention on the 5th-generation tensor cores (tcgen05 + TMEM + TMA),
// persistent version: one CTA per SM, balanced ranges of key-tile steps, many scenes per launch.
//
// Work unit: one (scene, KV head, pair of 128-row query tiles, rollout).  Query row r = i * G + g
// stacks block position i and the g-th query head of the GQA group, so 2 x 128 rows share every
// staged K/V tile.  Keys come in tiles of 128 from three segments: the shared prefix (contiguous
// or paged), the rollout's private suffix, the block itself.  A unit therefore is a run of
// "tile steps"; all units of all scenes of a call, laid end to end, form one global sequence of
// tile steps that is cut into equal contiguous ranges, one per CTA.  A CTA walks its range item
// by item (item = the part of one unit inside the range).  A unit that lies inside one range is
// written directly; a unit cut by a range border leaves normalised fp32 partials plus their
// log-sum-exp in scratch.  A unit in two pieces is merged at once by whichever CTA writes its piece
// second (a counter per unit, nobody waits).  A unit in more pieces is merged by all its piece
// holders together: once a CTA is through its range it waits until all pieces of the unit are
// written (the launch is cooperative, so the CTAs it waits for are running; the wait is bounded)
// and merges an equal share of the unit's rows into the bf16 output.
//
// Warp roles (384 threads): warps 0-3 and 4-7 are the two soft-max groups (thread = one query
// row = one TMEM lane), warp 8 lane 0 drives TMA, warps 9 and 10 issue the tcgen05.mma (one lane each:
// warp 9 the score products, warp 10 the output products), warp
// 11 only donates its registers.
// TMEM (512 columns): S | P0 | P1 | O0 | O1.  There is ONE fp32 score buffer S (128 columns) that the
// two query tiles use in turn: a soft-max group copies its scores into registers and hands the
// buffer back at once, so the next QK^T never waits for the exponentials.  The bf16 probabilities
// go to a buffer of their own (P0 / P1, 64 columns) and feed the PV product straight from TMEM.
// Per key tile and query tile:
//   S = Q K^T (smem x smem)  ->  soft-max warps: running max (rescaling O only when the max moved
//   by more than 2^8), P = exp2(S * c - m) -> TMEM  ->  O += P V (TMEM x smem, V keys-major).
// The MMA warp issues QK(1, j), PV(1, j - 1), QK(0, j + 1), PV(0, j) in that order, which keeps the
// tensor pipe fed while each soft-max group spends a whole period on one tile.
// Items follow one another without a meeting of the whole CTA: Q of the next item is staged as soon as
// the last score product of the current one has completed, its first scores are computed while
// the soft-max groups still write the current item's output, and each group moves on by itself.
// The exponentials can be split between the special-function unit (ex2.approx) and a cubic
// polynomial on the FMA pipe (one ex2 per score needs as many cycles as the MMAs).
// Every mbarrier wait is bounded; on a timeout the CTA records FDD_ERR_DEVICE_TIMEOUT, drains
// and returns (TMEM is always freed).
#include "fdd_internal.h"
#include "tc_ptx.cuh"
#include "tmap.h"

#include <math_constants.h>

#include <atomic>
#include <cstdlib>

namespace {

constexpr int kTcThreads = 384;
constexpr int kKeysPerTile = 128;
constexpr long long kWaitLimit = 4000000000LL;   // about two seconds of SM clocks
constexpr int kMaxGatedForks = kAttnMaxGatedForks;   // rollouts of one launch when any scene has a gate
constexpr int kMinTilesPerCta = 3;               // do not cut the work finer than this (every cut costs a piece to write and merge)
// Registers per thread after the hand-over.  The CTA starts with 384 x 168; 8 soft-max warps x
// kRegsSoftmax + 4 other warps x kRegsOther must not exceed that (2 * 208 + 88 = 3 * 168).
constexpr int kRegsSoftmax = 208;
constexpr int kRegsOther = 88;
static_assert(2 * kRegsSoftmax + kRegsOther <= 3 * 168, "register hand-over exceeds the CTA's pool");

struct SetParams {
    __nv_bfloat16* out;
    const int32_t* page_table;
    const int32_t* gate;       // per rollout, 0 = skip it; nullptr = every rollout takes part
    int fork_base;             // rollouts of the scenes before this one (index into the kernel's list)
    int units_per_fork;        // Hkv * row_pairs
    int n_forks, d, n_q_heads, G, R;
    int prefix_len, page_tokens, n_phys_pages, suffix_len;
    int tiles_prefix, tiles_suffix, tiles_total;
    int row_pairs;
    int causal;
};

template <int MAXSETS>
struct TcArgs {
    TcSetMaps maps[MAXSETS];
    SetParams sets[MAXSETS];
    float* part_o;             // [2 * ctas][D / 4][256] float4: normalised partial outputs, column-major per slot
    float* part_lse;           // [2 * ctas][256] log2-domain log-sum-exp of the partial
    int* unit_count;           // [2][max_units]: pieces written per unit, CTAs done with the unit's merge (self-resetting)
    int max_units;
    int* status;
    int min_tiles;             // do not cut the work into ranges shorter than this
    int n_sets;
    float scale_log2;
    long long merge_wait_limit; // SM clocks a CTA waits for the other pieces of a cut unit before it gives up
};

struct TileInfo {
    int segment;   // 0 prefix, 1 suffix, 2 block
    int index;     // tile index inside the segment
    int nvalid;    // valid keys in the tile (1..128)
};

__device__ __forceinline__ TileInfo tile_info(const SetParams& p, int g) {
    TileInfo t;
    if (g < p.tiles_prefix) {
        t.segment = 0; t.index = g;
        t.nvalid = min(kKeysPerTile, p.prefix_len - g * kKeysPerTile);
    } else if (g < p.tiles_prefix + p.tiles_suffix) {
        t.segment = 1; t.index = g - p.tiles_prefix;
        t.nvalid = min(kKeysPerTile, p.suffix_len - t.index * kKeysPerTile);
    } else {
        t.segment = 2; t.index = g - p.tiles_prefix - p.tiles_suffix;
        t.nvalid = min(kKeysPerTile, p.d - t.index * kKeysPerTile);
    }
    return t;
}

template <int D>
struct TcShape {
    static constexpr int kTileBytes = 128 * D * 2;      // one 128-row operand tile
    static constexpr int kChunks = D / 64;               // 64-element (128-byte) column chunks
    static constexpr int kChunkBytes = 128 * 128;        // 128 rows x 128 bytes
    static constexpr int kStages = D == 128 ? 2 : 4;     // K/V ring depth
    // Q (two tiles) + K ring + V ring + alignment slack; always more than half an SM's shared
    // memory, so two CTAs (each wanting all 512 TMEM columns) never share an SM.
    static constexpr int kSmemBytes = 2 * kTileBytes + 2 * kStages * kTileBytes + 1024;
};

// Issue the TMA loads of one 128-key tile of K or V into `dst` (layout [chunk][128 rows][128 B]).
template <int D>
__device__ __forceinline__ void load_kv_tile(const SetParams& p, const CUtensorMap* seg_map, const CUtensorMap* tail_map,
                                             const TileInfo& t, uint32_t dst, uint32_t bar, int h, int f,
                                             const int (&pages)[2]) {
    constexpr int kChunks = TcShape<D>::kChunks;
#pragma unroll
    for (int rh = 0; rh < 2; ++rh) {
        const int row0 = t.index * kKeysPerTile + rh * 64;
#pragma unroll
        for (int ch = 0; ch < kChunks; ++ch) {
            const uint32_t d_addr = dst + ch * TcShape<D>::kChunkBytes + rh * 8192;
            if (t.segment == 0) {
                if (p.page_tokens == 0) {
                    tc::tma_load_3d(d_addr, seg_map, bar, ch * 64, row0, h);
                } else {
                    // pages[rh]: physical page of this half tile, looked up by the caller ahead of time
                    // (n_phys_pages, one past the pool, for a half tile beyond the prefix: zeros)
                    const int lp = row0 / 64;
                    const int n_pages = (p.prefix_len + 63) / 64;
                    const bool tail = (lp == n_pages - 1) && (p.prefix_len % 64 != 0);
                    tc::tma_load_4d(d_addr, tail ? tail_map : seg_map, bar, ch * 64, 0, h, pages[rh]);
                }
            } else if (t.segment == 1) {
                tc::tma_load_4d(d_addr, seg_map, bar, ch * 64, row0, h, f);
            } else {
                tc::tma_load_4d(d_addr, seg_map, bar, ch * 64, h, row0, f);
            }
        }
    }
}

// One item of a CTA's range: tiles [t0, t1) of unit `unit` of scene `s`.
struct Item {
    int s, unit, t0, t1;
    long long unit_begin;      // global tile step of the unit's tile 0
};

// step_base[s]: first global tile step of scene s (scenes laid end to end, skipped rollouts left out)
template <int MAXSETS>
__device__ __forceinline__ Item locate(const TcArgs<MAXSETS>& a, const long long* step_base, long long pos, long long end) {
    Item it;
    int s = 0;
    while (s + 1 < a.n_sets && pos >= step_base[s + 1]) ++s;
    const SetParams& p = a.sets[s];
    const long long rel = pos - step_base[s];
    it.s = s;
    it.unit = static_cast<int>(rel / p.tiles_total);
    it.t0 = static_cast<int>(rel - static_cast<long long>(it.unit) * p.tiles_total);
    it.unit_begin = pos - it.t0;
    const long long left = end - pos;
    it.t1 = static_cast<int>(min(static_cast<long long>(p.tiles_total), it.t0 + left));
    return it;
}

// Cubic 2^f on [-0.5, 0.5] (relative error 7.5e-5, far below the bf16 rounding of P), with the
// factor 2^-112 of the range shift folded into the coefficients.
constexpr float kExpShift = 112.0f;
constexpr float kPolyScale = 1.92592994438723585e-34f;        // 2^-112
constexpr float kPoly0 = 0.9999281167984009f * kPolyScale;
constexpr float kPoly1 = 0.6932609677314758f * kPolyScale;
constexpr float kPoly2 = 0.2426108568906784f * kPolyScale;
constexpr float kPoly3 = 0.055171459913253784f * kPolyScale;
constexpr float kRoundMagic = 12582912.0f;                    // 1.5 * 2^23: adding it rounds to an integer

// Merge of a unit cut between CTAs:  out = sum_k w_k O_k / sum_k w_k,  w_k = 2^(lse_k - M), M = max_k lse_k.
// Every CTA that holds a piece merges an equal share of the unit's rows.  A thread takes CT float4
// columns of one row: 32 / CT pieces are read per round trip, 32 independent 16-byte reads (and the
// pieces' log-sum-exps) in flight.  M is not known in advance: the sums are kept relative to the
// largest log-sum-exp seen so far and rescaled when a chunk raises it, so the pieces are read once.
// Partials lie column-major in their slots ([D / 4][256 rows] float4).
template <int D, int CT>
__device__ __forceinline__ void merge_columns(const float* part_o, const float* part_lse, const int* slot_s, int n_pieces,
                                              int row, int col0, __nv_bfloat16* op) {
    constexpr int NC4 = D / 4;
    constexpr int PC = 32 / CT;                     // pieces per chunk
    const float4* po4 = reinterpret_cast<const float4*>(part_o);
    float4 acc[CT];
#pragma unroll
    for (int c = 0; c < CT; ++c) acc[c] = make_float4(0.f, 0.f, 0.f, 0.f);
    float M = -CUDART_INF_F, wsum = 0.0f;
    for (int k0 = 0; k0 < n_pieces; k0 += PC) {
        float ls[PC];
        float4 ov[PC][CT];
#pragma unroll
        for (int k = 0; k < PC; ++k) {
            const bool live = k0 + k < n_pieces;
            const size_t slot = slot_s[min(k0 + k, n_pieces - 1)];
            ls[k] = live ? __ldcg(part_lse + slot * 256 + row) : -CUDART_INF_F;
#pragma unroll
            for (int c = 0; c < CT; ++c)
                ov[k][c] = live ? __ldcg(po4 + (slot * NC4 + col0 + c) * 256 + row) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        float mc = ls[0];
#pragma unroll
        for (int k = 1; k < PC; ++k) mc = fmaxf(mc, ls[k]);
        const float mn = fmaxf(M, mc);
        if (!(mn > -CUDART_INF_F)) continue;                        // nothing but empty pieces so far
        const float back = exp2f(M - mn);                           // 0 the first time (M = -inf), 1 while M stands
        wsum *= back;
#pragma unroll
        for (int c = 0; c < CT; ++c) { acc[c].x *= back; acc[c].y *= back; acc[c].z *= back; acc[c].w *= back; }
        M = mn;
#pragma unroll
        for (int k = 0; k < PC; ++k) {
            const float wgt = exp2f(ls[k] - M);                     // 0 for a piece that is not there
            wsum += wgt;
#pragma unroll
            for (int c = 0; c < CT; ++c) {
                acc[c].x = fmaf(wgt, ov[k][c].x, acc[c].x); acc[c].y = fmaf(wgt, ov[k][c].y, acc[c].y);
                acc[c].z = fmaf(wgt, ov[k][c].z, acc[c].z); acc[c].w = fmaf(wgt, ov[k][c].w, acc[c].w);
            }
        }
    }
    const float iw = wsum > 0.0f ? 1.0f / wsum : 0.0f;
#pragma unroll
    for (int c = 0; c < CT; ++c) {
        const __nv_bfloat162 b0 = __floats2bfloat162_rn(acc[c].x * iw, acc[c].y * iw), b1 = __floats2bfloat162_rn(acc[c].z * iw, acc[c].w * iw);
        *reinterpret_cast<uint2*>(op + (col0 + c) * 4) =
            make_uint2(*reinterpret_cast<const uint32_t*>(&b0), *reinterpret_cast<const uint32_t*>(&b1));
    }
}

// A unit whose merge this CTA takes part in once its range is done.
struct Deferred {
    int s, unit, f, rp, h, c_first, n_pieces, gu;
    long long unit_begin;
};

template <int D, int MAXSETS, int EMU>
__global__ void __launch_bounds__(kTcThreads, 1)
attn_ptc_kernel(const __grid_constant__ TcArgs<MAXSETS> a) {
    using Shape = TcShape<D>;
    constexpr int kStages = Shape::kStages;
    static_assert(EMU % 8 == 0 && EMU >= 0 && EMU <= 128, "EMU: emulated exponentials per 128-key tile");
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t q_s = tc::smem_u32(smem);
    const uint32_t k_s = q_s + 2 * Shape::kTileBytes;
    const uint32_t v_s = k_s + kStages * Shape::kTileBytes;

    __shared__ __align__(8) unsigned long long bar_q_full, bar_k_full[kStages], bar_k_empty[kStages],
        bar_v_full[kStages], bar_v_empty[kStages], bar_s_full[2], bar_s_free[2], bar_p_full[2], bar_o_done[2], bar_o_final[2], bar_q_empty;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s, n_deferred_s, last_s;
    __shared__ Deferred deferred_s[2];                  // a range starts and ends inside at most one cut unit each
    constexpr int kMaxPieces = 160;                     // a unit is cut by CTA borders: at most one piece per CTA
    __shared__ int slot2_s[2][kMaxPieces];              // scratch slot of every piece of the (up to two) units being merged
    int* const slot_s = slot2_s[0];
    volatile int* abort_flag = &abort_s;

    // The rollouts that take part (gate != 0), scene after scene, and the layout of the work that
    // follows from them.  Every CTA derives the same lists from the same gate values.
    __shared__ unsigned short fork_s[kMaxGatedForks];
    __shared__ int n_act_s[MAXSETS], unit_base_s[MAXSETS];
    __shared__ long long step_base_s[MAXSETS + 1];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // A kernel launched behind this one for an early start (the unmasking step's streaming kernel)
    // may be made resident on SMs as their CTA of this launch exits; it waits for the whole of this
    // launch before it reads anything.
    tc::grid_launch_dependents();
    // (and this launch may itself have started early: the gate below is written by the kernel ahead of it)
    tc::grid_dependency_wait();

    for (int s = warp; s < a.n_sets; s += kTcThreads / 32) {
        const SetParams& p = a.sets[s];
        int cnt = p.n_forks;
        if (p.gate != nullptr) {
            cnt = 0;
            for (int j0 = 0; j0 < p.n_forks; j0 += 32) {
                const int j = j0 + lane;
                const bool on = j < p.n_forks && __ldcg(p.gate + j) != 0;
                const unsigned m = __ballot_sync(0xffffffffu, on);
                if (on) fork_s[p.fork_base + cnt + __popc(m & ((1u << lane) - 1u))] = static_cast<unsigned short>(j);
                cnt += __popc(m);
            }
        }
        if (lane == 0) n_act_s[s] = cnt;
    }
    __syncthreads();
    if (tid == 0) {
        long long steps = 0;
        int units = 0;
        for (int s = 0; s < a.n_sets; ++s) {
            step_base_s[s] = steps;
            unit_base_s[s] = units;
            const int u = a.sets[s].units_per_fork * n_act_s[s];
            steps += static_cast<long long>(u) * a.sets[s].tiles_total;
            units += u;
        }
        step_base_s[a.n_sets] = steps;
    }
    __syncthreads();
    const long long T = step_base_s[a.n_sets];
    const long long C = max(1LL, min(static_cast<long long>(gridDim.x), T / a.min_tiles));
    if (T == 0 || blockIdx.x >= C) return;          // nothing (left) to do: before any barrier or TMEM exists
    const long long range_begin = T * blockIdx.x / C;
    const long long range_end = T * (blockIdx.x + 1) / C;

    if (tid == 0) {
        abort_s = 0;
        n_deferred_s = 0;
        tc::mbar_init(tc::smem_u32(&bar_q_full), 1);
        tc::mbar_init(tc::smem_u32(&bar_q_empty), 1);      // every QK^T product of an item has completed: Q may be overwritten
        for (int s = 0; s < kStages; ++s) {
            tc::mbar_init(tc::smem_u32(&bar_k_full[s]), 1);
            tc::mbar_init(tc::smem_u32(&bar_k_empty[s]), 1);
            tc::mbar_init(tc::smem_u32(&bar_v_full[s]), 1);
            tc::mbar_init(tc::smem_u32(&bar_v_empty[s]), 1);
        }
        for (int q = 0; q < 2; ++q) {
            tc::mbar_init(tc::smem_u32(&bar_s_full[q]), 1);     // scores of query tile q are in S
            tc::mbar_init(tc::smem_u32(&bar_s_free[q]), 128);   // group q has copied them out of S
            tc::mbar_init(tc::smem_u32(&bar_p_full[q]), 128);   // group q has written P[q]
            tc::mbar_init(tc::smem_u32(&bar_o_done[q]), 1);     // a PV product of query tile q has completed
            tc::mbar_init(tc::smem_u32(&bar_o_final[q]), 1);    // the last PV product of query tile q in an item has completed
        }
        tc::fence_barrier_init();
    }
    if (warp == 9) {
        tc::tmem_alloc(tc::smem_u32(&tmem_base_s), 512);
        tc::tmem_relinquish();
    }
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem = tmem_base_s;
    const uint32_t tm_s = tmem;
    const uint32_t tm_p[2] = {tmem + 128, tmem + 192};
    const uint32_t tm_o[2] = {tmem + 256, tmem + 256 + D};

    // Each role runs its own copy of the item loop.  Nothing brings all of them together between two
    // items: the producer stages the next item's Q as soon as the last QK^T product of this one has
    // completed and its K/V tiles as ring stages come free, the first scores of the next item are
    // computed while the soft-max groups still read this item's output out of TMEM, and a group's
    // first P of the next item (written after its epilogue) is what lets the PV issuer overwrite O.
    struct ItemView {
        Item it;
        int f, rp, h, nt, rows_here, NQ;
    };
    auto view_item = [&](long long pos) {
        ItemView v;
        v.it = locate(a, step_base_s, pos, range_end);
        const SetParams& p = a.sets[v.it.s];
        int idx = v.it.unit;
        const int n_act = n_act_s[v.it.s];
        v.f = idx % n_act; idx /= n_act;
        if (p.gate != nullptr) v.f = fork_s[p.fork_base + v.f];
        v.rp = idx % p.row_pairs; idx /= p.row_pairs;
        v.h = idx;
        v.nt = v.it.t1 - v.it.t0;
        v.rows_here = min(256, p.R - v.rp * 256);
        v.NQ = v.rows_here > 128 ? 2 : 1;
        return v;
    };

    if (warp >= 8) {
        // The soft-max warps hold a 128-wide score row in registers; this warpgroup gives most of
        // its registers up for them.
        tc::reg_dealloc<kRegsOther>();
        if (warp == 8) {
            // ------------------------------------------------------------------ TMA producer
            uint32_t kv_cnt = 0;            // K/V tiles staged so far: ring stage and phase carry over between items
            uint32_t item_cnt = 0;
            bool ok = true;
            for (long long pos = range_begin; pos < range_end && ok;) {
                const ItemView v = view_item(pos);
                {
                    // warp-uniform loop, one elected lane issues the copies
                    const SetParams& p = a.sets[v.it.s];
                    const TcSetMaps& maps = a.maps[v.it.s];
                    const uint32_t bq = tc::smem_u32(&bar_q_full);
                    if (item_cnt > 0) {
                        // Q of the item before is still being read until its last QK^T product has completed
                        ok = tc::mbar_wait(tc::smem_u32(&bar_q_empty), (item_cnt - 1) & 1, abort_flag, kWaitLimit);
                        ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                    }
                    if (ok && tc::elect_one()) {
                        tc::prefetch_tmap(&maps.q);
                        tc::mbar_arrive_expect_tx(bq, v.NQ * Shape::kTileBytes);
                        for (int q = 0; q < v.NQ; ++q)
                            for (int ch = 0; ch < Shape::kChunks; ++ch)
                                tc::tma_load_4d(q_s + q * Shape::kTileBytes + ch * Shape::kChunkBytes, &maps.q, bq, ch * 64,
                                                v.h * p.G, (v.rp * 2 + q) * (128 / p.G), v.f);
                    }
                    __syncwarp();
                    for (int jl = 0; jl < v.nt && ok; ++jl) {
                        const TileInfo t = tile_info(p, v.it.t0 + jl);
                        const uint32_t n = kv_cnt + jl;
                        const int s = n % kStages;
                        const uint32_t ph = (n / kStages) & 1;
                        const CUtensorMap* mk = t.segment == 0 ? &maps.pk : (t.segment == 1 ? &maps.sk : &maps.bk);
                        const CUtensorMap* mv = t.segment == 0 ? &maps.pv : (t.segment == 1 ? &maps.sv : &maps.bv);
                        // the page table is read before the wait for a free stage, so that the lookup
                        // does not sit between a stage coming free and the copy into it
                        int pages[2] = {0, 0};
                        if (t.segment == 0 && p.page_tokens != 0) {
                            const int n_pages = (p.prefix_len + 63) / 64;
#pragma unroll
                            for (int rh = 0; rh < 2; ++rh) {
                                const int lp = t.index * 2 + rh;
                                pages[rh] = lp < n_pages ? __ldg(p.page_table + lp) : p.n_phys_pages;
                            }
                        }
                        ok = tc::mbar_wait(tc::smem_u32(&bar_k_empty[s]), ph ^ 1, abort_flag, kWaitLimit);
                        ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                        if (!ok) break;
                        if (tc::elect_one()) {
                            tc::mbar_arrive_expect_tx(tc::smem_u32(&bar_k_full[s]), Shape::kTileBytes);
                            load_kv_tile<D>(p, mk, &maps.pk_tail, t, k_s + s * Shape::kTileBytes, tc::smem_u32(&bar_k_full[s]), v.h, v.f, pages);
                        }
                        __syncwarp();
                        ok = tc::mbar_wait(tc::smem_u32(&bar_v_empty[s]), ph ^ 1, abort_flag, kWaitLimit);
                        ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                        if (!ok) break;
                        if (tc::elect_one()) {
                            tc::mbar_arrive_expect_tx(tc::smem_u32(&bar_v_full[s]), Shape::kTileBytes);
                            load_kv_tile<D>(p, mv, &maps.pv_tail, t, v_s + s * Shape::kTileBytes, tc::smem_u32(&bar_v_full[s]), v.h, v.f, pages);
                        }
                        __syncwarp();
                    }
                    if (!ok && lane == 0) {
                        if (*abort_flag == 0) atomicCAS(a.status, 0, FDD_ERR_DEVICE_TIMEOUT);
                        *abort_flag = 1;
                    }
                }
                __syncwarp();
                kv_cnt += v.nt;
                ++item_cnt;
                pos += v.nt;
            }
            if (*abort_flag != 0 && lane == 0) {
                const long long t0 = clock64();                  // let copies already in flight land
                while (clock64() - t0 < 2000000) {}
            }
            __syncwarp();
        } else if (warp == 9 || warp == 10) {
            // ------------------------------------------------------------------ MMA issuers
            // Warp 9 issues every QK^T, warp 10 every PV: while one of them checks the barriers of its
            // next product, the other one's MMAs keep the tensor pipe busy.  Nothing orders the two
            // streams against each other but the barriers (S handed back, P written).
            const bool qk_role = warp == 9;
            uint32_t kv_cnt = 0, item_cnt = 0;
            uint32_t sp_cnt[2] = {0, 0};    // key tiles handled so far per query tile
            // the soft-max group that read S last, and which of its tiles that was: S is not written
            // again before that group has copied its scores out, across items as well as inside one
            int s_prev_q = 0;
            uint32_t s_prev_idx = 0;
            bool s_has_prev = false;
            bool ok = true;
            for (long long pos = range_begin; pos < range_end && ok;) {
                const ItemView v = view_item(pos);
                const int nt = v.nt, NQ = v.NQ;
                {
                    // The whole warp runs this loop with warp-uniform values (so that descriptors and
                    // addresses can live in uniform registers); one elected lane issues the MMAs.
                    constexpr uint32_t kIdescQK = tc::idesc_bf16(128, 128, 0);
                    constexpr uint32_t kIdescPV = tc::idesc_bf16(128, D, 1);
                    // Descriptors are built once; inside the loops an operand address is one addition
                    // (the address field counts 16-byte units and never carries out of its 14 bits).
                    const uint64_t dq0 = tc::smem_desc_sw128(q_s, 0, 1024);
                    const uint64_t dk0 = tc::smem_desc_sw128(k_s, 0, 1024);
                    const uint64_t dv0 = tc::smem_desc_sw128(v_s, Shape::kChunkBytes, 1024);
                    // S = Q[q] . K^T
                    auto issue_qk = [&](int q, int s) {
                        const uint64_t dq = dq0 + static_cast<uint32_t>((q * Shape::kTileBytes) >> 4);
                        const uint64_t dk = dk0 + static_cast<uint32_t>((s * Shape::kTileBytes) >> 4);
#pragma unroll
                        for (int k = 0; k < D / 16; ++k) {
                            const uint32_t off = ((k >> 2) * Shape::kChunkBytes + (k & 3) * 32) >> 4;
                            if (k == 0) tc::mma_ss_first(tm_s, dq + off, dk + off, kIdescQK);
                            else tc::mma_ss_acc(tm_s, dq + off, dk + off, kIdescQK);
                        }
                    };
                    // O[q] (+)= P[q] . V
                    auto issue_pv = [&](int q, int s, bool accumulate) {
                        const uint64_t dv = dv0 + static_cast<uint32_t>((s * Shape::kTileBytes) >> 4);
                        if (accumulate) tc::mma_ts_acc(tm_o[q], tm_p[q], dv, kIdescPV);
                        else tc::mma_ts_first(tm_o[q], tm_p[q], dv, kIdescPV);
#pragma unroll
                        for (int j = 1; j < kKeysPerTile / 16; ++j)
                            tc::mma_ts_acc(tm_o[q], tm_p[q] + j * 8, dv + static_cast<uint32_t>((j * 2048) >> 4), kIdescPV);
                    };
                    auto stage_of = [&](int jl) { return static_cast<int>((kv_cnt + jl) % kStages); };
                    auto phase_of = [&](int jl) { return ((kv_cnt + jl) / kStages) & 1u; };
                    auto wait = [&](unsigned long long* bar, uint32_t parity) {
                        return tc::mbar_wait(tc::smem_u32(bar), parity & 1u, abort_flag, kWaitLimit);
                    };
                    // PV(q, jl): needs V tile jl and P[q] of that tile
                    auto do_pv = [&](int q, int jl, bool first_user_of_v, bool last_user_of_v) {
                        const int s = stage_of(jl);
                        bool good = true;
                        if (first_user_of_v) good = wait(&bar_v_full[s], phase_of(jl));
                        // (the first P of an item is written after the group has read the output of the
                        // item before out of TMEM: O[q] may be overwritten once that P is there)
                        good = good && wait(&bar_p_full[q], sp_cnt[q] + jl);
                        good = __shfl_sync(0xFFFFFFFFu, good ? 1 : 0, 0) != 0;
                        if (!good) return false;
                        tc::fence_after_sync();
                        if (tc::elect_one()) {
                            issue_pv(q, s, jl > 0);
                            tc::mma_commit(tc::smem_u32(&bar_o_done[q]));
                            if (last_user_of_v) tc::mma_commit(tc::smem_u32(&bar_v_empty[s]));
                            // the item's output for query tile q is complete (the products of one
                            // issuing thread complete in order)
                            if (jl == nt - 1) tc::mma_commit(tc::smem_u32(&bar_o_final[q]));
                        }
                        __syncwarp();
                        return true;
                    };
                    // QK(q, jl) into S: needs K tile jl and S handed back by its previous reader
                    auto do_qk = [&](int q, int jl, bool first_user_of_k, bool last_user_of_k) {
                        const int s = stage_of(jl);
                        bool good = true;
                        if (first_user_of_k) good = wait(&bar_k_full[s], phase_of(jl));
                        if (s_has_prev) good = good && wait(&bar_s_free[s_prev_q], s_prev_idx);
                        good = __shfl_sync(0xFFFFFFFFu, good ? 1 : 0, 0) != 0;
                        if (!good) return false;
                        tc::fence_after_sync();
                        if (tc::elect_one()) {
                            issue_qk(q, s);
                            tc::mma_commit(tc::smem_u32(&bar_s_full[q]));
                            if (last_user_of_k) tc::mma_commit(tc::smem_u32(&bar_k_empty[s]));
                            // the item's last score product: once it has completed nothing reads Q any more
                            if (jl == nt - 1 && q == NQ - 1) tc::mma_commit(tc::smem_u32(&bar_q_empty));
                        }
                        __syncwarp();
                        s_prev_q = q;
                        s_prev_idx = sp_cnt[q] + jl;
                        s_has_prev = true;
                        return true;
                    };
                    if (qk_role) {
                        // scores: QK(0,0) | QK(1,j) QK(0,j+1) | ...   (S is one buffer: each product waits
                        // until the group that owned the previous scores has copied them out)
                        ok = __shfl_sync(0xFFFFFFFFu, wait(&bar_q_full, item_cnt) ? 1 : 0, 0) != 0;
                        ok = ok && do_qk(0, 0, true, NQ == 1);
                        for (int jl = 0; jl < nt && ok; ++jl) {
                            if (NQ == 2) ok = do_qk(1, jl, false, true);
                            if (ok && jl + 1 < nt) ok = do_qk(0, jl + 1, true, NQ == 1);
                        }
                    } else {
                        // outputs: PV(1,j-1) PV(0,j) | ... | PV(1,nt-1), in the order the P tiles appear
                        for (int jl = 0; jl < nt && ok; ++jl) {
                            if (NQ == 2 && jl > 0) ok = do_pv(1, jl - 1, false, true);
                            if (ok) ok = do_pv(0, jl, true, NQ == 1);
                        }
                        if (ok && NQ == 2) ok = do_pv(1, nt - 1, false, true);
                    }
                    if (!ok && lane == 0) {
                        if (*abort_flag == 0) atomicCAS(a.status, 0, FDD_ERR_DEVICE_TIMEOUT);
                        *abort_flag = 1;
                    }
                }
                __syncwarp();
                kv_cnt += nt;
                for (int q = 0; q < NQ; ++q) sp_cnt[q] += nt;
                ++item_cnt;
                pos += nt;
            }
        }
        // (warp 11 has nothing to do but to have given up its registers)
    } else {
        tc::reg_alloc<kRegsSoftmax>();
        // ---------------------------------------------------------------------- soft-max groups
        const int q = warp >> 2;
        const int row_local = tid & 127;
        const uint32_t lane_base = (static_cast<uint32_t>(warp & 3) * 32u) << 16;
        const uint32_t bo = tc::smem_u32(&bar_o_done[q]);
        uint32_t sp0 = 0;                   // key tiles this group has handled so far
        uint32_t items_mine = 0;            // items this group has taken part in so far
        // After a wait has given up, the groups still walk the rest of the range (without computing):
        // both of them must meet at the same named barriers of the epilogues.
        for (long long pos = range_begin; pos < range_end;) {
            const ItemView v = view_item(pos);
            const Item& it = v.it;
            const SetParams& p = a.sets[it.s];
            const int f = v.f, rp = v.rp, h = v.h, nt = v.nt;
            const bool active = q < v.NQ;
            const int r = rp * 256 + q * 128 + row_local;       // row inside the unit
            const bool row_ok = r < p.R;
            const int qi = row_ok ? r / p.G : 0;
            const int qg = row_ok ? r - qi * p.G : 0;
            float m_used = -CUDART_INF_F, l = 0.0f;
            bool ok = *abort_flag == 0;
            if (active && ok) {
                const float c = a.scale_log2;
                const uint64_t c2 = tc::pack2(c, c);
                const float c_emu = c * (1.0f / 128.0f);
                const uint32_t bs = tc::smem_u32(&bar_s_full[q]), bf = tc::smem_u32(&bar_s_free[q]);
                const uint32_t bp = tc::smem_u32(&bar_p_full[q]);
                for (int jl = 0; jl < nt; ++jl) {
                    const TileInfo t = tile_info(p, it.t0 + jl);
                    ok = tc::mbar_wait(bs, (sp0 + jl) & 1, abort_flag, kWaitLimit);
                    if (!ok) break;
                    tc::fence_after_sync();
                    uint32_t sr[128];
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) tc::tmem_ld32(tm_s + lane_base + cc * 32, sr + cc * 32);
                    tc::wait_ld();
                    tc::fence_before_sync();
                    tc::mbar_arrive(bf);                                // S may be overwritten now
                    int limit = t.nvalid;                               // keys [0, limit) are visible
                    if (p.causal && t.segment == 2) limit = min(limit, qi - t.index * kKeysPerTile + 1);
                    if (limit < kKeysPerTile) {
#pragma unroll
                        for (int i = 0; i < 128; ++i)
                            if (i >= limit) sr[i] = 0xFF800000u;        // -inf
                    }
                    // the row's maximum: sixteen short chains, then a tree (the maximum sits on the path from
                    // the scores to the probabilities, so its depth counts, not its instruction count)
                    float mx[16];
#pragma unroll
                    for (int u = 0; u < 16; ++u) mx[u] = fmaxf(__uint_as_float(sr[2 * u]), __uint_as_float(sr[2 * u + 1]));
#pragma unroll
                    for (int i = 32; i < 128; i += 32) {
#pragma unroll
                        for (int u = 0; u < 16; ++u)
                            mx[u] = tc::max3(mx[u], __uint_as_float(sr[i + 2 * u]), __uint_as_float(sr[i + 2 * u + 1]));
                    }
#pragma unroll
                    for (int u = 0; u < 5; ++u) mx[u] = tc::max3(mx[3 * u], mx[3 * u + 1], mx[3 * u + 2]);   // 15 -> 5
                    const float tmax = fmaxf(tc::max3(mx[0], mx[1], mx[2]), tc::max3(mx[3], mx[4], mx[15]));
                    float m_tile = tmax * c;
                    if (!(m_tile > -CUDART_INF_F)) m_tile = m_used > -CUDART_INF_F ? m_used : 0.0f;
                    // The previous PV of this query tile must be complete before P is overwritten and
                    // before O is rescaled (it is one phase behind at most).  Usually only the first
                    // matters, so the wait sits after the exponentials.
                    bool pv_done = jl == 0;
                    if (jl == 0) {
                        m_used = m_tile;
                    } else {
                        const bool need = m_tile > m_used + 8.0f;
                        if (__any_sync(0xFFFFFFFFu, need)) {
                            ok = tc::mbar_wait(bo, (sp0 + jl - 1) & 1, abort_flag, kWaitLimit);
                            if (!ok) break;
                            pv_done = true;
                            tc::fence_after_sync();
                            const float alpha = need ? exp2f(m_used - m_tile) : 1.0f;
#pragma unroll
                            for (int cc = 0; cc < D / 32; ++cc) {
                                uint32_t o[32];
                                tc::tmem_ld32(tm_o[q] + lane_base + cc * 32, o);
                                tc::wait_ld();
#pragma unroll
                                for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                                tc::tmem_st32(tm_o[q] + lane_base + cc * 32, o);
                            }
                            tc::wait_st();
                            l *= alpha;
                            if (need) m_used = m_tile;
                        }
                    }
                    // P = 2^(S * c - m): the first 128 - EMU scores through ex2.approx, the rest
                    // through the polynomial; row sums in four packed accumulators.
                    uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
                    uint32_t packed[64];
                    const uint64_t nm2 = tc::pack2(-m_used, -m_used);
#pragma unroll
                    for (int i = 0; i < (128 - EMU) / 2; ++i) {
                        const uint64_t x2 = tc::fma2(tc::pack2(__uint_as_float(sr[2 * i]), __uint_as_float(sr[2 * i + 1])), c2, nm2);
                        float x0, x1;
                        tc::unpack2(x2, x0, x1);
                        const float e0 = tc::ex2(x0), e1 = tc::ex2(x1);
                        acc[i & 3] = tc::add2(acc[i & 3], tc::pack2(e0, e1));
                        const __nv_bfloat162 pk = __floats2bfloat162_rn(e0, e1);
                        packed[i] = *reinterpret_cast<const uint32_t*>(&pk);
                    }
                    if (EMU > 0) {
                        // y = (S * c - m + 112) / 128 clamped to [0, 1]; 2^(128 y - 112) = 2^n * 2^f with
                        // n = round(128 y), f = 128 y - n; 2^n enters through the exponent bits.
                        const float k_emu = (kExpShift - m_used) * (1.0f / 128.0f);
                        const uint64_t magic2 = tc::pack2(kRoundMagic, kRoundMagic);
                        const uint64_t m1_2 = tc::pack2(-1.0f, -1.0f);
                        const uint64_t s128_2 = tc::pack2(128.0f, 128.0f);
                        const uint64_t p0_2 = tc::pack2(kPoly0, kPoly0), p1_2 = tc::pack2(kPoly1, kPoly1);
                        const uint64_t p2_2 = tc::pack2(kPoly2, kPoly2), p3_2 = tc::pack2(kPoly3, kPoly3);
#pragma unroll
                        for (int i = (128 - EMU) / 2; i < 64; ++i) {
                            const float y0 = tc::fma_sat(__uint_as_float(sr[2 * i]), c_emu, k_emu);
                            const float y1 = tc::fma_sat(__uint_as_float(sr[2 * i + 1]), c_emu, k_emu);
                            const uint64_t y2 = tc::pack2(y0, y1);
                            const uint64_t t2 = tc::fma2(y2, s128_2, magic2);     // 128 y rounded to an integer (+ magic)
                            const uint64_t nn2 = tc::fma2(t2, m1_2, magic2);      // -n
                            const uint64_t f2 = tc::fma2(y2, s128_2, nn2);        // f in [-0.5, 0.5]
                            uint64_t pl = tc::fma2(f2, p3_2, p2_2);
                            pl = tc::fma2(pl, f2, p1_2);
                            pl = tc::fma2(pl, f2, p0_2);
                            float pa, pb, ta, tb;
                            tc::unpack2(pl, pa, pb);
                            tc::unpack2(t2, ta, tb);
                            const float e0 = __uint_as_float(__float_as_uint(pa) + (__float_as_uint(ta) << 23));
                            const float e1 = __uint_as_float(__float_as_uint(pb) + (__float_as_uint(tb) << 23));
                            acc[i & 3] = tc::add2(acc[i & 3], tc::pack2(e0, e1));
                            const __nv_bfloat162 pk = __floats2bfloat162_rn(e0, e1);
                            packed[i] = *reinterpret_cast<const uint32_t*>(&pk);
                        }
                    }
                    {
                        const uint64_t s01 = tc::add2(tc::add2(acc[0], acc[1]), tc::add2(acc[2], acc[3]));
                        float sa, sb;
                        tc::unpack2(s01, sa, sb);
                        l += sa + sb;
                    }
                    if (!pv_done) {
                        ok = tc::mbar_wait(bo, (sp0 + jl - 1) & 1, abort_flag, kWaitLimit);
                        if (!ok) break;
                        tc::fence_after_sync();
                    }
                    tc::tmem_st32(tm_p[q] + lane_base, packed);
                    tc::tmem_st32(tm_p[q] + lane_base + 32, packed + 32);
                    tc::wait_st();
                    tc::fence_before_sync();
                    tc::mbar_arrive(bp);
                }
                // the item's last PV product of this query tile (and with it every product before it)
                if (ok) ok = tc::mbar_wait(tc::smem_u32(&bar_o_final[q]), items_mine & 1, abort_flag, kWaitLimit);
                if (ok) tc::fence_after_sync();
            }

            // ---------------------------------------------------------------- epilogue
            const long long unit_end = it.unit_begin + p.tiles_total;
            const int c_first = static_cast<int>(((it.unit_begin + 1) * C + T - 1) / T) - 1;   // CTA of the unit's first step
            const int c_last = static_cast<int>((unit_end * C + T - 1) / T) - 1;                // CTA of its last step
            const int n_pieces = c_last - c_first + 1;
            const float inv = l > 0.0f ? 1.0f / l : 0.0f;
            if (n_pieces == 1) {
                if (active && ok) {
                    __nv_bfloat16* op = p.out + ((static_cast<size_t>(f) * p.d + qi) * p.n_q_heads + h * p.G + qg) * D;
#pragma unroll
                    for (int cc = 0; cc < D / 32; ++cc) {
                        uint32_t o[32];
                        tc::tmem_ld32(tm_o[q] + lane_base + cc * 32, o);
                        tc::wait_ld();
                        if (row_ok) {
                            // (a row is D * 2 bytes and starts on a multiple of that: 32-byte stores are aligned)
#pragma unroll
                            for (int v8 = 0; v8 < 2; ++v8) {
                                uint32_t w[8];
#pragma unroll
                                for (int x = 0; x < 8; ++x) {
                                    const __nv_bfloat162 pk = __floats2bfloat162_rn(__uint_as_float(o[v8 * 16 + 2 * x]) * inv,
                                                                                      __uint_as_float(o[v8 * 16 + 2 * x + 1]) * inv);
                                    w[x] = *reinterpret_cast<const uint32_t*>(&pk);
                                }
                                tc::st_global_32B(op + cc * 32 + v8 * 16, w);
                            }
                        }
                    }
                }
            } else {
                // A piece that starts at the CTA's range start uses the CTA's slot 0, a later one
                // (necessarily the CTA's last item) slot 1.
                const int own_slot = blockIdx.x * 2 + (pos == range_begin ? 0 : 1);
                // Two pieces, and the other one is there already (the usual case for a CTA's last item: its
                // neighbour wrote the unit's other piece as its first item, long ago): this piece does not
                // go through scratch at all, it is merged straight out of TMEM with the other one's partials.
                bool direct = false;
                if (n_pieces == 2) {
                    if (tid == 0) {
                        const int gu = unit_base_s[it.s] + it.unit;
                        const int there = *reinterpret_cast<volatile int*>(a.unit_count + gu) == 1;
                        if (there) a.unit_count[gu] = 0;         // (nobody else counts on this unit any more: ready for the next launch)
                        // the other piece was published before its count: one fence by the thread that read the
                        // count, ahead of the barrier behind which the others read the piece
                        if (there) __threadfence();
                        last_s = there;
                        slot_s[0] = c_first * 2 + (it.unit_begin <= T * c_first / C ? 0 : 1);
                        slot_s[1] = (c_first + 1) * 2;           // the second piece starts its CTA's range
                    }
                    tc::named_barrier(1, 256);
                    direct = last_s != 0;
                }
                if (direct) {
                    if (active && ok) {                          // (warp-uniform: the TMEM loads below are warp-wide)
                        const int other = slot_s[0] == own_slot ? slot_s[1] : slot_s[0];
                        // every read of the other piece goes out at once: the merge costs one round trip
                        const float4* po4 = reinterpret_cast<const float4*>(a.part_o) + static_cast<size_t>(other) * (D / 4) * 256 + tid;
                        float4 ov[D / 32][8];
#pragma unroll
                        for (int cc = 0; cc < D / 32; ++cc)
#pragma unroll
                            for (int v4 = 0; v4 < 8; ++v4)
                                ov[cc][v4] = row_ok ? __ldcg(po4 + (cc * 8 + v4) * 256) : make_float4(0.f, 0.f, 0.f, 0.f);
                        const float l_oth = row_ok ? __ldcg(a.part_lse + static_cast<size_t>(other) * 256 + tid) : -CUDART_INF_F;
                        const float l_own = m_used + log2f(l);
                        float M = fmaxf(l_own, l_oth);
                        if (!(M > -CUDART_INF_F)) M = 0.0f;
                        const float w_own = exp2f(l_own - M), w_oth = exp2f(l_oth - M);
                        const float wsum = w_own + w_oth;
                        const float iw = wsum > 0.0f ? 1.0f / wsum : 0.0f;
                        const float a_own = w_own * iw * inv, a_oth = w_oth * iw;     // (the other piece is stored normalised)
                        __nv_bfloat16* op = p.out + ((static_cast<size_t>(f) * p.d + qi) * p.n_q_heads + h * p.G + qg) * D;
#pragma unroll
                        for (int cc = 0; cc < D / 32; ++cc) {
                            uint32_t o[32];
                            tc::tmem_ld32(tm_o[q] + lane_base + cc * 32, o);
                            tc::wait_ld();
                            if (row_ok) {
#pragma unroll
                                for (int v8 = 0; v8 < 2; ++v8) {
                                    uint32_t wv[8];
#pragma unroll
                                    for (int x = 0; x < 8; ++x) {
                                        const int e0 = v8 * 16 + 2 * x;      // element inside the 32 columns
                                        const float4& src = ov[cc][e0 / 4];
                                        const float s0 = (e0 % 4 == 0) ? src.x : src.z, s1 = (e0 % 4 == 0) ? src.y : src.w;
                                        const __nv_bfloat162 pk = __floats2bfloat162_rn(fmaf(a_own, __uint_as_float(o[e0]), a_oth * s0),
                                                                                          fmaf(a_own, __uint_as_float(o[e0 + 1]), a_oth * s1));
                                        wv[x] = *reinterpret_cast<const uint32_t*>(&pk);
                                    }
                                    tc::st_global_32B(op + cc * 32 + v8 * 16, wv);
                                }
                            }
                        }
                    }
                    tc::named_barrier(1, 256);                   // slot_s is free again
                } else {
                if (active && ok) {
                    // column-major inside the slot ([D / 4 float4 columns][256 rows]): the 32 rows of a
                    // warp make one contiguous 512-byte store, and the merge reads them back the same way
                    float4* po = reinterpret_cast<float4*>(a.part_o) + static_cast<size_t>(own_slot) * (D / 4) * 256 + q * 128 + row_local;
#pragma unroll
                    for (int cc = 0; cc < D / 32; ++cc) {
                        uint32_t o[32];
                        tc::tmem_ld32(tm_o[q] + lane_base + cc * 32, o);
                        tc::wait_ld();
#pragma unroll
                        for (int v4 = 0; v4 < 8; ++v4)
                            __stcg(po + (cc * 8 + v4) * 256,
                                   make_float4(__uint_as_float(o[v4 * 4]) * inv, __uint_as_float(o[v4 * 4 + 1]) * inv,
                                               __uint_as_float(o[v4 * 4 + 2]) * inv, __uint_as_float(o[v4 * 4 + 3]) * inv));
                    }
                    __stcg(a.part_lse + static_cast<size_t>(own_slot) * 256 + q * 128 + row_local, m_used + log2f(l));
                }
                // Publishing the piece: every thread's stores are ordered before the barrier, the one thread
                // that counts the piece fences between the barrier and the count (and again after it, on
                // behalf of the threads that read the other pieces behind the next barrier).
                tc::named_barrier(1, 256);
                if (n_pieces == 2) {
                    // Two pieces: whichever of the two CTAs writes its piece second merges the unit
                    // at once; nobody waits.
                    if (tid == 0) {
                        const int gu = unit_base_s[it.s] + it.unit;
                        __threadfence();
                        const int last = atomicAdd(a.unit_count + gu, 1) == 1;
                        if (last) {
                            a.unit_count[gu] = 0;                // both pieces are there: ready for the next launch
                            __threadfence();
                        }
                        last_s = last;
                        slot_s[0] = c_first * 2 + (it.unit_begin <= T * c_first / C ? 0 : 1);
                        slot_s[1] = (c_first + 1) * 2;           // the second piece starts its CTA's range
                    }
                    tc::named_barrier(1, 256);
                    if (last_s) {
                        if (row_ok) {                            // thread = row
                            __nv_bfloat16* op = p.out + ((static_cast<size_t>(f) * p.d + qi) * p.n_q_heads + h * p.G + qg) * D;
#pragma unroll
                            for (int col0 = 0; col0 < D / 4; col0 += 16)
                                merge_columns<D, 16>(a.part_o, a.part_lse, slot_s, 2, tid, col0, op);
                        }
                    }
                    tc::named_barrier(1, 256);                   // slot_s is free again
                } else if (tid == 0) {
                    // More pieces: count this one, and note the unit for this CTA's share of its merge,
                    // which follows once the whole range is done (waiting here, in the middle of the
                    // range, would chain every CTA behind its neighbour).
                    const int gu = unit_base_s[it.s] + it.unit;
                    __threadfence();
                    atomicAdd(a.unit_count + gu, 1);
                    Deferred& dfr = deferred_s[n_deferred_s++];
                    dfr.s = it.s; dfr.unit = it.unit; dfr.f = f; dfr.rp = rp; dfr.h = h;
                    dfr.c_first = c_first; dfr.n_pieces = n_pieces; dfr.gu = gu;
                    dfr.unit_begin = it.unit_begin;
                }
                }   // not direct
            }
            if (!ok) {
                if (*abort_flag == 0) atomicCAS(a.status, 0, FDD_ERR_DEVICE_TIMEOUT);
                *abort_flag = 1;
            }
            if (active) {
                sp0 += nt;
                ++items_mine;
            }
            pos += nt;
        }

        // ------------------------------------------------------------ merges of the cut units
        // Every CTA that holds a piece of a unit (in more than two pieces) merges an equal share of
        // the unit's rows, once all pieces are there.  (All CTAs of the launch are resident at once:
        // the wait is for CTAs that are running, and it is bounded like every other wait.)  A CTA
        // with two such units gives half of its threads to each.
        tc::named_barrier(1, 256);
        const int n_deferred = *abort_flag ? 0 : n_deferred_s;
        if (n_deferred > 0) {
            if (tid == 0) {
                const long long t0 = clock64();
                for (int e = 0; e < n_deferred; ++e) {
                    volatile int* arrived = a.unit_count + deferred_s[e].gu;
                    while (*arrived < deferred_s[e].n_pieces) {
                        if (clock64() - t0 > a.merge_wait_limit) {
                            atomicCAS(a.status, 0, FDD_ERR_DEVICE_TIMEOUT);
                            *abort_flag = 1;
                            break;
                        }
                    }
                }
                __threadfence();                                      // the pieces were published before their counts
            }
            for (int e = 0; e < n_deferred; ++e)
                if (tid < deferred_s[e].n_pieces && tid < kMaxPieces) {
                    const int pc = deferred_s[e].c_first + tid;
                    slot2_s[e][tid] = pc * 2 + (deferred_s[e].unit_begin <= T * pc / C ? 0 : 1);
                }
            tc::named_barrier(1, 256);
            if (*abort_flag == 0) {
                const int threads_e = 256 / n_deferred;               // threads per unit
                const int e = tid / threads_e, lt = tid - e * threads_e;
                const Deferred dfr = deferred_s[e];
                const SetParams& p = a.sets[dfr.s];
                const int n_pieces = dfr.n_pieces;
                const int* slots = slot2_s[e];
                // this CTA's share of the rows; a row is split between `col_groups` threads
                const int rows_here = min(256, p.R - dfr.rp * 256);
                const int mine = static_cast<int>(blockIdx.x) - dfr.c_first;
                const int row_lo = rows_here * mine / n_pieces, row_hi = rows_here * (mine + 1) / n_pieces;
                const int share = row_hi - row_lo;                    // <= 86 (three pieces or more)
                int col_groups = 1;                                   // a power of two, share * col_groups <= threads_e
                while (col_groups < D / 4 && share * col_groups * 2 <= threads_e) col_groups *= 2;
                const int ct = (D / 4) / col_groups;                  // float4 columns per thread
                const int row_in_share = lt / col_groups, cg = lt - row_in_share * col_groups;
                if (share > 0 && row_in_share < share) {
                    const int rowu = row_lo + row_in_share;
                    const int r = dfr.rp * 256 + rowu;
                    const int qi2 = r / p.G, qg2 = r - qi2 * p.G;
                    __nv_bfloat16* op = p.out + ((static_cast<size_t>(dfr.f) * p.d + qi2) * p.n_q_heads + dfr.h * p.G + qg2) * D;
                    const int col0 = cg * ct;
                    switch (ct) {
                        case 1: merge_columns<D, 1>(a.part_o, a.part_lse, slots, n_pieces, rowu, col0, op); break;
                        case 2: merge_columns<D, 2>(a.part_o, a.part_lse, slots, n_pieces, rowu, col0, op); break;
                        case 4: merge_columns<D, 4>(a.part_o, a.part_lse, slots, n_pieces, rowu, col0, op); break;
                        case 8: merge_columns<D, 8>(a.part_o, a.part_lse, slots, n_pieces, rowu, col0, op); break;
                        case 16: merge_columns<D, 16>(a.part_o, a.part_lse, slots, n_pieces, rowu, col0, op); break;
                        default: merge_columns<D, 32>(a.part_o, a.part_lse, slots, n_pieces, rowu, col0, op); break;
                    }
                }
                tc::named_barrier(1, 256);
                if (tid < n_deferred) {
                    // the last CTA to finish its share leaves both counters at zero for the next launch
                    const Deferred& d2 = deferred_s[tid];
                    int* done = a.unit_count + a.max_units + d2.gu;
                    if (atomicAdd(done, 1) == d2.n_pieces - 1) {
                        *done = 0;
                        a.unit_count[d2.gu] = 0;
                    }
                }
            }
        }
    }

    tc::fence_before_sync();
    __syncthreads();
    if (warp == 9) tc::tmem_dealloc(tmem, 512);
}

bool make_call_maps(const AttnProblem& a, int D, TcSetMaps* m) {
    const uint64_t eb = 2;
    const int G = a.n_q_heads / a.n_kv_heads;
    {
        uint64_t dims[4] = {(uint64_t)D, (uint64_t)a.n_q_heads, (uint64_t)a.d, (uint64_t)a.n_forks};
        uint64_t str[3] = {D * eb, a.n_q_heads * D * eb, (uint64_t)a.d * a.n_q_heads * D * eb};
        uint32_t box[4] = {64, (uint32_t)G, (uint32_t)(128 / G), 1};
        if (!tmap::encode_bf16(&m->q, a.q, 4, dims, str, box)) return false;
    }
    {
        uint64_t dims[4] = {(uint64_t)D, (uint64_t)a.n_kv_heads, (uint64_t)a.d, (uint64_t)a.n_forks};
        uint64_t str[3] = {D * eb, a.n_kv_heads * D * eb, (uint64_t)a.d * a.n_kv_heads * D * eb};
        uint32_t box[4] = {64, 1, 64, 1};
        if (!tmap::encode_bf16(&m->bk, a.k_blk, 4, dims, str, box)) return false;
        if (!tmap::encode_bf16(&m->bv, a.v_blk, 4, dims, str, box)) return false;
    }
    return true;
}

bool make_cache_maps(const AttnProblem& a, int D, TcSetMaps* m) {
    const uint64_t eb = 2;
    if (a.suffix_len > 0) {
        uint64_t dims[4] = {(uint64_t)D, (uint64_t)a.suffix_len, (uint64_t)a.n_kv_heads, (uint64_t)a.n_forks};
        uint64_t str[3] = {D * eb, (uint64_t)a.suffix_capacity * D * eb, (uint64_t)a.n_kv_heads * a.suffix_capacity * D * eb};
        uint32_t box[4] = {64, 64, 1, 1};
        if (!tmap::encode_bf16(&m->sk, a.suffix_k, 4, dims, str, box)) return false;
        if (!tmap::encode_bf16(&m->sv, a.suffix_v, 4, dims, str, box)) return false;
    } else {
        m->sk = m->bk; m->sv = m->bv;    // never used (no suffix tiles)
    }
    m->pk_tail = m->bk; m->pv_tail = m->bv;
    if (a.prefix_len > 0) {
        if (a.page_tokens == 0) {
            uint64_t dims[3] = {(uint64_t)D, (uint64_t)a.prefix_len, (uint64_t)a.n_kv_heads};
            uint64_t str[2] = {D * eb, (uint64_t)a.prefix_capacity * D * eb};
            uint32_t box[3] = {64, 64, 1};
            if (!tmap::encode_bf16(&m->pk, a.prefix_k, 3, dims, str, box)) return false;
            if (!tmap::encode_bf16(&m->pv, a.prefix_v, 3, dims, str, box)) return false;
        } else {
            uint64_t dims[4] = {(uint64_t)D, (uint64_t)a.page_tokens, (uint64_t)a.n_kv_heads, (uint64_t)a.prefix_capacity};
            uint64_t str[3] = {D * eb, (uint64_t)a.page_tokens * D * eb, (uint64_t)a.n_kv_heads * a.page_tokens * D * eb};
            uint32_t box[4] = {64, 64, 1, 1};
            if (!tmap::encode_bf16(&m->pk, a.prefix_k, 4, dims, str, box)) return false;
            if (!tmap::encode_bf16(&m->pv, a.prefix_v, 4, dims, str, box)) return false;
            const int tail = a.prefix_len % a.page_tokens;
            if (tail) {
                dims[1] = tail;
                if (!tmap::encode_bf16(&m->pk_tail, a.prefix_k, 4, dims, str, box)) return false;
                if (!tmap::encode_bf16(&m->pv_tail, a.prefix_v, 4, dims, str, box)) return false;
            }
        }
    } else {
        m->pk = m->bk; m->pv = m->bv;    // never used (no prefix tiles)
    }
    return true;
}

// Tensor maps of one scene, reusing the cached ones while the pointers and lengths they were
// built from have not changed (the usual case: one set of buffers, many denoising steps).
const TcSetMaps* maps_for(const AttnProblem& a, int D, TcMapCache* cache) {
    const bool call_same = cache->valid && cache->q == a.q && cache->k_blk == a.k_blk && cache->v_blk == a.v_blk &&
                           cache->d == a.d;
    const bool cache_same = cache->valid && cache->suffix_len == a.suffix_len && cache->prefix_len == a.prefix_len;
    if (call_same && cache_same) return &cache->maps;
    if (!call_same) {
        if (!make_call_maps(a, D, &cache->maps)) { cache->valid = false; return nullptr; }
    }
    // the never-used entries of the cache part alias the call part, so it is rebuilt either way
    if (!make_cache_maps(a, D, &cache->maps)) { cache->valid = false; return nullptr; }
    cache->q = a.q; cache->k_blk = a.k_blk; cache->v_blk = a.v_blk; cache->d = a.d;
    cache->suffix_len = a.suffix_len;
    cache->prefix_len = a.prefix_len;
    cache->valid = true;
    return &cache->maps;
}

int emulated_exponentials() {
    // How many of the 128 exponentials of a key tile go through the polynomial.  FDD_ATTN_EMU
    // (0, 16 or 32) overrides the default; every choice computes the same thing.
    static int value = -1;
    if (value < 0) {
        value = 0;
        if (const char* e = std::getenv("FDD_ATTN_EMU")) {
            const int v = std::atoi(e);
            if (v == 0 || v == 16 || v == 32) value = v;
        }
    }
    return value;
}

template <int D, int MAXSETS, int EMU>
cudaError_t launch_one(const TcArgs<MAXSETS>& args, unsigned ctas, int device, cudaStream_t st) {
    const int smem = TcShape<D>::kSmemBytes;
    // the kernel's shared-memory size is a per-device attribute: set on the first launch on each device
    constexpr int kMaxDevices = 64;
    static std::atomic<bool> configured[kMaxDevices];
    if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!configured[device].load(std::memory_order_acquire)) {
        cudaError_t e = cudaFuncSetAttribute(attn_ptc_kernel<D, MAXSETS, EMU>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        configured[device].store(true, std::memory_order_release);
    }
    // The CTAs wait for one another's pieces at the end: a cooperative launch makes the runtime
    // guarantee that all of them are resident at once (or fail the launch).  The launch also asks for
    // an early start behind the kernel ahead of it on the stream (the kernel waits before it reads
    // anything); a runtime that does not take the two attributes together gets the first one alone.
    void* params[] = {const_cast<TcArgs<MAXSETS>*>(&args)};
    static std::atomic<int> early_start_refused[kMaxDevices];
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas);
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = static_cast<size_t>(smem);
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    const bool capturing = cudaStreamIsCapturing(st, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone;
    const void* fn = reinterpret_cast<const void*>(&attn_ptc_kernel<D, MAXSETS, EMU>);
    if (!capturing && !early_start_refused[device].load(std::memory_order_relaxed)) {
        cfg.numAttrs = 2;
        const cudaError_t e = cudaLaunchKernelExC(&cfg, fn, params);
        if (e == cudaSuccess) return e;
        (void)cudaGetLastError();                         // a refused configuration launches nothing and leaves no sticky error
        early_start_refused[device].store(1, std::memory_order_relaxed);
    }
    cfg.numAttrs = 1;
    return cudaLaunchKernelExC(&cfg, fn, params);
}

template <int MAXSETS>
cudaError_t launch_emu(const TcArgs<MAXSETS>& args, int head_dim, unsigned ctas, int device, cudaStream_t st) {
    if (head_dim == 64) return launch_one<64, MAXSETS, 0>(args, ctas, device, st);
    switch (emulated_exponentials()) {
        case 16: return launch_one<128, MAXSETS, 16>(args, ctas, device, st);
        case 32: return launch_one<128, MAXSETS, 32>(args, ctas, device, st);
        default: return launch_one<128, MAXSETS, 0>(args, ctas, device, st);
    }
}

template <int MAXSETS>
cudaError_t launch_group(fdd_ctx* ctx, const AttnProblem* probs, TcMapCache* const* caches, int n, int head_dim,
                         cudaStream_t st) {
    // 1-20 KB, kept off the stack in the context's own buffer (a context is used by one host thread at a time)
    if (ctx->attn_args.size() * sizeof(uint64_t) < sizeof(TcArgs<MAXSETS>)) ctx->attn_args.resize((sizeof(TcArgs<MAXSETS>) + 7) / 8);
    TcArgs<MAXSETS>& args = *reinterpret_cast<TcArgs<MAXSETS>*>(ctx->attn_args.data());
    long long steps = 0;
    int units = 0, forks = 0;
    bool gated = false;
    for (int s = 0; s < n; ++s) {
        const AttnProblem& a = probs[s];
        const TcSetMaps* m = maps_for(a, head_dim, caches[s]);
        if (!m) return cudaErrorInvalidValue;
        args.maps[s] = *m;
        SetParams& p = args.sets[s];
        p.out = a.out;
        p.page_table = a.page_table;
        p.n_forks = a.n_forks; p.d = a.d; p.n_q_heads = a.n_q_heads;
        p.G = a.n_q_heads / a.n_kv_heads;
        p.R = a.d * p.G;
        p.prefix_len = a.prefix_len; p.page_tokens = a.page_tokens; p.n_phys_pages = a.prefix_capacity;
        p.suffix_len = a.suffix_len;
        p.tiles_prefix = (a.prefix_len + kKeysPerTile - 1) / kKeysPerTile;
        p.tiles_suffix = (a.suffix_len + kKeysPerTile - 1) / kKeysPerTile;
        p.tiles_total = p.tiles_prefix + p.tiles_suffix + (a.d + kKeysPerTile - 1) / kKeysPerTile;
        p.row_pairs = (p.R + 255) / 256;
        p.units_per_fork = a.n_kv_heads * p.row_pairs;
        p.causal = a.causal_in_block;
        p.gate = a.gate;
        p.fork_base = forks;
        gated = gated || a.gate != nullptr;
        forks += a.n_forks;
        steps += static_cast<long long>(p.units_per_fork) * a.n_forks * p.tiles_total;
        units += p.units_per_fork * a.n_forks;
    }
    if (units > ctx->attn_max_units) return cudaErrorInvalidValue;
    if (gated && forks > kMaxGatedForks) return cudaErrorInvalidValue;
    static int min_tiles = 0;
    if (min_tiles == 0) {
        min_tiles = kMinTilesPerCta;
        if (const char* e = std::getenv("FDD_ATTN_MIN_TILES")) { const int v = std::atoi(e); if (v >= 1 && v <= 64) min_tiles = v; }
    }
    long long ctas = steps / min_tiles;
    if (ctas > ctx->attn_max_ctas) ctas = ctx->attn_max_ctas;
    if (ctas < 1) ctas = 1;
    args.part_o = static_cast<float*>(ctx->ws_attn);
    args.part_lse = args.part_o + static_cast<size_t>(2) * ctx->attn_max_ctas * 256 * head_dim;
    args.unit_count = ctx->attn_unit_count;
    args.max_units = ctx->attn_max_units;
    args.status = ctx->d_status;
    args.min_tiles = min_tiles;
    args.n_sets = n;
    args.scale_log2 = probs[0].scale * 1.4426950408889634f;
    args.merge_wait_limit = ctx->attn_merge_wait_limit;
    return launch_emu<MAXSETS>(args, head_dim, static_cast<unsigned>(ctas), ctx->device, st);
}

}  // namespace

// Whether the tensor-core kernel covers this problem.
bool attention_tc_supported(const AttnProblem& a, int head_dim) {
    const int G = a.n_q_heads / a.n_kv_heads;
    if (head_dim != 64 && head_dim != 128) return false;
    if (G < 1 || G > 16 || (G & (G - 1)) != 0) return false;
    if (a.page_tokens != 0 && a.page_tokens != 64) return false;
    return tmap::encode_fn() != nullptr;
}

// Scratch of the split-unit merge: two partial slots per CTA, each D / 4 float4 columns of 256 rows
// plus the rows' log-sum-exps.
size_t attention_ptc_workspace_bytes(int head_dim, int max_ctas) {
    return static_cast<size_t>(2) * max_ctas * 256 * (head_dim + 1) * sizeof(float);
}

// One launch for up to kTcMaxSets scenes (all with the same soft-max scale).
cudaError_t launch_attention_ptc(fdd_ctx* ctx, const AttnProblem* probs, TcMapCache* const* caches, int n,
                                 int head_dim, cudaStream_t st, int* n_launches) {
    if (n < 1 || n > kTcMaxSets) return cudaErrorInvalidValue;
    *n_launches += 1;
    if (n == 1) return launch_group<1>(ctx, probs, caches, n, head_dim, st);
    return launch_group<kTcMaxSets>(ctx, probs, caches, n, head_dim, st);
}
