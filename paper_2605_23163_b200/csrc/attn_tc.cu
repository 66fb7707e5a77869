// Block-causal decode attention on the 5th-generation tensor cores (tcgen05 + TMEM + TMA).
//
// Work unit: one (KV head, rollout, pair of 128-row query tiles) and a contiguous range of key
// tiles.  Query row r = i * G + g stacks block position i and the g-th query head of the GQA
// group, so 128 * 2 rows share every staged K/V tile.  Keys come in tiles of 128 from three
// segments: the shared prefix (contiguous or paged), the rollout's private suffix, the block.
//
// Warp roles (320 threads): warps 0-3 and 4-7 are the two soft-max groups (thread = one query
// row = one TMEM lane), warp 8 lane 0 drives TMA, warp 9 lane 0 issues every tcgen05.mma.
// TMEM (512 columns): S0 | S1 | O0 | O1; the bf16 probabilities P overwrite the first half of
// their S tile and feed the PV product straight from TMEM.  Per key tile and query tile:
//   S = Q K^T (smem x smem)  ->  soft-max warps: running max (rescaling O only when the max moved
//   by more than 2^8), P = exp2(S * c - m) -> TMEM  ->  O += P V (TMEM x smem, V keys-major).
// The two query tiles ping-pong, so one tile's soft-max overlaps the other tile's MMAs.
// Every mbarrier wait is bounded; on a timeout the CTA records FDD_ERR_DEVICE_TIMEOUT, drains
// and returns (TMEM is always freed).
#include "fdd_internal.h"
#include "tc_ptx.cuh"
#include "tmap.h"

#include <math_constants.h>

namespace {

constexpr int kTcThreads = 320;
constexpr int kKeysPerTile = 128;
constexpr int kStages = 2;
constexpr long long kWaitLimit = 4000000000LL;   // about two seconds of SM clocks

struct TcMaps {
    CUtensorMap q;                  // (D, Hq, d, N)
    CUtensorMap pk, pv;             // contiguous: (D, P, Hkv); paged: (D, 64, Hkv, pages)
    CUtensorMap pk_tail, pv_tail;   // paged only: token dimension cut to the last page's fill
    CUtensorMap sk, sv;             // (D, S, Hkv, N)
    CUtensorMap bk, bv;             // (D, Hkv, d, N)
};

struct TcParams {
    __nv_bfloat16* out;
    float* part_o;          // [cta][256][D] normalised partial outputs (split-KV only)
    float* part_lse;        // [cta][256] log2-domain log-sum-exp of the partial
    const int32_t* page_table;
    int* status;
    int n_forks, d, n_q_heads, n_kv_heads, G, R;
    int prefix_len, page_tokens, n_phys_pages, suffix_len;
    int tiles_prefix, tiles_suffix, tiles_block;
    int row_pairs, n_splits;
    int causal;
    float scale_log2;
};

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct TileInfo {
    int segment;   // 0 prefix, 1 suffix, 2 block
    int index;     // tile index inside the segment
    int nvalid;    // valid keys in the tile (1..128)
};

__device__ __forceinline__ TileInfo tile_info(const TcParams& p, int g) {
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
    static constexpr int kSmemBytes = 2 * kTileBytes + 2 * kStages * kTileBytes + 1024;
};

// Issue the TMA loads of one 128-key tile of K or V into `dst` (layout [chunk][128 rows][128 B]).
template <int D>
__device__ __forceinline__ void load_kv_tile(const TcParams& p, const CUtensorMap* seg_map, const CUtensorMap* tail_map,
                                             const TileInfo& t, uint32_t dst, uint32_t bar, int h, int f) {
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
                    const int lp = row0 / 64;
                    const int n_pages = (p.prefix_len + 63) / 64;
                    if (lp < n_pages) {
                        const int page = p.page_table[lp];
                        const bool tail = (lp == n_pages - 1) && (p.prefix_len % 64 != 0);
                        tc::tma_load_4d(d_addr, tail ? tail_map : seg_map, bar, ch * 64, 0, h, page);
                    } else {
                        tc::tma_load_4d(d_addr, seg_map, bar, ch * 64, 0, h, p.n_phys_pages);   // past the end: zeros
                    }
                }
            } else if (t.segment == 1) {
                tc::tma_load_4d(d_addr, seg_map, bar, ch * 64, row0, h, f);
            } else {
                tc::tma_load_4d(d_addr, seg_map, bar, ch * 64, h, row0, f);
            }
        }
    }
}

template <int D>
__global__ void __launch_bounds__(kTcThreads, 1)
attn_tc_kernel(const __grid_constant__ TcMaps maps, const TcParams p) {
    using Shape = TcShape<D>;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t q_s = tc::smem_u32(smem);
    const uint32_t k_s = q_s + 2 * Shape::kTileBytes;
    const uint32_t v_s = k_s + kStages * Shape::kTileBytes;

    __shared__ __align__(8) unsigned long long bar_q_full, bar_k_full[kStages], bar_k_empty[kStages],
        bar_v_full[kStages], bar_v_empty[kStages], bar_s_full[2], bar_p_full[2], bar_o_done[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    volatile int* abort_flag = &abort_s;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // decode the work unit
    int idx = blockIdx.x;
    const int split = idx % p.n_splits; idx /= p.n_splits;
    const int f = idx % p.n_forks; idx /= p.n_forks;
    const int rp = idx % p.row_pairs; idx /= p.row_pairs;
    const int h = idx;
    const int tiles_total = p.tiles_prefix + p.tiles_suffix + p.tiles_block;
    const int jt0 = static_cast<int>(static_cast<long long>(tiles_total) * split / p.n_splits);
    const int jt1 = static_cast<int>(static_cast<long long>(tiles_total) * (split + 1) / p.n_splits);
    const int nt = jt1 - jt0;
    const int rows_here = min(256, p.R - rp * 256);
    const int NQ = rows_here > 128 ? 2 : 1;

    if (tid == 0) {
        abort_s = 0;
        tc::mbar_init(tc::smem_u32(&bar_q_full), 1);
        for (int s = 0; s < kStages; ++s) {
            tc::mbar_init(tc::smem_u32(&bar_k_full[s]), 1);
            tc::mbar_init(tc::smem_u32(&bar_k_empty[s]), 1);
            tc::mbar_init(tc::smem_u32(&bar_v_full[s]), 1);
            tc::mbar_init(tc::smem_u32(&bar_v_empty[s]), 1);
        }
        for (int q = 0; q < 2; ++q) {
            tc::mbar_init(tc::smem_u32(&bar_s_full[q]), 1);
            tc::mbar_init(tc::smem_u32(&bar_p_full[q]), 128);
            tc::mbar_init(tc::smem_u32(&bar_o_done[q]), 1);
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
    const uint32_t tm_s[2] = {tmem, tmem + 128};
    const uint32_t tm_o[2] = {tmem + 256, tmem + 256 + D};

    if (warp == 8) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0 && nt > 0) {
            tc::prefetch_tmap(&maps.q);
            const uint32_t bq = tc::smem_u32(&bar_q_full);
            tc::mbar_arrive_expect_tx(bq, NQ * Shape::kTileBytes);
            for (int q = 0; q < NQ; ++q)
                for (int ch = 0; ch < Shape::kChunks; ++ch)
                    tc::tma_load_4d(q_s + q * Shape::kTileBytes + ch * Shape::kChunkBytes, &maps.q, bq, ch * 64,
                                    h * p.G, (rp * 2 + q) * (128 / p.G), f);
            bool ok = true;
            for (int jl = 0; jl < nt && ok; ++jl) {
                const TileInfo t = tile_info(p, jt0 + jl);
                const int s = jl % kStages;
                const uint32_t ph = (jl / kStages) & 1;
                const CUtensorMap* mk = t.segment == 0 ? &maps.pk : (t.segment == 1 ? &maps.sk : &maps.bk);
                const CUtensorMap* mv = t.segment == 0 ? &maps.pv : (t.segment == 1 ? &maps.sv : &maps.bv);
                ok = tc::mbar_wait(tc::smem_u32(&bar_k_empty[s]), ph ^ 1, abort_flag, kWaitLimit);
                if (!ok) break;
                tc::mbar_arrive_expect_tx(tc::smem_u32(&bar_k_full[s]), Shape::kTileBytes);
                load_kv_tile<D>(p, mk, &maps.pk_tail, t, k_s + s * Shape::kTileBytes, tc::smem_u32(&bar_k_full[s]), h, f);
                ok = tc::mbar_wait(tc::smem_u32(&bar_v_empty[s]), ph ^ 1, abort_flag, kWaitLimit);
                if (!ok) break;
                tc::mbar_arrive_expect_tx(tc::smem_u32(&bar_v_full[s]), Shape::kTileBytes);
                load_kv_tile<D>(p, mv, &maps.pv_tail, t, v_s + s * Shape::kTileBytes, tc::smem_u32(&bar_v_full[s]), h, f);
            }
            if (!ok) {
                if (*abort_flag == 0) atomicCAS(p.status, 0, FDD_ERR_DEVICE_TIMEOUT);
                *abort_flag = 1;
                const long long t0 = clock64();          // let copies already in flight land
                while (clock64() - t0 < 2000000) {}
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0 && nt > 0) {
            constexpr uint32_t kIdescQK = tc::idesc_bf16(128, 128, 0);
            constexpr uint32_t kIdescPV = tc::idesc_bf16(128, D, 1);
            auto issue_qk = [&](int q, int s) {
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (k >> 2) * Shape::kChunkBytes + (k & 3) * 32;
                    tc::mma_ss(tm_s[q], tc::smem_desc_sw128(q_s + q * Shape::kTileBytes + off, 0, 1024),
                               tc::smem_desc_sw128(k_s + s * Shape::kTileBytes + off, 0, 1024), kIdescQK, k > 0);
                }
            };
            auto issue_pv = [&](int q, int s, int accumulate) {
#pragma unroll
                for (int j = 0; j < kKeysPerTile / 16; ++j)
                    tc::mma_ts(tm_o[q], tm_s[q] + j * 8,
                               tc::smem_desc_sw128(v_s + s * Shape::kTileBytes + j * 2048, Shape::kChunkBytes, 1024),
                               kIdescPV, (accumulate || j > 0) ? 1u : 0u);
            };
            bool ok = tc::mbar_wait(tc::smem_u32(&bar_q_full), 0, abort_flag, kWaitLimit);
            ok = ok && tc::mbar_wait(tc::smem_u32(&bar_k_full[0]), 0, abort_flag, kWaitLimit);
            if (ok) {
                tc::fence_after_sync();
                for (int q = 0; q < NQ; ++q) {
                    issue_qk(q, 0);
                    tc::mma_commit(tc::smem_u32(&bar_s_full[q]));
                }
                tc::mma_commit(tc::smem_u32(&bar_k_empty[0]));
            }
            for (int jl = 0; jl < nt && ok; ++jl) {
                const int s = jl % kStages;
                const uint32_t ph = (jl / kStages) & 1;
                const int jn = jl + 1, sn = jn % kStages;
                const uint32_t phn = (jn / kStages) & 1;
                ok = tc::mbar_wait(tc::smem_u32(&bar_v_full[s]), ph, abort_flag, kWaitLimit);
                for (int q = 0; q < NQ && ok; ++q) {
                    ok = tc::mbar_wait(tc::smem_u32(&bar_p_full[q]), jl & 1, abort_flag, kWaitLimit);
                    if (!ok) break;
                    tc::fence_after_sync();
                    issue_pv(q, s, jl > 0);
                    tc::mma_commit(tc::smem_u32(&bar_o_done[q]));
                    if (jn < nt) {
                        if (q == 0) {
                            ok = tc::mbar_wait(tc::smem_u32(&bar_k_full[sn]), phn, abort_flag, kWaitLimit);
                            if (!ok) break;
                            tc::fence_after_sync();
                        }
                        issue_qk(q, sn);
                        tc::mma_commit(tc::smem_u32(&bar_s_full[q]));
                    }
                }
                if (!ok) break;
                tc::mma_commit(tc::smem_u32(&bar_v_empty[s]));
                if (jn < nt) tc::mma_commit(tc::smem_u32(&bar_k_empty[sn]));
            }
            if (!ok) {
                if (*abort_flag == 0) atomicCAS(p.status, 0, FDD_ERR_DEVICE_TIMEOUT);
                *abort_flag = 1;
            }
        }
    } else if (warp < 4 * NQ && nt > 0) {
        // ------------------------------------------------------------------ soft-max groups
        const int q = warp >> 2;
        const int row_local = tid & 127;
        const uint32_t lane_base = (static_cast<uint32_t>(warp & 3) * 32u) << 16;
        const int r = rp * 256 + q * 128 + row_local;       // row inside the (rollout, KV head) unit
        const bool row_ok = r < p.R;
        const int qi = row_ok ? r / p.G : 0;
        const int qg = row_ok ? r - qi * p.G : 0;
        const uint32_t bs = tc::smem_u32(&bar_s_full[q]), bp = tc::smem_u32(&bar_p_full[q]), bo = tc::smem_u32(&bar_o_done[q]);
        float m_used = -CUDART_INF_F, l = 0.0f;
        bool ok = true;
        for (int jl = 0; jl < nt; ++jl) {
            const TileInfo t = tile_info(p, jt0 + jl);
            ok = tc::mbar_wait(bs, jl & 1, abort_flag, kWaitLimit);
            if (!ok) break;
            tc::fence_after_sync();
            uint32_t sr[128];
#pragma unroll
            for (int c = 0; c < 4; ++c) tc::tmem_ld32(tm_s[q] + lane_base + c * 32, sr + c * 32);
            tc::wait_ld();
            int limit = t.nvalid;                               // keys [0, limit) are visible
            if (p.causal && t.segment == 2) limit = min(limit, qi - t.index * kKeysPerTile + 1);
            float tmax = -CUDART_INF_F;
            if (limit >= kKeysPerTile) {
#pragma unroll
                for (int i = 0; i < 128; ++i) tmax = fmaxf(tmax, __uint_as_float(sr[i]));
            } else {
#pragma unroll
                for (int i = 0; i < 128; ++i) {
                    if (i >= limit) sr[i] = 0xFF800000u;        // -inf
                    tmax = fmaxf(tmax, __uint_as_float(sr[i]));
                }
            }
            float m_tile = tmax * p.scale_log2;
            if (!(m_tile > -CUDART_INF_F)) m_tile = m_used > -CUDART_INF_F ? m_used : 0.0f;
            if (jl == 0) {
                m_used = m_tile;
            } else {
                const bool need = m_tile > m_used + 8.0f;
                if (__any_sync(0xFFFFFFFFu, need)) {
                    ok = tc::mbar_wait(bo, (jl - 1) & 1, abort_flag, kWaitLimit);
                    if (!ok) break;
                    tc::fence_after_sync();
                    const float alpha = need ? exp2f(m_used - m_tile) : 1.0f;
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        tc::tmem_ld32(tm_o[q] + lane_base + c * 32, o);
                        tc::wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tc::tmem_st32(tm_o[q] + lane_base + c * 32, o);
                    }
                    tc::wait_st();
                    l *= alpha;
                    if (need) m_used = m_tile;
                }
            }
            float psum = 0.0f;
            uint32_t packed[64];
#pragma unroll
            for (int i = 0; i < 64; ++i) {
                const float a = fast_exp2(fmaf(__uint_as_float(sr[2 * i]), p.scale_log2, -m_used));
                const float b = fast_exp2(fmaf(__uint_as_float(sr[2 * i + 1]), p.scale_log2, -m_used));
                psum += a + b;
                const __nv_bfloat162 pk = __floats2bfloat162_rn(a, b);
                packed[i] = *reinterpret_cast<const uint32_t*>(&pk);
            }
            l += psum;
            tc::tmem_st32(tm_s[q] + lane_base, packed);
            tc::tmem_st32(tm_s[q] + lane_base + 32, packed + 32);
            tc::wait_st();
            tc::fence_before_sync();
            tc::mbar_arrive(bp);
        }
        if (ok) ok = tc::mbar_wait(bo, (nt - 1) & 1, abort_flag, kWaitLimit);
        if (ok) {
            tc::fence_after_sync();
            const float inv = l > 0.0f ? 1.0f / l : 0.0f;
            if (p.n_splits == 1) {
                __nv_bfloat16* op = p.out + ((static_cast<size_t>(f) * p.d + qi) * p.n_q_heads + h * p.G + qg) * D;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    tc::tmem_ld32(tm_o[q] + lane_base + c * 32, o);
                    tc::wait_ld();
                    if (row_ok) {
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) {
                            uint32_t w[4];
#pragma unroll
                            for (int x = 0; x < 4; ++x) {
                                const __nv_bfloat162 pk = __floats2bfloat162_rn(__uint_as_float(o[v4 * 8 + 2 * x]) * inv,
                                                                                  __uint_as_float(o[v4 * 8 + 2 * x + 1]) * inv);
                                w[x] = *reinterpret_cast<const uint32_t*>(&pk);
                            }
                            *reinterpret_cast<uint4*>(op + c * 32 + v4 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                }
            } else {
                float* po = p.part_o + (static_cast<size_t>(blockIdx.x) * 256 + q * 128 + row_local) * D;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    tc::tmem_ld32(tm_o[q] + lane_base + c * 32, o);
                    tc::wait_ld();
#pragma unroll
                    for (int v4 = 0; v4 < 8; ++v4)
                        *reinterpret_cast<float4*>(po + c * 32 + v4 * 4) =
                            make_float4(__uint_as_float(o[v4 * 4]) * inv, __uint_as_float(o[v4 * 4 + 1]) * inv,
                                        __uint_as_float(o[v4 * 4 + 2]) * inv, __uint_as_float(o[v4 * 4 + 3]) * inv);
                }
                p.part_lse[static_cast<size_t>(blockIdx.x) * 256 + q * 128 + row_local] = m_used + log2f(l);
            }
        } else {
            if (*abort_flag == 0) atomicCAS(p.status, 0, FDD_ERR_DEVICE_TIMEOUT);
            *abort_flag = 1;
        }
    }

    tc::fence_before_sync();
    __syncthreads();
    if (warp == 9) tc::tmem_dealloc(tmem, 512);
}

// Merge the split-KV partials of one unit: out = sum_s w_s O_s / sum_s w_s, w_s = 2^(lse_s - max).
template <int D>
__global__ void __launch_bounds__(D)
attn_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse, __nv_bfloat16* __restrict__ out,
                  int n_forks, int d, int n_q_heads, int n_kv_heads, int G, int R, int row_pairs, int n_splits) {
    int idx = blockIdx.x;                 // (unit, row) with unit = (h, rp, f)
    const int row = idx % 256; idx /= 256;
    const int f = idx % n_forks; idx /= n_forks;
    const int rp = idx % row_pairs; idx /= row_pairs;
    const int h = idx;
    const int r = rp * 256 + row;
    if (r >= R) return;
    const int unit = (h * row_pairs + rp) * n_forks + f;
    const int c = threadIdx.x;
    float M = -CUDART_INF_F;
    for (int s = 0; s < n_splits; ++s) M = fmaxf(M, part_lse[(static_cast<size_t>(unit) * n_splits + s) * 256 + row]);
    float acc = 0.0f, wsum = 0.0f;
    for (int s = 0; s < n_splits; ++s) {
        const size_t cta = static_cast<size_t>(unit) * n_splits + s;
        const float w = exp2f(part_lse[cta * 256 + row] - M);
        acc = fmaf(w, part_o[(cta * 256 + row) * D + c], acc);
        wsum += w;
    }
    const int i = r / G, g = r - i * G;
    out[((static_cast<size_t>(f) * d + i) * n_q_heads + h * G + g) * D + c] = __float2bfloat16_rn(acc / wsum);
}

bool make_maps(const AttnProblem& a, int D, TcMaps* m) {
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

}  // namespace

// Whether the tensor-core kernel covers this problem.
bool attention_tc_supported(const AttnProblem& a, int head_dim) {
    const int G = a.n_q_heads / a.n_kv_heads;
    if (head_dim != 64 && head_dim != 128) return false;
    if (G < 1 || G > 16 || (G & (G - 1)) != 0) return false;
    if (a.page_tokens != 0 && a.page_tokens != 64) return false;
    return tmap::encode_fn() != nullptr;
}

// Bytes of scratch the split-KV path may need (sized once, at context creation).
size_t attention_tc_workspace_bytes(int head_dim, int sm_count) {
    const size_t ctas = static_cast<size_t>(3) * sm_count;
    return ctas * 256 * (head_dim + 1) * sizeof(float);
}

cudaError_t launch_attention_tc(fdd_ctx* ctx, const AttnProblem& a, int head_dim, cudaStream_t st, int* n_launches) {
    TcMaps maps;
    if (!make_maps(a, head_dim, &maps)) return cudaErrorInvalidValue;
    TcParams p;
    p.out = a.out;
    p.page_table = a.page_table;
    p.status = ctx->d_status;
    p.n_forks = a.n_forks; p.d = a.d; p.n_q_heads = a.n_q_heads; p.n_kv_heads = a.n_kv_heads;
    p.G = a.n_q_heads / a.n_kv_heads;
    p.R = a.d * p.G;
    p.prefix_len = a.prefix_len; p.page_tokens = a.page_tokens; p.n_phys_pages = a.prefix_capacity;
    p.suffix_len = a.suffix_len;
    p.tiles_prefix = (a.prefix_len + kKeysPerTile - 1) / kKeysPerTile;
    p.tiles_suffix = (a.suffix_len + kKeysPerTile - 1) / kKeysPerTile;
    p.tiles_block = (a.d + kKeysPerTile - 1) / kKeysPerTile;
    p.row_pairs = (p.R + 255) / 256;
    p.causal = a.causal_in_block;
    p.scale_log2 = a.scale * 1.4426950408889634f;
    const int units = a.n_kv_heads * p.row_pairs * a.n_forks;
    const int tiles_total = p.tiles_prefix + p.tiles_suffix + p.tiles_block;
    const int sms = ctx->sm_count > 0 ? ctx->sm_count : 148;
    int n_splits = 1;
    if (units < sms) {
        n_splits = sms / units;
        if (n_splits > tiles_total) n_splits = tiles_total;
        const size_t max_ctas = ctx->ws_attn_bytes / (256 * (head_dim + 1) * sizeof(float));
        while (n_splits > 1 && static_cast<size_t>(units) * n_splits > max_ctas) --n_splits;
        if (n_splits < 1) n_splits = 1;
    }
    p.n_splits = n_splits;
    const size_t ctas = static_cast<size_t>(units) * n_splits;
    p.part_o = static_cast<float*>(ctx->ws_attn);
    p.part_lse = p.part_o ? p.part_o + ctas * 256 * head_dim : nullptr;
    cudaError_t e;
    if (head_dim == 128) {
        const int smem = TcShape<128>::kSmemBytes;
        e = cudaFuncSetAttribute(attn_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        attn_tc_kernel<128><<<static_cast<unsigned>(ctas), kTcThreads, smem, st>>>(maps, p);
    } else {
        const int smem = 120 * 1024;      // more than half an SM's shared memory: one CTA (512 TMEM columns) per SM
        e = cudaFuncSetAttribute(attn_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        attn_tc_kernel<64><<<static_cast<unsigned>(ctas), kTcThreads, smem, st>>>(maps, p);
    }
    *n_launches += 1;
    e = cudaGetLastError();
    if (e != cudaSuccess || n_splits == 1) return e;
    const unsigned merge_grid = static_cast<unsigned>(units) * 256u;
    if (head_dim == 128)
        attn_merge_kernel<128><<<merge_grid, 128, 0, st>>>(p.part_o, p.part_lse, a.out, a.n_forks, a.d, a.n_q_heads,
                                                         a.n_kv_heads, p.G, p.R, p.row_pairs, n_splits);
    else
        attn_merge_kernel<64><<<merge_grid, 64, 0, st>>>(p.part_o, p.part_lse, a.out, a.n_forks, a.d, a.n_q_heads,
                                                       a.n_kv_heads, p.G, p.R, p.row_pairs, n_splits);
    *n_launches += 1;
    return cudaGetLastError();
}
