// Confidence-threshold parallel unmasking: vocabulary-wide soft-max statistics and
// (Gumbel-perturbed) arg-max per MASKED row, then the per-rollout commit rule.
//
// Kernel 1 (unmask_partial_kernel): persistent grid.  The MASKED rows of the call, cut into chunks
// of 8192 ids and laid end to end, are split into equal contiguous ranges, one per CTA (with few
// rows every chunk gets a CTA of its own).  A CTA streams each of its pieces from HBM once, 16
// consecutive logits per thread and step (32-byte loads, or 16-byte asynchronous copies through a
// per-thread ring in shared memory), and keeps running soft-max statistics; nothing but the few
// logits that can win the arg-max is looked at twice.  Rows that are not MASKED are never read.
//
// Noise (temperature > 0).  The Gumbel draws are g = -ln(E) with E an exponential race over groups
// of 16 consecutive ids: one 32-bit word R per group (a Philox block serves the four groups that a
// thread meets in four consecutive iterations) fixes the "leader" 16 j + R % 16, which holds the
// group's smallest E = -ln(U) / 16, U = ((R >> 4) + (f + 0.5) 2^-23) / 2^28; every other id of the
// group has E = E_leader - ln((f + 0.5) 2^-23) with 23 fine bits f of its own (second Philox
// stream, one block per 4 ids).  The word alone bounds all 16 draws, which is what makes the
// kernel cheap: the streaming pass tests one word per 16 logits, and the second stream and the
// logarithms are spent only on
//   (1) the leaders of the groups whose word lies in the top 2^-b of its range (b = 2..6, so that
//       a segment has 128 to 256 such groups), whose best exact score L is a lower bound of the
//       segment's best score, and
//   (2) the ids of threads whose largest logit could still beat L with the largest draw any other
//       group allows (g < 6.9237 for b = 6), filtered once more by their own group's bound.
// Any id left out cannot reach L, so the arg-max (lowest id on ties) is exact.
//
// Kernel 2 (unmask_finalize_kernel): one CTA per rollout merges the segment records of its
// rows, forms the confidences and applies the threshold / at-least-one rule.
#include "fdd_internal.h"

#include <math_constants.h>

namespace {

constexpr int kThreads = 256;
constexpr int kGroup = 16;                            // consecutive entries per load and per coarse Philox block
constexpr int kSegQuantum = kThreads * kGroup;        // ids a CTA covers per iteration (4096); segment lengths are multiples of it
constexpr int kMaxCand = 512;                         // groups with a top word kept per segment (148 expected for a 152k row)
constexpr int kMaxRows = kUnmaskMaxRows;              // rows whose state fits the CTA's compaction buffer
// "Top" words: the upper 2^-b of the word range, b chosen per launch so that a segment has 128 to
// 256 top-word groups (b = 6 for whole rows of 152k ids, b = 2 for 8192-id segments).  Every draw
// of the other groups lies below kGumbelPlain[b] > -ln(-ln(1 - 2^-b) / 16).
constexpr int kTopBitsMin = 2, kTopBitsMax = 6;
#ifndef FDD_UM_NOISY_CTAS
#define FDD_UM_NOISY_CTAS 3
#endif
constexpr int kNoisyCtasPerSm = FDD_UM_NOISY_CTAS;   // noisy kernel: CTAs per SM (2: four load buffers per thread, 3: two)
__device__ __forceinline__ float gumbel_plain(int b) {
    return b == 2 ? 4.0195f : (b == 3 ? 4.7870f : (b == 4 ? 5.5140f : (b == 5 ? 6.2235f : 6.9245f)));
}
constexpr float kLog2e = 1.4426950408889634f;

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

// Philox block and word of group j (16 ids): the four words of a block go to groups 256 apart.
__device__ __forceinline__ uint32_t group_counter(int j) { return static_cast<uint32_t>((j >> 10) * 256 + (j & 255)); }
__device__ __forceinline__ uint32_t pick_word(const uint4& r, int k) {
    return k == 0 ? r.x : (k == 1 ? r.y : (k == 2 ? r.z : r.w));
}

// E of a group's leader: -ln(U) / 16, U = (h + (f + 0.5) 2^-23) / 2^28, h = R >> 4.  In the upper
// half the logarithm goes through 1 - U, which fp32 holds almost exactly there.
__device__ __forceinline__ float leader_exponential(uint32_t R, uint32_t f23) {
    const uint32_t h = R >> 4;
    const float frac = (static_cast<float>(f23) + 0.5f) * 1.1920928955078125e-07f;
    float nl;                                               // -ln(U)
    if (h >= (1u << 27)) {
        const float y = (static_cast<float>((1u << 28) - h) - frac) * 3.7252902984619140625e-09f;   // 1 - U
        nl = -log1pf(-y);
    } else {
        nl = 19.408121055678468f - logf(static_cast<float>(h) + frac);                              // 28 ln 2 - ln(2^28 U)
    }
    return nl * 0.0625f;
}
// Lower bound of the leader's E (so of every E of the group) from the word alone.
__device__ __forceinline__ float group_floor(uint32_t R) {
    const float hp = static_cast<float>((R >> 4) + 1u);     // rounds to nearest: the slack below covers it
    return fmaxf(19.408121055678468f - logf(hp), 0.0f) * 0.0625f * 0.999f;
}
// E of an id that is not its group's leader: the leader's plus -ln((f + 0.5) 2^-23).
__device__ __forceinline__ float follower_exponential(float e_leader, uint32_t f23) {
    return e_leader + (15.942385152878742f - logf(static_cast<float>(f23) + 0.5f));                 // 23 ln 2 - ln(f + 0.5)
}

__device__ __forceinline__ float ex2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3f(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

__device__ __forceinline__ void load32(const void* p, uint32_t (&r)[8]) {
    asm volatile("ld.global.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "l"(p));
}

// Asynchronous 16-byte copies global -> shared (the thread that issues them also waits for them).
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Ring of bf16 groups in shared memory: every thread owns 32 bytes per stage, fills them with
// asynchronous copies several groups ahead and reads only what it copied itself (no barrier).
constexpr int kRingStages = 4;
constexpr int kRingStageBytes = kThreads * kGroup * 2;

// A group = 16 consecutive logits.  fetch() starts the 32-byte loads of a group into raw words,
// widen() turns the words into fp32 once they are needed (so several groups can be in flight).
template <typename T> struct Logit;
template <> struct Logit<__nv_bfloat16> {
    static constexpr int kWords = 8;
    __device__ static void fetch(const __nv_bfloat16* p, uint32_t (&w)[kWords]) { load32(p, w); }
    __device__ static void widen(const uint32_t (&w)[kWords], float* out) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            out[2 * i] = __uint_as_float(w[i] << 16);
            out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};
template <> struct Logit<float> {
    static constexpr int kWords = 16;
    __device__ static void fetch(const float* p, uint32_t (&w)[kWords]) {
        uint32_t a[8], b[8];
        load32(p, a);
        load32(p + 8, b);
#pragma unroll
        for (int i = 0; i < 8; ++i) { w[i] = a[i]; w[8 + i] = b[i]; }
    }
    __device__ static void widen(const uint32_t (&w)[kWords], float* out) {
#pragma unroll
        for (int i = 0; i < 16; ++i) out[i] = __uint_as_float(w[i]);
    }
    __device__ static float load1(const float* p) { return *p; }
};

// 16 logits starting at vocabulary id v0 (a multiple of 16); ids >= vocab read as -inf.
template <typename T>
__device__ __forceinline__ void load_group(const T* row_ptr, int v0, int vocab, int vec_ok, float* val) {
    if (vec_ok && v0 + kGroup <= vocab) {
        uint32_t w[Logit<T>::kWords];
        Logit<T>::fetch(row_ptr + v0, w);
        Logit<T>::widen(w, val);
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

template <typename T, bool NOISY>
__global__ void __launch_bounds__(kThreads, NOISY ? kNoisyCtasPerSm : 3)
unmask_partial_kernel(const T* __restrict__ logits, const uint8_t* __restrict__ state,
                      const __grid_constant__ UnmaskSets sets, UnmaskPartial* __restrict__ partial,
                      int vocab, int n_chunks, float temperature,
                      uint32_t block_idx, uint32_t step, int vec_ok, int select_state,
                      const uint32_t* __restrict__ step_counter) {
    if (step_counter != nullptr) step += *step_counter;    // the denoising step as counted on the device
    const int rows = sets.row_off[sets.n_sets];
    __shared__ uint16_t s_rows[kMaxRows];               // the selected rows (MASKED, or DRAFT for the verifier), ascending
    __shared__ int s_n_rows;
    __shared__ int s_warp_count[kThreads / 32];
    __shared__ int s_cand[kMaxCand];                    // groups with a top word: first id of the group ...
    __shared__ uint32_t s_cand_word[kMaxCand];          // ... the word ...
    __shared__ float s_cand_e[kMaxCand];                // ... and its leader's E, once known
    __shared__ int s_n_cand;
    __shared__ uint16_t s_redo[kThreads];               // threads whose groups pass 2 goes over again
    __shared__ int s_n_redo;
    __shared__ float red_max[kThreads / 32], red_sum[kThreads / 32], red_score[kThreads / 32];
    __shared__ Best red_best[kThreads / 32];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr bool noisy = NOISY;                       // temperature > 0

    // Every CTA compacts the list of MASKED rows for itself (the state array is a few KB): a thread
    // takes a run of consecutive rows, one block-wide prefix sum places the runs.
    {
        const int per = (rows + kThreads - 1) / kThreads;          // <= 32 (rows <= 8192)
        const int r_begin = min(rows, tid * per), r_end = min(rows, r_begin + per);
        uint32_t mine = 0;                                         // bit k: row r_begin + k is selected
        for (int r = r_begin; r < r_end; ++r) mine |= (state[r] == select_state ? 1u : 0u) << (r - r_begin);
        const int cnt = __popc(mine);
        int incl = cnt;                                            // inclusive prefix sum inside the warp
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += up;
        }
        if (lane == 31) s_warp_count[warp] = incl;
        __syncthreads();
        int before = incl - cnt, total = 0;
#pragma unroll
        for (int w2 = 0; w2 < kThreads / 32; ++w2) {
            if (w2 < warp) before += s_warp_count[w2];
            total += s_warp_count[w2];
        }
        while (mine) {
            const int k = __ffs(mine) - 1;
            mine &= mine - 1;
            s_rows[before++] = static_cast<uint16_t>(r_begin + k);
        }
        if (tid == 0) { s_n_rows = total; s_n_cand = 0; s_n_redo = 0; }
        __syncthreads();
    }
    const int n_rows = s_n_rows;
    if (n_rows == 0) return;
    // The selected rows, cut into chunks of 8192 ids and laid end to end, are split into equal
    // contiguous ranges, one per CTA: a CTA's range is the tail of one row, some whole rows and the
    // head of another, and every (row, CTA) pair leaves one record (at most n_chunks per row).  With
    // few rows every chunk gets its own CTA.  Every CTA derives the same numbers.
    const long long W = static_cast<long long>(n_rows) * n_chunks;
    const long long G = min(static_cast<long long>(gridDim.x), W);
    if (blockIdx.x >= G) return;
    const long long range_begin = W * blockIdx.x / G, range_end = W * (blockIdx.x + 1) / G;

    for (long long at = range_begin; at < range_end;) {
        const int ri = static_cast<int>(at / n_chunks);
        const int chunk0 = static_cast<int>(at - static_cast<long long>(ri) * n_chunks);
        const int chunk1 = static_cast<int>(min(static_cast<long long>(n_chunks), chunk0 + (range_end - at)));
        at += chunk1 - chunk0;
        const int row = s_rows[ri];
        const int seg_begin = chunk0 * kUnmaskChunk;
        const int seg_end = min(vocab, chunk1 * kUnmaskChunk);
        // which of the row's records this is, and how many there are (CTA c owns chunks [W c / G, W (c + 1) / G))
        const long long row_first = static_cast<long long>(ri) * n_chunks;
        const int cta_first = static_cast<int>(((row_first + 1) * G + W - 1) / W) - 1;
        const int cta_last = static_cast<int>(((row_first + n_chunks) * G + W - 1) / W) - 1;
        const int seg = static_cast<int>(blockIdx.x) - cta_first;
        const int segs = cta_last - cta_first + 1;
        // 2^-top_bits of the groups get their leader scored at once: 128 to 256 groups of this piece
        int top_bits = kTopBitsMin;
        while (top_bits < kTopBitsMax && ((seg_end - seg_begin) >> 4) >> (top_bits + 1) >= 128) ++top_bits;
        const uint32_t top_word = 0xFFFFFFFFu << (32 - top_bits);
        const T* row_ptr = logits + static_cast<size_t>(row) * vocab;
        int set = 0;
        while (set + 1 < sets.n_sets && row >= sets.row_off[set + 1]) ++set;
        const int local = row - sets.row_off[set];
        const int fork = local / sets.d[set], pos = local - fork * sets.d[set];   // rollout inside its set
        uint2 keys = make_uint2(0u, 0u);
        if (noisy) {
            const uint64_t seed = sets.seeds[set][fork];
            keys = make_uint2(static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32));
        }

        // ---- pass 1: stream the segment; running soft-max statistics, coarse bytes, candidates
        float m = -CUDART_INF_F, s = 0.0f;             // thread's running max and sum exp(l - m)
        Best best{-CUDART_INF_F, -CUDART_INF_F, 0x7FFFFFFF};
        // One group: `w` holds its raw words if it could be fetched with the wide loads.
        auto process = [&](int v0, const uint32_t (&w)[Logit<T>::kWords], uint32_t R) {
            float val[kGroup];
            if (vec_ok && v0 + kGroup <= vocab) {
                Logit<T>::widen(w, val);
            } else {
#pragma unroll
                for (int j = 0; j < kGroup; ++j) val[j] = (v0 + j < vocab) ? Logit<T>::load1(row_ptr + v0 + j) : -CUDART_INF_F;
            }
            float g4[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) g4[u] = max3f(val[4 * u], val[4 * u + 1], fmaxf(val[4 * u + 2], val[4 * u + 3]));
            const float gm = fmaxf(fmaxf(g4[0], g4[1]), fmaxf(g4[2], g4[3]));
            if (gm > -CUDART_INF_F) {
                if (!noisy && gm > m) {
                    // greedy: the arg-max so far moves into this group; find its first place
                    int at = kGroup;
#pragma unroll
                    for (int i = kGroup - 1; i >= 0; --i)
                        if (val[i] == gm) at = i;
                    best = Best{gm, gm, v0 + at};
                }
                const float mn = fmaxf(m, gm);
                const float mnl = mn * kLog2e;
                // packed fp32x2 arithmetic: one FMA and one add per two logits
                const float2 l2e2 = make_float2(kLog2e, kLog2e), nm2 = make_float2(-mnl, -mnl);
                float2 s2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
                for (int i = 0; i < kGroup; i += 2) {
                    const float2 x = __ffma2_rn(make_float2(val[i], val[i + 1]), l2e2, nm2);
                    s2[(i >> 1) & 1] = __fadd2_rn(s2[(i >> 1) & 1], make_float2(ex2_fast(x.x), ex2_fast(x.y)));
                }
                const float2 s01 = __fadd2_rn(s2[0], s2[1]);
                const float sa = s01.x, sb = s01.y;
                // rescale by 2^((m - mn) log2e): exactly 1 while the maximum stands (the rounded mnl must
                // not enter here, or a factor 1 + 1e-7 would compound over the groups)
                s = s * ex2_fast((m - mn) * kLog2e) + (sa + sb);
                m = mn;
            }
            if (noisy && R >= top_word && v0 < vocab) {
                const int slot = atomicAdd(&s_n_cand, 1);
                if (slot < kMaxCand) { s_cand[slot] = v0; s_cand_word[slot] = R; }
            }
        };
        auto fetch = [&](int v0, uint32_t (&w)[Logit<T>::kWords]) {
            if (vec_ok && v0 < seg_end && v0 + kGroup <= vocab) Logit<T>::fetch(row_ptr + v0, w);
        };
        if (NOISY && sizeof(T) == 2 && vec_ok) {
            // noisy step on bf16 rows that allow 16-byte copies: the groups travel through the thread's
            // slots of the ring (three copies in flight without holding registers); four consecutive
            // groups of a thread (4096 ids apart) share one Philox block.
            constexpr int S = kRingStages;
            extern __shared__ __align__(16) unsigned char s_ring[];
            const int v_first = seg_begin + tid * kGroup;
            const int n_g = v_first < seg_end ? (seg_end - v_first + kSegQuantum - 1) / kSegQuantum : 0;
            const int k0 = (v_first >> 12) & 3;         // word index of the first group inside its Philox block
            auto issue = [&](int g) {
                const int v = v_first + g * kSegQuantum;
                if (g < n_g && v + kGroup <= vocab) {
                    unsigned char* dst = s_ring + (g % S) * kRingStageBytes + tid * 32;
                    const unsigned char* src = reinterpret_cast<const unsigned char*>(row_ptr + v);
                    cp_async16(dst, src);
                    cp_async16(dst + 16, src + 16);
                }
                cp_async_commit();                      // an empty group keeps the count uniform
            };
#pragma unroll
            for (int g = 0; g < S - 1; ++g) issue(g);
            uint4 rq = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll 4
            for (int g = 0; g < n_g; ++g) {
                issue(g + S - 1);                       // into the slot that was consumed one iteration ago
                cp_async_wait<S - 1>();                 // group g has landed
                const int v = v_first + g * kSegQuantum;
                uint32_t R = 0u;
                if (noisy) {
                    const int k = (k0 + g) & 3;
                    if (g == 0 || k == 0) rq = philox4x32_10(make_uint4(group_counter(v >> 4), pos, step, block_idx), keys);
                    R = pick_word(rq, k);
                }
                uint32_t w[Logit<T>::kWords];
                const uint4* slot = reinterpret_cast<const uint4*>(s_ring + (g % S) * kRingStageBytes + tid * 32);
                const uint4 lo = slot[0], hi = slot[1];
                w[0] = lo.x; w[1] = lo.y; w[2] = lo.z; w[3] = lo.w;
                w[Logit<T>::kWords - 4] = hi.x; w[Logit<T>::kWords - 3] = hi.y; w[Logit<T>::kWords - 2] = hi.z; w[Logit<T>::kWords - 1] = hi.w;
                process(v, w, R);
            }
            cp_async_wait<0>();
        } else if (noisy) {
            // Four iterations (four groups 4096 ids apart) share one Philox block; two register buffers
            // take turns, so the next group's load is in flight while this one is reduced.
            constexpr int Q = kSegQuantum;
            uint32_t wa[Logit<T>::kWords], wb[Logit<T>::kWords];
            int v0 = seg_begin + tid * kGroup;
            const int k0 = (v0 >> 12) & 3;              // word index of the first group inside its Philox block
            fetch(v0, wa);
            if (k0 != 0 && v0 < seg_end) {
                // a segment that starts inside a run of four: finish the run (one to three groups)
                const uint4 rq = philox4x32_10(make_uint4(group_counter(v0 >> 4), pos, step, block_idx), keys);
                if (k0 < 3) fetch(v0 + Q, wb);
                process(v0, wa, pick_word(rq, k0));
                if (k0 < 3 && v0 + Q < seg_end) {
                    if (k0 < 2) fetch(v0 + 2 * Q, wa);
                    process(v0 + Q, wb, pick_word(rq, k0 + 1));
                    if (k0 < 2 && v0 + 2 * Q < seg_end) process(v0 + 2 * Q, wa, rq.w);
                }
                v0 += (4 - k0) * Q;
                fetch(v0, wa);
            }
            if (kNoisyCtasPerSm >= 3) {
                while (v0 < seg_end) {
                    const uint4 rq = philox4x32_10(make_uint4(group_counter(v0 >> 4), pos, step, block_idx), keys);
                    fetch(v0 + Q, wb);
                    process(v0, wa, rq.x);
                    if (v0 + Q < seg_end) { fetch(v0 + 2 * Q, wa); process(v0 + Q, wb, rq.y); }
                    if (v0 + 2 * Q < seg_end) { fetch(v0 + 3 * Q, wb); process(v0 + 2 * Q, wa, rq.z); }
                    if (v0 + 3 * Q < seg_end) { fetch(v0 + 4 * Q, wa); process(v0 + 3 * Q, wb, rq.w); }
                    v0 += 4 * Q;
                }
            } else {
                // four buffers, three loads in flight
                uint32_t wc[Logit<T>::kWords], wd[Logit<T>::kWords];
                fetch(v0 + Q, wb);
                fetch(v0 + 2 * Q, wc);
                while (v0 < seg_end) {
                    const uint4 rq = philox4x32_10(make_uint4(group_counter(v0 >> 4), pos, step, block_idx), keys);
                    fetch(v0 + 3 * Q, wd);
                    process(v0, wa, rq.x);
                    if (v0 + Q < seg_end) { fetch(v0 + 4 * Q, wa); process(v0 + Q, wb, rq.y); }
                    if (v0 + 2 * Q < seg_end) { fetch(v0 + 5 * Q, wb); process(v0 + 2 * Q, wc, rq.z); }
                    if (v0 + 3 * Q < seg_end) { fetch(v0 + 6 * Q, wc); process(v0 + 3 * Q, wd, rq.w); }
                    v0 += 4 * Q;
                }
            }
        } else if (sizeof(T) == 4) {
            uint32_t wa[Logit<T>::kWords], wb[Logit<T>::kWords];
            int v0 = seg_begin + tid * kGroup;
            fetch(v0, wa);
            while (v0 < seg_end) {
                fetch(v0 + kSegQuantum, wb);
                process(v0, wa, 0u);
                if (v0 + kSegQuantum < seg_end) {
                    fetch(v0 + 2 * kSegQuantum, wa);
                    process(v0 + kSegQuantum, wb, 0u);
                }
                v0 += 2 * kSegQuantum;
            }
        } else {
            // the greedy step has little arithmetic per logit to hide the memory latency behind: four
            // buffers, three loads in flight
            uint32_t wa[Logit<T>::kWords], wb[Logit<T>::kWords], wc[Logit<T>::kWords], wd[Logit<T>::kWords];
            int v0 = seg_begin + tid * kGroup;
            fetch(v0, wa);
            fetch(v0 + kSegQuantum, wb);
            fetch(v0 + 2 * kSegQuantum, wc);
            while (v0 < seg_end) {
                fetch(v0 + 3 * kSegQuantum, wd);
                process(v0, wa, 0u);
                if (v0 + kSegQuantum < seg_end) { fetch(v0 + 4 * kSegQuantum, wa); process(v0 + kSegQuantum, wb, 0u); }
                if (v0 + 2 * kSegQuantum < seg_end) { fetch(v0 + 5 * kSegQuantum, wb); process(v0 + 2 * kSegQuantum, wc, 0u); }
                if (v0 + 3 * kSegQuantum < seg_end) { fetch(v0 + 6 * kSegQuantum, wc); process(v0 + 3 * kSegQuantum, wd, 0u); }
                v0 += 4 * kSegQuantum;
            }
        }

        if (noisy) {
            __syncthreads();
            // Exact score of an id of group v0 whose word is R; e_leader < 0: not computed yet.
            auto fine23 = [&](int v) {
                const uint4 r = philox4x32_10(make_uint4(static_cast<uint32_t>(v >> 2), pos | kFineStream, step, block_idx), keys);
                return pick_word(r, v & 3) >> 9;
            };
            // ---- exact scores of the leaders of the top-word groups: their best is a lower bound L of
            // the segment's best
            const int n_cand = s_n_cand;
            const bool overflow = n_cand > kMaxCand;    // (never for random words) then nothing is pruned
            if (!overflow) {
                for (int c = tid; c < n_cand; c += kThreads) {
                    const int v = s_cand[c] + static_cast<int>(s_cand_word[c] & 15u);
                    const float e = leader_exponential(s_cand_word[c], fine23(v));
                    s_cand_e[c] = e;
                    if (v >= vocab) continue;           // the leader of a cut last group may lie beyond the row
                    const float l = Logit<T>::load1(row_ptr + v);
                    best = better(best, Best{fmaf(temperature, -logf(e), l), l, v});
                }
            }
            float lb = best.score;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) lb = fmaxf(lb, __shfl_xor_sync(0xFFFFFFFFu, lb, off));
            if (lane == 0) red_score[warp] = lb;
            __syncthreads();
            lb = red_score[0];
#pragma unroll
            for (int w2 = 1; w2 < kThreads / 32; ++w2) lb = fmaxf(lb, red_score[w2]);
            if (overflow) lb = -CUDART_INF_F;
            // ---- pass 2: every id that can still reach L is scored exactly.  Two kinds of groups are
            // gone over again, by the whole CTA (one group per thread): all groups of the threads whose
            // largest logit can reach L with the largest draw a plain group allows, and the top-word
            // groups (their other 15 ids are bounded by their leader's draw only).
            const float reach = lb - temperature * gumbel_plain(top_bits) - 1e-3f;
            if (m >= reach) {
                const int slot = atomicAdd(&s_n_redo, 1);
                if (slot < kThreads) s_redo[slot] = static_cast<uint16_t>(tid);
            }
            __syncthreads();
            const int n_redo = min(s_n_redo, kThreads);
            const int groups_per_thread = (seg_end - seg_begin + kSegQuantum - 1) / kSegQuantum;
            const int n_plain = n_redo * groups_per_thread;
            const int n_top = overflow ? 0 : n_cand;
            for (int w = tid; w < n_plain + n_top; w += kThreads) {
                int v0;
                uint32_t R;
                bool top;
                if (w < n_plain) {
                    const int owner = s_redo[w / groups_per_thread];
                    v0 = seg_begin + owner * kGroup + (w % groups_per_thread) * kSegQuantum;
                    if (v0 >= seg_end) continue;
                } else {
                    v0 = s_cand[w - n_plain];
                }
                float val[kGroup];
                load_group(row_ptr, v0, vocab, vec_ok, val);
                float e_lead = -1.0f;                   // < 0: not known yet
                if (w < n_plain) {
                    bool some = false;
#pragma unroll
                    for (int i = 0; i < kGroup; ++i) some = some || (val[i] >= reach && val[i] > -CUDART_INF_F);
                    if (!some) continue;
                    const int j = v0 >> 4;
                    R = pick_word(philox4x32_10(make_uint4(group_counter(j), pos, step, block_idx), keys), (j >> 8) & 3);
                    top = R >= top_word;
                    if (top && !overflow) continue;     // comes again as a top-word group
                } else {
                    R = s_cand_word[w - n_plain];
                    e_lead = s_cand_e[w - n_plain];
                    top = true;
                }
                // the bound every draw of the group obeys: exact for a top-word group, from the word
                // alone otherwise (the leader's fine bits are fetched only if some id passes it)
                const int lead = v0 + static_cast<int>(R & 15u);
                if (top && e_lead < 0.0f) e_lead = leader_exponential(R, fine23(lead));
                const float bar = lb - 1e-3f - temperature * -logf(top ? e_lead * 0.999f : group_floor(R));
                uint32_t pass = 0;                      // ids whose logit clears the bar
#pragma unroll
                for (int i = 0; i < kGroup; ++i) pass |= (val[i] >= bar && val[i] > -CUDART_INF_F) ? (1u << i) : 0u;
                while (pass) {
                    const int i = __ffs(pass) - 1;
                    pass &= pass - 1;
                    float l = val[0];
#pragma unroll
                    for (int x = 1; x < kGroup; ++x) if (x == i) l = val[x];
                    const int v = v0 + i;
                    if (e_lead < 0.0f) e_lead = leader_exponential(R, fine23(lead));
                    const float e = v == lead ? e_lead : follower_exponential(e_lead, fine23(v));
                    best = better(best, Best{fmaf(temperature, -logf(e), l), l, v});
                }
            }
        }

        // ---- block reduction
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float m2 = __shfl_xor_sync(0xFFFFFFFFu, m, off);
            const float s2 = __shfl_xor_sync(0xFFFFFFFFu, s, off);
            const float mn = fmaxf(m, m2);
            if (mn > -CUDART_INF_F) s = s * __expf(m - mn) + s2 * __expf(m2 - mn);
            m = mn;
        }
        best = warp_best(best);
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
            out.best_index = B.index;
            out.pad[0] = segs;                          // how many records this row has (read from record 0)
            out.pad[1] = out.pad[2] = 0;
            partial[static_cast<size_t>(row) * n_chunks + seg] = out;
            s_n_cand = 0;
            s_n_redo = 0;
        }
        __syncthreads();                                // red_* and the candidate list are reused by the next item
    }
}

__global__ void __launch_bounds__(128)
unmask_finalize_kernel(const UnmaskPartial* __restrict__ partial, int32_t* __restrict__ tokens,
                       uint8_t* __restrict__ state, int32_t* __restrict__ n_committed,
                       int32_t* __restrict__ n_left, float* __restrict__ conf_out,
                       const __grid_constant__ UnmaskSets sets, int n_chunks, float threshold, int commit_state,
                       uint32_t* __restrict__ step_bump) {
    // (the streaming kernel of this call has read the counter; the next call sees it advanced)
    if (step_bump != nullptr && blockIdx.x == 0 && threadIdx.x == 0) *step_bump += 1u;
    const int fork = blockIdx.x;                        // rollout index over all sets of the call
    const int i = threadIdx.x;
    int set = 0;
    while (set + 1 < sets.n_sets && fork >= sets.fork_off[set + 1]) ++set;
    const int d = sets.d[set];
    const int row0 = sets.row_off[set] + (fork - sets.fork_off[set]) * d;
    __shared__ float s_conf[128];
    __shared__ int s_masked, s_pass;
    if (i == 0) { s_masked = 0; s_pass = 0; }
    __syncthreads();

    const int row = row0 + i;
    bool masked = false;
    float conf = -1.0f;
    int tok = 0;
    if (i < d) {
        masked = state[row] == FDD_MASKED;
        if (masked) {
            const UnmaskPartial* p = partial + static_cast<size_t>(row) * n_chunks;
            const int n_rec = p[0].pad[0];              // records the first kernel wrote for this row
            float M = -CUDART_INF_F;
            for (int c = 0; c < n_rec; ++c) M = fmaxf(M, p[c].row_max);
            float S = 0.0f;
            Best B{-CUDART_INF_F, -CUDART_INF_F, 0x7FFFFFFF};
            for (int c = 0; c < n_rec; ++c) {
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
        state[row] = static_cast<uint8_t>(commit_state);
    }
    if (i == 0) {
        const int nc = (n_masked == 0) ? 0 : (n_pass > 0 ? n_pass : 1);
        n_committed[fork] = nc;
        n_left[fork] = n_masked - nc;
    }
}


// Accept scan of Scaffold Speculative Decoding: one CTA per rollout.  The first kernel has left, for
// every DRAFT row, the verifier's token (arg-max of its perturbed logits).  Going left to right, a
// draft is accepted while it equals the verifier's token; at the first mismatch the verifier's token
// replaces it and every later draft goes back to MASKED.
__global__ void __launch_bounds__(128)
ss_accept_kernel(const UnmaskPartial* __restrict__ partial, int32_t* __restrict__ tokens,
                 uint8_t* __restrict__ state, int32_t* __restrict__ n_accepted, int32_t* __restrict__ n_left,
                 const __grid_constant__ UnmaskSets sets, int n_chunks) {
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
            const UnmaskPartial* p = partial + static_cast<size_t>(row) * n_chunks;
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

// Both entry points launch the same two kernels; only the home of the records differs.
// mode 0: unmasking step; 1: draft of Scaffold Speculative Decoding (every MASKED row becomes DRAFT);
// 2: its accept scan (rows in state DRAFT are read, then the scan runs).
cudaError_t launch_unmask_kernels(const UnmaskProblem& p, UnmaskPartial* partial, cudaStream_t st, int mode = 0) {
    const int select_state = mode == 2 ? FDD_DRAFT : FDD_MASKED;
    const int rows = p.sets.row_off[p.sets.n_sets];
    const int forks = p.sets.fork_off[p.sets.n_sets];
    if (rows > kMaxRows) return cudaErrorInvalidValue;
    const int n_chunks = unmask_chunks(p.vocab);
    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count <= 0)
            sm_count = 148;
    }
    const long long ctas = static_cast<long long>(sm_count) * (p.temperature != 0.0f ? kNoisyCtasPerSm : 3);   // persistent: as many CTAs as fit on the SMs
    const dim3 grid(static_cast<unsigned>(ctas));
    if (p.logits_dtype == FDD_LOGITS_BF16) {
        const int vec_ok = (p.vocab % 16 == 0) && (reinterpret_cast<uintptr_t>(p.logits) % 32 == 0);
        // the noisy bf16 kernel streams through a ring in dynamic shared memory (more than the 48 KB a
        // kernel gets without asking, together with its static arrays)
        constexpr int kRingNoisy = kRingStages * kRingStageBytes, kRingGreedy = 0;
        static bool configured = false;
        if (!configured) {
            cudaError_t ea = cudaFuncSetAttribute(unmask_partial_kernel<__nv_bfloat16, true>,
                                                  cudaFuncAttributeMaxDynamicSharedMemorySize, kRingNoisy);
            if (ea != cudaSuccess) return ea;
            configured = true;
        }
        if (p.temperature != 0.0f)
            unmask_partial_kernel<__nv_bfloat16, true><<<grid, kThreads, kRingNoisy, st>>>(
                static_cast<const __nv_bfloat16*>(p.logits), p.state, p.sets, partial, p.vocab,
                n_chunks, p.temperature, p.block_idx, p.step, vec_ok, select_state, p.step_counter);
        else
            unmask_partial_kernel<__nv_bfloat16, false><<<grid, kThreads, kRingGreedy, st>>>(
                static_cast<const __nv_bfloat16*>(p.logits), p.state, p.sets, partial, p.vocab,
                n_chunks, p.temperature, p.block_idx, p.step, vec_ok, select_state, p.step_counter);
    } else {
        const int vec_ok = (p.vocab % 8 == 0) && (reinterpret_cast<uintptr_t>(p.logits) % 32 == 0);
        if (p.temperature != 0.0f)
            unmask_partial_kernel<float, true><<<grid, kThreads, 0, st>>>(
                static_cast<const float*>(p.logits), p.state, p.sets, partial, p.vocab,
                n_chunks, p.temperature, p.block_idx, p.step, vec_ok, select_state, p.step_counter);
        else
            unmask_partial_kernel<float, false><<<grid, kThreads, 0, st>>>(
                static_cast<const float*>(p.logits), p.state, p.sets, partial, p.vocab,
                n_chunks, p.temperature, p.block_idx, p.step, vec_ok, select_state, p.step_counter);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (mode == 2)
        ss_accept_kernel<<<forks, 128, 0, st>>>(partial, p.tokens, p.state, p.n_committed, p.n_left, p.sets, n_chunks);
    else
        unmask_finalize_kernel<<<forks, 128, 0, st>>>(partial, p.tokens, p.state, p.n_committed, p.n_left, p.conf,
                                                     p.sets, n_chunks, p.threshold, mode == 1 ? FDD_DRAFT : FDD_COMMITTED,
                                                     p.bump_counter ? p.step_counter : nullptr);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_unmask(fdd_ctx* ctx, const UnmaskProblem& p, cudaStream_t st, int* n_launches, int mode) {
    *n_launches += 2;
    return launch_unmask_kernels(p, static_cast<UnmaskPartial*>(ctx->ws_unmask), st, mode);
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
    UnmaskProblem p;
    p.logits = logits; p.tokens = tokens; p.state = state;
    p.n_committed = n_committed; p.n_left = n_left; p.conf = conf;
    p.sets.n_sets = 1;
    p.sets.row_off[0] = 0; p.sets.row_off[1] = n_forks * block_len;
    p.sets.fork_off[0] = 0; p.sets.fork_off[1] = n_forks;
    p.sets.d[0] = block_len; p.sets.seeds[0] = seeds;
    p.vocab = vocab; p.logits_dtype = logits_dtype;
    p.threshold = threshold; p.temperature = temperature; p.block_idx = block_idx; p.step = step;
    e = launch_unmask_kernels(p, g_static_ptr[dev], static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        if (err && err_len) snprintf(err, err_len, "fdd_unmask_static: launch failed: %s", cudaGetErrorString(e));
        return FDD_ERR_CUDA;
    }
    return FDD_OK;
}
