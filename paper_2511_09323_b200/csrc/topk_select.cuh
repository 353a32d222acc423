// Exact row-wise Top-K selector (the mask definition of Section 3.2 of the paper).
//
// One CTA owns one row.  The row's gate values are turned into order-preserving 32-bit keys in
// shared memory; a most-significant-digit radix select (4 passes of 8 bits over a 256-bin
// histogram) finds the exact key tau of the K-th largest element and how many elements are
// strictly larger; two sweeps then emit, in ascending channel order, every channel with
// key > tau plus the first (K - n_gt) channels with key == tau.  The sweep order gives both the
// ascending output and the "ties go to the lower channel" rule for free, so the result is unique
// and can be compared bit for bit.
//
// Cost control:
//  * the first pass counts into one private histogram per warp (padded so that equal bins of different
//    warps sit in different banks), because gate values of one row share sign and exponent and would
//    otherwise serialise on a handful of counters;
//  * after the first pass only the keys of the chosen bin are still candidates; when they fit, they
//    are copied to a short list and passes 2..4 read the list instead of the whole row;
//  * the ordered emission needs only a fixed number of block barriers: per-(chunk, warp) counts go to
//    a table, one scan of the table gives every warp its output offset.
#pragma once

#include "moc_common.cuh"

namespace moc {

constexpr int kSelectThreads = 256;
constexpr int kSelectMaxN = 32768;                      // int16 channel indices
constexpr int kSelectCandCap = 2048;                    // candidate list entries
constexpr int kSelectTable = kSelectMaxN / 256 * 8;     // (chunk, warp) slots: 128 chunks x 8 warps

constexpr int kPrivStride = 257;  // per-warp histogram stride: equal bins of different warps hit different banks

template <int NW>
struct SelectSmemT {
    uint32_t hist[256];
    uint32_t warp_tot[32];
    uint32_t cand[kSelectCandCap];
    uint32_t table[kSelectTable];
    uint32_t priv[NW * kPrivStride];  // one private first-pass histogram per warp
    uint32_t chosen_bin;
    uint32_t remaining;
    uint32_t cand_count;
};
using SelectSmem = SelectSmemT<kSelectThreads / 32>;

// From hist[256] and sm.remaining: the bin holding the remaining-th largest, and how many lie above it.
// Result in sm.chosen_bin = bin | (count_above << 8).  All threads call; contains block barriers.
template <int THREADS>
__device__ __forceinline__ void block_pick_bin(SelectSmemT<THREADS / 32> &sm) {
    const int tid = threadIdx.x;
    uint32_t h = 0, s = 0;
    if (tid < 256) {
        h = sm.hist[tid];
        s = h;  // inclusive suffix sum over bins >= tid
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t v = __shfl_down_sync(0xffffffffu, s, o);
            if ((tid & 31) + o < 32) s += v;
        }
        if ((tid & 31) == 0) sm.warp_tot[tid >> 5] = s;
    }
    __syncthreads();
    if (tid < 256) {
        for (int w = (tid >> 5) + 1; w < 8; ++w) s += sm.warp_tot[w];
        const uint32_t rem = sm.remaining;
        if (s >= rem && s - h < rem) sm.chosen_bin = (uint32_t)tid | ((s - h) << 8);
    }
    __syncthreads();
}

// Finds tau (key of the K-th largest) and need (how many keys == tau are to be kept).
// keys: shared memory, n entries.  All threads of the CTA must call it.  THREADS >= 256.
template <int THREADS>
__device__ __forceinline__ void block_radix_threshold(const uint32_t *keys, int n, int k,
                                                      SelectSmemT<THREADS / 32> &sm, uint32_t &tau, int &need) {
    static_assert(THREADS >= 256 && THREADS % 32 == 0, "selector needs at least 256 threads");
    constexpr int NW = THREADS / 32;
    const int tid = threadIdx.x, warp = tid >> 5;
    // ---- pass 1 over the whole row: top 8 bits (sign and exponent).  The gate values of a row share
    // these bits almost entirely, so a single histogram would serialise on a few counters: every warp
    // counts into its own copy and the copies are summed afterwards.
    for (int i = tid; i < NW * kPrivStride; i += THREADS) sm.priv[i] = 0;
    if (tid == 0) {
        sm.remaining = (uint32_t)k;
        sm.cand_count = 0;
    }
    __syncthreads();
    for (int j = tid; j < n; j += THREADS) atomicAdd(&sm.priv[warp * kPrivStride + (keys[j] >> 24)], 1u);
    __syncthreads();
    if (tid < 256) {
        uint32_t h = 0;
#pragma unroll 8
        for (int w = 0; w < NW; ++w) h += sm.priv[w * kPrivStride + tid];
        sm.hist[tid] = h;
    }
    block_pick_bin<THREADS>(sm);
    uint32_t cb = sm.chosen_bin;
    uint32_t prefix = (cb & 255u) << 24, mask = 255u << 24;
    const uint32_t in_bin = sm.hist[cb & 255u];
    __syncthreads();
    if (tid == 0) sm.remaining -= (cb >> 8);
    // ---- candidates of the chosen bin: copy them to the list when they fit
    const bool use_list = in_bin <= (uint32_t)kSelectCandCap;
    if (use_list) {
        for (int base = 0; base < n; base += THREADS) {
            const int j = base + tid;
            const uint32_t key = j < n ? keys[j] : 0u;
            const bool c = j < n && (key & mask) == prefix;
            const uint32_t b = __ballot_sync(0xffffffffu, c);
            uint32_t at = 0;
            if ((tid & 31) == 0 && b) at = atomicAdd(&sm.cand_count, (uint32_t)__popc(b));
            at = __shfl_sync(0xffffffffu, at, 0);
            if (c) sm.cand[at + __popc(b & ((1u << (tid & 31)) - 1u))] = key;
        }
    }
    __syncthreads();
    const uint32_t *src = use_list ? sm.cand : keys;
    const int m = use_list ? (int)in_bin : n;
    // ---- passes 2..4
#pragma unroll 1
    for (int pass = 1; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) sm.hist[tid] = 0;
        __syncthreads();
        for (int j = tid; j < m; j += THREADS) {
            const uint32_t key = src[j];
            if ((key & mask) == prefix) atomicAdd(&sm.hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        block_pick_bin<THREADS>(sm);
        cb = sm.chosen_bin;
        prefix |= (cb & 255u) << shift;
        mask |= 255u << shift;
        __syncthreads();
        if (tid == 0) sm.remaining -= (cb >> 8);
    }
    __syncthreads();
    tau = prefix;
    need = (int)sm.remaining;
    __syncthreads();
}

// ---- threshold by guess and verify ------------------------------------------------------------------
// A CTA that walks many rows of one projection sees thresholds that move little from row to row.
// Given a bracket [lo, hi] around the previous row's threshold, one fused pass over the new row
// (the same pass that converts and stores the keys) counts the keys above hi and the keys not below
// lo and copies the keys inside the bracket to a short list.  If the counts prove that the K-th
// largest key lies inside the bracket and the list did not overflow, one warp finds it exactly by a
// bitwise search over the list; otherwise the row falls back to the full radix select.  Either way
// the result is the exact threshold: the guess only decides how much work finding it takes.
struct SelectGuess {
    float center = 0.f;  // previous threshold (as a float)
    float delta = 0.f;   // half width of the bracket
    bool valid = false;
};

__device__ __forceinline__ float key_to_float(uint32_t key) {
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Loads row g[0..n) into keys[] (shared) and returns tau / need like block_radix_threshold.
// All threads call; `guess` must hold the same values in every thread (it is updated uniformly).
template <int THREADS>
__device__ __forceinline__ void block_select_row(const float *__restrict__ g, int n, int k, uint32_t *keys,
                                                 SelectSmemT<THREADS / 32> &sm, SelectGuess &guess, uint32_t &tau,
                                                 int &need, bool post_silu = false) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t lo = 1u, hi = 0u;  // empty bracket
    if (guess.valid) {
        lo = gate_key(guess.center - guess.delta);
        hi = gate_key(guess.center + guess.delta);
    }
    if (tid == 0) sm.cand_count = 0;
    __syncthreads();
    uint32_t cnt = 0;  // low half: keys > hi, high half: keys >= lo
    for (int base = 0; base < n; base += THREADS) {
        const int j = base + tid;
        uint32_t key = 0u;
        if (j < n) {
            key = gate_key(post_silu ? silu_f(g[j]) : g[j]);  // the key the ranking uses: g, or SiLU(g)
            keys[j] = key;
        }
        if (guess.valid) {
            const bool above = key > hi, not_below = key >= lo;
            cnt += (above ? 1u : 0u) + (not_below ? 0x10000u : 0u);
            const bool band = not_below && !above;
            const uint32_t b = __ballot_sync(0xffffffffu, band);
            if (b) {
                uint32_t at = 0;
                if (lane == 0) at = atomicAdd(&sm.cand_count, (uint32_t)__popc(b));
                at = __shfl_sync(0xffffffffu, at, 0);
                const uint32_t slot = at + (uint32_t)__popc(b & ((1u << lane) - 1u));
                if (band && slot < (uint32_t)kSelectCandCap) sm.cand[slot] = key;
            }
        }
    }
    bool solved = false, overflow = false;
    if (guess.valid) {
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if (lane == 0) sm.warp_tot[warp] = cnt;
        __syncthreads();
        uint32_t tot = 0;
#pragma unroll
        for (int w = 0; w < THREADS / 32; ++w) tot += sm.warp_tot[w];
        const uint32_t c_hi = tot & 0xffffu, c_lo = tot >> 16;
        const uint32_t in_band = sm.cand_count;
        overflow = in_band > (uint32_t)kSelectCandCap;
        solved = c_hi < (uint32_t)k && c_lo >= (uint32_t)k && in_band <= (uint32_t)kSelectCandCap;
        if (solved) {
            if (warp == 0) {
                // the m-th largest of the list, bit by bit below the highest bit in which lo and hi differ
                const uint32_t m = (uint32_t)k - c_hi;
                uint32_t res = hi;
                if (lo != hi) {
                    const int top = 31 - __clz(lo ^ hi);
                    res = hi & ~((2u << top) - 1u);
                    for (int bit = top; bit >= 0; --bit) {
                        const uint32_t trial = res | (1u << bit);
                        uint32_t c = 0;
                        for (uint32_t i = lane; i < in_band; i += 32) c += sm.cand[i] >= trial ? 1u : 0u;
                        c = __reduce_add_sync(0xffffffffu, c);
                        if (c >= m) res = trial;
                    }
                }
                uint32_t gt = 0;
                for (uint32_t i = lane; i < in_band; i += 32) gt += sm.cand[i] > res ? 1u : 0u;
                gt = __reduce_add_sync(0xffffffffu, gt);
                if (lane == 0) {
                    sm.chosen_bin = res;
                    sm.remaining = m - gt;
                }
            }
            __syncthreads();
            tau = sm.chosen_bin;
            need = (int)sm.remaining;
        }
    }
    __syncthreads();
    if (!solved) block_radix_threshold<THREADS>(keys, n, k, sm, tau, need);
    // next row's bracket
    const float t = key_to_float(tau);
    if (!(fabsf(t) <= 3.0e38f)) {
        guess.valid = false;  // infinite threshold: no bracket
    } else if (!guess.valid) {
        guess.center = t;
        guess.delta = 0.05f * fabsf(t) + 1e-30f;
        guess.valid = true;
    } else {
        const float err = fabsf(t - guess.center);
        // converge to about 3.5 standard deviations of the row-to-row change; widen after a miss,
        // narrow when the bracket held too many keys
        guess.delta = solved ? 0.9f * guess.delta + 0.44f * err
                             : (overflow ? 0.5f * guess.delta : 2.0f * err + guess.delta);
        guess.delta = fminf(fmaxf(guess.delta, 1e-30f), 1.0e37f);
        guess.center = t;
    }
}

// Ordered compaction.  emit(pos, j) is called exactly once for each kept channel j, pos = its rank
// among the kept channels in ascending channel order (0 <= pos < k).
template <int THREADS, typename Emit>
__device__ __forceinline__ void block_ordered_emit(const uint32_t *keys, int n, uint32_t tau, int need,
                                                   SelectSmemT<THREADS / 32> &sm, Emit emit) {
    static_assert(THREADS == 256 || THREADS == 1024, "table holds (n / THREADS) x (THREADS / 32) <= 1024 slots");
    constexpr int NW = THREADS / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t lt_mask = (1u << lane) - 1u;
    const int chunks = (n + THREADS - 1) / THREADS;
    const int slots = chunks * NW;
    // sweep 1: per (chunk, warp) counts of key > tau (low half) and key == tau (high half)
    for (int c = 0; c < chunks; ++c) {
        const int j = c * THREADS + tid;
        const uint32_t key = j < n ? keys[j] : 0u;
        const uint32_t bg = __ballot_sync(0xffffffffu, j < n && key > tau);
        const uint32_t be = __ballot_sync(0xffffffffu, j < n && key == tau);
        if (lane == 0) sm.table[c * NW + warp] = (uint32_t)__popc(bg) | ((uint32_t)__popc(be) << 16);
    }
    __syncthreads();
    // exclusive scan of the table in slot order; thread t owns slots [per*t, per*t + per)
    {
        const int per = (slots + THREADS - 1) / THREADS;
        const int s0 = per * tid;
        uint32_t local = 0;
        for (int i = 0; i < per; ++i)
            if (s0 + i < slots) local += sm.table[s0 + i];
        uint32_t inc = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += v;
        }
        if (lane == 31) sm.warp_tot[warp] = inc;
        __syncthreads();
        uint32_t before = inc - local;
        for (int w = 0; w < warp; ++w) before += sm.warp_tot[w];
        for (int i = 0; i < per; ++i) {
            if (s0 + i < slots) {
                const uint32_t v = sm.table[s0 + i];
                sm.table[s0 + i] = before;
                before += v;
            }
        }
    }
    __syncthreads();
    // sweep 2: emit
    for (int c = 0; c < chunks; ++c) {
        const int j = c * THREADS + tid;
        const uint32_t key = j < n ? keys[j] : 0u;
        const bool gt = j < n && key > tau;
        const bool eq = j < n && key == tau;
        const uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
        const uint32_t before = sm.table[c * NW + warp];
        const uint32_t gt_before = (before & 0xffffu) + (uint32_t)__popc(bg & lt_mask);
        const uint32_t eq_before = (before >> 16) + (uint32_t)__popc(be & lt_mask);
        if (gt || (eq && eq_before < (uint32_t)need)) emit((int)(gt_before + min(eq_before, (uint32_t)need)), j);
    }
    __syncthreads();
}

// Stand-alone selector: gate [rows, n_ld] fp32 -> idx_out [rows, k] int16.  grid.x = rows (strided).
template <int THREADS>
__global__ void __launch_bounds__(THREADS) topk_select_kernel(const float *__restrict__ gate, int64_t rows, int n,
                                                               int n_ld, int k, int16_t *__restrict__ idx_out) {
    extern __shared__ __align__(16) uint32_t select_keys[];
    __shared__ SelectSmem sm;
    SelectGuess guess;
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        const float *g = gate + r * (int64_t)n_ld;
        uint32_t tau;
        int need;
        block_select_row<THREADS>(g, n, k, select_keys, sm, guess, tau, need);
        int16_t *o = idx_out + r * (int64_t)k;
        block_ordered_emit<THREADS>(select_keys, n, tau, need, sm, [&](int pos, int j) { o[pos] = (int16_t)j; });
        __syncthreads();
    }
}

}  // namespace moc
