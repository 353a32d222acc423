// Exact row-wise Top-K selector (the mask definition of Section 3.2 of the paper).
//
// One CTA owns one row.  The row's gate values are turned into order-preserving 32-bit keys in
// shared memory; a most-significant-digit radix select (4 passes of 8 bits over a 256-bin
// histogram) finds the exact key tau of the K-th largest element and how many elements are
// strictly larger; one ordered sweep then emits, in ascending channel order, every channel with
// key > tau plus the first (K - n_gt) channels with key == tau.  The sweep order gives both the
// ascending output and the "ties go to the lower channel" rule for free, so the result is unique
// and can be compared bit for bit.
#pragma once

#include "moc_common.cuh"

namespace moc {

constexpr int kSelectThreads = 256;

struct SelectSmem {
    uint32_t hist[256];
    uint32_t warp_tot[32];
    uint32_t chosen_bin;
    uint32_t remaining;
};

// Finds tau (key of the K-th largest) and need (how many keys == tau are to be kept).
// keys: shared memory, n entries.  All threads of the CTA must call it.  THREADS >= 256.
template <int THREADS>
__device__ __forceinline__ void block_radix_threshold(const uint32_t *keys, int n, int k, SelectSmem &sm,
                                                      uint32_t &tau, int &need) {
    static_assert(THREADS >= 256 && THREADS % 32 == 0, "selector needs at least 256 threads");
    const int tid = threadIdx.x;
    uint32_t prefix = 0, mask = 0;
    if (tid == 0) sm.remaining = (uint32_t)k;
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) sm.hist[tid] = 0;
        __syncthreads();
        for (int j = tid; j < n; j += THREADS) {
            uint32_t key = keys[j];
            if ((key & mask) == prefix) atomicAdd(&sm.hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        // inclusive suffix sums S[b] = sum_{c >= b} hist[c] over the 256 bins (threads 0..255)
        uint32_t h = 0, s = 0;
        if (tid < 256) {
            h = sm.hist[tid];
            s = h;
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
            // bin b holds the K-th largest iff  S[b+1] < rem <= S[b]
            if (s >= rem && s - h < rem) sm.chosen_bin = (uint32_t)tid | ((s - h) << 8);
        }
        __syncthreads();
        const uint32_t cb = sm.chosen_bin;
        prefix |= (cb & 255u) << shift;
        mask |= 255u << shift;
        __syncthreads();
        if (tid == 0) sm.remaining -= (cb >> 8);
        // next pass's first __syncthreads orders this update before its use
    }
    __syncthreads();
    tau = prefix;
    need = (int)sm.remaining;
    __syncthreads();
}

// Ordered compaction.  emit(pos, j) is called exactly once for each kept channel j, pos = its rank
// among the kept channels in ascending channel order (0 <= pos < k).
template <int THREADS, typename Emit>
__device__ __forceinline__ void block_ordered_emit(const uint32_t *keys, int n, uint32_t tau, int need,
                                                   SelectSmem &sm, Emit emit) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int NW = THREADS / 32;
    uint32_t run_gt = 0, run_eq = 0;
    for (int base = 0; base < n; base += THREADS) {
        const int j = base + tid;
        const uint32_t key = j < n ? keys[j] : 0u;
        const bool gt = j < n && key > tau;
        const bool eq = j < n && key == tau;
        const uint32_t bg = __ballot_sync(0xffffffffu, gt), be = __ballot_sync(0xffffffffu, eq);
        const uint32_t lt_mask = (1u << lane) - 1u;
        if (lane == 0) sm.warp_tot[warp] = (uint32_t)__popc(bg) | ((uint32_t)__popc(be) << 16);
        __syncthreads();
        uint32_t before = 0, total = 0;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            uint32_t v = sm.warp_tot[w];
            if (w < warp) before += v;
            total += v;
        }
        const uint32_t gt_before = run_gt + (before & 0xffffu) + (uint32_t)__popc(bg & lt_mask);
        const uint32_t eq_before = run_eq + (before >> 16) + (uint32_t)__popc(be & lt_mask);
        if (gt || (eq && eq_before < (uint32_t)need)) {
            emit((int)(gt_before + min(eq_before, (uint32_t)need)), j);
        }
        run_gt += total & 0xffffu;
        run_eq += total >> 16;
        __syncthreads();
    }
}

// Stand-alone selector: gate [rows, n_ld] fp32 -> idx_out [rows, k] int16.  grid.x = rows (strided).
template <int THREADS>
__global__ void __launch_bounds__(THREADS) topk_select_kernel(const float *__restrict__ gate, int64_t rows, int n,
                                                               int n_ld, int k, int16_t *__restrict__ idx_out) {
    extern __shared__ __align__(16) uint32_t select_keys[];
    __shared__ SelectSmem sm;
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        const float *g = gate + r * (int64_t)n_ld;
        for (int j = threadIdx.x; j < n; j += THREADS) select_keys[j] = gate_key(g[j]);
        __syncthreads();
        uint32_t tau;
        int need;
        block_radix_threshold<THREADS>(select_keys, n, k, sm, tau, need);
        int16_t *o = idx_out + r * (int64_t)k;
        block_ordered_emit<THREADS>(select_keys, n, tau, need, sm, [&](int pos, int j) { o[pos] = (int16_t)j; });
        __syncthreads();
    }
}

}  // namespace moc
