// Small-batch inference path (Section 5 of the paper): tokens <= 16, bf16.
//
// Decode is bound by reading weights from HBM once: the whole gate matrix (F*d elements) plus the
// selected rows of W_up and W_down.  With several tokens, a row selected by more than one token is
// read once (the union of the tokens' channel sets), which is what keeps a batch of 16 cheaper than
// a dense FFN.  Four kernels, all streaming through shared-memory rings filled by bulk async copies
// (the bytes in flight live in shared memory, not in registers):
//   1. gate GEMV   : rows of W_gate dealt out evenly to two CTAs per SM; a producer warp copies
//                    8-row x 1 KiB stages, 8 consumer warps split each stage along the contraction.
//                    The tokens are the M dimension of m16n8k16 tensor-core MMAs, so 16 tokens cost no
//                    more issue slots than one (one FMA per loaded weight and token would be ALU-bound).
//   2. select      : one 1024-thread CTA per token, exact Top-K by a radix select whose digits are taken
//                    relative to the range the candidates lie in (see the kernel).  Decode needs the set,
//                    not the order: each token's selection is a bitmap written word by word from warp
//                    ballots; the last CTA to finish lists the union of the bitmaps (ascending channels).
//   3. up          : the same GEMV over the listed rows of W_up; z = SiLU(g) u for the tokens whose bitmap
//                    holds the channel (zero for the others), stored as bf16 in MMA-ready blocks.
//   4. down        : CTA = (512-column slice, part of the list).  Stages of 16 rows x 1 KiB; the rows are
//                    the contraction index, so the B fragments are read transposed with ldmatrix.
//                    Per-slice partial sums are added to an fp32 accumulator with vector reductions and the last
//                    CTA of a slice writes the bf16 output (the summation order across CTAs is not
//                    fixed, so the last bit of `out` may vary from run to run).
#pragma once

#include "moc_common.cuh"
#include "tc_gemm.cuh"  // mbarrier helpers
#include "topk_select.cuh"

namespace moc {
namespace dec {



constexpr int kSelThreads = 1024;
constexpr int kSelListCap = 4096;   // candidate list entries (two lists)
constexpr int kSelCached = 12;      // keys per thread held in registers by the CTA selector (rows up to 12288 channels)
constexpr int kSliceCols = 512;     // down projection: columns per CTA (1 KiB of a bf16 row)
constexpr int kMaxPart = 512;       // list entries per down CTA (bound of its shared arrays)

// GEMV ring: a stage is 8 rows x 512 contraction elements; rows are padded to 1088 bytes so that the
// 16-byte fragment loads of a quarter warp fall into distinct bank groups
constexpr int kGemvChunk = 512, kGemvPitch = 1088, kGemvStageBytes = 8 * kGemvPitch, kGemvStages = 11;
constexpr int kGemvThreads = 288;   // 8 consumer warps + 1 producer warp
constexpr int kGemvMaxTiles = 8;    // 8-row tiles per CTA: the host sizes the grid so that a CTA owns <= 64 rows
constexpr int kGemvMaxRows = kGemvMaxTiles * 8;
constexpr size_t kGemvSmem = (size_t)kGemvStages * kGemvStageBytes + 128;
// down ring: a stage is 16 rows x 1 KiB, pitch 1040 so that ldmatrix rows fall into distinct bank groups
constexpr int kDownPitch = 1040, kDownStageBytes = 16 * kDownPitch, kDownStages = 4;
constexpr size_t kDownSmem = (size_t)kDownStages * kDownStageBytes + (size_t)kMaxPart * (32 + 2) + 128;

struct Workspace {
    float *G;             // [T, ldf] gate projection
    __nv_bfloat16 *Zb;    // [list position / 16][16 tokens][16 positions] z = SiLU(g) u (0 where not selected)
    uint32_t *sel_bits;   // [T][sel_words] bit j % 32 of word j / 32: token t selected channel j
    int sel_words;        // ceil(F / 32)
    uint16_t *list;       // [F] used channels in order of first selection
    int *list_count;      // number of used channels
    float *out_acc;       // [T, d]
    int *counters;        // [slices] arrival counters of the down kernel
    int ldf;
};

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void consumer_bar_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------- 1 + 3. GEMV
// R[t, r] = sum_i x[t,i] W[row(r), i] for the CTA's share of the rows, all tokens at once.
//   GATHER == false: rows are the channels 0..F-1 of W_gate; result -> G          (Eq. (Moc-1))
//   GATHER == true : rows are the listed channels of W_up;   result -> z = SiLU(g) u on the selection bitmaps
// CTA b owns row slots [b n / grid, (b+1) n / grid).  Each lane reads 16 contiguous bytes (8 contraction
// elements) of a weight row per fragment; the same permutation of the contraction index is applied to the
// x fragment, so the MMA operands need no data movement.
template <bool GATHER>
__global__ void __launch_bounds__(kGemvThreads, 2) gemv_rows_kernel(const __nv_bfloat16 *__restrict__ x,
                                                                    const __nv_bfloat16 *__restrict__ w, int T, int d,
                                                                    int F, Workspace ws, int slices,
                                                                    int *__restrict__ status) {
    extern __shared__ __align__(128) uint8_t gsm[];
    __shared__ uint64_t bars[2 * kGemvStages];
    __shared__ int s_abort;
    __shared__ uint16_t s_rows[kGemvMaxRows];                          // this CTA's rows when gathering
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    tc::pdl_launch_dependents();
    // Gathering: the list of used channels comes from the select kernel, so every thread waits for it here.
    // Gate projection: the weights do not depend on earlier kernels, so the producer warp starts streaming them
    // at once (while the previous kernel of the stream may still be draining); only the consumers wait, before
    // they touch x or the workspace.
    if (GATHER) tc::pdl_wait();
    const int n = GATHER ? min(*ws.list_count, F) : F;
    const int r0 = (int)(((int64_t)blockIdx.x * n) / gridDim.x);
    const int r1 = (int)(((int64_t)(blockIdx.x + 1) * n) / gridDim.x);
    const int tiles = (r1 - r0 + 7) >> 3;
    if (GATHER)
        for (int i = tid; i < r1 - r0 && i < kGemvMaxRows; i += kGemvThreads) s_rows[i] = ws.list[r0 + i];
    const int nkc = (d + kGemvChunk - 1) / kGemvChunk;
    const uint32_t ring = tc::smem_u32(gsm);
    auto full_bar = [&](int s) { return tc::smem_u32(&bars[s]); };
    auto empty_bar = [&](int s) { return tc::smem_u32(&bars[kGemvStages + s]); };

    // When the last chunk of a row is short, the bytes it leaves untouched are multiplied by zero x entries and
    // must therefore be finite: the ring then starts out as zeros.  (Rows of a partial tile that are never
    // copied only feed outputs that are never written.)
    if (d % kGemvChunk != 0)
        for (int i = tid; i < (int)(kGemvStages * kGemvStageBytes / 16); i += kGemvThreads)
            reinterpret_cast<uint4 *>(gsm)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int s = 0; s < kGemvStages; ++s) {
            tc::mbar_init(full_bar(s), 1);
            tc::mbar_init(empty_bar(s), 8);
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // zero fill before the async copies
    __syncthreads();
    if (tiles <= 0 && GATHER) return;  // (the gate kernel's grid never leaves a CTA without rows)

    if (warp == 8) {
        // ------------------------------------------------------------------ producer
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        // stages go chunk by chunk of the contraction index, all the CTA's row tiles within a chunk (the
        // consumers keep a chunk's x fragments in registers across the tiles)
        for (int kc = 0; kc < nkc && ok; ++kc) {
            const int k0 = kc * kGemvChunk;
            const uint32_t bytes = (uint32_t)min(kGemvChunk, d - k0) * 2;
            for (int tile = 0; tile < tiles; ++tile) {
                const int slot = r0 + tile * 8 + lane;  // lanes 0..7 own one row each
                const bool valid = lane < 8 && slot < r1;
                const int row = valid ? (GATHER ? (int)s_rows[slot - r0] : slot) : 0;
                const int nvalid = min(8, r1 - (r0 + tile * 8));
                if (!__all_sync(0xffffffffu, tc::mbar_wait(empty_bar(stage), phase ^ 1u, &s_abort, status))) {
                    ok = false;
                    break;
                }
                if (lane == 0) tc::mbar_expect_tx(full_bar(stage), bytes * (uint32_t)nvalid);
                __syncwarp();
                if (valid)
                    bulk_copy_g2s(ring + stage * kGemvStageBytes + lane * kGemvPitch, w + (int64_t)row * d + k0,
                                  bytes, full_bar(stage));
                if (++stage == kGemvStages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers (warps 0..7)
        // The partial sums of all the CTA's tiles (at most kGemvMaxTiles, the host sizes the grid for that)
        // stay in registers; the eight warps' sums are combined once, after the last stage, in the ring's
        // memory (idle by then).
        if (!GATHER) {
            tc::pdl_wait();
            // housekeeping for the later kernels: clear the accumulators and the arrival counters
            for (int64_t i = (int64_t)blockIdx.x * 256 + tid; i < (int64_t)T * d; i += (int64_t)gridDim.x * 256)
                ws.out_acc[i] = 0.f;
            if (blockIdx.x == 0)
                for (int i = tid; i <= slices; i += 256) ws.counters[i] = 0;  // [slices]: arrivals of the select kernel
        }
        // gathering: the factor SiLU(g) of every output this thread will write (0 where the token did not select
        // the channel) is fetched now, so that the loads are long done when the sums are ready
        const int width = r1 - r0;
        float sfac[4] = {0.f, 0.f, 0.f, 0.f};  // 16 tokens x at most 64 rows / 256 threads
        if (GATHER) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int o = tid + 256 * k;
                if (o < 16 * width) {
                    const int t = o / width, j = s_rows[o - t * width];
                    if (t < T && ((ws.sel_bits[t * ws.sel_words + (j >> 5)] >> (j & 31)) & 1u))
                        sfac[k] = silu_f(ws.G[(int64_t)t * ws.ldf + j]);
                }
            }
        }
        const int g = lane >> 2, q = lane & 3;
        const __nv_bfloat16 *xa_row = x + (int64_t)g * d, *xb_row = x + (int64_t)(g + 8) * d;
        const bool has_a = g < T, has_b = g + 8 < T;
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        float acc[kGemvMaxTiles][4];
#pragma unroll
        for (int ti = 0; ti < kGemvMaxTiles; ++ti) acc[ti][0] = acc[ti][1] = acc[ti][2] = acc[ti][3] = 0.f;
        for (int kc = 0; kc < nkc && ok; ++kc) {
            // this warp's 64 contraction elements of the chunk: two 16-byte fragments per lane and token row
            const int k0 = kc * kGemvChunk + warp * 64 + q * 8;
            uint4 xa0 = make_uint4(0, 0, 0, 0), xa1 = xa0, xb0 = xa0, xb1 = xa0;
            if (has_a) {
                if (k0 < d) xa0 = *reinterpret_cast<const uint4 *>(xa_row + k0);
                if (k0 + 32 < d) xa1 = *reinterpret_cast<const uint4 *>(xa_row + k0 + 32);
            }
            if (has_b) {
                if (k0 < d) xb0 = *reinterpret_cast<const uint4 *>(xb_row + k0);
                if (k0 + 32 < d) xb1 = *reinterpret_cast<const uint4 *>(xb_row + k0 + 32);
            }
#pragma unroll
            for (int ti = 0; ti < kGemvMaxTiles; ++ti) {
                if (ti < tiles && ok) {  // uniform
                    if (!__all_sync(0xffffffffu, tc::mbar_wait(full_bar(stage), phase, &s_abort, status))) {
                        ok = false;
                        break;
                    }
                    const uint8_t *src = gsm + stage * kGemvStageBytes + g * kGemvPitch + warp * 128 + q * 16;
                    const uint4 w0 = *reinterpret_cast<const uint4 *>(src);
                    const uint4 w1 = *reinterpret_cast<const uint4 *>(src + 64);
                    mma_bf16_16816(acc[ti], xa0.x, xb0.x, xa0.y, xb0.y, w0.x, w0.y);
                    mma_bf16_16816(acc[ti], xa0.z, xb0.z, xa0.w, xb0.w, w0.z, w0.w);
                    mma_bf16_16816(acc[ti], xa1.x, xb1.x, xa1.y, xb1.y, w1.x, w1.y);
                    mma_bf16_16816(acc[ti], xa1.z, xb1.z, xa1.w, xb1.w, w1.z, w1.w);
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(empty_bar(stage));
                    if (++stage == kGemvStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
        // every warp passes both barriers, also after a failed wait
        consumer_bar_sync();
        float *red = reinterpret_cast<float *>(gsm);  // [8 warps][16 tokens][kGemvMaxTiles * 8 + 1]
        constexpr int RP = kGemvMaxTiles * 8 + 1;
#pragma unroll
        for (int ti = 0; ti < kGemvMaxTiles; ++ti) {
            float *r = red + (warp * 16) * RP + ti * 8 + 2 * q;
            r[g * RP] = acc[ti][0];
            r[g * RP + 1] = acc[ti][1];
            r[(g + 8) * RP] = acc[ti][2];
            r[(g + 8) * RP + 1] = acc[ti][3];
        }
        consumer_bar_sync();
        ok = ok && !s_abort;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int o = tid + 256 * k;
            if (ok && o < 16 * width) {
                const int t = o / width, c = o - t * width;
                const int slot = r0 + c;
                float sum = 0.f;
#pragma unroll
                for (int wi = 0; wi < 8; ++wi) sum += red[(wi * 16 + t) * RP + c];
                if (!GATHER) {
                    if (t < T) ws.G[(int64_t)t * ws.ldf + slot] = sum;
                } else {
                    ws.Zb[((int64_t)(slot >> 4) * 16 + t) * 16 + (slot & 15)] = __float2bfloat16_rn(sfac[k] * sum);
                }
            }
        }
    }
    __syncwarp();
    if (s_abort) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
}

// Last step of both select kernels: the last CTA to get here (one CTA per token) lists the used channels (ascending)
// for the up and down kernels.  dyn: the CTA's dynamic shared memory (free by now, at least d_ff / 2 + 1 words).
__device__ __forceinline__ void list_used_channels(const Workspace &ws, int F, int *arrivals, uint32_t *dyn) {
    constexpr int NW = kSelThreads / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ int s_is_last, s_warp_cnt[NW];
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        s_is_last = atomicAdd(arrivals, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (!s_is_last) return;
    __threadfence();
    // union of the tokens' bitmaps, one word per thread (at most 1024 words), block-wide exclusive scan of the
    // popcounts, then every thread writes the channels of its word
    uint32_t word = 0;
    if (tid < ws.sel_words) {
        uint32_t part[16];  // at most 16 tokens: all loads in flight together
#pragma unroll
        for (int tt = 0; tt < 16; ++tt)
            part[tt] = tt < (int)gridDim.x ? __ldcg(&ws.sel_bits[(int64_t)tt * ws.sel_words + tid]) : 0u;
#pragma unroll
        for (int tt = 0; tt < 16; ++tt) word |= part[tt];
    }
    const int v = __popc(word);
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += u;
    }
    if (lane == 31) s_warp_cnt[warp] = inc;
    __syncthreads();
    int wt = s_warp_cnt[lane], winc = wt;  // NW == 32: one warp total per lane
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, winc, o);
        if (lane >= o) winc += u;
    }
    const int before_warp = __shfl_sync(0xffffffffu, winc - wt, warp), total = __shfl_sync(0xffffffffu, winc, 31);
    // the list is put together in shared memory (the keys' memory, free by now) and leaves in whole words:
    // consecutive 2-byte stores of one thread to global memory serialise on their sector
    uint16_t *slist = reinterpret_cast<uint16_t *>(dyn);
    __syncthreads();  // all threads are done with the keys
    int pos = before_warp + inc - v;
    while (word) {
        const int bpos = __ffs(word) - 1;
        word &= word - 1u;
        slist[pos++] = (uint16_t)(tid * 32 + bpos);
    }
    __syncthreads();
    for (int i = tid; i < (total + 1) / 2; i += kSelThreads)  // the list array holds F (rounded up to even) entries
        reinterpret_cast<uint32_t *>(ws.list)[i] = reinterpret_cast<const uint32_t *>(slist)[i];
    if (tid == 0) *ws.list_count = total;
}

// ---------------------------------------------------------------------------------------------- 2'. grouped select
// MoC 2:8 (Section 4): the 2 largest of every 8 consecutive channels.  One CTA per token as above, but the mask is
// local: the eight lanes that hold a group rank their keys against each other with shuffles, and the ballot of
// "rank < 2" is a word of the token's selection bitmap.
__global__ void __launch_bounds__(kSelThreads) select_grouped_bits_kernel(Workspace ws, int F, int *arrivals) {
    extern __shared__ __align__(16) uint32_t dyn[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int NW = kSelThreads / 32;
    const int t = blockIdx.x;
    tc::pdl_launch_dependents();
    tc::pdl_wait();
    const float *g = ws.G + (int64_t)t * ws.ldf;
    uint32_t *my_bits = ws.sel_bits + (int64_t)t * ws.sel_words;
    const int nch = (F + kSelThreads - 1) / kSelThreads;
    for (int c = 0; c < nch; ++c) {
        const int j = c * kSelThreads + tid;  // d_ff is a multiple of 8: a group never straddles the end
        const uint32_t key = j < F ? gate_key(g[j]) : 0u;
        const int first = lane & ~7, me = lane & 7;
        int before = 0;
#pragma unroll
        for (int f = 0; f < 8; ++f) {
            const uint32_t o = __shfl_sync(0xffffffffu, key, first + f);
            before += (o > key || (o == key && f < me)) ? 1 : 0;
        }
        const uint32_t b = __ballot_sync(0xffffffffu, j < F && before < 2);
        if (lane == 0 && c * kSelThreads + warp * 32 < F) my_bits[c * NW + warp] = b;
    }
    list_used_channels(ws, F, arrivals, dyn);
}

// ---------------------------------------------------------------------------------------------- 2. select
// One CTA per token: exact Top-K set of G[t, 0..F).
//
// A single CTA has to find the K-th largest of ~10^4 keys with as few block-wide steps as possible.
// Radix select with digits taken from the top of the key fails at that here: the keys of one row share
// sign and exponent, so the first digits put almost everything into a few bins (serialised counters) and
// narrow the candidates very slowly.  Instead the digits are taken relative to the range the candidates
// are known to lie in: with [lo, hi] the current range, bin = (key - lo) >> shift with shift chosen so
// that the range maps onto at most 2048 bins.  The first level uses the row's minimum and maximum key;
// the bin that holds the K-th largest then holds a handful of keys, which are copied to a short list and
// ranked directly.  Further levels (only for very uneven data) repeat the step on the list.
// Decode needs the set, not the order: consecutive lanes hold consecutive channels, so a warp ballot of
// "key >= threshold" is one word of the token's selection bitmap; only when ties at the threshold must be
// cut does the ordered emission run.  The kernels are chained with programmatic dependent launch: each
// calls pdl_wait before it touches what an earlier kernel wrote.
struct SelectLevel {
    uint32_t lo, hi;  // candidates lie in [lo, hi]
    uint32_t m;       // the m-th largest of them is wanted
    uint32_t count;   // number of candidates
};

// One bulk copy of `bytes` (a multiple of 16) from global `src` to shared `dst` (both 16-byte aligned), or two when
// src2 is given (begin), and a bounded wait for them (wait).  Every thread of the CTA calls both; the result is the
// same for all (false: the wait ran out and MOC_ERR_TIMEOUT was raised).  `bar` / `abort_flag`: shared scratch.
__device__ __forceinline__ void cta_stage_rows_begin(uint64_t *bar, int *abort_flag, void *dst, const void *src,
                                                     uint32_t bytes, void *dst2 = nullptr,
                                                     const void *src2 = nullptr) {
    const uint32_t b = tc::smem_u32(bar);
    if (threadIdx.x == 0) {
        tc::mbar_init(b, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        tc::mbar_expect_tx(b, src2 ? 2 * bytes : bytes);
        tc::bulk_copy_g2s(tc::smem_u32(dst), src, bytes, b);
        if (src2) tc::bulk_copy_g2s(tc::smem_u32(dst2), src2, bytes, b);
    }
    __syncthreads();  // the barrier is initialised before anyone polls it
}
__device__ __forceinline__ bool cta_stage_rows_wait(uint64_t *bar, int *abort_flag, int *status) {
    const bool ok = tc::mbar_wait(tc::smem_u32(bar), 0u, abort_flag, status);
    return __syncthreads_or(ok ? 0 : 1) == 0;
}
__device__ __forceinline__ bool cta_stage_rows(uint64_t *bar, int *abort_flag, int *status, void *dst, const void *src,
                                               uint32_t bytes) {
    cta_stage_rows_begin(bar, abort_flag, dst, src, bytes);
    return cta_stage_rows_wait(bar, abort_flag, status);
}

// The threshold search of one CTA (kSelThreads threads) over the row g[0..F): fills keys[0..F) and returns the
// K-th largest key `tau`, how many keys equal to tau belong to the set (`need`), and whether some keys equal to
// tau must be left out (`ties_cut`; false: the set is exactly "key >= tau").
// g == nullptr: keys[] already holds the row's fp32 values (staged by a bulk copy) and is converted in place.
// lists0: two candidate lists of kSelListCap entries; sm: the full radix select's state (its arrays double as scratch).
// kreg: the calling thread's keys when the row is short enough to be held in registers (F <= kSelCached * kSelThreads;
// element i = channel tid + i * kSelThreads, 0 beyond the row), for callers that go over the row once more.
__device__ __forceinline__ void cta_select_threshold(const float *__restrict__ g, int F, int K, uint32_t *keys,
                                                     uint32_t *lists0, SelectSmemT<kSelThreads / 32> &sm,
                                                     uint32_t &tau_out, int &need_out, bool &ties_cut_out,
                                                     uint32_t (&kreg)[kSelCached]) {
    __shared__ uint32_t s_min[32], s_max[32], s_pick, s_above, s_inbin, s_n;
    uint32_t *lists[2] = {lists0, lists0 + kSelListCap};
    uint32_t *hist = sm.priv;  // 2048 entries
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int NW = kSelThreads / 32;

    // ---- keys, minimum and maximum.  Rows of up to kSelCached * kSelThreads channels also stay in registers (element
    // i of a thread is channel tid + i * kSelThreads): the first level's passes then run without loads.
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    const bool cached = F <= kSelCached * kSelThreads;
    if (cached) {
#pragma unroll
        for (int i = 0; i < kSelCached; ++i) {
            const int j = tid + i * kSelThreads;
            kreg[i] = 0u;
            if (j < F) {
                const uint32_t key = gate_key(g ? g[j] : __uint_as_float(keys[j]));
                keys[j] = key;
                kreg[i] = key;
                kmin = min(kmin, key);
                kmax = max(kmax, key);
            }
        }
    } else {
        for (int j = tid; j < F; j += kSelThreads) {
            const uint32_t key = gate_key(g ? g[j] : __uint_as_float(keys[j]));
            keys[j] = key;
            kmin = min(kmin, key);
            kmax = max(kmax, key);
        }
    }
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if (lane == 0) {
        s_min[warp] = kmin;
        s_max[warp] = kmax;
    }
    for (int i = tid; i < 2048; i += kSelThreads) hist[i] = 0;
    if (tid == 0) s_n = 0;
    __syncthreads();
    kmin = s_min[lane];
    kmax = s_max[lane];
    kmin = __reduce_min_sync(0xffffffffu, kmin);
    kmax = __reduce_max_sync(0xffffffffu, kmax);

    SelectLevel lv{kmin, kmax, (uint32_t)K, (uint32_t)F};
    const uint32_t *src = keys;
    int which = 0;
    bool failed = false, by_value = true;
    uint32_t tau = 0, in_bin = 0;
    int need = 0, level = 0;
    // ---- levels: histogram the candidates over their own range, keep the bin that holds the m-th largest
    while (true) {
        const uint32_t span = lv.hi - lv.lo;
        if (span == 0) {  // all candidates equal
            tau = lv.lo;
            need = (int)lv.m;
            in_bin = lv.count;
            break;
        }
        if (lv.count <= 128u && src != keys) {
            // The usual end of the search: a handful of candidates, ranked by the whole CTA at once.  Eight threads
            // share a candidate and split the others between them; candidate i is the answer when exactly m-1
            // others precede it in (value descending, list position ascending) order.
            const uint32_t cand = (uint32_t)tid >> 3, sub = (uint32_t)tid & 7u;
            const bool act = cand < lv.count;
            const uint32_t mine = act ? src[cand] : 0u;
            uint32_t before = 0, equal = 0, gt = 0;
            if (act) {
                for (uint32_t j = sub; j < lv.count; j += 8) {
                    const uint32_t o = src[j];
                    gt += o > mine ? 1u : 0u;
                    before += (o > mine || (o == mine && j < cand)) ? 1u : 0u;
                    equal += o == mine ? 1u : 0u;
                }
            }
#pragma unroll
            for (int o = 1; o < 8; o <<= 1) {
                before += __shfl_xor_sync(0xffffffffu, before, o);
                equal += __shfl_xor_sync(0xffffffffu, equal, o);
                gt += __shfl_xor_sync(0xffffffffu, gt, o);
            }
            if (act && sub == 0 && before == lv.m - 1) {
                s_pick = mine;
                s_above = lv.m - gt;  // how many keys equal to tau are wanted
                s_inbin = equal;
            }
            __syncthreads();
            tau = s_pick;
            need = (int)s_above;
            in_bin = s_inbin;
            break;
        }
        // Bins are taken over the candidates' VALUE range where that is possible: the keys of one row share sign and
        // exponent, so equal steps of the key put a quarter of an octave into one bin (hundreds of candidates around
        // the threshold), while equal steps of the value leave a handful.  The map value -> bin is monotone, which is
        // all the search needs; ranks inside the kept bin are decided on the exact keys.  Where the value range is
        // not finite, or a level made no progress, the bins are equal steps of the key (which always narrow).
        const float lo_f = key_to_float(lv.lo), hi_f = key_to_float(lv.hi);
        const float inv = 2048.0f / (hi_f - lo_f);
        const bool lin = by_value && isfinite(lo_f) && isfinite(hi_f) && isfinite(inv) && inv > 0.f;
        const int bits = 32 - __clz(span);
        const int shift = bits > 11 ? bits - 11 : 0;
        auto bin_of = [&](uint32_t key) -> uint32_t {
            if (lin) return (uint32_t)min(2047, max(0, __float2int_rd((key_to_float(key) - lo_f) * inv)));
            return (key - lv.lo) >> shift;
        };
        // histogram over the candidates (hist is zero on entry)
        if (src == keys && cached) {
#pragma unroll
            for (int i = 0; i < kSelCached; ++i)
                if (tid + i * kSelThreads < F) atomicAdd(&hist[bin_of(kreg[i])], 1u);
        } else {
            for (uint32_t i = tid; i < lv.count; i += kSelThreads) {
                const uint32_t key = src[i];
                if (key >= lv.lo && key <= lv.hi) atomicAdd(&hist[bin_of(key)], 1u);
            }
        }
        __syncthreads();
        // suffix sums: thread i owns bins 2i, 2i+1
        const uint32_t h0 = hist[2 * tid], h1 = hist[2 * tid + 1];
        uint32_t s = h0 + h1;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_down_sync(0xffffffffu, s, o);
            if (lane + o < 32) s += v;
        }
        if (lane == 0) sm.warp_tot[warp] = s;
        __syncthreads();
        {
            // totals of the warps after this one: a second-level suffix scan done by every warp on its own
            uint32_t w = sm.warp_tot[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t v = __shfl_down_sync(0xffffffffu, w, o);
                if (lane + o < 32) w += v;
            }
            const uint32_t after = __shfl_sync(0xffffffffu, w, (warp + 1) & 31);
            if (warp + 1 < NW) s += after;
        }
        if (s - h0 >= lv.m && s - h0 - h1 < lv.m) {
            s_pick = 2 * tid + 1;
            s_above = s - h0 - h1;
            s_inbin = h1;
        } else if (s >= lv.m && s - h0 < lv.m) {
            s_pick = 2 * tid;
            s_above = s - h0;
            s_inbin = h0;
        }
        if (tid == 0) {
            s_min[0] = 0xffffffffu;  // range of the kept bin's keys, for the next level
            s_max[0] = 0u;
        }
        __syncthreads();
        const uint32_t bin = s_pick;
        const uint32_t new_m = lv.m - s_above, new_count = s_inbin;
        if (!lin && shift == 0) {  // the bin is a single key value
            tau = lv.lo + bin;
            need = (int)new_m;
            in_bin = new_count;
            break;
        }
        if (new_count > (uint32_t)kSelListCap) {
            failed = true;
            break;
        }
        // copy the bin's keys to the other list (with their range) and clear the histogram for the next level
        uint32_t *dst = lists[which];
        auto keep = [&](uint32_t key) {
            if (key >= lv.lo && key <= lv.hi && bin_of(key) == bin) {
                dst[atomicAdd(&s_n, 1u)] = key;
                atomicMin(&s_min[0], key);
                atomicMax(&s_max[0], key);
            }
        };
        if (src == keys && cached) {
#pragma unroll
            for (int i = 0; i < kSelCached; ++i)
                if (tid + i * kSelThreads < F) keep(kreg[i]);
        } else {
            for (uint32_t i = tid; i < lv.count; i += kSelThreads) keep(src[i]);
        }
        for (int i = tid; i < 2048; i += kSelThreads) hist[i] = 0;
        __syncthreads();
        if (++level >= 6) by_value = false;  // rows whose values thin out over many octaves: key steps end in three levels
        lv = SelectLevel{s_min[0], s_max[0], new_m, new_count};
        src = dst;
        which ^= 1;
        __syncthreads();
        if (tid == 0) s_n = 0;
    }
    bool ties_cut = true;  // true: some keys equal to tau must be left out -> ordered emission
    if (failed)
        block_radix_threshold<kSelThreads>(keys, F, K, sm, tau, need);
    else
        ties_cut = in_bin != (uint32_t)need;
    tau_out = tau;
    need_out = need;
    ties_cut_out = ties_cut;
}

__global__ void __launch_bounds__(kSelThreads) select_mask_kernel(Workspace ws, int F, int K, int *arrivals,
                                                                  int *__restrict__ status) {
    static_assert(kSelThreads == 1024, "the listing step scans one count per lane");
    extern __shared__ __align__(16) uint32_t dyn[];  // keys [F rounded up to 4] | candidate lists 2 x [kSelListCap]
    __shared__ SelectSmemT<kSelThreads / 32> sm;
    __shared__ uint64_t s_bar;
    __shared__ int s_abort;
    const uint32_t *keys = dyn;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int NW = kSelThreads / 32;
    const int t = blockIdx.x;
    const int Fp = (F + 3) & ~3;
    tc::pdl_launch_dependents();
    tc::pdl_wait();
    // the token's gate row arrives with one bulk copy instead of a chain of dependent loads
    if (!cta_stage_rows(&s_bar, &s_abort, status, dyn, ws.G + (int64_t)t * ws.ldf, (uint32_t)Fp * 4u)) return;
    uint32_t tau;
    int need;
    bool ties_cut;
    uint32_t kreg[kSelCached];
    cta_select_threshold(nullptr, F, K, dyn, dyn + Fp, sm, tau, need, ties_cut, kreg);
    uint32_t *my_bits = ws.sel_bits + (int64_t)t * ws.sel_words;
    const int nch = (F + kSelThreads - 1) / kSelThreads;
    if (!ties_cut) {
        // every key >= tau is kept: consecutive lanes hold consecutive channels, so a ballot IS a word of the
        // token's selection bitmap (plain stores, no atomics, nothing read back)
        for (int c = 0; c < nch; ++c) {
            const int j = c * kSelThreads + tid;
            const uint32_t b = __ballot_sync(0xffffffffu, j < F && keys[j] >= tau);
            if (lane == 0 && c * kSelThreads + warp * 32 < F) my_bits[c * NW + warp] = b;
        }
    } else {
        for (int i = tid; i < ws.sel_words; i += kSelThreads) my_bits[i] = 0u;
        __syncthreads();
        block_ordered_emit<kSelThreads>(keys, F, tau, need, sm,
                                        [&](int, int j) { atomicOr(&my_bits[j >> 5], 1u << (j & 31)); });
    }
    list_used_channels(ws, F, arrivals, dyn);
}


// Stand-alone form of the CTA-per-row selector (test hook): gate [rows, n_ld] fp32 -> idx_out [rows, k] int16 ascending.
__global__ void __launch_bounds__(kSelThreads) cta_select_idx_kernel(const float *__restrict__ gate, int n, int n_ld,
                                                                      int k, int16_t *__restrict__ idx_out,
                                                                      int *__restrict__ status) {
    extern __shared__ __align__(16) uint32_t dyn[];
    __shared__ SelectSmemT<kSelThreads / 32> sm;
    __shared__ uint64_t s_bar;
    __shared__ int s_abort;
    const int np = (n + 3) & ~3;
    const float *g = gate + (int64_t)blockIdx.x * n_ld;
    // rows that start on a 16-byte boundary and can be read four values at a time arrive with a bulk copy
    const bool staged = (n_ld & 3) == 0 && np <= n_ld && (reinterpret_cast<uintptr_t>(gate) & 15u) == 0;
    if (staged && !cta_stage_rows(&s_bar, &s_abort, status, dyn, g, (uint32_t)np * 4u)) return;
    uint32_t tau;
    int need;
    bool ties_cut;
    uint32_t kreg[kSelCached];
    cta_select_threshold(staged ? nullptr : g, n, k, dyn, dyn + np, sm, tau, need, ties_cut, kreg);
    int16_t *out = idx_out + (int64_t)blockIdx.x * k;
    block_ordered_emit<kSelThreads>(dyn, n, tau, need, sm, [&](int pos, int j) { out[pos] = (int16_t)j; });
}

// ---------------------------------------------------------------------------------------------- 4. down
// out[t, c] = sum_{j in C_t} z[t,j] Wd[j, c]   (Section 5, final output) for the CTA's column slice and its
// part of the list of used channels.  grid = (slices, parts).  Tokens are the M dimension of the MMA, the
// listed channels its contraction index: B[k = channel][n = column] is row-major in shared memory and is
// read transposed with ldmatrix.
__global__ void __launch_bounds__(kGemvThreads, 2) down_rows_kernel(const __nv_bfloat16 *__restrict__ wd, int T, int d,
                                                                    int F, Workspace ws,
                                                                    __nv_bfloat16 *out, const __nv_bfloat16 *resid,
                                                                    int *__restrict__ status) {
    extern __shared__ __align__(128) uint8_t dsm[];
    // layout: ring [kDownStages][16][kDownPitch] | z blocks [kMaxPart / 16][16 tokens][16] bf16 | channel [kMaxPart]
    uint8_t *ring = dsm;
    __nv_bfloat16 *zl = reinterpret_cast<__nv_bfloat16 *>(dsm + kDownStages * kDownStageBytes);
    uint16_t *lch = reinterpret_cast<uint16_t *>(zl + kMaxPart * 16);
    __shared__ uint64_t bars[2 * kDownStages];
    __shared__ int s_abort, s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slice = blockIdx.x, c0 = slice * kSliceCols;
    const int cols = min(kSliceCols, d - c0);       // multiple of 8
    const uint32_t row_bytes = (uint32_t)cols * 2;  // multiple of 16
    tc::pdl_launch_dependents();
    auto full_bar = [&](int s) { return tc::smem_u32(&bars[s]); };
    auto empty_bar = [&](int s) { return tc::smem_u32(&bars[kDownStages + s]); };
    for (int i = tid; i < (int)(kDownStages * kDownStageBytes / 16); i += kGemvThreads)
        reinterpret_cast<uint4 *>(ring)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int s = 0; s < kDownStages; ++s) {
            tc::mbar_init(full_bar(s), 1);
            tc::mbar_init(empty_bar(s), 8);
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    tc::pdl_wait();  // the list and z come from the kernels before
    const int total = min(*ws.list_count, F);
    // parts are whole 16-position blocks, so that a part's z blocks are the ones the up kernel wrote
    const int blocks_total = (total + 15) >> 4;
    const int per_blocks = min(kMaxPart / 16, (blocks_total + (int)gridDim.y - 1) / (int)gridDim.y);
    const int b0 = min(blocks_total, (int)blockIdx.y * per_blocks);
    const int nblocks = min(per_blocks, blocks_total - b0);
    const int p0 = b0 * 16;
    const int count = min(nblocks * 16, total - p0);
    for (int i = tid; i < count; i += kGemvThreads) lch[i] = ws.list[p0 + i];
    // z blocks of this part: nblocks x 512 bytes, contiguous
    for (int i = tid; i < nblocks * 32; i += kGemvThreads)
        reinterpret_cast<uint4 *>(zl)[i] = reinterpret_cast<const uint4 *>(ws.Zb + (int64_t)b0 * 256)[i];
    __syncthreads();
    // positions past the end of the list were never written by the up kernel: they must count as zero
    if (nblocks > 0 && count < nblocks * 16) {
        for (int i = tid; i < 256; i += kGemvThreads)
            if ((nblocks - 1) * 16 + (i & 15) >= count) zl[(nblocks - 1) * 256 + i] = __float2bfloat16_rn(0.f);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();

    if (warp == 8) {
        // ------------------------------------------------------------------ producer: 16 rows per stage
        int stage = 0;
        uint32_t phase = 0;
        for (int blk = 0; blk < nblocks; ++blk) {
            if (!__all_sync(0xffffffffu, tc::mbar_wait(empty_bar(stage), phase ^ 1u, &s_abort, status))) break;
            const int p = blk * 16 + lane;
            const bool valid = lane < 16 && p < count;
            const int nvalid = min(16, count - blk * 16);
            if (lane == 0) tc::mbar_expect_tx(full_bar(stage), row_bytes * (uint32_t)nvalid);
            __syncwarp();
            if (valid)
                bulk_copy_g2s(tc::smem_u32(ring + stage * kDownStageBytes + lane * kDownPitch),
                              wd + (int64_t)lch[p] * d + c0, row_bytes, full_bar(stage));
            if (++stage == kDownStages) {
                stage = 0;
                phase ^= 1u;
            }
        }
    } else {
        // ------------------------------------------------------------------ consumers: warp w owns columns 64w..64w+63
        const int g = lane >> 2, q = lane & 3;
        float acc[8][4];
#pragma unroll
        for (int nb = 0; nb < 8; ++nb)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[nb][e] = 0.f;
        int stage = 0;
        uint32_t phase = 0;
        for (int blk = 0; blk < nblocks; ++blk) {
            // A fragment: z[t][position] of this block (tokens g and g+8, positions 2q.. and 2q+8..)
            const uint32_t *zb = reinterpret_cast<const uint32_t *>(zl + blk * 256);
            const uint32_t a0 = zb[g * 8 + q], a1 = zb[(g + 8) * 8 + q];
            const uint32_t a2 = zb[g * 8 + 4 + q], a3 = zb[(g + 8) * 8 + 4 + q];
            if (!__all_sync(0xffffffffu, tc::mbar_wait(full_bar(stage), phase, &s_abort, status))) break;
            // ldmatrix.x4.trans: lanes 0..15 address rows k = 0..15 at this column pair's first tile,
            // lanes 16..31 the same rows 8 columns further: one instruction yields two n-tiles
            const uint32_t base = tc::smem_u32(ring + stage * kDownStageBytes) + (uint32_t)(lane & 15) * kDownPitch +
                                  (uint32_t)(warp * 128 + (lane >> 4) * 16);
#pragma unroll
            for (int pr = 0; pr < 4; ++pr) {
                uint32_t b0r, b1r, b2r, b3r;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                             : "=r"(b0r), "=r"(b1r), "=r"(b2r), "=r"(b3r)
                             : "r"(base + pr * 32));
                mma_bf16_16816(acc[2 * pr], a0, a1, a2, a3, b0r, b1r);
                mma_bf16_16816(acc[2 * pr + 1], a0, a1, a2, a3, b2r, b3r);
            }
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(empty_bar(stage));
            if (++stage == kDownStages) {
                stage = 0;
                phase ^= 1u;
            }
        }
        // add this CTA's partial sums.  A lane holds columns 64 warp + 8 nb + 2q, +1 of tokens g and g + 8; lanes q
        // and q ^ 1 swap halves so that an even lane owns four consecutive columns of token g and an odd lane of
        // token g + 8: one 16-byte vector reduction each instead of four scalar ones
        if (nblocks > 0) {
            const bool odd = q & 1;
            const int tok = odd ? g + 8 : g;
#pragma unroll
            for (int nb = 0; nb < 8; ++nb) {
                const float s0 = odd ? acc[nb][0] : acc[nb][2], s1 = odd ? acc[nb][1] : acc[nb][3];
                const float r0v = __shfl_xor_sync(0xffffffffu, s0, 1), r1v = __shfl_xor_sync(0xffffffffu, s1, 1);
                const float k0 = odd ? acc[nb][2] : acc[nb][0], k1 = odd ? acc[nb][3] : acc[nb][1];
                // even lane: (own, partner's) = columns c .. c+3; odd lane: (partner's, own) = columns c-2 .. c+1
                const float v0 = odd ? r0v : k0, v1 = odd ? r1v : k1, v2 = odd ? k0 : r0v, v3 = odd ? k1 : r1v;
                const int c = warp * 64 + nb * 8 + 2 * (q & ~1);
                if (tok < T) {
                    float *dst = ws.out_acc + (int64_t)tok * d + c0 + c;
                    if (c + 3 < cols) {
                        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(v0), "f"(v1), "f"(v2),
                                     "f"(v3)
                                     : "memory");
                    } else {
                        if (c < cols) atomicAdd(dst, v0);
                        if (c + 1 < cols) atomicAdd(dst + 1, v1);
                        if (c + 2 < cols) atomicAdd(dst + 2, v2);
                        if (c + 3 < cols) atomicAdd(dst + 3, v3);
                    }
                }
            }
        }
    }
    __syncwarp();
    if (s_abort) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    // the last CTA of the slice converts the totals to bf16
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(&ws.counters[slice], 1) == (int)gridDim.y - 1;
    __syncthreads();
    if (s_last) {
        __threadfence();
        for (int i = tid; i < T * (cols >> 1); i += kGemvThreads) {
            const int t = i / (cols >> 1), c = (i % (cols >> 1)) * 2;
            const float *a = ws.out_acc + (int64_t)t * d + c0 + c;
            float v0 = __ldcg(a), v1 = __ldcg(a + 1);
            if (resid) {  // the residual connection of the block form: out = h + D (out may be h itself)
                const __nv_bfloat162 h2 = *reinterpret_cast<const __nv_bfloat162 *>(resid + (int64_t)t * d + c0 + c);
                v0 += __low2float(h2);
                v1 += __high2float(h2);
            }
            *reinterpret_cast<__nv_bfloat162 *>(out + (int64_t)t * d + c0 + c) = __floats2bfloat162_rn(v0, v1);
        }
    }
}

// RMSNorm of the residual stream in front of the layer (Section 2, "RMSNorm"): y = h / sqrt(mean(h^2) + eps) . weight
// for one token, rounded to bf16 (the layer's input type), by the first 256 threads of a CTA (all of its threads call:
// there is a block-wide barrier inside).  s_part: 8 floats of shared memory.
__device__ __forceinline__ void rmsnorm_row(const __nv_bfloat16 *__restrict__ row, const __nv_bfloat16 *__restrict__ weight,
                                            float eps, int d, __nv_bfloat16 *__restrict__ y, float *s_part) {
    const int tid = threadIdx.x;
    float ss = 0.f;
    if (tid < 256) {
        for (int i = tid * 8; i < d; i += 256 * 8) {  // d is a multiple of 8
            float v[8];
            Vec8<__nv_bfloat16>::load(row + i, v);
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(v[e], v[e], ss);
        }
        ss = warp_sum(ss);
        if ((tid & 31) == 0) s_part[tid >> 5] = ss;
    }
    __syncthreads();
    if (tid < 256) {
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) tot += s_part[w];
        const float scale = rsqrtf(tot / (float)d + eps);
        for (int i = tid * 8; i < d; i += 256 * 8) {
            float v[8], g[8];
            Vec8<__nv_bfloat16>::load(row + i, v);
            Vec8<__nv_bfloat16>::load(weight + i, g);
            uint32_t w4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) w4[e] = tc::pack_bf16(v[2 * e] * scale * g[2 * e], v[2 * e + 1] * scale * g[2 * e + 1]);
            *reinterpret_cast<uint4 *>(y + i) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
    }
}

// One CTA per token.
__global__ void __launch_bounds__(256) rmsnorm_rows_kernel(const __nv_bfloat16 *__restrict__ h,
                                                           const __nv_bfloat16 *__restrict__ weight, float eps, int d,
                                                           __nv_bfloat16 *__restrict__ y) {
    __shared__ float s_part[8];
    const int t = blockIdx.x;
    tc::pdl_launch_dependents();
    // waits although h is an input of the call: the kernels after this one wait for THIS kernel only, and rely on
    // everything before it in the stream being over when it is
    tc::pdl_wait();
    rmsnorm_row(h + (int64_t)t * d, weight, eps, d, y + (int64_t)t * d, s_part);
}


// ---------------------------------------------------------------------------------------------- stream probe
// A bare streaming read (diagnostics): up to three byte ranges are read once, in 8 KiB bulk copies through a ring of
// kProbeStages stages per CTA, two CTAs per SM, nothing computed: the time below which no schedule that has to read those
// bytes from HBM can finish.  The ranges are split evenly over the CTAs.
constexpr int kProbeStages = 11, kProbeChunk = 8192, kProbeThreads = 64;
struct ProbeRanges {
    const uint8_t *base[3];
    unsigned long long bytes[3];  // multiples of 16
};
__global__ void __launch_bounds__(kProbeThreads, 2) stream_probe_kernel(const ProbeRanges r, int *__restrict__ status) {
    extern __shared__ __align__(128) uint8_t dsm[];
    __shared__ uint64_t bars[2 * kProbeStages];
    __shared__ int s_abort;
    const int tid = threadIdx.x;
    auto full_bar = [&](int s) { return tc::smem_u32(&bars[s]); };
    auto empty_bar = [&](int s) { return tc::smem_u32(&bars[kProbeStages + s]); };
    if (tid == 0) {
        for (int s = 0; s < kProbeStages; ++s) {
            tc::mbar_init(full_bar(s), 1);
            tc::mbar_init(empty_bar(s), 1);
        }
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    tc::pdl_launch_dependents();
    // this CTA's share of every range, in chunks
    if (tid == 0) {  // producer
        int stage = 0;
        uint32_t phase = 0;
        for (int i = 0; i < 3; ++i) {
            const unsigned long long chunks = (r.bytes[i] + kProbeChunk - 1) / kProbeChunk;
            const unsigned long long c0 = chunks * blockIdx.x / gridDim.x, c1 = chunks * (blockIdx.x + 1) / gridDim.x;
            for (unsigned long long c = c0; c < c1; ++c) {
                if (!tc::mbar_wait(empty_bar(stage), phase ^ 1u, &s_abort, status)) return;
                const unsigned long long off = c * kProbeChunk;
                const uint32_t n = (uint32_t)min((unsigned long long)kProbeChunk, r.bytes[i] - off);
                tc::mbar_expect_tx(full_bar(stage), n);
                bulk_copy_g2s(tc::smem_u32(dsm + stage * kProbeChunk), r.base[i] + off, n, full_bar(stage));
                if (++stage == kProbeStages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
        }
    } else if (tid == 32) {  // consumer: hands every stage straight back
        int stage = 0;
        uint32_t phase = 0;
        for (int i = 0; i < 3; ++i) {
            const unsigned long long chunks = (r.bytes[i] + kProbeChunk - 1) / kProbeChunk;
            const unsigned long long c0 = chunks * blockIdx.x / gridDim.x, c1 = chunks * (blockIdx.x + 1) / gridDim.x;
            for (unsigned long long c = c0; c < c1; ++c) {
                if (!tc::mbar_wait(full_bar(stage), phase, &s_abort, status)) return;
                tc::mbar_arrive(empty_bar(stage));
                if (++stage == kProbeStages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
        }
    }
}

}  // namespace dec
}  // namespace moc
