// Decode for one or two tokens as ONE cooperative kernel (bf16, d_model <= 4096).
//
// The four-kernel decode plan reads the right bytes (Section 5: the gate matrix once, then only the selected rows of
// W_up and W_down) but spends two thirds of its time on the hand-overs between kernels.  Here every SM keeps a fixed
// share of the CHANNELS for the whole call, so that nothing but a few words per token has to cross between SMs:
//
//   phase 1   the CTA streams its channels' rows of W_gate and keeps their gate values g[t][j] in shared memory
//             (Eq. (Moc-1)); it adds them to a global 2048-bin histogram of the order-preserving keys
//   select    grid barrier; every CTA scans the histogram for the bin that holds the K-th largest key, appends its
//             own keys of that bin (with their channels) to a global list; grid barrier; every CTA ranks its own
//             candidates against the list: a channel is kept when fewer than K channels precede it in
//             (value descending, channel ascending) order -- the mask definition of Section 3.2 with the tie rule
//             of the library, decided without any single SM ever seeing the whole row
//   phase 3   the CTA streams the rows of W_up and W_down of ITS kept channels only, forms z = SiLU(g) u (Eq. (MoC-2))
//             and its partial output, adds it to a global fp32 accumulator; grid barrier; the CTAs round slices of
//             the accumulator to bf16.
//
// Grid barriers are cooperative-groups grid syncs (the launch is cooperative: all CTAs are resident, or the launch
// fails).  No CTA ever leaves before the last barrier: a bounded wait that runs out raises MOC_ERR_TIMEOUT, stops the
// CTA's streaming, and the CTA still walks through every barrier.
#pragma once

#include <cooperative_groups.h>

#include "grouped_select.cuh"
#include "moc_common.cuh"
#include "tc_gemm.cuh"

namespace moc {
namespace dc {


constexpr int kMaxTokens = 2;         // the dot products are plain FMAs: beyond two tokens the four-kernel plan's MMAs win
constexpr int kMaxD = 4096;          // a thread owns 8 output columns
constexpr int kConsumerWarps = 16;
constexpr int kThreads = (kConsumerWarps + 1) * 32;  // + one producer warp
constexpr int kMaxRows = 256;        // channels per CTA
constexpr int kBins = 2048;          // top 11 bits of the key
constexpr int kMaxStages = 32;         // a multiple of kConsumerWarps
constexpr int kFirstRows = 8;  // gate rows requested before x is staged and the shared arrays are cleared (16 or 32 of them
                               // made that start-up 0.9 us longer and the call 1 us slower: they compete with it for the path from L2)

struct Params {
    const __nv_bfloat16 *x, *wg, *wu, *wd;
    __nv_bfloat16 *out;
    int T, d, F, K, grouped;
    int unit;            // channels are dealt to the CTAs in units of this many (8 when F % 8 == 0, else 1)
    int stages;          // ring stages of one weight row each
    // workspace
    uint32_t *hist;      // [T][kBins]
    uint32_t *cand_n;    // [T]
    uint2 *cand;         // [T][F]  (key, channel)
    float *acc;          // [T][d]
    int *status;
    // the block form (Section 2, "LLM structure"): x holds the residual stream h, the layer reads RMSNorm(h) with
    // weight rms_w and adds h to its output; rms_w == nullptr: the plain layer on x
    const __nv_bfloat16 *rms_w;
    float rms_eps;
    // test hook: when not null, [T][F] bytes that receive 1 for every channel a token keeps and 0 for the others
    uint8_t *kept_out;
};

inline size_t smem_bytes(int T, int d, int stages) {
    // x [T][d] bf16 | ring [stages][d] bf16 | g [T][kMaxRows] f32 | z [T][kMaxRows] f32
    return (size_t)T * d * 2 + (size_t)stages * d * 2 + (size_t)2 * T * kMaxRows * 4;
}

template <int T>
__global__ void __launch_bounds__(kThreads, 1) decode_coop_kernel(const Params p) {
    namespace cg = cooperative_groups;
    cg::grid_group grid = cg::this_grid();
    extern __shared__ __align__(128) uint8_t dsm[];
    __shared__ uint64_t bars[2 * kMaxStages];
    __shared__ int s_abort;
    __shared__ uint32_t s_scan[kConsumerWarps];
    __shared__ uint32_t s_bin[T], s_above[T];
    __shared__ uint16_t s_list[kMaxRows];   // the CTA's kept channels (offsets in its range), kept by any token
    __shared__ __align__(4) uint8_t s_mask[kMaxRows];  // per channel of the range: which tokens keep it (bit t)
    __shared__ int s_nsel;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool producer = warp == kConsumerWarps;
    MOC_TL_CTA(256);
    const int d = p.d, F = p.F;
    __nv_bfloat16 *sx = reinterpret_cast<__nv_bfloat16 *>(dsm);
    uint8_t *ring = dsm + (size_t)T * d * 2;
    float *sg = reinterpret_cast<float *>(ring + (size_t)p.stages * d * 2);
    float *sz = sg + T * kMaxRows;
    const uint32_t row_bytes = (uint32_t)d * 2u;
    auto full_bar = [&](int s) { return tc::smem_u32(&bars[s]); };
    auto empty_bar = [&](int s) { return tc::smem_u32(&bars[kMaxStages + s]); };
    auto consumer_sync = [&]() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory"); };

    // the CTA's channels: units [u0, u1) of `unit` channels each
    const int units = (F + p.unit - 1) / p.unit;
    const int u0 = (int)(((int64_t)blockIdx.x * units) / gridDim.x);
    const int u1 = (int)(((int64_t)(blockIdx.x + 1) * units) / gridDim.x);
    const int c0 = u0 * p.unit, c1 = min(F, u1 * p.unit);
    const int rows = max(0, c1 - c0);  // <= kMaxRows (the host checks)

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            tc::mbar_init(full_bar(s), 1);
            tc::mbar_init(empty_bar(s), kConsumerWarps);
        }
        s_abort = 0;
        s_nsel = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // ---- ring: the producer lane issues one bulk copy per weight row; rows are consumed in the order issued
    int p_stage = 0, c_stage = 0;
    uint32_t p_phase = 0, c_phase = 0;
    auto produce_row = [&](const __nv_bfloat16 *w, int row) -> bool {  // producer lane only
        if (!tc::mbar_wait(empty_bar(p_stage), p_phase ^ 1u, &s_abort, p.status)) return false;
        tc::mbar_expect_tx(full_bar(p_stage), row_bytes);
        tc::bulk_copy_g2s(tc::smem_u32(ring + (size_t)p_stage * row_bytes), w + (int64_t)row * d, row_bytes,
                          full_bar(p_stage));
        if (++p_stage == p.stages) {
            p_stage = 0;
            p_phase ^= 1u;
        }
        return true;
    };
    auto advance = [&]() {
        if (++c_stage == p.stages) {
            c_stage = 0;
            c_phase ^= 1u;
        }
    };
    auto release = [&](uint32_t count) {  // the calling lane frees the current stage on behalf of `count` warps
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(empty_bar(c_stage)), "r"(count) : "memory");
    };
    // A parity test only tells an odd from an even number of completed rounds of a stage, so a warp must see every round
    // of the stages it waits on (a stage two rounds behind would pass the test for the current round at once).  The
    // number of stages is therefore a multiple of the number of consumer warps: row r goes to stage r mod stages and to
    // warp r mod 16, so a stage is always consumed by the same warp.  (In the last phase every warp sees every row.)
    auto wait_row = [&](int) -> bool { return tc::mbar_wait(full_bar(c_stage), c_phase, &s_abort, p.status); };
    // dot products of one staged row with the T tokens, by one warp (every lane gets the sums)
    auto row_dots = [&](const uint8_t *row, float (&sum)[T]) {
#pragma unroll
        for (int t = 0; t < T; ++t) sum[t] = 0.f;
        for (int c = lane * 8; c < d; c += 256) {
            float w8[8];
            Vec8<__nv_bfloat16>::load(reinterpret_cast<const __nv_bfloat16 *>(row) + c, w8);
#pragma unroll
            for (int t = 0; t < T; ++t) {
                float x8[8];
                Vec8<__nv_bfloat16>::load(sx + (size_t)t * d + c, x8);
#pragma unroll
                for (int e = 0; e < 8; ++e) sum[t] = fmaf(w8[e], x8[e], sum[t]);
            }
        }
#pragma unroll
        for (int t = 0; t < T; ++t) sum[t] = warp_sum(sum[t]);
    };

    // ---- start: the first gate rows leave at once (the ring is empty: nothing to wait for); x is staged and the
    //      CTA clears its slices of the arrays all CTAs share
    const int first = min(min(p.stages, kFirstRows), rows);  // (the producer lane joins the barrier below: it must not be late)
    if (producer && lane == 0)
        for (int i = 0; i < first; ++i) produce_row(p.wg, c0 + i);
    {
        for (int i = tid * 8; i < T * d; i += kThreads * 8)
            *reinterpret_cast<uint4 *>(sx + i) = *reinterpret_cast<const uint4 *>(p.x + i);
        if (p.rms_w) {
            // RMSNorm of the staged rows, in place: y = h / sqrt(mean(h^2) + eps) . weight, rounded to bf16 as the
            // layer's input (every CTA normalises all T rows: 2 d values)
            __syncthreads();
            float ss[T];
#pragma unroll
            for (int t = 0; t < T; ++t) {
                ss[t] = 0.f;
                for (int i = tid; i < d; i += kThreads) {
                    const float v = __bfloat162float(sx[t * d + i]);
                    ss[t] = fmaf(v, v, ss[t]);
                }
                ss[t] = warp_sum(ss[t]);
            }
            if (lane == 0)
#pragma unroll
                for (int t = 0; t < T; ++t) sz[t * kMaxRows + warp] = ss[t];  // (z is not in use yet)
            __syncthreads();
#pragma unroll
            for (int t = 0; t < T; ++t) {
                float tot = 0.f;
                for (int w = 0; w < kThreads / 32; ++w) tot += sz[t * kMaxRows + w];
                const float scale = rsqrtf(tot / (float)d + p.rms_eps);
                for (int i = tid; i < d; i += kThreads)
                    sx[t * d + i] = __float2bfloat16_rn(__bfloat162float(sx[t * d + i]) * scale * __bfloat162float(p.rms_w[i]));
            }
        }
        for (int i = tid; i < kMaxRows; i += kThreads) s_mask[i] = 0;
        const int nthr = (int)gridDim.x * kThreads, gtid = (int)blockIdx.x * kThreads + tid;
        for (int i = gtid; i < T * kBins; i += nthr) p.hist[i] = 0u;
        for (int i = gtid; i < T; i += nthr) p.cand_n[i] = 0u;
        for (int i = gtid; i < T * d; i += nthr) p.acc[i] = 0.f;
    }
    // #0, split: the CTA announces that its slices are clear now and waits for the others only when it is about to
    // touch the shared arrays, after phase 1 (the arrival is a block-wide barrier too: x is staged)
    auto clear_token = grid.barrier_arrive();
    MOC_TL_CTA(512);

    // ---- phase 1: gate values of the CTA's channels (one warp per row), histogram of their keys
    if (producer) {
        if (lane == 0)
            for (int i = first; i < rows; ++i)
                if (!produce_row(p.wg, c0 + i)) break;
    } else {
        for (int r = 0; r < rows; ++r) {
            if (r % kConsumerWarps == warp) {
                const bool ok = __all_sync(0xffffffffu, wait_row(r));
                float sum[T];
                if (ok) row_dots(ring + (size_t)c_stage * row_bytes, sum);
                __syncwarp();
                if (lane == 0) {
                    release(kConsumerWarps);
#pragma unroll
                    for (int t = 0; t < T; ++t) sg[t * kMaxRows + r] = ok ? sum[t] : 0.f;
                }
            }
            advance();
        }
    }
    __syncthreads();
    grid.barrier_wait(std::move(clear_token));  // every CTA's slices of the shared arrays are clear
    MOC_TL_CTA(768);

    // ---- selection
    if (!p.grouped) {
        for (int i = tid; i < T * rows; i += kThreads) {
            const int t = i / rows, r = i - t * rows;
            atomicAdd(&p.hist[t * kBins + (gate_key(sg[t * kMaxRows + r]) >> 21)], 1u);
        }
        grid.sync();  // #1 (the barrier's release / acquire pair orders the CTAs' writes before the others' reads): every CTA's keys are in the histogram
        MOC_TL_CTA(1024);
        // the bin of the K-th largest key and the number of keys above that bin, per token (suffix sums over 2048 bins:
        // four bins per consumer thread)
        for (int t = 0; t < T; ++t) {
            uint32_t h[4] = {0u, 0u, 0u, 0u}, s = 0u;
            if (!producer) {
#pragma unroll
                for (int i = 0; i < 4; ++i) h[i] = __ldcg(&p.hist[t * kBins + 4 * tid + i]);
                s = h[0] + h[1] + h[2] + h[3];
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t v = __shfl_down_sync(0xffffffffu, s, o);
                    if (lane + o < 32) s += v;
                }
                if (lane == 0) s_scan[warp] = s;
            }
            __syncthreads();
            if (!producer) {
                uint32_t after = 0u;
                for (int w = warp + 1; w < kConsumerWarps; ++w) after += s_scan[w];
                s += after;  // keys in this thread's bins and all higher ones
                uint32_t above = s - (h[0] + h[1] + h[2] + h[3]);  // keys in strictly higher bins than this thread's
#pragma unroll
                for (int i = 3; i >= 0; --i) {
                    if (above < (uint32_t)p.K && above + h[i] >= (uint32_t)p.K) {
                        s_bin[t] = (uint32_t)(4 * tid + i);
                        s_above[t] = above;
                    }
                    above += h[i];
                }
            }
            __syncthreads();
        }
        // the CTA's keys of that bin join the global candidate list
        for (int i = tid; i < T * rows; i += kThreads) {
            const int t = i / rows, r = i - t * rows;
            const uint32_t key = gate_key(sg[t * kMaxRows + r]);
            if ((key >> 21) == s_bin[t]) {
                const uint32_t pos = atomicAdd(&p.cand_n[t], 1u);
                p.cand[(int64_t)t * F + pos] = make_uint2(key, (uint32_t)(c0 + r));
            }
        }
        grid.sync();  // #2: the candidate lists are complete
        MOC_TL_CTA(1280);
        // rank the CTA's own candidates: one warp per candidate, the lanes share the list -- which is first copied to
        // shared memory (the ring is idle between the phases) when it fits, so that the ranking loops do not pay a
        // trip to L2 per step
        uint32_t n_of[T], off_of[T], total = 0;
#pragma unroll
        for (int t = 0; t < T; ++t) {
            n_of[t] = min(__ldcg(&p.cand_n[t]), (uint32_t)F);
            off_of[t] = total;
            total += n_of[t];
        }
        uint2 *scand = reinterpret_cast<uint2 *>(ring);
        const bool staged = (size_t)total * sizeof(uint2) <= (size_t)p.stages * row_bytes;
        if (staged) {
#pragma unroll
            for (int t = 0; t < T; ++t)
                for (uint32_t j = tid; j < n_of[t]; j += kThreads) scand[off_of[t] + j] = __ldcg(&p.cand[(int64_t)t * F + j]);
        }
        __syncthreads();
        for (int i = warp; i < T * rows; i += kConsumerWarps + 1) {
            const int t = i / rows, r = i - t * rows;
            const uint32_t key = gate_key(sg[t * kMaxRows + r]);
            const uint32_t bin = key >> 21;
            bool kept = bin > s_bin[t];
            if (bin == s_bin[t]) {
                uint32_t nt = 0, ot = 0;
#pragma unroll
                for (int tt = 0; tt < T; ++tt)
                    if (tt == t) {
                        nt = n_of[tt];
                        ot = off_of[tt];
                    }
                const uint32_t ch = (uint32_t)(c0 + r);
                uint32_t before = 0;
                for (uint32_t j = lane; j < nt; j += 32) {
                    const uint2 o = staged ? scand[ot + j] : __ldcg(&p.cand[(int64_t)t * F + j]);
                    before += (o.x > key || (o.x == key && o.y < ch)) ? 1u : 0u;
                }
                before = __reduce_add_sync(0xffffffffu, before);
                kept = s_above[t] + before < (uint32_t)p.K;
            }
            if (kept && lane == 0) atomicOr(reinterpret_cast<unsigned int *>(s_mask) + (r >> 2), (1u << t) << (8 * (r & 3)));
        }
        __syncthreads();  // the ring is the producer's again
    } else {
        // MoC 2:8 (Section 4): the CTA's range is made of whole groups of eight channels; the mask is local
        for (int i = tid; i < T * (rows >> 3); i += kThreads) {
            const int t = i / (rows >> 3), q = i - t * (rows >> 3);
            uint32_t key[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) key[e] = gate_key(sg[t * kMaxRows + 8 * q + e]);
            int lo, hi;
            top2_of_8(key, lo, hi);
            atomicOr(reinterpret_cast<unsigned int *>(s_mask) + ((8 * q + lo) >> 2), (1u << t) << (8 * ((8 * q + lo) & 3)));
            atomicOr(reinterpret_cast<unsigned int *>(s_mask) + ((8 * q + hi) >> 2), (1u << t) << (8 * ((8 * q + hi) & 3)));
        }
    }
    __syncthreads();
    if (p.kept_out)
        for (int i = tid; i < T * rows; i += kThreads) {
            const int t = i / rows, r = i - t * rows;
            p.kept_out[(int64_t)t * F + c0 + r] = (uint8_t)((s_mask[r] >> t) & 1);
        }
    if (warp == 0) {  // the kept channels in ascending order
        int n = 0;
        for (int base = 0; base < rows; base += 32) {
            const int r = base + lane;
            const bool f = r < rows && s_mask[r] != 0;
            const uint32_t b = __ballot_sync(0xffffffffu, f);
            if (f) s_list[n + __popc(b & ((1u << lane) - 1u))] = (uint16_t)r;
            n += __popc(b);
        }
        if (lane == 0) s_nsel = n;
    }
    __syncthreads();
    const int nsel = s_nsel;
    MOC_TL_CTA(1536);

    // ---- phase 3: up rows (one warp per row: u, z = SiLU(g) u), then down rows (every thread owns 8 columns)
    float acc[T][8];
#pragma unroll
    for (int t = 0; t < T; ++t)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[t][e] = 0.f;
    if (producer) {
        if (lane == 0) {
            bool ok = true;
            for (int i = 0; i < nsel && ok; ++i) ok = produce_row(p.wu, c0 + s_list[i]);
            for (int i = 0; i < nsel && ok; ++i) ok = produce_row(p.wd, c0 + s_list[i]);
        }
    } else {
        for (int i = 0; i < nsel; ++i) {
            if (i % kConsumerWarps == warp) {
                const bool ok = __all_sync(0xffffffffu, wait_row(rows + i));
                float sum[T];
                if (ok) row_dots(ring + (size_t)c_stage * row_bytes, sum);
                __syncwarp();
                if (lane == 0) {
                    release(kConsumerWarps);
                    const int r = s_list[i];
#pragma unroll
                    for (int t = 0; t < T; ++t)
                        sz[t * kMaxRows + i] = (ok && ((s_mask[r] >> t) & 1)) ? silu_f(sg[t * kMaxRows + r]) * sum[t] : 0.f;
                }
            }
            advance();
        }
        consumer_sync();  // every z is in shared memory
        const int col = tid * 8;
        for (int i = 0; i < nsel; ++i) {
            const bool ok = __all_sync(0xffffffffu, tc::mbar_wait(full_bar(c_stage), c_phase, &s_abort, p.status));
            if (ok && col < d) {
                float w8[8];
                Vec8<__nv_bfloat16>::load(reinterpret_cast<const __nv_bfloat16 *>(ring + (size_t)c_stage * row_bytes) + col, w8);
#pragma unroll
                for (int t = 0; t < T; ++t) {
                    const float z = sz[t * kMaxRows + i];
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[t][e] = fmaf(z, w8[e], acc[t][e]);
                }
            }
            __syncwarp();
            if (lane == 0) release(1u);
            advance();
        }
        if (col < d && nsel > 0) {
#pragma unroll
            for (int t = 0; t < T; ++t) {
                float *dst = p.acc + (int64_t)t * d + col;
                asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(acc[t][0]), "f"(acc[t][1]),
                             "f"(acc[t][2]), "f"(acc[t][3])
                             : "memory");
                asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + 4), "f"(acc[t][4]), "f"(acc[t][5]),
                             "f"(acc[t][6]), "f"(acc[t][7])
                             : "memory");
            }
        }
    }
    __syncthreads();
    MOC_TL_CTA(1792);
    grid.sync();  // #3: every CTA's partial output is in the accumulator
    MOC_TL_CTA(2048);

    // ---- out = bf16(accumulator), a slice per CTA
    {
        const int vecs = T * d / 8;
        for (int v = (int)blockIdx.x * kThreads + tid; v < vecs; v += (int)gridDim.x * kThreads) {
            float4 a = __ldcg(reinterpret_cast<const float4 *>(p.acc) + 2 * v);
            float4 b = __ldcg(reinterpret_cast<const float4 *>(p.acc) + 2 * v + 1);
            if (p.rms_w) {  // the residual connection: out = h + D
                float h8[8];
                Vec8<__nv_bfloat16>::load(p.x + (size_t)v * 8, h8);
                a.x += h8[0], a.y += h8[1], a.z += h8[2], a.w += h8[3];
                b.x += h8[4], b.y += h8[5], b.z += h8[6], b.w += h8[7];
            }
            reinterpret_cast<uint4 *>(p.out)[v] =
                make_uint4(tc::pack_bf16(a.x, a.y), tc::pack_bf16(a.z, a.w), tc::pack_bf16(b.x, b.y), tc::pack_bf16(b.z, b.w));
        }
    }
    MOC_TL_CTA(2304);
    if (s_abort) {  // copies still in flight must land before shared memory goes away
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
}

}  // namespace dc
}  // namespace moc
