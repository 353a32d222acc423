// Small-batch forward (bf16, up to 32 tokens, nothing saved) as ONE cooperative kernel.
//
// The kernels of small_batch.cuh each stream one or two weight matrices; every kernel boundary costs a hand-over, a
// cold start of the next kernel's ring and an epilogue during which HBM idles -- about a third of the call at 16
// tokens.  Here the grid is one CTA per SM for the whole call.  T of the CTAs are selectors (one token each, the
// CTA-per-row selector of the decode plan); every other CTA is a streamer whose ring of shared-memory stages never
// drains:
//
//   phase G   stream the CTA's channels' rows of W_gate  -> fp32 gate values (Eq. (Moc-1)) to the workspace and to
//             shared memory; count the CTA in flags[0]
//   (select)  the selector CTAs wait for flags[0], find their token's Top-K set (Section 3.2), leave it as a bitmap
//             and count themselves in flags[1] -- while the streamers are in
//   phase U   stream the same channels' rows of W_up     -> accumulators; once flags[1] is complete, form
//             Z' = SiLU(g) u on the kept channels (Eq. (MoC-2)) and store it; count the CTA in flags[2]
//   phase D   stream the CTA's share of W_down (its weight boxes are requested while phases G and U still compute, the
//             Z' boxes once flags[2] says every CTA's Z' is written) -> partial sums, added to an fp32 accumulator; the
//             last CTA of a column block rounds to bf16
//
// Two warps issue the MMAs, stage about: with 16 or 32 tokens an MMA is short (some 45 cycles), and the instruction that
// hands a stage back once its MMAs have read it (tcgen05.commit) stalls the issuing thread for some 450 cycles -- as long
// as a whole stage's MMAs.  The stall is the thread's, not the tensor core's: a second issuer fills it.  Each issuer
// accumulates into its own tensor-memory columns.
//
// CTAs wait on one another, so the launch is cooperative: all CTAs are resident, or the launch fails.  Every wait is
// bounded as everywhere else in the library.
//
// The flags and the column blocks' counters live in a block of the library's own device memory (one per workspace
// address; the caller's workspace is the caller's between calls).  A run that completes leaves them zero and writes a
// 64-bit mark behind them; a run that finds the mark starts at once (and removes it as soon as every CTA has read it,
// so that a run that does not complete leaves no mark).  A run that finds no mark -- the first one, or the one after a
// run that gave up on a wait -- has CTA 0 zero the block and publishes that with a grid barrier, some 4 us during
// which only the first ring of requests is in flight.
#pragma once

#include <cooperative_groups.h>

#include "small_batch.cuh"

namespace moc {
namespace sbf {

using sb::kBK;
using sb::kTile;

constexpr int kBlock = dec::kSelThreads;  // the selector's block size; a streamer CTA uses its first eleven warps:
                                          // warp 0 TMA, warps 1 and 2 MMA, warps 3..10 epilogue (two per TMEM lane quarter)
constexpr int kEpiWarps = 8;
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kMaxTokens = 32;            // one 32-token accumulator chunk
constexpr int kTn = 32;                   // columns of tensor memory per accumulator (MMA N is 16 or 32)
constexpr int kStagesMax = 8;
constexpr int kStateCounters = 112;        // counters of the column blocks; the flags follow them in the state block
constexpr unsigned long long kCleanMark = 0x6d6f632d66757365ull;  // "the flags and counters of this workspace are zero"
// Tensor memory: every MMA issuer has its own accumulators (the epilogue adds them).  32 columns per tile;
// issuer w: gate tiles at 64 w (+32), up tiles at 128 + 64 w (+32), down accumulators at 256 + 64 w (+32).
constexpr uint32_t kTmemCols = 512;

struct FusedParams {
    CUtensorMap wg_map, wu_map;  // [F, d]: boxes of `rows` channels x 64
    CUtensorMap x_map;           // [T, d]: boxes of tn tokens x 64 (rows >= T read as zero)
    CUtensorMap wd_map;          // [F, d]: boxes of 64 columns x 64 channels (the M-major operand of the down projection)
    CUtensorMap z_map;           // Z' [T, F]: boxes of tn tokens x 64 channels
    int T, F, K, d;
    int grouped;                 // MoC 2:8 (Section 4): the mask is local to groups of 8 channels -- no selector CTAs, the streamers'
                                 // epilogue picks the two largest of every group itself (rows is then a multiple of 8)
    int tn;                      // MMA N and rows of an activation box: 16 (up to 16 tokens) or 32
    int n_stream;                // streamer CTAs: blocks [0, n_stream); block n_stream + t selects for token t
    int n_gu;                    // streamers that own channels: ceil(F / rows)
    int rows;                    // channels per streamer in phases G and U (<= 256; a multiple of 8 beyond 128)
    uint32_t w_pitch;            // shared-memory bytes of one weight box of those phases: rows * 128 rounded up to 1024
    int gu_boxes;                // 64-element contraction blocks per stage of phases G and U
    int gu_stages;               // stages per matrix: ceil(d / (64 * gu_boxes))
    int accs, m_tiles, splits, kb_down;  // down projection: 128 * accs columns per CTA, CTAs (m, split), 64-channel blocks
    uint32_t slot_bytes;         // one ring slot (the larger of the two stage shapes)
    int stages;
    uint32_t tail_off;           // from the ring's base: gate values [32][rows] fp32 | barriers (the ring's over-read room)
    float *G;                    // [T, ldf]
    int ldf;
    uint32_t *kept_bits;         // [T, kept_words]
    int kept_words;
    __nv_bfloat16 *Z;            // [T, ldz]
    int ldz;
    float *acc;                  // [T, d] fp32
    __nv_bfloat16 *out;
    const __nv_bfloat16 *resid;  // the block form's residual, or nullptr
    // the block form with the normalisation inside the kernel (Top-K form only): the selector CTAs, idle until the gate
    // values exist, first write xn = RMSNorm(rms_h; rms_w, rms_eps) -- the array x_map reads -- a token each, and the
    // producers request activation boxes only once flags[5] counts all of them.  rms_w == nullptr: x is given.
    const __nv_bfloat16 *rms_h, *rms_w;
    __nv_bfloat16 *xn;
    float rms_eps;
    int *counters;               // [kStateCounters], of which m_tiles are used
    unsigned int *flags;         // [0] streamers done with G, [1] tokens selected, [2] streamers done with Z', [3] CTAs that
                                 // have read the mark, [4] CTAs that have finished, [5] tokens normalised, [6..7] the mark (8-byte aligned)
    int *status;
    long long wait_limit;        // cycles after which a wait gives up (tc::kWaitLimitCycles; shorter in the time-out test)
    int stall;                   // the time-out test: the selectors wait for this many streamers more than exist
};

// shared memory of the selector role: keys [Fp] | two candidate lists | the radix select's state
inline size_t selector_smem(int F) {
    const size_t Fp = (size_t)((F + 3) & ~3);
    return (Fp + 2 * dec::kSelListCap) * sizeof(uint32_t) + 16 + sizeof(SelectSmemT<kBlock / 32>);
}

__device__ __forceinline__ unsigned int ld_acquire(const unsigned int *p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Bounded wait until *flag >= target.  False: it gave up (MOC_ERR_TIMEOUT raised) or another role already had.
__device__ __forceinline__ bool flag_wait(const unsigned int *flag, unsigned int target, volatile int *abort_flag, int *status,
                                          long long limit_cycles) {
    if (ld_acquire(flag) >= target) return true;
    const long long t0 = clock64();
    while (ld_acquire(flag) < target) {
        __nanosleep(40);
        if (*abort_flag) return false;
        if (clock64() - t0 > limit_cycles) {
            *abort_flag = 1;
            raise_status(status, MOC_ERR_TIMEOUT);
            return false;
        }
    }
    return true;
}

// 16 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}
// sum of the two issuers' accumulators: 16 columns at `taddr` and at `taddr` + 64 (when the second issuer had work)
__device__ __forceinline__ void tmem_ld16_sum(uint32_t taddr, bool two, float (&v)[16]) {
    uint32_t a[16];
    tmem_ld16(taddr, a);
    tc::tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(a[i]);
    if (two) {  // (warp-uniform)
        tmem_ld16(taddr + 64u, a);
        tc::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] += __uint_as_float(a[i]);
    }
}
// An MMA whose descriptors are given as their low words (address and leading-dimension fields) and the high word both
// share: the issuing thread's instruction stream is what limits a run of short MMAs, so it is kept to two additions each.
__device__ __forceinline__ void umma_lohi(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %4, p;\n\t}"
        ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc), "r"(accumulate)
        : "memory");
}

// One thread of a CTA that has used the flags for the last time: the last CTA of the grid to get here zeroes them for
// the next run and leaves the mark.  (A CTA that gave up on a wait never gets here: no mark.)
__device__ __forceinline__ void cta_finished(const FusedParams &p) {
    __threadfence();
    if (atomicAdd(p.flags + 4, 1u) == gridDim.x - 1) {
#pragma unroll
        for (int i = 0; i < 6; ++i) p.flags[i] = 0u;
        __threadfence();
        *reinterpret_cast<volatile unsigned long long *>(p.flags + 6) = kCleanMark;
    }
}

// ------------------------------------------------------------------------------------------------ selector role
__device__ __forceinline__ void selector_role(const FusedParams &p, uint32_t *dyn) {
    __shared__ uint64_t s_bar;
    __shared__ int s_abort;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int t = (int)blockIdx.x - p.n_stream;
    const int Fp = (p.F + 3) & ~3;
    uint32_t *keys = dyn, *lists = dyn + Fp, *bits = lists;
    auto &sm = *reinterpret_cast<SelectSmemT<kBlock / 32> *>(
        (reinterpret_cast<uintptr_t>(lists + 2 * dec::kSelListCap) + 15) & ~(uintptr_t)15);
    if (p.rms_w) {  // the layer's input for this token: the streamers' first stages wait for it
        __shared__ float s_part[8];
        dec::rmsnorm_row(p.rms_h + (int64_t)t * p.d, p.rms_w, p.rms_eps, p.d, p.xn + (int64_t)t * p.d, s_part);
        __threadfence();
        __syncthreads();
        if (tid == 0) atomicAdd(p.flags + 5, 1u);
    }
    for (int i = tid; i < p.d / 4; i += kBlock)  // the token's row of the output accumulator
        reinterpret_cast<float4 *>(p.acc + (int64_t)t * p.d)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (tid == 0) {
        s_abort = 0;
        flag_wait(p.flags, (unsigned int)(p.n_gu + p.stall), &s_abort, p.status, p.wait_limit);  // every streamer's gate values are in G
        asm volatile("fence.proxy.async;" ::: "memory");               // ... written by ordinary stores; a bulk copy reads them
    }
    __syncthreads();
    if (s_abort) return;
    MOC_TL_CTA(1280);
    if (!dec::cta_stage_rows(&s_bar, &s_abort, p.status, keys, p.G + (int64_t)t * p.ldf, (uint32_t)Fp * 4u)) return;
    MOC_TL_CTA(3072);
    uint32_t tau;
    int need;
    bool ties_cut;
    uint32_t kreg[dec::kSelCached];
    dec::cta_select_threshold(nullptr, p.F, p.K, keys, lists, sm, tau, need, ties_cut, kreg);
    MOC_TL_CTA(3328);
    uint32_t *my_bits = p.kept_bits + (int64_t)t * p.kept_words;
    constexpr int NW = kBlock / 32;
    if (!ties_cut) {
        // consecutive lanes hold consecutive channels: a ballot is a word of the bitmap
        const int nch = (p.F + kBlock - 1) / kBlock;
        for (int c = 0; c < nch; ++c) {
            const int j = c * kBlock + tid;
            const uint32_t b = __ballot_sync(0xffffffffu, j < p.F && keys[j] >= tau);
            if (lane == 0 && c * kBlock + warp * 32 < p.F) my_bits[c * NW + warp] = b;
        }
    } else {
        __syncthreads();
        for (int i = tid; i < p.kept_words; i += kBlock) bits[i] = 0u;
        __syncthreads();
        block_ordered_emit<kBlock>(keys, p.F, tau, need, sm, [&](int, int j) { atomicOr(&bits[j >> 5], 1u << (j & 31)); });
        __syncthreads();
        for (int i = tid; i < p.kept_words; i += kBlock) my_bits[i] = bits[i];
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        atomicAdd(p.flags + 1, 1u);
        MOC_TL_CTA_ANY(3840);
        cta_finished(p);
    }
    MOC_TL_CTA(1536);
}

// ------------------------------------------------------------------------------------------------ the kernel
// GROUPED: the MoC 2:8 mask (p.grouped; a template parameter so that the Top-K form carries none of its code or registers)
template <bool GROUPED>
__global__ void __launch_bounds__(kBlock, 1) sb_fused_kernel(const __grid_constant__ FusedParams p) {
    namespace cg = cooperative_groups;
    extern __shared__ __align__(16) uint8_t smem_raw[];
    __shared__ int s_last, s_clean;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool streamer = (int)blockIdx.x < p.n_stream;
    tc::pdl_launch_dependents();  // the next kernel in the stream may become resident as this one's CTAs leave
    if (streamer && warp == 2 && lane < 5) {  // the tensor maps' first use would otherwise wait for their fetch
        const CUtensorMap *m = lane == 0 ? &p.wg_map : lane == 1 ? &p.x_map : lane == 2 ? &p.wu_map : lane == 3 ? &p.wd_map : &p.z_map;
        asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
    }
    MOC_TL_CTA(256);
#ifdef MOC_TIMELINE
    if (blockIdx.x == 0 && threadIdx.x == 0) {  // the starts of the last 64 calls
        const unsigned long long n = atomicAdd(&g_timeline[4095], 1ull);
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        g_timeline[3584 + (int)(n & 63ull)] = t;
    }
#endif

    // ---- the streamer's shared memory and work (a selector CTA computes the same numbers and uses none of them)
    const uint32_t raw = tc::smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    float *sg = reinterpret_cast<float *>(smem_raw + (base - raw) + p.tail_off);  // gate values [32][rows]
    const uint32_t bar_base = base + p.tail_off + (uint32_t)(kTn * p.rows * 4);
    uint8_t *bar_ptr = smem_raw + (bar_base - raw);
    auto slot = [&](int s) { return base + (uint32_t)s * p.slot_bytes; };
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kStagesMax + s); };
    const uint32_t tfull_g = bar_base + 8u * (2 * kStagesMax), tfull_u = tfull_g + 8u, tfull_d = tfull_g + 16u;
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(bar_ptr + 8 * (2 * kStagesMax + 3));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);

    const uint32_t kXBox = (uint32_t)p.tn * kBK * 2;  // one activation box: tn tokens x 64 elements
    const int ch0 = (int)blockIdx.x * p.rows;
    const bool has_gu = streamer && ch0 < p.F;
    const int extra = p.rows > kTile ? p.rows - kTile : 0;  // rows of the second MMA tile that are new
    const uint32_t nb = (uint32_t)p.gu_boxes;
    const uint32_t gu_bytes = nb * (kXBox + (uint32_t)p.rows * kBK * 2u);  // what arrives in one stage of phases G, U
    const int n_gu = has_gu ? p.gu_stages : 0;
    const int k_shift = has_gu ? (int)(((int64_t)blockIdx.x * p.gu_stages) / p.n_gu) : 0;
    const bool has_d = streamer && (int)blockIdx.x < p.m_tiles * p.splits;
    const int m_blk = (int)blockIdx.x / p.splits, split = (int)blockIdx.x - m_blk * p.splits;
    const int kb0 = has_d ? (int)(((int64_t)split * p.kb_down) / p.splits) : 0;
    const int kb1 = has_d ? (int)(((int64_t)(split + 1) * p.kb_down) / p.splits) : 0;
    const int n_d = kb1 - kb0;
    const int col0 = m_blk * kTile * p.accs;
    const uint32_t d_w_bytes = (uint32_t)(2 * p.accs) * (64 * kBK * 2), d_bytes = d_w_bytes + kXBox;

    // producer state (thread 0 before the grid barrier, the same thread after it)
    int pr_stage = 0, pr_item = 0;
    uint32_t pr_phase = 0;
    auto pr_next = [&]() {
        ++pr_item;
        if (++pr_stage == p.stages) {
            pr_stage = 0;
            pr_phase ^= 1u;
        }
    };
    // stage `item` of phases G and U: activation boxes first (their size is fixed), then the weight boxes
    auto gu_block0 = [&](int item) {
        // CTAs walk the contraction dimension from different starting points, so that at any moment they ask for
        // different lines of x
        int s = (item >= n_gu ? item - n_gu : item) + k_shift;
        if (s >= n_gu) s -= n_gu;
        return p.gu_boxes * s;
    };
    auto issue_gu_w = [&](int item, int stage) {
        const CUtensorMap *wm = item >= n_gu ? &p.wu_map : &p.wg_map;
        const int kb = gu_block0(item);
        tc::mbar_expect_tx(full_bar(stage), gu_bytes);
        for (int b = 0; b < p.gu_boxes; ++b)
            tc::tma_load_2d(slot(stage) + nb * kXBox + (uint32_t)b * p.w_pitch, wm, full_bar(stage), (kb + b) * kBK, ch0);
    };
    auto issue_gu_x = [&](int item, int stage) {
        const int kb = gu_block0(item);
        for (int b = 0; b < p.gu_boxes; ++b)
            tc::tma_load_2d(slot(stage) + (uint32_t)b * kXBox, &p.x_map, full_bar(stage), (kb + b) * kBK, 0);
    };
    const int ahead = min(p.stages, 2 * n_gu);  // stages requested before the grid barrier

    if (streamer) {
        if (threadIdx.x == 0) {
            for (int s = 0; s < p.stages; ++s) {
                tc::mbar_init(full_bar(s), 1);
                tc::mbar_init(empty_bar(s), 1);
            }
            tc::mbar_init(tfull_g, 2);  // one arrival per MMA issuer
            tc::mbar_init(tfull_u, 2);
            tc::mbar_init(tfull_d, 2);
            *abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            // the first ring of weight boxes leaves at once: the weights depend on nothing earlier in the stream
            for (int i = 0; i < ahead; ++i) issue_gu_w(i, i);
        }
        if (warp == 1) {
            tc::tmem_alloc(tc::smem_u32(const_cast<uint32_t *>(tmem_holder)), kTmemCols);
            tc::tmem_relinquish();
        }
    }
    // everything below touches what earlier kernels in the stream may still read or write (x, the workspace, out)
    tc::pdl_wait();
    if (streamer && threadIdx.x == 0 && !p.rms_w) {
        for (int i = 0; i < ahead; ++i) {
            issue_gu_x(i, i);
            pr_next();
        }
    }
    // (a thread other than the one that is busy requesting the first ring reads the mark)
    if (threadIdx.x == 96) s_clean = __ldcg(reinterpret_cast<const unsigned long long *>(p.flags + 6)) == kCleanMark ? 1 : 0;
    tc::tc_fence_before();
    __syncthreads();  // this CTA's barriers and TMEM address are set
    // the last CTA to have read the mark removes it: from here on a run that does not complete leaves none
    if (threadIdx.x == 96 && atomicAdd(p.flags + 3, 1u) == gridDim.x - 1 && s_clean)
        *reinterpret_cast<volatile unsigned long long *>(p.flags + 6) = 0ull;
    if (!s_clean) {   // (the same answer in every CTA: the mark changes only once all have read it)
        if (blockIdx.x == 0) {
            if (threadIdx.x < 6) p.flags[threadIdx.x] = 0u;
            for (int i = (int)threadIdx.x; i < kStateCounters; i += kBlock) p.counters[i] = 0;
        }
        cg::this_grid().sync();  // the flags and counters are zero for everyone
    }
    tc::tc_fence_after();
    MOC_TL_CTA(512);

    if (!streamer) {
        selector_role(p, reinterpret_cast<uint32_t *>(smem_raw));
        return;
    }
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            bool ok = true;
            if (p.rms_w) {  // the first ring's activation boxes: once the selector CTAs have normalised every token
                ok = flag_wait(p.flags + 5, (unsigned int)p.T, abort_flag, p.status, p.wait_limit);
                asm volatile("fence.proxy.async;" ::: "memory");
                for (int i = 0; i < ahead && ok; ++i) {
                    issue_gu_x(i, i);
                    pr_next();
                }
            }
            while (ok && pr_item < 2 * n_gu) {  // W_gate, then W_up
                if (!tc::mbar_wait(empty_bar(pr_stage), pr_phase ^ 1u, abort_flag, p.status, p.wait_limit)) {
                    ok = false;
                    break;
                }
                issue_gu_w(pr_item, pr_stage);
                issue_gu_x(pr_item, pr_stage);
                pr_next();
            }
            // W_down: the weight boxes of as many stages as the ring gives leave before Z' is complete
            auto load_wd = [&](int st, int kb) {
                for (int b = 0; b < 2 * p.accs; ++b)
                    tc::tma_load_2d(slot(st) + (uint32_t)b * (64 * kBK * 2), &p.wd_map, full_bar(st), col0 + 64 * b, kb * kBK);
            };
            const int first_stage = pr_stage;
            int issued = 0;
            for (; issued < n_d && issued < p.stages && ok; ++issued) {
                if (!tc::mbar_wait(empty_bar(pr_stage), pr_phase ^ 1u, abort_flag, p.status, p.wait_limit)) {
                    ok = false;
                    break;
                }
                tc::mbar_expect_tx(full_bar(pr_stage), d_bytes);
                load_wd(pr_stage, kb0 + issued);
                pr_next();
            }
            if (ok && n_d > 0) {
                ok = flag_wait(p.flags + 2, (unsigned int)p.n_gu, abort_flag, p.status, p.wait_limit);  // every streamer's part of Z' is written
                asm volatile("fence.proxy.async;" ::: "memory");                           // ... by ordinary stores; TMA reads it
                MOC_TL_CTA_ANY(2304);
                int st = first_stage;
                for (int i = 0; i < issued && ok; ++i) {
                    tc::tma_load_2d(slot(st) + d_w_bytes, &p.z_map, full_bar(st), (kb0 + i) * kBK, 0);
                    if (++st == p.stages) st = 0;
                }
            }
            for (int i = issued; i < n_d && ok; ++i) {
                if (!tc::mbar_wait(empty_bar(pr_stage), pr_phase ^ 1u, abort_flag, p.status, p.wait_limit)) break;
                tc::mbar_expect_tx(full_bar(pr_stage), d_bytes);
                load_wd(pr_stage, kb0 + i);
                tc::tma_load_2d(slot(pr_stage) + d_w_bytes, &p.z_map, full_bar(pr_stage), (kb0 + i) * kBK, 0);
                pr_next();
            }
        }
    } else if (warp <= 2) {
        // ------------------------------------------------------------------ MMA issuers: stages about.  Both walk the
        // whole sequence of stages and wait for every one (a parity test only tells an odd from an even number of
        // completed rounds, so a thread must see every round of a barrier it waits on); issuer w works on the stages
        // whose number within their phase is w modulo 2.
        if (lane == 0) {
            const uint32_t w = (uint32_t)(warp - 1);
            const uint32_t idesc_gu = sb::idesc_bf16(false, p.tn), idesc_d = sb::idesc_bf16(true, p.tn);
            const uint64_t dk = tc::make_smem_desc(0, 16, 1024), dm = tc::make_smem_desc(0, kBK * 128, 1024);
            const uint32_t hi = (uint32_t)(dk >> 32), lo_k = (uint32_t)dk, lo_m = (uint32_t)dm;  // (the high words agree)
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            auto next = [&]() {
                if (++stage == p.stages) {
                    stage = 0;
                    phase ^= 1u;
                }
            };
            const uint32_t xp = kXBox >> 4, wp = p.w_pitch >> 4;
            for (int m = 0; m < 2 && ok; ++m) {
                const uint32_t acc0 = tmem_base + (uint32_t)(128 * m) + 64u * w;
                uint32_t accum = 0u;
                for (int s = 0; s < n_gu; ++s) {
                    if (!tc::mbar_wait(full_bar(stage), phase, abort_flag, p.status, p.wait_limit)) {
                        ok = false;
                        break;
                    }
                    if (((uint32_t)s & 1u) == w) {
                        tc::tc_fence_after();
                        const uint32_t x_lo = lo_k + (slot(stage) >> 4), w_lo = x_lo + nb * xp;
                        for (uint32_t b = 0; b < nb; ++b) {
#pragma unroll
                            for (uint32_t k = 0; k < kBK / 16; ++k) {
                                umma_lohi(acc0, w_lo + b * wp + 2u * k, x_lo + b * xp + 2u * k, hi, idesc_gu, accum);
                                if (extra) umma_lohi(acc0 + (uint32_t)kTn, w_lo + b * wp + 8u * (uint32_t)extra + 2u * k, x_lo + b * xp + 2u * k, hi, idesc_gu, accum);
                                accum = 1u;
                            }
                        }
                        tc::umma_commit(empty_bar(stage));
                    }
                    next();
                }
                if (ok && n_gu > 0) tc::umma_commit(m == 0 ? tfull_g : tfull_u);
                MOC_TL_IF((m == 0 ? 768 : 1792) + (int)blockIdx.x, w == 1u);
            }
            const uint32_t accd = tmem_base + 256u + 64u * w;
            uint32_t accum = 0u;
            for (int i = 0; i < n_d && ok; ++i) {
                if (!tc::mbar_wait(full_bar(stage), phase, abort_flag, p.status, p.wait_limit)) {
                    ok = false;
                    break;
                }
                if (((uint32_t)i & 1u) == w) {
                    tc::tc_fence_after();
                    const uint32_t a_lo = lo_m + (slot(stage) >> 4), z_lo = lo_k + ((slot(stage) + d_w_bytes) >> 4);
#pragma unroll
                    for (uint32_t k = 0; k < kBK / 16; ++k) {
                        for (uint32_t a = 0; a < (uint32_t)p.accs; ++a)
                            umma_lohi(accd + a * (uint32_t)kTn, a_lo + a * 1024u + k * 128u, z_lo + 2u * k, hi, idesc_d, accum);
                        accum = 1u;
                    }
                    tc::umma_commit(empty_bar(stage));
                }
                next();
            }
            if (ok && n_d > 0) tc::umma_commit(tfull_d);
            MOC_TL_IF(2560 + (int)blockIdx.x, w == 1u);
        }
    } else if (warp < 3 + kEpiWarps) {
        // ------------------------------------------------------------------ epilogue warps 3..10
        // Work items are (tile, 16-token chunk); the two warps of a TMEM lane quarter take alternate items.
        const int quarter = warp & 3, half = (warp - 3) >> 2, etid = (int)threadIdx.x - 96;
        const int valid = min(p.rows, p.F - ch0);  // channels of this CTA inside the matrix
        const int trow = quarter * 32 + lane;      // row of the MMA tile this thread reads
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int chunks = p.tn >> 4;
        bool ok = true;
        if (has_gu) {
            const int items = (extra ? 2 : 1) * chunks;
            const bool two = n_gu >= 2;  // the second issuer had stages of its own
            uint32_t kept0 = 0u;         // MoC 2:8: bit i = this lane's channel is kept by token i of the warp's first item
            // MoC 2:8: the kept bits of tokens t0 .. t0 + 15 for this lane's channel, from the gate values in shared memory.
            // The 8 channels of a group sit in 8 adjacent lanes: a channel is kept when fewer than two of its group come
            // before it in (key descending, channel ascending) order.  (A plain loop: few registers are live.)
            auto group_mask = [&](int row, bool mine, int t0) {
                uint32_t bits = 0u;
#pragma unroll 1
                for (int i = 0; i < 16; ++i) {
                    const uint32_t key = (mine && t0 + i < p.T) ? gate_key(sg[(t0 + i) * p.rows + row]) : 0u;
                    int before = 0;
#pragma unroll
                    for (int m = 1; m < 8; ++m) {
                        const uint32_t other = __shfl_xor_sync(0xffffffffu, key, m);
                        before += (other > key || (other == key && ((lane ^ m) & 7) < (lane & 7))) ? 1 : 0;
                    }
                    bits |= (before < kGroupKeep ? 1u : 0u) << i;
                }
                return bits;
            };
            // ---- gate values
            ok = __all_sync(0xffffffffu, tc::mbar_wait(tfull_g, 0u, abort_flag, p.status, p.wait_limit));
            if (ok) {
                tc::tc_fence_after();
                for (int item = half; item < items; item += 2) {
                    const int tile = item / chunks, t0 = (item - tile * chunks) << 4;
                    if (tile == 1 && quarter * 32 + 31 < kTile - extra) continue;  // warp-uniform: nothing new in this quarter
                    const int row = tile == 0 ? trow : extra + trow;  // channel within the CTA's range
                    const bool mine = (tile == 0 ? trow < p.rows : trow >= kTile - extra) && row < valid;
                    float g[16];
                    tmem_ld16_sum(lane_addr + (uint32_t)(tile * kTn + t0), two, g);
                    if (mine) {
                        float *dst = p.G + ch0 + row + (int64_t)t0 * p.ldf;
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            if (t0 + i < p.T) {
                                if (!GROUPED) dst[(int64_t)i * p.ldf] = g[i];  // a warp's store: 128 contiguous bytes
                                sg[(t0 + i) * p.rows + row] = g[i];
                            }
                        }
                    }
                }
            }
            if (GROUPED && ok && half < items && !((half / chunks) == 1 && quarter * 32 + 31 < kTile - extra)) {
                // the mask needs the gate values only: for the warp's first item it is worked out now, while the up
                // projection streams, not after it
                const int tile = half / chunks, t0 = (half - tile * chunks) << 4;
                const int row = tile == 0 ? trow : extra + trow;
                __syncwarp();
                kept0 = group_mask(row, (tile == 0 ? trow < p.rows : trow >= kTile - extra) && row < valid, t0);
            }
            if (GROUPED) {
                // no selector CTAs: the streamers clear the output accumulator, a slice each (ordered before every
                // addition to it by the count of streamers whose Z' is written, which each joins only afterwards)
                const int64_t vecs = (int64_t)p.T * p.d / 4;
                const int64_t v0 = vecs * blockIdx.x / p.n_gu, v1 = vecs * (blockIdx.x + 1) / p.n_gu;
                for (int64_t i = v0 + etid; i < v1; i += kEpiThreads) reinterpret_cast<float4 *>(p.acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            } else {
                __threadfence();
                asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
                if (etid == 0 && !*abort_flag) atomicAdd(p.flags, 1u);  // (a CTA that gave up is never counted: those that
                                                                          //  wait for it give up in turn, nothing half-done is read)
            }
            MOC_TL_IF(1024 + (int)blockIdx.x, etid == 0);
            // ---- Z' = SiLU(g) u on the kept channels.  The products are formed for every channel as soon as the up
            // projection is complete; the bitmaps, which usually arrive last, then only decide which of them are stored.
            ok = ok && __all_sync(0xffffffffu, tc::mbar_wait(tfull_u, 0u, abort_flag, p.status, p.wait_limit));
            // (the CTAs of a problem with at most 128 channels per CTA and at most 16 tokens have one item per warp)
            const int item0 = half;
            const int tile0 = item0 / chunks, t00 = (item0 - tile0 * chunks) << 4;
            float z0[16];
            const bool pre = ok && item0 < items && !(tile0 == 1 && quarter * 32 + 31 < kTile - extra);
            if (pre) {
                tc::tc_fence_after();
                const int row = tile0 == 0 ? trow : extra + trow;
                tmem_ld16_sum(lane_addr + (uint32_t)(128 + tile0 * kTn + t00), two, z0);
                if (row < valid && (tile0 == 0 ? trow < p.rows : trow >= kTile - extra)) {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (t00 + i < p.T) z0[i] *= silu_f(key_to_float(gate_key(sg[(t00 + i) * p.rows + row])));
                }
            }
            if (!GROUPED) {
                int fine = 1;
                if (lane == 0) fine = ok && flag_wait(p.flags + 1, (unsigned int)p.T, abort_flag, p.status, p.wait_limit) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, fine, 0) != 0;
            }
            if (ok) {
                tc::tc_fence_after();
                for (int item = half; item < items; item += 2) {
                    const int tile = item / chunks, t0 = (item - tile * chunks) << 4;
                    if (tile == 1 && quarter * 32 + 31 < kTile - extra) continue;
                    const int row = tile == 0 ? trow : extra + trow;
                    const bool mine = (tile == 0 ? trow < p.rows : trow >= kTile - extra) && row < valid;
                    // the warp's 32 channels lie in at most two words of a token's bitmap: lane i fetches those of token
                    // t0 + i (one trip to L2 for the whole warp), the loop below hands them round
                    const int ch_lo = ch0 + (tile == 0 ? quarter * 32 : extra + quarter * 32);  // lane 0's channel
                    uint32_t w_lo = 0u, w_hi = 0u;
                    if (!GROUPED && lane < 16 && t0 + lane < p.T && (ch_lo >> 5) < p.kept_words) {
                        const uint32_t *kb = p.kept_bits + (int64_t)(t0 + lane) * p.kept_words + (ch_lo >> 5);
                        w_lo = __ldcg(kb);
                        if ((ch_lo >> 5) + 1 < p.kept_words) w_hi = __ldcg(kb + 1);
                    }
                    float z[16];
                    if (item == item0) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) z[i] = z0[i];
                    } else {  // (warp-uniform)
                        tmem_ld16_sum(lane_addr + (uint32_t)(128 + tile * kTn + t0), two, z);
                        if (mine) {
#pragma unroll
                            for (int i = 0; i < 16; ++i)
                                if (t0 + i < p.T) z[i] *= silu_f(key_to_float(gate_key(sg[(t0 + i) * p.rows + row])));
                        }
                    }
                    const int bit = (ch_lo & 31) + lane;  // position in the 64-bit pair
                    const uint32_t kmask = !GROUPED ? 0u : item == item0 ? kept0 : group_mask(row, mine, t0);
                    __nv_bfloat16 *dst = p.Z + ch_lo + lane + (int64_t)t0 * p.ldz;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        bool kept;
                        if (GROUPED) {
                            kept = ((kmask >> i) & 1u) != 0u;
                        } else {
                            const uint32_t lo = __shfl_sync(0xffffffffu, w_lo, i), hi = __shfl_sync(0xffffffffu, w_hi, i);
                            kept = ((bit < 32 ? lo >> bit : hi >> (bit - 32)) & 1u) != 0u;
                        }
                        if (t0 + i < p.T && mine) dst[(int64_t)i * p.ldz] = __float2bfloat16_rn(kept ? z[i] : 0.f);
                    }
                }
            }
            __threadfence();
            asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
            if (etid == 0 && !*abort_flag) atomicAdd(p.flags + 2, 1u);
            MOC_TL_IF(2048 + (int)blockIdx.x, etid == 0);
        }
        // ---- D: partial sums into the fp32 accumulator, the last CTA of the column block rounds
        if (has_d) {
            const bool done = ok && __all_sync(0xffffffffu, tc::mbar_wait(tfull_d, 0u, abort_flag, p.status, p.wait_limit));
            if (done) {
                tc::tc_fence_after();
                const bool two = n_d >= 2;
                for (int item = half; item < p.accs * chunks; item += 2) {
                    const int a = item / chunks, t0 = (item - a * chunks) << 4;
                    const int col = col0 + a * kTile + quarter * 32 + lane;
                    float r[16];
                    tmem_ld16_sum(lane_addr + (uint32_t)(256 + a * kTn + t0), two, r);
                    // 4 x 4 transposes among the four lanes that hold four adjacent columns: lane l of the group ends up
                    // with the four columns of token 4 g + l, which leave as one 16-byte vector reduction
                    const int l4 = lane & 3;
                    const bool odd = (l4 & 1) != 0, hi = (l4 & 2) != 0;
#pragma unroll
                    for (int g4 = 0; g4 < 4; ++g4) {
                        float v0 = r[4 * g4], v1 = r[4 * g4 + 1], v2 = r[4 * g4 + 2], v3 = r[4 * g4 + 3];
                        float x0 = __shfl_xor_sync(0xffffffffu, odd ? v0 : v1, 1);
                        float x1 = __shfl_xor_sync(0xffffffffu, odd ? v2 : v3, 1);
                        if (odd) {
                            v0 = x0;
                            v2 = x1;
                        } else {
                            v1 = x0;
                            v3 = x1;
                        }
                        x0 = __shfl_xor_sync(0xffffffffu, hi ? v0 : v2, 2);
                        x1 = __shfl_xor_sync(0xffffffffu, hi ? v1 : v3, 2);
                        if (hi) {
                            v0 = x0;
                            v1 = x1;
                        } else {
                            v2 = x0;
                            v3 = x1;
                        }
                        const int tok = t0 + 4 * g4 + l4;
                        if (tok < p.T && col < p.d)
                            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p.acc + (int64_t)tok * p.d + (col - l4)),
                                         "f"(v0), "f"(v1), "f"(v2), "f"(v3)
                                         : "memory");
                    }
                }
            }
            __threadfence();
            asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
            if (etid == 0) s_last = !*abort_flag && atomicAdd(&p.counters[m_blk], 1) == p.splits - 1;
            asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
            if (s_last) {
                __threadfence();
                const int cols = min(kTile * p.accs, p.d - col0), vecs = cols / 4;  // cols is a multiple of 8
                for (int i = etid; i < p.T * vecs; i += kEpiThreads) {
                    const int t = i / vecs, c = (i - t * vecs) * 4;
                    float4 v = __ldcg(reinterpret_cast<const float4 *>(p.acc + (int64_t)t * p.d + col0 + c));
                    if (p.resid) {  // out = h + D (out may be h itself: the same thread reads and writes an element)
                        const uint2 hb = *reinterpret_cast<const uint2 *>(p.resid + (int64_t)t * p.d + col0 + c);
                        v.x += __uint_as_float(hb.x << 16);
                        v.y += __uint_as_float(hb.x & 0xffff0000u);
                        v.z += __uint_as_float(hb.y << 16);
                        v.w += __uint_as_float(hb.y & 0xffff0000u);
                    }
                    *reinterpret_cast<uint2 *>(p.out + (int64_t)t * p.d + col0 + c) =
                        make_uint2(tc::pack_bf16(v.x, v.y), tc::pack_bf16(v.z, v.w));
                }
                if (etid == 0) p.counters[m_blk] = 0;  // ready for the next run
            }
        }
    }

    __syncwarp();
    if (warp < 3 + kEpiWarps && *abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tc::tc_fence_before();
    __syncthreads();
    MOC_TL_CTA(2816);
    if (threadIdx.x == 0 && !*abort_flag) cta_finished(p);
    if (warp == 1) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace sbf
}  // namespace moc
