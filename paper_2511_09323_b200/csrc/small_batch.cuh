// Small-batch plan (bf16, up to 256 tokens): the forward as three weight-streaming kernels on tcgen05.
//
// With a few dozen tokens the union of the tokens' Top-K sets covers nearly every channel
// (1 - (1 - K/F)^T), so the row gathers of the decode plan (Section 5) no longer save bytes: the whole
// of W_gate, W_up and W_down is read once, and the job is to keep HBM busy.  The token count is far
// below a 128-row MMA tile, so the operands are swapped: the WEIGHTS are the M side of the MMA and the
// tokens are its N side (T rounded up to 32).
//
//   1. sb_gate_up_kernel   G^T | U^T [channel, token] = [Wg ; Wu] x^T          (Eq. (Moc-1) and U = X W_up)
//                          every CTA owns `rows` consecutive channels of one matrix, rows chosen so that the
//                          grid is one CTA per SM; fp32 G and U [T, ldf] go to the workspace
//   2. sb_select_kernel    per token: exact Top-K of G (or 2 of every 8), Z' = SiLU(G) . M . U  (mask, Eq. (MoC-2))
//                          as a dense bf16 row; optionally the compact saved triple; zeroes the output accumulator
//   3. sb_down_kernel      D^T [column, token] = Wd^T Z'^T; a CTA owns 128 or 256 output columns and a share of
//                          the channels; partial sums meet in an fp32 accumulator (16-byte red.add), the last CTA of a
//                          column block rounds to bf16.  The backward of a small batch uses the same kernel for
//                          grad_x = dG' Wg + dU' Wu (Eq. (bp-5)): two contraction segments into one accumulator
//
// One CTA per SM with the deepest ring of stages shared memory allows: the bytes in flight set the pace.
// The kernels are chained with programmatic dependent launch: weights stream before the dependency
// wait, activations and the workspace are touched after it.  Waits are bounded as everywhere else in
// the library.
#pragma once

#include "decode_kernels.cuh"
#include "grouped_select.cuh"
#include "tc_gemm.cuh"
#include "topk_select.cuh"

namespace moc {
namespace sb {

constexpr int kTile = 128;      // MMA M
constexpr int kBK = 64;         // contraction elements per stage: one 128-byte swizzle row
constexpr int kThreads = 320;   // warp 0 TMA, warp 1 MMA + TMEM, warps 2..9 epilogue (two per TMEM lane quarter)
constexpr int kEpiThreads = kThreads - 64;
constexpr int kMaxStages = 16;  // narrow stages (few rows per CTA) need many of them to keep enough bytes in flight
constexpr int kMaxTokens = 256;
constexpr int kMaxRows = 256;   // weight rows per CTA: two MMA tiles
constexpr uint32_t kBarRegion = 512;
constexpr size_t kSmemBudget = 224 * 1024;
constexpr size_t kSmemSlack = 1024 /*alignment*/ + kTile * kBK * 2 /*an MMA over a short tile reads 128 rows*/;

struct GemmShape {
    int tn;            // tokens rounded up to a multiple of 32 (MMA N, rows of the activation box)
    int tmem_cols;     // power of two >= accumulators * tn
    int stages;
    uint32_t w_bytes;  // weight bytes per stage
    uint32_t stage_bytes;
    size_t smem;
};

// weight_rows: rows (gate/up: channels; down: output columns) per CTA, at most kMaxRows
// boxes: 64-element contraction blocks per stage (gate/up kernel only: with few rows per CTA a stage of one block is
// so small that the per-stage hand-overs, not HBM, set the pace; two blocks per stage halve their number)
inline GemmShape gemm_shape(int tokens, int weight_rows, int boxes = 1) {
    GemmShape s{};
    s.tn = (tokens + 31) & ~31;
    const int cols = s.tn * (weight_rows > kTile ? 2 : 1);
    s.tmem_cols = cols <= 32 ? 32 : cols <= 64 ? 64 : cols <= 128 ? 128 : cols <= 256 ? 256 : 512;
    s.w_bytes = (uint32_t)weight_rows * kBK * 2 * (uint32_t)boxes;
    s.stage_bytes = s.w_bytes + (uint32_t)s.tn * kBK * 2 * (uint32_t)boxes;
    const size_t room = kSmemBudget - kSmemSlack - kBarRegion;
    s.stages = (int)std::min<size_t>(kMaxStages, room / s.stage_bytes);
    s.smem = kSmemSlack + (size_t)s.stages * s.stage_bytes + kBarRegion;
    return s;
}

struct GateUpParams {
    CUtensorMap w_map[2];  // W_gate, W_up: [F, d] rows of d contiguous elements, boxes of `rows` rows x 64
    CUtensorMap x_map;     // x [T, d], boxes of tn rows x 64 (rows >= T read as zero)
    int T, tn, tmem_cols, stages;
    uint32_t w_bytes, stage_bytes;
    int F, k_blocks;
    int rows, ctas_per_matrix;  // channels per CTA (multiple of 8, <= 256); grid = 2 * ctas_per_matrix
    float *G, *U;               // [T, ldf]
    int ldf;
    int *counters, n_counters;  // zeroed here for the down kernel
    int *status;
    int boxes;  // 64-element contraction blocks per stage (1 or 2); k_blocks counts stages
    // Which matrices the grid covers: CTA b works on matrix prob0 + b / ctas_per_matrix (prob0 = 0 and a grid of
    // 2 * ctas_per_matrix: both, as one launch; the overlapped form launches the kernel once per matrix).
    int prob0;
    // mask_mode (the up projection of the overlapped form): instead of storing U, the epilogue forms the masked hidden
    // state Z' = SiLU(G) . M . U (Eq. (MoC-2)) for its channels from the gate values in G and the selection bitmaps
    // that the select kernel left, and stores it as bf16 [T, ldz].  The kernel then reads x without waiting for the
    // kernels before it: it is only launched once the kernel that wrote G has completed, which itself read x.
    int mask_mode;
    const uint32_t *kept_bits;  // [T, kept_words]: bit j of a token's words = channel j is kept
    int kept_words;
    __nv_bfloat16 *Z;           // [T, ldz]
    int ldz;
};

struct DownParams {
    // One or two contraction segments, each a weight matrix [F, d] read as the M-major operand (boxes of 64 channels x
    // 64 columns) and an activation array [T, F] (boxes of tn rows x 64 channels): the forward's D = Z' Wd has one,
    // the backward's dX = dG' Wg + dU' Wu (Eq. (bp-5)) two that add into the same accumulator.
    CUtensorMap wd_map[2];
    CUtensorMap z_map[2];
    int segments;
    int T, tn, tmem_cols, stages;
    uint32_t w_bytes, stage_bytes;
    int d, k_blocks, m_tiles, splits;  // k_blocks: channel blocks of ONE segment; the splits share segments * k_blocks
    int accs;            // 1 or 2: the CTA owns 128 * accs output columns
    float *acc;          // [T, d] fp32, zero on entry
    __nv_bfloat16 *out;  // [T, d]
    const __nv_bfloat16 *resid;  // [T, d] added to the sums before rounding (the block form's residual), or nullptr
    int *counters;       // [m_tiles], zero on entry, left zero
    int *status;
};

__device__ __forceinline__ uint32_t idesc_bf16(bool a_mn, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(kTile >> 4) << 24);
}

// Shared-memory carve-up common to both GEMM kernels: stages | barriers | TMEM address | abort flag.
struct Ring {
    uint32_t base, bar_base;
    uint32_t stage_bytes;
    __device__ __forceinline__ uint32_t stage(int s) const { return base + (uint32_t)s * stage_bytes; }
    __device__ __forceinline__ uint32_t full(int s) const { return bar_base + 8u * s; }
    __device__ __forceinline__ uint32_t empty(int s) const { return bar_base + 8u * (kMaxStages + s); }
    __device__ __forceinline__ uint32_t tfull() const { return bar_base + 8u * (2 * kMaxStages); }
    __device__ __forceinline__ uint32_t extra() const { return bar_base + 8u * (2 * kMaxStages + 2); }  // after the TMEM address and the abort flag
};

// ---------------------------------------------------------------------------------------------- 1. gate + up
// A CTA's `rows` channels are covered by one MMA tile (rows <= 128; the rows of the tile beyond `rows` are whatever
// follows in shared memory and land in accumulator lanes nobody reads) or by two overlapping ones: tile 0 = rows
// 0..127, tile 1 = rows (rows - 128)..(rows - 1), of which only the last rows - 128 lanes are new.
__global__ void __launch_bounds__(kThreads, 1) sb_gate_up_kernel(const __grid_constant__ GateUpParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = tc::smem_u32(smem_raw);
    Ring ring;
    ring.base = (raw + 1023u) & ~1023u;
    ring.stage_bytes = p.stage_bytes;
    ring.bar_base = ring.base + (uint32_t)p.stages * p.stage_bytes + kTile * kBK * 2;
    uint8_t *bar_ptr = smem_raw + (ring.bar_base - raw);
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(bar_ptr + 8 * (2 * kMaxStages + 1));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    tc::pdl_launch_dependents();
    MOC_TL(p.mask_mode ? 32 : 0);
    MOC_TL_CTA(p.mask_mode ? 1536 : 256);

    const int prob = p.prob0 + (int)blockIdx.x / p.ctas_per_matrix;
    const int ch0 = ((int)blockIdx.x % p.ctas_per_matrix) * p.rows;
    const int ahead = min(p.stages, p.k_blocks);
    const uint32_t w_box = (uint32_t)p.rows * kBK * 2, x_box = (uint32_t)p.tn * kBK * 2;  // one 64-element block of each

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            tc::mbar_init(ring.full(s), 1);
            tc::mbar_init(ring.empty(s), 1);
        }
        tc::mbar_init(ring.tfull(), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        // the weights depend on nothing earlier in the stream: the first stages' weight boxes leave at once,
        // their activation boxes after the dependency wait
        for (int kb = 0; kb < ahead; ++kb) {
            tc::mbar_expect_tx(ring.full(kb), p.stage_bytes);
            for (int b = 0; b < p.boxes; ++b)
                tc::tma_load_2d(ring.stage(kb) + (uint32_t)b * w_box, &p.w_map[prob], ring.full(kb), (kb * p.boxes + b) * kBK, ch0);
        }
    }
    if (warp == 1) {
        tc::tmem_alloc(tc::smem_u32(const_cast<uint32_t *>(tmem_holder)), (uint32_t)p.tmem_cols);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    const int extra = p.rows > kTile ? p.rows - kTile : 0;  // rows of the second tile that are new

    if (warp == 0) {
        if (lane == 0) {
            if (!p.mask_mode) tc::pdl_wait();
            for (int kb = 0; kb < ahead; ++kb)
                for (int b = 0; b < p.boxes; ++b)
                    tc::tma_load_2d(ring.stage(kb) + p.w_bytes + (uint32_t)b * x_box, &p.x_map, ring.full(kb),
                                    (kb * p.boxes + b) * kBK, 0);
            int stage = 0;
            uint32_t phase = 1;  // the ring has gone round once
            for (int kb = ahead; kb < p.k_blocks; ++kb) {
                if (!tc::mbar_wait(ring.empty(stage), phase ^ 1u, abort_flag, p.status)) break;
                tc::mbar_expect_tx(ring.full(stage), p.stage_bytes);
                for (int b = 0; b < p.boxes; ++b) {
                    tc::tma_load_2d(ring.stage(stage) + (uint32_t)b * w_box, &p.w_map[prob], ring.full(stage),
                                    (kb * p.boxes + b) * kBK, ch0);
                    tc::tma_load_2d(ring.stage(stage) + p.w_bytes + (uint32_t)b * x_box, &p.x_map, ring.full(stage),
                                    (kb * p.boxes + b) * kBK, 0);
                }
                if (++stage == p.stages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16(false, p.tn);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int kb = 0; kb < p.k_blocks; ++kb) {
                if (!tc::mbar_wait(ring.full(stage), phase, abort_flag, p.status)) {
                    ok = false;
                    break;
                }
                tc::tc_fence_after();
                for (int b = 0; b < p.boxes; ++b) {
                    const uint32_t sa = ring.stage(stage) + (uint32_t)b * w_box, sb = ring.stage(stage) + p.w_bytes + (uint32_t)b * x_box;
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k) {
                        const uint64_t bd = tc::make_smem_desc(sb + k * 32, 16, 1024);
                        tc::umma_bf16(tmem_base, tc::make_smem_desc(sa + k * 32, 16, 1024), bd, idesc,
                                      (kb | b | k) != 0 ? 1u : 0u);
                        if (extra)
                            tc::umma_bf16(tmem_base + (uint32_t)p.tn,
                                          tc::make_smem_desc(sa + (uint32_t)extra * 128u + k * 32, 16, 1024), bd, idesc,
                                          (kb | b | k) != 0 ? 1u : 0u);
                    }
                }
                tc::umma_commit(ring.empty(stage));
                if (++stage == p.stages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
            if (ok) tc::umma_commit(ring.tfull());
            MOC_TL_IF(p.mask_mode ? 34 : 2, blockIdx.x == 0);
            MOC_TL_CTA_ANY(p.mask_mode ? 1792 : 512);
        }
    } else {
        // ---- epilogue: lane = channel, columns = tokens; a warp's store of one token is 128 contiguous bytes
        const int quarter = warp & 3;
        tc::pdl_wait();  // the workspace may still be read by the previous call's kernels
        MOC_TL_IF(p.mask_mode ? 35 : 3, blockIdx.x == 0 && threadIdx.x == 64);
        if (blockIdx.x == 0)
            for (int i = (int)threadIdx.x - 64; i < p.n_counters; i += kEpiThreads) p.counters[i] = 0;
        const int valid = min(p.rows, p.F - ch0);  // channels of this CTA inside the matrix
        // mask mode: the factors SiLU(g) . M of this thread's first items (four channels of one token each, as the loop
        // after the accumulators' transposition deals them out) are fetched now, while the main loop still runs
        constexpr int kPre = 4;
        float4 sf[kPre];
        const int quads_pre = valid >> 2;
        if (p.mask_mode) {
#pragma unroll
            for (int q = 0; q < kPre; ++q) {
                sf[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                const int i = (int)threadIdx.x - 64 + q * kEpiThreads;
                if ((valid & 3) == 0 && i < p.T * quads_pre) {
                    const int t = i / quads_pre, ch = ch0 + ((i - t * quads_pre) << 2);
                    const uint32_t nib = (p.kept_bits[(int64_t)t * p.kept_words + (ch >> 5)] >> (ch & 31)) & 0xfu;
                    if (nib) {
                        const float4 g4 = *reinterpret_cast<const float4 *>(p.G + (int64_t)t * p.ldf + ch);
                        if (nib & 1u) sf[q].x = silu_f(key_to_float(gate_key(g4.x)));
                        if (nib & 2u) sf[q].y = silu_f(key_to_float(gate_key(g4.y)));
                        if (nib & 4u) sf[q].z = silu_f(key_to_float(gate_key(g4.z)));
                        if (nib & 8u) sf[q].w = silu_f(key_to_float(gate_key(g4.w)));
                    }
                }
            }
        }
        if (__all_sync(0xffffffffu, tc::mbar_wait(ring.tfull(), 0u, abort_flag, p.status))) {
            tc::tc_fence_after();
            float *base = prob == 0 ? p.G : p.U;
            if (p.mask_mode) base = nullptr;  // nothing of U is stored
            const int trow = quarter * 32 + lane;  // row of the MMA tile this thread reads
            // The tile goes through the (now idle) stage ring, transposed to [token][channel], and leaves as one
            // bulk store per token: 128 scalar stores per thread would add microseconds to the end of the kernel.
            // A channel count that is not a multiple of 4 (a ragged last CTA) cannot be a bulk copy, and the tile of a
            // large batch of long rows may not fit the ring: direct stores.
            const bool fits = (uint32_t)p.T * (uint32_t)p.rows * 4u <= (uint32_t)p.stages * p.stage_bytes;
            const bool bulk = (valid & 3) == 0 && fits;
            const uint32_t pitch = (uint32_t)p.rows * 4u;
            float *stage_f = reinterpret_cast<float *>(smem_raw + (ring.base - raw));
            // work items = (tile, 32-token chunk); the two warps of a lane quarter take alternate items
            const int chunks = p.tn >> 5, half = (warp - 2) >> 2;
            for (int item = half; item < (extra ? 2 : 1) * chunks; item += 2) {
                const int tile = item / chunks, c0 = (item - tile * chunks) << 5;
                const int row = tile == 0 ? trow : extra + trow;  // row within the CTA's channels
                const bool mine = (tile == 0 ? trow < p.rows : trow >= kTile - extra) && row < valid;
                if (tile == 1 && quarter * 32 + 31 < kTile - extra) continue;  // warp-uniform: nothing new in this quarter
                uint32_t r[32];
                __syncwarp();
                tc::tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(tile * p.tn + c0), r);
                tc::tmem_ld_wait();
                if (!mine) {
                    // (no early exit: the TMEM load above is warp-collective)
                } else if (p.mask_mode && !bulk) {
                    // ragged channel count or a tile too large for the ring: this thread's channel, token by token
                    const int ch = ch0 + row;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int t = c0 + i;
                        if (t < p.T) {
                            const bool kept = (p.kept_bits[(int64_t)t * p.kept_words + (ch >> 5)] >> (ch & 31)) & 1u;
                            float z = 0.f;
                            if (kept) z = silu_f(key_to_float(gate_key(p.G[(int64_t)t * p.ldf + ch]))) * __uint_as_float(r[i]);
                            p.Z[(int64_t)t * p.ldz + ch] = __float2bfloat16_rn(z);
                        }
                    }
                } else if (bulk) {
                    float *dst = stage_f + (size_t)c0 * p.rows + row;
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c0 + i < p.T) dst[i * p.rows] = __uint_as_float(r[i]);
                } else {
                    float *dst = base + ch0 + row + (int64_t)c0 * p.ldf;
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c0 + i < p.T) dst[(int64_t)i * p.ldf] = __uint_as_float(r[i]);
                }
            }
            if (bulk && p.mask_mode) {
                // the tile lies in shared memory as [token][channel]: four channels per step, kept ones multiplied by
                // SiLU of their gate value (recovered from its key, so that a NaN acts as -inf here as in the selection)
                asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
                const int etid = (int)threadIdx.x - 64, quads = valid >> 2;
#pragma unroll
                for (int q = 0; q < kPre; ++q) {  // the items whose factors are in registers already
                    const int i = etid + q * kEpiThreads;
                    if (i < p.T * quads) {
                        const int t = i / quads, c = (i - t * quads) << 2;
                        const float4 u4 = *reinterpret_cast<const float4 *>(stage_f + (size_t)t * p.rows + c);
                        *reinterpret_cast<uint2 *>(p.Z + (int64_t)t * p.ldz + ch0 + c) =
                            make_uint2(tc::pack_bf16(sf[q].x * u4.x, sf[q].y * u4.y), tc::pack_bf16(sf[q].z * u4.z, sf[q].w * u4.w));
                    }
                }
                for (int i = etid + kPre * kEpiThreads; i < p.T * quads; i += kEpiThreads) {
                    const int t = i / quads, c = (i - t * quads) << 2, ch = ch0 + c;
                    const float4 u4 = *reinterpret_cast<const float4 *>(stage_f + (size_t)t * p.rows + c);
                    const uint32_t nib = (p.kept_bits[(int64_t)t * p.kept_words + (ch >> 5)] >> (ch & 31)) & 0xfu;
                    float z[4] = {0.f, 0.f, 0.f, 0.f};
                    if (nib) {
                        const float4 g4 = *reinterpret_cast<const float4 *>(p.G + (int64_t)t * p.ldf + ch);
                        const float gv[4] = {g4.x, g4.y, g4.z, g4.w}, uv[4] = {u4.x, u4.y, u4.z, u4.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if ((nib >> e) & 1u) z[e] = silu_f(key_to_float(gate_key(gv[e]))) * uv[e];
                    }
                    *reinterpret_cast<uint2 *>(p.Z + (int64_t)t * p.ldz + ch) =
                        make_uint2(tc::pack_bf16(z[0], z[1]), tc::pack_bf16(z[2], z[3]));
                }
            } else if (bulk) {
                tc::fence_async_smem();
                asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
                const int etid = (int)threadIdx.x - 64;
                if (etid < p.T) {
                    tc::bulk_copy_s2g(base + (int64_t)etid * p.ldf + ch0, ring.base + (uint32_t)etid * pitch,
                                      (uint32_t)valid * 4u);
                    tc::bulk_store_wait_read<0>();  // shared memory must outlive the copy's reads
                }
            }
        }
    }

    __syncwarp();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tc::tc_fence_before();
    __syncthreads();
    MOC_TL(p.mask_mode ? 36 : 4);
    MOC_TL_CTA(p.mask_mode ? 2048 : 768);
    if (warp == 1) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------------- 2. select
struct SelectParams {
    const float *G, *U;  // [T, ldf]
    int ldf, F, K, d;
    __nv_bfloat16 *Z;    // [T, ldz] dense masked hidden state
    int ldz;
    float *acc;          // [T, d], zeroed here
    int16_t *idx_out;    // compact saved activations [T, K] (all three or none)
    __nv_bfloat16 *g_out, *u_out;
    int stage_u;         // 1: shared memory has room for the token's up row as well
    int *status;
    // the overlapped form: when not null the kernel writes only the token's selection bitmap (kept_words words: bit j =
    // channel j is kept) and zeroes the accumulator; U and Z are not touched (the up kernel's epilogue forms Z')
    uint32_t *kept_bits;
    int kept_words;
};

// dynamic shared memory of sb_select_kernel: keys [Fp] | 2 candidate lists | up row [Fp] (when staged)
inline size_t select_smem(int F, bool stage_u) {
    const size_t Fp = (size_t)((F + 3) & ~3);
    return (Fp * (stage_u ? 2 : 1) + 2 * dec::kSelListCap) * sizeof(uint32_t);
}

// One CTA per token.  The token's gate row (and up row) arrive with bulk copies; the threshold search is the decode
// plan's; the set then leaves as the token's dense masked row Z' (and, when asked for, as the compact triple in
// ascending channel order).  Gate values are recovered from their keys, so a NaN gate value acts as -inf in the
// product as well as in the selection.
__global__ void __launch_bounds__(dec::kSelThreads) sb_select_kernel(const SelectParams p) {
    extern __shared__ __align__(16) uint32_t dyn[];
    __shared__ SelectSmemT<dec::kSelThreads / 32> sm;
    __shared__ uint64_t s_bar;
    __shared__ int s_abort;
    const int tid = threadIdx.x;
    const int t = blockIdx.x;
    const int Fp = (p.F + 3) & ~3;
    uint32_t *keys = dyn, *lists = dyn + Fp;
    uint32_t *bits = lists;  // bitmap of the kept channels once the search is over
    const float *u_row = p.stage_u ? reinterpret_cast<const float *>(lists + 2 * dec::kSelListCap)
                                   : p.U + (int64_t)t * p.ldf;
    MOC_TL(16);
    if (p.kept_bits) {
        // the up kernel behind this one streams its weights while the selection runs; it may start only now that the
        // gate kernel has completed (it reads x without a wait of its own)
        tc::pdl_wait();
        tc::pdl_launch_dependents();
        MOC_TL(17);
        MOC_TL_CTA(1024);
    } else {
        tc::pdl_launch_dependents();
        tc::pdl_wait();
    }
    dec::cta_stage_rows_begin(&s_bar, &s_abort, keys, p.G + (int64_t)t * p.ldf, (uint32_t)Fp * 4u,
                              p.stage_u ? lists + 2 * dec::kSelListCap : nullptr,
                              p.stage_u ? p.U + (int64_t)t * p.ldf : nullptr);
    for (int i = tid; i < p.d / 4; i += dec::kSelThreads)  // while the rows travel
        reinterpret_cast<float4 *>(p.acc + (int64_t)t * p.d)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (!dec::cta_stage_rows_wait(&s_bar, &s_abort, p.status)) return;
    uint32_t tau;
    int need;
    bool ties_cut;
    uint32_t kreg[dec::kSelCached];
    dec::cta_select_threshold(nullptr, p.F, p.K, keys, lists, sm, tau, need, ties_cut, kreg);
    if (p.kept_bits) {
        uint32_t *my_bits = p.kept_bits + (int64_t)t * p.kept_words;
        const int lane = tid & 31, warp = tid >> 5;
        constexpr int NW = dec::kSelThreads / 32;
        if (!ties_cut) {
            // consecutive lanes hold consecutive channels: a ballot is a word of the bitmap
            const int nch = (p.F + dec::kSelThreads - 1) / dec::kSelThreads;
            for (int c = 0; c < nch; ++c) {
                const int j = c * dec::kSelThreads + tid;
                const uint32_t b = __ballot_sync(0xffffffffu, j < p.F && keys[j] >= tau);
                if (lane == 0 && c * dec::kSelThreads + warp * 32 < p.F) my_bits[c * NW + warp] = b;
            }
        } else {
            __syncthreads();
            for (int i = tid; i < p.kept_words; i += dec::kSelThreads) bits[i] = 0u;
            __syncthreads();
            block_ordered_emit<dec::kSelThreads>(keys, p.F, tau, need, sm,
                                                 [&](int, int j) { atomicOr(&bits[j >> 5], 1u << (j & 31)); });
            __syncthreads();
            for (int i = tid; i < p.kept_words; i += dec::kSelThreads) my_bits[i] = bits[i];
        }
        MOC_TL(18);
        MOC_TL_CTA(1280);
        return;
    }
    const bool save = p.idx_out != nullptr;
    const bool by_bitmap = ties_cut || save;
    if (by_bitmap) {
        __syncthreads();
        for (int i = tid; i < (p.F + 31) / 32; i += dec::kSelThreads) bits[i] = 0u;
        __syncthreads();
        int16_t *io = save ? p.idx_out + (int64_t)t * p.K : nullptr;
        __nv_bfloat16 *go = save ? p.g_out + (int64_t)t * p.K : nullptr;
        __nv_bfloat16 *uo = save ? p.u_out + (int64_t)t * p.K : nullptr;
        block_ordered_emit<dec::kSelThreads>(keys, p.F, tau, need, sm, [&](int pos, int j) {
            atomicOr(&bits[j >> 5], 1u << (j & 31));
            if (save) {
                io[pos] = (int16_t)j;
                go[pos] = __float2bfloat16_rn(key_to_float(keys[j]));
                uo[pos] = __float2bfloat16_rn(u_row[j]);
            }
        });
    }
    // Z' row.  When the triple is saved the up value is rounded to bf16 before it is used, so that the backward pass,
    // which recomputes z from the saved pair, sees the same product.
    __nv_bfloat16 *z = p.Z + (int64_t)t * p.ldz;
    auto z_of = [&](uint32_t key, int j) {
        const float uv = save ? __bfloat162float(__float2bfloat16_rn(u_row[j])) : u_row[j];
        return __float2bfloat16_rn(silu_f(key_to_float(key)) * uv);
    };
    if (p.F <= dec::kSelCached * dec::kSelThreads) {
        // The thread's keys are still in registers: the row is zero-filled with 16-byte stores (into the padding up
        // to ldz as well), then every thread drops the values of its own kept channels (one in eight) into place.
        for (int q = tid; q * 8 < p.F; q += dec::kSelThreads) *reinterpret_cast<uint4 *>(z + q * 8) = make_uint4(0u, 0u, 0u, 0u);
        __syncthreads();
#pragma unroll
        for (int i = 0; i < dec::kSelCached; ++i) {
            const int j = tid + i * dec::kSelThreads;
            if (j < p.F) {
                const bool kept = by_bitmap ? ((bits[j >> 5] >> (j & 31)) & 1u) != 0u : kreg[i] >= tau;
                if (kept) z[j] = z_of(kreg[i], j);
            }
        }
    } else {
        // long rows: eight channels (one 16-byte store) per thread and step
        for (int q = tid; q * 8 < p.F; q += dec::kSelThreads) {
            const int j0 = q * 8;
            uint32_t kept = 0;
            if (by_bitmap) {
                kept = (bits[j0 >> 5] >> (j0 & 31)) & 0xffu;
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (j0 + e < p.F && keys[j0 + e] >= tau) kept |= 1u << e;
            }
            uint32_t w[4] = {0u, 0u, 0u, 0u};
            while (kept) {
                const int e = __ffs(kept) - 1;
                kept &= kept - 1u;
                const uint32_t hbits = (uint32_t)__bfloat16_as_ushort(z_of(keys[j0 + e], j0 + e)) << (16 * (e & 1));
#pragma unroll
                for (int q2 = 0; q2 < 4; ++q2)
                    if ((e >> 1) == q2) w[q2] |= hbits;
            }
            *reinterpret_cast<uint4 *>(z + j0) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

// MoC 2:8 (Section 4): the mask is local, one thread per group of 8 channels.
__global__ void __launch_bounds__(dec::kSelThreads) sb_select_grouped_kernel(const SelectParams p) {
    const int tid = threadIdx.x;
    const int t = blockIdx.x;
    tc::pdl_launch_dependents();
    tc::pdl_wait();
    const float *g = p.G + (int64_t)t * p.ldf, *u = p.U + (int64_t)t * p.ldf;
    for (int i = tid; i < p.d / 4; i += dec::kSelThreads)
        reinterpret_cast<float4 *>(p.acc + (int64_t)t * p.d)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    const bool save = p.idx_out != nullptr;
    __nv_bfloat16 *z = p.Z + (int64_t)t * p.ldz;
    for (int q = tid; q < p.F / kGroup; q += dec::kSelThreads) {
        const float4 g0 = reinterpret_cast<const float4 *>(g + q * kGroup)[0];
        const float4 g1 = reinterpret_cast<const float4 *>(g + q * kGroup)[1];
        const float4 u0 = reinterpret_cast<const float4 *>(u + q * kGroup)[0];
        const float4 u1 = reinterpret_cast<const float4 *>(u + q * kGroup)[1];
        const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
        const float uv[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
        uint32_t key[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) key[e] = gate_key(gv[e]);
        int lo, hi;
        top2_of_8(key, lo, hi);
        float zv[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        const int sel[2] = {lo, hi};
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            float gs = 0.f, us = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (e == sel[s]) {
                    gs = gv[e];
                    us = uv[e];
                }
            if (save) {
                const int64_t o = (int64_t)t * p.K + 2 * q + s;
                p.idx_out[o] = (int16_t)(q * kGroup + sel[s]);
                p.g_out[o] = __float2bfloat16_rn(gs);
                p.u_out[o] = __float2bfloat16_rn(us);
                us = __bfloat162float(__float2bfloat16_rn(us));
            }
            const float zz = silu_f(gs) * us;
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (e == sel[s]) zv[e] = zz;
        }
        *reinterpret_cast<uint4 *>(z + q * kGroup) =
            make_uint4(tc::pack_bf16(zv[0], zv[1]), tc::pack_bf16(zv[2], zv[3]), tc::pack_bf16(zv[4], zv[5]),
                       tc::pack_bf16(zv[6], zv[7]));
    }
}

// ---------------------------------------------------------------------------------------------- 3. down
// grid = m_tiles * splits; CTA (m, s) contracts its share of the channel blocks for output columns
// 128 * accs * m ..; with accs == 2 the activation box of a stage feeds two MMA tiles.
__global__ void __launch_bounds__(kThreads, 1) sb_down_kernel(const __grid_constant__ DownParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ int s_last;
    const uint32_t raw = tc::smem_u32(smem_raw);
    Ring ring;
    ring.base = (raw + 1023u) & ~1023u;
    ring.stage_bytes = p.stage_bytes;
    ring.bar_base = ring.base + (uint32_t)p.stages * p.stage_bytes + kTile * kBK * 2;
    uint8_t *bar_ptr = smem_raw + (ring.bar_base - raw);
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(bar_ptr + 8 * (2 * kMaxStages + 1));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    tc::pdl_launch_dependents();
    MOC_TL(48);
    MOC_TL_CTA(2304);

    const int m_blk = (int)blockIdx.x / p.splits, split = (int)blockIdx.x - m_blk * p.splits;
    const int kb_all = p.k_blocks * p.segments;
    const int kb0 = (int)(((int64_t)split * kb_all) / p.splits);
    const int kb1 = (int)(((int64_t)(split + 1) * kb_all) / p.splits);
    const int nkb = kb1 - kb0;  // >= 1: the host keeps splits <= k_blocks
    const int col0 = m_blk * kTile * p.accs;
    const int ahead = min(p.stages, nkb);
    auto load_w = [&](int stage, int kb) {
        // boxes of 64 columns x 64 channels, 8 KiB each: the M-major operand layout, two boxes per MMA tile
        const int sg = kb >= p.k_blocks ? 1 : 0;
        for (int b = 0; b < 2 * p.accs; ++b)
            tc::tma_load_2d(ring.stage(stage) + (uint32_t)b * (64 * kBK * 2), &p.wd_map[sg], ring.full(stage), col0 + 64 * b,
                            (kb - sg * p.k_blocks) * kBK);
    };
    auto load_z = [&](int stage, int kb) {
        const int sg = kb >= p.k_blocks ? 1 : 0;
        tc::tma_load_2d(ring.stage(stage) + p.w_bytes, &p.z_map[sg], ring.full(stage), (kb - sg * p.k_blocks) * kBK, 0);
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            tc::mbar_init(ring.full(s), 1);
            tc::mbar_init(ring.empty(s), 1);
        }
        tc::mbar_init(ring.tfull(), 1);
        tc::mbar_init(ring.extra(), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        for (int i = 0; i < ahead; ++i) {  // weights first: they depend on nothing earlier in the stream
            tc::mbar_expect_tx(ring.full(i), p.stage_bytes);
            load_w(i, kb0 + i);
        }
    }
    if (warp == 1) {
        tc::tmem_alloc(tc::smem_u32(const_cast<uint32_t *>(tmem_holder)), (uint32_t)p.tmem_cols);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp == 0) {
        if (lane == 0) {
            tc::pdl_wait();  // Z' comes from the select kernel
            MOC_TL_IF(49, blockIdx.x == 0);
            MOC_TL_CTA_ANY(2560);
            for (int i = 0; i < ahead; ++i) load_z(i, kb0 + i);
            int stage = 0;
            uint32_t phase = 1;
            for (int i = ahead; i < nkb; ++i) {
                if (!tc::mbar_wait(ring.empty(stage), phase ^ 1u, abort_flag, p.status)) break;
                tc::mbar_expect_tx(ring.full(stage), p.stage_bytes);
                load_w(stage, kb0 + i);
                load_z(stage, kb0 + i);
                if (++stage == p.stages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = idesc_bf16(true, p.tn);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int i = 0; i < nkb; ++i) {
                if (!tc::mbar_wait(ring.full(stage), phase, abort_flag, p.status)) {
                    ok = false;
                    break;
                }
                tc::tc_fence_after();
                const uint32_t sa = ring.stage(stage), sb = sa + p.w_bytes;
#pragma unroll
                for (int k = 0; k < kBK / 16; ++k) {
                    const uint64_t bd = tc::make_smem_desc(sb + k * 32, 16, 1024);
                    for (int a = 0; a < p.accs; ++a)
                        tc::umma_bf16(tmem_base + (uint32_t)(a * p.tn),
                                      tc::make_smem_desc(sa + (uint32_t)a * (2 * 64 * kBK * 2) + k * 2048, kBK * 128, 1024),
                                      bd, idesc, (i | k) != 0 ? 1u : 0u);
                }
                tc::umma_commit(ring.empty(stage));
                if (++stage == p.stages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
            if (ok) tc::umma_commit(ring.tfull());
            MOC_TL_CTA_ANY(2816);
        }
    } else {
        // ---- epilogue: lane = output column, TMEM columns = tokens
        const int quarter = warp & 3;
        const int etid = (int)threadIdx.x - 64;
        tc::pdl_wait();
        const bool done = __all_sync(0xffffffffu, tc::mbar_wait(ring.tfull(), 0u, abort_flag, p.status));
        if (done) {
            tc::tc_fence_after();
            const int chunks = p.tn >> 5, half = (warp - 2) >> 2;
            for (int item = half; item < p.accs * chunks; item += 2) {
                const int a = item / chunks, c0 = (item - a * chunks) << 5;
                const int col = col0 + a * kTile + quarter * 32 + lane;
                uint32_t r[32];
                __syncwarp();
                tc::tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * p.tn + c0), r);
                tc::tmem_ld_wait();
                // 4 x 4 transposes among the four lanes that hold four adjacent columns: lane l of the group ends up
                // with the four columns of token 4 g + l, which leave as one 16-byte vector reduction (d is a
                // multiple of 8, so a group of four columns is inside the row or outside it as a whole)
                const int l4 = lane & 3;
                const bool odd = (l4 & 1) != 0, hi = (l4 & 2) != 0;
#pragma unroll
                for (int g4 = 0; g4 < 8; ++g4) {
                    float v0 = __uint_as_float(r[4 * g4]), v1 = __uint_as_float(r[4 * g4 + 1]);
                    float v2 = __uint_as_float(r[4 * g4 + 2]), v3 = __uint_as_float(r[4 * g4 + 3]);
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
                    const int tok = c0 + 4 * g4 + l4;
                    if (tok < p.T && col < p.d)
                        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(
                                         p.acc + (int64_t)tok * p.d + (col - l4)),
                                     "f"(v0), "f"(v1), "f"(v2), "f"(v3)
                                     : "memory");
                }
            }
        }
        // the last CTA of this column block to get here rounds the sums to bf16
        __threadfence();
        asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
        if (etid == 0) s_last = atomicAdd(&p.counters[m_blk], 1) == p.splits - 1;
        asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
        if (s_last) {
            __threadfence();
            // The sums of this column block come back with one bulk copy per token into the (now idle) stage ring
            // -- a handful of plain loads per thread would take longer than the whole main loop -- and leave as bf16.
            asm volatile("fence.proxy.async;" ::: "memory");
            const int cols = min(kTile * p.accs, p.d - col0);  // a multiple of 8
            const uint32_t row_bytes = (uint32_t)cols * 4u;
            const int per_round = (int)min((uint32_t)p.T, ((uint32_t)p.stages * p.stage_bytes) / row_bytes);  // tokens the ring holds
            const uint8_t *stage_ptr = smem_raw + (ring.base - raw);
            const int vecs = cols / 4;
            uint32_t parity = 0;
            if (p.T * vecs <= 4 * kEpiThreads) {
                // a few vectors per thread: independent loads from L2 (where the reductions left the sums) cost one round
                // trip, less than setting up and awaiting the bulk copies
                for (int i = etid; i < p.T * vecs; i += kEpiThreads) {
                    const int t = i / vecs, c = (i - t * vecs) * 4;
                    float4 v = __ldcg(reinterpret_cast<const float4 *>(p.acc + (int64_t)t * p.d + col0 + c));
                    if (p.resid) {
                        const uint2 hb = *reinterpret_cast<const uint2 *>(p.resid + (int64_t)t * p.d + col0 + c);
                        v.x += __uint_as_float(hb.x << 16);
                        v.y += __uint_as_float(hb.x & 0xffff0000u);
                        v.z += __uint_as_float(hb.y << 16);
                        v.w += __uint_as_float(hb.y & 0xffff0000u);
                    }
                    *reinterpret_cast<uint2 *>(p.out + (int64_t)t * p.d + col0 + c) =
                        make_uint2(tc::pack_bf16(v.x, v.y), tc::pack_bf16(v.z, v.w));
                }
            } else
            for (int t0 = 0; t0 < p.T; t0 += per_round, parity ^= 1u) {
                const int nt = min(per_round, p.T - t0);
                asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");  // the ring is free again
                if (etid == 0) tc::mbar_expect_tx(ring.extra(), row_bytes * (uint32_t)nt);
                asm volatile("bar.sync 1, %0;" ::"n"(kEpiThreads) : "memory");
                for (int t = etid; t < nt; t += kEpiThreads)
                    tc::bulk_copy_g2s(ring.base + (uint32_t)t * row_bytes, p.acc + (int64_t)(t0 + t) * p.d + col0, row_bytes,
                                      ring.extra());
                // (after a failed wait the rounds go on, so that every warp meets the barriers above; their waits
                //  return at once because the abort flag is set)
                const bool landed = __all_sync(0xffffffffu, tc::mbar_wait(ring.extra(), parity, abort_flag, p.status));
                for (int i = etid; landed && i < nt * vecs; i += kEpiThreads) {
                    const int t = i / vecs, c = (i - t * vecs) * 4;
                    float4 v = *reinterpret_cast<const float4 *>(stage_ptr + (size_t)t * row_bytes + (size_t)c * 4);
                    if (p.resid) {  // out = h + D (out may be h itself: the same thread reads and writes an element)
                        const uint2 hb = *reinterpret_cast<const uint2 *>(p.resid + (int64_t)(t0 + t) * p.d + col0 + c);
                        v.x += __uint_as_float(hb.x << 16);
                        v.y += __uint_as_float(hb.x & 0xffff0000u);
                        v.z += __uint_as_float(hb.y << 16);
                        v.w += __uint_as_float(hb.y & 0xffff0000u);
                    }
                    *reinterpret_cast<uint2 *>(p.out + (int64_t)(t0 + t) * p.d + col0 + c) =
                        make_uint2(tc::pack_bf16(v.x, v.y), tc::pack_bf16(v.z, v.w));
                }
            }
            if (etid == 0) p.counters[m_blk] = 0;
        }
    }

    __syncwarp();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    tc::tc_fence_before();
    __syncthreads();
    MOC_TL(52);
    MOC_TL_CTA(3072);
    if (warp == 1) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

}  // namespace sb
}  // namespace moc
