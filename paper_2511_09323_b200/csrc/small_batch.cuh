// Small-batch plan (bf16, 17..128 tokens): the forward as three weight-streaming kernels on tcgen05.
//
// With a few dozen tokens the union of the tokens' Top-K sets covers nearly every channel
// (1 - (1 - K/F)^T), so the row gathers of the decode plan (Section 5) no longer save bytes: the whole
// of W_gate, W_up and W_down is read once, and the job is to keep HBM busy.  The token count is far
// below a 128-row MMA tile, so the operands are swapped: the WEIGHTS are the M side of the MMA
// (128 channels, or 128 output columns, per CTA) and the tokens are its N side (T rounded up to 32).
//
//   1. sb_gate_up_kernel   G^T | U^T [channel, token] = [Wg ; Wu] x^T          (Eq. (Moc-1) and U = X W_up)
//                          one CTA per (matrix, 128 channels); fp32 G and U [T, ldf] in the workspace
//   2. sb_select_kernel    per token: exact Top-K of G (or 2 of every 8), Z' = SiLU(G) . M . U  (mask, Eq. (MoC-2))
//                          as a dense bf16 row; optionally the compact saved triple; zeroes the output accumulator
//   3. sb_down_kernel      D^T [column, token] = Wd^T Z'^T, the channels split over several CTAs per 128 columns;
//                          partial sums meet in an fp32 accumulator (vector-free red.add), the last CTA of a
//                          column block rounds to bf16
//
// Every CTA owns one tile and two CTAs share an SM, so that all tiles are resident at once and the
// bytes in flight, not a tile schedule, set the pace.  The kernels are chained with programmatic
// dependent launch: weights stream before the dependency wait, activations and the workspace are
// touched after it.  Waits are bounded as everywhere else in the library.
#pragma once

#include "decode_kernels.cuh"
#include "grouped_select.cuh"
#include "tc_gemm.cuh"
#include "topk_select.cuh"

namespace moc {
namespace sb {

constexpr int kTile = 128;      // MMA M: weight rows (channels / output columns) per CTA
constexpr int kBK = 64;         // contraction elements per stage: one 128-byte swizzle row
constexpr int kThreads = 192;   // warp 0 TMA, warp 1 MMA + TMEM, warps 2..5 epilogue
constexpr int kMaxStages = 8;
constexpr int kMaxTokens = 128;
constexpr uint32_t kWeightStageBytes = kTile * kBK * 2;  // 16 KiB
constexpr uint32_t kBarRegion = 256;
constexpr size_t kSmemBudget = 108 * 1024;  // per CTA, two CTAs per SM

struct GemmShape {
    int tn;        // tokens rounded up to a multiple of 32 (MMA N, rows of the activation box)
    int tmem_cols; // power of two >= tn
    int stages;
    uint32_t stage_bytes;
    size_t smem;
};

inline GemmShape gemm_shape(int tokens) {
    GemmShape s{};
    s.tn = (tokens + 31) & ~31;
    s.tmem_cols = s.tn <= 32 ? 32 : s.tn <= 64 ? 64 : 128;
    s.stage_bytes = kWeightStageBytes + (uint32_t)s.tn * kBK * 2;
    const size_t room = kSmemBudget - 1024 - kBarRegion;
    s.stages = (int)std::min<size_t>(kMaxStages, room / s.stage_bytes);
    s.smem = 1024 + (size_t)s.stages * s.stage_bytes + kBarRegion;
    return s;
}

struct GateUpParams {
    CUtensorMap w_map[2];  // W_gate, W_up: [F, d] rows of d contiguous elements, boxes of 128 rows x 64
    CUtensorMap x_map;     // x [T, d], boxes of tn rows x 64 (rows >= T read as zero)
    int T, tn, tmem_cols, stages;
    uint32_t stage_bytes;
    int F, k_blocks, tiles;  // tiles = ceil(F / 128) per matrix
    float *G, *U;            // [T, ldf]
    int ldf;
    int *counters, n_counters;  // zeroed here for the down kernel
    int *status;
};

struct DownParams {
    CUtensorMap wd_map;  // W_down [F, d] read as the M-major operand: boxes of 64 channels x 64 columns
    CUtensorMap z_map;   // Z' [T, F], boxes of tn rows x 64 channels
    int T, tn, tmem_cols, stages;
    uint32_t stage_bytes;
    int d, k_blocks, m_tiles, splits;
    float *acc;          // [T, d] fp32, zero on entry
    __nv_bfloat16 *out;  // [T, d]
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
};

// ---------------------------------------------------------------------------------------------- 1. gate + up
__global__ void __launch_bounds__(kThreads, 2) sb_gate_up_kernel(const __grid_constant__ GateUpParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = tc::smem_u32(smem_raw);
    Ring ring;
    ring.base = (raw + 1023u) & ~1023u;
    ring.stage_bytes = p.stage_bytes;
    ring.bar_base = ring.base + (uint32_t)p.stages * p.stage_bytes;
    uint8_t *bar_ptr = smem_raw + (ring.bar_base - raw);
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(bar_ptr + 8 * (2 * kMaxStages + 1));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    tc::pdl_launch_dependents();

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            tc::mbar_init(ring.full(s), 1);
            tc::mbar_init(ring.empty(s), 1);
        }
        tc::mbar_init(ring.tfull(), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tc::tmem_alloc(tc::smem_u32(const_cast<uint32_t *>(tmem_holder)), (uint32_t)p.tmem_cols);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    const int prob = (int)blockIdx.x / p.tiles;
    const int ch0 = ((int)blockIdx.x - prob * p.tiles) * kTile;

    if (warp == 0) {
        if (lane == 0) {
            tc::prefetch_tmap(&p.w_map[prob]);
            tc::prefetch_tmap(&p.x_map);
            // the weights depend on nothing earlier in the stream: the first stages' weight boxes leave at once,
            // their activation boxes after the dependency wait
            const int ahead = min(p.stages, p.k_blocks);
            for (int kb = 0; kb < ahead; ++kb) {
                tc::mbar_expect_tx(ring.full(kb), p.stage_bytes);
                tc::tma_load_2d(ring.stage(kb), &p.w_map[prob], ring.full(kb), kb * kBK, ch0);
            }
            tc::pdl_wait();
            for (int kb = 0; kb < ahead; ++kb)
                tc::tma_load_2d(ring.stage(kb) + kWeightStageBytes, &p.x_map, ring.full(kb), kb * kBK, 0);
            int stage = 0;
            uint32_t phase = 1;  // the ring has gone round once
            for (int kb = ahead; kb < p.k_blocks; ++kb) {
                if (!tc::mbar_wait(ring.empty(stage), phase ^ 1u, abort_flag, p.status)) break;
                tc::mbar_expect_tx(ring.full(stage), p.stage_bytes);
                tc::tma_load_2d(ring.stage(stage), &p.w_map[prob], ring.full(stage), kb * kBK, ch0);
                tc::tma_load_2d(ring.stage(stage) + kWeightStageBytes, &p.x_map, ring.full(stage), kb * kBK, 0);
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
                const uint32_t sa = ring.stage(stage), sb = sa + kWeightStageBytes;
#pragma unroll
                for (int k = 0; k < kBK / 16; ++k)
                    tc::umma_bf16(tmem_base, tc::make_smem_desc(sa + k * 32, 16, 1024),
                                  tc::make_smem_desc(sb + k * 32, 16, 1024), idesc, (kb | k) != 0 ? 1u : 0u);
                tc::umma_commit(ring.empty(stage));
                if (++stage == p.stages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
            if (ok) tc::umma_commit(ring.tfull());
        }
    } else {
        // ---- epilogue: lane = channel, columns = tokens; a warp's store of one token is 128 contiguous bytes
        const int quarter = warp & 3;
        tc::pdl_wait();  // the workspace may still be read by the previous call's kernels
        if (blockIdx.x == 0)
            for (int i = (int)threadIdx.x - 64; i < p.n_counters; i += 128) p.counters[i] = 0;
        if (__all_sync(0xffffffffu, tc::mbar_wait(ring.tfull(), 0u, abort_flag, p.status))) {
            tc::tc_fence_after();
            const int ch = ch0 + quarter * 32 + lane;
            float *dst = (prob == 0 ? p.G : p.U) + ch;
            for (int c0 = 0; c0 < p.tn; c0 += 32) {
                uint32_t r[32];
                __syncwarp();
                tc::tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r);
                tc::tmem_ld_wait();
                if (ch < p.F) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c0 + i < p.T) dst[(int64_t)(c0 + i) * p.ldf] = __uint_as_float(r[i]);
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
};

// One CTA per token.  The threshold search is the decode plan's; the set then leaves as the token's dense
// masked row Z' (and, when asked for, as the compact triple in ascending channel order).
__global__ void __launch_bounds__(dec::kSelThreads) sb_select_kernel(const SelectParams p) {
    extern __shared__ __align__(16) uint32_t dyn[];  // keys [F] | 2 candidate lists (the first doubles as the bitmap)
    __shared__ SelectSmemT<dec::kSelThreads / 32> sm;
    const int tid = threadIdx.x;
    const int t = blockIdx.x;
    tc::pdl_launch_dependents();
    tc::pdl_wait();
    const float *g = p.G + (int64_t)t * p.ldf, *u = p.U + (int64_t)t * p.ldf;
    for (int i = tid; i < p.d / 4; i += dec::kSelThreads)
        reinterpret_cast<float4 *>(p.acc + (int64_t)t * p.d)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    uint32_t tau;
    int need;
    bool ties_cut;
    dec::cta_select_threshold(g, p.F, p.K, dyn, sm, tau, need, ties_cut);
    const uint32_t *keys = dyn;
    uint32_t *bits = dyn + p.F;  // bitmap of the kept channels, only when ties are cut or the triple is wanted
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
                go[pos] = __float2bfloat16_rn(g[j]);
                uo[pos] = __float2bfloat16_rn(u[j]);
            }
        });
    }
    // Z' row, two channels per thread.  The saved up value is rounded to bf16 before it is used, so that the
    // backward pass, which recomputes z from the saved pair, sees the same product.
    __nv_bfloat16 *z = p.Z + (int64_t)t * p.ldz;
    for (int j = 2 * tid; j < p.F; j += 2 * dec::kSelThreads) {
        float v[2] = {0.f, 0.f};
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int jj = j + e;
            if (jj >= p.F) continue;
            const bool kept = by_bitmap ? ((bits[jj >> 5] >> (jj & 31)) & 1u) != 0u : keys[jj] >= tau;
            if (kept) {
                const float uv = save ? __bfloat162float(__float2bfloat16_rn(u[jj])) : u[jj];
                v[e] = silu_f(g[jj]) * uv;
            }
        }
        if (j + 1 < p.ldz)
            *reinterpret_cast<__nv_bfloat162 *>(z + j) = __floats2bfloat162_rn(v[0], v[1]);
        else
            z[j] = __float2bfloat16_rn(v[0]);
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
        const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
        uint32_t key[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) key[e] = gate_key(gv[e]);
        int lo, hi;
        top2_of_8(key, lo, hi);
        float zv[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        const int sel[2] = {lo, hi};
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            float gs = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (e == sel[s]) gs = gv[e];
            float us = u[q * kGroup + sel[s]];
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
// grid = m_tiles * splits; CTA (m, s) contracts its share of the channel blocks for output columns 128 m ..
__global__ void __launch_bounds__(kThreads, 2) sb_down_kernel(const __grid_constant__ DownParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ int s_last;
    const uint32_t raw = tc::smem_u32(smem_raw);
    Ring ring;
    ring.base = (raw + 1023u) & ~1023u;
    ring.stage_bytes = p.stage_bytes;
    ring.bar_base = ring.base + (uint32_t)p.stages * p.stage_bytes;
    uint8_t *bar_ptr = smem_raw + (ring.bar_base - raw);
    volatile uint32_t *tmem_holder = reinterpret_cast<volatile uint32_t *>(bar_ptr + 8 * (2 * kMaxStages + 1));
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_holder + 1);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    tc::pdl_launch_dependents();

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            tc::mbar_init(ring.full(s), 1);
            tc::mbar_init(ring.empty(s), 1);
        }
        tc::mbar_init(ring.tfull(), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tc::tmem_alloc(tc::smem_u32(const_cast<uint32_t *>(tmem_holder)), (uint32_t)p.tmem_cols);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    const int m_blk = (int)blockIdx.x / p.splits, split = (int)blockIdx.x - m_blk * p.splits;
    const int kb0 = (int)(((int64_t)split * p.k_blocks) / p.splits);
    const int kb1 = (int)(((int64_t)(split + 1) * p.k_blocks) / p.splits);
    const int nkb = kb1 - kb0;  // >= 1: the host keeps splits <= k_blocks
    const int col0 = m_blk * kTile;

    if (warp == 0) {
        if (lane == 0) {
            tc::prefetch_tmap(&p.wd_map);
            tc::prefetch_tmap(&p.z_map);
            auto load_w = [&](int stage, int kb) {
                // two boxes of 64 columns x 64 channels: the M-major operand layout
                tc::tma_load_2d(ring.stage(stage), &p.wd_map, ring.full(stage), col0, kb * kBK);
                tc::tma_load_2d(ring.stage(stage) + 64 * kBK * 2, &p.wd_map, ring.full(stage), col0 + 64, kb * kBK);
            };
            const int ahead = min(p.stages, nkb);
            for (int i = 0; i < ahead; ++i) {
                tc::mbar_expect_tx(ring.full(i), p.stage_bytes);
                load_w(i, kb0 + i);
            }
            tc::pdl_wait();  // Z' comes from the select kernel
            for (int i = 0; i < ahead; ++i)
                tc::tma_load_2d(ring.stage(i) + kWeightStageBytes, &p.z_map, ring.full(i), (kb0 + i) * kBK, 0);
            int stage = 0;
            uint32_t phase = 1;
            for (int i = ahead; i < nkb; ++i) {
                if (!tc::mbar_wait(ring.empty(stage), phase ^ 1u, abort_flag, p.status)) break;
                tc::mbar_expect_tx(ring.full(stage), p.stage_bytes);
                load_w(stage, kb0 + i);
                tc::tma_load_2d(ring.stage(stage) + kWeightStageBytes, &p.z_map, ring.full(stage), (kb0 + i) * kBK, 0);
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
                const uint32_t sa = ring.stage(stage), sb = sa + kWeightStageBytes;
#pragma unroll
                for (int k = 0; k < kBK / 16; ++k)
                    tc::umma_bf16(tmem_base, tc::make_smem_desc(sa + k * 2048, kBK * 128, 1024),
                                  tc::make_smem_desc(sb + k * 32, 16, 1024), idesc, (i | k) != 0 ? 1u : 0u);
                tc::umma_commit(ring.empty(stage));
                if (++stage == p.stages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
            if (ok) tc::umma_commit(ring.tfull());
        }
    } else {
        // ---- epilogue: lane = output column, TMEM columns = tokens
        const int quarter = warp & 3;
        const int etid = (int)threadIdx.x - 64;
        tc::pdl_wait();
        const bool done = __all_sync(0xffffffffu, tc::mbar_wait(ring.tfull(), 0u, abort_flag, p.status));
        if (done) {
            tc::tc_fence_after();
            const int col = col0 + quarter * 32 + lane;
            float *dst = p.acc + col;
            for (int c0 = 0; c0 < p.tn; c0 += 32) {
                uint32_t r[32];
                __syncwarp();
                tc::tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r);
                tc::tmem_ld_wait();
                if (col < p.d) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c0 + i < p.T) atomicAdd(dst + (int64_t)(c0 + i) * p.d, __uint_as_float(r[i]));
                }
            }
        }
        // the last CTA of this column block to get here rounds the sums to bf16
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (etid == 0) s_last = atomicAdd(&p.counters[m_blk], 1) == p.splits - 1;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (s_last) {
            __threadfence();
            const int cols = min(kTile, p.d - col0);  // even: d is a multiple of 8
            const int half = cols / 2;
            for (int i = etid; i < p.T * half; i += 128) {
                const int t = i / half, c = (i - t * half) * 2;
                const float2 v = __ldcg(reinterpret_cast<const float2 *>(p.acc + (int64_t)t * p.d + col0 + c));
                *reinterpret_cast<__nv_bfloat162 *>(p.out + (int64_t)t * p.d + col0 + c) = __floats2bfloat162_rn(v.x, v.y);
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
    if (warp == 1) {
        tc::tc_fence_after();
        tc::tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

}  // namespace sb
}  // namespace moc
