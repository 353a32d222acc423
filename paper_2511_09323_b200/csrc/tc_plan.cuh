// Tensor-core plan of the MoC FFN for bf16 training shapes: "compute dense on tcgen05, keep compact".
// At 12.5 % unstructured density the tensor cores finish the dense contraction several times faster
// than the ALUs finish the sparse one, so every contraction runs as a dense GEMM over the full
// channel range and the Top-K structure is applied around it: the forward selects from the fp32
// gate tile and turns the dense up projection into the masked Z' in place; the backward samples
// dD Wd^T at the saved indices in the GEMM epilogue.  Only idx / g / u in compact [T,K] form leave
// the forward; all dense [T,F] arrays are transient workspace.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include "moc_common.cuh"
#include "tc_gemm.cuh"
#include "topk_select.cuh"

namespace moc {
namespace tc {

// ---- driver entry point for tensor-map encoding (looked up once; no link-time dependency on libcuda)
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// bf16 matrix [rows, cols] row-major with leading dimension ld (elements); box = box_cols x box_rows.
// Out-of-range parts of a box read as zero.
inline bool make_map(CUtensorMap *m, const void *ptr, int64_t rows, int64_t cols, int64_t ld, int box_cols,
                     int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// K-major operand: tensor [mn, k], k contiguous; a tile is `tile_mn` rows of 64 k-elements
inline bool map_k_major(CUtensorMap *m, const void *ptr, int64_t mn, int64_t k, int64_t ld, int tile_mn) {
    return make_map(m, ptr, mn, k, ld, BK, tile_mn);
}
// MN-major operand: tensor [k, mn], mn contiguous; loaded as 64 x 64 boxes
inline bool map_mn_major(CUtensorMap *m, const void *ptr, int64_t k, int64_t mn, int64_t ld) {
    return make_map(m, ptr, k, mn, ld, 64, BK);
}

inline int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    }
    return n;
}

inline void init_params(Params &p) {
    memset(&p, 0, sizeof(p));
    p.num_problems = 1;
    p.k_segments = 1;
}

template <bool A_MN, bool B_MN, int EPI>
inline int launch_gemm(const Params &p, cudaStream_t st) {
    auto kern = gemm_kernel<A_MN, B_MN, EPI>;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess)
            return MOC_ERR_CUDA;
        configured = true;
    }
    const int tiles = p.m_tiles * p.n_tiles * p.num_problems;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    if (grid <= 0) return MOC_OK;
    kern<<<grid, THREADS, SMEM_BYTES, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? MOC_OK : MOC_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------
// Threshold hint shared by all selector CTAs / warps of one forward call: {center, half width} of a
// bracket around the threshold of the call's first token.  It only seeds the guess-and-verify
// selection (the result is exact whatever the hint holds); a non-finite center means "no hint".
__device__ __forceinline__ SelectGuess guess_from_hint(const float *hint) {
    SelectGuess g;
    if (hint) {
        const float c = hint[0], d = hint[1];
        if (fabsf(c) <= 3.0e38f && d > 0.f && d <= 1.0e37f) {
            g.center = c;
            g.delta = d;
            g.valid = true;
        }
    }
    return g;
}

// One CTA: exact threshold of row 0 by the radix select -> hint[0..1].
__global__ void __launch_bounds__(kSelectThreads) select_hint_kernel(const float *__restrict__ G, int F, int K,
                                                                      float *__restrict__ hint) {
    extern __shared__ __align__(16) uint32_t select_keys[];
    __shared__ SelectSmem sm;
    for (int j = threadIdx.x; j < F; j += kSelectThreads) select_keys[j] = gate_key(G[j]);
    __syncthreads();
    uint32_t tau;
    int need;
    block_radix_threshold<kSelectThreads>(select_keys, F, K, sm, tau, need);
    if (threadIdx.x == 0) {
        const float t = key_to_float(tau);
        hint[0] = t;  // +-inf stays non-finite and is rejected by guess_from_hint
        hint[1] = 0.15f * fabsf(t) + 1e-30f;
    }
}

// ------------------------------------------------------------------------------------------------
// Forward selector for rows of at most NV * 128 channels: ONE WARP per token, the row's keys live in
// registers (NV float4 loads per lane), no block barriers.  Same outputs as the CTA-per-token kernel
// below.  Threshold: bracket from the hint / the warp's previous row, verified by counting; inside
// the bracket an exact bitwise search over the few keys it holds; if the bracket fails, the same
// bitwise search over all registers.  Emission is an ordered warp scan, so indices come out
// ascending and ties go to the lower channel.
constexpr int kWarpSelCand = 384;

template <int NV>
__global__ void __launch_bounds__(256) select_mask_rows_warp_kernel(
    const float *__restrict__ G, int ldg, __nv_bfloat16 *__restrict__ U, int ldu, int64_t rows, int F, int K,
    int16_t *__restrict__ idx_out, __nv_bfloat16 *__restrict__ g_out, __nv_bfloat16 *__restrict__ u_out,
    const float *__restrict__ hint) {
    extern __shared__ __align__(16) uint32_t warp_sel_smem[];  // per warp: kWarpSelCand + 2 K words
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    uint32_t *cand = warp_sel_smem + (size_t)wib * (kWarpSelCand + 2 * K);
    uint32_t *packed = cand + kWarpSelCand;  // [K] key of the kept channel, later its z (bf16 bits)
    uint32_t *packed_j = packed + K;         // [K] channel
    const uint32_t lt_mask = (1u << lane) - 1u;
    const int64_t gw = (int64_t)blockIdx.x * 8 + wib, nw = (int64_t)gridDim.x * 8;
    SelectGuess guess = guess_from_hint(hint);

    for (int64_t r = gw; r < rows; r += nw) {
        const float *g = G + r * (int64_t)ldg;
        __nv_bfloat16 *u = U + r * (int64_t)ldu;
        // ---- keys: lane holds channels (v*32 + lane)*4 .. +3 of every 128-channel group v
        uint32_t key[NV][4];
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int c0 = (v * 32 + lane) * 4;
            float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
            if (c0 < F) f = *reinterpret_cast<const float4 *>(g + c0);
            key[v][0] = c0 + 0 < F ? gate_key(f.x) : 0u;
            key[v][1] = c0 + 1 < F ? gate_key(f.y) : 0u;
            key[v][2] = c0 + 2 < F ? gate_key(f.z) : 0u;
            key[v][3] = c0 + 3 < F ? gate_key(f.w) : 0u;
        }
        // ---- bracket: count and collect
        uint32_t tau = 0;
        int need = 0;
        bool solved = false, overflow = false;
        if (guess.valid) {
            const uint32_t lo = gate_key(guess.center - guess.delta), hi = gate_key(guess.center + guess.delta);
            uint32_t cnt = 0, n_band = 0;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t k32 = key[v][e];
                    const bool above = k32 > hi, not_below = k32 >= lo;
                    cnt += (above ? 1u : 0u) + (not_below ? 0x10000u : 0u);
                    const bool band = not_below && !above;
                    const uint32_t b = __ballot_sync(0xffffffffu, band);
                    if (b) {
                        const uint32_t slot = n_band + (uint32_t)__popc(b & lt_mask);
                        if (band && slot < (uint32_t)kWarpSelCand) cand[slot] = k32;
                        n_band += (uint32_t)__popc(b);
                    }
                }
            }
            cnt = __reduce_add_sync(0xffffffffu, cnt);
            const uint32_t c_hi = cnt & 0xffffu, c_lo = cnt >> 16;
            overflow = n_band > (uint32_t)kWarpSelCand;
            solved = c_hi < (uint32_t)K && c_lo >= (uint32_t)K && !overflow;
            if (solved) {
                __syncwarp();
                const uint32_t m = (uint32_t)K - c_hi;
                uint32_t res = hi;
                if (lo != hi) {
                    const int top = 31 - __clz(lo ^ hi);
                    res = hi & ~((2u << top) - 1u);
                    for (int bit = top; bit >= 0; --bit) {
                        const uint32_t trial = res | (1u << bit);
                        uint32_t c = 0;
                        for (uint32_t i = lane; i < n_band; i += 32) c += cand[i] >= trial ? 1u : 0u;
                        c = __reduce_add_sync(0xffffffffu, c);
                        if (c >= m) res = trial;
                    }
                }
                uint32_t gt = 0;
                for (uint32_t i = lane; i < n_band; i += 32) gt += cand[i] > res ? 1u : 0u;
                gt = __reduce_add_sync(0xffffffffu, gt);
                tau = res;
                need = (int)(m - gt);
            }
        }
        if (!solved) {
            // exact K-th largest by bitwise search over the registers
            uint32_t res = 0;
#pragma unroll 1
            for (int bit = 31; bit >= 0; --bit) {
                const uint32_t trial = res | (1u << bit);
                uint32_t c = 0;
#pragma unroll
                for (int v = 0; v < NV; ++v)
#pragma unroll
                    for (int e = 0; e < 4; ++e) c += key[v][e] >= trial ? 1u : 0u;
                c = __reduce_add_sync(0xffffffffu, c);
                if (c >= (uint32_t)K) res = trial;
            }
            uint32_t gt = 0;
#pragma unroll
            for (int v = 0; v < NV; ++v)
#pragma unroll
                for (int e = 0; e < 4; ++e) gt += key[v][e] > res ? 1u : 0u;
            gt = __reduce_add_sync(0xffffffffu, gt);
            tau = res;
            need = K - (int)gt;
        }
        // ---- ordered emission (group v, then lane, then element)
        uint32_t run_gt = 0, run_eq = 0;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            uint32_t local = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e)
                local += (key[v][e] > tau ? 1u : 0u) + (key[v][e] == tau ? 0x10000u : 0u);
            uint32_t inc = local;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t nb = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += nb;
            }
            const uint32_t total = __shfl_sync(0xffffffffu, inc, 31);
            if (local) {
                uint32_t gt_b = run_gt + ((inc - local) & 0xffffu), eq_b = run_eq + ((inc - local) >> 16);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint32_t k32 = key[v][e];
                    const bool gt = k32 > tau, eq = k32 == tau;
                    if (gt || (eq && eq_b < (uint32_t)need)) {
                        // only shared-memory stores here: global loads inside this ordered walk would
                        // serialise one memory round trip per element
                        const int pos = (int)(gt_b + min(eq_b, (uint32_t)need));
                        packed[pos] = k32;
                        packed_j[pos] = (uint32_t)((v * 32 + lane) * 4 + e);
                    }
                    gt_b += gt ? 1u : 0u;
                    eq_b += eq ? 1u : 0u;
                }
            }
            run_gt += total & 0xffffu;
            run_eq += total >> 16;
        }
        __syncwarp();
        // ---- values of the kept channels: independent iterations, so the scattered loads of u overlap;
        //      the compact outputs are written with consecutive lanes on consecutive slots
#pragma unroll 4
        for (int i = lane; i < K; i += 32) {
            const uint32_t j = packed_j[i];
            const float gv = key_to_float(packed[i]);
            const __nv_bfloat16 ub = u[j];
            const __nv_bfloat16 zb = __float2bfloat16_rn(silu_f(gv) * __bfloat162float(ub));
            packed[i] = (uint32_t)(*reinterpret_cast<const uint16_t *>(&zb));
            if (idx_out) {
                idx_out[r * K + i] = (int16_t)j;
                g_out[r * K + i] = __float2bfloat16_rn(gv);
                u_out[r * K + i] = ub;
            }
        }
        __syncwarp();
        // ---- U row -> masked Z' in place
        uint4 *row16 = reinterpret_cast<uint4 *>(u);
        for (int i = lane; i < (ldu >> 3); i += 32) row16[i] = make_uint4(0, 0, 0, 0);
        __syncwarp();
        for (int i = lane; i < K; i += 32) {
            const uint16_t zb = (uint16_t)packed[i];
            u[packed_j[i]] = *reinterpret_cast<const __nv_bfloat16 *>(&zb);
        }
        __syncwarp();
        // ---- next row's bracket
        const float t = key_to_float(tau);
        if (!(fabsf(t) <= 3.0e38f)) {
            guess.valid = false;
        } else if (!guess.valid) {
            guess.center = t;
            guess.delta = 0.15f * fabsf(t) + 1e-30f;
            guess.valid = true;
        } else {
            const float err = fabsf(t - guess.center);
            guess.delta = solved ? 0.9f * guess.delta + 0.44f * err
                                 : (overflow ? 0.5f * guess.delta : 2.0f * err + guess.delta);
            guess.delta = fminf(fmaxf(guess.delta, 1e-30f), 1.0e37f);
            guess.center = t;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Forward selector of the tensor-core plan, one CTA per token.
//   G [rows, ldg] fp32 and U [rows, ldu] bf16 are the dense projections of the token chunk.
//   Emits idx / g / u of the K kept channels (when saving) and rewrites the token's U row IN PLACE
//   into the masked hidden Z' = SiLU(g) u on the kept channels, 0 elsewhere -- the A operand of the
//   down projection.
__global__ void __launch_bounds__(kSelectThreads) select_mask_rows_kernel(
    const float *__restrict__ G, int ldg, __nv_bfloat16 *__restrict__ U, int ldu, int64_t rows, int F, int K,
    int16_t *__restrict__ idx_out, __nv_bfloat16 *__restrict__ g_out, __nv_bfloat16 *__restrict__ u_out,
    const float *__restrict__ hint) {
    extern __shared__ __align__(16) uint32_t select_keys[];  // F keys, then K packed (z bf16, j) entries
    __shared__ SelectSmem sm;
    uint32_t *packed = select_keys + F;
    SelectGuess guess = guess_from_hint(hint);
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        const float *g = G + r * (int64_t)ldg;
        __nv_bfloat16 *u = U + r * (int64_t)ldu;
        uint32_t tau;
        int need;
        block_select_row<kSelectThreads>(g, F, K, select_keys, sm, guess, tau, need);
        // the ordered walk only records the kept channels; values are fetched afterwards in independent
        // iterations so that the scattered loads overlap
        block_ordered_emit<kSelectThreads>(select_keys, F, tau, need, sm,
                                           [&](int pos, int j) { packed[pos] = (uint32_t)j; });
        __syncthreads();
#pragma unroll 4
        for (int i = threadIdx.x; i < K; i += kSelectThreads) {
            const uint32_t j = packed[i];
            const float gv = key_to_float(select_keys[j]);
            const __nv_bfloat16 ub = u[j];
            const __nv_bfloat16 zb = __float2bfloat16_rn(silu_f(gv) * __bfloat162float(ub));
            packed[i] = ((uint32_t)(*reinterpret_cast<const uint16_t *>(&zb)) << 16) | j;
            if (idx_out) {
                idx_out[r * K + i] = (int16_t)j;
                g_out[r * K + i] = __float2bfloat16_rn(gv);
                u_out[r * K + i] = ub;
            }
        }
        __syncthreads();
        // zero the row (ldu is a multiple of 8 and the row start is 16-byte aligned), then scatter Z'
        uint4 *row16 = reinterpret_cast<uint4 *>(u);
        for (int v = threadIdx.x; v < (ldu >> 3); v += kSelectThreads) row16[v] = make_uint4(0, 0, 0, 0);
        __syncthreads();
        for (int k = threadIdx.x; k < K; k += kSelectThreads) {
            const uint32_t e = packed[k];
            const uint16_t zb = (uint16_t)(e >> 16);
            u[e & 0xffffu] = *reinterpret_cast<const __nv_bfloat16 *>(&zb);
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// Backward element-wise step, one CTA per token (Eqs. (bp-1)..(bp-3) on the mask, with S' and Z'
// recomputed from the saved values):
//   dz = dZ[t, j] for each saved channel j, s = SiLU(g), z = s u, dU = s dz, dG = u dz SiLU'(g).
// dZ [T, ld] is the dense product dD Wd^T; its row is read at the saved indices only and then
// overwritten IN PLACE by the masked Z'; dU' and dG' rows are written masked (zeros elsewhere).
// A saved index outside [0, F) is skipped and raises MOC_ERR_BAD_INDEX.
__global__ void __launch_bounds__(256) backward_sample_rows_kernel(
    const int16_t *__restrict__ idx, const __nv_bfloat16 *__restrict__ gval, const __nv_bfloat16 *__restrict__ uval,
    int64_t T, int K, int F, int ld, __nv_bfloat16 *__restrict__ dz_z, __nv_bfloat16 *__restrict__ du,
    __nv_bfloat16 *__restrict__ dg, int *__restrict__ status) {
    extern __shared__ __align__(16) uint32_t sample_smem[];  // K x {j | z<<16, dU | dG<<16}
    for (int64_t t = blockIdx.x; t < T; t += gridDim.x) {
        __nv_bfloat16 *zr = dz_z + t * (int64_t)ld, *ur = du + t * (int64_t)ld, *gr = dg + t * (int64_t)ld;
        for (int k = threadIdx.x; k < K; k += 256) {
            const int j = idx[t * K + k];
            uint32_t w0 = 0xffffu, w1 = 0;  // j = 0xffff marks a skipped entry
            if (j >= 0 && j < F) {
                const float dz = __bfloat162float(zr[j]);
                const float g = __bfloat162float(gval[t * K + k]);
                const float u = __bfloat162float(uval[t * K + k]);
                const float s = silu_f(g);
                const __nv_bfloat16 zb = __float2bfloat16_rn(s * u);
                w0 = (uint32_t)j | ((uint32_t)(*reinterpret_cast<const uint16_t *>(&zb)) << 16);
                w1 = pack_bf16(s * dz, u * dz * dsilu_f(g));
            } else {
                raise_status(status, MOC_ERR_BAD_INDEX);
            }
            sample_smem[2 * k] = w0;
            sample_smem[2 * k + 1] = w1;
        }
        __syncthreads();
        uint4 *z16 = reinterpret_cast<uint4 *>(zr), *u16 = reinterpret_cast<uint4 *>(ur),
              *g16 = reinterpret_cast<uint4 *>(gr);
        const uint4 zero = make_uint4(0, 0, 0, 0);
        for (int v = threadIdx.x; v < (ld >> 3); v += 256) {
            z16[v] = zero;
            u16[v] = zero;
            g16[v] = zero;
        }
        __syncthreads();
        for (int k = threadIdx.x; k < K; k += 256) {
            const uint32_t w0 = sample_smem[2 * k], w1 = sample_smem[2 * k + 1];
            const uint32_t j = w0 & 0xffffu;
            if (j == 0xffffu) continue;
            const uint16_t zb = (uint16_t)(w0 >> 16), ub = (uint16_t)(w1 & 0xffffu), gb = (uint16_t)(w1 >> 16);
            zr[j] = *reinterpret_cast<const __nv_bfloat16 *>(&zb);
            ur[j] = *reinterpret_cast<const __nv_bfloat16 *>(&ub);
            gr[j] = *reinterpret_cast<const __nv_bfloat16 *>(&gb);
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
struct TcForwardLayout {
    int64_t chunk;  // tokens per gate/up pass
    int ldf;        // leading dimension of the dense [*, F] arrays (multiple of 8)
    size_t off_g;   // fp32 G of one chunk [chunk, ldf]
    size_t off_u;   // bf16 U, rewritten in place into Z', for ALL tokens [T, ldf]
    size_t off_hint;  // two floats: threshold hint of the call (see select_hint_kernel)
    size_t total;
};
struct TcBackwardLayout {
    int ldf;
    size_t off_z, off_du, off_dg, total;  // three dense bf16 [T, ldf] arrays
};

inline int round_up8(int v) { return (v + 7) & ~7; }

inline TcForwardLayout tc_forward_layout(const moc_ffn_desc &d) {
    TcForwardLayout L{};
    L.ldf = round_up8(d.d_ff);
    // Tokens go through the gate/up GEMM and the selector in chunks whose G (fp32) + U (bf16) stay
    // around 96 MiB, so that the selector reads them back while they are still in L2.  Among the
    // chunk sizes near that budget, take the one whose tile count fills whole waves of the GPU best.
    const size_t per_token = (size_t)L.ldf * 6;
    const int n_tiles = 2 * ((d.d_ff + BN - 1) / BN);
    const int64_t all_m = (d.tokens + BM - 1) / BM;
    int64_t hi = std::max<int64_t>(1, (int64_t)(((size_t)96 << 20) / per_token) / BM);
    hi = std::min(hi, all_m);
    const int64_t lo = std::max<int64_t>(1, hi - hi / 3);
    const int sms = sm_count();
    int64_t best = hi;
    double best_eff = 0.0;
    for (int64_t m = hi; m >= lo; --m) {
        const int64_t tiles = m * n_tiles;
        const double eff = (double)tiles / (double)(((tiles + sms - 1) / sms) * sms);
        if (eff > best_eff + 1e-9) {
            best_eff = eff;
            best = m;
        }
    }
    L.chunk = best * BM;
    size_t off = 0;
    L.off_g = off;
    off = align_up(off + (size_t)L.chunk * L.ldf * 4, 256);
    L.off_u = off;
    off = align_up(off + (size_t)all_m * BM * L.ldf * 2, 256);
    L.off_hint = off;
    off += 256;
    L.total = off;
    return L;
}

inline TcBackwardLayout tc_backward_layout(const moc_ffn_desc &d) {
    TcBackwardLayout L{};
    L.ldf = round_up8(d.d_ff);
    const size_t dense = align_up((size_t)d.tokens * L.ldf * 2, 256);
    size_t off = 0;
    L.off_z = off;
    off += dense;
    L.off_du = off;
    off += dense;
    L.off_dg = off;
    off += dense;
    L.total = off;
    return L;
}

}  // namespace tc
}  // namespace moc
