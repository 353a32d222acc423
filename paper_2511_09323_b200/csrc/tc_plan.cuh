// Tensor-core plan of the MoC FFN for bf16 training shapes: "compute dense on tcgen05, keep compact".
// At 12.5 % unstructured density the tensor cores finish the dense contraction several times faster
// than the ALUs finish the sparse one, so every contraction runs as a dense GEMM over the full
// channel range and the Top-K structure is applied around it: the forward selects from the fp32
// gate rows and turns the dense up projection into the masked Z' in place; the backward samples the
// dense dD Wd^T at the saved indices in a per-token kernel that also writes the masked dU' and dG' rows
// the gradient GEMMs contract.  Only idx / g / u in compact [T,K] form leave the forward; all dense
// [T,F] arrays are transient workspace.  The per-token kernels stage a token's rows in shared memory
// with bulk async copies and give each token a warp or a team of two or four warps.
#pragma once

#include <cuda.h>
#include <cstdlib>
#include <cstring>
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

// CTA pairs (clusters of two, one MMA across both) are the default; MOC_FFN_GEMM=single in the environment selects
// the one-CTA kernel (kept for comparison and for devices that refuse the cluster launch).
inline bool pair_mode() {
    static int mode = -1;
    if (mode < 0) {
        const char *e = getenv("MOC_FFN_GEMM");
        mode = (e && strcmp(e, "single") == 0) ? 0 : 1;
    }
    return mode == 1;
}
// rows of a K-major B box: a CTA of a pair stages half of the 256 B rows of a tile
inline int b_box_rows() { return pair_mode() ? BN / 2 : BN; }

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

// Output [rows, cols] with leading dimension ld as 32-row boxes of 128 bytes.  False when the tensor-map rules
// (16-byte aligned base and row pitch) do not hold.
inline bool make_out_map(CUtensorMap *m, void *ptr, int64_t rows, int64_t cols, int64_t ld, bool f32) {
    EncodeTiledFn fn = encode_fn();
    const size_t esz = f32 ? 4 : 2;
    if (!fn || (reinterpret_cast<uintptr_t>(ptr) & 15u) || ((size_t)ld * esz) % 16 != 0 || rows <= 0 || cols <= 0)
        return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * esz};
    cuuint32_t box[2] = {(cuuint32_t)(128 / esz), 32};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ptr, dims, strides, box,
              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <bool A_MN, bool B_MN, int EPI>
inline int launch_gemm(const Params &p_in, cudaStream_t st) {
    Params p = p_in;
    p.direct_store = 0;
    for (int i = 0; i < p.num_problems && !p.direct_store; ++i) {
        const bool f32 = EPI == EPI_F32 || (EPI == EPI_GATE_UP && i == 0);
        if (!make_out_map(&p.c_map[i], p.c[i], p.M, p.N, p.ldc[i], f32)) p.direct_store = 1;
    }
    if (pair_mode() && !(p.single_cta && A_MN && B_MN)) {  // K-major B boxes are sized for the mode: no choice there
        auto kern = gemm_pair_kernel<A_MN, B_MN, EPI>;
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.blockDim = dim3(pair_threads(EPI));
        cfg.dynamicSmemBytes = SMEM_BYTES;
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        static int max_pairs = 0;  // pairs that can be resident at once
        if (!max_pairs) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess)
                return MOC_ERR_CUDA;
            cfg.gridDim = dim3(2 * (unsigned)sm_count());
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) return MOC_ERR_CUDA;
            max_pairs = n;
        }
        const int tiles = ((p.m_tiles + 1) / 2) * p.n_tiles * p.num_problems;
        const int pairs = tiles < max_pairs ? tiles : max_pairs;
        if (pairs <= 0) return MOC_OK;
        cfg.gridDim = dim3(2 * (unsigned)pairs);
        return cudaLaunchKernelEx(&cfg, kern, p) == cudaSuccess ? MOC_OK : MOC_ERR_CUDA;
    }
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
// Forward selector for rows that fit a slice of shared memory: a TEAM of two or four warps per token, no block
// barriers (the warps of a team meet at a named barrier of their own).  nv = number of 128-channel groups of a row.
// Same outputs as the CTA-per-token kernel below.
//
// Every team owns a slice of shared memory into which its first thread bulk-copies the token's gate row (fp32)
// and up row (bf16); the team works on those copies, turns the up row into the masked Z' row in place and
// bulk-stores it back.  All global traffic of a row is therefore three asynchronous, fully coalesced
// copies plus the compact outputs, and the scattered accesses of the method (K values per token) stay in
// shared memory.
//
// The launch starts from one bracket [center - width, center + width] that is expected to contain every
// row's threshold; it comes from the thresholds of the previous launch (kept in the workspace).  A row whose
// threshold lies outside moves the bracket (tripling its reach on that side) and tries again; without a
// bracket from an earlier launch a team derives one from the first threshold it finds.  Per row:
//   1. the gate values are classified with plain float compares: values above the bracket are counted,
//      values inside it are parked (raw bits) in the lane's column of shared memory;
//   2. if the counts prove that the K-th largest value is a parked one, a 64-bin histogram over the
//      bracket's key range finds its bin and the few keys of that bin are ranked exactly: threshold tau;
//   3. when no tie has to be cut, the kept set is {g >= tau}: one compare per value, four flags per
//      lane and 128-channel group go to a shared bitmap, which is then enumerated in ascending order;
//   4. values of the kept channels, compact outputs, masked row.
// Rows for which 1-3 do not apply (no bracket yet, too many parked keys, ties to cut, non-finite
// threshold, inconsistent counts) take the general exact path (8-bit radix selection over the
// staged row).  Either way the result is exact: indices ascending, ties to the lower channel.
// Parked values per lane: 14 for rows of up to 2048 channels, growing with the square root of the row length
// (the spread of a row's threshold shrinks with the square root, so the values inside the bracket grow likewise).
__host__ __device__ constexpr int warp_select_slots(int nv) {
    int s = 14;
    while (s * s * 16 < 196 * nv) ++s;  // s >= 14 sqrt(nv / 16)
    return s;
}
__host__ __device__ constexpr int warp_select_cand_words(int nv) {
    return (warp_select_slots(nv) + 1) * 32;  // one more row absorbs the overflow of a column (>= 256: histogram)
}
constexpr int kWarpSelWords = 128;                       // bitmap words, at least (also scratch of the search)
constexpr float kBracketTag = 20251109.0f;

// Words of shared memory one warp needs: gate row, up row, parked keys, bitmap, kept list, mbarrier.
__host__ __device__ constexpr int warp_select_bitmap_words(int nv) { return nv * 4 > kWarpSelWords ? nv * 4 : kWarpSelWords; }
struct SelectMeta {
    float *bracket;      // {center, half width, tag}; rewritten by the last CTA of the launch
    float *acc;          // {sum of thresholds, sum of |threshold - center|, rows}: this launch's statistics
    unsigned int *done;  // CTAs finished
};

// General exact path for one staged row: most-significant-digit radix selection with 8-bit digits.
// g: the row in shared memory (ncols values, channels past the end hold -inf and are never counted because
// only the first F are visited); hist: 256 words of the warp's shared memory.  Leaves the kept channels
// (ascending) in kept[0..K) and returns the threshold key.
__device__ __noinline__ uint32_t warp_select_row_general(const float *g, int F, int K, uint32_t *hist,
                                                         uint32_t *kept) {
    const int lane = threadIdx.x & 31;
    const uint32_t lt_mask = (1u << lane) - 1u;
    uint32_t prefix = 0, kk = (uint32_t)K;  // kk: rank of the threshold among the keys that share the prefix
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        for (int i = lane; i < 256; i += 32) hist[i] = 0u;
        __syncwarp();
        for (int j = lane; j < F; j += 32) {
            const uint32_t key = gate_key(g[j]);
            if (pass == 0 || (key >> (shift + 8)) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
        __syncwarp();
        // lane owns digits 8 lane .. 8 lane + 7; counts of all higher digits come from a suffix scan over lanes
        uint32_t h[8], tot = 0;
#pragma unroll
        for (int b = 0; b < 8; ++b) {
            h[b] = hist[lane * 8 + b];
            tot += h[b];
        }
        uint32_t suf = tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t nb = __shfl_down_sync(0xffffffffu, suf, o);
            if (lane + o < 32) suf += nb;
        }
        uint32_t gt = suf - tot, digit = 0, next_kk = 0;
        bool found = false;
#pragma unroll
        for (int b = 7; b >= 0; --b) {
            const uint32_t ge = gt + h[b];
            if (gt < kk && kk <= ge) {
                found = true;
                digit = (uint32_t)(lane * 8 + b);
                next_kk = kk - gt;
            }
            gt = ge;
        }
        const int src = __ffs(__ballot_sync(0xffffffffu, found)) - 1;  // exactly one lane, since 1 <= kk <= keys left
        digit = __shfl_sync(0xffffffffu, digit, src);
        kk = __shfl_sync(0xffffffffu, next_kk, src);
        prefix = (prefix << 8) | digit;
        __syncwarp();
    }
    const uint32_t res = prefix, need = kk;  // kk keys equal to the threshold are kept, lowest channels first
    uint32_t run_gt = 0, run_eq = 0;
    for (int base = 0; base < F; base += 32) {
        const int j = base + lane;
        const uint32_t key = j < F ? gate_key(g[j]) : 0u;
        const bool isgt = j < F && key > res, iseq = j < F && key == res;
        const uint32_t bg = __ballot_sync(0xffffffffu, isgt), be = __ballot_sync(0xffffffffu, iseq);
        const uint32_t gt_b = run_gt + (uint32_t)__popc(bg & lt_mask), eq_b = run_eq + (uint32_t)__popc(be & lt_mask);
        if (isgt || (iseq && eq_b < need)) kept[gt_b + min(eq_b, need)] = (uint32_t)j;
        run_gt += (uint32_t)__popc(bg);
        run_eq += (uint32_t)__popc(be);
    }
    __syncwarp();
    return res;
}

// ------------------------------------------------------------------------------------------------
// The kernel.  Warp w of a team of W takes the 128-channel groups w, w + W, ... in steps 1 and 3 and every W-th
// batch of kept channels in step 4; the warps meet at the team's named barrier between the steps.  The shared
// memory of an SM bounds the tokens in flight, so W warps per token make it feed W times as many warps (measured
// against one warp per token: 2048 channels 0.086 -> 0.080 ms with pairs; 5504 channels 0.85 -> 0.50 ms and 11008
// channels 0.68 -> 0.41 ms with teams of four).
// shared_u: the up row is copied into the gate row's buffer once the gate values are no longer needed there
// (less shared memory per token, so longer rows still fit; no prefetch of the next gate row).  It is a template
// parameter: as a run-time flag it slowed the common path by a quarter.
__host__ __device__ constexpr size_t pair_select_words(int nv, int K, bool shared_u, int W = 2) {
    return (size_t)nv * 128 + (shared_u ? 0 : (size_t)nv * 64) + (size_t)W * warp_select_cand_words(nv) +
           warp_select_bitmap_words(nv) + (size_t)((K + 3) & ~3) + 40 /* exchange */ + 4 /* two mbarriers */;
}
__host__ __device__ constexpr bool pair_select_parks_gates(int nv, int K, int W = 2) {
    return K <= W * warp_select_cand_words(nv) + warp_select_bitmap_words(nv);
}
constexpr int kPairSelMaxWarps = 12;  // warps per CTA, at most (six pairs or three teams of four; two CTAs per SM)

template <int NV, bool shared_u, int W>
__global__ void __launch_bounds__(kPairSelMaxWarps * 32, 2) select_mask_rows_pair_kernel(
    const float *__restrict__ G, int ldg, __nv_bfloat16 *__restrict__ U, int ldu, int64_t rows, int F, int nv_runtime, int K,
    int16_t *__restrict__ idx_out, __nv_bfloat16 *__restrict__ g_out, __nv_bfloat16 *__restrict__ u_out,
    SelectMeta meta, int *status) {
    extern __shared__ __align__(128) uint32_t warp_sel_smem[];
    static_assert(W == 2 || W == 4, "teams of two or four warps");
    constexpr int TT = 32 * W;  // threads of a team
    __shared__ float s_stat[kPairSelMaxWarps / 2][3];
    __shared__ int s_abort;
    const int nv = NV > 0 ? NV : nv_runtime;
    const int slots = warp_select_slots(nv), cw = warp_select_cand_words(nv);
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5, ppc = blockDim.x / TT;  // teams per CTA
    const int pair = wib / W, w = wib % W, pl = (w << 5) | lane;                       // pl: thread index within the team
    uint32_t *base = warp_sel_smem + (size_t)pair * pair_select_words(nv, K, shared_u, W);
    float *sg = reinterpret_cast<float *>(base);
    __nv_bfloat16 *su = reinterpret_cast<__nv_bfloat16 *>(shared_u ? base : base + nv * 128);
    uint32_t *cand0 = base + nv * 128 + (shared_u ? 0 : nv * 64);  // [W warps][slot][lane] parked values
    uint32_t *cand = cand0 + w * cw;
    uint32_t *bitmap = cand0 + W * cw;
    uint32_t *kept = bitmap + warp_select_bitmap_words(nv);
    uint32_t *xch = kept + ((K + 3) & ~3);  // [2 parities][W warps][4] counts exchanged between the warps
    uint64_t *bar_mem = reinterpret_cast<uint64_t *>(xch + 40);  // (xch[32..35]: the warps' wait verdicts)
    const uint32_t bar_g = smem_u32(bar_mem), bar_u = smem_u32(bar_mem + 1);
    float *gkept = reinterpret_cast<float *>(cand0);
    const bool early_gate = pair_select_parks_gates(nv, K, W);
    auto pair_sync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(pair + 1), "n"(TT) : "memory"); };
    const int64_t gp = (int64_t)blockIdx.x * ppc + pair, np = (int64_t)gridDim.x * ppc;
    const float b_center = meta.bracket[0], b_width = meta.bracket[1];
    const bool have_bracket = meta.bracket[2] == kBracketTag && b_width > 0.f && fabsf(b_center) <= 3.0e38f;
    float cen = b_center, wid = b_width;
    bool have = have_bracket;
    float st_sum = 0.f, st_abs = 0.f, st_n = 0.f;
    const int words = (F + 31) >> 5;
    const uint32_t g_bytes = (uint32_t)ldg * 4u, u_bytes = (uint32_t)ldu * 2u;

    if (threadIdx.x == 0) s_abort = 0;
    if (pl == 0) {
        mbar_init(bar_g, 1);
        mbar_init(bar_u, 1);
    }
    for (int c = ldg + pl; c < nv * 128; c += TT) sg[c] = -INFINITY;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    uint32_t phase = 0;
    int xp = 0;  // parity of the exchange slot in use
    bool dead = false;
    if (pl == 0 && gp < rows && !shared_u) {
        mbar_expect_tx(bar_g, g_bytes);
        bulk_copy_g2s(smem_u32(sg), G + gp * (int64_t)ldg, g_bytes, bar_g);
    }
    // the warps of a team take every branch below together: all conditions come from values they share

    for (int64_t r = gp; r < rows && !dead; r += np) {
        __nv_bfloat16 *u = U + r * (int64_t)ldu;
        if (pl == 0) {
            bulk_store_wait_read<0>();
            fence_async_smem();
            if (shared_u) {
                mbar_expect_tx(bar_g, g_bytes);
                bulk_copy_g2s(smem_u32(sg), G + r * (int64_t)ldg, g_bytes, bar_g);
            } else {
                mbar_expect_tx(bar_u, u_bytes);
                bulk_copy_g2s(smem_u32(su), u, u_bytes, bar_u);
            }
        }
        // a wait that gave up ends the team: the warps exchange their verdicts so that all of them leave together
        // (another team's time-out can make one warp's wait return early and not its partner's)
        const auto team_agrees = [&](bool ok) {
            if (lane == 0) xch[32 + w] = ok ? 1u : 0u;
            pair_sync();
            bool all_ok = true;
#pragma unroll
            for (int i = 0; i < W; ++i) all_ok = all_ok && xch[32 + i] != 0u;
            return all_ok;
        };
        const bool g_ok = __all_sync(0xffffffffu, mbar_wait(bar_g, phase, &s_abort, status));
        if (g_ok)
            for (int c = F + pl; c < ldg; c += TT) sg[c] = -INFINITY;
        if (!team_agrees(g_ok)) {
            dead = true;
            break;
        }

        uint32_t tau = 0, res = 0;
        bool fast = false, settled = false, no_cut = false;
        float lo_f = cen - wid, hi_f = cen + wid;
        for (int attempt = 0; have && attempt < 8; ++attempt) {
            // ---- 1. classify: this warp's groups v = w, w + 2, ...
            uint32_t n_above = 0, n_mine = 0;
#pragma unroll 4
            for (int v = w; v < nv; v += W) {
                const float4 q = *reinterpret_cast<const float4 *>(sg + (v * 32 + lane) * 4);
                const float e4[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float x = e4[e];
                    n_above += x > hi_f ? 1u : 0u;
                    const bool inside = x >= lo_f && x <= hi_f;
                    if (inside) cand[min(n_mine, (uint32_t)slots) * 32 + lane] = __float_as_uint(x);
                    n_mine += inside ? 1u : 0u;
                }
            }
            const uint32_t my_hi = __reduce_add_sync(0xffffffffu, n_above);
            const uint32_t my_band = __reduce_add_sync(0xffffffffu, n_mine);
            const uint32_t my_max = __reduce_max_sync(0xffffffffu, n_mine);
            uint32_t *xs = xch + xp * (4 * W);
            xp ^= 1;
            if (lane == 0) {
                xs[w * 4 + 0] = my_hi;
                xs[w * 4 + 1] = my_band;
                xs[w * 4 + 2] = my_max;
            }
            // scratch of the search, cleared here so that the barrier below also publishes it
            uint32_t *hist = bitmap, *list = bitmap + 64, *list_n = bitmap + 96;
            if (pl < 64) hist[pl] = 0u;
            if (pl == 0) *list_n = 0u;
            pair_sync();
            uint32_t c_hi = 0, n_band = 0, max_mine = 0;
#pragma unroll
            for (int i = 0; i < W; ++i) {
                c_hi += xs[4 * i];
                n_band += xs[4 * i + 1];
                max_mine = max(max_mine, xs[4 * i + 2]);
            }
            if (max_mine > (uint32_t)slots) {  // too many values inside: halve the bracket
                const float c = 0.5f * (lo_f + hi_f), wd = 0.25f * (hi_f - lo_f);
                lo_f = c - wd;
                hi_f = c + wd;
                continue;
            }
            if (c_hi >= (uint32_t)K) {
                const float wd = hi_f - lo_f;
                lo_f = hi_f;
                hi_f += 2.f * wd;
                continue;
            }
            if (c_hi + n_band < (uint32_t)K) {
                const float wd = hi_f - lo_f;
                hi_f = lo_f;
                lo_f -= 2.f * wd;
                continue;
            }
            // ---- 2. histogram of both warps' parked keys, bin of the m-th largest, exact ranking inside it
            //         (both warps compute the scan and the ranking: same inputs, same result, no exchange)
            const uint32_t lo_k = gate_key(lo_f), hi_k = gate_key(hi_f);
            const uint32_t m = (uint32_t)K - c_hi;
            const uint32_t span = hi_k - lo_k;
            const int shift = max(0, 26 - __clz(span | 1u));
            for (uint32_t s = 0; s < n_mine; ++s) {
                const uint32_t key = gate_key(__uint_as_float(cand[s * 32 + lane]));
                atomicAdd(&hist[(key - lo_k) >> shift], 1u);
            }
            pair_sync();
            const uint32_t h0 = hist[2 * lane], h1 = hist[2 * lane + 1], tot = h0 + h1;
            uint32_t suf = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t nb = __shfl_down_sync(0xffffffffu, suf, o);
                if (lane + o < 32) suf += nb;
            }
            const uint32_t above = suf - tot;
            const bool f1 = above < m && m <= above + h1, f0 = above + h1 < m && m <= above + tot;
            const int src = __ffs(__ballot_sync(0xffffffffu, f0 || f1)) - 1;
            const uint32_t tbin = __shfl_sync(0xffffffffu, (uint32_t)(2 * lane + (f1 ? 1 : 0)), src);
            const uint32_t m2 = m - __shfl_sync(0xffffffffu, f1 ? above : above + h1, src);
            const uint32_t nbin = __shfl_sync(0xffffffffu, f1 ? h1 : h0, src);
            if (nbin <= 32u) {
                for (uint32_t s = 0; s < n_mine; ++s) {
                    const uint32_t key = gate_key(__uint_as_float(cand[s * 32 + lane]));
                    if (((key - lo_k) >> shift) == tbin) list[atomicAdd(list_n, 1u)] = key;
                }
                pair_sync();
                const uint32_t mykey = (uint32_t)lane < nbin ? list[lane] : 0u;
                uint32_t n_gt = 0, n_eq = 0;
                for (uint32_t i = 0; i < nbin; ++i) {
                    const uint32_t o = list[i];
                    n_gt += o > mykey ? 1u : 0u;
                    n_eq += o == mykey ? 1u : 0u;
                }
                const bool is_tau = (uint32_t)lane < nbin && n_gt < m2 && m2 <= n_gt + n_eq;
                const int tl = __ffs(__ballot_sync(0xffffffffu, is_tau)) - 1;
                res = __shfl_sync(0xffffffffu, mykey, tl);
                no_cut = __shfl_sync(0xffffffffu, n_gt + n_eq, tl) == m2;
                settled = true;
            }
            break;
        }
        pair_sync();  // the search scratch is about to become the bitmap
        const float tau_f = key_to_float(res);
        if (settled && no_cut && fabsf(tau_f) <= 3.0e38f) {
            // ---- 3. kept set = {g >= tau}: each warp writes the bitmap words of its own groups
            for (int v = w; v < nv; v += W)
                if (lane < 4 && v * 4 + lane < warp_select_bitmap_words(nv)) bitmap[v * 4 + lane] = 0u;
            __syncwarp();
#pragma unroll 4
            for (int v = w; v < nv; v += W) {
                const float4 q = *reinterpret_cast<const float4 *>(sg + (v * 32 + lane) * 4);
                const uint32_t nib = (q.x >= tau_f ? 1u : 0u) | (q.y >= tau_f ? 2u : 0u) |
                                     (q.z >= tau_f ? 4u : 0u) | (q.w >= tau_f ? 8u : 0u);
                if (nib) atomicOr(&bitmap[v * 4 + (lane >> 3)], nib << ((lane & 7) * 4));
            }
            pair_sync();
            // enumerate in ascending channel order: thread pl of the pair owns words [pl*wpl, (pl+1)*wpl)
            const int wpl = (words + TT - 1) / TT;
            uint32_t mine = 0;
            for (int i = 0; i < wpl; ++i) {
                const int wd = pl * wpl + i;
                mine += wd < words ? (uint32_t)__popc(bitmap[wd]) : 0u;
            }
            uint32_t pre = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t nb = __shfl_up_sync(0xffffffffu, pre, o);
                if (lane >= o) pre += nb;
            }
            uint32_t *xs = xch + xp * (4 * W);
            xp ^= 1;
            if (lane == 31) xs[w * 4 + 3] = pre;  // this warp's total
            pair_sync();
            uint32_t total = 0, before = 0;
#pragma unroll
            for (int i = 0; i < W; ++i) {
                total += xs[4 * i + 3];
                before += i < w ? xs[4 * i + 3] : 0u;
            }
            if (total == (uint32_t)K) {  // counts and compares agree
                uint32_t pos = pre - mine + before;
                for (int i = 0; i < wpl; ++i) {
                    const int wd = pl * wpl + i;
                    uint32_t bits = wd < words ? bitmap[wd] : 0u;
                    while (bits) {
                        const int b = __ffs(bits) - 1;
                        bits &= bits - 1u;
                        kept[pos++] = (uint32_t)(wd * 32 + b);
                    }
                }
                tau = res;
                fast = true;
            }
        }
        pair_sync();
        if (!fast) {
            // general exact path (rare): one warp works on the whole row, its partner waits
            if (w == 0) {
                const uint32_t t0 = warp_select_row_general(sg, F, K, cand0, kept);
                if (lane == 0) xch[0] = t0;
            }
            xp = 0;
            pair_sync();
            tau = xch[0];
            pair_sync();
        }
        // ---- 4. values of the kept channels, entries pl, pl + 64, ...
        auto request_next_gate = [&]() {
            if (pl == 0 && r + np < rows) {
                fence_async_smem();
                mbar_expect_tx(bar_g, g_bytes);
                bulk_copy_g2s(smem_u32(sg), G + (r + np) * (int64_t)ldg, g_bytes, bar_g);
            }
        };
        if (early_gate) {
            for (int i = pl; i < K; i += TT) gkept[i] = sg[kept[i]];
            pair_sync();
            if (!shared_u) {
                request_next_gate();
            } else if (pl == 0) {
                fence_async_smem();
                mbar_expect_tx(bar_u, u_bytes);
                bulk_copy_g2s(smem_u32(su), u, u_bytes, bar_u);
            }
        }
        if (!team_agrees(__all_sync(0xffffffffu, mbar_wait(bar_u, phase, &s_abort, status)))) {
            dead = true;
            break;
        }
        phase ^= 1u;
        for (int i = pl; i < K; i += TT) {
            const uint32_t j = kept[i];
            const float gval = early_gate ? gkept[i] : sg[j];
            const __nv_bfloat16 ub = su[j];
            const __nv_bfloat16 zb = __float2bfloat16_rn(silu_f(gval) * __bfloat162float(ub));
            kept[i] = j | ((uint32_t)(*reinterpret_cast<const uint16_t *>(&zb)) << 16);
            if (idx_out) {
                idx_out[r * K + i] = (int16_t)j;
                g_out[r * K + i] = __float2bfloat16_rn(gval);
                u_out[r * K + i] = ub;
            }
        }
        pair_sync();
        if (!early_gate) request_next_gate();
        // ---- up row -> masked Z' row, in shared memory, then one bulk store
        uint4 *row16 = reinterpret_cast<uint4 *>(su);
        for (int i = pl; i < (ldu >> 3); i += TT) row16[i] = make_uint4(0, 0, 0, 0);
        pair_sync();
        for (int i = pl; i < K; i += TT) {
            const uint32_t e = kept[i];
            const uint16_t zb = (uint16_t)(e >> 16);
            su[e & 0xffffu] = *reinterpret_cast<const __nv_bfloat16 *>(&zb);
        }
        fence_async_smem();
        pair_sync();
        if (pl == 0) bulk_copy_s2g(u, smem_u32(su), u_bytes);
        // ---- statistics for the next launch's bracket (kept by both warps, published by the first)
        const float t = key_to_float(tau);
        if (fabsf(t) <= 3.0e38f) {
            st_sum += t;
            st_abs += have_bracket ? fabsf(t - b_center) : 0.f;
            st_n += 1.f;
            if (!have) {
                cen = t;
                wid = 0.15f * fabsf(t) + 1e-30f;
                have = true;
            }
        }
    }
    if (pl == 0) bulk_store_wait_all();
    if (pl == 0) {
        s_stat[pair][0] = st_sum;
        s_stat[pair][1] = st_abs;
        s_stat[pair][2] = st_n;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float a = 0.f, b = 0.f, c = 0.f;
        for (int i = 0; i < ppc; ++i) {
            a += s_stat[i][0];
            b += s_stat[i][1];
            c += s_stat[i][2];
        }
        if (c > 0.f) {
            atomicAdd(&meta.acc[0], a);
            atomicAdd(&meta.acc[1], b);
            atomicAdd(&meta.acc[2], c);
        }
        __threadfence();
        if (atomicInc(meta.done, gridDim.x - 1) == gridDim.x - 1) {
            __threadfence();
            const float sum = atomicAdd(&meta.acc[0], 0.f), dev = atomicAdd(&meta.acc[1], 0.f),
                        n = atomicAdd(&meta.acc[2], 0.f);
            if (n > 0.f) {
                const float center = sum / n;
                float width = have_bracket ? 5.0f * dev / n : 0.15f * fabsf(center);
                width = fmaxf(width, 0.02f * fabsf(center) + 1e-30f);
                meta.bracket[0] = center;
                meta.bracket[1] = width;
                meta.bracket[2] = kBracketTag;
            } else {
                meta.bracket[2] = 0.f;
            }
            meta.acc[0] = meta.acc[1] = meta.acc[2] = 0.f;
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
// The same step with ONE WARP per token and the rows staged in the warp's slice of shared memory: the dZ
// row arrives by a bulk copy (the next token's row is already in flight while this one is worked on), the
// three masked rows are built in shared memory and leave as bulk stores.  Global traffic is fully
// coalesced and the scattered accesses stay on chip.  Used when the four rows of a token fit a slice.
__host__ __device__ constexpr size_t sample_warp_words(int ld, int K) {
    return (size_t)2 * ld /* four bf16 rows */ + (size_t)2 * ((K + 1) & ~1) /* entries */ +
           (size_t)3 * ((K + 7) & ~7) /* saved idx, g, u of two tokens */ + 4 /* two mbarriers */ + 4 /* verdicts */;
}
constexpr int kSampleMaxWarps = 10;

// W warps work on a token (W = 1 or 2: with two, the token's rows occupy the slice for about half as long and the
// same shared memory feeds twice the warps); they meet at a named barrier of their own between the phases.
template <int W>
__global__ void __launch_bounds__(kSampleMaxWarps * 32) backward_sample_rows_warp_kernel(
    const int16_t *__restrict__ idx, const __nv_bfloat16 *__restrict__ gval, const __nv_bfloat16 *__restrict__ uval,
    int64_t T, int K, int F, int ld, __nv_bfloat16 *__restrict__ dz_z, __nv_bfloat16 *__restrict__ du,
    __nv_bfloat16 *__restrict__ dg, int *__restrict__ status) {
    extern __shared__ __align__(128) uint32_t sample_warp_smem[];
    __shared__ int s_abort;
    constexpr int TT = 32 * W;  // threads of a team
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5, wpc = blockDim.x / TT;  // teams per CTA
    const int team = wib / W, pl = ((wib % W) << 5) | lane;                            // pl: thread index within the team
    auto team_sync = [&]() {
        if (W == 1) __syncwarp();
        else asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "n"(TT) : "memory");
    };
    uint32_t *base = sample_warp_smem + (size_t)team * sample_warp_words(ld, K);
    const int row_words = ld >> 1;  // ld is a multiple of 8: rows are multiples of 16 bytes
    __nv_bfloat16 *zbuf0 = reinterpret_cast<__nv_bfloat16 *>(base);  // two dZ rows, used alternately
    __nv_bfloat16 *ubuf = reinterpret_cast<__nv_bfloat16 *>(base + 2 * row_words);
    __nv_bfloat16 *gbuf = reinterpret_cast<__nv_bfloat16 *>(base + 3 * row_words);
    uint32_t *entry = base + 4 * row_words;  // K x {j | z << 16, dU | dG << 16}
    // saved idx | g | u rows of the two tokens in flight, K8 16-bit entries each (arrive with the dZ row when K is a
    // multiple of 8, i.e. when the rows are 16-byte multiples; plain loads otherwise)
    const int K8 = (K + 7) & ~7;
    uint16_t *saved0 = reinterpret_cast<uint16_t *>(entry + 2 * ((K + 1) & ~1));
    const bool staged_saved = (K & 7) == 0;
    uint64_t *bar_mem = reinterpret_cast<uint64_t *>(saved0 + 6 * K8);
    const uint32_t bar0 = smem_u32(bar_mem);  // two mbarriers, 8 bytes apart
    const uint32_t row_bytes = (uint32_t)ld * 2u, saved_bytes = (uint32_t)K * 2u;
    const int64_t gw = (int64_t)blockIdx.x * wpc + team, nw = (int64_t)gridDim.x * wpc;

    if (threadIdx.x == 0) s_abort = 0;
    if (pl == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8u, 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    uint32_t phases = 0;  // bit b: parity to wait for on barrier b
    auto request = [&](int64_t tok, int buf) {  // lane 0: dZ row (+ saved rows) of a token into buffer `buf`
        const uint32_t nbar = bar0 + 8u * (uint32_t)buf;
        mbar_expect_tx(nbar, row_bytes + (staged_saved ? 3u * saved_bytes : 0u));
        bulk_copy_g2s(smem_u32(zbuf0 + (size_t)buf * ld), dz_z + tok * (int64_t)ld, row_bytes, nbar);
        if (staged_saved) {
            uint16_t *sv = saved0 + (size_t)buf * 3 * K8;
            bulk_copy_g2s(smem_u32(sv), idx + tok * K, saved_bytes, nbar);
            bulk_copy_g2s(smem_u32(sv + K8), gval + tok * K, saved_bytes, nbar);
            bulk_copy_g2s(smem_u32(sv + 2 * K8), uval + tok * K, saved_bytes, nbar);
        }
    };
    if (pl == 0 && gw < T) request(gw, 0);
    int b = 0;
    for (int64_t t = gw; t < T; t += nw, b ^= 1) {
        // a wait that gave up ends the team: the warps exchange their verdicts so that all of them leave together
        const bool ok = __all_sync(0xffffffffu, mbar_wait(bar0 + 8u * (uint32_t)b, (phases >> b) & 1u, &s_abort, status));
        if (W > 1) {
            uint32_t *verdict = reinterpret_cast<uint32_t *>(bar_mem + 2);
            if (lane == 0) verdict[wib % W] = ok ? 1u : 0u;
            team_sync();
            bool all_ok = true;
#pragma unroll
            for (int i = 0; i < W; ++i) all_ok = all_ok && verdict[i] != 0u;
            if (!all_ok) break;
        } else if (!ok) {
            break;
        }
        phases ^= 1u << b;
        __nv_bfloat16 *zr = zbuf0 + (size_t)b * ld;
        const uint16_t *sv = saved0 + (size_t)b * 3 * K8;
        for (int k0 = 0; k0 < K; k0 += 8 * TT) {
            // eight saved entries per lane, their loads issued together
            int jv[8];
            __nv_bfloat16 gb[8], ub[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int k = k0 + i * TT + pl;
                jv[i] = -1;
                if (k < K) {
                    if (staged_saved) {
                        jv[i] = (int16_t)sv[k];
                        gb[i] = *reinterpret_cast<const __nv_bfloat16 *>(sv + K8 + k);
                        ub[i] = *reinterpret_cast<const __nv_bfloat16 *>(sv + 2 * K8 + k);
                    } else {
                        jv[i] = idx[t * K + k];
                        gb[i] = gval[t * K + k];
                        ub[i] = uval[t * K + k];
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int k = k0 + i * TT + pl;
                if (k >= K) continue;
                const int j = jv[i];
                uint32_t w0 = 0xffffu, w1 = 0;  // j = 0xffff marks a skipped entry
                if (j >= 0 && j < F) {
                    const float dz = __bfloat162float(zr[j]);
                    const float g = __bfloat162float(gb[i]);
                    const float u = __bfloat162float(ub[i]);
                    const float s = silu_f(g);
                    const __nv_bfloat16 zb = __float2bfloat16_rn(s * u);
                    w0 = (uint32_t)j | ((uint32_t)(*reinterpret_cast<const uint16_t *>(&zb)) << 16);
                    w1 = pack_bf16(s * dz, u * dz * dsilu_f(g));
                } else {
                    raise_status(status, MOC_ERR_BAD_INDEX);
                }
                entry[2 * k] = w0;
                entry[2 * k + 1] = w1;
            }
        }
        // by now the stores of the previous token have read their rows: the other dZ buffer (next token's row goes
        // there) and the dU / dG rows are free
        team_sync();  // every thread has sampled the dZ row
        if (pl == 0) {
            bulk_store_wait_read<0>();
            fence_async_smem();
            if (t + nw < T) request(t + nw, b ^ 1);
        }
        team_sync();
        {
            uint4 *z16 = reinterpret_cast<uint4 *>(zr), *u16 = reinterpret_cast<uint4 *>(ubuf),
                  *g16 = reinterpret_cast<uint4 *>(gbuf);
            const uint4 zero = make_uint4(0, 0, 0, 0);
            for (int v = pl; v < (ld >> 3); v += TT) {
                z16[v] = zero;
                u16[v] = zero;
                g16[v] = zero;
            }
        }
        team_sync();
        for (int k = pl; k < K; k += TT) {
            const uint32_t w0 = entry[2 * k], w1 = entry[2 * k + 1];
            const uint32_t j = w0 & 0xffffu;
            if (j == 0xffffu) continue;
            const uint16_t zb = (uint16_t)(w0 >> 16), ub = (uint16_t)(w1 & 0xffffu), gb = (uint16_t)(w1 >> 16);
            zr[j] = *reinterpret_cast<const __nv_bfloat16 *>(&zb);
            ubuf[j] = *reinterpret_cast<const __nv_bfloat16 *>(&ub);
            gbuf[j] = *reinterpret_cast<const __nv_bfloat16 *>(&gb);
        }
        fence_async_smem();
        team_sync();
        if (pl == 0) {
            bulk_copy_s2g(dz_z + t * (int64_t)ld, smem_u32(zr), row_bytes);
            bulk_copy_s2g(du + t * (int64_t)ld, smem_u32(ubuf), row_bytes);
            bulk_copy_s2g(dg + t * (int64_t)ld, smem_u32(gbuf), row_bytes);
        }
    }
    if (pl == 0) bulk_store_wait_all();
}

// ------------------------------------------------------------------------------------------------
struct TcForwardLayout {
    int64_t chunk;  // tokens per gate/up pass
    int ldf;        // leading dimension of the dense [*, F] arrays (multiple of 8)
    size_t off_g;   // fp32 G of one chunk [chunk, ldf]
    size_t off_u;   // bf16 U, rewritten in place into Z', for ALL tokens [T, ldf]
    size_t off_hint;  // bracket {center, width, tag}, statistics {sum, sum|dev|, rows}, CTA counter
    // MoC 2:8 on the sparse MMA: Z' in compressed form lives where U would (it is half as large), its metadata here
    size_t off_meta, meta_bytes;
    int sp_k_stages;  // blocks of 128 channels
    size_t total;
};
struct TcBackwardLayout {
    int ldf;
    size_t off_z, off_du, off_dg, total;  // three dense bf16 [T, ldf] arrays
    size_t off_small, small_bytes;        // batches of up to 256 tokens: fp32 accumulator [T, d] + counters of the dX kernel
    // MoC 2:8 with grad_x on the sparse MMA: dG' and dU' in compressed form [T, F / 2] with their metadata (sp_bytes == 0:
    // not used)
    size_t off_gc, off_uc, off_gmeta, off_umeta, sp_bytes;
    size_t off_split, split_bytes;        // a few hundred tokens: two fp32 partial outputs [T, d] of the grad_x GEMM
};

inline int round_up8(int v) { return (v + 7) & ~7; }

// grad_x of the MoC 2:8 variant on the sparse MMA is built and checked but off by default: compressing dG' and dU' costs
// what the shorter GEMM saves (LLaMA-1B shape, 65536 tokens: grad_x 2.14 -> 1.38 ms, two compression passes 0.8 ms).
// MOC_FFN_SPARSE_DX=1 in the environment turns it on.
inline bool sparse_dx_requested() {
    static const bool on = [] {
        const char *e = getenv("MOC_FFN_SPARSE_DX");
        return e && strcmp(e, "1") == 0;
    }();
    return on;
}

inline TcForwardLayout tc_forward_layout(const moc_ffn_desc &d) {
    TcForwardLayout L{};
    L.ldf = round_up8(d.d_ff);
    // Tokens go through the gate/up GEMM and the selector in as few equal chunks as keep the transient fp32 G and
    // the chunk's U within 1.25 GiB.  (Fewer, longer launches measured faster than chunks small enough for G to
    // stay in L2: LLaMA-130M shapes 0.109 -> 0.087 ms for the GEMM and 0.114 -> 0.091 ms for the selector.)
    const size_t per_token = (size_t)L.ldf * 6;
    const int64_t all_m = (d.tokens + BM - 1) / BM;
    // MOC_FFN_FWD_CHUNK_MIB in the environment overrides the bound (smaller workspace, more launches)
    size_t bound_mib = 1280;
    if (const char *e = getenv("MOC_FFN_FWD_CHUNK_MIB")) {
        const long v = atol(e);
        if (v >= 1 && v <= (1 << 20)) bound_mib = (size_t)v;
    }
    int64_t hi = std::max<int64_t>(1, (int64_t)((bound_mib << 20) / per_token) / BM);
    hi = std::min(hi, all_m);
    const int64_t n_chunks = (all_m + hi - 1) / hi;
    const int64_t best = (all_m + n_chunks - 1) / n_chunks;  // equal chunks
    L.chunk = best * BM;
    size_t off = 0;
    L.off_g = off;
    off = align_up(off + (size_t)L.chunk * L.ldf * 4, 256);
    L.off_u = off;
    off = align_up(off + (size_t)all_m * BM * L.ldf * 2, 256);
    L.off_hint = off;
    off += 256;
    L.sp_k_stages = (d.d_ff + 127) / 128;
    L.off_meta = off;
    L.meta_bytes = (d.flags & MOC_FLAG_SELECT_2_OF_8) ? align_up((size_t)all_m * L.sp_k_stages * 128 * 16, 256) : 0;
    off += L.meta_bytes;
    L.total = off;
    return L;
}

// A GEMM whose output has so few tiles that half of the CTA pairs would idle (a few hundred tokens: 32 tiles of
// 256 x 256 for 512 tokens and d_model = 4096, each with the whole d_ffn to contract) is split in two along its
// contraction: the halves run as two problems of one launch into fp32 partial outputs, which a small kernel adds.
// MOC_FFN_SPLIT_K=0 in the environment switches the split off (comparisons).
inline bool split_contraction_pays(int64_t T, int n_cols) {
    static const bool on = [] {
        const char *e = getenv("MOC_FFN_SPLIT_K");
        return !(e && atoi(e) == 0);
    }();
    if (!on || !pair_mode() || (n_cols & 7)) return false;
    const int64_t tiles = ((T + BM - 1) / BM + 1) / 2 * ((n_cols + BN - 1) / BN);
    return 2 * tiles <= sm_count() / 2;
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
    L.off_small = off;
    L.small_bytes = d.tokens <= 256 ? align_up((size_t)d.tokens * d.d_model * sizeof(float) + 1024, 256) : 0;
    off += L.small_bytes;
    L.sp_bytes = 0;
    if ((d.flags & MOC_FLAG_SELECT_2_OF_8) && sparse_dx_requested() && !L.small_bytes) {
        const size_t rows = (size_t)((d.tokens + 127) / 128) * 128;
        const size_t k_stages = (size_t)(d.d_ff + 127) / 128;
        const size_t comp = align_up(rows * k_stages * 64 * 2, 256), meta = align_up(rows / 128 * k_stages * 2048, 256);
        L.off_gc = off;
        L.off_uc = off + comp;
        L.off_gmeta = off + 2 * comp;
        L.off_umeta = off + 2 * comp + meta;
        L.sp_bytes = 2 * comp + 2 * meta;
        off += L.sp_bytes;
    }
    // fp32 partial outputs of the grad_x GEMM when its contraction is split (its two segments as two problems)
    L.off_split = off;
    L.split_bytes = (!L.small_bytes && !L.sp_bytes && split_contraction_pays(d.tokens, d.d_model))
                        ? align_up((size_t)2 * d.tokens * d.d_model * sizeof(float), 256) : 0;
    off += L.split_bytes;
    L.total = off;
    return L;
}

}  // namespace tc
}  // namespace moc
