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
// Forward selector of the tensor-core plan, one CTA per token.
//   G [rows, ldg] fp32 and U [rows, ldu] bf16 are the dense projections of the token chunk.
//   Emits idx / g / u of the K kept channels (when saving) and rewrites the token's U row IN PLACE
//   into the masked hidden Z' = SiLU(g) u on the kept channels, 0 elsewhere -- the A operand of the
//   down projection.
__global__ void __launch_bounds__(kSelectThreads) select_mask_rows_kernel(
    const float *__restrict__ G, int ldg, __nv_bfloat16 *__restrict__ U, int ldu, int64_t rows, int F, int K,
    int16_t *__restrict__ idx_out, __nv_bfloat16 *__restrict__ g_out, __nv_bfloat16 *__restrict__ u_out) {
    extern __shared__ __align__(16) uint32_t select_keys[];  // F keys, then K packed (z bf16, j) entries
    __shared__ SelectSmem sm;
    uint32_t *packed = select_keys + F;
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        const float *g = G + r * (int64_t)ldg;
        __nv_bfloat16 *u = U + r * (int64_t)ldu;
        for (int j = threadIdx.x; j < F; j += kSelectThreads) select_keys[j] = gate_key(g[j]);
        __syncthreads();
        uint32_t tau;
        int need;
        block_radix_threshold<kSelectThreads>(select_keys, F, K, sm, tau, need);
        block_ordered_emit<kSelectThreads>(select_keys, F, tau, need, sm, [&](int pos, int j) {
            const float gv = g[j];
            const __nv_bfloat16 ub = u[j];
            const float z = silu_f(gv) * __bfloat162float(ub);
            const __nv_bfloat16 zb = __float2bfloat16_rn(z);
            packed[pos] = ((uint32_t)(*reinterpret_cast<const uint16_t *>(&zb)) << 16) | (uint32_t)j;
            if (idx_out) {
                idx_out[r * K + pos] = (int16_t)j;
                g_out[r * K + pos] = __float2bfloat16_rn(gv);
                u_out[r * K + pos] = ub;
            }
        });
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
// Backward helper: validates the saved indices (in range, strictly ascending) and records, per token
// and per 256-column tile of the channel range, where that tile's entries start in the token's list.
__global__ void __launch_bounds__(256) tile_start_kernel(const int16_t *__restrict__ idx, int64_t T, int K, int F,
                                                         int n_tiles, int32_t *__restrict__ tile_start,
                                                         int *__restrict__ status) {
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);  // warp per token
    if (t >= T) return;
    const int16_t *row = idx + t * K;
    int32_t *ts = tile_start + t * n_tiles;
    bool bad = false;
    for (int k = lane; k < K; k += 32) {
        const int j = row[k];
        const int prev = k > 0 ? (int)row[k - 1] : -1;
        if (j < 0 || j >= F || j <= prev) bad = true;
        // entry k is the first of every tile b with  prev < b*BN <= j
        if (!bad) {
            const int b_lo = prev < 0 ? 0 : prev / BN + 1;
            const int b_hi = j / BN;
            for (int b = b_lo; b <= b_hi && b < n_tiles; ++b) ts[b] = k;
        }
    }
    // tiles after the last entry start at K
    if (lane == 0) {
        const int last = (int)row[K - 1];
        const int b0 = (last < 0 || last >= F) ? 0 : last / BN + 1;
        for (int b = b0; b < n_tiles; ++b) ts[b] = K;
    }
    __syncwarp();
    if (__any_sync(0xffffffffu, bad)) {
        // a corrupted list: the token contributes nothing (all its tiles start at K)
        if (lane == 0) {
            raise_status(status, MOC_ERR_BAD_INDEX);
            for (int b = 0; b < n_tiles; ++b) ts[b] = K;
        }
    }
}

// ------------------------------------------------------------------------------------------------
struct TcForwardLayout {
    int64_t chunk;  // tokens per gate/up pass
    int ldf;        // leading dimension of the dense [*, F] arrays (multiple of 8)
    size_t off_g;   // fp32 G of one chunk [chunk, ldf]
    size_t off_u;   // bf16 U, rewritten in place into Z', for ALL tokens [T, ldf]
    size_t total;
};
struct TcBackwardLayout {
    int ldf;
    int n_tiles;
    size_t off_z, off_du, off_dg, off_tile_start, total;
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
    L.total = off;
    return L;
}

inline TcBackwardLayout tc_backward_layout(const moc_ffn_desc &d) {
    TcBackwardLayout L{};
    L.ldf = round_up8(d.d_ff);
    L.n_tiles = (d.d_ff + BN - 1) / BN;
    const size_t dense = align_up((size_t)d.tokens * L.ldf * 2, 256);
    size_t off = 0;
    L.off_z = off;
    off += dense;
    L.off_du = off;
    off += dense;
    L.off_dg = off;
    off += dense;
    L.off_tile_start = off;
    off = align_up(off + (size_t)d.tokens * L.n_tiles * 4, 256);
    L.total = off;
    return L;
}

}  // namespace tc
}  // namespace moc
