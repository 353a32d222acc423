// Small-batch inference path (Section 5 of the paper): tokens <= 16, bf16.
//
// Decode is bound by reading weights from HBM once: the whole gate matrix (F*d elements) plus the
// selected rows of W_up and W_down.  With several tokens, a row selected by more than one token is
// read once (the union of the tokens' channel sets), which is what keeps a batch of 16 cheaper than
// a dense FFN.  Four kernels, all streaming:
//   1. gate GEMV   : the channels are dealt out evenly to two CTAs per SM; a CTA's 8 warps split the
//                    contraction into contiguous parts; the tokens are the M dimension of m16n8k16
//                    tensor-core MMAs so that 16 tokens cost no more issue slots than one (one FMA per
//                    loaded weight and token would be ALU-bound at 16 tokens).
//   2. select      : one 1024-thread CTA per token, exact Top-K (same selector as training); sets the
//                    token's bit in a per-channel mask and appends a channel to the list of used
//                    channels the first time any token selects it.
//   3. up          : one warp per used channel, u = x . Wu[j,:] for the tokens in its mask,
//                    z = SiLU(g) u, stored next to the channel's list position.
//   4. down        : CTA = (512-column slice, part of the list); rows arrive through a double-buffered
//                    shared-memory ring filled by bulk async copies; per-slice partial sums are added to
//                    an fp32 accumulator with atomics and the last CTA of a slice writes the bf16 output
//                    (summation order across CTAs is not fixed, so the last bit of `out` may vary).
#pragma once

#include "moc_common.cuh"
#include "tc_gemm.cuh"  // mbarrier helpers
#include "topk_select.cuh"

namespace moc {
namespace dec {

constexpr int kGemvMaxTiles = 8;   // 8-channel MMA tiles per CTA (<= 64 channels)
constexpr int kSelThreads = 1024;
constexpr int kSliceCols = 512;    // down projection: columns per CTA (1 KiB of a bf16 row)
constexpr int kBatchRows = 32;     // rows per ring buffer
constexpr int kMaxPart = 512;      // list entries per down CTA (bound of its shared arrays)

struct Workspace {
    float *G;           // [T, ldf] gate projection
    float *Zc;          // [list position][16] z = SiLU(g) u per token
    uint32_t *chmask;   // [F] bit t set: token t selected the channel
    uint16_t *list;     // [F] used channels in order of first selection
    int *list_count;    // number of used channels
    float *out_acc;     // [T, d]
    int *counters;      // [slices] arrival counters of the down kernel
    int ldf;
};

__device__ __forceinline__ uint4 ld_stream16(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// ---------------------------------------------------------------------------------------------- 1. gate GEMV
// G[t, j] = sum_i x[t,i] Wg[j,i]   (Eq. (Moc-1), per token as in Section 5).
// CTA b owns channels [b F / grid, (b+1) F / grid).  Each lane loads 16 contiguous bytes (8 contraction
// elements) of a weight row per step; the same permutation of the contraction index is applied to the
// x fragment, so no data movement is needed to form the MMA operands.
__global__ void __launch_bounds__(256, 2) gate_gemv_kernel(const __nv_bfloat16 *__restrict__ x,
                                                           const __nv_bfloat16 *__restrict__ wg, int T, int d, int F,
                                                           Workspace ws, int slices) {
    __shared__ float red[8][16][kGemvMaxTiles * 8 + 1];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, q = lane & 3;
    const int r0 = (int)(((int64_t)blockIdx.x * F) / gridDim.x);
    const int r1 = (int)(((int64_t)(blockIdx.x + 1) * F) / gridDim.x);
    const int nt = (r1 - r0 + 7) >> 3;
    // housekeeping for the later kernels: clear masks, accumulators, counters
    for (int j = r0 + tid; j < r1; j += 256) ws.chmask[j] = 0u;
    for (int64_t i = (int64_t)blockIdx.x * 256 + tid; i < (int64_t)T * d; i += (int64_t)gridDim.x * 256)
        ws.out_acc[i] = 0.f;
    if (blockIdx.x == 0) {
        if (tid < slices) ws.counters[tid] = 0;
        if (tid == 0) *ws.list_count = 0;
    }

    float acc[kGemvMaxTiles][4];
#pragma unroll
    for (int nb = 0; nb < kGemvMaxTiles; ++nb)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[nb][e] = 0.f;
    const int ksteps = (d + 31) >> 5;
    const int per_warp = (ksteps + 7) >> 3;
    const int s_begin = warp * per_warp, s_end = min(ksteps, s_begin + per_warp);
    const __nv_bfloat16 *xa_row = x + (int64_t)g * d, *xb_row = x + (int64_t)(g + 8) * d;
    const bool has_a = g < T, has_b = g + 8 < T;
    const __nv_bfloat16 *wrow[kGemvMaxTiles];
    bool wok[kGemvMaxTiles];
#pragma unroll
    for (int nb = 0; nb < kGemvMaxTiles; ++nb) {
        const int ch = r0 + nb * 8 + g;
        wok[nb] = nb < nt && ch < r1;
        wrow[nb] = wg + (int64_t)(wok[nb] ? ch : r0) * d;
    }
#pragma unroll 2
    for (int s = s_begin; s < s_end; ++s) {
        const int koff = (s << 5) + (q << 3);
        const bool kv = koff < d;
        uint4 wv[kGemvMaxTiles];
#pragma unroll
        for (int nb = 0; nb < kGemvMaxTiles; ++nb) {
            wv[nb] = make_uint4(0, 0, 0, 0);
            if (kv && wok[nb]) wv[nb] = ld_stream16(wrow[nb] + koff);
        }
        uint4 xa = make_uint4(0, 0, 0, 0), xb = make_uint4(0, 0, 0, 0);
        if (kv && has_a) xa = *reinterpret_cast<const uint4 *>(xa_row + koff);
        if (kv && has_b) xb = *reinterpret_cast<const uint4 *>(xb_row + koff);
#pragma unroll
        for (int nb = 0; nb < kGemvMaxTiles; ++nb) {
            if (nb < nt) {  // uniform
                mma_bf16_16816(acc[nb], xa.x, xb.x, xa.y, xb.y, wv[nb].x, wv[nb].y);
                mma_bf16_16816(acc[nb], xa.z, xb.z, xa.w, xb.w, wv[nb].z, wv[nb].w);
            }
        }
    }
#pragma unroll
    for (int nb = 0; nb < kGemvMaxTiles; ++nb) {
        red[warp][g][nb * 8 + 2 * q] = acc[nb][0];
        red[warp][g][nb * 8 + 2 * q + 1] = acc[nb][1];
        red[warp][g + 8][nb * 8 + 2 * q] = acc[nb][2];
        red[warp][g + 8][nb * 8 + 2 * q + 1] = acc[nb][3];
    }
    __syncthreads();
    const int width = r1 - r0;
    for (int o = tid; o < T * width; o += 256) {
        const int t = o / width, c = o - t * width;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += red[w][t][c];
        ws.G[(int64_t)t * ws.ldf + r0 + c] = s;
    }
}

// ---------------------------------------------------------------------------------------------- 2. select
// One CTA per token: exact Top-K of G[t, 0..F).
__global__ void __launch_bounds__(kSelThreads) select_mask_kernel(Workspace ws, int F, int K) {
    extern __shared__ __align__(16) uint32_t select_keys[];
    __shared__ SelectSmemT<kSelThreads / 32> sm;
    const int t = blockIdx.x;
    const float *g = ws.G + (int64_t)t * ws.ldf;
    for (int j = threadIdx.x; j < F; j += kSelThreads) select_keys[j] = gate_key(g[j]);
    __syncthreads();
    uint32_t tau;
    int need;
    block_radix_threshold<kSelThreads>(select_keys, F, K, sm, tau, need);
    const uint32_t bit = 1u << t;
    block_ordered_emit<kSelThreads>(select_keys, F, tau, need, sm, [&](int, int j) {
        if (atomicOr(&ws.chmask[j], bit) == 0u) ws.list[atomicAdd(ws.list_count, 1)] = (uint16_t)j;
    });
}

// ---------------------------------------------------------------------------------------------- 3. up
// One warp per used channel j: u_t = x_t . Wu[j,:] for every token t in the channel's mask,
// z_t = SiLU(G[t,j]) u_t.   (Eq. (MoC-2) on the mask.)
__global__ void __launch_bounds__(256) up_rows_kernel(const __nv_bfloat16 *__restrict__ x,
                                                      const __nv_bfloat16 *__restrict__ wu, int T, int d, int F,
                                                      Workspace ws) {
    const int lane = threadIdx.x & 31;
    const int gw = blockIdx.x * 8 + (threadIdx.x >> 5), nw = gridDim.x * 8;
    const int nvec = d >> 3;  // 16-byte vectors per row
    const int count = min(*ws.list_count, F);
    for (int p = gw; p < count; p += nw) {
        const int j = ws.list[p];
        const uint32_t m = ws.chmask[j];
        const __nv_bfloat16 *row = wu + (int64_t)j * d;
        float part[16];
#pragma unroll
        for (int t = 0; t < 16; ++t) part[t] = 0.f;
        // the row is consumed in segments of 8 vectors per lane (2048 elements), weights in registers
        for (int v0 = 0; v0 < nvec; v0 += 256) {
            uint4 w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int v = v0 + i * 32 + lane;
                w[i] = make_uint4(0, 0, 0, 0);
                if (v < nvec) w[i] = ld_stream16(row + 8 * v);
            }
#pragma unroll
            for (int t = 0; t < 16; ++t) {
                if (!((m >> t) & 1u)) continue;  // uniform across the warp
                const __nv_bfloat16 *xt = x + (int64_t)t * d;
                float a = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int v = v0 + i * 32 + lane;
                    if (v < nvec) {
                        const uint4 xv = *reinterpret_cast<const uint4 *>(xt + 8 * v);
                        const uint32_t ww[4] = {w[i].x, w[i].y, w[i].z, w[i].w};
                        const uint32_t xx[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            a = fmaf(__uint_as_float(ww[e] << 16), __uint_as_float(xx[e] << 16), a);
                            a = fmaf(__uint_as_float(ww[e] & 0xffff0000u), __uint_as_float(xx[e] & 0xffff0000u), a);
                        }
                    }
                }
                part[t] += a;
            }
        }
#pragma unroll
        for (int t = 0; t < 16; ++t) {
            if (!((m >> t) & 1u)) continue;
            const float u = warp_sum(part[t]);
            if (lane == 0) ws.Zc[(int64_t)p * 16 + t] = silu_f(ws.G[(int64_t)t * ws.ldf + j]) * u;
        }
    }
}

// ---------------------------------------------------------------------------------------------- 4. down
// out[t, c] = sum_{j in C_t} z[t,j] Wd[j, c]   (Section 5, final output), for the CTA's column slice
// and its part of the list of used channels.  grid = (slices, parts).
__global__ void __launch_bounds__(256) down_rows_kernel(const __nv_bfloat16 *__restrict__ wd, int T, int d, int F,
                                                        Workspace ws, __nv_bfloat16 *__restrict__ out,
                                                        int *__restrict__ status) {
    extern __shared__ __align__(128) uint8_t dsm[];
    // layout: ring [2][kBatchRows][1 KiB] | z [kMaxPart][16] floats | channel [kMaxPart] u16 | mask [kMaxPart] u16
    uint8_t *ring = dsm;
    float *zl = reinterpret_cast<float *>(dsm + 2 * kBatchRows * 1024);
    uint16_t *lch = reinterpret_cast<uint16_t *>(zl + kMaxPart * 16);
    uint16_t *lmask = lch + kMaxPart;
    __shared__ uint64_t bars[2];
    __shared__ int s_abort, s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int slice = blockIdx.x, c0 = slice * kSliceCols;
    const int cols = min(kSliceCols, d - c0);       // multiple of 8
    const uint32_t row_bytes = (uint32_t)cols * 2;  // multiple of 16
    const int total = min(*ws.list_count, F);
    const int per = min(kMaxPart, (total + (int)gridDim.y - 1) / (int)gridDim.y);
    const int p0 = min(total, (int)blockIdx.y * per);
    const int count = min(per, total - p0);

    if (tid == 0) {
        tc::mbar_init(tc::smem_u32(&bars[0]), 1);
        tc::mbar_init(tc::smem_u32(&bars[1]), 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = tid; i < count; i += 256) {
        const int j = ws.list[p0 + i];
        lch[i] = (uint16_t)j;
        lmask[i] = (uint16_t)ws.chmask[j];
    }
    for (int i = tid; i < count * 16; i += 256) zl[i] = ws.Zc[(int64_t)p0 * 16 + i];
    __syncthreads();

    const int batches = (count + kBatchRows - 1) / kBatchRows;
    auto issue = [&](int b) {  // warp 0: one bulk copy per lane
        const int buf = b & 1;
        const int rows = min(kBatchRows, count - b * kBatchRows);
        const uint32_t bar = tc::smem_u32(&bars[buf]);
        if (lane == 0) tc::mbar_expect_tx(bar, (uint32_t)rows * row_bytes);
        __syncwarp();
        if (lane < rows) {
            const int j = lch[b * kBatchRows + lane];
            const uint32_t dst = tc::smem_u32(ring + ((size_t)buf * kBatchRows + lane) * 1024);
            const __nv_bfloat16 *src = wd + (int64_t)j * d + c0;
            asm volatile(
                "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                ::"r"(dst), "l"(src), "r"(row_bytes), "r"(bar)
                : "memory");
        }
    };
    float acc[16][2];
#pragma unroll
    for (int t = 0; t < 16; ++t) acc[t][0] = acc[t][1] = 0.f;
    if (warp == 0 && batches > 0) issue(0);
    uint32_t phase0 = 0, phase1 = 0;
    for (int b = 0; b < batches; ++b) {
        const int buf = b & 1;
        if (warp == 0 && b + 1 < batches) issue(b + 1);  // the other buffer was released by the barrier below
        const bool ok = tc::mbar_wait(tc::smem_u32(&bars[buf]), buf ? phase1 : phase0, &s_abort, status);
        if (buf) phase1 ^= 1u; else phase0 ^= 1u;
        if (!__syncthreads_and(ok)) break;
        const int rows = min(kBatchRows, count - b * kBatchRows);
        if (2 * tid < cols) {
            for (int r = 0; r < rows; ++r) {
                const int p = b * kBatchRows + r;
                const uint32_t w2 =
                    *reinterpret_cast<const uint32_t *>(ring + ((size_t)buf * kBatchRows + r) * 1024 + 4 * tid);
                const float w0 = __uint_as_float(w2 << 16), w1 = __uint_as_float(w2 & 0xffff0000u);
                const uint32_t m = lmask[p];
                const float *zp = zl + p * 16;
#pragma unroll
                for (int t = 0; t < 16; ++t) {
                    if ((m >> t) & 1u) {
                        const float z = zp[t];
                        acc[t][0] = fmaf(z, w0, acc[t][0]);
                        acc[t][1] = fmaf(z, w1, acc[t][1]);
                    }
                }
            }
        }
        __syncthreads();  // everyone is done with `buf` before it is refilled
    }
    if (s_abort) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) __nanosleep(1000);
    }
    // add this CTA's partial sums, then the last CTA of the slice converts the totals to bf16
    if (2 * tid < cols && count > 0) {
#pragma unroll
        for (int t = 0; t < 16; ++t) {
            if (t < T) {
                float *o = ws.out_acc + (int64_t)t * d + c0 + 2 * tid;
                if (acc[t][0] != 0.f) atomicAdd(o, acc[t][0]);
                if (acc[t][1] != 0.f) atomicAdd(o + 1, acc[t][1]);
            }
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(&ws.counters[slice], 1) == (int)gridDim.y - 1;
    __syncthreads();
    if (s_last) {
        __threadfence();
        for (int i = tid; i < T * (cols >> 1); i += 256) {
            const int t = i / (cols >> 1), c = (i % (cols >> 1)) * 2;
            const float *a = ws.out_acc + (int64_t)t * d + c0 + c;
            const float v0 = __ldcg(a), v1 = __ldcg(a + 1);
            *reinterpret_cast<__nv_bfloat162 *>(out + (int64_t)t * d + c0 + c) = __floats2bfloat162_rn(v0, v1);
        }
    }
}

}  // namespace dec
}  // namespace moc
