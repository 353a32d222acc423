// Gathered (ALU) kernels of the MoC FFN: exact fp32-accumulate implementations of every step of
// the operator that touch only the selected channels.  They serve the fp32 storage type, shapes
// the tensor-core path does not take, and small batches, where reading only the K selected rows
// of W_up / W_down is the whole point (Section 5 of the paper).
//
// All weights are channel-major [F_ld, d]: a selected channel is one contiguous d-vector, read
// with 16-byte (bf16) / 32-byte (fp32) vector loads by consecutive threads.
#pragma once

#include "moc_common.cuh"
#include "topk_select.cuh"

namespace moc {

constexpr int kTokenThreads = 256;

// ------------------------------------------------------------------------------------------------
// Dense gate projection on the ALUs:  C[M,N] (fp32) = A[M,Kd] * B[N,Kd]^T, both operands K-major.
// 64x64 tile, 256 threads, 4x4 outputs per thread.  (Eq. (Moc-1), G = X W_gate.)
template <typename T>
__global__ void __launch_bounds__(256) gemm_nt_alu_kernel(const T *__restrict__ A, const T *__restrict__ B,
                                                          float *__restrict__ C, int M, int N, int Kd, int ldc) {
    constexpr int BM = 64, BN = 64, BK = 16;
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int tx = tid % 16, ty = tid / 16;
    float acc[4][4] = {};
    // each thread stages 4 A and 4 B elements per k-step: row = tid / 4, cols (tid % 4) * 4 .. +3
    const int lr = tid / 4, lc = (tid % 4) * 4;
    for (int k0 = 0; k0 < Kd; k0 += BK) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int kk = k0 + lc + c;
            float a = 0.f, b = 0.f;
            if (kk < Kd) {
                if (m0 + lr < M) a = to_f32<T>(A[(int64_t)(m0 + lr) * Kd + kk]);
                if (n0 + lr < N) b = to_f32<T>(B[(int64_t)(n0 + lr) * Kd + kk]);
            }
            As[lc + c][lr] = a;
            Bs[lc + c][lr] = b;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                a[i] = As[kk][ty * 4 + i];
                b[i] = Bs[kk][tx * 4 + i];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n < N) C[(int64_t)m * ldc + n] = acc[i][j];
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Row selector fused with the gather of the gate values: one CTA per token of the chunk.
//   G [rows, ldg] fp32 (transient) -> idx [rows,K] int16 ascending, and optionally the saved gate
//   values topk_gate [rows,K] in the storage type.
template <typename T>
__global__ void __launch_bounds__(kSelectThreads) select_rows_kernel(const float *__restrict__ G, int64_t rows,
                                                                      int F, int ldg, int K,
                                                                      int16_t *__restrict__ idx_out,
                                                                      T *__restrict__ topk_gate, int post_silu) {
    extern __shared__ __align__(16) uint32_t select_keys[];
    __shared__ SelectSmem sm;
    SelectGuess guess;
    for (int64_t r = blockIdx.x; r < rows; r += gridDim.x) {
        const float *g = G + r * (int64_t)ldg;
        uint32_t tau;
        int need;
        block_select_row<kSelectThreads>(g, F, K, select_keys, sm, guess, tau, need, post_silu != 0);
        int16_t *o = idx_out + r * (int64_t)K;
        T *og = topk_gate ? topk_gate + r * (int64_t)K : nullptr;
        block_ordered_emit<kSelectThreads>(select_keys, F, tau, need, sm, [&](int pos, int j) {
            o[pos] = (int16_t)j;
            // the value comes back from the key in shared memory: a global load inside the ordered walk
            // would cost a memory round trip per chunk
            // (keys of SiLU(g) do not give g back: the post-SiLU variant reads it)
            if (og) og[pos] = from_f32<T>(post_silu ? g[j] : key_to_float(select_keys[j]));
        });
        __syncthreads();
    }
}

// Accumulates  acc[v-th 8-vector] += sum_k coef[k] * W[rowidx[k], 8v..8v+7]  over the token's K rows,
// with the CTA's threads laid out as (row-group g) x (vector lane vl); partial sums of the groups
// are combined through shared memory.  Used by the down projection and by grad_x.
// red: shared scratch of at least THREADS/min(nvec,THREADS) * d floats when more than one group exists.
template <typename T, int NSRC, typename RowW, typename Coef>
__device__ __forceinline__ void token_row_combine(int d, int K, const int *rowidx, RowW roww, Coef coef,
                                                  float *red, T *__restrict__ dst) {
    const int tid = threadIdx.x;
    const int nvec = d >> 3;
    const int lanes_v = nvec < kTokenThreads ? nvec : kTokenThreads;
    const int G = kTokenThreads / lanes_v;
    const int g = tid / lanes_v, vl = tid % lanes_v;
    for (int v = vl; v < nvec; v += lanes_v) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (g < G) {
            for (int k = g; k < K; k += G) {
                const int j = rowidx[k];
                if (j < 0) continue;  // invalid saved index: skipped (status already raised)
#pragma unroll
                for (int s = 0; s < NSRC; ++s) {
                    float w[8];
                    Vec8<T>::load(roww(s) + (int64_t)j * d + 8 * v, w);
                    const float c = coef(s, k);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[e] = fmaf(c, w[e], acc[e]);
                }
            }
        }
        if (G == 1) {
            Vec8<T>::store(dst + 8 * v, acc);
        } else {
            // G > 1 only when nvec < THREADS, i.e. this loop body runs once per thread
            if (g < G) {
#pragma unroll
                for (int e = 0; e < 8; ++e) red[g * d + 8 * v + e] = acc[e];
            }
            __syncthreads();
            if (g == 0) {
                for (int gg = 1; gg < G; ++gg)
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[e] += red[gg * d + 8 * v + e];
                Vec8<T>::store(dst + 8 * v, acc);
            }
            __syncthreads();
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Forward, per token (grid.x = tokens of the chunk):
//   u_k = x . W_up[idx_k,:]        (Eq. (Moc-1) on the mask only)
//   z_k = SiLU(g_k) * u_k          (Eq. (MoC-2))
//   out = sum_k z_k W_down[idx_k,:]
// gate values come from the transient fp32 gate projection G (unrounded).
// Dynamic shared memory: d floats (x) + K floats (z) + K ints (idx) + reduction scratch.
template <typename T>
__global__ void __launch_bounds__(kTokenThreads) forward_token_kernel(
    const T *__restrict__ x, const T *__restrict__ w_up, const T *__restrict__ w_down,
    const float *__restrict__ G, int ldg, const int16_t *__restrict__ idx, int d, int K, T *__restrict__ out,
    T *__restrict__ topk_up, int red_floats) {
    extern __shared__ __align__(16) float fsm[];
    float *xs = fsm;
    float *zs = xs + d;
    int *js = reinterpret_cast<int *>(zs + K);
    float *red = reinterpret_cast<float *>(js + K);
    (void)red_floats;
    const int64_t t = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T *xt = x + t * d;
    for (int v = tid; v < (d >> 3); v += kTokenThreads) {
        float f[8];
        Vec8<T>::load(xt + 8 * v, f);
#pragma unroll
        for (int e = 0; e < 8; ++e) xs[8 * v + e] = f[e];
    }
    for (int k = tid; k < K; k += kTokenThreads) js[k] = idx[t * K + k];
    __syncthreads();
    const float *gt = G + t * (int64_t)ldg;
    for (int k = warp; k < K; k += kTokenThreads / 32) {
        const int j = js[k];
        const T *wr = w_up + (int64_t)j * d;
        float acc = 0.f;
        for (int v = lane; v < (d >> 3); v += 32) {
            float w[8];
            Vec8<T>::load(wr + 8 * v, w);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc = fmaf(xs[8 * v + e], w[e], acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) {
            const float g = gt[j];
            zs[k] = silu_f(g) * acc;
            if (topk_up) topk_up[t * K + k] = from_f32<T>(acc);
        }
    }
    __syncthreads();
    token_row_combine<T, 1>(
        d, K, js, [&](int) { return w_down; }, [&](int, int k) { return zs[k]; }, red, out + t * d);
}

// ------------------------------------------------------------------------------------------------
// Backward, per token (grid.x = tokens):  Eqs. (bp-1)..(bp-3) on the mask and Eq. (bp-5).
//   dz_k = grad_out . W_down[idx_k,:];  s = SiLU(g);  z = s u;  dU = s dz;  dG = u dz SiLU'(g)
//   grad_x = sum_k dG_k W_gate[idx_k,:] + dU_k W_up[idx_k,:]
// The compact coefficients z, dU, dG go to coef [3, T*K] fp32 for the weight-gradient kernels.
template <typename T>
__global__ void __launch_bounds__(kTokenThreads) backward_token_kernel(
    const T *__restrict__ w_gate, const T *__restrict__ w_up, const T *__restrict__ w_down,
    const int16_t *__restrict__ idx, const T *__restrict__ topk_gate, const T *__restrict__ topk_up,
    const T *__restrict__ grad_out, int d, int F, int K, int64_t TK, T *__restrict__ grad_x,
    float *__restrict__ coef, int *__restrict__ status) {
    extern __shared__ __align__(16) float fsm[];
    float *ds = fsm;
    float *dgs = ds + d;
    float *dus = dgs + K;
    int *js = reinterpret_cast<int *>(dus + K);
    float *red = reinterpret_cast<float *>(js + K);
    const int64_t t = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T *dt = grad_out + t * d;
    for (int v = tid; v < (d >> 3); v += kTokenThreads) {
        float f[8];
        Vec8<T>::load(dt + 8 * v, f);
#pragma unroll
        for (int e = 0; e < 8; ++e) ds[8 * v + e] = f[e];
    }
    for (int k = tid; k < K; k += kTokenThreads) {
        int j = idx[t * K + k];
        if (j < 0 || j >= F) {
            raise_status(status, MOC_ERR_BAD_INDEX);
            j = -1;
        }
        js[k] = j;
    }
    __syncthreads();
    for (int k = warp; k < K; k += kTokenThreads / 32) {
        const int j = js[k];
        float z = 0.f, dU = 0.f, dG = 0.f;
        if (j >= 0) {
            const T *wr = w_down + (int64_t)j * d;
            float acc = 0.f;
            for (int v = lane; v < (d >> 3); v += 32) {
                float w[8];
                Vec8<T>::load(wr + 8 * v, w);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc = fmaf(ds[8 * v + e], w[e], acc);
            }
            const float dz = warp_sum(acc);
            const float g = to_f32<T>(topk_gate[t * K + k]);
            const float u = to_f32<T>(topk_up[t * K + k]);
            const float s = silu_f(g);
            z = s * u;
            dU = s * dz;
            dG = u * dz * dsilu_f(g);
        }
        if (lane == 0) {
            dgs[k] = dG;
            dus[k] = dU;
            if (coef) {
                coef[t * K + k] = z;
                coef[TK + t * K + k] = dU;
                coef[2 * TK + t * K + k] = dG;
            }
        }
    }
    __syncthreads();
    if (grad_x) {
        token_row_combine<T, 2>(
            d, K, js, [&](int s) { return s == 0 ? w_gate : w_up; },
            [&](int s, int k) { return s == 0 ? dgs[k] : dus[k]; }, red, grad_x + t * d);
    }
}

// ------------------------------------------------------------------------------------------------
// Per-channel token lists (a CSR transpose of idx), built deterministically so that every weight
// gradient row is a sum over its tokens in ascending token order.
//   counts [nb, F]  : per token-block, per channel occurrence counts, then exclusive offsets
//   row_start [F+1] : list start of each channel
//   pairs [T*K]     : pair id p = t*K + k, grouped by channel, tokens ascending
// Token block b covers tokens [b*tb, min(T,(b+1)*tb)).
__global__ void __launch_bounds__(256) csr_count_kernel(const int16_t *__restrict__ idx, int64_t T, int K, int F,
                                                        int tb, uint32_t *__restrict__ counts) {
    extern __shared__ __align__(16) uint32_t cnt[];
    for (int j = threadIdx.x; j < F; j += 256) cnt[j] = 0;
    __syncthreads();
    const int64_t t0 = (int64_t)blockIdx.x * tb;
    const int64_t t1 = t0 + tb < T ? t0 + tb : T;
    const int64_t e0 = t0 * K, e1 = t1 * K;
    for (int64_t e = e0 + threadIdx.x; e < e1; e += 256) {
        const int j = idx[e];
        if (j >= 0 && j < F) atomicAdd(&cnt[j], 1u);
    }
    __syncthreads();
    uint32_t *o = counts + (int64_t)blockIdx.x * F;
    for (int j = threadIdx.x; j < F; j += 256) o[j] = cnt[j];
}

// thread per channel: exclusive prefix over the token blocks; totals[j] = list length
__global__ void __launch_bounds__(256) csr_scan_blocks_kernel(uint32_t *__restrict__ counts, int nb, int F,
                                                              uint32_t *__restrict__ totals) {
    const int j = blockIdx.x * 256 + threadIdx.x;
    if (j >= F) return;
    uint32_t run = 0;
    for (int b = 0; b < nb; ++b) {
        const uint32_t c = counts[(int64_t)b * F + j];
        counts[(int64_t)b * F + j] = run;
        run += c;
    }
    totals[j] = run;
}

// single CTA: exclusive scan of totals[F] -> row_start[F+1]
__global__ void __launch_bounds__(1024) csr_scan_channels_kernel(const uint32_t *__restrict__ totals, int F,
                                                                 uint32_t *__restrict__ row_start) {
    __shared__ uint32_t wtot[32];
    __shared__ uint32_t carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < F; base += 1024) {
        const int j = base + tid;
        const uint32_t v = j < F ? totals[j] : 0u;
        uint32_t s = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t n = __shfl_up_sync(0xffffffffu, s, o);
            if (lane >= o) s += n;
        }
        if (lane == 31) wtot[warp] = s;
        __syncthreads();
        uint32_t before = carry;
        for (int w = 0; w < warp; ++w) before += wtot[w];
        if (j < F) row_start[j] = before + s - v;
        __syncthreads();
        if (tid == 1023) carry = before + s;
        __syncthreads();
    }
    if (tid == 0) row_start[F] = carry;
}

__global__ void __launch_bounds__(256) csr_fill_kernel(const int16_t *__restrict__ idx, int64_t T, int K, int F,
                                                       int tb, const uint32_t *__restrict__ counts,
                                                       const uint32_t *__restrict__ row_start,
                                                       uint32_t *__restrict__ pairs) {
    extern __shared__ __align__(16) uint32_t cursor[];
    const uint32_t *c = counts + (int64_t)blockIdx.x * F;
    for (int j = threadIdx.x; j < F; j += 256) cursor[j] = row_start[j] + c[j];
    __syncthreads();
    const int64_t t0 = (int64_t)blockIdx.x * tb;
    const int64_t t1 = t0 + tb < T ? t0 + tb : T;
    for (int64_t t = t0; t < t1; ++t) {
        // channels of one token are distinct, so the order inside a list is the token order
        for (int k = threadIdx.x; k < K; k += 256) {
            const int j = idx[t * K + k];
            if (j >= 0 && j < F) {
                const uint32_t pos = atomicAdd(&cursor[j], 1u);
                pairs[pos] = (uint32_t)(t * K + k);
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// Weight gradients, one CTA per channel row j (Eqs. (bp-1) and (bp-4) restricted to the mask):
//   grad_w_down[j,:] = sum_p z_p  * grad_out[t_p,:]
//   grad_w_up  [j,:] = sum_p dU_p * x[t_p,:]
//   grad_w_gate[j,:] = sum_p dG_p * x[t_p,:]          p over the channel's (token, slot) pairs
// Rows no token selected (and padding rows) are written as exact zeros.
template <typename T>
__global__ void __launch_bounds__(kTokenThreads) wgrad_rows_kernel(
    const T *__restrict__ x, const T *__restrict__ grad_out, const float *__restrict__ coef, int64_t TK,
    const uint32_t *__restrict__ row_start, const uint32_t *__restrict__ pairs, int d, int F, int K,
    T *__restrict__ gw_gate, T *__restrict__ gw_up, T *__restrict__ gw_down, int accumulate) {
    extern __shared__ __align__(16) float red[];  // [G][3][d] when G > 1
    const int j = blockIdx.x;
    const int tid = threadIdx.x;
    const int nvec = d >> 3;
    const int lanes_v = nvec < kTokenThreads ? nvec : kTokenThreads;
    const int G = kTokenThreads / lanes_v;
    const int g = tid / lanes_v, vl = tid % lanes_v;
    uint32_t p0 = 0, p1 = 0;
    if (j < F) {
        p0 = row_start[j];
        p1 = row_start[j + 1];
    }
    for (int v = vl; v < nvec; v += lanes_v) {
        float a_dn[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        float a_up[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        float a_gt[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (g < G) {
            for (uint32_t q = p0 + g; q < p1; q += G) {
                const uint32_t p = pairs[q];
                const int64_t t = p / (uint32_t)K;
                float xv[8], dv[8];
                if (gw_down) {
                    Vec8<T>::load(grad_out + t * d + 8 * v, dv);
                    const float z = coef[p];
#pragma unroll
                    for (int e = 0; e < 8; ++e) a_dn[e] = fmaf(z, dv[e], a_dn[e]);
                }
                if (gw_up || gw_gate) {
                    Vec8<T>::load(x + t * d + 8 * v, xv);
                    const float dU = coef[TK + p], dG = coef[2 * TK + p];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        a_up[e] = fmaf(dU, xv[e], a_up[e]);
                        a_gt[e] = fmaf(dG, xv[e], a_gt[e]);
                    }
                }
            }
        }
        if (G > 1) {
            if (g < G) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    red[(g * 3 + 0) * d + 8 * v + e] = a_dn[e];
                    red[(g * 3 + 1) * d + 8 * v + e] = a_up[e];
                    red[(g * 3 + 2) * d + 8 * v + e] = a_gt[e];
                }
            }
            __syncthreads();
            if (g == 0) {
                for (int gg = 1; gg < G; ++gg)
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        a_dn[e] += red[(gg * 3 + 0) * d + 8 * v + e];
                        a_up[e] += red[(gg * 3 + 1) * d + 8 * v + e];
                        a_gt[e] += red[(gg * 3 + 2) * d + 8 * v + e];
                    }
            }
        }
        if (g == 0) {
            const int64_t o = (int64_t)j * d + 8 * v;
            T *dst[3] = {gw_down, gw_up, gw_gate};
            float *src[3] = {a_dn, a_up, a_gt};
#pragma unroll
            for (int s = 0; s < 3; ++s) {
                if (!dst[s]) continue;
                float r[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) r[e] = src[s][e];
                if (accumulate) {
                    float old[8];
                    Vec8<T>::load(dst[s] + o, old);
#pragma unroll
                    for (int e = 0; e < 8; ++e) r[e] += old[e];
                }
                Vec8<T>::store(dst[s] + o, r);
            }
        }
        if (G > 1) __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------- up values again
// topk_up[t, k] = U[t, idx[t, k]] from a dense U [T, ldu] (the tensor-core plan recomputes U with its GEMM), or, with
// U == nullptr, the dot product x[t, :] . w_up[idx[t, k], :] itself in fp32 (one warp per kept channel).
// An index outside [0, F) is skipped (its output is set to zero) and reported.
template <typename T>
__global__ void __launch_bounds__(256) recompute_up_kernel(const T *__restrict__ x, const T *__restrict__ w_up,
                                                           const __nv_bfloat16 *__restrict__ U, int ldu,
                                                           const int16_t *__restrict__ idx, int64_t tokens, int K, int F,
                                                           int d, T *__restrict__ up_out, int *__restrict__ status) {
    const int lane = threadIdx.x & 31;
    const int64_t total = tokens * K;
    if (U) {
        for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < total; i += (int64_t)gridDim.x * 256) {
            const int64_t t = i / K;
            const int j = idx[i];
            if (j < 0 || j >= F) {
                raise_status(status, MOC_ERR_BAD_INDEX);
                up_out[i] = from_f32<T>(0.f);
            } else {
                up_out[i] = from_f32<T>(__bfloat162float(U[t * ldu + j]));
            }
        }
        return;
    }
    const int64_t warps = (int64_t)gridDim.x * 8;
    for (int64_t i = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); i < total; i += warps) {
        const int64_t t = i / K;
        const int j = idx[i];
        if (j < 0 || j >= F) {
            if (lane == 0) {
                raise_status(status, MOC_ERR_BAD_INDEX);
                up_out[i] = from_f32<T>(0.f);
            }
            continue;
        }
        const T *xr = x + t * d, *wr = w_up + (int64_t)j * d;
        float sum = 0.f;
        for (int c = lane * 8; c < d; c += 256) {
            float a[8], b[8];
            Vec8<T>::load(xr + c, a);
            Vec8<T>::load(wr + c, b);
#pragma unroll
            for (int e = 0; e < 8; ++e) sum = fmaf(a[e], b[e], sum);
        }
        sum = warp_sum(sum);
        if (lane == 0) up_out[i] = from_f32<T>(sum);
    }
}

}  // namespace moc
