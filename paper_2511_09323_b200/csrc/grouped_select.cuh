// Grouped selection, MoC 2:8 (Section 4, "MoC with structured 2:8 sparsity"; Theorem 1 for the a:b form): in every
// group of 8 consecutive channels the 2 with the largest signed pre-SiLU gate values are kept (equal values: the
// lower channel; NaN as -inf; -0 equals +0).  The mask is local, so no search is needed: one thread per group.
// Everything after the mask (Eq. (MoC-2), the backward of Section 4) is the same as with the row Top-K mask, with
// K = d_ff / 4 and the kept channels of group q in slots 2q and 2q + 1 of the compact arrays.
#pragma once

#include "moc_common.cuh"

namespace moc {

constexpr int kGroup = 8, kGroupKeep = 2;

// the two kept offsets of a group, ascending
__device__ __forceinline__ void top2_of_8(const uint32_t (&key)[8], int &lo, int &hi) {
    // (the running best keys are carried in registers: indexing key[] with a run-time index would put it in local memory)
    uint32_t k1 = key[0], k2 = 0u;
    int i1 = 0, i2 = -1;
#pragma unroll
    for (int e = 1; e < 8; ++e)
        if (key[e] > k1) {  // strict: among equal keys the lowest channel stays
            k1 = key[e];
            i1 = e;
        }
#pragma unroll
    for (int e = 0; e < 8; ++e)
        if (e != i1 && (i2 < 0 || key[e] > k2)) {
            k2 = key[e];
            i2 = e;
        }
    lo = min(i1, i2);
    hi = max(i1, i2);
}

// Tensor-core plan: G [rows, ldg] fp32 and U [rows, ldu] bf16 (dense, from the gate+up GEMM) -> compact idx / g / u
// (any of them may be null together: inference) and the U row rewritten in place into the masked Z' = SiLU(g) u.
// One thread per group: 32 bytes of G and 16 bytes of U in, 16 bytes of Z' out, all coalesced.
__global__ void __launch_bounds__(256) select_grouped_mask_kernel(const float *__restrict__ G, int ldg,
                                                                  __nv_bfloat16 *__restrict__ U, int ldu, int64_t rows,
                                                                  int F, int16_t *__restrict__ idx_out,
                                                                  __nv_bfloat16 *__restrict__ g_out,
                                                                  __nv_bfloat16 *__restrict__ u_out) {
    const int groups = F / kGroup;
    const int64_t total = rows * groups;
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < total; i += (int64_t)gridDim.x * 256) {
        const int64_t r = i / groups;
        const int q = (int)(i - r * groups);
        const float4 *gp = reinterpret_cast<const float4 *>(G + r * ldg + q * kGroup);
        const float4 g0 = gp[0], g1 = gp[1];
        uint4 *up = reinterpret_cast<uint4 *>(U + r * ldu + q * kGroup);
        const uint4 uw = *up;
        const float g[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
        uint32_t key[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) key[e] = gate_key(g[e]);
        int lo, hi;
        top2_of_8(key, lo, hi);
        const uint32_t uwords[4] = {uw.x, uw.y, uw.z, uw.w};
        uint32_t zwords[4] = {0u, 0u, 0u, 0u};
        __nv_bfloat16 ub[2], gb[2];
        const int sel[2] = {lo, hi};
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            const int e = sel[s];
            float gv = 0.f;
            uint32_t uword = 0u;
#pragma unroll
            for (int f = 0; f < 8; ++f) {  // register arrays: no dynamic indexing
                if (f == e) {
                    gv = g[f];
                    uword = uwords[f >> 1];
                }
            }
            const uint16_t ubits = (uint16_t)((e & 1) ? (uword >> 16) : (uword & 0xffffu));
            ub[s] = *reinterpret_cast<const __nv_bfloat16 *>(&ubits);
            gb[s] = __float2bfloat16_rn(gv);
            const __nv_bfloat16 zb = __float2bfloat16_rn(silu_f(gv) * __bfloat162float(ub[s]));
            const uint32_t zbits = (uint32_t)(*reinterpret_cast<const uint16_t *>(&zb)) << ((e & 1) * 16);
#pragma unroll
            for (int wd = 0; wd < 4; ++wd)
                if (wd == (e >> 1)) zwords[wd] |= zbits;
        }
        *up = make_uint4(zwords[0], zwords[1], zwords[2], zwords[3]);
        if (idx_out) {
            const int64_t o = r * (int64_t)(groups * kGroupKeep) + q * kGroupKeep;
            *reinterpret_cast<short2 *>(idx_out + o) = make_short2((short)(q * kGroup + lo), (short)(q * kGroup + hi));
            *reinterpret_cast<__nv_bfloat162 *>(g_out + o) = __halves2bfloat162(gb[0], gb[1]);
            *reinterpret_cast<__nv_bfloat162 *>(u_out + o) = __halves2bfloat162(ub[0], ub[1]);
        }
    }
}

// Gathered plan: G [rows, ldg] fp32 -> idx [rows, F / 4] and optionally the saved gate values.
template <typename T>
__global__ void __launch_bounds__(256) select_grouped_idx_kernel(const float *__restrict__ G, int64_t rows, int F, int ldg,
                                                                 int16_t *__restrict__ idx_out, T *__restrict__ topk_gate) {
    const int groups = F / kGroup;
    const int64_t total = rows * groups;
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < total; i += (int64_t)gridDim.x * 256) {
        const int64_t r = i / groups;
        const int q = (int)(i - r * groups);
        const float *gp = G + r * ldg + q * kGroup;
        float g[8];
        uint32_t key[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            g[e] = gp[e];
            key[e] = gate_key(g[e]);
        }
        int lo, hi;
        top2_of_8(key, lo, hi);
        float glo = 0.f, ghi = 0.f;
#pragma unroll
        for (int f = 0; f < 8; ++f) {
            if (f == lo) glo = g[f];
            if (f == hi) ghi = g[f];
        }
        const int64_t o = r * (int64_t)(groups * kGroupKeep) + q * kGroupKeep;
        idx_out[o] = (int16_t)(q * kGroup + lo);
        idx_out[o + 1] = (int16_t)(q * kGroup + hi);
        if (topk_gate) {
            topk_gate[o] = from_f32<T>(glo);
            topk_gate[o + 1] = from_f32<T>(ghi);
        }
    }
}

}  // namespace moc
