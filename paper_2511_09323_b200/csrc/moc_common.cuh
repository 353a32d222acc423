// Shared device/host helpers of the MoC FFN library (internal; not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/moc_ffn.h"

namespace moc {

// ---- device status word ---------------------------------------------------------------------
// One sticky int per device; kernels raise it with atomicMin (statuses are negative, the most
// negative wins), the host reads and clears it in moc_last_device_status().
int *device_status_ptr();  // host: device address of the current device's status word (nullptr on error)

__device__ __forceinline__ void raise_status(int *status, int code) {
    if (status) atomicMin(status, code);
}

// ---- scalar conversions ---------------------------------------------------------------------
template <typename T>
__device__ __forceinline__ float to_f32(T v);
template <>
__device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T>
__device__ __forceinline__ T from_f32(float v);
template <>
__device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Vector of 8 storage elements (16 bytes for bf16, 32 for fp32) widened to fp32.
template <typename T>
struct Vec8;
template <>
struct Vec8<__nv_bfloat16> {
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float (&f)[8]) {
        uint4 raw = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, const float (&f)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t *>(&h);
        }
        *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};
template <>
struct Vec8<float> {
    static __device__ __forceinline__ void load(const float *p, float (&f)[8]) {
        float4 a = *reinterpret_cast<const float4 *>(p);
        float4 b = *reinterpret_cast<const float4 *>(p + 4);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
        f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    }
    static __device__ __forceinline__ void store(float *p, const float (&f)[8]) {
        *reinterpret_cast<float4 *>(p) = make_float4(f[0], f[1], f[2], f[3]);
        *reinterpret_cast<float4 *>(p + 4) = make_float4(f[4], f[5], f[6], f[7]);
    }
};

// ---- SiLU (paper Eq. (silu)) and its derivative, fp32 -------------------------------------------
__device__ __forceinline__ float sigmoid_f(float g) {
    // evaluated from exp(-|g|) so that large |g| neither overflows nor produces NaN
    float e = expf(-fabsf(g));
    float r = 1.0f / (1.0f + e);
    return g >= 0.0f ? r : e * r;
}
__device__ __forceinline__ float silu_f(float g) { return g * sigmoid_f(g); }
__device__ __forceinline__ float dsilu_f(float g) {
    float s = sigmoid_f(g);
    return s * (1.0f + g * (1.0f - s));
}

// ---- warp helpers -----------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---- selection key ------------------------------------------------------------------------------
// Order-preserving map fp32 -> uint32 (larger value <=> larger key); NaN -> key of -inf, -0 -> +0.
__device__ __forceinline__ uint32_t gate_key(float g) {
    if (g != g) g = __int_as_float(0xff800000);  // NaN orders as -infinity
    g = g + 0.0f;                                // -0.0 + 0.0 = +0.0
    uint32_t b = __float_as_uint(g);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---- development aid: device-clock stamps (only in builds with -DMOC_TIMELINE) ---------------------------------
// MOC_TL(slot) lets the first thread of the first CTA of a kernel note the GPU's nanosecond timer in g_timeline[slot].
#ifdef MOC_TIMELINE
__device__ unsigned long long g_timeline[4096];
__device__ __forceinline__ void timeline_stamp(int slot, bool who) {
    if (who) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        g_timeline[slot] = t;
    }
}
// MOC_TL_CTA(base): every CTA's first thread notes the timer in g_timeline[base + blockIdx.x]
#define MOC_TL_CTA(base) ::moc::timeline_stamp((base) + (int)blockIdx.x, threadIdx.x == 0)
#define MOC_TL_CTA_ANY(base) ::moc::timeline_stamp((base) + (int)blockIdx.x, true)
#define MOC_TL(slot) ::moc::timeline_stamp(slot, blockIdx.x == 0 && threadIdx.x == 0)
#define MOC_TL_IF(slot, cond) ::moc::timeline_stamp(slot, cond)
#else
#define MOC_TL(slot) ((void)0)
#define MOC_TL_CTA(base) ((void)0)
#define MOC_TL_CTA_ANY(base) ((void)0)
#define MOC_TL_IF(slot, cond) ((void)0)
#endif

}  // namespace moc
