// Device-side building blocks of the 4-bit AdamW step: the two 4-bit tables, exact nearest-entry
// searches, nibble unpacking and the Adam arithmetic. Every operation that decides a stored bit
// (codes, scales) is written with explicit round-to-nearest intrinsics so that no compiler flag can
// fuse a multiply with an add: the stored state is a pure function of the gradient stream.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "lpmm_de_lut.cuh"

namespace lpmm {

constexpr float kFltMin = 1.17549435e-38f;  // smallest normal binary32

// Signed 4-bit dynamic-exponent table (App. D.2 with b = 1 + E + 1 + F = 4), sorted increasingly:
// +-{0.2125, 0.4375, 0.6625, 0.8875}, +-{0.0325, 0.0775}, +-0.0055, 0 and +1 (no -1).
__device__ __constant__ float kDeTable[16] = {
    -0.8875f, -0.6625f, -0.4375f, -0.2125f, -0.0775f, -0.0325f, -0.0055f, 0.0f,
    0.0055f,  0.0325f,  0.0775f,  0.2125f,  0.4375f,  0.6625f,  0.8875f,  1.0f};

// Nearest-entry rule for the table above (Sec. 2.2 "Mapping": argmin_i |n - T(i)|, exact, ties to the
// lower entry). Each constant is the largest binary32 value not above the exact midpoint of two
// adjacent entries, so "n > thr" means "n is strictly nearer to the upper entry" for every binary32 n;
// the code is the number of thresholds strictly below n.
__device__ __forceinline__ uint32_t de_nearest(float n) {
    uint32_t c = 0;
    c += (n > __uint_as_float(0xbf466667u));
    c += (n > __uint_as_float(0xbf0ccccdu));
    c += (n > __uint_as_float(0xbea66667u));
    c += (n > __uint_as_float(0xbe147ae2u));
    c += (n > __uint_as_float(0xbd6147aeu));
    c += (n > __uint_as_float(0xbc9ba5e3u));
    c += (n > __uint_as_float(0xbb343958u));
    c += (n > __uint_as_float(0x3b343958u));
    c += (n > __uint_as_float(0x3c9ba5e3u));
    c += (n > __uint_as_float(0x3d6147aeu));
    c += (n > __uint_as_float(0x3e147ae1u));
    c += (n > __uint_as_float(0x3ea66666u));
    c += (n > __uint_as_float(0x3f0ccccdu));
    c += (n > __uint_as_float(0x3f466666u));
    c += (n > __uint_as_float(0x3f719999u));
    return c;
}

// Zero-free linear table T(i) = (i+1)/16 (Sec. 4.1). The midpoints (2i+3)/32 are exact in binary32 and
// 16 n - 1.5 is exact whenever n >= 3/32 (below that only its sign matters), so
// code = clamp(ceil(16 n - 1.5), 0, 15) equals the exact argmin with ties going down.
__device__ __forceinline__ uint32_t lin_nearest(float n) {
    float y = __fmaf_rn(n, 16.0f, -1.5f);
    int q = __float2int_ru(y);
    q = max(q, 0);
    q = min(q, 15);
    return (uint32_t)q;
}

__device__ __forceinline__ float lin_value(uint32_t q) {  // (q+1)/16, exact
    return __fmul_rn((float)(q + 1u), 0.0625f);
}

// Same value without an integer conversion: `word` holds the nibble at bits [shift, shift+4); it is
// moved to the top of the mantissa of 1.0f (giving 1 + q/16 exactly) and 15/16 is subtracted (exact).
template <int SHIFT>
__device__ __forceinline__ float lin_value_at(uint32_t word) {
    const uint32_t moved = (SHIFT <= 19) ? (word << (19 - SHIFT)) : (word >> (SHIFT - 19));
    return __fadd_rn(__uint_as_float((moved & 0x00780000u) | 0x3f800000u), -0.9375f);
}

// Nearest linear code as the low mantissa bits of 2^23 + ceil(max(16 n - 1.5, 0)), added with
// round-up; valid for n <= 1 + 2^-22 (then the code is at most 15). The caller removes the 2^23 pattern.
constexpr uint32_t kMagicBits = 0x4b000000u;  // 2^23 as binary32
__device__ __forceinline__ uint32_t lin_nearest_magic(float n) {
    const float y = fmaxf(__fmaf_rn(n, 16.0f, -1.5f), 0.0f);
    return __float_as_uint(__fadd_ru(y, 8388608.0f));
}

// Shared-memory image used by the step kernel: the non-negative half of kDeLut at byte 0, the negative
// half at byte 16384 (so that the sign bit of the key selects it without an extra instruction), and the
// 16-entry dequantization table in between.
constexpr int kLutNegOffset = 16384;
constexpr int kLutDeTableOffset = 1024;
constexpr int kLutSmemBytes = kLutNegOffset + kDeLutBins * 8;

__device__ __forceinline__ void load_lut_smem(unsigned char* smem) {
    for (int i = threadIdx.x; i < kDeLutBins; i += blockDim.x) {
        reinterpret_cast<uint2*>(smem)[i] = kDeLut[i];
        reinterpret_cast<uint2*>(smem + kLutNegOffset)[i] = kDeLut[kDeLutBins + i];
    }
    if (threadIdx.x < 16) reinterpret_cast<float*>(smem + kLutDeTableOffset)[threadIdx.x] = kDeTable[threadIdx.x];
}

// Table-driven equivalent of de_nearest() for |n| < 2 (always true for m / blockmax(|m|)); NaN gives code 7.
__device__ __forceinline__ uint32_t de_nearest_lut(float n, const unsigned char* smem) {
    const float a = fminf(fmaxf(fabsf(n), kDeLutMinAbs), 1.9999999f);
    const uint32_t nb = __float_as_uint(n);
    const uint32_t cs = (__float_as_uint(a) & 0x7fffffffu) | (nb & 0x80000000u);   // copysign(a, n)
    const uint32_t off = (cs >> 17) & 0x7ff8u;      // bit 14 = sign -> +16384; bits 3..13 = key * 8
    const uint2 e = *reinterpret_cast<const uint2*>(smem + off - kDeLutKeyBias);
    const uint32_t c = e.y + (a > __uint_as_float(e.x) ? 1u : 0u);
    return c ^ ((uint32_t)((int32_t)nb >> 31) & 15u);
}

// 1/s for a usable scale, 0 for a zero or denormal one (everything under it quantizes as zero).
__device__ __forceinline__ float scale_rcp(float s) {
    return (s >= kFltMin) ? __fdiv_rn(1.0f, s) : 0.0f;
}

struct Hyper {
    float lr, beta1, beta2, eps;
    float omb1, omb2;  // 1 - beta, evaluated in binary32
    float bc1, bc2;    // 1 - beta^t, evaluated in binary64 on the host and rounded once
    float decay;       // 1 - lr * weight_decay
    float step_size;   // lr / bc1, evaluated in binary64 and rounded once (fast update)
    float rbc2;        // 1 / bc2, likewise
};

// Eq. 1 moment updates; separate roundings, in the order written there.
__device__ __forceinline__ float ema_m(float m, float g, const Hyper& h) {
    return __fadd_rn(__fmul_rn(h.beta1, m), __fmul_rn(h.omb1, g));
}
__device__ __forceinline__ float ema_v(float v, float g, const Hyper& h) {
    return __fadd_rn(__fmul_rn(h.beta2, v), __fmul_rn(h.omb2, __fmul_rn(g, g)));
}

// Eq. 1 bias correction and update with decoupled weight decay, IEEE division and square root.
__device__ __forceinline__ float adam_update(float w, float mt, float vt, const Hyper& h) {
    float mhat = __fdiv_rn(mt, h.bc1);
    float vhat = __fdiv_rn(vt, h.bc2);
    float denom = __fadd_rn(__fsqrt_rn(vhat), h.eps);
    float upd = __fmul_rn(h.lr, __fdiv_rn(mhat, denom));
    return __fsub_rn(__fmul_rn(w, h.decay), upd);
}

// The same update with one approximate square root and one approximate reciprocal (each within about
// one ulp) and the constant divisions folded into host-side factors: a handful of roundings away from
// adam_update(), far inside the 1e-6 * max(|w|, lr) parameter tolerance. A denormal bias-corrected
// second moment is flushed to zero before the square root, which is harmless once eps is added; the host
// therefore selects adam_update() instead when eps is (almost) zero. The stored states never depend on
// this function.
__device__ __forceinline__ float adam_update_fast(float w, float mt, float vt, const Hyper& h) {
    float sq, rc;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(sq) : "f"(__fmul_rn(vt, h.rbc2)));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rc) : "f"(__fadd_rn(sq, h.eps)));
    const float upd = __fmul_rn(__fmul_rn(mt, h.step_size), rc);
    return __fmaf_rn(w, h.decay, -upd);
}

__device__ __forceinline__ float bf16_lo(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t pair) { return __uint_as_float(pair & 0xffff0000u); }

// max over the 16 lanes that share one 128-element block (8 elements per lane)
__device__ __forceinline__ float half_warp_max(float x) {
    x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 8));
    x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 4));
    x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 2));
    x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 1));
    return x;
}
__device__ __forceinline__ float warp_max(float x) {
    x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 16));
    return half_warp_max(x);
}

// Non-negative floats order like their bit patterns, so an unsigned atomicMax reduces them exactly.
__device__ __forceinline__ void atomic_max_nonneg(float* addr, float v) {
    atomicMax(reinterpret_cast<unsigned int*>(addr), __float_as_uint(v));
}

}  // namespace lpmm
