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

// Signed 4-bit dynamic-exponent table (App. E.2 with b = 1 + E + 1 + F = 4), sorted increasingly:
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

// Nearest linear code as the low mantissa bits of 2^23 + ceil(max(16 n - 1.5, 0)), added with
// round-up; valid for n <= 1 + 2^-22 (then the code is at most 15). The caller removes the 2^23 pattern.
constexpr uint32_t kMagicBits = 0x4b000000u;  // 2^23 as binary32
__device__ __forceinline__ uint32_t lin_nearest_magic(float n) {
    const float y = fmaxf(__fmaf_rn(n, 16.0f, -1.5f), 0.0f);
    return __float_as_uint(__fadd_ru(y, 8388608.0f));
}

// Shared-memory image of the nearest-entry table, directly indexed by the top 11 bits of n: 1024 eight-byte
// entries for n >= 0 followed by 1024 for n < 0, so that no clamping is needed and every bit pattern (NaN
// and infinities included) stays inside the table.
constexpr int kLutSmemBytes = 2 * 1024 * 8;

__device__ __forceinline__ void load_lut_smem(unsigned char* smem) {
    for (uint32_t i = threadIdx.x; i < 2048u; i += blockDim.x) {
        const uint32_t key = i & 1023u, neg = i >> 10;
        uint2 e;
        if (key < kDeLutFirstKey) e = make_uint2(0x7f7fffffu, 7u);
        else if (key >= kDeLutFirstKey + kDeLutBins) e = make_uint2(0x7f7fffffu, neg ? 0u : 15u);
        else e = kDeLut[neg * kDeLutBins + key - kDeLutFirstKey];
        reinterpret_cast<uint2*>(smem)[i] = e;
    }
}

// Table-driven equivalent of de_nearest(): one lookup, one comparison, one add.
__device__ __forceinline__ uint32_t de_nearest_lut(float n, const unsigned char* smem) {
    const uint2 e = *reinterpret_cast<const uint2*>(smem + ((__float_as_uint(n) >> 18) & 0x3ff8u));
    return e.y + (n > __uint_as_float(e.x) ? 1u : 0u);
}

// 1/s (correctly rounded) for a usable scale, 0 for a zero or denormal one (everything under it
// quantizes as zero).
__device__ __forceinline__ float scale_rcp(float s) {
    return (s >= kFltMin) ? __frcp_rn(s) : 0.0f;
}

struct Hyper {
    float lr, beta1, beta2, eps;
    float omb1, omb2;  // 1 - beta, evaluated in binary32
    float bc1, bc2;    // 1 - beta^t, evaluated in binary64 on the host and rounded once
    float decay;       // 1 - lr * weight_decay
    float step_size;   // lr / bc1, evaluated in binary64 and rounded once (fast update)
    float rbc2;        // 1 / bc2, likewise
    float one;         // 1.0f, passed as data (see ema_m2)
    float upd_c1;      // -sqrt(1 / bc2) / step_size and
    float upd_e1;      // -eps / step_size (binary64 on the host, rounded once): see adam_update_fast2()
};

// The same constants as pairs, for the packed two-lane fp32 instructions of sm_100 (mul/add/fma.f32x2:
// two independent IEEE operations per instruction, so results are bit-identical to the scalar forms).
struct Hyper2 {
    float2 beta1, omb1, beta2, omb2;
    float2 rbc2, eps, neg_step, decay, one, upd_c1, upd_e1;
    float2 c16, cm15, magic;   // 16, -1.5 and 2^23 for the linear quantizer
    float2 lin_a01, lin_a23, lin_b01, lin_b23;   // see lin_dequant8()
};
__host__ __device__ __forceinline__ float2 splat(float x) { return make_float2(x, x); }

// Packed operations written as PTX with an explicit rounding mode: such instructions are never
// contracted into a fused multiply-add, which the stored states rely on.
__device__ __forceinline__ unsigned long long pack2(float2 a) {
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a.x), "f"(a.y));
    return r;
}
__device__ __forceinline__ float2 unpack2(unsigned long long r) {
    float2 a;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a.x), "=f"(a.y) : "l"(r));
    return a;
}
__device__ __forceinline__ float2 mul2_rn(float2 a, float2 b) {
    unsigned long long d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(pack2(a)), "l"(pack2(b)));
    return unpack2(d);
}
__device__ __forceinline__ float2 add2_rn(float2 a, float2 b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(pack2(a)), "l"(pack2(b)));
    return unpack2(d);
}
__device__ __forceinline__ float2 add2_ru(float2 a, float2 b) {
    unsigned long long d;
    asm("add.rp.f32x2 %0, %1, %2;" : "=l"(d) : "l"(pack2(a)), "l"(pack2(b)));
    return unpack2(d);
}
__device__ __forceinline__ float2 fma2_rn(float2 a, float2 b, float2 c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(pack2(a)), "l"(pack2(b)), "l"(pack2(c)));
    return unpack2(d);
}
__host__ __device__ __forceinline__ Hyper2 make_hyper2(const Hyper& h) {
    Hyper2 p;
    p.beta1 = splat(h.beta1); p.omb1 = splat(h.omb1); p.beta2 = splat(h.beta2); p.omb2 = splat(h.omb2);
    p.rbc2 = splat(h.rbc2); p.eps = splat(h.eps); p.neg_step = splat(-h.step_size); p.decay = splat(h.decay);
    p.one = splat(h.one); p.upd_c1 = splat(h.upd_c1); p.upd_e1 = splat(h.upd_e1);
    p.c16 = splat(16.0f); p.cm15 = splat(-1.5f); p.magic = splat(8388608.0f);
    // a_k = 2^-(4k+4), b_k = 2^-4 - 2^(19-4k): (2^23 + q 16^k) a_k + b_k = (q + 1)/16 exactly
    p.lin_a01 = make_float2(0.0625f, 0.00390625f);
    p.lin_a23 = make_float2(0.000244140625f, 0.0000152587890625f);
    p.lin_b01 = make_float2(0.0625f - 524288.0f, 0.0625f - 32768.0f);
    p.lin_b23 = make_float2(0.0625f - 2048.0f, 0.0625f - 128.0f);
    return p;
}
// T_lin(q) = (q + 1)/16 (App. E.2) for the eight codes of one word, without a table: a nibble at bit 4k
// (k <= 3), OR-ed into the mantissa of 2^23, is the number 2^23 + q 16^k, and one fused multiply-add maps it
// to (q + 1)/16. Every intermediate and the result are exactly representable, so nothing is rounded.
// t[i] holds the entries of elements 2i and 2i + 1.
__device__ __forceinline__ void lin_dequant8(uint32_t q, const Hyper2& h, float2 (&t)[4]) {
    const uint32_t hi = q >> 16;
    const uint32_t magic = __float_as_uint(h.magic.x);     // 2^23: its mantissa field is empty
    uint32_t f[8];
#define LPMM_NIB(dst, src, m) asm("lop3.b32 %0, %1, " #m ", %2, 0xEA;" : "=r"(dst) : "r"(src), "r"(magic))
    LPMM_NIB(f[0], q, 0xf);   LPMM_NIB(f[1], q, 0xf0);   LPMM_NIB(f[2], q, 0xf00);   LPMM_NIB(f[3], q, 0xf000);
    LPMM_NIB(f[4], hi, 0xf);  LPMM_NIB(f[5], hi, 0xf0);  LPMM_NIB(f[6], hi, 0xf00);  LPMM_NIB(f[7], hi, 0xf000);
#undef LPMM_NIB
    t[0] = fma2_rn(make_float2(__uint_as_float(f[0]), __uint_as_float(f[1])), h.lin_a01, h.lin_b01);
    t[1] = fma2_rn(make_float2(__uint_as_float(f[2]), __uint_as_float(f[3])), h.lin_a23, h.lin_b23);
    t[2] = fma2_rn(make_float2(__uint_as_float(f[4]), __uint_as_float(f[5])), h.lin_a01, h.lin_b01);
    t[3] = fma2_rn(make_float2(__uint_as_float(f[6]), __uint_as_float(f[7])), h.lin_a23, h.lin_b23);
}
// Both products must be rounded before the sum (Eq. 1 evaluated operation by operation). The assembler
// was observed to merge a packed multiply with a following packed add into a fused multiply-add even with
// explicit rounding modes, so the sum is written as fma(p1, 1, p2) with the 1 supplied at run time:
// fl(p1 * 1 + p2) = fl(p1 + p2) exactly, and nothing is left to merge.
__device__ __forceinline__ float2 ema_m2(float2 m, float2 g, const Hyper2& h) {
    return fma2_rn(mul2_rn(h.beta1, m), h.one, mul2_rn(h.omb1, g));
}
__device__ __forceinline__ float2 ema_v2(float2 v, float2 g, const Hyper2& h) {
    return fma2_rn(mul2_rn(h.beta2, v), h.one, mul2_rn(h.omb2, mul2_rn(g, g)));
}
// adam_update_fast() on a pair, with the constants folded on the host so that three packed operations and the
// two approximate special functions remain:
//   -step / (sqrt(v_t / bc2) + eps) = 1 / (sqrt(v_t) * c1 + e1),  c1 = -sqrt(1 / bc2) / step,  e1 = -eps / step.
// The host falls back to adam_update() when step is (almost) zero, where c1 and e1 do not exist.
__device__ __forceinline__ float2 adam_update_fast2(float2 w, float2 mt, float2 vt, const Hyper2& h) {
    float2 sq, rc;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(sq.x) : "f"(vt.x));
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(sq.y) : "f"(vt.y));
    const float2 den = fma2_rn(sq, h.upd_c1, h.upd_e1);
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rc.x) : "f"(den.x));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(rc.y) : "f"(den.y));
    return fma2_rn(w, h.decay, mul2_rn(mt, rc));
}

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

// The same with a look first: a value that does not exceed what the slot already holds needs no atomic at all.
// The slot only ever grows within a pass, so a stale read can cost a redundant atomic but never lose a maximum;
// the read bypasses L1 to see other SMs' updates early. Over a stream of values the number of atomics per slot
// drops from the number of elements to roughly the number of running maxima.
__device__ __forceinline__ void atomic_max_nonneg_filtered(float* addr, float v) {
    if (v > __ldcg(addr)) atomicMax(reinterpret_cast<unsigned int*>(addr), __float_as_uint(v));
}

}  // namespace lpmm
