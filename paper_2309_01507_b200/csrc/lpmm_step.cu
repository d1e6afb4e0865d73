// Kernels of the fused 4-bit AdamW step (Alg. 3 with Eq. 1) for sm_100a.
//
// One step is three launches over a device-side tensor table:
//   pass 1  (rank-1 tensors only) recomputes the new second moment v_t from the gradient and the old
//           codes and reduces its row and column maxima r', c' (Sec. 4.2) with an unsigned atomicMax
//           on the float bit patterns (v_t >= 0);
//   rcp     inverts r', c' once (1/s, or 0 for a scale below FLT_MIN);
//   pass 2  (all tensors) dequantizes m and v, applies the moment updates, bias correction, decoupled
//           decay and the parameter update, reduces each 128-block's |m_t| maximum inside 16 lanes,
//           and re-quantizes both moments to the nearest code, two codes per byte.
// Work is cut into tiles; tile -> tensor is a binary search over prefix sums, so one launch covers
// every tensor. A lane always owns 8 consecutive elements: 32 B of fp32 parameters, 16 B of bf16 (32 B
// of fp32) gradient and one 32-bit word of each moment's codes; 16 lanes own one 128-element block.
#include "lpmm_internal.h"

// The update pass has 80 instantiations; to build in parallel this file can be compiled four times with
// -DLPMM_STEP_PART=0..3, each part holding the update-pass launchers of one (gradient type, update math) pair and
// part 0 the remaining launchers as well. Without the macro one translation unit holds everything.
#ifndef LPMM_STEP_PART
#define LPMM_STEP_ALL 1
#define LPMM_STEP_PART 0
#endif

namespace lpmm {

namespace {

__device__ __forceinline__ int find_tensor(const int32_t* __restrict__ start, int n, int tile) {
    int lo = 0, hi = n;  // invariant: start[lo] <= tile < start[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (__ldg(start + mid) <= tile) lo = mid; else hi = mid;
    }
    return lo;
}

// One of the three rank-1 scale buffers of a tensor (selected without indexing the by-value descriptor dynamically).
__device__ __forceinline__ float* rc_pick(const TensorDesc& d, int i) { return i == 0 ? d.rc[0] : (i == 1 ? d.rc[1] : d.rc[2]); }

// The row / column scale vectors a tiled kernel works with: a matrix's own r, c, or a composite tensor's expanded ones.
__device__ __forceinline__ float* stats_old(const TensorDesc& d, RcSel sel) { return d.exp_old ? d.exp_old : rc_pick(d, sel.old_i); }
__device__ __forceinline__ float* stats_new(const TensorDesc& d, RcSel sel) { return d.exp_old ? d.exp_new : rc_pick(d, sel.new_i); }

// ---- tile hand-out --------------------------------------------------------------------------------
//
// The CTAs of a launch take tiles from a counter in the arena header in the order they become free, so an SM
// that gets less memory bandwidth than its neighbours simply takes fewer tiles (with a fixed stride the whole
// launch waits for the slowest SM). Thread 0 asks for the next index while the current tile is processed and
// publishes it through one of two shared words; the CTA that finishes last puts both counters back to zero for
// the next launch on the stream.

__device__ __forceinline__ int tiles_first(int32_t* ctr, int* s_next) {
    if (threadIdx.x == 0) s_next[0] = atomicAdd(ctr, 1);
    __syncthreads();
    return s_next[0];
}
__device__ __forceinline__ int tiles_fetch(int32_t* ctr) { return threadIdx.x == 0 ? atomicAdd(ctr, 1) : 0; }
__device__ __forceinline__ int tiles_next(int* s_next, int& buf, int fetched) {
    buf ^= 1;
    if (threadIdx.x == 0) s_next[buf] = fetched;
    __syncthreads();
    return s_next[buf];
}
__device__ __forceinline__ void tiles_done(int32_t* ctr) {
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(ctr + 1, 1) == (int)gridDim.x - 1) { ctr[0] = 0; ctr[1] = 0; }
    }
}

// ---- 8-element loads ------------------------------------------------------------------------

__device__ __forceinline__ void load8_f32(const float* p, float (&x)[8]) {
    float4 a = __ldg(reinterpret_cast<const float4*>(p));
    float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void load8_rw(const float* p, float (&x)[8]) {  // read-modify-write data: no __ldg
    float4 a = *reinterpret_cast<const float4*>(p);
    float4 b = *(reinterpret_cast<const float4*>(p) + 1);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void store8_f32(float* p, const float (&x)[8]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
    *(reinterpret_cast<float4*>(p) + 1) = make_float4(x[4], x[5], x[6], x[7]);
}
// Eight parameters as bfloat16 (round to nearest even), one 16-byte store.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ void store8_bf16(uint16_t* p, const float (&x)[8]) {
    *reinterpret_cast<uint4*>(p) = make_uint4(pack_bf16x2(x[0], x[1]), pack_bf16x2(x[2], x[3]),
                                              pack_bf16x2(x[4], x[5]), pack_bf16x2(x[6], x[7]));
}
__device__ __forceinline__ void store8_bf16_guard(uint16_t* p, int64_t e, int64_t numel, const float (&x)[8]) {
#pragma unroll
    for (int k = 0; k < 8; k += 2) {
        const uint32_t pr = pack_bf16x2(x[k], x[k + 1]);
        if (e + k < numel) p[e + k] = (uint16_t)(pr & 0xffffu);
        if (e + k + 1 < numel) p[e + k + 1] = (uint16_t)(pr >> 16);
    }
}
__device__ __forceinline__ void load8_bf16(const uint16_t* p, float (&x)[8]) {
    uint4 r = __ldg(reinterpret_cast<const uint4*>(p));
    x[0] = bf16_lo(r.x); x[1] = bf16_hi(r.x); x[2] = bf16_lo(r.y); x[3] = bf16_hi(r.y);
    x[4] = bf16_lo(r.z); x[5] = bf16_hi(r.z); x[6] = bf16_lo(r.w); x[7] = bf16_hi(r.w);
}
template <bool BF16>
__device__ __forceinline__ void load8_grad(const void* g, int64_t e, float (&x)[8]) {
    if (BF16) load8_bf16(reinterpret_cast<const uint16_t*>(g) + e, x);
    else load8_f32(reinterpret_cast<const float*>(g) + e, x);
}
template <bool BF16>
__device__ __forceinline__ float load1_grad(const void* g, int64_t e) {
    if (BF16) return __uint_as_float(((uint32_t)__ldg(reinterpret_cast<const uint16_t*>(g) + e)) << 16);
    return __ldg(reinterpret_cast<const float*>(g) + e);
}

// Guarded variants for the ragged end of a tensor: elements at or beyond `numel` read as zero.
template <bool BF16>
__device__ __forceinline__ void load8_grad_guard(const void* g, int64_t e, int64_t numel, float (&x)[8]) {
#pragma unroll
    for (int k = 0; k < 8; ++k) x[k] = (e + k < numel) ? load1_grad<BF16>(g, e + k) : 0.0f;
}
__device__ __forceinline__ void load8_guard(const float* p, int64_t e, int64_t numel, float (&x)[8]) {
#pragma unroll
    for (int k = 0; k < 8; ++k) x[k] = (e + k < numel) ? p[e + k] : 0.0f;
}
__device__ __forceinline__ void store8_guard(float* p, int64_t e, int64_t numel, const float (&x)[8]) {
#pragma unroll
    for (int k = 0; k < 8; ++k) if (e + k < numel) p[e + k] = x[k];
}
// 8 codes of elements e..e+7 (e is a multiple of 8); bytes beyond the tensor read as 0.
__device__ __forceinline__ uint32_t load_codes_guard(const uint8_t* codes, int64_t e, int64_t numel) {
    int64_t nbytes = (numel + 1) >> 1;
    uint32_t q = 0;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        int64_t byte = (e >> 1) + b;
        if (byte < nbytes) q |= ((uint32_t)codes[byte]) << (8 * b);
    }
    return q;
}
// Stores the codes of the valid elements; a trailing odd element leaves its byte's high nibble 0.
__device__ __forceinline__ void store_codes_guard(uint8_t* codes, int64_t e, int64_t numel, uint32_t q) {
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        int64_t lo = e + 2 * b;
        if (lo < numel) {
            uint32_t byte = (q >> (8 * b)) & 0xffu;
            if (lo + 1 >= numel) byte &= 0x0fu;
            codes[lo >> 1] = (uint8_t)byte;
        }
    }
}

// ---- per-lane arithmetic ----------------------------------------------------------------------

template <bool EXACT>
__device__ __forceinline__ float update_param(float w, float mt, float vt, const Hyper& h) {
    return EXACT ? adam_update(w, mt, vt, h) : adam_update_fast(w, mt, vt, h);
}

// Per-lane constants of the shuffle-based table lookups: lane l of every 16-lane group holds entry
// l & 15 of the signed DE table and of the linear table; a code is dequantized by reading the lane whose
// index is the code (shuffle width 16 takes the source lane modulo 16, so the nibble needs no masking).
struct LaneTables {
    float de;    // T_DE[lane & 15]
    float lin;   // (lane & 15 + 1) / 16 (the maxima pass looks second-moment codes up with a shuffle)
    unsigned mask;   // the 16 lanes of this lane's group
};
__device__ __forceinline__ LaneTables make_lane_tables() {
    const int lane = threadIdx.x & 31;
    LaneTables t;
    t.de = kDeTable[lane & 15];
    t.lin = __fmul_rn((float)((lane & 15) + 1), 0.0625f);
    t.mask = 0xffffu << (lane & 16);
    return t;
}

// Dequantize (Sec. 2.2), update the moments (Eq. 1) and the parameters for 8 elements, two at a time.
// m_prod is T_DE[lane & 15] * (old block scale of m); vs[k] the old scale of element k's second moment.
// FACT: the second moment is not dequantized and averaged but given (vs[k] is the reconstructed v_ij itself).
template <bool EXACT, bool FACT = false>
__device__ __forceinline__ void moments_and_update8(float (&w)[8], const float (&g)[8], uint32_t qm, uint32_t qv,
                                                    float m_prod, const float (&vs)[8], const Hyper& h,
                                                    const Hyper2& h2, const LaneTables& lt, float (&mt)[8],
                                                    float (&vt)[8]) {
    float2 tlin[4];
    if (!FACT) lin_dequant8(qv, h2, tlin);
#pragma unroll
    for (int k = 0; k < 8; k += 2) {
        const float2 m = make_float2(__shfl_sync(lt.mask, m_prod, (int)(qm >> (4 * k)), 16),
                                     __shfl_sync(lt.mask, m_prod, (int)(qm >> (4 * k + 4)), 16));
        const float2 g2 = make_float2(g[k], g[k + 1]);
        const float2 m2 = ema_m2(m, g2, h2);
        float2 v2;
        if (FACT) {
            v2 = make_float2(vs[k], vs[k + 1]);
        } else {
            v2 = ema_v2(mul2_rn(tlin[k >> 1], make_float2(vs[k], vs[k + 1])), g2, h2);
        }
        mt[k] = m2.x; mt[k + 1] = m2.y;
        vt[k] = v2.x; vt[k + 1] = v2.y;
        if (EXACT) {
            w[k] = adam_update(w[k], m2.x, v2.x, h);
            w[k + 1] = adam_update(w[k + 1], m2.y, v2.y, h);
        } else {
            const float2 w2 = adam_update_fast2(make_float2(w[k], w[k + 1]), m2, v2, h2);
            w[k] = w2.x; w[k + 1] = w2.y;
        }
    }
}

__device__ __forceinline__ float absmax8(const float (&x)[8]) {
    float a = 0.0f;
#pragma unroll
    for (int k = 0; k < 8; ++k) a = fmaxf(a, fabsf(x[k]));
    return a;
}
__device__ __forceinline__ float group_max(float x, unsigned mask) {   // over the 16 lanes of one block
    x = fmaxf(x, __shfl_xor_sync(mask, x, 8));
    x = fmaxf(x, __shfl_xor_sync(mask, x, 4));
    x = fmaxf(x, __shfl_xor_sync(mask, x, 2));
    x = fmaxf(x, __shfl_xor_sync(mask, x, 1));
    return x;
}

// Maximum over one first-moment block. B128: the 16 lanes that own it. B2048: the whole CTA (its 8 warps
// cover exactly one block per step and move in lockstep); the two halves of s_red alternate from step to
// step, so one barrier per step is enough.
__device__ __forceinline__ float block_max(float x, int m_shift, const LaneTables& lt, float* s_red, uint32_t& step) {
    if (m_shift == 7) return group_max(x, lt.mask);
    x = warp_max(x);
    float* slot = s_red + (step++ & 1u) * kWarps;   // the counter runs across tiles: every thread calls this equally often
    if ((threadIdx.x & 31) == 0) slot[threadIdx.x >> 5] = x;
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kWarps; ++i) x = fmaxf(x, slot[i]);
    return x;
}

// Eight nearest codes packed little-nibble-first: acc = acc * 16 + code, from element 7 down to 0.
__device__ __forceinline__ uint32_t quantize8_de(const float (&x)[8], float rcp, const unsigned char* s_lut) {
    uint32_t q = 0;
    const float2 r2 = splat(rcp);
#pragma unroll
    for (int k = 6; k >= 0; k -= 2) {
        const float2 n = mul2_rn(make_float2(x[k], x[k + 1]), r2);
        q = q * 16u + de_nearest_lut(n.y, s_lut);
        q = q * 16u + de_nearest_lut(n.x, s_lut);
    }
    return q;
}
// Linear codes as the low mantissa bits of 2^23 + ceil(max(16 n - 1.5, 0)) (see lin_nearest_magic()).
__device__ __forceinline__ uint32_t quantize8_lin(const float (&x)[8], const float (&rcp)[8], const Hyper2& h2) {
    uint32_t q = 0;
    const float2 c16 = h2.c16, cm = h2.cm15, magic = h2.magic;
#pragma unroll
    for (int k = 6; k >= 0; k -= 2) {
        float2 y = fma2_rn(mul2_rn(make_float2(x[k], x[k + 1]), make_float2(rcp[k], rcp[k + 1])), c16, cm);
        y.x = fmaxf(y.x, 0.0f);
        y.y = fmaxf(y.y, 0.0f);
        const float2 t = add2_ru(y, magic);
        q = q * 16u + __float_as_uint(t.y);
        q = q * 16u + __float_as_uint(t.x);
    }
    return q - kMagicBits * 0x11111111u;   // removes the eight 2^23 patterns (mod 2^32)
}

template <bool BF16>
__device__ __forceinline__ void unpack_grad8(const uint4& g0, const uint4& g1, float (&g)[8]) {
    if (BF16) {
        g[0] = bf16_lo(g0.x); g[1] = bf16_hi(g0.x); g[2] = bf16_lo(g0.y); g[3] = bf16_hi(g0.y);
        g[4] = bf16_lo(g0.z); g[5] = bf16_hi(g0.z); g[6] = bf16_lo(g0.w); g[7] = bf16_hi(g0.w);
    } else {
        g[0] = __uint_as_float(g0.x); g[1] = __uint_as_float(g0.y); g[2] = __uint_as_float(g0.z);
        g[3] = __uint_as_float(g0.w); g[4] = __uint_as_float(g1.x); g[5] = __uint_as_float(g1.y);
        g[6] = __uint_as_float(g1.z); g[7] = __uint_as_float(g1.w);
    }
}

// 256-bit global accesses (sm_100): a lane's 8 fp32 values in one instruction instead of two. The address must be
// 32-byte aligned; callers check the tensor's base pointer once per tile and fall back to two 128-bit accesses.
__device__ __forceinline__ void load8_f32_256(const float* p, float4& a, float4& b) {
    asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w), "=f"(b.x), "=f"(b.y), "=f"(b.z), "=f"(b.w) : "l"(p));
}
__device__ __forceinline__ void load8_u32_256_nc(const void* p, uint4& a, uint4& b) {
    asm volatile("ld.global.nc.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "l"(p));
}
__device__ __forceinline__ void store8_f32_256(float* p, const float (&x)[8]) {
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "l"(p), "f"(x[0]), "f"(x[1]), "f"(x[2]), "f"(x[3]), "f"(x[4]), "f"(x[5]), "f"(x[6]), "f"(x[7]) : "memory");
}

// ---- L2 residency hints (fused schedule) --------------------------------------------------------------
//
// In the fused schedule the maxima pass and the update pass of a tensor run close together and the update pass
// should find the gradient and the second-moment codes still in L2. The maxima pass therefore reads the part of a
// tensor that is meant to stay with the "evict last" priority. (Marking the update pass's accesses "evict first" as
// well was measured and dropped: the hinted forms of its loads and stores cost more than the few extra hits saved.)
struct L2Policies {
    uint64_t last, normal;
};
__device__ __forceinline__ L2Policies make_l2_policies() {
    L2Policies p;
    asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p.last));
    asm("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p.normal));
    return p;
}
__device__ __forceinline__ uint4 load4_u32_nc_h(const void* p, uint64_t pol) {
    uint4 a;
    asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w) : "l"(p), "l"(pol));
    return a;
}
__device__ __forceinline__ uint32_t load1_u32_nc_h(const void* p, uint64_t pol) {
    uint32_t a;
    asm volatile("ld.global.nc.L2::cache_hint.u32 %0, [%1], %2;" : "=r"(a) : "l"(p), "l"(pol));
    return a;
}
__device__ __forceinline__ void load8_f32_cg(const float* p, float (&x)[8]) {   // data written earlier in the same launch
    float4 a = __ldcg(reinterpret_cast<const float4*>(p));
    float4 b = __ldcg(reinterpret_cast<const float4*>(p) + 1);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}

template <bool A32>
__device__ __forceinline__ void load8_rw_a(const float* p, float (&x)[8]) {
    if (A32) {
        float4 a, b;
        load8_f32_256(p, a, b);
        x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
    } else {
        load8_rw(p, x);
    }
}
template <bool A32>
__device__ __forceinline__ void store8_f32_a(float* p, const float (&x)[8]) {
    if (A32) store8_f32_256(p, x); else store8_f32(p, x);
}
template <bool BF16, bool A32>
__device__ __forceinline__ void load8_grad_a(const void* g, int64_t e, float (&x)[8]) {
    if (!BF16 && A32) {
        uint4 a, b;
        load8_u32_256_nc(reinterpret_cast<const float*>(g) + e, a, b);
        x[0] = __uint_as_float(a.x); x[1] = __uint_as_float(a.y); x[2] = __uint_as_float(a.z); x[3] = __uint_as_float(a.w);
        x[4] = __uint_as_float(b.x); x[5] = __uint_as_float(b.y); x[6] = __uint_as_float(b.z); x[7] = __uint_as_float(b.w);
    } else {
        load8_grad<BF16>(g, e, x);
    }
}

// ---- pass 2, rank-1 tensors with cols % 128 == 0 ---------------------------------------------------

template <bool BF16>
struct RowRegs {           // one lane's share of one row: raw, still packed
    float4 w0, w1;
    uint4 g0, g1;          // bf16: g0 holds all 8 values; fp32: g0, g1
    uint32_t qm, qv;
    float am, r_old, r_rcp;
};

// Per-lane view of a tile: base pointers at the lane's first element and 32-bit offsets from there.
struct TileView {
    float* w;
    uint16_t* w16;         // optional bfloat16 copy of the parameters (same indexing as w), or nullptr
    const void* g;
    uint8_t* m_codes;
    uint8_t* v_codes;
    float* m_scale;
    float* v_bscale;       // VM == 2: block maxima of the second moment (same indexing as m_scale with B128)
    const float* r_old;
    const float* r_rcp;
    uint32_t row_step;     // elements between two rows this warp handles
    uint32_t row_stride;   // rows between them
    int m_shift;           // log2 of the first-moment block size
    float* s_red;          // CTA scratch for B2048 block maxima
    uint32_t* red_step;    // running count of CTA-wide reductions
    const char* pf_base;   // this lane's share of the row prefetch: one cache line of one of the arrays
    uint32_t pf_step;      // bytes between two of the warp's rows in that array (0: this lane prefetches nothing)
    const float* s_rows;   // fused schedule: shared memory, the tile's old row maxima [kFusedTileRows] followed by the
                           // reciprocals of its new ones, starting at this warp's first row
};

// Fused schedule: most rows an update tile may have (its row scalars are staged in shared memory).
constexpr int kFusedTileRows = 1024;
// Asks L2 to fetch this lane's share of row k ahead of time (no register is tied up): the later
// loads then find their data in L2 instead of waiting for DRAM.
constexpr uint32_t kL2Ahead = 4;   // rows
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// One instruction per row for the whole warp: the 256 elements a warp owns in a row are 8 lines of parameters,
// 4 (bf16) or 8 (fp32) lines of gradient, one line of each code array and one of block scales, and each of the
// first lanes asks for one of those lines.
template <bool BF16, int MSHIFT, int VM, bool FU = false>
__device__ __forceinline__ void prefetch_row(const TileView& t, uint32_t k) {
    if (t.pf_step != 0) prefetch_l2(t.pf_base + (size_t)k * t.pf_step);
}
// Assigns the lane its line (warp_* point at the warp's first element of row 0; row_step in elements).
// `valid` = how many of the warp's 256 columns exist (128 in a tensor's last warp column when cols % 256 == 128):
// no lane asks for a line past the end of the row.
template <bool BF16, int MSHIFT, int VM>
__device__ __forceinline__ void prefetch_roles(TileView& t, int lane, int valid, const float* warp_w, const void* warp_g,
                                               const uint8_t* warp_mq, const uint8_t* warp_vq, const float* warp_ms,
                                               const float* warp_vs) {
    constexpr int kGLines = BF16 ? 4 : 8;
    constexpr int kGLineElems = BF16 ? 64 : 32;
    t.pf_base = nullptr;
    t.pf_step = 0;
    if (lane < 8) {
        if (lane * 32 < valid) {
            t.pf_base = reinterpret_cast<const char*>(warp_w) + lane * 128;
            t.pf_step = t.row_step * 4u;
        }
    } else if (lane < 8 + kGLines) {
        if ((lane - 8) * kGLineElems < valid) {
            t.pf_base = reinterpret_cast<const char*>(warp_g) + (lane - 8) * 128;
            t.pf_step = t.row_step * (BF16 ? 2u : 4u);
        }
    } else if (lane == 8 + kGLines) {
        t.pf_base = reinterpret_cast<const char*>(warp_mq);
        t.pf_step = t.row_step / 2u;
    } else if (lane == 9 + kGLines && VM != 1) {
        t.pf_base = reinterpret_cast<const char*>(warp_vq);
        t.pf_step = t.row_step / 2u;
    } else if (lane == 10 + kGLines) {
        t.pf_base = reinterpret_cast<const char*>(warp_ms);
        t.pf_step = (t.row_step >> MSHIFT) * 4u;
    } else if (lane == 11 + kGLines && VM == 2) {
        t.pf_base = reinterpret_cast<const char*>(warp_vs);
        t.pf_step = (t.row_step >> 7) * 4u;
    }
}

// A32: the parameter rows (and fp32 gradient rows) of this tensor are 32-byte aligned.
template <bool BF16, int MSHIFT, int VM, bool A32, bool FU = false>
__device__ __forceinline__ void load_row(RowRegs<BF16>& r, const TileView& t, uint32_t k) {
    const uint32_t off = k * t.row_step;
    if (A32) {
        load8_f32_256(t.w + off, r.w0, r.w1);
    } else {
        r.w0 = *reinterpret_cast<const float4*>(t.w + off);
        r.w1 = *reinterpret_cast<const float4*>(t.w + off + 4);
    }
    if (BF16) {
        r.g0 = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(t.g) + off));
    } else if (A32) {
        load8_u32_256_nc(reinterpret_cast<const float*>(t.g) + off, r.g0, r.g1);
    } else {
        r.g0 = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(t.g) + off));
        r.g1 = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(t.g) + off + 4));
    }
    r.qm = *reinterpret_cast<const uint32_t*>(t.m_codes + (off >> 1));
    r.am = t.m_scale[off >> MSHIFT];
    if (VM == 2) {                                        // block-wise second moment: r_old carries the block's scale
        r.qv = *reinterpret_cast<const uint32_t*>(t.v_codes + (off >> 1));
        r.r_old = t.v_bscale[off >> 7];
        r.r_rcp = 0.0f;
        return;
    }
    if (FU) {
        r.qv = *reinterpret_cast<const uint32_t*>(t.v_codes + (off >> 1));
        r.r_old = t.s_rows[k * t.row_stride];
        r.r_rcp = t.s_rows[kFusedTileRows + k * t.row_stride];
        return;
    }
    r.r_rcp = __ldg(t.r_rcp + k * t.row_stride);        // VM == 1: the row factor R_i / sum(R)
    if (VM == 1) {
        r.qv = 0;
        r.r_old = 0.0f;
    } else {
        r.qv = *reinterpret_cast<const uint32_t*>(t.v_codes + (off >> 1));
        r.r_old = __ldg(t.r_old + k * t.row_stride);
    }
}

template <bool BF16, bool EXACT, int MSHIFT, int VM, bool WB, bool A32, bool FU = false>
__device__ __forceinline__ void process_row(const RowRegs<BF16>& r, const TileView& t, uint32_t k,
                                            const float (&c_old)[8], const float (&c_rcp)[8], const Hyper& h,
                                            const Hyper2& h2, const LaneTables& lt, const unsigned char* s_lut) {
    const uint32_t off = k * t.row_step;
    float wv[8] = {r.w0.x, r.w0.y, r.w0.z, r.w0.w, r.w1.x, r.w1.y, r.w1.z, r.w1.w};
    float gv[8], mt[8], vt[8], vs[8], vr[8];
    unpack_grad8<BF16>(r.g0, r.g1, gv);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        if (VM == 1) {
            vs[j] = __fmul_rn(r.r_rcp, c_rcp[j]);  // Sec. 4.3: v_ij = (R_i / sum R) * C_j
            vr[j] = 0.0f;
        } else if (VM == 2) {
            vs[j] = r.r_old;                       // Sec. 2.2: the block's maximum
            vr[j] = 0.0f;
        } else {
            vs[j] = fminf(r.r_old, c_old[j]);      // Sec. 4.2: scale = min(r_i, c_j)
            vr[j] = fmaxf(r.r_rcp, c_rcp[j]);      // 1/min(r', c') = max(1/r', 1/c')
        }
    }
    moments_and_update8<EXACT, VM == 1>(wv, gv, r.qm, r.qv, __fmul_rn(lt.de, r.am), vs, h, h2, lt, mt, vt);
    if (A32) store8_f32_256(t.w + off, wv); else store8_f32(t.w + off, wv);
    if (WB) store8_bf16(t.w16 + off, wv);
    const float am_new = block_max(absmax8(mt), MSHIFT, lt, t.s_red, *t.red_step);
    if ((threadIdx.x & (MSHIFT == 7 ? 15 : 2047)) == 0) t.m_scale[off >> MSHIFT] = am_new;
    *reinterpret_cast<uint32_t*>(t.m_codes + (off >> 1)) = quantize8_de(mt, scale_rcp(am_new), s_lut);
    if (VM == 2) {       // new block maximum of v_t (non-negative), its reciprocal for all eight elements
        const float av_new = group_max(absmax8(vt), lt.mask);
        if ((threadIdx.x & 15) == 0) t.v_bscale[off >> 7] = av_new;
        const float rv = scale_rcp(av_new);
#pragma unroll
        for (int j = 0; j < 8; ++j) vr[j] = rv;
    }
    if (VM != 1) *reinterpret_cast<uint32_t*>(t.v_codes + (off >> 1)) = quantize8_lin(vt, vr, h2);
}

// VM: how the second moment is kept: 0 rank-1 codes (Sec. 4.2), 1 factorized statistics (Sec. 4.3), 2 block-wise codes.
template <bool BF16, bool EXACT, int MSHIFT, int VM = 0, bool WB = false, bool A32 = false, bool FU = false>
__device__ __forceinline__ void pass2_rank1_fast(const TensorDesc& d, float* __restrict__ w, uint16_t* __restrict__ w16,
                                                 const void* __restrict__ g,
                                                 int tile, RcSel sel, const Hyper& h, const Hyper2& h2,
                                                 const LaneTables& lt, const unsigned char* s_lut, float* s_red,
                                                 uint32_t& red_step, float* s_rows = nullptr) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wx = d.wx, wy_count = kWarps / wx;
    const int tx = tile % d.tiles_x, ty = tile / d.tiles_x;
    if (FU) {
        // The tile's row scalars go to shared memory first (before any warp leaves): the old row maxima, and the
        // reciprocals of the new ones, which the maxima pass reduced earlier in this launch (read past L1).
        const int64_t r0 = (int64_t)ty * d.tile_rows;
        const int nr = (int)min((int64_t)d.tile_rows, d.rows - r0);
        const float* ro = rc_pick(d, sel.old_i) + r0;
        const float* rn = rc_pick(d, sel.new_i) + r0;
        for (int i = threadIdx.x; i < nr; i += kThreads) {
            s_rows[i] = __ldg(ro + i);
            s_rows[kFusedTileRows + i] = scale_rcp(__ldcg(rn + i));
        }
        __syncthreads();
    }
    const int64_t col0 = (int64_t)tx * (kWarpElems * wx) + (warp % wx) * kWarpElems + lane * kLaneElems;
    // cols % 128 == 0: a whole 16-lane group (one block) is in or out together. With B2048 the tile is one
    // block wide (wx = 8, cols % 2048 == 0), every warp is inside and all of them run the same rows.
    if (col0 >= d.cols) return;
    const float* rc_old = stats_old(d, sel);
    const float* rcp_new = d.rcp_new;
    const int64_t row0 = (int64_t)ty * d.tile_rows + warp / wx;
    const int64_t row_end = min((int64_t)(ty + 1) * d.tile_rows, d.rows);
    if (row0 >= row_end) return;
    const uint32_t nrows = (uint32_t)((row_end - row0 + wy_count - 1) / wy_count);
    // checking build: the lane's first and last accesses of this tile lie inside the tensor (B2048 tiles end rows in a
    // CTA-wide barrier, so there the failure is recorded and the tile goes on)
    if (!LPMM_DBG_OK(d, tile >= 0 && tile < d.tiles2 && col0 + kLaneElems <= d.cols && row0 + (int64_t)(nrows - 1) * wy_count < d.rows &&
                        (row0 + (int64_t)(nrows - 1) * wy_count) * d.cols + col0 + kLaneElems <= d.numel, 1) && MSHIFT == 7) return;

    float c_old[8], c_rcp[8];
    if (VM == 2) {   // no row / column statistics at all
#pragma unroll
        for (int j = 0; j < 8; ++j) { c_old[j] = 0.0f; c_rcp[j] = 0.0f; }
    } else if (VM == 1) {      // the new column statistics C_j sit in the "new" buffer; nothing old is needed
        load8_f32(rc_pick(d, sel.new_i) + d.c_off + col0, c_rcp);
#pragma unroll
        for (int j = 0; j < 8; ++j) c_old[j] = 0.0f;
    } else {
        load8_f32(rc_old + d.c_off + col0, c_old);
        if (FU) {   // the new column maxima c' were reduced earlier in this launch: read past L1, invert here
            load8_f32_cg(rc_pick(d, sel.new_i) + d.c_off + col0, c_rcp);
#pragma unroll
            for (int j = 0; j < 8; ++j) c_rcp[j] = scale_rcp(c_rcp[j]);
        } else {
            load8_f32(rcp_new + d.c_off + col0, c_rcp);
        }
    }
    const int64_t e0 = row0 * d.cols + col0;
    TileView t;
    t.w = w + e0;
    t.w16 = WB ? w16 + e0 : nullptr;
    t.g = BF16 ? static_cast<const void*>(reinterpret_cast<const uint16_t*>(g) + e0)
               : static_cast<const void*>(reinterpret_cast<const float*>(g) + e0);
    t.m_codes = d.m_codes + (e0 >> 1);
    t.v_codes = VM == 1 ? nullptr : d.v_codes + (e0 >> 1);
    t.v_bscale = VM == 2 ? d.v_bscale + (e0 >> 7) : nullptr;
    t.m_scale = d.m_scale + (e0 >> MSHIFT);
    t.r_old = rc_old + row0;
    t.r_rcp = rcp_new + row0;
    t.s_rows = FU ? s_rows + warp / wx : nullptr;
    t.row_step = (uint32_t)(wy_count * d.cols);
    t.row_stride = (uint32_t)wy_count;
    t.m_shift = d.m_shift;
    t.s_red = s_red;
    t.red_step = &red_step;
    {
        const int64_t ew = e0 - lane * kLaneElems;       // the warp's first element of its first row
        const int64_t left = d.cols - (col0 - lane * kLaneElems);
        prefetch_roles<BF16, MSHIFT, VM>(t, lane, left < kWarpElems ? (int)left : kWarpElems, w + ew,
                                           BF16 ? static_cast<const void*>(reinterpret_cast<const uint16_t*>(g) + ew)
                                                : static_cast<const void*>(reinterpret_cast<const float*>(g) + ew),
                                           d.m_codes + (ew >> 1), VM == 1 ? nullptr : d.v_codes + (ew >> 1), d.m_scale + (ew >> MSHIFT),
                                           VM == 2 ? d.v_bscale + (ew >> 7) : nullptr);
    }

    // Two register sets alternate: while one row is processed the next one is already in flight.
    RowRegs<BF16> ra, rb;
#pragma unroll
    for (uint32_t k = 1; k < kL2Ahead; ++k) if (k < nrows) prefetch_row<BF16, MSHIFT, VM, FU>(t, k);
    load_row<BF16, MSHIFT, VM, A32, FU>(ra, t, 0);
    uint32_t k = 0;
    // (B2048 rows end in a CTA-wide barrier, where the longer straight-line body only costs registers: guarded loop only)
    for (; MSHIFT == 7 && k + 1 + kL2Ahead < nrows; k += 2) {        // every row touched below exists: no guards
        prefetch_row<BF16, MSHIFT, VM, FU>(t, k + kL2Ahead);
        load_row<BF16, MSHIFT, VM, A32, FU>(rb, t, k + 1);
        process_row<BF16, EXACT, MSHIFT, VM, WB, A32, FU>(ra, t, k, c_old, c_rcp, h, h2, lt, s_lut);
        prefetch_row<BF16, MSHIFT, VM, FU>(t, k + 1 + kL2Ahead);
        load_row<BF16, MSHIFT, VM, A32, FU>(ra, t, k + 2);
        process_row<BF16, EXACT, MSHIFT, VM, WB, A32, FU>(rb, t, k + 1, c_old, c_rcp, h, h2, lt, s_lut);
    }
    for (; k < nrows; k += 2) {                       // the last rows of the tile
        const bool has_b = k + 1 < nrows;
        if (k + kL2Ahead < nrows) prefetch_row<BF16, MSHIFT, VM, FU>(t, k + kL2Ahead);
        if (has_b) load_row<BF16, MSHIFT, VM, A32, FU>(rb, t, k + 1);
        process_row<BF16, EXACT, MSHIFT, VM, WB, A32, FU>(ra, t, k, c_old, c_rcp, h, h2, lt, s_lut);
        if (!has_b) break;
        if (k + 1 + kL2Ahead < nrows) prefetch_row<BF16, MSHIFT, VM, FU>(t, k + 1 + kL2Ahead);
        if (k + 2 < nrows) load_row<BF16, MSHIFT, VM, A32, FU>(ra, t, k + 2);
        process_row<BF16, EXACT, MSHIFT, VM, WB, A32, FU>(rb, t, k + 1, c_old, c_rcp, h, h2, lt, s_lut);
    }
}

// ---- rank-1 normalization in the general form of Alg. 4 (element-indexed paths) --------------------
//
// The leading axes of the tensor are flattened into "rows". For row i the contribution of the leading axes to
// an element's scale is the minimum of their statistics at the row's multi-index (for the reciprocals of the
// new statistics: the maximum). A matrix has one leading axis and this is a single load.

// Row and column of flat element e of a rows x cols tensor (one 32-bit division when the indices allow it).
__device__ __forceinline__ void split_index(const TensorDesc& d, int64_t e, int64_t& i, int64_t& j) {
    if (d.numel <= 0xffffffffLL) {
        const uint32_t q = (uint32_t)e / (uint32_t)d.cols;
        i = q;
        j = (uint32_t)e - q * (uint32_t)d.cols;
    } else {
        i = e / d.cols;
        j = e - i * d.cols;
    }
}

// CG: the statistics were written earlier in the same launch (fused schedule): read them past L1.
template <bool MAX, bool CG = false>
__device__ __forceinline__ float outer_stat(const TensorDesc& d, const float* __restrict__ base, int64_t i) {
    if (d.n_outer == 1) return CG ? __ldcg(base + i) : __ldg(base + i);
    uint32_t rem = (uint32_t)i;                          // rows <= 2^30 (checked on the host)
    float s = MAX ? 0.0f : 3.402823466e38f;
#pragma unroll
    for (int a = 2; a >= 0; --a) {                       // the last leading axis varies fastest; constant indices keep
        if (a < d.n_outer) {                             // the descriptor in registers
            const uint32_t q = rem / (uint32_t)d.outer_dim[a];
            const float* px = base + d.outer_off[a] + (rem - q * (uint32_t)d.outer_dim[a]);
            const float x = CG ? __ldcg(px) : __ldg(px);
            s = MAX ? fmaxf(s, x) : fminf(s, x);
            rem = q;
        }
    }
    return s;
}
// Publishes the maximum of a run of elements of row i to every leading axis.
__device__ __forceinline__ void outer_publish(const TensorDesc& d, float* base, int64_t i, float x) {
    if (d.n_outer == 1) { atomic_max_nonneg_filtered(base + i, x); return; }
    uint32_t rem = (uint32_t)i;
#pragma unroll
    for (int a = 2; a >= 0; --a) {
        if (a < d.n_outer) {
            const uint32_t q = rem / (uint32_t)d.outer_dim[a];
            atomic_max_nonneg_filtered(base + d.outer_off[a] + (rem - q * (uint32_t)d.outer_dim[a]), x);
            rem = q;
        }
    }
}

// ---- pass 2, flat (element-indexed) tensors: block-wise v, or rank-1 with arbitrary cols ------

// Interior tiles of a matrix whose rows hold a whole number of lanes (cols % 8 == 0, cols >= 256) but not of
// first-moment blocks: the flat 128-aligned walk of pass2_flat() with everything that walk recomputes per chunk taken
// out of the loop. 32-bit offsets from the tile's first element; the (row, column) of a lane's elements is divided out
// once per tile and then stepped (a chunk step of 2048 elements passes at most eight row ends); the streaming operands of
// the next chunk are loaded before the current one is processed (two alternating register sets), the row and column
// statistics - which come from L1 - when they are needed.
template <bool BF16>
struct FlatRegs {
    float4 w0, w1;
    uint4 g0, g1;          // bf16: g0 only
    uint32_t qm, qv;
    float am;
};
template <bool BF16, bool A32>
__device__ __forceinline__ void flat_load(FlatRegs<BF16>& r, const float* w, const void* g, const uint8_t* mq, const uint8_t* vq,
                                          const float* ms, uint32_t off) {
    if (A32) {
        load8_f32_256(w + off, r.w0, r.w1);
    } else {
        r.w0 = *reinterpret_cast<const float4*>(w + off);
        r.w1 = *reinterpret_cast<const float4*>(w + off + 4);
    }
    if (BF16) {
        r.g0 = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(g) + off));
    } else if (A32) {
        load8_u32_256_nc(reinterpret_cast<const float*>(g) + off, r.g0, r.g1);
    } else {
        r.g0 = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(g) + off));
        r.g1 = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(g) + off + 4));
    }
    r.qm = *reinterpret_cast<const uint32_t*>(mq + (off >> 1));
    r.qv = *reinterpret_cast<const uint32_t*>(vq + (off >> 1));
    r.am = ms[off >> 7];
}
template <bool BF16, bool EXACT, bool WB, bool A32, bool FU>
__device__ __forceinline__ void pass2_flat_interior(const TensorDesc& d, float* __restrict__ w, uint16_t* __restrict__ w16,
                                                    const void* __restrict__ g, int tile, RcSel sel, const Hyper& h,
                                                    const Hyper2& h2, const LaneTables& lt, const unsigned char* s_lut) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t base = (int64_t)tile * d.flat_chunks * (kWarps * kWarpElems);
    const float* rc_old = stats_old(d, sel);
    const float* rcp_new = d.rcp_new;
    float* wb = w + base;
    uint16_t* w16b = WB ? w16 + base : nullptr;
    const void* gb = BF16 ? static_cast<const void*>(reinterpret_cast<const uint16_t*>(g) + base)
                          : static_cast<const void*>(reinterpret_cast<const float*>(g) + base);
    uint8_t* mq = d.m_codes + (base >> 1);
    uint8_t* vq = d.v_codes + (base >> 1);
    float* ms = d.m_scale + (base >> 7);
    uint32_t off = (uint32_t)(warp * kWarpElems + lane * kLaneElems);
    int64_t i64, j64;
    split_index(d, base + off, i64, j64);
    uint32_t i = (uint32_t)i64, j = (uint32_t)j64;
    const uint32_t cols = (uint32_t)d.cols;
    constexpr uint32_t kStep = kWarps * kWarpElems;
    FlatRegs<BF16> ra, rb;
    flat_load<BF16, A32>(ra, wb, gb, mq, vq, ms, off);
    const int n = d.flat_chunks;
    for (int c = 0; c < n; ++c) {
        FlatRegs<BF16>& cur = (c & 1) ? rb : ra;
        FlatRegs<BF16>& nxt = (c & 1) ? ra : rb;
        if (c + 1 < n) flat_load<BF16, A32>(nxt, wb, gb, mq, vq, ms, off + kStep);
        float wv[8] = {cur.w0.x, cur.w0.y, cur.w0.z, cur.w0.w, cur.w1.x, cur.w1.y, cur.w1.z, cur.w1.w};
        float gv[8], mt[8], vt[8], vs[8], vr[8], co[8], cr[8];
        unpack_grad8<BF16>(cur.g0, cur.g1, gv);
        const float so = __ldg(rc_old + i);
        const float ro = FU ? __ldcg(rcp_new + i) : __ldg(rcp_new + i);
        load8_f32(rc_old + d.c_off + j, co);
        if (FU) load8_f32_cg(rcp_new + d.c_off + j, cr);
        else load8_f32(rcp_new + d.c_off + j, cr);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            vs[k] = fminf(so, co[k]);
            vr[k] = fmaxf(ro, cr[k]);
        }
        moments_and_update8<EXACT>(wv, gv, cur.qm, cur.qv, __fmul_rn(lt.de, cur.am), vs, h, h2, lt, mt, vt);
        store8_f32_a<A32>(wb + off, wv);
        if (WB) store8_bf16(w16b + off, wv);
        const float am_new = group_max(absmax8(mt), lt.mask);
        if ((lane & 15) == 0) ms[off >> 7] = am_new;
        *reinterpret_cast<uint32_t*>(mq + (off >> 1)) = quantize8_de(mt, scale_rcp(am_new), s_lut);
        *reinterpret_cast<uint32_t*>(vq + (off >> 1)) = quantize8_lin(vt, vr, h2);
        off += kStep;
        j += kStep;
        while (j >= cols) { j -= cols; ++i; }     // cols >= 256: at most eight rows per chunk step
    }
}

// (FU: called from the fused kernel, which reads the new reciprocals past L1 and, to keep its register allocation,
// does without the interior loop.)
template <bool BF16, bool RANK1, bool EXACT, int MSHIFT, bool WB = false, bool A32 = false, bool FU = false>
__device__ __forceinline__ void pass2_flat(const TensorDesc& d, float* __restrict__ w, uint16_t* __restrict__ w16,
                                           const void* __restrict__ g,
                                           int tile, RcSel sel, const Hyper& h, const Hyper2& h2, const LaneTables& lt,
                                           const unsigned char* s_lut, float* s_red, uint32_t& red_step) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float* rc_old = stats_old(d, sel);
    const float* rcp_new = d.rcp_new;
    const int64_t m_mask = ((int64_t)1 << MSHIFT) - 1;
    // checking build: the tile starts inside the tensor (B2048: recorded only, the CTA-wide barrier needs every warp)
    if (!LPMM_DBG_OK(d, tile >= 0 && (int64_t)tile * d.flat_chunks * kWarps * kWarpElems < d.numel, 3) && MSHIFT == 7) return;
    if (!FU && RANK1 && MSHIFT == 7 && d.n_outer == 1 && (d.cols & 7) == 0 && d.cols >= kWarpElems &&
        (int64_t)(tile + 1) * d.flat_chunks * (kWarps * kWarpElems) <= d.numel) {   // uniform over the CTA
        pass2_flat_interior<BF16, EXACT, WB, A32, FU>(d, w, w16, g, tile, sel, h, h2, lt, s_lut);
        return;
    }
    for (int c = 0; c < d.flat_chunks; ++c) {
        const int64_t chunk0 = ((int64_t)tile * d.flat_chunks + c) * kWarps;   // the CTA's 8 chunks = 2048 elements
        const int64_t chunk = chunk0 + warp;
        const int64_t e = chunk * kWarpElems + lane * kLaneElems;
        if (chunk0 * kWarpElems >= d.numel) break;          // uniform over the CTA
        // B128: a warp past the end has nothing to do. B2048: it still joins the CTA-wide block maximum
        // (with zeros; its loads and stores are all guarded away).
        if (MSHIFT == 7 && chunk * kWarpElems >= d.numel) break;
        const bool full = (chunk + 1) * kWarpElems <= d.numel;
        if (c + 2 < d.flat_chunks) {
            // L2 hint for the warp's chunk after next (one line per lane: 8 of parameters, 4 or 8 of gradient, one of
            // each code array), so that its loads find their data in L2
            const int64_t en = (chunk + 2 * kWarps) * kWarpElems;
            if (en + kWarpElems <= d.numel) {
                constexpr int kG = BF16 ? 4 : 8;
                const char* p = nullptr;
                if (lane < 8) p = reinterpret_cast<const char*>(w + en) + lane * 128;
                else if (lane < 8 + kG) p = reinterpret_cast<const char*>(g) + en * (BF16 ? 2 : 4) + (lane - 8) * 128;
                else if (lane == 8 + kG) p = reinterpret_cast<const char*>(d.m_codes) + (en >> 1);
                else if (lane == 9 + kG) p = reinterpret_cast<const char*>(d.v_codes) + (en >> 1);
                if (p) prefetch_l2(p);
            }
        }
        float wv[8], gv[8], mt[8], vt[8], vs[8], vr[8];
        uint32_t qm, qv;
        if (full) {
            load8_rw_a<A32>(w + e, wv);
            load8_grad_a<BF16, A32>(g, e, gv);
            qm = __ldg(reinterpret_cast<const uint32_t*>(d.m_codes + (e >> 1)));
            qv = __ldg(reinterpret_cast<const uint32_t*>(d.v_codes + (e >> 1)));
        } else {
            load8_guard(w, e, d.numel, wv);
            load8_grad_guard<BF16>(g, e, d.numel, gv);
            qm = load_codes_guard(d.m_codes, e, d.numel);
            qv = load_codes_guard(d.v_codes, e, d.numel);
        }
        const bool lane_live = e < d.numel;
        // every lane of a 16-lane group that still holds an element needs the block's scale: the
        // shuffle-based table lookup reads T[q] * scale from the group's other lanes
        const bool group_live = (e & ~m_mask) < d.numel;
        const float am = group_live ? d.m_scale[e >> MSHIFT] : 0.0f;
        if (RANK1 && full && (d.cols & 7) == 0) {
            // cols % 8 == 0: the lane's eight elements lie in one row, their column statistics are two 16-byte loads
            int64_t i, j;
            split_index(d, e, i, j);
            const float so = outer_stat<false>(d, rc_old, i), ro = outer_stat<true, FU>(d, rcp_new, i);
            float co[8], cr[8];
            load8_f32(rc_old + d.c_off + j, co);
            if (FU) load8_f32_cg(rcp_new + d.c_off + j, cr);
            else load8_f32(rcp_new + d.c_off + j, cr);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                vs[k] = fminf(so, co[k]);
                vr[k] = fmaxf(ro, cr[k]);
            }
        } else if (RANK1) {
            int64_t i, j;
            split_index(d, e, i, j);
            float so = 0.0f, ro = 0.0f;          // leading axes' share of the old scale / the new reciprocal, row i
            bool fresh = true;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if (e + k < d.numel) {
                    if (fresh) {
                        so = outer_stat<false>(d, rc_old, i);
                        ro = outer_stat<true, FU>(d, rcp_new, i);
                        fresh = false;
                    }
                    vs[k] = fminf(so, __ldg(rc_old + d.c_off + j));
                    vr[k] = fmaxf(ro, FU ? __ldcg(rcp_new + d.c_off + j) : __ldg(rcp_new + d.c_off + j));
                } else {
                    vs[k] = 0.0f; vr[k] = 0.0f;
                }
                if (++j == d.cols) { j = 0; ++i; fresh = true; }
            }
        } else {
            const float av = lane_live ? d.v_bscale[e >> 7] : 0.0f;
#pragma unroll
            for (int k = 0; k < 8; ++k) vs[k] = av;
        }
        moments_and_update8<EXACT>(wv, gv, qm, qv, __fmul_rn(lt.de, am), vs, h, h2, lt, mt, vt);
        if (!full) {   // elements beyond the tensor must not reach a block maximum
#pragma unroll
            for (int k = 0; k < 8; ++k) if (e + k >= d.numel) { mt[k] = 0.0f; vt[k] = 0.0f; }
        }
        const float am_new = block_max(absmax8(mt), MSHIFT, lt, s_red, red_step);
        if (!RANK1) {
            const float av_new = half_warp_max(absmax8(vt));
            const float r = scale_rcp(av_new);
#pragma unroll
            for (int k = 0; k < 8; ++k) vr[k] = r;
            if (lane_live && (lane & 15) == 0) d.v_bscale[e >> 7] = av_new;
        }
        if (lane_live && (threadIdx.x & (MSHIFT == 7 ? 15 : 2047)) == 0) d.m_scale[e >> MSHIFT] = am_new;
        const uint32_t qm_new = quantize8_de(mt, scale_rcp(am_new), s_lut);
        const uint32_t qv_new = quantize8_lin(vt, vr, h2);
        if (WB) {
            if (full) store8_bf16(w16 + e, wv); else store8_bf16_guard(w16, e, d.numel, wv);
        }
        if (full) {
            store8_f32_a<A32>(w + e, wv);
            *reinterpret_cast<uint32_t*>(d.m_codes + (e >> 1)) = qm_new;
            *reinterpret_cast<uint32_t*>(d.v_codes + (e >> 1)) = qv_new;
        } else {
            store8_guard(w, e, d.numel, wv);
            store_codes_guard(d.m_codes, e, d.numel, qm_new);
            store_codes_guard(d.v_codes, e, d.numel, qv_new);
        }
    }
}

// ---- pass 2, small tensors with fp32 states (App. D.1) ------------------------------------------

template <bool BF16, bool EXACT, bool WB = false, bool A32 = false>
__device__ __forceinline__ void pass2_fp32(const TensorDesc& d, float* __restrict__ w, uint16_t* __restrict__ w16,
                                           const void* __restrict__ g, int tile, const Hyper& h) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (!LPMM_DBG_OK(d, tile >= 0 && (int64_t)tile * d.flat_chunks * kWarps * kWarpElems < d.numel && d.m32 != nullptr && d.v32 != nullptr, 4)) return;
    for (int c = 0; c < d.flat_chunks; ++c) {
        const int64_t chunk = ((int64_t)tile * d.flat_chunks + c) * kWarps + warp;
        const int64_t e = chunk * kWarpElems + lane * kLaneElems;
        if (chunk * kWarpElems >= d.numel) break;
        const bool full = (chunk + 1) * kWarpElems <= d.numel;
        float wv[8], gv[8], m[8], v[8];
        if (full) {
            // (the fp32 states live in the arena at 256-byte aligned offsets: always 32-byte aligned here)
            load8_rw_a<A32>(w + e, wv); load8_grad_a<BF16, A32>(g, e, gv); load8_rw_a<true>(d.m32 + e, m); load8_rw_a<true>(d.v32 + e, v);
        } else {
            load8_guard(w, e, d.numel, wv); load8_grad_guard<BF16>(g, e, d.numel, gv);
            load8_guard(d.m32, e, d.numel, m); load8_guard(d.v32, e, d.numel, v);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            m[k] = ema_m(m[k], gv[k], h);
            v[k] = ema_v(v[k], gv[k], h);
            wv[k] = update_param<EXACT>(wv[k], m[k], v[k], h);
        }
        if (WB) {
            if (full) store8_bf16(w16 + e, wv); else store8_bf16_guard(w16, e, d.numel, wv);
        }
        if (full) {
            store8_f32_a<A32>(w + e, wv); store8_f32_a<true>(d.m32 + e, m); store8_f32_a<true>(d.v32 + e, v);
        } else {
            store8_guard(w, e, d.numel, wv); store8_guard(d.m32, e, d.numel, m); store8_guard(d.v32, e, d.numel, v);
        }
    }
}

// VF: how the state keeps the second moment of its tiled tensors: 0 rank-1 codes, 1 factorized, 2 block-wise codes.
// A state has tiled tensors of one of these kinds only, so each instantiation carries only one tiled path.
// WB: a bfloat16 copy of every updated parameter is written as well (a.params_bf16).
// A32: every parameter pointer (and, with fp32 gradients, every gradient pointer) of the step is 32-byte aligned,
// checked on the host: the tiled path then moves a lane's 8 values with one 256-bit access.
// MISC: false = the tensors on the tiled path and the small tensors with fp32 states; true = the element-indexed ones
// (odd shapes, ragged or short 1-D tensors). They are two kernels (two launches per step when a state has both) so that
// the register allocation of the tiled path - where nearly all parameters of a real model are - is not shared with
// the element-indexed paths: with both in one kernel the update pass of the LLaMA-7B list took 13.9-14.0 ms instead
// of 13.3-13.4.
template <bool BF16, bool EXACT, int MSHIFT, int VF, bool WB, bool A32, bool MISC = false>
__global__ void __launch_bounds__(kThreads, 2) pass2_kernel(StepArgs a) {
    __shared__ __align__(16) unsigned char s_lut[kLutSmemBytes];
    __shared__ float s_red[2 * kWarps];
    load_lut_smem(s_lut);
    __syncthreads();
    const LaneTables lt = make_lane_tables();
    const Hyper2& h2 = a.h2;
    uint32_t red_step = 0;
    __shared__ int s_next[2];
    int buf = 0;
    for (int tile = a.tile_begin + tiles_first(a.tile_counter, s_next); tile < a.tile_end;) {
        const int fetched = tiles_fetch(a.tile_counter);
        const int t = find_tensor(a.tile_start, a.n_tensors, tile);
        const TensorDesc d = a.descs[t];   // by value: the fields stay in registers across the stores below
        float* w = a.params[t];
        uint16_t* w16 = WB ? a.params_bf16[t] : nullptr;
        const void* g = a.grads[t];
        const int local = tile - __ldg(a.tile_start + t);
        if (MISC) {
            switch (d.kind) {
                case K_RANK1_FLAT: pass2_flat<BF16, true, EXACT, MSHIFT, WB, A32>(d, w, w16, g, local, a.sel, a.h, h2, lt, s_lut, s_red, red_step); break;
                case K_BLOCK:      pass2_flat<BF16, false, EXACT, MSHIFT, WB, A32>(d, w, w16, g, local, a.sel, a.h, h2, lt, s_lut, s_red, red_step); break;
                default: break;
            }
        } else {
            switch (d.kind) {
                case K_RANK1_FAST:
                    if (VF == 0) pass2_rank1_fast<BF16, EXACT, MSHIFT, 0, WB, A32>(d, w, w16, g, local, a.sel, a.h, h2, lt, s_lut, s_red, red_step);
                    break;
                case K_FACT:
                    if (VF == 1) pass2_rank1_fast<BF16, EXACT, MSHIFT, 1, WB>(d, w, w16, g, local, a.sel, a.h, h2, lt, s_lut, s_red, red_step);
                    break;
                case K_BLOCK_TILED:   // matrices of a block-wise state; long 1-D tensors folded into rows (in states of another
                                      // kind these get a launch of their own, so that the default kernels stay lean)
                    if (VF == 2) pass2_rank1_fast<BF16, EXACT, MSHIFT, 2, WB, A32>(d, w, w16, g, local, a.sel, a.h, h2, lt, s_lut, s_red, red_step);
                    break;
                case K_FP32:      // small tensors with fp32 states ride along (a short, register-light path)
                    pass2_fp32<BF16, EXACT, WB, A32>(d, w, w16, g, local, a.h);
                    break;
                default: break;
            }
        }
        tile = a.tile_begin + tiles_next(s_next, buf, fetched);
    }
    tiles_done(a.tile_counter);
}

// ---- pass 1: new row / column maxima of v_t for rank-1 tensors -----------------------------------
//
// Maxima are idempotent, so ragged edges are handled by clamping indices onto valid rows / column
// groups (a duplicate contributes the same value again) instead of predicating the loads.

template <bool BF16>
struct P1Row {             // one lane's share of one row
    uint4 g0, g1;          // bf16: g0 only
    uint32_t qv;
};

struct P1View {
    const void* g;             // at the lane's first element of the tile (row i0, the lane's 8 columns)
    const uint8_t* v_codes;    // likewise
    uint32_t row_step;         // elements between two rows this warp handles
    const char* pf_base;       // this lane's share of the prefetch of a group of rows: one line of one array in one row
    uint32_t pf_step;          // bytes between two of the warp's rows in that array (0: nothing to prefetch)
    uint32_t pf_row;           // which row of the group
    uint64_t pol;              // fused schedule: cache policy of the loads (evict last where the tile is meant to stay in L2)
    bool keep;                 // fused schedule: whether the prefetch hints ask for evict-last lines
};

template <bool BF16, bool FU = false>
__device__ __forceinline__ void load_p1_row(P1Row<BF16>& b, const P1View& t, uint32_t k) {
    const uint32_t off = k * t.row_step;
    if (FU) {
        if (BF16) {
            b.g0 = load4_u32_nc_h(reinterpret_cast<const uint16_t*>(t.g) + off, t.pol);
        } else {
            b.g0 = load4_u32_nc_h(reinterpret_cast<const float*>(t.g) + off, t.pol);
            b.g1 = load4_u32_nc_h(reinterpret_cast<const float*>(t.g) + off + 4, t.pol);
        }
        b.qv = load1_u32_nc_h(t.v_codes + (off >> 1), t.pol);
        return;
    }
    if (BF16) {
        b.g0 = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(t.g) + off));
    } else {
        b.g0 = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(t.g) + off));
        b.g1 = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(t.g) + off + 4));
    }
    b.qv = __ldg(reinterpret_cast<const uint32_t*>(t.v_codes + (off >> 1)));
}

// L2 prefetch of a group of rows with one instruction for the whole warp: a row of the warp is 4 (bf16) or 8
// (fp32) lines of gradient and one line of codes, so 4 (2) rows fit the 32 lanes.
template <bool BF16> struct P1Pf {
    static constexpr int kGLines = BF16 ? 4 : 8;
    static constexpr int kLines = kGLines + 1;
    static constexpr int kRows = BF16 ? 4 : 2;          // rows per instruction
};
template <bool BF16>
__device__ __forceinline__ void p1_prefetch_roles(P1View& t, int lane, int valid, const void* warp_g, const uint8_t* warp_vq) {
    const int u = lane / P1Pf<BF16>::kLines, item = lane - u * P1Pf<BF16>::kLines;
    t.pf_base = nullptr;
    t.pf_step = 0;
    t.pf_row = (uint32_t)u;
    if (u >= P1Pf<BF16>::kRows) return;
    if (item < P1Pf<BF16>::kGLines) {
        if (item * (BF16 ? 64 : 32) < valid) {
            t.pf_base = reinterpret_cast<const char*>(warp_g) + item * 128;
            t.pf_step = t.row_step * (BF16 ? 2u : 4u);
        }
    } else {
        t.pf_base = reinterpret_cast<const char*>(warp_vq);
        t.pf_step = t.row_step / 2u;
    }
}
// Rows k .. k + kRows - 1 (those below nrows).
__device__ __forceinline__ void prefetch_l2_keep(const void* p) { asm volatile("prefetch.global.L2::evict_last [%0];" ::"l"(p)); }
template <bool BF16, bool FU = false>
__device__ __forceinline__ void prefetch_p1_group(const P1View& t, uint32_t k, uint32_t nrows) {
    const uint32_t row = k + t.pf_row;
    if (t.pf_step != 0 && row < nrows) {
        if (FU && t.keep) prefetch_l2_keep(t.pf_base + (size_t)row * t.pf_step);
        else prefetch_l2(t.pf_base + (size_t)row * t.pf_step);
    }
}

// Maxima of four per-lane values over the warp with 6 shuffles: afterwards the lanes with
// (lane & 7) == 0 hold the warp-wide maximum of value number 2 * bit4(lane) + bit3(lane).
__device__ __forceinline__ float warp_max4(const float (&r)[4], int lane) {
    const bool h16 = lane & 16, h8 = lane & 8;
    float k0 = h16 ? r[2] : r[0], k1 = h16 ? r[3] : r[1];
    const float s0 = h16 ? r[0] : r[2], s1 = h16 ? r[1] : r[3];
    k0 = fmaxf(k0, __shfl_xor_sync(0xffffffffu, s0, 16));
    k1 = fmaxf(k1, __shfl_xor_sync(0xffffffffu, s1, 16));
    float k = h8 ? k1 : k0;
    const float s = h8 ? k0 : k1;
    k = fmaxf(k, __shfl_xor_sync(0xffffffffu, s, 8));
    k = fmaxf(k, __shfl_xor_sync(0xffffffffu, k, 4));
    k = fmaxf(k, __shfl_xor_sync(0xffffffffu, k, 2));
    k = fmaxf(k, __shfl_xor_sync(0xffffffffu, k, 1));
    return k;
}

// New second moments of one row; accumulates the column maxima and returns the lane's row maximum.
template <bool BF16>
__device__ __forceinline__ float p1_process_row(const P1Row<BF16>& b, float r_old, const float (&c_old)[8],
                                                float (&c_max)[8], const Hyper2& h2, const LaneTables& lt) {
    float gv[8];
    unpack_grad8<BF16>(b.g0, b.g1, gv);
    float rm = 0.0f;
#pragma unroll
    for (int k = 0; k < 8; k += 2) {
        // (this pass is bound by the logic/min-max pipe, so the table entry comes from a shuffle here, not from
        // the arithmetic of lin_dequant8() as in the update pass, which is short of shuffle/shared-memory slots)
        const float2 tl = make_float2(__shfl_sync(0xffffffffu, lt.lin, (int)(b.qv >> (4 * k)), 16),
                                      __shfl_sync(0xffffffffu, lt.lin, (int)(b.qv >> (4 * k + 4)), 16));
        const float2 sc = make_float2(fminf(r_old, c_old[k]), fminf(r_old, c_old[k + 1]));
        const float2 vt = ema_v2(mul2_rn(tl, sc), make_float2(gv[k], gv[k + 1]), h2);
        rm = fmaxf(rm, fmaxf(vt.x, vt.y));
        c_max[k] = fmaxf(c_max[k], vt.x);
        c_max[k + 1] = fmaxf(c_max[k + 1], vt.y);
    }
    return rm;
}

// Two rows at once: the column maxima take one three-input maximum per column for both rows.
template <bool BF16>
__device__ __forceinline__ void p1_process_2rows(const P1Row<BF16>& a, const P1Row<BF16>& b, float ra_old, float rb_old,
                                                 const float (&c_old)[8], float (&c_max)[8], const Hyper2& h2,
                                                 const LaneTables& lt, float& rm_a, float& rm_b) {
    float ga[8], gb[8];
    unpack_grad8<BF16>(a.g0, a.g1, ga);
    unpack_grad8<BF16>(b.g0, b.g1, gb);
    rm_a = 0.0f;
    rm_b = 0.0f;
#pragma unroll
    for (int k = 0; k < 8; k += 2) {
        const float2 ta = make_float2(__shfl_sync(0xffffffffu, lt.lin, (int)(a.qv >> (4 * k)), 16),
                                      __shfl_sync(0xffffffffu, lt.lin, (int)(a.qv >> (4 * k + 4)), 16));
        const float2 tb = make_float2(__shfl_sync(0xffffffffu, lt.lin, (int)(b.qv >> (4 * k)), 16),
                                      __shfl_sync(0xffffffffu, lt.lin, (int)(b.qv >> (4 * k + 4)), 16));
        const float2 sa = make_float2(fminf(ra_old, c_old[k]), fminf(ra_old, c_old[k + 1]));
        const float2 sb = make_float2(fminf(rb_old, c_old[k]), fminf(rb_old, c_old[k + 1]));
        const float2 va = ema_v2(mul2_rn(ta, sa), make_float2(ga[k], ga[k + 1]), h2);
        const float2 vb = ema_v2(mul2_rn(tb, sb), make_float2(gb[k], gb[k + 1]), h2);
        rm_a = fmaxf(rm_a, fmaxf(va.x, va.y));
        rm_b = fmaxf(rm_b, fmaxf(vb.x, vb.y));
        c_max[k] = fmaxf(c_max[k], fmaxf(va.x, vb.x));
        c_max[k + 1] = fmaxf(c_max[k + 1], fmaxf(va.y, vb.y));
    }
}

constexpr uint32_t kP1L2Ahead = 8;  // rows the L2 prefetch hints run ahead

template <bool BF16, bool FU = false>
__device__ __forceinline__ void pass1_rank1_fast(const TensorDesc& d, const void* __restrict__ g, int tile, RcSel sel,
                                                 const Hyper2& h2, const LaneTables& lt, float* s_col, uint64_t pol = 0,
                                                 bool keep = false) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wx = d.wx, wy_count = kWarps / wx;
    const int tx = tile % d.tiles_x, ty = tile / d.tiles_x;
    const int64_t col_w = (int64_t)tx * (kWarpElems * wx) + (warp % wx) * kWarpElems;   // first column of this warp
    int64_t col0 = col_w + lane * kLaneElems;
    // Maxima are idempotent: lanes beyond the last column (cols % 256 != 0) repeat its last eight columns.
    if (col0 >= d.cols) col0 = d.cols - kLaneElems;
    const float* rc_old = stats_old(d, sel);
    float* rc_new = stats_new(d, sel);
    const int64_t row0 = (int64_t)ty * d.tile_rows1 + warp / wx;
    const int64_t row_end = min((int64_t)(ty + 1) * d.tile_rows1, d.rows);
    if (row0 >= row_end) return;                      // uniform over the warp
    const uint32_t nrows = (uint32_t)((row_end - row0 + wy_count - 1) / wy_count);
    if (!LPMM_DBG_OK(d, tile >= 0 && tile < d.tiles1 && col0 >= 0 && col0 + kLaneElems <= d.cols &&
                        row0 + (int64_t)(nrows - 1) * wy_count < d.rows, 2)) return;

    float c_old[8], c_max[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) c_max[k] = 0.0f;
    load8_f32(rc_old + d.c_off + col0, c_old);
    const int64_t e0 = row0 * d.cols + col0;
    P1View t;
    t.pol = pol;
    t.keep = keep;
    t.g = BF16 ? static_cast<const void*>(reinterpret_cast<const uint16_t*>(g) + e0)
               : static_cast<const void*>(reinterpret_cast<const float*>(g) + e0);
    t.v_codes = d.v_codes + (e0 >> 1);
    t.row_step = (uint32_t)(wy_count * d.cols);

    {
        const int64_t ew = row0 * d.cols + col_w;          // the warp's first element of its first row
        const int64_t left = d.cols - col_w;
        p1_prefetch_roles<BF16>(t, lane, left < kWarpElems ? (int)left : kWarpElems,
                                BF16 ? static_cast<const void*>(reinterpret_cast<const uint16_t*>(g) + ew)
                                     : static_cast<const void*>(reinterpret_cast<const float*>(g) + ew),
                                d.v_codes + (ew >> 1));
    }
#pragma unroll
    for (uint32_t k = 0; k < kP1L2Ahead; k += P1Pf<BF16>::kRows) prefetch_p1_group<BF16, FU>(t, k, nrows);
    // Lane j keeps the old row scale of the warp's row number base + j (32 rows per refill); a row's scale is
    // then read with one shuffle instead of a load.
    float r_vec = 0.0f;
    // Four register sets: the rows of a trip were loaded during the previous trip (four rows of loads in flight per
    // lane). Maxima are idempotent, so row numbers are clamped to the tile's last row instead of guarded: a trip
    // past the end re-reads that row and contributes the same values again, and the loop body has no branches.
    P1Row<BF16> s0, s1, s2, s3;
    const uint32_t last = nrows - 1;
    load_p1_row<BF16, FU>(s0, t, 0);
    load_p1_row<BF16, FU>(s1, t, min(1u, last));
    load_p1_row<BF16, FU>(s2, t, min(2u, last));
    load_p1_row<BF16, FU>(s3, t, min(3u, last));
    for (uint32_t k = 0; k < nrows; k += 4) {         // four rows per trip so that their maxima reduce together
        if ((k & 31) == 0) {
            const uint32_t kk = min(k + lane, last);
            r_vec = __ldg(rc_old + row0 + (int64_t)kk * wy_count);
        }
#pragma unroll
        for (uint32_t u = 0; u < 4; u += P1Pf<BF16>::kRows) prefetch_p1_group<BF16, FU>(t, k + kP1L2Ahead + u, nrows);
        float r_max[4];
        p1_process_2rows<BF16>(s0, s1, __shfl_sync(0xffffffffu, r_vec, k & 31), __shfl_sync(0xffffffffu, r_vec, (k + 1) & 31),
                               c_old, c_max, h2, lt, r_max[0], r_max[1]);
        load_p1_row<BF16, FU>(s0, t, min(k + 4, last));
        load_p1_row<BF16, FU>(s1, t, min(k + 5, last));
        p1_process_2rows<BF16>(s2, s3, __shfl_sync(0xffffffffu, r_vec, (k + 2) & 31), __shfl_sync(0xffffffffu, r_vec, (k + 3) & 31),
                               c_old, c_max, h2, lt, r_max[2], r_max[3]);
        load_p1_row<BF16, FU>(s2, t, min(k + 6, last));
        load_p1_row<BF16, FU>(s3, t, min(k + 7, last));
        const float rm = warp_max4(r_max, lane);
        const uint32_t kr = min(k + ((lane >> 4) & 1) * 2 + ((lane >> 3) & 1), last);   // the row whose maximum this lane holds
        if ((lane & 7) == 0) atomic_max_nonneg(rc_new + row0 + (int64_t)kr * wy_count, rm);
    }
    // Column maxima: transpose through this warp's slice of shared memory so that consecutive lanes hold
    // consecutive columns, then one atomic per column. Only the warp itself touches its slice.
    float* mine = s_col + warp * kWarpElems;
    __syncwarp();
#pragma unroll
    for (int k = 0; k < 8; ++k) mine[lane * kLaneElems + k] = c_max[k];
    __syncwarp();
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int cc = lane + 32 * k;
        if (col_w + cc < d.cols) atomic_max_nonneg(rc_new + d.c_off + col_w + cc, mine[cc]);
    }
}

// ---- pass 1 of the factorized second moment: row and column sums of g^2 (Sec. 4.3) ---------------------
//
// Same tiling as the maxima pass. Nothing is accumulated with atomics: every tile writes partial sums to a scratch
// region of the arena and two small kernels add them up in a fixed order, so R and C are reproducible bit for bit
// from run to run (and from GPU to GPU).
//   row i:    one partial per 256-column strip (a lane adds its eight squares in order, then a shuffle tree over the
//             warp), rowpart[i * nstrips + strip];
//   column j: one partial per tile row-block: every warp adds its rows in increasing order with a compensated
//             (Kahan) sum, so that the rounding error does not grow with the tile's height; the warps that share a
//             column strip are combined in warp order through shared memory, colpart[ty * cols + j].
// All arithmetic is binary32; the finalize kernels add the partials in binary64.

[[maybe_unused]] __device__ __forceinline__ void kahan_add(float& s, float& c, float x) {
    const float y = __fsub_rn(x, c);
    const float t = __fadd_rn(s, y);
    c = __fsub_rn(__fsub_rn(t, s), y);
    s = t;
}

template <bool BF16>
__device__ __forceinline__ void pass1_fact(const TensorDesc& d, const void* __restrict__ g, int tile, float* s_col) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wx = d.wx, wy_count = kWarps / wx;
    const int tx = tile % d.tiles_x, ty = tile / d.tiles_x;
    const int64_t col_w = (int64_t)tx * (kWarpElems * wx) + (warp % wx) * kWarpElems;
    const int64_t col0 = col_w + lane * kLaneElems;
    const bool active = col0 < d.cols;                  // cols % 256 == 128: the upper half-warp adds zeros
    const bool strip_exists = col_w < d.cols;
    const int64_t strip = col_w / kWarpElems;
    const int64_t row0 = (int64_t)ty * d.tile_rows1 + warp / wx;
    const int64_t row_end = min((int64_t)(ty + 1) * d.tile_rows1, d.rows);
    float c_sum[8], c_cmp[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) { c_sum[k] = 0.0f; c_cmp[k] = 0.0f; }
    for (int64_t i = row0; i < row_end; i += 4 * wy_count) {     // four rows of loads in flight
        float gv[4][8];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t r = i + (int64_t)u * wy_count;
            if (active && r < row_end) {
                load8_grad<BF16>(g, r * d.cols + col0, gv[u]);
            } else {
#pragma unroll
                for (int k = 0; k < 8; ++k) gv[u][k] = 0.0f;
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t r = i + (int64_t)u * wy_count;
            float rs = 0.0f;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const float gg = __fmul_rn(gv[u][k], gv[u][k]);
                rs = __fadd_rn(rs, gg);
                kahan_add(c_sum[k], c_cmp[k], gg);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) rs = __fadd_rn(rs, __shfl_xor_sync(0xffffffffu, rs, o));
            if (lane == 0 && strip_exists && r < row_end) d.fact_rowpart[r * d.fact_nstrips + strip] = rs;
        }
    }
    float* mine = s_col + warp * kWarpElems;
#pragma unroll
    for (int k = 0; k < 8; ++k) mine[lane * kLaneElems + k] = c_sum[k];
    __syncthreads();
    if (warp < wx) {                                    // the first warp of every column strip adds the strip's warps in order
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int cc = lane + 32 * k;
            float t = 0.0f;
            for (int wy = 0; wy < wy_count; ++wy) t = __fadd_rn(t, s_col[(wy * wx + warp) * kWarpElems + cc]);
            if (col_w + cc < d.cols) d.fact_colpart[(int64_t)ty * d.cols + col_w + cc] = t;
        }
    }
    // (the tile loop's barrier comes before anybody writes s_col again)
}

#if LPMM_STEP_PART == 0   // non-template kernels live in one part only
// Finalize: one CTA per 32 consecutive statistics of one factorized tensor ([R | C] index space), eight warps per
// statistic: warp w adds the w-th eighth of the statistic's partial sums in order, the eighths are added in warp order
// (binary64), the moving average is applied (R <- b2 R + (1 - b2) sum, reading of Sec. 4.3) and the CTA's share of
// sum(R) goes to fact_blockpart[chunk]. The CTA that finishes a tensor's last chunk (a counter, no waiting) then adds
// the shares in a fixed tree and stores the row factors R_i / sum(R). Every order is fixed, whichever CTA comes last.
constexpr int kFactChunk = 32;

__global__ void __launch_bounds__(256) factor_finalize_kernel(StepArgs a) {
    const int chunk_g = a.tile_begin + blockIdx.x;
    const int t = find_tensor(a.tile_start, a.n_tensors, chunk_g);
    const TensorDesc d = a.descs[t];
    const int chunk = chunk_g - __ldg(a.tile_start + t);
    const int n_chunks = __ldg(a.tile_start + t + 1) - __ldg(a.tile_start + t);
    const float* old = rc_pick(d, a.sel.old_i);
    float* cur = rc_pick(d, a.sel.new_i);
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t idx = (int64_t)chunk * kFactChunk + lane;
    const bool is_row = idx < d.rows, is_col = idx >= d.c_off && idx < d.c_off + d.cols;
    __shared__ double s_part[8][32];
    __shared__ double s_tree[256];
    __shared__ int s_last;
    // (binary64 additions are scarce on this part: an eighth is added in binary32 with a compensated sum, which is as
    // good as exact for a few hundred terms, and only the eighths and what follows are added in binary64)
    float part = 0.0f, comp = 0.0f;
    if (is_row) {
        const float* p = d.fact_rowpart + idx * d.fact_nstrips;
        const int n = d.fact_nstrips, lo = n * w / 8, hi = n * (w + 1) / 8;
        for (int k = lo; k < hi; ++k) kahan_add(part, comp, p[k]);
    } else if (is_col) {
        const float* p = d.fact_colpart + (idx - d.c_off);
        const int n = d.fact_tiles_y, lo = n * w / 8, hi = n * (w + 1) / 8;
        int k = lo;
        for (; k + 4 <= hi; k += 4) {                              // four loads in flight, added in order
            const float x0 = p[(int64_t)k * d.cols], x1 = p[(int64_t)(k + 1) * d.cols];
            const float x2 = p[(int64_t)(k + 2) * d.cols], x3 = p[(int64_t)(k + 3) * d.cols];
            kahan_add(part, comp, x0); kahan_add(part, comp, x1); kahan_add(part, comp, x2); kahan_add(part, comp, x3);
        }
        for (; k < hi; ++k) kahan_add(part, comp, p[(int64_t)k * d.cols]);
    }
    s_part[w][lane] = (double)part - (double)comp;
    __syncthreads();
    if (w == 0) {
        double sum = 0.0;
#pragma unroll
        for (int k = 0; k < 8; ++k) sum += s_part[k][lane];
        double r_share = 0.0;
        if (is_row || is_col) {
            const float v = __fadd_rn(__fmul_rn(a.h.beta2, old[idx]), __fmul_rn(a.h.omb2, (float)sum));
            cur[idx] = v;
            if (is_row) r_share = (double)v;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) r_share += __shfl_xor_sync(0xffffffffu, r_share, o);
        if (lane == 0) {
            d.fact_blockpart[chunk] = r_share;
            __threadfence();
            s_last = (atomicAdd(&a.tsync[t].maxima_done, 1u) == (uint32_t)(n_chunks - 1));
        }
    }
    __syncthreads();
    if (!s_last) return;
    // the tensor's last chunk: every statistic and every share is in place
    __threadfence();
    if (threadIdx.x == 0) a.tsync[t].maxima_done = 0u;
    const int row_chunks = (int)((d.rows + kFactChunk - 1) / kFactChunk);
    double mine = 0.0;
    for (int c = threadIdx.x; c < row_chunks; c += 256) mine += __ldcg(d.fact_blockpart + c);
    s_tree[threadIdx.x] = mine;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) s_tree[threadIdx.x] += s_tree[threadIdx.x + o];
        __syncthreads();
    }
    const float r_total = scale_rcp((float)s_tree[0]);
    for (int64_t i0 = 0; i0 < d.rows; i0 += 8 * 256) {           // eight loads in flight per thread, then eight stores
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int64_t i = i0 + u * 256 + threadIdx.x;
            v[u] = i < d.rows ? __ldcg(cur + i) : 0.0f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int64_t i = i0 + u * 256 + threadIdx.x;
            if (i < d.rows) d.rcp_new[i] = __fmul_rn(v[u], r_total);
        }
    }
}
#endif

template <bool BF16>
__device__ __forceinline__ void pass1_rank1_flat(const TensorDesc& d, const void* __restrict__ g, int tile, RcSel sel,
                                                 const Hyper& h) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float* rc_old = rc_pick(d, sel.old_i);
    float* rc_new = rc_pick(d, sel.new_i);
    for (int c = 0; c < d.flat_chunks; ++c) {
        const int64_t chunk = ((int64_t)tile * d.flat_chunks + c) * kWarps + warp;
        const int64_t e = chunk * kWarpElems + lane * kLaneElems;
        if (chunk * kWarpElems >= d.numel) break;
        if (e >= d.numel) continue;
        float gv[8];
        load8_grad_guard<BF16>(g, e, d.numel, gv);
        const uint32_t qv = load_codes_guard(d.v_codes, e, d.numel);
        int64_t i, j;
        split_index(d, e, i, j);
        float run = 0.0f;                      // maximum of the lane's current run of elements in row i
        float so = 0.0f;                       // leading axes' share of the old scale in row i
        bool fresh = true;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            if (e + k < d.numel) {
                if (fresh) { so = outer_stat<false>(d, rc_old, i); fresh = false; }
                const float s = fminf(so, __ldg(rc_old + d.c_off + j));
                const float vt = ema_v(__fmul_rn(lin_value((qv >> (4 * k)) & 15u), s), gv[k], h);
                run = fmaxf(run, vt);
                atomic_max_nonneg_filtered(rc_new + d.c_off + j, vt);
            }
            if (++j == d.cols) {               // the row ends inside the lane's elements: publish and start over
                outer_publish(d, rc_new, i, run);
                run = 0.0f;
                j = 0;
                ++i;
                fresh = true;
            }
        }
        if (i < d.rows) outer_publish(d, rc_new, i, run);
    }
}

// MINB: CTAs per SM the kernel is compiled for. The tiled maxima path keeps four rows of loads in registers and
// runs best at two (128 registers); the element-indexed and the sum-of-squares paths hold little state and want
// three. The host picks the instantiation by which kind holds most of a state's elements.
template <bool BF16, int MINB>
__global__ void __launch_bounds__(kThreads, MINB) pass1_kernel(StepArgs a) {
    __shared__ float s_col[kWarps * kWarpElems];
    const LaneTables lt = make_lane_tables();
    const Hyper2& h2 = a.h2;
    __shared__ int s_next[2];
    int buf = 0;
    for (int tile = a.tile_begin + tiles_first(a.tile_counter, s_next); tile < a.tile_end;) {
        const int fetched = tiles_fetch(a.tile_counter);
        const int t = find_tensor(a.tile_start, a.n_tensors, tile);
        const TensorDesc d = a.descs[t];
        const void* g = a.grads[t];
        const int local = tile - __ldg(a.tile_start + t);
        if (d.kind == K_RANK1_FAST || d.p1_tiled) pass1_rank1_fast<BF16>(d, g, local, a.sel, h2, lt, s_col);
        else if (d.kind == K_FACT) pass1_fact<BF16>(d, g, local, s_col);
        else pass1_rank1_flat<BF16>(d, g, local, a.sel, a.h);
        tile = a.tile_begin + tiles_next(s_next, buf, fetched);
    }
    tiles_done(a.tile_counter);
}

// ---- the fused schedule: both passes of every tensor in one launch --------------------------------------
//
// The launch walks an explicit work list (built on the host) whose items are tiles of the maxima pass and tiles of
// the update pass. The update tiles of a rank-1 tensor come after all of its maxima tiles in the list, close
// enough that the gradient and the second-moment codes read by the maxima pass are still in L2 when the update
// pass reads them again (the loads carry eviction priorities, see L2Policies), and the list interleaves the next
// tensor's maxima tiles with the current tensor's update tiles.
//
// Dependencies are counted per tensor in the arena (TensorSync). Items are handed out in list order, so whatever an
// update tile waits for was handed out earlier to a CTA that is already running and never waits itself: the oldest
// unfinished item always makes progress, whether or not all CTAs of the grid are resident. Every wait is bounded:
// when it runs out the CTA records kStatusWaitTimeout in the device status word and stops taking work.

constexpr uint32_t kStatusWaitTimeout = 2u;

// Polls until the counter has reached `target` (compared modulo 2^32: the counters are never reset, a tensor's
// target grows by its tile count with every launch). False when the limit ran out or another CTA has already reported
// an error. A wait that did not succeed at the first look adds its duration to the statistics words.
__device__ __forceinline__ bool wait_count(const uint32_t* counter, uint32_t target, uint32_t limit, const uint32_t* dev_status,
                                           unsigned long long* stats) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if ((int32_t)(v - target) >= 0) return true;
    unsigned long long t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    bool ok = false;
    for (uint32_t it = 0; it < limit; ++it) {
        __nanosleep(it < 64u ? 50u : 500u);
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
        if ((int32_t)(v - target) >= 0) { ok = true; break; }
        if ((it & 63u) == 63u && *reinterpret_cast<const volatile uint32_t*>(dev_status) != 0u) break;
    }
    if (stats) {
        unsigned long long t1;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        atomicAdd(stats, 1ull);
        atomicAdd(stats + 1, t1 - t0);
    }
    return ok;
}

template <bool BF16, bool EXACT, bool A32>
__global__ void __launch_bounds__(kThreads, 2) step_fused_kernel(StepArgs a) {
    __shared__ __align__(16) unsigned char s_lut[kLutSmemBytes];
    __shared__ float s_col[kWarps * kWarpElems];
    __shared__ float s_red[2 * kWarps];
    __shared__ float s_rows[2 * kFusedTileRows];
    __shared__ int s_next[2];
    __shared__ int s_flag;
    load_lut_smem(s_lut);
    __syncthreads();
    const LaneTables lt = make_lane_tables();
    const Hyper2& h2 = a.h2;
    uint32_t red_step = 0;
    int buf = 0;
    int ready_tensor = -1;     // the last tensor this CTA has seen complete its maxima pass (uniform over the CTA)
    for (int tile = a.tile_begin + tiles_first(a.tile_counter, s_next); tile < a.tile_end;) {
        const int fetched = tiles_fetch(a.tile_counter);
        const uint2 item = __ldg(a.work + tile);
        const int t = (int)(item.x & kWorkTensorMask);
        const bool update = (item.x & kWorkUpdate) != 0, keep = (item.x & kWorkKeep) != 0;
        const int local = (int)item.y;
        if (t >= a.n_tensors) {            // (never: the host built the list; the checking build says so before stopping)
#ifdef LPMM_DEBUG
            atomicCAS(a.dev_status, 0u, kStatusCheckBase + 6u);
#endif
            break;
        }
        const TensorDesc d = a.descs[t];
        const void* g = a.grads[t];
        TensorSync* sy = a.tsync + t;
        const bool rank1 = d.kind == K_RANK1_FAST || d.kind == K_RANK1_FLAT;
        if (!update) {
            {   // this tile's share of clearing the buffer that will receive the NEXT step's maxima (nothing reads or
                // writes it during this step)
                float4* z = reinterpret_cast<float4*>(rc_pick(d, a.sel.zero_i));
                const int n4 = d.rc_floats >> 2;
                const int z0 = (int)((int64_t)n4 * local / d.tiles1), z1 = (int)((int64_t)n4 * (local + 1) / d.tiles1);
                for (int i = z0 + (int)threadIdx.x; i < z1; i += kThreads) z[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            }
            if (d.kind == K_RANK1_FAST || d.p1_tiled) {
                const L2Policies pol = make_l2_policies();
                pass1_rank1_fast<BF16, true>(d, g, local, a.sel, h2, lt, s_col, (keep && a.l2_hints) ? pol.last : pol.normal, keep && a.l2_hints);
            } else {
                pass1_rank1_flat<BF16>(d, g, local, a.sel, a.h);
            }
            if (d.kind == K_RANK1_FAST) {
                // Count the tile. The barrier orders every thread's atomic maxima before thread 0's fence, which is
                // cumulative; nobody waits for the counter's old value.
                __syncthreads();
                if (threadIdx.x == 0) {
                    __threadfence();
                    atomicAdd(&sy->maxima_done, 1u);
                }
            } else {
                // Element-indexed tensors (odd shapes, three or four axes): their update path reads the reciprocals of
                // the new statistics from memory, so the CTA that finishes the tensor's last maxima tile inverts them
                // and only then announces the tensor (`ready` takes the launch number).
                __syncthreads();
                if (threadIdx.x == 0) {
                    __threadfence();
                    s_flag = (atomicAdd(&sy->maxima_done, 1u) + 1u == a.epoch * (uint32_t)d.tiles1);
                }
                __syncthreads();
                if (s_flag) {
                    __threadfence();
                    const float4* src = reinterpret_cast<const float4*>(rc_pick(d, a.sel.new_i));
                    float4* dst = reinterpret_cast<float4*>(d.rcp_new);
                    for (int i = threadIdx.x; i < (d.rc_floats >> 2); i += kThreads) {
                        const float4 v = __ldcg(src + i);
                        dst[i] = make_float4(scale_rcp(v.x), scale_rcp(v.y), scale_rcp(v.z), scale_rcp(v.w));
                    }
                    __threadfence();
                    __syncthreads();
                    if (threadIdx.x == 0) asm volatile("st.release.gpu.global.u32 [%0], %1;" :: "l"(&sy->ready), "r"(a.epoch) : "memory");
                }
            }
        } else {
            if (rank1 && t != ready_tensor) {
                if (threadIdx.x == 0) {
                    const bool ok = d.kind == K_RANK1_FAST
                        ? wait_count(&sy->maxima_done, a.epoch * (uint32_t)d.tiles1, a.spin_limit, a.dev_status, a.wait_stats)
                        : wait_count(&sy->ready, a.epoch, a.spin_limit, a.dev_status, a.wait_stats);
                    if (!ok) atomicCAS(a.dev_status, 0u, kStatusWaitTimeout);
                    s_flag = ok;
                }
                __syncthreads();
                if (!s_flag) break;                // uniform over the CTA; the states of this step are incomplete
                ready_tensor = t;
            }
            float* w = a.params[t];
            switch (d.kind) {
                case K_RANK1_FAST:
                    pass2_rank1_fast<BF16, EXACT, 7, 0, false, A32, true>(d, w, nullptr, g, local, a.sel, a.h, h2, lt, s_lut, s_red, red_step, s_rows);
                    break;
                case K_RANK1_FLAT: pass2_flat<BF16, true, EXACT, 7, false, A32, true>(d, w, nullptr, g, local, a.sel, a.h, h2, lt, s_lut, s_red, red_step); break;
                case K_BLOCK:      pass2_flat<BF16, false, EXACT, 7, false, A32>(d, w, nullptr, g, local, a.sel, a.h, h2, lt, s_lut, s_red, red_step); break;
                case K_FP32:       pass2_fp32<BF16, EXACT, false, A32>(d, w, nullptr, g, local, a.h); break;
                default: break;                    // (tiled block-wise tensors have a launch of their own)
            }
        }
        tile = a.tile_begin + tiles_next(s_next, buf, fetched);
    }
    tiles_done(a.tile_counter);
}

#if LPMM_STEP_PART == 0
// Two CTAs wait for a count that nothing will ever reach (test hook for the bounded wait): each gives up after
// `limit` polls, records the timeout in the status word and returns.
__global__ void wait_selftest_kernel(const uint32_t* flag, uint32_t want, uint32_t limit, uint32_t* dev_status, int32_t* gave_up) {
    if (threadIdx.x == 0) {
        if (!wait_count(flag, want, limit, dev_status, nullptr)) {
            atomicCAS(dev_status, 0u, kStatusWaitTimeout);
            atomicAdd(gave_up, 1);
        }
    }
}
#endif

// ---- compressed SGDM (Alg. 2): m = beta m + g ; w = w - lr m ; compress m. One pass, element-indexed -------

// One full chunk of a B128 tensor: the lane's eight elements, already loaded.
template <bool A32>
__device__ __forceinline__ void sgdm_chunk(float* w, uint8_t* mq, float* ms, float (&wv)[8], const float (&gv)[8], uint32_t qm,
                                           float prod, const Hyper2& h2, const LaneTables& lt, const unsigned char* s_lut) {
    float mt[8];
#pragma unroll
    for (int k = 0; k < 8; k += 2) {
        const float2 mo = make_float2(__shfl_sync(lt.mask, prod, (int)(qm >> (4 * k)), 16),
                                      __shfl_sync(lt.mask, prod, (int)(qm >> (4 * k + 4)), 16));
        const float2 m2 = fma2_rn(mul2_rn(h2.beta1, mo), h2.one, make_float2(gv[k], gv[k + 1]));
        const float2 w2 = fma2_rn(mul2_rn(h2.neg_step, m2), h2.one, make_float2(wv[k], wv[k + 1]));
        mt[k] = m2.x; mt[k + 1] = m2.y;
        wv[k] = w2.x; wv[k + 1] = w2.y;
    }
    store8_f32_a<A32>(w, wv);
    const float am_new = group_max(absmax8(mt), lt.mask);
    if ((threadIdx.x & 15) == 0) *ms = am_new;
    *reinterpret_cast<uint32_t*>(mq) = quantize8_de(mt, scale_rcp(am_new), s_lut);
}

template <bool BF16, bool A32>
__global__ void __launch_bounds__(kThreads, 3) sgdm_kernel(StepArgs a) {
    __shared__ __align__(16) unsigned char s_lut[kLutSmemBytes];
    __shared__ float s_red[2 * kWarps];
    load_lut_smem(s_lut);
    __syncthreads();
    const LaneTables lt = make_lane_tables();
    const Hyper2& h2 = a.h2;          // beta1 = momentum, neg_step = -lr, one = 1
    uint32_t red_step = 0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __shared__ int s_next[2];
    int buf = 0;
    for (int tile = a.tile_begin + tiles_first(a.tile_counter, s_next); tile < a.tile_end;) {
        const int fetched = tiles_fetch(a.tile_counter);
        const int t = find_tensor(a.tile_start, a.n_tensors, tile);
        const TensorDesc d = a.descs[t];
        float* w = a.params[t];
        const void* g = a.grads[t];
        const int local = tile - __ldg(a.tile_start + t);
        const int64_t m_mask = ((int64_t)1 << d.m_shift) - 1;
        int c_first = 0;
        // A tile that lies wholly inside a B128 tensor takes its chunks two at a time: both chunks' loads are in flight
        // before either is processed, and nothing needs a guard.
        if (d.kind != K_FP32 && d.m_shift == 7 && ((int64_t)(local + 1) * d.flat_chunks) * kWarps * kWarpElems <= d.numel) {
            for (; c_first + 1 < d.flat_chunks; c_first += 2) {
                const int64_t e0 = (((int64_t)local * d.flat_chunks + c_first) * kWarps + warp) * kWarpElems + lane * kLaneElems;
                const int64_t e1 = e0 + (int64_t)kWarps * kWarpElems;
                float w0[8], w1[8], g0[8], g1[8];
                load8_rw_a<A32>(w + e0, w0);
                load8_rw_a<A32>(w + e1, w1);
                load8_grad_a<BF16, A32>(g, e0, g0);
                load8_grad_a<BF16, A32>(g, e1, g1);
                const uint32_t q0 = *reinterpret_cast<const uint32_t*>(d.m_codes + (e0 >> 1));
                const uint32_t q1 = *reinterpret_cast<const uint32_t*>(d.m_codes + (e1 >> 1));
                const float p0 = __fmul_rn(lt.de, d.m_scale[e0 >> 7]), p1 = __fmul_rn(lt.de, d.m_scale[e1 >> 7]);
                sgdm_chunk<A32>(w + e0, d.m_codes + (e0 >> 1), d.m_scale + (e0 >> 7), w0, g0, q0, p0, h2, lt, s_lut);
                sgdm_chunk<A32>(w + e1, d.m_codes + (e1 >> 1), d.m_scale + (e1 >> 7), w1, g1, q1, p1, h2, lt, s_lut);
            }
        }
        for (int c = c_first; c < d.flat_chunks; ++c) {
            const int64_t chunk0 = ((int64_t)local * d.flat_chunks + c) * kWarps;
            const int64_t chunk = chunk0 + warp;
            const int64_t e = chunk * kWarpElems + lane * kLaneElems;
            if (chunk0 * kWarpElems >= d.numel) break;                               // uniform over the CTA
            const bool quant = d.kind != K_FP32;
            if (!(quant && d.m_shift == 11) && chunk * kWarpElems >= d.numel) break;  // B2048 warps stay for the barrier
            const bool full = (chunk + 1) * kWarpElems <= d.numel;
            float wv[8], gv[8], mo[8];
            uint32_t qm = 0;
            if (full) { load8_rw(w + e, wv); load8_grad<BF16>(g, e, gv); }
            else { load8_guard(w, e, d.numel, wv); load8_grad_guard<BF16>(g, e, d.numel, gv); }
            if (quant) {
                qm = full ? __ldg(reinterpret_cast<const uint32_t*>(d.m_codes + (e >> 1))) : load_codes_guard(d.m_codes, e, d.numel);
                const bool group_live = (e & ~m_mask) < d.numel;
                const float prod = __fmul_rn(lt.de, group_live ? d.m_scale[e >> d.m_shift] : 0.0f);
#pragma unroll
                for (int k = 0; k < 8; ++k) mo[k] = __shfl_sync(lt.mask, prod, (int)(qm >> (4 * k)), 16);
            } else {
                if (full) load8_rw(d.m32 + e, mo); else load8_guard(d.m32, e, d.numel, mo);
            }
            float mt[8];
#pragma unroll
            for (int k = 0; k < 8; k += 2) {
                // fl(fl(beta m) + g) and fl(w + fl(-lr m_t)), each sum written as fma(p, 1, q) (see ema_m2)
                const float2 m2 = fma2_rn(mul2_rn(h2.beta1, make_float2(mo[k], mo[k + 1])), h2.one, make_float2(gv[k], gv[k + 1]));
                const float2 w2 = fma2_rn(mul2_rn(h2.neg_step, m2), h2.one, make_float2(wv[k], wv[k + 1]));
                mt[k] = m2.x; mt[k + 1] = m2.y;
                wv[k] = w2.x; wv[k + 1] = w2.y;
            }
            if (!full) {
#pragma unroll
                for (int k = 0; k < 8; ++k) if (e + k >= d.numel) mt[k] = 0.0f;
            }
            if (full) store8_f32(w + e, wv); else store8_guard(w, e, d.numel, wv);
            if (quant) {
                const float am_new = block_max(absmax8(mt), d.m_shift, lt, s_red, red_step);
                if (e < d.numel && (threadIdx.x & (d.m_shift == 7 ? 15 : 2047)) == 0) d.m_scale[e >> d.m_shift] = am_new;
                const uint32_t q_new = quantize8_de(mt, scale_rcp(am_new), s_lut);
                if (full) *reinterpret_cast<uint32_t*>(d.m_codes + (e >> 1)) = q_new;
                else store_codes_guard(d.m_codes, e, d.numel, q_new);
            } else {
                if (full) store8_f32(d.m32 + e, mt); else store8_guard(d.m32, e, d.numel, mt);
            }
        }
        tile = a.tile_begin + tiles_next(s_next, buf, fetched);
    }
    tiles_done(a.tile_counter);
}

#if LPMM_STEP_PART == 0
__global__ void rcp_kernel(const float* __restrict__ src, float* __restrict__ dst, int64_t n) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = scale_rcp(src[i]);
}
#endif

}  // namespace

#if LPMM_STEP_PART == 0
cudaError_t launch_pass1(const StepArgs& a, bool bf16, int ctas_per_sm, int grid, cudaStream_t s) {
    if (a.tile_end <= a.tile_begin) return cudaSuccess;
    if (ctas_per_sm == 2) {
        if (bf16) pass1_kernel<true, 2><<<grid, kThreads, 0, s>>>(a);
        else pass1_kernel<false, 2><<<grid, kThreads, 0, s>>>(a);
    } else {
        if (bf16) pass1_kernel<true, 3><<<grid, kThreads, 0, s>>>(a);
        else pass1_kernel<false, 3><<<grid, kThreads, 0, s>>>(a);
    }
    return cudaGetLastError();
}

#endif

template <bool BF16, bool EXACT, int MSHIFT>
cudaError_t launch_pass2_t(const StepArgs& a, int v_kind, int grid, cudaStream_t s) {
    if (v_kind == 3) {   // the tensors that are not on the tiled path
        if (a.params_bf16 != nullptr) {
            if (a.aligned32) pass2_kernel<BF16, EXACT, MSHIFT, 0, true, true, true><<<grid, kThreads, 0, s>>>(a);
            else pass2_kernel<BF16, EXACT, MSHIFT, 0, true, false, true><<<grid, kThreads, 0, s>>>(a);
        } else {
            if (a.aligned32) pass2_kernel<BF16, EXACT, MSHIFT, 0, false, true, true><<<grid, kThreads, 0, s>>>(a);
            else pass2_kernel<BF16, EXACT, MSHIFT, 0, false, false, true><<<grid, kThreads, 0, s>>>(a);
        }
    } else if (v_kind == 1) {
        pass2_kernel<BF16, EXACT, MSHIFT, 1, false, false><<<grid, kThreads, 0, s>>>(a);
    } else if (v_kind == 2) {
        if (a.params_bf16 != nullptr) {
            if (a.aligned32) pass2_kernel<BF16, EXACT, MSHIFT, 2, true, true><<<grid, kThreads, 0, s>>>(a);
            else pass2_kernel<BF16, EXACT, MSHIFT, 2, true, false><<<grid, kThreads, 0, s>>>(a);
        } else {
            if (a.aligned32) pass2_kernel<BF16, EXACT, MSHIFT, 2, false, true><<<grid, kThreads, 0, s>>>(a);
            else pass2_kernel<BF16, EXACT, MSHIFT, 2, false, false><<<grid, kThreads, 0, s>>>(a);
        }
    } else if (a.params_bf16 != nullptr) {
        if (a.aligned32) pass2_kernel<BF16, EXACT, MSHIFT, 0, true, true><<<grid, kThreads, 0, s>>>(a);
        else pass2_kernel<BF16, EXACT, MSHIFT, 0, true, false><<<grid, kThreads, 0, s>>>(a);
    } else if (a.aligned32) {
        pass2_kernel<BF16, EXACT, MSHIFT, 0, false, true><<<grid, kThreads, 0, s>>>(a);
    } else {
        pass2_kernel<BF16, EXACT, MSHIFT, 0, false, false><<<grid, kThreads, 0, s>>>(a);
    }
    return cudaGetLastError();
}

template <bool BF16, bool EXACT>
cudaError_t launch_pass2_m(const StepArgs& a, int m_shift, int v_kind, int grid, cudaStream_t s) {
    return m_shift == 11 ? launch_pass2_t<BF16, EXACT, 11>(a, v_kind, grid, s) : launch_pass2_t<BF16, EXACT, 7>(a, v_kind, grid, s);
}

template <bool BF16, bool EXACT>
cudaError_t launch_fused_t(const StepArgs& a, int grid, cudaStream_t s) {
    if (a.aligned32) step_fused_kernel<BF16, EXACT, true><<<grid, kThreads, 0, s>>>(a);
    else step_fused_kernel<BF16, EXACT, false><<<grid, kThreads, 0, s>>>(a);
    return cudaGetLastError();
}

// One launcher per (gradient type, update math) pair, each in its own part of the build.
#if defined(LPMM_STEP_ALL) || LPMM_STEP_PART == 0
cudaError_t launch_pass2_bf16_fast(const StepArgs& a, int m_shift, int v_kind, int grid, cudaStream_t s) { return launch_pass2_m<true, false>(a, m_shift, v_kind, grid, s); }
cudaError_t launch_fused_bf16_fast(const StepArgs& a, int grid, cudaStream_t s) { return launch_fused_t<true, false>(a, grid, s); }
#endif
#if defined(LPMM_STEP_ALL) || LPMM_STEP_PART == 1
cudaError_t launch_pass2_bf16_ieee(const StepArgs& a, int m_shift, int v_kind, int grid, cudaStream_t s) { return launch_pass2_m<true, true>(a, m_shift, v_kind, grid, s); }
cudaError_t launch_fused_bf16_ieee(const StepArgs& a, int grid, cudaStream_t s) { return launch_fused_t<true, true>(a, grid, s); }
#endif
#if defined(LPMM_STEP_ALL) || LPMM_STEP_PART == 2
cudaError_t launch_pass2_f32_fast(const StepArgs& a, int m_shift, int v_kind, int grid, cudaStream_t s) { return launch_pass2_m<false, false>(a, m_shift, v_kind, grid, s); }
cudaError_t launch_fused_f32_fast(const StepArgs& a, int grid, cudaStream_t s) { return launch_fused_t<false, false>(a, grid, s); }
#endif
#if defined(LPMM_STEP_ALL) || LPMM_STEP_PART == 3
cudaError_t launch_pass2_f32_ieee(const StepArgs& a, int m_shift, int v_kind, int grid, cudaStream_t s) { return launch_pass2_m<false, true>(a, m_shift, v_kind, grid, s); }
cudaError_t launch_fused_f32_ieee(const StepArgs& a, int grid, cudaStream_t s) { return launch_fused_t<false, true>(a, grid, s); }
#endif

#if LPMM_STEP_PART == 0
// v_kind: 0 rank-1 second moments, 1 factorized, 2 block-wise (which tiled path the state's matrices take);
// 3: the kernel of the tensors that are not on the tiled path.
cudaError_t launch_pass2(const StepArgs& a, bool bf16, bool exact, int m_shift, int v_kind, int grid, cudaStream_t s) {
    if (a.tile_end <= a.tile_begin) return cudaSuccess;
    if (bf16) return exact ? launch_pass2_bf16_ieee(a, m_shift, v_kind, grid, s) : launch_pass2_bf16_fast(a, m_shift, v_kind, grid, s);
    return exact ? launch_pass2_f32_ieee(a, m_shift, v_kind, grid, s) : launch_pass2_f32_fast(a, m_shift, v_kind, grid, s);
}

// The fused schedule (rank-1 states with B128 first moments): one launch over the work list [tile_begin, tile_end).
cudaError_t launch_fused(const StepArgs& a, bool bf16, bool exact, int grid, cudaStream_t s) {
    if (a.tile_end <= a.tile_begin) return cudaSuccess;
    if (bf16) return exact ? launch_fused_bf16_ieee(a, grid, s) : launch_fused_bf16_fast(a, grid, s);
    return exact ? launch_fused_f32_ieee(a, grid, s) : launch_fused_f32_fast(a, grid, s);
}

// ---- composite tensors (three or four axes on the tiled path): expanded statistics -------------------------
//
// One thread per entry of a composite tensor's expanded vector [rows padded to 4 | cols]; one CTA per 256 entries.
// The side's axes are walked from the last (fastest) to the first; `digit` is the entry's index along the axis.
template <typename F>
__device__ __forceinline__ void nd_for_axes(const TensorDesc& d, int a0, int a1, uint32_t idx, F f) {
    uint32_t rem = idx;
#pragma unroll
    for (int a = 3; a >= 0; --a) {
        if (a >= a0 && a < a1) {
            const uint32_t q = rem / (uint32_t)d.nd_dim[a];
            f(d.nd_off[a] + (int)(rem - q * (uint32_t)d.nd_dim[a]));
            rem = q;
        }
    }
}
__global__ void __launch_bounds__(256) nd_stats_kernel(StepArgs a, int mode) {
    const int chunk_g = a.tile_begin + blockIdx.x;
    const int t = find_tensor(a.tile_start, a.n_tensors, chunk_g);
    const TensorDesc d = a.descs[t];
    const int e = (chunk_g - __ldg(a.tile_start + t)) * 256 + (int)threadIdx.x;
    if (e >= d.exp_len) return;
    const bool is_row = e < d.rows, is_col = e >= d.c_off && e < d.c_off + d.cols;
    const int a0 = is_row ? 0 : d.nd_split, a1 = is_row ? d.nd_split : d.nd;
    const uint32_t idx = (uint32_t)(is_row ? e : e - d.c_off);
    if (mode == 0) {
        float s = 0.0f;
        if (is_row || is_col) {
            const float* old = rc_pick(d, a.sel.old_i);
            s = 3.402823466e38f;
            nd_for_axes(d, a0, a1, idx, [&](int off) { s = fminf(s, old[off]); });
        }
        d.exp_old[e] = s;
        d.exp_new[e] = 0.0f;
    } else if (mode == 1) {
        if (is_row || is_col) {
            const float v = d.exp_new[e];
            float* cur = rc_pick(d, a.sel.new_i);
            nd_for_axes(d, a0, a1, idx, [&](int off) { atomic_max_nonneg_filtered(cur + off, v); });
        }
    } else {
        float r = 0.0f;
        if (is_row || is_col) {
            const float* cur = rc_pick(d, a.sel.new_i);
            nd_for_axes(d, a0, a1, idx, [&](int off) { r = fmaxf(r, scale_rcp(cur[off])); });
        }
        d.rcp_new[e] = r;
    }
}
cudaError_t launch_nd_stats(const StepArgs& a, int mode, cudaStream_t s) {
    if (a.tile_end <= a.tile_begin) return cudaSuccess;
    nd_stats_kernel<<<a.tile_end - a.tile_begin, 256, 0, s>>>(a, mode);
    return cudaGetLastError();
}

// Checking build: counts the bytes of one guard zone that no longer hold the pattern.
__global__ void guard_check_kernel(const unsigned char* zone, int bytes, unsigned char want, uint32_t* damaged) {
    for (int i = threadIdx.x; i < bytes; i += blockDim.x)
        if (zone[i] != want) atomicAdd(damaged, 1u);
}
cudaError_t launch_guard_check(const unsigned char* zone, int bytes, unsigned char want, uint32_t* damaged, cudaStream_t s) {
    guard_check_kernel<<<1, 256, 0, s>>>(zone, bytes, want, damaged);
    return cudaGetLastError();
}
// A check that fails on purpose (host-requested): shows that a failed index check reaches the status word.
__global__ void check_selftest_kernel(uint32_t* dev_status) {
#ifdef LPMM_DEBUG
    TensorDesc d = {};
    d.dbg_status = dev_status;
    d.numel = 0;
    if (!LPMM_DBG_OK(d, d.numel > 0, 0x7f)) return;
#else
    (void)dev_status;      // (the normal build never launches this kernel)
#endif
}
cudaError_t launch_check_selftest(uint32_t* dev_status, cudaStream_t s) {
    check_selftest_kernel<<<1, 1, 0, s>>>(dev_status);
    return cudaGetLastError();
}

cudaError_t launch_wait_selftest(const uint32_t* flag, uint32_t want, uint32_t limit, uint32_t* dev_status, int32_t* gave_up,
                                 cudaStream_t s) {
    wait_selftest_kernel<<<2, 32, 0, s>>>(flag, want, limit, dev_status, gave_up);
    return cudaGetLastError();
}

// a.tile_start / tile_begin / tile_end: the table of 32-statistic chunks of the factorized tensors.
cudaError_t launch_factor_finalize(const StepArgs& a, cudaStream_t s) {
    if (a.tile_end <= a.tile_begin) return cudaSuccess;
    factor_finalize_kernel<<<a.tile_end - a.tile_begin, 256, 0, s>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_sgdm(const StepArgs& a, bool bf16, int grid, cudaStream_t s) {
    if (a.tile_end <= a.tile_begin) return cudaSuccess;
    if (a.aligned32) {
        if (bf16) sgdm_kernel<true, true><<<grid, kThreads, 0, s>>>(a);
        else sgdm_kernel<false, true><<<grid, kThreads, 0, s>>>(a);
    } else {
        if (bf16) sgdm_kernel<true, false><<<grid, kThreads, 0, s>>>(a);
        else sgdm_kernel<false, false><<<grid, kThreads, 0, s>>>(a);
    }
    return cudaGetLastError();
}

cudaError_t launch_rcp(const float* src, float* dst, int64_t n, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    int grid = (int)((n + 255) / 256);
    if (grid > 2048) grid = 2048;
    rcp_kernel<<<grid, 256, 0, s>>>(src, dst, n);
    return cudaGetLastError();
}

cudaError_t step_kernel_occupancy(int pass1_ctas_per_sm, int* p1, int* p2) {
    cudaError_t e = pass1_ctas_per_sm == 2 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(p1, pass1_kernel<true, 2>, kThreads, 0)
                                           : cudaOccupancyMaxActiveBlocksPerMultiprocessor(p1, pass1_kernel<true, 3>, kThreads, 0);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(p2, pass2_kernel<true, false, 7, 0, false, true>, kThreads, 0);
}

#endif  // LPMM_STEP_PART == 0

}  // namespace lpmm
