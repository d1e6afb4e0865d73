// Stand-alone quantizer / dequantizer kernels (Sec. 2.2: Q = M o N, x~ = N^-1 o T(q)) for sm_100a.
// They serve inspection, checkpoint tooling and the parity tests; the fused step does not call them.
#include <mutex>

#include "../../include/lpmm.h"
#include "lpmm_internal.h"

namespace lpmm {

namespace {

constexpr int kQThreads = 256;

// Block-wise scales: one warp per block of B elements (B = 128 or 2048), any numel.
__global__ void block_scale_kernel(const float* __restrict__ x, int64_t numel, int64_t B, int64_t nblocks,
                                   float* __restrict__ scale) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t b = warp0; b < nblocks; b += nwarps) {
        const int64_t lo = b * B, hi = min(lo + B, numel);
        float mx = 0.0f;
        for (int64_t i = lo + lane; i < hi; i += 32) mx = fmaxf(mx, fabsf(__ldg(x + i)));
        mx = warp_max(mx);
        if (lane == 0) scale[b] = mx;
    }
}

// Rank-1 statistics (Sec. 4.2): each CTA owns a strip of 32 rows x 256 columns; a thread walks one
// column down the strip, so row maxima reduce inside a warp and column maxima stay in a register.
__global__ void rank1_scale_kernel(const float* __restrict__ x, int64_t rows, int64_t cols,
                                   float* __restrict__ r, float* __restrict__ c) {
    const int64_t col_tiles = (cols + kQThreads - 1) / kQThreads;
    const int64_t row_tiles = (rows + 31) / 32;
    const int lane = threadIdx.x & 31;
    for (int64_t tile = blockIdx.x; tile < col_tiles * row_tiles; tile += gridDim.x) {
        const int64_t j = (tile % col_tiles) * kQThreads + threadIdx.x;
        const int64_t i0 = (tile / col_tiles) * 32;
        float cm = 0.0f;
        for (int64_t i = i0; i < min(i0 + 32, rows); ++i) {
            const float a = (j < cols) ? fabsf(__ldg(x + i * cols + j)) : 0.0f;
            cm = fmaxf(cm, a);
            const float rm = warp_max(a);
            if (lane == 0) atomic_max_nonneg(r + i, rm);
        }
        if (j < cols) atomic_max_nonneg(c + j, cm);
    }
}

// One thread per byte of codes (two elements), any numel.
template <bool DE, bool RANK1>
__global__ void map_kernel(const float* __restrict__ x, int64_t rows, int64_t cols, int64_t B,
                           const float* __restrict__ s0, const float* __restrict__ s1, uint8_t* __restrict__ codes) {
    const int64_t numel = rows * cols;
    const int64_t nbytes = (numel + 1) >> 1;
    for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nbytes; b += (int64_t)gridDim.x * blockDim.x) {
        uint32_t byte = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int64_t e = 2 * b + h;
            if (e >= numel) continue;
            float xv = __ldg(x + e);
            float rcp;
            if (RANK1) {
                const int64_t i = e / cols, j = e - i * cols;
                rcp = fmaxf(scale_rcp(__ldg(s0 + i)), scale_rcp(__ldg(s1 + j)));
            } else {
                rcp = scale_rcp(__ldg(s0 + e / B));
            }
            if (RANK1) xv = fabsf(xv);   // Alg. 4 takes |x|; block-wise keeps the sign (negative -> lowest code)
            const float n = __fmul_rn(xv, rcp);
            const uint32_t q = DE ? de_nearest(n) : lin_nearest(n);
            byte |= q << (4 * h);
        }
        codes[b] = (uint8_t)byte;
    }
}

template <bool DE, bool RANK1>
__global__ void unmap_kernel(const uint8_t* __restrict__ codes, int64_t rows, int64_t cols, int64_t B,
                             const float* __restrict__ s0, const float* __restrict__ s1, float* __restrict__ out) {
    const int64_t numel = rows * cols;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < numel; e += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t q = (codes[e >> 1] >> (4 * (e & 1))) & 15u;
        float s;
        if (RANK1) {
            const int64_t i = e / cols, j = e - i * cols;
            s = fminf(__ldg(s0 + i), __ldg(s1 + j));
        } else {
            s = __ldg(s0 + e / B);
        }
        const float t = DE ? kDeTable[q] : lin_value(q);
        out[e] = __fmul_rn(t, s);
    }
}

int grid_for(int64_t work_items) {
    int64_t g = (work_items + kQThreads - 1) / kQThreads;
    if (g < 1) g = 1;
    if (g > 148 * 16) g = 148 * 16;
    return (int)g;
}

}  // namespace

cudaError_t launch_quantize(const float* x, int64_t rows, int64_t cols, int norm, int map, int block,
                            bool given, uint8_t* codes, float* s0, float* s1, cudaStream_t s) {
    const int64_t numel = rows * cols;
    const bool rank1 = (norm == 1), de = (map == 0);
    if (!given) {
        if (rank1) {
            cudaError_t e = cudaMemsetAsync(s0, 0, sizeof(float) * rows, s);
            if (e != cudaSuccess) return e;
            e = cudaMemsetAsync(s1, 0, sizeof(float) * cols, s);
            if (e != cudaSuccess) return e;
            const int64_t tiles = ((cols + kQThreads - 1) / kQThreads) * ((rows + 31) / 32);
            rank1_scale_kernel<<<(int)(tiles < 148 * 16 ? tiles : 148 * 16), kQThreads, 0, s>>>(x, rows, cols, s0, s1);
        } else {
            const int64_t nblocks = (numel + block - 1) / block;
            block_scale_kernel<<<grid_for(nblocks * 32), kQThreads, 0, s>>>(x, numel, block, nblocks, s0);
        }
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    const int grid = grid_for((numel + 1) / 2);
    if (rank1) map_kernel<false, true><<<grid, kQThreads, 0, s>>>(x, rows, cols, block, s0, s1, codes);
    else if (de) map_kernel<true, false><<<grid, kQThreads, 0, s>>>(x, rows, cols, block, s0, s1, codes);
    else map_kernel<false, false><<<grid, kQThreads, 0, s>>>(x, rows, cols, block, s0, s1, codes);
    return cudaGetLastError();
}

cudaError_t launch_dequantize(const uint8_t* codes, const float* s0, const float* s1, int64_t rows, int64_t cols,
                              int norm, int map, int block, float* out, cudaStream_t s) {
    const bool rank1 = (norm == 1), de = (map == 0);
    const int grid = grid_for(rows * cols);
    if (rank1) unmap_kernel<false, true><<<grid, kQThreads, 0, s>>>(codes, rows, cols, block, s0, s1, out);
    else if (de) unmap_kernel<true, false><<<grid, kQThreads, 0, s>>>(codes, rows, cols, block, s0, s1, out);
    else unmap_kernel<false, false><<<grid, kQThreads, 0, s>>>(codes, rows, cols, block, s0, s1, out);
    return cudaGetLastError();
}

// ---- rank-1 quantizer whose scratch lives inside the library image ---------------------------------
//
// The reciprocals of the row and column maxima are computed once into a scratch array and the mapping
// kernel reads them from there (instead of dividing twice per element). The scratch is a fixed
// file-scope device array, so this path needs no allocation from anybody.

constexpr int64_t kStaticScratchFloats = LPMM_NOALLOC_MAX_SCALES;
static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

namespace {

__global__ void rcp_to_scratch_kernel(const float* __restrict__ r, const float* __restrict__ c, int64_t rows,
                                      int64_t c_off, int64_t cols, float* __restrict__ scratch) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < rows + cols; i += (int64_t)gridDim.x * blockDim.x) {
        if (i < rows) scratch[i] = scale_rcp(r[i]);
        else scratch[c_off + (i - rows)] = scale_rcp(c[i - rows]);
    }
}

__global__ void map_rank1_scratch_kernel(const float* __restrict__ x, int64_t rows, int64_t cols, int64_t c_off,
                                         const float* __restrict__ scratch, uint8_t* __restrict__ codes) {
    const int64_t numel = rows * cols;
    const int64_t nbytes = (numel + 1) >> 1;
    for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b < nbytes; b += (int64_t)gridDim.x * blockDim.x) {
        uint32_t byte = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int64_t e = 2 * b + h;
            if (e >= numel) continue;
            const int64_t i = e / cols, j = e - i * cols;
            const float rcp = fmaxf(scratch[i], scratch[c_off + j]);
            byte |= lin_nearest(__fmul_rn(fabsf(__ldg(x + e)), rcp)) << (4 * h);
        }
        codes[b] = (uint8_t)byte;
    }
}

// Device address of g_static_scratch on the current device, looked up once per device. In host code the
// array's name is only a handle for the runtime; the kernels must be given this address.
cudaError_t static_scratch_address(float** out) {
    constexpr int kMaxDevices = 64;
    static float* cached[kMaxDevices] = {};
    static std::mutex mu;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!cached[dev]) {
        float* p = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch);
        if (e != cudaSuccess) return e;
        cached[dev] = p;
    }
    *out = cached[dev];
    return cudaSuccess;
}

}  // namespace

cudaError_t launch_quantize_rank1_noalloc(const float* x, int64_t rows, int64_t cols, uint8_t* codes, float* r,
                                          float* c, cudaStream_t s) {
    float* scratch = nullptr;
    cudaError_t e = static_scratch_address(&scratch);
    if (e != cudaSuccess) return e;
    const int64_t c_off = (rows + 3) / 4 * 4;
    // The outputs accumulate maxima and must start at zero; the scratch needs no clearing because the part
    // used by this call is overwritten below before anything reads it.
    e = cudaMemsetAsync(r, 0, sizeof(float) * rows, s);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(c, 0, sizeof(float) * cols, s);
    if (e != cudaSuccess) return e;
    const int64_t tiles = ((cols + kQThreads - 1) / kQThreads) * ((rows + 31) / 32);
    rank1_scale_kernel<<<(int)(tiles < 148 * 16 ? tiles : 148 * 16), kQThreads, 0, s>>>(x, rows, cols, r, c);
    rcp_to_scratch_kernel<<<grid_for(rows + cols), kQThreads, 0, s>>>(r, c, rows, c_off, cols, scratch);
    map_rank1_scratch_kernel<<<grid_for((rows * cols + 1) / 2), kQThreads, 0, s>>>(x, rows, cols, c_off, scratch, codes);
    return cudaGetLastError();
}

}  // namespace lpmm
