// Internal structures shared by the host API and the kernels of the fused step.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "lpmm_device.cuh"

namespace lpmm {

// Work kinds inside the step kernels. RANK1_FAST needs cols % 128 == 0 (a 128-block then lies inside
// one row and every row starts on a 16-byte boundary of every operand); other 2-D shapes take the
// element-indexed RANK1_FLAT path. BLOCK_TILED: a matrix with a block-wise second moment (LPMM_V_BLOCK) and
// cols % 128 == 0 on the tiled path; BLOCK: every other block-wise tensor, element-indexed.
enum : int32_t { K_FP32 = 0, K_BLOCK = 1, K_RANK1_FAST = 2, K_RANK1_FLAT = 3, K_FACT = 4, K_BLOCK_TILED = 5 };

constexpr int kThreads = 256;          // threads per CTA in the step kernels
constexpr int kWarps = kThreads / 32;
constexpr int kLaneElems = 8;          // consecutive elements per lane
constexpr int kWarpElems = 32 * kLaneElems;  // 256: two 128-element blocks per warp

// One entry of the device-side tensor table (lives at the head of the arena).
struct TensorDesc {
    uint8_t* m_codes;   // ceil(numel/2) bytes
    float* m_scale;     // ceil(numel / m_block) block maxima of |m|
    uint8_t* v_codes;
    float* v_bscale;    // K_BLOCK: ceil(numel/128) block maxima of v
    float* rc[3];       // K_RANK1_*: three buffers of [r (rows, padded to 4) | c (cols)] that rotate from step to step
                        // (current, new, being cleared for the step after); K_FACT: [R | C] statistics
    float* rcp_new;     // K_RANK1_*: reciprocals of the new r, c (same layout), per-step scratch; K_FACT: R_i / sum(R)
    float* m32;         // K_FP32
    float* v32;
    int64_t rows, cols, numel;
    int32_t kind;
    int32_t c_off;      // float offset of c inside rc[] and rcp_new
    int32_t wx;         // K_RANK1_FAST: warps across a tile (1, 2 or 4); tile is 256*wx columns wide
    int32_t tiles_x;    // K_RANK1_FAST: column tiles
    int32_t tile_rows;  // K_RANK1_FAST: rows per tile of the update pass
    int32_t flat_chunks;  // other kinds: 256-element chunks per warp per tile
    int32_t m_shift;    // log2 of the first-moment block size: 7 (B128) or 11 (B2048)
    // K_RANK1_FLAT, general form of Alg. 4: the tensor is [outer_dim[0] x .. x outer_dim[n_outer-1]] x cols,
    // rows = the product of the leading extents. The statistics of leading axis a start at float outer_off[a]
    // of rc[] / rcp_new (axis 0 at 0), those of the last axis at c_off. A matrix has n_outer = 1.
    int32_t n_outer;
    int32_t outer_dim[3];
    int32_t outer_off[3];
    int32_t tile_rows1; // K_RANK1_FAST: rows per tile of the maxima pass (at least tile_rows; same tile width)
    int32_t tiles1;     // rank-1 kinds: tiles of the maxima pass
    int32_t tiles2;     // tiles of the update pass
    int32_t rc_floats;  // rank-1 kinds: floats of this tensor's share of rc[] / rcp_new (c_off + cols rounded up to 4)
    // K_FACT: partial sums of g^2 written by the sums pass and added up in a fixed order by the finalize kernels
    float* fact_rowpart;    // rows x fact_nstrips: one partial per row and 256-column strip
    float* fact_colpart;    // fact_tiles_y x cols: one partial per column and tile row-block of the sums pass
    double* fact_blockpart; // ceil(rc_floats / 32): each finalize CTA's share of sum(R)
    int32_t fact_nstrips;
    int32_t fact_tiles_y;
    uint32_t* dbg_status;   // the arena's device status word (written by the checking build's index checks)
    // K_RANK1_FAST for a tensor with three or four axes ("composite", Alg. 4): the leading nd_split axes are flattened
    // into rows, the others into columns (rows, cols, c_off above describe that matrix). The persistent statistics stay one
    // vector per axis (axis a at float nd_off[a] of rc[]); every step they are expanded into per-row / per-column vectors
    // (minimum over the axes of a side) which the tiled kernels read and reduce into exactly like a matrix's r and c:
    //   exp_old [rows padded to 4 | cols]   current scales, exp_new: maxima of this step, rcp_new: their reciprocals.
    float* exp_old;         // nullptr: not a composite tensor
    float* exp_new;
    int32_t exp_len;        // floats of each expanded vector
    int32_t nd, nd_split;
    int32_t p1_tiled;       // K_RANK1_FLAT matrix with cols % 8 == 0: its maxima pass runs on the tiled kernel (ragged last
                            // column group clamped onto valid columns: maxima are idempotent)
    int32_t nd_dim[4];
    int32_t nd_off[4];
};

// Index checks of the checking build (-DLPMM_DEBUG): a failed check records its code in the device status word (the
// first failure wins) and evaluates to false, on which the tile functions return without touching memory. Nothing
// traps. In the normal build the macro is the constant true.
constexpr uint32_t kStatusCheckBase = 0x100u;   // status words >= this: a failed index check, low byte = which one
#ifdef LPMM_DEBUG
#define LPMM_DBG_OK(desc, cond, code) \
    ((cond) ? true : (atomicCAS((desc).dbg_status, 0u, kStatusCheckBase + (uint32_t)(code)), false))
#else
#define LPMM_DBG_OK(desc, cond, code) (true)
#endif

// Fused schedule: progress of one tensor. The counter is never reset: launch number e (1, 2, ...) of a state waits for
// e * tiles1, modulo 2^32.
struct TensorSync {
    uint32_t maxima_done;  // finished tiles of the maxima pass, summed over all launches
    uint32_t ready;        // element-indexed tensors: the last launch whose new reciprocals are in place
};

// Which of a tensor's three scale buffers is which in this step.
struct RcSel {
    int32_t old_i;    // current r, c (read)
    int32_t new_i;    // receives the new r', c' (all zero when the step starts)
    int32_t zero_i;   // fused schedule: cleared during this step, becomes new_i of the next one
};

// Fused schedule: one item of the work list = one tile. x = tensor index | flags, y = tile number inside the
// tensor's pass (the maxima pass and the update pass have tilings of their own).
constexpr uint32_t kWorkTensorMask = 0x0fffffffu;
constexpr uint32_t kWorkUpdate = 0x40000000u;   // a tile of the update pass (else: of the maxima pass)
constexpr uint32_t kWorkKeep = 0x80000000u;     // maxima pass: load this tile so that it stays in L2 for the update pass

struct StepArgs {
    const TensorDesc* descs;
    float* const* params;        // n device pointers, fp32
    uint16_t* const* params_bf16;  // n device pointers to bfloat16 copies of the parameters, or nullptr (no copy)
    const void* const* grads;    // n device pointers
    const int32_t* tile_start;   // n + 1 prefix sums of tiles (pass-specific)
    int32_t n_tensors;
    int32_t tile_begin, tile_end;  // this launch covers tiles [tile_begin, tile_end) of the prefix table
    RcSel sel;                   // roles of the three scale buffers in this step
    const uint2* work;           // fused schedule: the work list
    TensorSync* tsync;           // fused schedule: per-tensor progress counters
    uint32_t spin_limit;         // fused schedule: polls before a wait gives up
    uint32_t epoch;              // fused schedule: number of this launch on the state (1, 2, ...)
    int32_t l2_hints;            // fused schedule: 1 = accesses carry L2 eviction priorities
    unsigned long long* wait_stats;   // fused schedule: {waits that had to poll, their summed nanoseconds}, or nullptr
    int32_t aligned32;           // every parameter (and fp32 gradient) pointer is 32-byte aligned: 256-bit accesses
    uint32_t* dev_status;        // device error word in the arena header (0 = ok)
    int32_t* tile_counter;       // two words in the arena header: next tile of this launch, finished CTAs (both 0 between launches)
    Hyper h;
    Hyper2 h2;                   // the same constants as pairs (kernel-parameter space: usable as operands)
};

cudaError_t launch_pass1(const StepArgs& a, bool bf16, int ctas_per_sm, int grid, cudaStream_t s);
cudaError_t launch_pass2(const StepArgs& a, bool bf16, bool exact, int m_shift, int v_kind, int grid, cudaStream_t s);
cudaError_t launch_pass2_bf16_fast(const StepArgs& a, int m_shift, int v_kind, int grid, cudaStream_t s);
cudaError_t launch_pass2_bf16_ieee(const StepArgs& a, int m_shift, int v_kind, int grid, cudaStream_t s);
cudaError_t launch_pass2_f32_fast(const StepArgs& a, int m_shift, int v_kind, int grid, cudaStream_t s);
cudaError_t launch_pass2_f32_ieee(const StepArgs& a, int m_shift, int v_kind, int grid, cudaStream_t s);
cudaError_t launch_fused(const StepArgs& a, bool bf16, bool exact, int grid, cudaStream_t s);
cudaError_t launch_fused_bf16_fast(const StepArgs& a, int grid, cudaStream_t s);
cudaError_t launch_fused_bf16_ieee(const StepArgs& a, int grid, cudaStream_t s);
cudaError_t launch_fused_f32_fast(const StepArgs& a, int grid, cudaStream_t s);
cudaError_t launch_fused_f32_ieee(const StepArgs& a, int grid, cudaStream_t s);
cudaError_t launch_wait_selftest(const uint32_t* flag, uint32_t want, uint32_t limit, uint32_t* dev_status, int32_t* gave_up,
                                 cudaStream_t s);
cudaError_t launch_check_selftest(uint32_t* dev_status, cudaStream_t s);
// mode 0: expand the current per-axis statistics and clear exp_new; 1: fold exp_new into the new per-axis statistics
// (atomic maxima into the cleared buffer); 2: expanded reciprocals of the new statistics. a.tile_*: the chunk table.
cudaError_t launch_nd_stats(const StepArgs& a, int mode, cudaStream_t s);
cudaError_t launch_guard_check(const unsigned char* zone, int bytes, unsigned char want, uint32_t* damaged, cudaStream_t s);
cudaError_t launch_factor_finalize(const StepArgs& a, cudaStream_t s);
cudaError_t launch_sgdm(const StepArgs& a, bool bf16, int grid, cudaStream_t s);
cudaError_t launch_rcp(const float* src, float* dst, int64_t n, cudaStream_t s);
cudaError_t step_kernel_occupancy(int pass1_ctas_per_sm, int* pass1_blocks_per_sm, int* pass2_blocks_per_sm);

cudaError_t launch_quantize(const float* x, int64_t rows, int64_t cols, int norm, int map, int block,
                            bool given, uint8_t* codes, float* s0, float* s1, cudaStream_t s);
cudaError_t launch_dequantize(const uint8_t* codes, const float* s0, const float* s1, int64_t rows, int64_t cols,
                              int norm, int map, int block, float* out, cudaStream_t s);

cudaError_t launch_quantize_rank1_noalloc(const float* x, int64_t rows, int64_t cols, uint8_t* codes, float* r,
                                          float* c, cudaStream_t s);

}  // namespace lpmm
