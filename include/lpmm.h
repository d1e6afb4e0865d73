/*
 * lpmm.h - C ABI of the B200 (sm_100a) fused 4-bit AdamW step.
 *
 * Implements the hot path of "Memory Efficient Optimizers with 4-bit States" (arXiv 2309.01507):
 * Alg. 3 (compressed Adam) with Eq. 1, decoupled weight decay, the first moment kept as
 * B128/DE (Sec. 3, App. E.2) and the second moment as Rank-1/Linear (Sec. 4.1, 4.2), B128/Linear
 * for one-dimensional tensors (Sec. 4.2) and fp32 states for tensors of <= 4096 elements (App. D.1).
 *
 * Conventions
 *  - Pointers named d_* are DEVICE pointers, h_* are HOST pointers; everything else is host memory.
 *  - The caller owns every device buffer (parameters, gradients, the state arena). The library
 *    allocates no device memory; it owns only the small host-side handle (lpmm_state).
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). Work is
 *    enqueued on it and the call returns without synchronizing unless stated otherwise.
 *  - Every function validates its arguments on the host before launching anything and returns a
 *    negative lpmm_status on error; nothing throws, traps or exits. Launch failures are reported
 *    as LPMM_ERR_CUDA (see lpmm_last_cuda_error()).
 *  - Tensors are row-major and contiguous. Codes are 4-bit; element 2k of the flattened tensor sits
 *    in bits 0-3 of byte k and element 2k+1 in bits 4-7; ceil(numel/2) bytes per moment.
 *  - NaN/Inf gradients are not detected; the result is then unspecified (but nothing faults).
 *  - There is no CPU fallback: without a CUDA device every launching call returns LPMM_ERR_CUDA.
 *  - The device that owns the arena must be the current device of the calling thread. A state handle is not
 *    thread-safe: use it from one thread at a time. Steps on one state must also be ordered on the device (the
 *    same stream, or streams ordered by events): the kernels of a step share work counters in the arena header
 *    that each launch leaves at zero for the next one.
 */
#ifndef LPMM_H
#define LPMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t lpmm_status;
#define LPMM_OK 0
#define LPMM_ERR_INVALID_ARG (-1)     /* null pointer, non-positive size, bad enum, bad hyper-parameter */
#define LPMM_ERR_UNSUPPORTED (-2)     /* a combination this build does not implement */
#define LPMM_ERR_ALIGNMENT (-3)       /* a device pointer is not 16-byte aligned */
#define LPMM_ERR_ARENA_TOO_SMALL (-4) /* arena_bytes < lpmm_state_bytes() */
#define LPMM_ERR_CUDA (-5)            /* a CUDA runtime call or launch failed */
#define LPMM_ERR_TOO_LARGE (-6)       /* larger than the fixed capacity of lpmm_quantize_rank1_noalloc */

typedef enum { LPMM_F32 = 0, LPMM_BF16 = 1 } lpmm_dtype;
typedef enum { LPMM_NORM_BLOCK = 0, LPMM_NORM_RANK1 = 1 } lpmm_norm;          /* Sec. 2.2 / Sec. 4.2 */
typedef enum { LPMM_MAP_DE_SIGNED = 0, LPMM_MAP_LINEAR_NOZERO = 1 } lpmm_map; /* App. E.2 / Sec. 4.1 */
/* Second moment of 2-D tensors: 4-bit with rank-1 or block-wise normalization, or not stored at all but
 * reconstructed from fp32 row / column statistics ("4-bit Factor", Sec. 4.3; 1-D tensors stay quantized). */
typedef enum { LPMM_V_RANK1 = 0, LPMM_V_BLOCK = 1, LPMM_V_FACTORED = 2 } lpmm_vmode;

/* How Eq. 1's last line (bias correction, sqrt, division) is evaluated. The stored states (codes and
 * scales) are bit-identical in both modes; only the rounding of the updated parameters differs.
 *   FAST: lr/(1-beta1^t) and 1/(1-beta2^t) folded on the host, one approximate square root and one
 *         approximate reciprocal per element; within 1e-6 * max(|w|, lr) of the IEEE evaluation.
 *   IEEE: every division and the square root correctly rounded, in the order Eq. 1 writes them. */
typedef enum { LPMM_UPDATE_FAST = 0, LPMM_UPDATE_IEEE = 1 } lpmm_update_math;

/* Order of the work inside one step (Sec. 4.2: the row and column maxima of the NEW second moment depend on the whole
 * tensor, so every rank-1 tensor is read twice: once to reduce r', c' and once to update and re-quantize).
 *   TWO_PASS: the maxima pass over all tensors, then the update pass over all tensors (three launches, see
 *             lpmm_adamw4_step). The second read of the gradient and the second-moment codes comes from DRAM.
 *   FUSED:    one launch whose work list puts the update tiles of a tensor closely behind its maxima tiles (the maxima
 *             pass loads the tail of a tensor with the "evict last" L2 priority), so that part of the second read is
 *             served by L2, and that needs no memset node. Needs the default quantizers (LPMM_V_RANK1, m_block 128);
 *             other states and lpmm_adamw4_step_bf16w / lpmm_adamw4_step_host run TWO_PASS. CTAs wait for one
 *             another through counters in the arena; every wait is bounded (see lpmm_state_device_status).
 *   OVERLAP:  TWO_PASS on groups of tensors, with the maxima pass of group k + 1 launched on a second stream (owned by
 *             the handle) beside the update pass of group k; ordered by events, no device-side waiting.
 *   AUTO:     by measurement on B200: FUSED for eligible states of fewer than 63 Mi elements (it is 11-14 % faster
 *             there: fewer launches), else TWO_PASS (faster from there on; the L2-resident re-read saves DRAM bytes
 *             but not time).
 * The stored states and the parameters are bit-identical under all schedules. */
typedef enum { LPMM_SCHEDULE_AUTO = 0, LPMM_SCHEDULE_TWO_PASS = 1, LPMM_SCHEDULE_FUSED = 2, LPMM_SCHEDULE_OVERLAP = 3 } lpmm_schedule;

/* lpmm_shape.flags */
#define LPMM_FORCE_QUANT 1u /* quantize even if numel <= min_quant_numel */
#define LPMM_FORCE_FP32 2u  /* keep fp32 states whatever the size */

/* lpmm_quantize flags */
#define LPMM_Q_GIVEN_SCALES 1u /* use the scales already in d_scale0/d_scale1 instead of recomputing them */

#define LPMM_MAX_NDIM 4
typedef struct {
    int64_t rows, cols; /* ndim 1: rows = numel, cols = 1; ndim 2: rows x cols, row-major;
                           ndim >= 3: rows = product of the leading extents, cols = the last extent */
    int32_t ndim;       /* 1 .. LPMM_MAX_NDIM */
    uint32_t flags;
    int64_t dims[LPMM_MAX_NDIM]; /* ndim >= 3: the extents, row-major (read only then; rows and cols must agree
                                    with them). Such tensors use the general rank-1 normalization of Alg. 4 (App. G):
                                    one vector of maxima per axis, scale of an element = the minimum over its axes. */
} lpmm_shape;

typedef struct {
    int32_t bits;            /* 4 */
    int32_t m_block;         /* first-moment block size B: 128 (Sec. 3) or 2048 (the 8-bit optimizer's size, Sec. 2.2) */
    int32_t v_block;         /* second-moment block size for 1-D tensors and LPMM_V_BLOCK (Sec. 4.2: 128) */
    int32_t v_mode;          /* lpmm_vmode */
    int64_t min_quant_numel; /* tensors with numel <= this keep fp32 states (App. D.1: 4096) */
    int32_t update_math;     /* lpmm_update_math: arithmetic of the parameter update only */
    int32_t schedule;        /* lpmm_schedule: how the two passes over a rank-1 tensor are ordered on the GPU */
    /* Tuning of the schedules; 0 everywhere = the library's choice. None of them changes any result. */
    int32_t tile_elems;        /* elements per tile of the update pass (a power of two, 2048 .. 4 Mi) */
    int32_t tile_elems_maxima; /* elements per tile of the maxima pass (likewise; at least tile_elems) */
    int32_t l2_keep_mbytes;    /* fused: MiB of gradient + second-moment codes at the end of a tensor's maxima pass that
                                  are loaded "evict last" so that the update pass finds them in L2 */
    int32_t lead_melems;       /* fused: Mi elements of ready update work the maxima pass stays ahead of the update pass */
    int32_t gap_items;         /* fused: work items between a tensor's last maxima tile and its first update tile */
    int32_t no_l2_hints;       /* fused: 1 = plain accesses without eviction priorities (to measure what the hints buy) */
    int32_t overlap_groups;    /* overlap: number of tensor groups (0 = 8) */
} lpmm_config;

typedef struct lpmm_state lpmm_state; /* opaque host handle */

/* State kind chosen per tensor (App. D.1 size rule; Sec. 4.2: a tensor that is 1-D, or has an
 * extent of 1, uses block-wise normalization for v). */
#define LPMM_KIND_FP32 0
#define LPMM_KIND_BLOCK 1
#define LPMM_KIND_RANK1 2
#define LPMM_KIND_FACTORED 3 /* LPMM_V_FACTORED: v_scale0 = R (rows), v_scale1 = C (cols), no second-moment codes */

/* Size in bytes of the device arena that holds the states of n tensors (codes, scales, fp32 states
 * of small tensors, the device-side tensor table and the per-step scratch for the rank-1 maxima).
 * Host-only; launches nothing. */
lpmm_status lpmm_state_bytes(const lpmm_config* cfg, const lpmm_shape* shapes, int32_t n, size_t* arena_bytes);

/* Alg. 1 / Alg. 3 "initial state 0": lays the arena out and enqueues its initialisation on `stream`
 * (first-moment codes = the table's zero entry, second-moment codes 0, every scale 0, fp32 states 0;
 * a zero scale dequantizes to exactly 0 whatever the code). d_arena must be 256-byte aligned and stay
 * alive until lpmm_state_destroy. *out receives the handle. */
lpmm_status lpmm_state_init(const lpmm_config* cfg, const lpmm_shape* shapes, int32_t n,
                            void* d_arena, size_t arena_bytes, lpmm_state** out, void* stream);

/* Re-creates a handle over an arena that already holds states (checkpoint restore): the arena bytes
 * are a copy of an arena previously produced with the same cfg/shapes, `phase` is the value
 * lpmm_state_phase() returned when that copy was taken. The arena starts with a header (magic word, layout
 * version, total size, a hash of cfg's quantizer fields and of the shapes); if it does not match what cfg/shapes
 * describe - another library version, another parameter list, not an arena at all - the call changes nothing and
 * returns LPMM_ERR_INVALID_ARG. Otherwise only the tensor table, the work list and the per-step scratch are
 * rewritten. The schedule and tuning fields of cfg may differ from the original's: the states occupy the same
 * offsets under every schedule (the fused schedule's work list lies behind them), so a copy of the first
 * lpmm_state_bytes(original cfg) bytes restored into an arena of lpmm_state_bytes(cfg) bytes is enough.
 * Synchronizes `stream`. */
lpmm_status lpmm_state_attach(const lpmm_config* cfg, const lpmm_shape* shapes, int32_t n,
                              void* d_arena, size_t arena_bytes, int32_t phase, lpmm_state** out, void* stream);

/* One fused step of Alg. 3 over every tensor of the state: decompress m, v; Eq. 1 moment updates,
 * bias correction, decoupled decay w <- w (1 - lr*wd), update w <- w - lr * m^/(sqrt(v^) + eps) with
 * the un-quantized new moments; new block / row / column maxima; compress to the nearest code.
 *   d_params[i] : device pointer to tensor i's fp32 parameters (updated in place)
 *   d_grads[i]  : device pointer to tensor i's gradient in grad_dtype (read only)
 * Both arrays are HOST arrays of n device pointers, each 16-byte aligned (when all of them are 32-byte aligned, as
 * framework allocations are, the update pass uses 256-bit accesses and is ~6 % faster). step is t >= 1.
 * Requires 0 <= beta1, beta2 < 1, lr >= 0, eps >= 0, weight_decay >= 0, all finite.
 * Kernels launched (two-pass schedule; see lpmm_schedule for the others): one pass over the rank-1 tensors that
 * reduces the new row/column maxima, one small pass that inverts them, one pass that updates and re-quantizes the
 * tensors on the tiled path (rows of whole first-moment blocks) and the small fp32 ones; one more update launch each
 * for the element-indexed tensors (other shapes) and for 1-D tensors of 65536 elements or more whose length is a
 * multiple of 128 (folded into rows and updated by the block-wise form of the tiled kernel) when the state's matrices
 * are not block-wise; three more small launches when tensors with three or four axes run as composite matrices
 * (their per-axis statistics are expanded per step). lpmm_state_last_launches() reports the count.
 * LPMM_V_FACTORED (reading of Sec. 4.3, which gives no formula): R <- b2 R + (1-b2) rowsum(g^2), C likewise,
 * v_ij = R_i C_j / sum(R), then Eq. 1 as usual. The first pass writes per-tile partial sums of g^2, a small kernel adds
 * them in a fixed order and updates R, C and sum(R): R and C are reproducible bit for bit (no floating-point atomics).
 * Such tensors need cols % m_block == 0 (else LPMM_ERR_UNSUPPORTED at state creation). */
lpmm_status lpmm_adamw4_step(lpmm_state* st, void* const* d_params, const void* const* d_grads,
                             int32_t grad_dtype, float lr, float beta1, float beta2, float eps,
                             float weight_decay, int64_t step, void* stream);

/* The same step, which also writes a bfloat16 copy (round to nearest even) of every updated parameter, for training
 * set-ups that keep fp32 master parameters here and run the model on a bf16 copy (+2 bytes per parameter of traffic;
 * the paper's method has no such output: its states and fp32 parameters are updated exactly as by lpmm_adamw4_step).
 *   d_params_bf16[i] : device pointer to numel bfloat16 values of tensor i (written), 16-byte aligned; a HOST array
 *                      of n device pointers like d_params.
 * Not available with LPMM_V_FACTORED (LPMM_ERR_UNSUPPORTED). */
lpmm_status lpmm_adamw4_step_bf16w(lpmm_state* st, void* const* d_params, void* const* d_params_bf16,
                                   const void* const* d_grads, int32_t grad_dtype, float lr, float beta1, float beta2,
                                   float eps, float weight_decay, int64_t step, void* stream);

/* One fused step of Alg. 2 (compressed SGDM) over every tensor of the state: decompress m (B128 or B2048 / DE);
 * m <- beta m + g ; w <- w - lr m ; new block maxima ; compress m. Only the first-moment part of the state
 * is used (tensors of <= min_quant_numel elements keep m in fp32); do not mix with lpmm_adamw4_step on one
 * state. One kernel launch; the parameters follow the same operation order as the algorithm's lines 4-5, so
 * they are reproducible bit for bit. Arguments as lpmm_adamw4_step; 0 <= beta < 1, lr >= 0. */
lpmm_status lpmm_sgdm4_step(lpmm_state* st, void* const* d_params, const void* const* d_grads,
                            int32_t grad_dtype, float lr, float beta, void* stream);

/* The same step for callers whose parameters and gradients live in HOST memory (optimizer
 * offloading): copies every tensor's parameters and gradient into the caller's device staging
 * buffers, runs the step there and copies the updated parameters back. The tensors are processed in
 * groups so that copy-in, update and copy-out of neighbouring groups overlap (two internal copy
 * streams owned by the handle, chained to `stream` by events): `stream` waits for earlier work before
 * the first copy and is complete only after the last copy-out.
 *   h_params[i], h_grads[i] : host pointers (pinned memory makes the copies asynchronous)
 *   d_param_stage / d_grad_stage : device buffers of at least lpmm_stage_bytes() bytes each
 * Returns after enqueueing; synchronize the stream before reading h_params. The number of kernels is
 * three per group that holds a rank-1 tensor. */
lpmm_status lpmm_adamw4_step_host(lpmm_state* st, void* const* h_params, const void* const* h_grads,
                                  int32_t grad_dtype, float lr, float beta1, float beta2, float eps,
                                  float weight_decay, int64_t step,
                                  void* d_param_stage, void* d_grad_stage, size_t stage_bytes, void* stream);

/* Bytes needed by each staging buffer of lpmm_adamw4_step_host (tensors packed at 256-byte
 * boundaries, 4 bytes per element). */
lpmm_status lpmm_stage_bytes(const lpmm_state* st, size_t* bytes);

/* Stand-alone quantizer Q = M o N of Sec. 2.2 for a rows x cols fp32 tensor (cols = 1 for 1-D).
 *   norm BLOCK : d_scale0 receives ceil(numel/block) block maxima of |x| (block = 128 or 2048)
 *   norm RANK1 : d_scale0 receives the rows row maxima, d_scale1 the cols column maxima (Sec. 4.2)
 *   map DE_SIGNED (signed input) or LINEAR_NOZERO (meant for non-negative input: RANK1 takes |x|,
 *       BLOCK keeps the sign and sends negative values to code 0)
 * n = x * (1/scale) in fp32 (a scale below FLT_MIN counts as 0 and gives n = 0), code = nearest
 * table entry, exact, lower entry on a tie. d_codes receives ceil(numel/2) bytes. RANK1 + DE_SIGNED
 * is LPMM_ERR_UNSUPPORTED. With LPMM_Q_GIVEN_SCALES the scale buffers are inputs. */
lpmm_status lpmm_quantize(const float* d_x, int64_t rows, int64_t cols, int32_t norm, int32_t map,
                          int32_t block, uint32_t flags, uint8_t* d_codes, float* d_scale0, float* d_scale1,
                          void* stream);

/* Allocation-free rank-1 quantizer. (No counterpart in the paper: this is a deployment variant of
 * lpmm_quantize(..., LPMM_NORM_RANK1, LPMM_MAP_LINEAR_NOZERO, ...) and produces the same codes and scales.)
 *
 * Who it is for: callers that cannot get device memory at the moment of the call and have nothing to
 * lend as scratch - a process whose whole GPU memory is already held by a framework's pool, a serving
 * loop that runs under a fixed memory budget, code that must not call cudaMalloc because that call
 * synchronizes the device. They pass only the input and the three outputs; the intermediate buffer
 * (the reciprocals of the row and column maxima) lives in a fixed array inside the library image.
 *
 *  - Capacity: round_up(rows, 4) + cols <= LPMM_NOALLOC_MAX_SCALES; beyond that the call launches nothing
 *    and returns LPMM_ERR_TOO_LARGE. The array costs LPMM_NOALLOC_MAX_SCALES * 4 bytes (1 MiB) of device
 *    memory on every GPU that loads the library, from load until the process exits.
 *  - The first call on each device looks up the array's device address (a host-side query, no allocation).
 *    Make that first call before starting any stream capture on that device. The address is remembered per
 *    device for the life of the process and does not survive cudaDeviceReset(): do not call this function
 *    again after a reset of a device it has already been used on.
 *  - All calls on a device share the one array and it keeps whatever the last call left there. Nothing
 *    in it needs to start at zero (each call overwrites the part it uses before reading it; the outputs
 *    d_scale0 / d_scale1 are cleared by the call itself). Two calls that overlap on the GPU - different
 *    streams, or different host threads - race on it: run them one after the other.
 *  - It calls neither cudaMalloc nor cudaFree nor any library routine that allocates. */
#define LPMM_NOALLOC_MAX_SCALES 262144
lpmm_status lpmm_quantize_rank1_noalloc(const float* d_x, int64_t rows, int64_t cols, uint8_t* d_codes,
                                        float* d_scale0 /* rows */, float* d_scale1 /* cols */, void* stream);

/* Dequantizer of Sec. 2.2: d_out[i] = T(code_i) * scale_i, scale_i = block maximum or min(r, c). */
lpmm_status lpmm_dequantize(const uint8_t* d_codes, const float* d_scale0, const float* d_scale1,
                            int64_t rows, int64_t cols, int32_t norm, int32_t map, int32_t block,
                            float* d_out, void* stream);

/* Device pointers into the arena for tensor i's current state (for inspection and parity checks).
 * Pointers that do not apply to the tensor's kind are set to NULL. Sizes: codes ceil(numel/2) bytes;
 * m_scale ceil(numel/m_block); BLOCK v_scale0 ceil(numel/v_block); RANK1 v_scale0 rows, v_scale1 cols;
 * FP32 m32/v32 numel floats. Valid until the next step (rank-1 scales alternate between two buffers). */
lpmm_status lpmm_state_view(const lpmm_state* st, int32_t tensor, int32_t* kind,
                            const uint8_t** m_codes, const float** m_scale,
                            const uint8_t** v_codes, const float** v_scale0, const float** v_scale1,
                            const float** m32, const float** v32);

/* Statistics of one axis of a tensor with rank-1 normalization (Alg. 4: mu_r, one maximum per index of axis r):
 * *mu receives a device pointer into the arena, *extent the axis' length. axis counts the tensor's own axes
 * (a matrix has axis 0 = r, axis 1 = c). The pointer is valid until the next step (the buffers alternate).
 * LPMM_ERR_INVALID_ARG for tensors of another kind or an axis out of range. */
lpmm_status lpmm_state_view_axis(const lpmm_state* st, int32_t tensor, int32_t axis, const float** mu, int64_t* extent);

/* Reads the device-side error word of the state (synchronizes `stream`). 0 = no error; 2 = a CTA of the fused
 * schedule waited for another tile's result longer than the limit (about two seconds) and stopped taking work: the
 * states written by that step are incomplete and the arena must be re-initialised or restored from a checkpoint.
 * Kernels never trap or spin without limit. */
lpmm_status lpmm_state_device_status(lpmm_state* st, int32_t* status, void* stream);

/* Self-test of the bounded wait the fused schedule relies on: launches two CTAs that wait (with a limit of a few
 * milliseconds) for a counter in the arena header that nothing ever advances. *ctas_gave_up receives how many of them
 * ran out of patience (2), *status_word what they left in the device status word (2). The word and the counters are
 * put back to zero afterwards, so the state stays usable. Synchronizes `stream`. */
lpmm_status lpmm_state_selftest_wait(lpmm_state* st, int32_t* ctas_gave_up, int32_t* status_word, void* stream);

/* Fused schedule: how many waits of an update tile for its tensor's maxima tiles did not succeed at the first look
 * since the last call, and how many nanoseconds they took in all (summed over CTAs). Reads and clears the two
 * counters; synchronizes `stream`. A tuning aid for lead_melems / gap_items. */
lpmm_status lpmm_state_wait_stats(lpmm_state* st, int64_t* waits, int64_t* wait_ns, void* stream);

/* The checking build. The library can be compiled with -DLPMM_DEBUG (paper_2309_01507_b200/build.py builds it as
 * liblpmm_debug.so beside the normal one); it stands in for a memory checker where none can be run:
 *   - every sub-buffer of the arena is followed by a 256-byte guard zone filled with a pattern (so lpmm_state_bytes is
 *     larger and arenas of the two builds cannot be attached to one another), and
 *   - the step kernels check, per tile, that the first and last element they are about to touch lie inside the tensor;
 *     a failed check puts 0x100 + its number into the device status word (lpmm_state_device_status) and the tile is
 *     skipped - nothing traps.
 * lpmm_build_is_checking() tells the two builds apart. lpmm_state_check_guards() counts the guard bytes that no longer
 * hold the pattern (*zones receives the number of guard zones); lpmm_state_selftest_check() runs one check that fails on
 * purpose and returns the status word it produced (0x17f), then clears it. Both return LPMM_ERR_UNSUPPORTED in the
 * normal build and synchronize `stream`. */
int32_t lpmm_build_is_checking(void);
lpmm_status lpmm_state_check_guards(lpmm_state* st, int64_t* zones, int64_t* damaged, void* stream);
lpmm_status lpmm_state_selftest_check(lpmm_state* st, int32_t* status_word, void* stream);

/* LPMM_SCHEDULE_TWO_PASS, LPMM_SCHEDULE_FUSED or LPMM_SCHEDULE_OVERLAP: what lpmm_adamw4_step runs on this state. */
int32_t lpmm_state_schedule(const lpmm_state* st);

/* 0, 1 or 2: which of the three rank-1 scale buffers is current (they rotate: current, new, being cleared for the
 * step after). Save it with a copy of the arena. */
int32_t lpmm_state_phase(const lpmm_state* st);

/* Optional per-kernel timing. While enabled, every lpmm_adamw4_step records CUDA events on its stream
 * around its kernels (host-side event objects only, created by this call, none by a step; at most 256 steps are
 * recorded between two reads). Under the fused schedule the whole launch is reported as the update pass. */
lpmm_status lpmm_state_profile(lpmm_state* st, int32_t enable);

/* Waits for the recorded steps to finish, returns the summed durations in milliseconds of the rank-1
 * maxima pass, the reciprocal pass and the update/re-quantize pass over `steps` recorded steps, and
 * clears the record. Any output pointer may be NULL. */
lpmm_status lpmm_state_profile_read(lpmm_state* st, double* pass1_ms, double* rcp_ms, double* pass2_ms, int32_t* steps);

/* Number of kernels the last lpmm_adamw4_step on this state launched. Two-pass schedule: 3 when a rank-1 tensor is
 * present, else 1, and one additional memset node clears the new row/column maxima. Fused schedule: 1 (no memset
 * node: a tensor's last update tile clears the buffer that receives the next step's maxima). */
int32_t lpmm_state_last_launches(const lpmm_state* st);

/* Frees the host handle only; the arena stays the caller's. NULL is allowed. */
void lpmm_state_destroy(lpmm_state* st);

const char* lpmm_status_string(lpmm_status s);

/* The cudaError_t (as int) of the most recent failed CUDA call made by this library in this thread. */
int32_t lpmm_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* LPMM_H */
