/*
 * CPU oracle for the 4-bit AdamW step of "Memory Efficient Optimizers with 4-bit States".
 *
 * TEST INFRASTRUCTURE ONLY. This is a plain, slow, loop-by-loop restatement of what the paper
 * defines, used to check the CUDA library and to report a CPU baseline. Only the test-suite,
 * the smoke check and the benchmark's CPU-baseline leg may call it; the CUDA library shares no
 * code, header, table or constant with it.
 *
 * Arithmetic contract: every floating-point operation below is a single IEEE-754 binary32
 * operation (compile with -ffp-contract=off, no fast-math), in the order written; denormals are
 * kept. Codes are 4-bit unsigned integers stored two per byte (even element in bits 0-3).
 *
 * Parity pins (tests/test_oracle_*.py): every function here is pinned to values the paper prints,
 * closed forms, brute force, or a library routine, except the 100-step closeness of the 4-bit
 * trajectory to an fp32 AdamW trajectory, which the paper does not quantify: parity unpinned for
 * that closeness (the step itself is pinned piecewise).
 */
#ifndef LPMM_ORACLE_H
#define LPMM_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Sec. 2.2 "Mapping" and App. E.2 "Linear mapping": T(i) = (i+1)/2^b, i = 0 .. 2^b-1. Returns 2^b. */
int lpmm_oracle_linear_map(int bits, float* T);

/* App. E.2 "Dynamic exponent mapping". Builds the table from the bit patterns:
 * unsigned  b = E + 1 + F : E leading zeros, indicator bit, F fraction bits,
 *           value 10^-E * fraction_F[k]; corner cases 0...0 -> 0 and 0...01 -> 1;
 * signed    b = 1 + E + 1 + F : first bit is the sign; corner cases 00..0 -> 0, 10..0 -> +1
 *           (-1 is not representable).
 * drop_zero removes the entry 0 (the "DE-0" variant of Sec. 4.1). The result is sorted
 * increasingly; T(i) is its i-th entry. Returns the number of entries. */
int lpmm_oracle_de_map(int bits, int is_signed, int drop_zero, float* T);

/* App. E.2: fraction_F[k] = (p_k + p_{k+1})/2 with p_j = 0.9 j / 2^F + 0.1, as a double. */
double lpmm_oracle_de_fraction(int F, int k);

/* Sec. 2.2 "Mapping": argmin_i |n - T(i)| in exact arithmetic on the binary32 values
 * (differences taken in binary64); the first minimiser wins a tie. */
int lpmm_oracle_nearest(const float* T, int n_entries, float n);

/* Reciprocal of a quantization scale: 1/s in binary32 when s >= FLT_MIN, else 0 (a zero or
 * denormal scale means "everything under it quantizes as zero"). */
float lpmm_oracle_rcp(float s);

/* Sec. 2.2 "Normalization", block-wise: scale[k] = max |x_i| over block k of B consecutive
 * elements of the flattened tensor; ceil(numel/B) scales, the last block may be short. */
void lpmm_oracle_block_scales(const float* x, int64_t numel, int64_t B, float* scale);

/* Alg. 4 (rank-1 normalization, any number of dimensions): mu[r][j] = max over all other
 * indices of |x[..., j at axis r, ...]|. mu_flat holds mu_1 (d_1 values), then mu_2, ... */
void lpmm_oracle_rank1_stats(const float* x, int ndim, const int64_t* dims, float* mu_flat);

/* Alg. 4, second loop: M_i = min_r mu[r][Phi(i)_r] for every flat index i. */
void lpmm_oracle_rank1_scale_field(int ndim, const int64_t* dims, const float* mu_flat, float* M);

/* Quantize x with per-element scales already chosen (scale_of_elem[i]) onto table T.
 * n_i = x_i * rcp(scale_i) (true_division != 0: n_i = x_i / scale_i when scale_i >= FLT_MIN).
 * codes: one byte per element, value 0..n_entries-1. */
void lpmm_oracle_map_codes(const float* x, const float* scale_of_elem, int64_t numel,
                           const float* T, int n_entries, int true_division, uint8_t* codes);

/* Block-wise quantizer (Sec. 2.2). given_scales != 0: use scale[] as passed instead of recomputing. */
void lpmm_oracle_quantize_block(const float* x, int64_t numel, int64_t B, const float* T, int n_entries,
                                int given_scales, int true_division, float* scale, uint8_t* codes);

/* Rank-1 quantizer for a rows x cols matrix (Sec. 4.2): r_i = max_j x_ij, c_j = max_i x_ij,
 * n_ij = x_ij * max(rcp r_i, rcp c_j). Input is taken as non-negative (|x| is used, as Alg. 4). */
void lpmm_oracle_quantize_rank1(const float* x, int64_t rows, int64_t cols, const float* T, int n_entries,
                                int given_scales, int true_division, float* r, float* c, uint8_t* codes);

/* Dequantizers (Sec. 2.2 "Dequantization"): x~ = T(q) * scale. */
void lpmm_oracle_dequantize_block(const uint8_t* codes, int64_t numel, int64_t B, const float* T,
                                  const float* scale, float* out);
void lpmm_oracle_dequantize_rank1(const uint8_t* codes, int64_t rows, int64_t cols, const float* T,
                                  const float* r, const float* c, float* out);

/* Two 4-bit codes per byte: element 2k in bits 0-3, element 2k+1 in bits 4-7 of byte k;
 * ceil(numel/2) bytes; an odd tail leaves the last high nibble 0. */
void lpmm_oracle_pack4(const uint8_t* codes, int64_t numel, uint8_t* packed);
void lpmm_oracle_unpack4(const uint8_t* packed, int64_t numel, uint8_t* codes);

/* bfloat16 bit pattern -> binary32 (exact). */
void lpmm_oracle_bf16_to_f32(const uint16_t* in, int64_t numel, float* out);

/* binary32 -> bfloat16 bit pattern: round to nearest, ties to even; NaN -> 0x7fff. (Not part of the paper's method:
 * checks the optional bfloat16 copy of the parameters that the CUDA library can write.) */
void lpmm_oracle_f32_to_bf16(const float* in, int64_t numel, uint16_t* out);

/* Hyper-parameters of Eq. 1 plus decoupled weight decay. */
typedef struct {
    float lr, beta1, beta2, eps, weight_decay;
    int64_t step;          /* t >= 1 */
    int32_t true_division; /* 0: multiply by reciprocal scale (contract); 1: divide by the scale */
} lpmm_oracle_hyper;

/* State kinds chosen by the rule of App. D.1 and Sec. 4.2. */
enum { LPMM_ORACLE_FP32 = 0, LPMM_ORACLE_BLOCK = 1, LPMM_ORACLE_RANK1 = 2 };

/* numel <= min_quant_numel (and not forced) -> FP32; one-dimensional or any extent 1 -> BLOCK;
 * otherwise RANK1. force: 0 none, 1 force quantization, 2 force fp32. */
int lpmm_oracle_kind(int64_t rows, int64_t cols, int ndim, int64_t min_quant_numel, int force);

/* One compressed-AdamW step on one tensor (Alg. 3 with Eq. 1, decoupled decay):
 *   decompress m, v -> moment EMAs -> bias correction -> decay + update -> new scales -> compress.
 * g is binary32. Packed states are updated in place.
 *   FP32 : m32, v32 (numel floats each); the other state pointers are ignored.
 *   BLOCK: m_codes/m_scale (block m_block), v_codes/v_s0 (block v_block, linear map).
 *   RANK1: m as BLOCK; v_codes with v_s0 = r (rows), v_s1 = c (cols).
 * Returns 0, or -1 on a bad argument. */
int lpmm_oracle_adamw4_step(float* w, const float* g, int64_t rows, int64_t cols, int kind,
                            int64_t m_block, int64_t v_block,
                            uint8_t* m_codes, float* m_scale,
                            uint8_t* v_codes, float* v_s0, float* v_s1,
                            float* m32, float* v32,
                            const lpmm_oracle_hyper* h);

/* The same step on a tensor of any rank p >= 1 (row-major dims[0..p-1]) whose second moment uses rank-1
 * normalization in the general form of Alg. 4: mu_flat holds the per-axis maxima mu_1 (dims[0] values), mu_2, ...
 * of the stored second moment; the scale of element i is M_i = min_r mu_r[Phi(i)_r] and n_i = v_i * rcp(M_i).
 * The first moment is compressed block-wise over the flattened tensor. With p = 2 this is the RANK1 case of
 * lpmm_oracle_adamw4_step (mu_1 = r, mu_2 = c). Returns 0, or -1 on a bad argument. */
int lpmm_oracle_adamw4_step_nd(float* w, const float* g, int ndim, const int64_t* dims, int64_t m_block,
                               uint8_t* m_codes, float* m_scale, uint8_t* v_codes, float* mu_flat,
                               const lpmm_oracle_hyper* h);

/* Initial compressed state s_0 = 0 (Alg. 1): m codes all "the entry 0" of the signed DE table,
 * v codes 0, every scale 0. */
void lpmm_oracle_state_init(int64_t rows, int64_t cols, int kind, int64_t m_block, int64_t v_block,
                            uint8_t* m_codes, float* m_scale, uint8_t* v_codes, float* v_s0, float* v_s1,
                            float* m32, float* v32);

/* One step of the factorized variant ("4-bit Factor", Sec. 4.3 and Sec. 5) on one rows x cols matrix: the first
 * moment is compressed as in lpmm_oracle_adamw4_step; the second moment is replaced by Adafactor's rank-1
 * reconstruction from fp32 row and column statistics. The paper gives no formula; the reading is:
 *   rs_i = sum_j g_ij^2, cs_j = sum_i g_ij^2   (squares in binary32, sums accumulated in binary64, rounded once)
 *   R <- beta2 R + (1 - beta2) rs ; C <- beta2 C + (1 - beta2) cs            (binary32, R_0 = C_0 = 0)
 *   v_ij = (R_i * (1 / sum_k R_k)) * C_j    (sum in binary64, rounded once; 0 when the sum is below FLT_MIN)
 * followed by Eq. 1's bias correction and update with this v (no update clipping, no relative step size).
 * Parity unpinned beyond the invariants tested in tests/test_oracle_factor.py. Returns 0 or -1. */
int lpmm_oracle_adamw4_factor_step(float* w, const float* g, int64_t rows, int64_t cols, int64_t m_block,
                                   uint8_t* m_codes, float* m_scale, float* R, float* C,
                                   const lpmm_oracle_hyper* h);

/* One compressed-SGDM step on one tensor (Alg. 2): m_t = beta * m_{t-1} + g ; w = w - lr * m_t ; compress m_t
 * (block-wise normalization with block m_block, signed dynamic-exponent map). quantized != 0: m_codes / m_scale
 * hold the state; else m32 (numel floats). Returns 0, or -1 on a bad argument. */
int lpmm_oracle_sgdm4_step(float* w, const float* g, int64_t numel, int quantized, int64_t m_block,
                           uint8_t* m_codes, float* m_scale, float* m32, float lr, float beta, int true_division);

/* Number of OpenMP threads the loops above use (1 when built without OpenMP). */
int lpmm_oracle_threads(void);
void lpmm_oracle_set_threads(int n);

#ifdef __cplusplus
}
#endif
#endif
