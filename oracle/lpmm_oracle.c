/*
 * CPU oracle: see lpmm_oracle.h. TEST INFRASTRUCTURE ONLY.
 *
 * Build: gcc -O2 -std=c99 -ffp-contract=off -fno-fast-math [-fopenmp] -shared -fPIC
 * Every float expression below is written one operation per rounding, in the order the paper's
 * equations state; nothing is blocked, fused or reordered.
 */
#include "lpmm_oracle.h"

#include <float.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ quantization mappings */

int lpmm_oracle_linear_map(int bits, float* T) {
    /* App. E.2: the 2^b + 1 evenly spaced points of [0, 1] with the first (zero) dropped. */
    int n = 1 << bits;
    for (int i = 0; i < n; ++i) T[i] = (float)((double)(i + 1) / (double)n);
    return n;
}

double lpmm_oracle_de_fraction(int F, int k) {
    /* p_j = (1 - 0.1)/2^F * j + 0.1 ; fraction[k] = (p_k + p_{k+1}) / 2.
     * Kept as an exact rational: (2^(F+1) + 9 (2k+1)) / (10 * 2^(F+1)). */
    double two = (double)(1 << (F + 1));
    return (two + 9.0 * (double)(2 * k + 1)) / (10.0 * two);
}

static double de_value(int width, unsigned pattern) {
    /* pattern has `width` bits and is non-zero: E leading zeros, one indicator bit, F fraction bits. */
    int E = 0;
    while (((pattern >> (width - 1 - E)) & 1u) == 0u) ++E;
    int F = width - 1 - E;
    unsigned k = pattern & ((1u << F) - 1u);
    /* 10^-E * fraction_F[k], numerator and denominator kept integral so only one rounding occurs. */
    double num = (double)(1 << (F + 1)) + 9.0 * (double)(2 * k + 1);
    double den = 10.0 * (double)(1 << (F + 1));
    for (int e = 0; e < E; ++e) den *= 10.0;
    return num / den;
}

static int cmp_float(const void* a, const void* b) {
    float x = *(const float*)a, y = *(const float*)b;
    return (x > y) - (x < y);
}

int lpmm_oracle_de_map(int bits, int is_signed, int drop_zero, float* T) {
    int n = 0;
    if (!is_signed) {
        for (unsigned p = 0; p < (1u << bits); ++p) {
            double val;
            if (p == 0u) val = 0.0;            /* corner case: all zeros -> 0 */
            else if (p == 1u) val = 1.0;       /* corner case: 0...01   -> 1 */
            else val = de_value(bits, p);
            if (drop_zero && val == 0.0) continue;
            T[n++] = (float)val;
        }
    } else {
        int width = bits - 1;
        for (unsigned s = 0; s < 2u; ++s) {
            for (unsigned p = 0; p < (1u << width); ++p) {
                double val;
                if (p == 0u) val = s ? 1.0 : 0.0; /* 00..0 -> 0, 10..0 -> +1; -1 does not exist */
                else val = (s ? -1.0 : 1.0) * de_value(width, p);
                if (drop_zero && val == 0.0) continue;
                T[n++] = (float)val;
            }
        }
    }
    qsort(T, (size_t)n, sizeof(float), cmp_float);
    return n;
}

int lpmm_oracle_nearest(const float* T, int n_entries, float n) {
    int best = 0;
    double best_d = fabs((double)n - (double)T[0]);
    for (int i = 1; i < n_entries; ++i) {
        double d = fabs((double)n - (double)T[i]);
        if (d < best_d) { best_d = d; best = i; }
    }
    return best;
}

float lpmm_oracle_rcp(float s) {
    return (s >= FLT_MIN) ? (1.0f / s) : 0.0f;
}

/* ------------------------------------------------------------------ normalization statistics */

void lpmm_oracle_block_scales(const float* x, int64_t numel, int64_t B, float* scale) {
    int64_t nb = (numel + B - 1) / B;
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < nb; ++k) {
        int64_t lo = k * B, hi = lo + B < numel ? lo + B : numel;
        float mx = 0.0f;
        for (int64_t i = lo; i < hi; ++i) mx = fmaxf(mx, fabsf(x[i]));
        scale[k] = mx;
    }
}

void lpmm_oracle_rank1_stats(const float* x, int ndim, const int64_t* dims, float* mu_flat) {
    int64_t total = 1, nstat = 0;
    for (int r = 0; r < ndim; ++r) { total *= dims[r]; nstat += dims[r]; }
    for (int64_t k = 0; k < nstat; ++k) mu_flat[k] = 0.0f;
    int64_t idx[16];
    for (int64_t i = 0; i < total; ++i) {
        int64_t rem = i; /* Phi(i): row-major multi-index of flat position i */
        for (int r = ndim - 1; r >= 0; --r) { idx[r] = rem % dims[r]; rem /= dims[r]; }
        float a = fabsf(x[i]);
        int64_t off = 0;
        for (int r = 0; r < ndim; ++r) {
            float* mu = mu_flat + off + idx[r];
            *mu = fmaxf(*mu, a);
            off += dims[r];
        }
    }
}

void lpmm_oracle_rank1_scale_field(int ndim, const int64_t* dims, const float* mu_flat, float* M) {
    int64_t total = 1;
    for (int r = 0; r < ndim; ++r) total *= dims[r];
    int64_t idx[16];
    for (int64_t i = 0; i < total; ++i) {
        int64_t rem = i;
        for (int r = ndim - 1; r >= 0; --r) { idx[r] = rem % dims[r]; rem /= dims[r]; }
        int64_t off = 0;
        float mn = 0.0f;
        for (int r = 0; r < ndim; ++r) {
            float mu = mu_flat[off + idx[r]];
            mn = (r == 0) ? mu : fminf(mn, mu);
            off += dims[r];
        }
        M[i] = mn;
    }
}

/* ------------------------------------------------------------------ quantize / dequantize */

static float normalize(float x, float scale, int true_division) {
    if (true_division) return (scale >= FLT_MIN) ? (x / scale) : 0.0f;
    return x * lpmm_oracle_rcp(scale);
}

void lpmm_oracle_map_codes(const float* x, const float* scale_of_elem, int64_t numel,
                           const float* T, int n_entries, int true_division, uint8_t* codes) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < numel; ++i) {
        float n = normalize(x[i], scale_of_elem[i], true_division);
        codes[i] = (uint8_t)lpmm_oracle_nearest(T, n_entries, n);
    }
}

void lpmm_oracle_quantize_block(const float* x, int64_t numel, int64_t B, const float* T, int n_entries,
                                int given_scales, int true_division, float* scale, uint8_t* codes) {
    if (!given_scales) lpmm_oracle_block_scales(x, numel, B, scale);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < numel; ++i) {
        float n = normalize(x[i], scale[i / B], true_division);
        codes[i] = (uint8_t)lpmm_oracle_nearest(T, n_entries, n);
    }
}

void lpmm_oracle_quantize_rank1(const float* x, int64_t rows, int64_t cols, const float* T, int n_entries,
                                int given_scales, int true_division, float* r, float* c, uint8_t* codes) {
    if (!given_scales) {
        for (int64_t i = 0; i < rows; ++i) r[i] = 0.0f;
        for (int64_t j = 0; j < cols; ++j) c[j] = 0.0f;
        for (int64_t i = 0; i < rows; ++i)
            for (int64_t j = 0; j < cols; ++j) {
                float a = fabsf(x[i * cols + j]);
                r[i] = fmaxf(r[i], a);
                c[j] = fmaxf(c[j], a);
            }
    }
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j) {
            float xv = fabsf(x[i * cols + j]);
            float n;
            if (true_division) {
                float s = fminf(r[i], c[j]);
                n = (s >= FLT_MIN) ? (xv / s) : 0.0f;
            } else {
                /* 1/min(r,c) = max(1/r, 1/c): the binary32 reciprocal is monotone. */
                n = xv * fmaxf(lpmm_oracle_rcp(r[i]), lpmm_oracle_rcp(c[j]));
            }
            codes[i * cols + j] = (uint8_t)lpmm_oracle_nearest(T, n_entries, n);
        }
}

void lpmm_oracle_dequantize_block(const uint8_t* codes, int64_t numel, int64_t B, const float* T,
                                  const float* scale, float* out) {
    for (int64_t i = 0; i < numel; ++i) out[i] = T[codes[i]] * scale[i / B];
}

void lpmm_oracle_dequantize_rank1(const uint8_t* codes, int64_t rows, int64_t cols, const float* T,
                                  const float* r, const float* c, float* out) {
    for (int64_t i = 0; i < rows; ++i)
        for (int64_t j = 0; j < cols; ++j)
            out[i * cols + j] = T[codes[i * cols + j]] * fminf(r[i], c[j]);
}

void lpmm_oracle_pack4(const uint8_t* codes, int64_t numel, uint8_t* packed) {
    int64_t nbytes = (numel + 1) / 2;
    for (int64_t k = 0; k < nbytes; ++k) {
        uint8_t lo = codes[2 * k];
        uint8_t hi = (2 * k + 1 < numel) ? codes[2 * k + 1] : 0;
        packed[k] = (uint8_t)(lo | (hi << 4));
    }
}

void lpmm_oracle_unpack4(const uint8_t* packed, int64_t numel, uint8_t* codes) {
    for (int64_t i = 0; i < numel; ++i) {
        uint8_t byte = packed[i / 2];
        codes[i] = (i % 2 == 0) ? (uint8_t)(byte & 0x0F) : (uint8_t)(byte >> 4);
    }
}

void lpmm_oracle_bf16_to_f32(const uint16_t* in, int64_t numel, float* out) {
    for (int64_t i = 0; i < numel; ++i) {
        uint32_t bits = ((uint32_t)in[i]) << 16;
        memcpy(&out[i], &bits, sizeof(float));
    }
}

/* ------------------------------------------------------------------ the compressed AdamW step */

int lpmm_oracle_kind(int64_t rows, int64_t cols, int ndim, int64_t min_quant_numel, int force) {
    int64_t numel = rows * cols;
    if (force == 2) return LPMM_ORACLE_FP32;
    if (force != 1 && numel <= min_quant_numel) return LPMM_ORACLE_FP32; /* App. D.1: size <= 4096 */
    if (ndim <= 1 || rows == 1 || cols == 1) return LPMM_ORACLE_BLOCK;   /* Sec. 4.2: 1-D uses B128 */
    return LPMM_ORACLE_RANK1;
}

static int zero_code_of(const float* T, int n) {
    for (int i = 0; i < n; ++i) if (T[i] == 0.0f) return i;
    return -1;
}

void lpmm_oracle_state_init(int64_t rows, int64_t cols, int kind, int64_t m_block, int64_t v_block,
                            uint8_t* m_codes, float* m_scale, uint8_t* v_codes, float* v_s0, float* v_s1,
                            float* m32, float* v32) {
    int64_t numel = rows * cols;
    if (kind == LPMM_ORACLE_FP32) {
        for (int64_t i = 0; i < numel; ++i) { m32[i] = 0.0f; v32[i] = 0.0f; }
        return;
    }
    float Tde[16];
    int nde = lpmm_oracle_de_map(4, 1, 0, Tde);
    uint8_t z = (uint8_t)zero_code_of(Tde, nde);
    int64_t nbytes = (numel + 1) / 2;
    for (int64_t k = 0; k < nbytes; ++k) {
        int has_hi = (2 * k + 1 < numel);
        m_codes[k] = (uint8_t)(z | (has_hi ? (z << 4) : 0));
        v_codes[k] = 0;
    }
    for (int64_t k = 0; k < (numel + m_block - 1) / m_block; ++k) m_scale[k] = 0.0f;
    if (kind == LPMM_ORACLE_BLOCK) {
        for (int64_t k = 0; k < (numel + v_block - 1) / v_block; ++k) v_s0[k] = 0.0f;
    } else {
        for (int64_t i = 0; i < rows; ++i) v_s0[i] = 0.0f;
        for (int64_t j = 0; j < cols; ++j) v_s1[j] = 0.0f;
    }
}

int lpmm_oracle_adamw4_step(float* w, const float* g, int64_t rows, int64_t cols, int kind,
                            int64_t m_block, int64_t v_block,
                            uint8_t* m_codes, float* m_scale,
                            uint8_t* v_codes, float* v_s0, float* v_s1,
                            float* m32, float* v32,
                            const lpmm_oracle_hyper* h) {
    if (!w || !g || !h || rows <= 0 || cols <= 0 || h->step < 1) return -1;
    const int64_t numel = rows * cols;
    const float beta1 = h->beta1, beta2 = h->beta2;
    const float omb1 = 1.0f - beta1;   /* (1 - beta) evaluated in binary32 */
    const float omb2 = 1.0f - beta2;
    /* Eq. 1: 1 - beta^t, evaluated in binary64 and rounded once. */
    const float bc1 = (float)(1.0 - pow((double)beta1, (double)h->step));
    const float bc2 = (float)(1.0 - pow((double)beta2, (double)h->step));
    const float decay = 1.0f - h->lr * h->weight_decay;

    float* m = (float*)malloc(sizeof(float) * (size_t)numel);
    float* v = (float*)malloc(sizeof(float) * (size_t)numel);
    if (!m || !v) { free(m); free(v); return -1; }

    float Tde[16], Tlin[16];
    lpmm_oracle_de_map(4, 1, 0, Tde);
    lpmm_oracle_linear_map(4, Tlin);
    uint8_t* q = NULL;

    /* Alg. 3 line 3: decompress. */
    if (kind == LPMM_ORACLE_FP32) {
        memcpy(m, m32, sizeof(float) * (size_t)numel);
        memcpy(v, v32, sizeof(float) * (size_t)numel);
    } else {
        q = (uint8_t*)malloc((size_t)numel);
        if (!q) { free(m); free(v); return -1; }
        lpmm_oracle_unpack4(m_codes, numel, q);
        lpmm_oracle_dequantize_block(q, numel, m_block, Tde, m_scale, m);
        lpmm_oracle_unpack4(v_codes, numel, q);
        if (kind == LPMM_ORACLE_BLOCK) lpmm_oracle_dequantize_block(q, numel, v_block, Tlin, v_s0, v);
        else lpmm_oracle_dequantize_rank1(q, rows, cols, Tlin, v_s0, v_s1, v);
    }

    /* Alg. 3 lines 4-8 (Eq. 1), with the decoupled decay applied to w_{t-1} first. */
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < numel; ++i) {
        float gi = g[i];
        float a = beta1 * m[i];
        float b = omb1 * gi;
        float mt = a + b;
        float gg = gi * gi;
        float c = beta2 * v[i];
        float d = omb2 * gg;
        float vt = c + d;
        float mhat = mt / bc1;
        float vhat = vt / bc2;
        float denom = sqrtf(vhat) + h->eps;
        float ratio = mhat / denom;
        float upd = h->lr * ratio;
        float wd = w[i] * decay;
        w[i] = wd - upd;
        m[i] = mt;
        v[i] = vt;
    }

    /* Alg. 3 line 9: compress the new moments. */
    if (kind == LPMM_ORACLE_FP32) {
        memcpy(m32, m, sizeof(float) * (size_t)numel);
        memcpy(v32, v, sizeof(float) * (size_t)numel);
    } else {
        lpmm_oracle_quantize_block(m, numel, m_block, Tde, 16, 0, h->true_division, m_scale, q);
        lpmm_oracle_pack4(q, numel, m_codes);
        if (kind == LPMM_ORACLE_BLOCK)
            lpmm_oracle_quantize_block(v, numel, v_block, Tlin, 16, 0, h->true_division, v_s0, q);
        else
            lpmm_oracle_quantize_rank1(v, rows, cols, Tlin, 16, 0, h->true_division, v_s0, v_s1, q);
        lpmm_oracle_pack4(q, numel, v_codes);
        free(q);
    }
    free(m);
    free(v);
    return 0;
}

/* binary32 -> bfloat16 bit pattern, round to nearest, ties to even (IEEE 754 roundTiesToEven on the 16 dropped
 * bits); a NaN becomes the canonical 0x7fff. */
void lpmm_oracle_f32_to_bf16(const float* in, int64_t numel, uint16_t* out) {
    for (int64_t i = 0; i < numel; ++i) {
        uint32_t u;
        memcpy(&u, &in[i], 4);
        if ((u & 0x7fffffffu) > 0x7f800000u) { out[i] = 0x7fffu; continue; }
        uint32_t keep = u >> 16, rest = u & 0xffffu;
        if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1u;   /* may carry into the exponent: that is the rounding to the next binade or to infinity */
        out[i] = (uint16_t)keep;
    }
}

/* ------------------------------------------------------------------ Alg. 3 on a tensor of any rank (Alg. 4) */

int lpmm_oracle_adamw4_step_nd(float* w, const float* g, int ndim, const int64_t* dims, int64_t m_block,
                               uint8_t* m_codes, float* m_scale, uint8_t* v_codes, float* mu_flat,
                               const lpmm_oracle_hyper* h) {
    if (!w || !g || !h || !dims || ndim < 1 || ndim > 16 || h->step < 1) return -1;
    int64_t numel = 1;
    for (int r = 0; r < ndim; ++r) { if (dims[r] <= 0) return -1; numel *= dims[r]; }
    const float beta1 = h->beta1, beta2 = h->beta2;
    const float omb1 = 1.0f - beta1, omb2 = 1.0f - beta2;
    const float bc1 = (float)(1.0 - pow((double)beta1, (double)h->step));
    const float bc2 = (float)(1.0 - pow((double)beta2, (double)h->step));
    const float decay = 1.0f - h->lr * h->weight_decay;
    float* m = (float*)malloc(sizeof(float) * (size_t)numel);
    float* v = (float*)malloc(sizeof(float) * (size_t)numel);
    float* M = (float*)malloc(sizeof(float) * (size_t)numel);
    uint8_t* q = (uint8_t*)malloc((size_t)numel);
    if (!m || !v || !M || !q) { free(m); free(v); free(M); free(q); return -1; }
    float Tde[16], Tlin[16];
    lpmm_oracle_de_map(4, 1, 0, Tde);
    lpmm_oracle_linear_map(4, Tlin);

    /* decompress: m block-wise; v with the scale field M_i = min_r mu_r[Phi(i)_r] of the stored statistics */
    lpmm_oracle_unpack4(m_codes, numel, q);
    lpmm_oracle_dequantize_block(q, numel, m_block, Tde, m_scale, m);
    lpmm_oracle_unpack4(v_codes, numel, q);
    lpmm_oracle_rank1_scale_field(ndim, dims, mu_flat, M);
    for (int64_t i = 0; i < numel; ++i) v[i] = Tlin[q[i]] * M[i];

    /* Eq. 1 with the decoupled decay, operation by operation as in lpmm_oracle_adamw4_step */
    for (int64_t i = 0; i < numel; ++i) {
        float gi = g[i];
        float a = beta1 * m[i];
        float b = omb1 * gi;
        float mt = a + b;
        float gg = gi * gi;
        float c = beta2 * v[i];
        float d = omb2 * gg;
        float vt = c + d;
        float mhat = mt / bc1;
        float vhat = vt / bc2;
        float denom = sqrtf(vhat) + h->eps;
        float ratio = mhat / denom;
        float upd = h->lr * ratio;
        float wd = w[i] * decay;
        w[i] = wd - upd;
        m[i] = mt;
        v[i] = vt;
    }

    /* compress: new per-axis maxima (Alg. 4, first loop), their scale field (second loop), nearest codes */
    lpmm_oracle_quantize_block(m, numel, m_block, Tde, 16, 0, h->true_division, m_scale, q);
    lpmm_oracle_pack4(q, numel, m_codes);
    lpmm_oracle_rank1_stats(v, ndim, dims, mu_flat);
    lpmm_oracle_rank1_scale_field(ndim, dims, mu_flat, M);
    lpmm_oracle_map_codes(v, M, numel, Tlin, 16, h->true_division, q);
    lpmm_oracle_pack4(q, numel, v_codes);
    free(m); free(v); free(M); free(q);
    return 0;
}

/* ------------------------------------------------------------------ factorized second moment (Sec. 4.3) */

int lpmm_oracle_adamw4_factor_step(float* w, const float* g, int64_t rows, int64_t cols, int64_t m_block,
                                   uint8_t* m_codes, float* m_scale, float* R, float* C,
                                   const lpmm_oracle_hyper* h) {
    if (!w || !g || !h || !R || !C || rows <= 0 || cols <= 0 || h->step < 1) return -1;
    const int64_t numel = rows * cols;
    const float beta1 = h->beta1, beta2 = h->beta2;
    const float omb1 = 1.0f - beta1, omb2 = 1.0f - beta2;
    const float bc1 = (float)(1.0 - pow((double)beta1, (double)h->step));
    const float bc2 = (float)(1.0 - pow((double)beta2, (double)h->step));
    const float decay = 1.0f - h->lr * h->weight_decay;
    float* m = (float*)malloc(sizeof(float) * (size_t)numel);
    uint8_t* q = (uint8_t*)malloc((size_t)numel);
    double* cs = (double*)calloc((size_t)cols, sizeof(double));
    if (!m || !q || !cs) { free(m); free(q); free(cs); return -1; }
    float Tde[16];
    lpmm_oracle_de_map(4, 1, 0, Tde);
    lpmm_oracle_unpack4(m_codes, numel, q);
    lpmm_oracle_dequantize_block(q, numel, m_block, Tde, m_scale, m);

    /* row and column sums of the squared gradient, then the statistics' moving averages */
    for (int64_t i = 0; i < rows; ++i) {
        double rs = 0.0;
        for (int64_t j = 0; j < cols; ++j) {
            float gg = g[i * cols + j] * g[i * cols + j];
            rs += (double)gg;
            cs[j] += (double)gg;
        }
        float a = beta2 * R[i];
        float b = omb2 * (float)rs;
        R[i] = a + b;
    }
    double total = 0.0;
    for (int64_t i = 0; i < rows; ++i) total += (double)R[i];
    for (int64_t j = 0; j < cols; ++j) {
        float a = beta2 * C[j];
        float b = omb2 * (float)cs[j];
        C[j] = a + b;
    }
    const float rS = lpmm_oracle_rcp((float)total);

#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        const float ai = R[i] * rS;
        for (int64_t j = 0; j < cols; ++j) {
            const int64_t e = i * cols + j;
            float gi = g[e];
            float x = beta1 * m[e];
            float y = omb1 * gi;
            float mt = x + y;
            float vt = ai * C[j];
            float mhat = mt / bc1;
            float vhat = vt / bc2;
            float denom = sqrtf(vhat) + h->eps;
            float upd = h->lr * (mhat / denom);
            float wd = w[e] * decay;
            w[e] = wd - upd;
            m[e] = mt;
        }
    }
    lpmm_oracle_quantize_block(m, numel, m_block, Tde, 16, 0, h->true_division, m_scale, q);
    lpmm_oracle_pack4(q, numel, m_codes);
    free(m); free(q); free(cs);
    return 0;
}

/* ------------------------------------------------------------------ the compressed SGDM step (Alg. 2) */

int lpmm_oracle_sgdm4_step(float* w, const float* g, int64_t numel, int quantized, int64_t m_block,
                           uint8_t* m_codes, float* m_scale, float* m32, float lr, float beta, int true_division) {
    if (!w || !g || numel <= 0) return -1;
    float* m = (float*)malloc(sizeof(float) * (size_t)numel);
    if (!m) return -1;
    float Tde[16];
    lpmm_oracle_de_map(4, 1, 0, Tde);
    uint8_t* q = NULL;
    if (quantized) {                                   /* line 3: decompress */
        q = (uint8_t*)malloc((size_t)numel);
        if (!q) { free(m); return -1; }
        lpmm_oracle_unpack4(m_codes, numel, q);
        lpmm_oracle_dequantize_block(q, numel, m_block, Tde, m_scale, m);
    } else {
        memcpy(m, m32, sizeof(float) * (size_t)numel);
    }
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < numel; ++i) {
        float a = beta * m[i];
        float mt = a + g[i];                           /* line 4 */
        float upd = lr * mt;
        w[i] = w[i] - upd;                             /* line 5 */
        m[i] = mt;
    }
    if (quantized) {                                   /* line 6: compress */
        lpmm_oracle_quantize_block(m, numel, m_block, Tde, 16, 0, true_division, m_scale, q);
        lpmm_oracle_pack4(q, numel, m_codes);
        free(q);
    } else {
        memcpy(m32, m, sizeof(float) * (size_t)numel);
    }
    free(m);
    return 0;
}

int lpmm_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void lpmm_oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
