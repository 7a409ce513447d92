/*
 * QuEST quantized-linear forward -- CPU ORACLE.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what the
 * method computes, written from the paper.  Only the test-suite, the smoke check and
 * the benchmark's cpu_baseline / reference legs may build, load or call it.  It shares
 * no code, header, table or helper with the CUDA library and never calls it.
 *
 * What it computes, per row x of length d (Algorithm 1: rotation, projection and product):
 *   1. x_h = HT(x)           Hadamard rotation along the matmul dimension (Eq. 2):
 *                            block-diagonal Sylvester-Hadamard H_g on contiguous blocks
 *                            of g elements, kept UN-normalised (u = H_g * block); the
 *                            orthonormal transform is u / sqrt(g).
 *   2. RMS normalisation     r = sqrt(mean(u^2)) over the whole row (Section 3.1,
 *                            "Gaussian Fitting").
 *   3. clip + round          onto the b-bit zero-free uniform grid of Eq. 1, clipping at
 *                            alpha*(b) * RMS (Section 3.1); level index k in [0, 2^b-1],
 *                            grid value c = 2k - (2^b-1) in units of the half step.
 *   4. trust mask            M = [ |x_h - xq_h| <= trust_factor * alpha* * RMS / (2^b-1) ]
 *                            (Section 3.2; the factor s of "The 1-bit Case").
 *   5. y = xq_h wq_h^T       integer contraction of the grid values, then the product of
 *                            the two per-row scales (the product step of Algorithm 1).
 *
 * Arithmetic: the paper fixes no precision.  Rounding decisions (codes, masks) are taken
 * in IEEE binary32 with one rounding per operation in a fixed order, stated at each step,
 * so that a GPU implementation can reproduce them bit for bit.  Everything that is only
 * tolerance-checked (dequantised outputs) is computed in binary64.
 *
 * Readings of the paper where it is silent are marked "READING".
 *
 * Pins (see tests/test_oracle_*.py): H H^T = g I, Parseval, involution; alpha*(b) against a
 * brute-force minimisation of the Gaussian quantisation MSE; codes against an exhaustive
 * nearest-grid-point search in binary64; masks against the inequality in binary64; the
 * integer contraction against numpy int64 matmul.  The tie-break (half to even), the
 * bit order inside a byte, the zero-row rule and the reading of trust_factor are
 * PARITY UNPINNED by the paper: they are pinned only by the stated reading.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -fno-fast-math -shared -fPIC.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define QO_OK 0
#define QO_BAD_ARG 1
#define QO_OVERFLOW 2

/* alpha*(b), b = 1..8: the minimiser of E (xi - alpha*round(clip(xi,alpha)/alpha))^2 for
 * xi ~ N(0,1) on the 2^b-point grid (Section 3.1).  Frozen binary32 values; re-derived by
 * brute force in tests/test_oracle_alpha.py. */
static const float QO_ALPHA_STAR[9] = {
    0.0f,
    0.7978846f,  /* b=1: sqrt(2/pi) */
    1.4935300f,  /* b=2 */
    2.0510680f,  /* b=3 */
    2.5140045f,  /* b=4 */
    2.9161513f,  /* b=5 */
    3.2779846f,  /* b=6 */
    3.6110970f,  /* b=7 */
    3.9222038f,  /* b=8 */
};

float qo_alpha_star(int bits) {
    if (bits < 1 || bits > 8) return 0.0f;
    return QO_ALPHA_STAR[bits];
}

/* READING: storage container per code: 1, 2, 4, 4, 8, 8, 8, 8 bits for b = 1..8
 * (the paper only says INT4 pairs are packed into UINT8, Section 5). */
int qo_container_bits(int bits) {
    if (bits == 1) return 1;
    if (bits == 2) return 2;
    if (bits <= 4) return 4;
    return 8;
}

static float bf16_to_f32(uint16_t h) {
    uint32_t w = (uint32_t)h << 16;
    float f;
    memcpy(&f, &w, 4);
    return f;
}

/* u = H_g * v, H_g[i][j] = (-1)^popcount(i & j) (Sylvester order), un-normalised.
 * READING (evaluation order): butterflies (a,b) -> (a+b, a-b), one binary32 rounding each,
 * stages in DESCENDING stride h = g/2, g/4, ..., 1. */
void qo_fwht_block(float *v, int g) {
    for (int h = g / 2; h >= 1; h /= 2) {
        for (int i = 0; i < g; i += 2 * h) {
            for (int j = i; j < i + h; ++j) {
                float a = v[j];
                float b = v[j + h];
                v[j] = a + b;
                v[j + h] = a - b;
            }
        }
    }
}

/* Sum of squares of a row in binary32.
 * READING (evaluation order): squares rounded to binary32, then pairwise summation over
 * ADJACENT elements (0+1, 2+3, ... then pairs of pairs ...) of the row padded with zeros
 * to the next power of two. */
static float sumsq_pairwise(const float *u, int64_t d, float *tmp, int64_t p2) {
    for (int64_t i = 0; i < d; ++i) tmp[i] = u[i] * u[i];
    for (int64_t i = d; i < p2; ++i) tmp[i] = 0.0f;
    for (int64_t n = p2; n > 1; n /= 2)
        for (int64_t i = 0; i < n / 2; ++i) tmp[i] = tmp[2 * i] + tmp[2 * i + 1];
    return tmp[0];
}

static int is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }

/*
 * Quantize every row of x [rows x cols], row stride ld elements.
 *   dtype: 0 = binary32, 1 = bfloat16 (widened exactly).
 *   codes: packed level indices, row stride cols*container/8 bytes, element e at bit
 *          offset (e mod (8/container))*container of its byte (element 0 lowest). Nullable.
 *   scales: per row, the half step of the grid in the ORTHONORMAL Hadamard domain:
 *          xq_h = scale * (2k - (2^b-1)).  Nullable.
 *   mask:  bitmap, element e at bit (e mod 8) of byte e/8, 1 = trusted.  Nullable.
 *   u_out: the un-normalised rotated row (binary32), [rows x cols] dense.  Nullable.
 *   t_out: the position on the level axis before rounding, [rows x cols].  Nullable.
 */
int qo_quantize(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                int bits, int had_block, float trust_factor,
                uint8_t *codes, float *scales, uint8_t *mask,
                float *u_out, float *t_out) {
    if (!x || rows < 0 || cols <= 0 || ld < cols) return QO_BAD_ARG;
    if (bits < 1 || bits > 8) return QO_BAD_ARG;
    if (!is_pow2(had_block) || cols % had_block != 0) return QO_BAD_ARG;
    if (dtype != 0 && dtype != 1) return QO_BAD_ARG;
    if (cols % 8 != 0) return QO_BAD_ARG;
    if (!(trust_factor >= 0.0f) || isinf(trust_factor)) return QO_BAD_ARG;

    const int L1 = (1 << bits) - 1;            /* 2^b - 1: number of steps across the grid */
    const float alpha = QO_ALPHA_STAR[bits];
    const float c0 = 0.5f * (float)L1;         /* level axis: t = x_n*(L1/(2 alpha)) + L1/2 */
    const float A = (float)L1 / (2.0f * alpha);
    const float B = alpha / ((float)L1 * sqrtf((float)had_block));
    const float h = 0.5f * trust_factor;       /* trust bound in units of one level step */
    const int cb = qo_container_bits(bits);
    const int64_t code_row_bytes = cols * cb / 8;
    const int64_t mask_row_bytes = cols / 8;
    int64_t p2 = 1;
    while (p2 < cols) p2 *= 2;

#pragma omp parallel
    {
        float *u = (float *)malloc(sizeof(float) * (size_t)cols);
        float *tmp = (float *)malloc(sizeof(float) * (size_t)p2);
#pragma omp for schedule(static)
        for (int64_t r = 0; r < rows; ++r) {
            /* Algorithm 1, rotation step (x_h = HT(x), w_h = HT(w)) */
            if (dtype == 0) {
                const float *xr = (const float *)x + r * ld;
                for (int64_t e = 0; e < cols; ++e) u[e] = xr[e];
            } else {
                const uint16_t *xr = (const uint16_t *)x + r * ld;
                for (int64_t e = 0; e < cols; ++e) u[e] = bf16_to_f32(xr[e]);
            }
            for (int64_t blk = 0; blk < cols; blk += had_block) qo_fwht_block(u + blk, had_block);

            /* RMS of the rotated row (un-normalised units) */
            const float ss = sumsq_pairwise(u, cols, tmp, p2);
            const float rms = sqrtf(ss / (float)cols);
            /* READING: a zero row has no scale; it gets inv = 0, scale = 0. */
            const float inv = (rms > 0.0f) ? (A / rms) : 0.0f;
            if (scales) scales[r] = rms * B;

            uint8_t *cr = codes ? codes + r * code_row_bytes : 0;
            uint8_t *mr = mask ? mask + r * mask_row_bytes : 0;
            if (cr) memset(cr, 0, (size_t)code_row_bytes);
            if (mr) memset(mr, 0, (size_t)mask_row_bytes);
            for (int64_t e = 0; e < cols; ++e) {
                /* Algorithm 1, projection step: clip to [-alpha*, alpha*] RMS and round to the nearest of the
                 * 2^b grid points; on the level axis the grid points are the integers
                 * 0..L1.  READING: ties go to the even level (rintf, default mode). */
                const float t = fmaf(u[e], inv, c0);
                const float tc = fminf(fmaxf(t, 0.0f), (float)L1);
                const float kf = rintf(tc);
                const int k = (int)kf;
                /* trust mask: |x_h - xq_h| <= trust_factor * (half step)  <=>
                 * |t - k| <= trust_factor / 2 on the level axis.  "<=": ties are trusted. */
                const int trusted = fabsf(t - kf) <= h;
                if (cr) {
                    const int per = 8 / cb;
                    cr[e / per] |= (uint8_t)(k << ((e % per) * cb));
                }
                if (mr && trusted) mr[e / 8] |= (uint8_t)(1u << (e % 8));
                if (t_out) t_out[r * cols + e] = t;
            }
            if (u_out) memcpy(u_out + r * cols, u, sizeof(float) * (size_t)cols);
        }
        free(u);
        free(tmp);
    }
    return QO_OK;
}

/* Grid values c = 2k - (2^b - 1) (odd integers) from packed level indices. */
int qo_unpack_grid_values(const uint8_t *codes, int64_t rows, int64_t cols, int bits, int16_t *c) {
    if (!codes || !c || bits < 1 || bits > 8) return QO_BAD_ARG;
    const int cb = qo_container_bits(bits);
    const int per = 8 / cb;
    const int L1 = (1 << bits) - 1;
    const int64_t row_bytes = cols * cb / 8;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t e = 0; e < cols; ++e) {
            const int k = (codes[r * row_bytes + e / per] >> ((e % per) * cb)) & ((1 << cb) - 1);
            c[r * cols + e] = (int16_t)(2 * k - L1);
        }
    return QO_OK;
}

/* Algorithm 1, product step, integer part: acc[i][j] = sum_k cx[i][k] * cw[j][k], exact.
 * Accumulated in 64 bits and checked to fit 32. */
int qo_gemm_acc(const uint8_t *xq, int bits_x, const uint8_t *wq, int bits_w,
                int64_t M, int64_t N, int64_t K, int32_t *acc) {
    if (!xq || !wq || !acc || M < 0 || N < 0 || K <= 0) return QO_BAD_ARG;
    int16_t *cx = (int16_t *)malloc(sizeof(int16_t) * (size_t)(M * K + 1));
    int16_t *cw = (int16_t *)malloc(sizeof(int16_t) * (size_t)(N * K + 1));
    int status = QO_OK;
    if (qo_unpack_grid_values(xq, M, K, bits_x, cx) || qo_unpack_grid_values(wq, N, K, bits_w, cw)) {
        free(cx); free(cw);
        return QO_BAD_ARG;
    }
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i) {
        for (int64_t j = 0; j < N; ++j) {
            int64_t s = 0;
            for (int64_t k = 0; k < K; ++k) s += (int32_t)cx[i * K + k] * (int32_t)cw[j * K + k];
            if (s > INT32_MAX || s < INT32_MIN) {
#pragma omp atomic write
                status = QO_OVERFLOW;
            }
            acc[i * N + j] = (int32_t)s;
        }
    }
    free(cx); free(cw);
    return status;
}

/* Algorithm 1, product step, scale part: y[i][j] = sx[i] * sw[j] * acc[i][j] in binary64. */
int qo_dequant(const int32_t *acc, const float *sx, const float *sw, int64_t M, int64_t N, double *y) {
    if (!acc || !sx || !sw || !y) return QO_BAD_ARG;
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j)
            y[i * N + j] = (double)sx[i] * (double)sw[j] * (double)acc[i * N + j];
    return QO_OK;
}

/*
 * Algorithm 1 end to end: quantize x rows and w rows with the same Hadamard block and
 * bit-width, contract, scale.  Every output is nullable except y.
 */
int qo_linear_fwd(const void *x, const void *w, int dtype, int64_t M, int64_t N, int64_t K,
                  int bits, int had_block, float trust_factor,
                  double *y, int32_t *acc_out,
                  uint8_t *xq, float *sx, uint8_t *mx,
                  uint8_t *wq, float *sw, uint8_t *mw) {
    if (!y) return QO_BAD_ARG;
    const int cb = qo_container_bits(bits);
    uint8_t *xq_ = xq ? xq : (uint8_t *)malloc((size_t)(M * K * cb / 8 + 1));
    uint8_t *wq_ = wq ? wq : (uint8_t *)malloc((size_t)(N * K * cb / 8 + 1));
    float *sx_ = sx ? sx : (float *)malloc(sizeof(float) * (size_t)(M + 1));
    float *sw_ = sw ? sw : (float *)malloc(sizeof(float) * (size_t)(N + 1));
    int32_t *acc = acc_out ? acc_out : (int32_t *)malloc(sizeof(int32_t) * (size_t)(M * N + 1));
    int st = qo_quantize(x, dtype, M, K, K, bits, had_block, trust_factor, xq_, sx_, mx, 0, 0);
    if (!st) st = qo_quantize(w, dtype, N, K, K, bits, had_block, trust_factor, wq_, sw_, mw, 0, 0);
    if (!st) st = qo_gemm_acc(xq_, bits, wq_, bits, M, N, K, acc);
    if (!st) st = qo_dequant(acc, sx_, sw_, M, N, y);
    if (!xq) free(xq_);
    if (!wq) free(wq_);
    if (!sx) free(sx_);
    if (!sw) free(sw_);
    if (!acc_out) free(acc);
    return st;
}

/* ------------------------------------------------------------------------------------------
 * FP4 variant (Section 4.4, "The FP4 Format"): the rounding of Eq. 1 is replaced by rounding to
 * the FP4 (E2M1) grid scaled to [-1, 1], alpha*_FP4 is the minimiser of the same Gaussian MSE with
 * that grid, and the trust bound is the largest half-interval of the grid.
 *
 * E2M1 values: +-{0, 0.5, 1, 1.5, 2, 3, 4, 6}; a code is sign << 3 | magnitude index.  On the value
 * axis t = x_h * 6 / (alpha* RMS) the grid points are the E2M1 values themselves, the largest
 * interval is [4, 6], so T = 1 in these units.
 * READING: ties between two neighbouring codes go to the even code (round-to-nearest-even of the
 * E2M1 encoding); values beyond +-6 saturate; the sign of a value that rounds to zero is kept in
 * the code (as a hardware conversion does).  PARITY UNPINNED by the paper.
 * ------------------------------------------------------------------------------------------ */
#define QO_ALPHA_STAR_FP4 2.9224751f

static const float QO_E2M1[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};

float qo_alpha_star_fp4(void) { return QO_ALPHA_STAR_FP4; }

static int e2m1_index(float a) { /* a >= 0; interval midpoints, ties to the even index */
    if (a <= 0.25f) return 0;
    if (a < 0.75f) return 1;
    if (a <= 1.25f) return 2;
    if (a < 1.75f) return 3;
    if (a <= 2.5f) return 4;
    if (a < 3.5f) return 5;
    if (a <= 5.0f) return 6;
    return 7;
}

/* The E2M1 code (sign << 3 | magnitude index) of a position t on the value axis. */
int qo_e2m1_code(float t) { return (signbit(t) ? 8 : 0) | e2m1_index(fabsf(t)); }

/* Same rotation, RMS and outputs as qo_quantize; codes are E2M1 nibbles (element 0 in the low
 * nibble), scales[r] = alpha*_FP4 RMS(x_h) / 6 so that xq_h = scale * E2M1 value. */
int qo_quantize_fp4(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                    int had_block, float trust_factor,
                    uint8_t *codes, float *scales, uint8_t *mask, float *t_out) {
    if (!x || rows < 0 || cols <= 0 || ld < cols) return QO_BAD_ARG;
    if (!is_pow2(had_block) || cols % had_block != 0) return QO_BAD_ARG;
    if (dtype != 0 && dtype != 1) return QO_BAD_ARG;
    if (cols % 8 != 0) return QO_BAD_ARG;
    if (!(trust_factor >= 0.0f) || isinf(trust_factor)) return QO_BAD_ARG;
    const float alpha = QO_ALPHA_STAR_FP4;
    const float A = 6.0f / alpha;                           /* RMS-normalised value -> E2M1 value axis */
    const float B = alpha / (6.0f * sqrtf((float)had_block));
    const float h = trust_factor;                           /* largest half-interval of the grid: 1 */
    int64_t p2 = 1;
    while (p2 < cols) p2 *= 2;
#pragma omp parallel
    {
        float *u = (float *)malloc(sizeof(float) * (size_t)cols);
        float *tmp = (float *)malloc(sizeof(float) * (size_t)p2);
#pragma omp for schedule(static)
        for (int64_t r = 0; r < rows; ++r) {
            if (dtype == 0) {
                const float *xr = (const float *)x + r * ld;
                for (int64_t e = 0; e < cols; ++e) u[e] = xr[e];
            } else {
                const uint16_t *xr = (const uint16_t *)x + r * ld;
                for (int64_t e = 0; e < cols; ++e) u[e] = bf16_to_f32(xr[e]);
            }
            for (int64_t blk = 0; blk < cols; blk += had_block) qo_fwht_block(u + blk, had_block);
            const float ss = sumsq_pairwise(u, cols, tmp, p2);
            const float rms = sqrtf(ss / (float)cols);
            const float inv = (rms > 0.0f) ? (A / rms) : 0.0f;
            if (scales) scales[r] = rms * B;
            uint8_t *cr = codes ? codes + r * (cols / 2) : 0;
            uint8_t *mr = mask ? mask + r * (cols / 8) : 0;
            if (cr) memset(cr, 0, (size_t)(cols / 2));
            if (mr) memset(mr, 0, (size_t)(cols / 8));
            for (int64_t e = 0; e < cols; ++e) {
                const float t = u[e] * inv;
                const int code = qo_e2m1_code(t);
                const int m = code & 7;
                const float v = signbit(t) ? -QO_E2M1[m] : QO_E2M1[m];
                const int trusted = fabsf(t - v) <= h;
                if (cr) cr[e / 2] |= (uint8_t)(code << ((e % 2) * 4));
                if (mr && trusted) mr[e / 8] |= (uint8_t)(1u << (e % 8));
                if (t_out) t_out[r * cols + e] = t;
            }
        }
        free(u);
        free(tmp);
    }
    return QO_OK;
}

/* Twice the E2M1 value of every code (an integer in [-12, 12]). */
int qo_unpack_fp4_twice(const uint8_t *codes, int64_t rows, int64_t cols, int16_t *c2) {
    if (!codes || !c2) return QO_BAD_ARG;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t e = 0; e < cols; ++e) {
            const int code = (codes[r * (cols / 2) + e / 2] >> ((e % 2) * 4)) & 15;
            const int two_v = (int)(2.0f * QO_E2M1[code & 7]);
            c2[r * cols + e] = (int16_t)((code & 8) ? -two_v : two_v);
        }
    return QO_OK;
}

/* acc4[i][j] = sum_k (2 v_x[i][k]) (2 v_w[j][k]) = 4 * (xq_h wq_h^T)[i][j] / (sx[i] sw[j]), exact. */
int qo_gemm_acc_fp4(const uint8_t *xq, const uint8_t *wq, int64_t M, int64_t N, int64_t K, int32_t *acc4) {
    if (!xq || !wq || !acc4 || M < 0 || N < 0 || K <= 0) return QO_BAD_ARG;
    int16_t *cx = (int16_t *)malloc(sizeof(int16_t) * (size_t)(M * K + 1));
    int16_t *cw = (int16_t *)malloc(sizeof(int16_t) * (size_t)(N * K + 1));
    qo_unpack_fp4_twice(xq, M, K, cx);
    qo_unpack_fp4_twice(wq, N, K, cw);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j) {
            int64_t s = 0;
            for (int64_t k = 0; k < K; ++k) s += (int32_t)cx[i * K + k] * (int32_t)cw[j * K + k];
            acc4[i * N + j] = (int32_t)s;
        }
    free(cx);
    free(cw);
    return QO_OK;
}
