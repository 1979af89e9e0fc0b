/*
 * nvfp4_oracle.c -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, obviously-correct CPU statement of the NVFP4 linear layer
 * (activation / weight quantizer, block-scaled FP4 matmul, BF16 matmul) that the
 * CUDA library is checked against.  Only tests, the smoke check and the CPU
 * baseline leg of the benchmark may call it.  It shares no code, table or helper
 * with the CUDA path.
 *
 * What the paper fixes (Section 2, "FP4 Quantization and Hardware Acceleration"):
 *   - an FP4 element has 1 sign, 2 exponent and 1 mantissa bit (E2M1);
 *   - NVFP4 groups 16 contiguous elements under one E4M3 scale;
 *   - quantization is  x~ = Q(x) = S * Pi_FP4(x / S)  with a shared scale S and a
 *     projection Pi_FP4 onto the FP4 grid.
 * Everything the paper leaves open (E2M1 bias/subnormal, which E4M3, the second
 * level FP32 per-tensor scale T, rounding rules, FP32 operation order, zero
 * handling, nibble order) follows the readings listed in the design notes; they
 * are restated next to each function below.
 *
 * Quantizer = an ENCODING, so the oracle takes the steps in order, in IEEE
 * binary32 with round-to-nearest-even and no contraction (build with
 * -ffp-contract=off, never -ffast-math).  The matmuls have a plain definition
 * (real-number sum of products of the dequantized operands, plus bias), written
 * out in FP64 with no blocking or reordering.
 *
 * Pins (tests/test_oracle_*.py): closed-form tables, exhaustive E2M1/E4M3
 * rounding against an exact-rational brute force written separately in Python,
 * hand-worked block, exact round trips, metamorphic invariants, integer-exact
 * tiny matmuls; for the adapter merge: integer-exact cases, agreement with an FP64 library
 * product up to the last BF16 place, two hand-worked cases that fix the order and the
 * single rounding of the final multiply-add.  Not pinned: byte-for-byte agreement with NVIDIA Transformer
 * Engine's quantizer (the paper's backend; not available) -- "parity with
 * Transformer Engine unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ scalar formats */

/* BF16 is the upper half of an IEEE binary32. */
float oracle_bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* One rounding, FP64 -> BF16, nearest-even (finite inputs).  Done directly on the
 * double so that no intermediate FP32 rounding happens. */
uint16_t oracle_f64_to_bf16(double y) {
    uint16_t sign = (uint16_t)(signbit(y) ? 0x8000u : 0u);
    double a = fabs(y);
    if (a == 0.0) return sign;
    int e;
    (void)frexp(a, &e);          /* a = f * 2^e, f in [0.5, 1)  ->  a in [2^(e-1), 2^e) */
    int ex = e - 1;              /* floor(log2 a) */
    if (ex < -126) ex = -126;    /* subnormal range shares the quantum of the lowest binade */
    double quantum = ldexp(1.0, ex - 7);         /* 8 significant bits */
    double r = nearbyint(a / quantum) * quantum; /* default rounding mode: nearest-even */
    if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80u); /* overflow -> inf */
    float f = (float)r;          /* exact: r has at most 8 significant bits */
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return (uint16_t)(sign | (uint16_t)(u >> 16));
}

/* E2M1 (paper Section 2: 1 sign, 2 exponent, 1 mantissa bit).  Reading: bias 1,
 * subnormal at exponent field 0, no Inf/NaN.  Code = s e e m. */
double oracle_e2m1_decode(uint8_t code) {
    int s = (code >> 3) & 1, e = (code >> 1) & 3, m = code & 1;
    double mag = (e == 0) ? 0.5 * m : ldexp(1.0 + 0.5 * m, e - 1);
    return s ? -mag : mag;
}

/* The decode closed forms above, tabulated once (a speed-up of the table lookup
 * only; the values are those the closed forms give). */
double oracle_e4m3_decode(uint8_t code);
static double e2m1_tab[8];
static double e4m3_tab[127];
static int tabs_ready = 0;
static void fill_tabs(void) {
    if (tabs_ready) return;
    for (int c = 0; c < 8; ++c) e2m1_tab[c] = oracle_e2m1_decode((uint8_t)c);
    for (int c = 0; c < 127; ++c) e4m3_tab[c] = oracle_e4m3_decode((uint8_t)c);
    tabs_ready = 1;
}
__attribute__((constructor)) static void oracle_init(void) { fill_tabs(); }

/* Projection Pi_FP4: nearest grid value; a tie goes to the even code; anything
 * beyond the largest magnitude saturates to it; the sign bit is the input's. */
uint8_t oracle_e2m1_encode(float y) {
    double a = fabs((double)y);
    if (a >= e2m1_tab[7]) return (uint8_t)((signbit(y) ? 8 : 0) | 7); /* saturate */
    int best = 0;
    double best_d = fabs(a - e2m1_tab[0]);
    for (int c = 1; c < 8; ++c) {
        double d = fabs(a - e2m1_tab[c]);
        if (d < best_d || (d == best_d && (c & 1) == 0)) {
            best = c;
            best_d = d;
        }
    }
    return (uint8_t)((signbit(y) ? 8 : 0) | best);
}

/* FP8 E4M3 in the "fn" variant: bias 7, subnormal m*2^-9, max 448 (0x7E), no Inf,
 * 0x7F is NaN.  Used unsigned for block scales. */
double oracle_e4m3_decode(uint8_t code) {
    int e = (code >> 3) & 15, m = code & 7;
    double mag = (e == 0) ? ldexp((double)m, -9) : ldexp(1.0 + m / 8.0, e - 7);
    return (code & 0x80) ? -mag : mag;
}

/* Non-negative finite v -> nearest of the 127 finite codes 0x00..0x7E, a tie goes
 * to the even mantissa (= even code); above 448 saturates to 0x7E. */
uint8_t oracle_e4m3_encode(float v) {
    double a = (double)v;
    if (a >= 448.0) return 0x7E;
    int best = 0;
    double best_d = a;
    for (int c = 1; c <= 0x7E; ++c) {
        double d = fabs(a - e4m3_tab[c]);
        if (d < best_d || (d == best_d && (c & 1) == 0)) {
            best = c;
            best_d = d;
        }
    }
    return (uint8_t)best;
}

/* ------------------------------------------------------------------ quantizer */

/* Second-level per-tensor scale (not in the paper; the reading is
 * T = amax / (6 * 448) so block scales span E4M3's range; T = 1 for a zero tensor). */
float oracle_tensor_scale(const uint16_t *x, int64_t rows, int64_t K, int64_t ld) {
    float amax = 0.0f;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            float a = fabsf(oracle_bf16_to_f32(x[r * ld + k]));
            if (a > amax) amax = a;
        }
    if (amax == 0.0f) return 1.0f;
    return amax / 2688.0f;
}

/* Q(x) of Section 2 with S = s_block * T, per 16 contiguous elements along K:
 *   a   = max |x| over the block
 *   v   = a / (6*T)                       (binary32 division)
 *   sb  = E4M3(v)                         (nearest-even, saturating; one byte)
 *   d   = float(sb) * T;  rcp = 1/d       (binary32; rcp = 0 when sb == 0)
 *   y_k = x_k * rcp;  code_k = E2M1(y_k)
 * Outputs: q[r][j] = code(x[r][2j]) | code(x[r][2j+1]) << 4   (rows x K/2 bytes)
 *          sf[r][b] = sb                                     (rows x K/16 bytes, row major) */
void oracle_nvfp4_quantize(const uint16_t *x, int64_t rows, int64_t K, int64_t ld, float T,
                           uint8_t *q, uint8_t *sf) {
    const int64_t nb = K / 16;
    const float c = 6.0f * T;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t b = 0; b < nb; ++b) {
            const uint16_t *xb = x + r * ld + b * 16;
            float a = 0.0f;
            for (int k = 0; k < 16; ++k) {
                float t = fabsf(oracle_bf16_to_f32(xb[k]));
                if (t > a) a = t;
            }
            float v = a / c;
            uint8_t sb = oracle_e4m3_encode(v);
            float d = (float)oracle_e4m3_decode(sb) * T;
            float rcp = (sb == 0) ? 0.0f : 1.0f / d;
            sf[r * nb + b] = sb;
            for (int j = 0; j < 8; ++j) {
                float y0 = oracle_bf16_to_f32(xb[2 * j]) * rcp;
                float y1 = oracle_bf16_to_f32(xb[2 * j + 1]) * rcp;
                q[r * (K / 2) + b * 8 + j] =
                    (uint8_t)(oracle_e2m1_encode(y0) | (oracle_e2m1_encode(y1) << 4));
            }
        }
    }
}

/* Byte offset of the scale of (row r, block kb) in the 128x4-chunked storage the
 * tensor core consumes: 512-byte chunks of 128 rows x 4 blocks, chunk order
 * [row tile][k chunk]; inside a chunk 32 lines of 16 bytes. */
int64_t oracle_sf_swizzled_offset(int64_t r, int64_t kb, int64_t K) {
    int64_t chunks_k = (K / 16 + 3) / 4;
    int64_t chunk = (r / 128) * chunks_k + kb / 4;
    int64_t rr = r % 128;
    return chunk * 512 + (rr % 32) * 16 + (rr / 32) * 4 + kb % 4;
}

int64_t oracle_sf_swizzled_bytes(int64_t rows, int64_t K) {
    return ((rows + 127) / 128) * ((K / 16 + 3) / 4) * 512;
}

/* Row-major scales -> chunked storage; padding bytes are zero. */
void oracle_sf_swizzle(const uint8_t *sf, int64_t rows, int64_t K, uint8_t *out) {
    memset(out, 0, (size_t)oracle_sf_swizzled_bytes(rows, K));
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t b = 0; b < K / 16; ++b)
            out[oracle_sf_swizzled_offset(r, b, K)] = sf[r * (K / 16) + b];
}

/* x^ = E2M1(code) * E4M3(sb) * T, in FP64 (every factor is exact in FP64). */
void oracle_nvfp4_dequantize(const uint8_t *q, const uint8_t *sf, float T, int64_t rows, int64_t K,
                             double *out) {
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            uint8_t byte = q[r * (K / 2) + k / 2];
            uint8_t code = (k & 1) ? (uint8_t)(byte >> 4) : (uint8_t)(byte & 0xF);
            out[r * K + k] =
                oracle_e2m1_decode(code) * oracle_e4m3_decode(sf[r * (K / 16) + k / 16]) * (double)T;
        }
}

/* ------------------------------------------------------------------ matmuls */

/* Y[i][n] = sum_k A[i][k] * B[n][k] + bias[n], FP64, k ascending, for the rows given. */
static void matmul_nt_f64(const double *A, const double *B, const uint16_t *bias, int64_t n_rows,
                          int64_t N, int64_t K, double *Y) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t i = 0; i < n_rows; ++i)
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) acc += A[i * K + k] * B[n * K + k];
            if (bias) acc += (double)oracle_bf16_to_f32(bias[n]);
            Y[i * N + n] = acc;
        }
}

/* NVFP4 linear: Y = dequant(X) . dequant(W)^T + bias for the selected rows of X.
 * q_x/sf_x are [M][K/2], [M][K/16] row-major; q_w/sf_w are [N][K/2], [N][K/16].
 * row_idx == NULL means rows 0..n_rows-1.  Y is [n_rows][N] FP64.  Returns 0, or 1
 * if memory for the dequantized operands could not be had. */
int oracle_nvfp4_linear(const uint8_t *q_x, const uint8_t *sf_x, float T_x, const uint8_t *q_w,
                        const uint8_t *sf_w, float T_w, const uint16_t *bias, int64_t N, int64_t K,
                        const int64_t *row_idx, int64_t n_rows, double *Y) {
    double *A = (double *)malloc(sizeof(double) * (size_t)n_rows * (size_t)K);
    double *B = (double *)malloc(sizeof(double) * (size_t)N * (size_t)K);
    if (!A || !B) {
        free(A);
        free(B);
        return 1;
    }
    for (int64_t i = 0; i < n_rows; ++i) {
        int64_t r = row_idx ? row_idx[i] : i;
        oracle_nvfp4_dequantize(q_x + r * (K / 2), sf_x + r * (K / 16), T_x, 1, K, A + i * K);
    }
    oracle_nvfp4_dequantize(q_w, sf_w, T_w, N, K, B);
    matmul_nt_f64(A, B, bias, n_rows, N, K, Y);
    free(A);
    free(B);
    return 0;
}

/* BF16 linear: Y = X . W^T + bias on the raw BF16 values (exact in FP64). */
int oracle_bf16_linear(const uint16_t *x, int64_t ldx, const uint16_t *w, int64_t ldw,
                       const uint16_t *bias, int64_t N, int64_t K, const int64_t *row_idx,
                       int64_t n_rows, double *Y) {
    double *A = (double *)malloc(sizeof(double) * (size_t)n_rows * (size_t)K);
    double *B = (double *)malloc(sizeof(double) * (size_t)N * (size_t)K);
    if (!A || !B) {
        free(A);
        free(B);
        return 1;
    }
    for (int64_t i = 0; i < n_rows; ++i) {
        int64_t r = row_idx ? row_idx[i] : i;
        for (int64_t k = 0; k < K; ++k) A[i * K + k] = (double)oracle_bf16_to_f32(x[r * ldx + k]);
    }
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) B[n * K + k] = (double)oracle_bf16_to_f32(w[n * ldw + k]);
    matmul_nt_f64(A, B, bias, n_rows, N, K, Y);
    free(A);
    free(B);
    return 0;
}

/* ------------------------------------------------------------------ MXFP4 (the other FP4 format of Section 2) */

/* Section 2 names two block formats: NVFP4 above, and OCP MXFP4 -- 32 elements under one E8M0
 * scale.  E8M0 is a bare biased exponent: byte b stands for 2^(b - 127) (0xFF is NaN, unused).
 * Q(x) = S * Pi_FP4(x / S) with S a power of two and no tensor-level scale.  The reading taken for
 * the scale is the OCP Microscaling rule: shared exponent = floor(log2(max|x|)) - 2 (2 = the
 * exponent of E2M1's largest value 6 = 1.5 * 2^2), clamped to [-127, 127]; a block maximum in
 * [4S, 8S) therefore has elements above 6S, which saturate.  Pi_FP4 is the same nearest-even,
 * saturating projection as for NVFP4; x / S is exact (a power-of-two scaling). */
double oracle_e8m0_decode(uint8_t b) { return ldexp(1.0, (int)b - 127); }

void oracle_mxfp4_quantize(const uint16_t *x, int64_t rows, int64_t K, int64_t ld, uint8_t *q, uint8_t *sf) {
    const int64_t nb = K / 32;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t b = 0; b < nb; ++b) {
            const uint16_t *xb = x + r * ld + b * 32;
            double a = 0.0;
            for (int k = 0; k < 32; ++k) {
                double t = fabs((double)oracle_bf16_to_f32(xb[k]));
                if (t > a) a = t;
            }
            int se = -127;
            if (a > 0.0) {
                int e;
                (void)frexp(a, &e);      /* a in [2^(e-1), 2^e)  ->  floor(log2 a) = e - 1 */
                se = (e - 1) - 2;
                if (se < -127) se = -127;
                if (se > 127) se = 127;
            }
            sf[r * nb + b] = (uint8_t)(se + 127);
            for (int j = 0; j < 16; ++j) {
                float y0 = (float)ldexp((double)oracle_bf16_to_f32(xb[2 * j]), -se);
                float y1 = (float)ldexp((double)oracle_bf16_to_f32(xb[2 * j + 1]), -se);
                q[r * (K / 2) + b * 16 + j] = (uint8_t)(oracle_e2m1_encode(y0) | (oracle_e2m1_encode(y1) << 4));
            }
        }
    }
}

/* The same 512-byte chunks of 128 rows x 4 scales as for NVFP4; a chunk now spans 128 elements of K. */
int64_t oracle_mx_sf_swizzled_offset(int64_t r, int64_t kb, int64_t K) {
    int64_t chunks_k = (K / 32 + 3) / 4;
    int64_t chunk = (r / 128) * chunks_k + kb / 4;
    int64_t rr = r % 128;
    return chunk * 512 + (rr % 32) * 16 + (rr / 32) * 4 + kb % 4;
}

int64_t oracle_mx_sf_swizzled_bytes(int64_t rows, int64_t K) {
    return ((rows + 127) / 128) * ((K / 32 + 3) / 4) * 512;
}

void oracle_mx_sf_swizzle(const uint8_t *sf, int64_t rows, int64_t K, uint8_t *out) {
    memset(out, 0, (size_t)oracle_mx_sf_swizzled_bytes(rows, K));
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t b = 0; b < K / 32; ++b)
            out[oracle_mx_sf_swizzled_offset(r, b, K)] = sf[r * (K / 32) + b];
}

void oracle_mxfp4_dequantize(const uint8_t *q, const uint8_t *sf, int64_t rows, int64_t K, double *out) {
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t k = 0; k < K; ++k) {
            uint8_t byte = q[r * (K / 2) + k / 2];
            uint8_t code = (k & 1) ? (uint8_t)(byte >> 4) : (uint8_t)(byte & 0xF);
            out[r * K + k] = oracle_e2m1_decode(code) * oracle_e8m0_decode(sf[r * (K / 32) + k / 32]);
        }
}

static void matmul_nt_f64(const double *A, const double *B, const uint16_t *bias, int64_t n_rows, int64_t N,
                          int64_t K, double *Y);

/* MXFP4 linear: Y = dequant(X) . dequant(W)^T + bias in FP64 for the selected rows of X. */
int oracle_mxfp4_linear(const uint8_t *q_x, const uint8_t *sf_x, const uint8_t *q_w, const uint8_t *sf_w,
                        const uint16_t *bias, int64_t N, int64_t K, const int64_t *row_idx, int64_t n_rows,
                        double *Y) {
    double *A = (double *)malloc(sizeof(double) * (size_t)n_rows * (size_t)K);
    double *B = (double *)malloc(sizeof(double) * (size_t)N * (size_t)K);
    if (!A || !B) {
        free(A);
        free(B);
        return 1;
    }
    for (int64_t i = 0; i < n_rows; ++i) {
        int64_t r = row_idx ? row_idx[i] : i;
        oracle_mxfp4_dequantize(q_x + r * (K / 2), sf_x + r * (K / 32), 1, K, A + i * K);
    }
    oracle_mxfp4_dequantize(q_w, sf_w, N, K, B);
    matmul_nt_f64(A, B, bias, n_rows, N, K, Y);
    free(A);
    free(B);
    return 0;
}

/* ------------------------------------------------------------------ activation between two linears */

/* GELU in its tanh form, the activation of the DiT feed-forward blocks whose linears the rollout
 * runs in NVFP4 (the paper does not restate it):
 *     gelu(x) = x/2 * (1 + tanh( sqrt(2/pi) * (x + 0.044715 x^3) )),   evaluated in FP64. */
double oracle_gelu_tanh(double x) {
    const double c = 0.79788456080286535588;  /* sqrt(2/pi) */
    return 0.5 * x * (1.0 + tanh(c * (x + 0.044715 * x * x * x)));
}

void oracle_gelu_tanh_array(const double *x, int64_t n, double *out) {
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_gelu_tanh(x[i]);
}

/* Adaptive layer norm in front of a DiT linear (the producer of most quantized activations; the
 * paper does not restate it): per row, with no learned affine,
 *     mu = mean(x),  var = mean((x - mu)^2),  xhat = (x - mu) / sqrt(var + eps),
 *     y[k] = xhat[k] * (1 + scale[s][k]) + shift[s][k],      s = row / rows_per_sample,
 * evaluated in FP64 on the BF16 inputs.  x [rows, K] pitch ld; scale, shift [samples, K] dense. */
void oracle_layernorm_modulate(const uint16_t *x, int64_t rows, int64_t K, int64_t ld, const uint16_t *scale,
                               const uint16_t *shift, int64_t rows_per_sample, double eps, double *out) {
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        const uint16_t *xr = x + r * ld;
        const int64_t s = r / rows_per_sample;
        double mu = 0.0;
        for (int64_t k = 0; k < K; ++k) mu += (double)oracle_bf16_to_f32(xr[k]);
        mu /= (double)K;
        double var = 0.0;
        for (int64_t k = 0; k < K; ++k) {
            double d = (double)oracle_bf16_to_f32(xr[k]) - mu;
            var += d * d;
        }
        var /= (double)K;
        const double inv = 1.0 / sqrt(var + eps);
        for (int64_t k = 0; k < K; ++k) {
            double xh = ((double)oracle_bf16_to_f32(xr[k]) - mu) * inv;
            out[r * K + k] = xh * (1.0 + (double)oracle_bf16_to_f32(scale[s * K + k])) +
                             (double)oracle_bf16_to_f32(shift[s * K + k]);
        }
    }
}

/* ------------------------------------------------------------------ weight refresh (LoRA merge) */

/* The policy is trained through rank-r adapters (Section 4.1: r = 32, alpha = 64) and its
 * weights are re-quantized into the NVFP4 engine after every update (Section 3.4,
 * Appendix B.2).  The paper does not say how the adapters reach the engine; the reading taken
 * here is the usual merge
 *     W'[n][k] = W[n][k] + s * sum_j B[n][j] * A[j][k],      s = alpha / r,
 * with W [N, K], A [r, K] ("down"), B [N, r] ("up") in BF16 and W' rounded to BF16, after
 * which W' goes through the weight quantizer above.  Because W' decides quantized codes, its
 * arithmetic is fixed as a sequence in IEEE binary32:
 *     acc = 0;  for j = 0 .. r-1 in this order:  acc = fma(B[n][j], A[j][k], acc)
 *     W'  = bf16_rne( fma(s, acc, W[n][k]) )
 * (each fma rounds once; the BF16 products are exact in binary32).  `out` is dense [N, K]. */
void oracle_lora_merge(const uint16_t *w, int64_t ldw, const uint16_t *a, int64_t lda, const uint16_t *b,
                       int64_t ldb, int64_t N, int64_t K, int64_t r, float s, uint16_t *out) {
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) {
            float acc = 0.0f;
            for (int64_t j = 0; j < r; ++j)
                acc = fmaf(oracle_bf16_to_f32(b[n * ldb + j]), oracle_bf16_to_f32(a[j * lda + k]), acc);
            const float merged = fmaf(s, acc, oracle_bf16_to_f32(w[n * ldw + k]));
            out[n * K + k] = oracle_f64_to_bf16((double)merged);  /* widening is exact: one rounding */
        }
}

void oracle_f64_to_bf16_array(const double *y, int64_t n, uint16_t *out) {
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_f64_to_bf16(y[i]);
}

/* Threads the row-parallel loops above actually use. */
int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
