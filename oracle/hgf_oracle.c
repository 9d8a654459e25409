/*
 * CPU oracle for the forward pass of the Hybrid Gated Flow (HGF) dual-stream linear layer.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, scalar restatement of the
 * paper's definitions (Section 2.2 "Ternary Weight Quantization", Section 2.2.1 "Activation
 * Quantization", Section 2.3 "Gated Low-Rank Correction", Algorithm 1 "HGF 1.0 Forward Pass").
 * Only the tests, the smoke check and the benchmark's cpu-baseline leg may call it.  It shares no
 * code, header, table or helper with the CUDA library; the packed-weight layout is re-implemented
 * here from its written description (two bits per weight, see oracle_pack below).
 *
 * Precision: every real-valued quantity is a C double; integer quantities are int32/int64.
 * Loops are written in the order of the definitions; the only concession to run time is one
 * OpenMP "parallel for" over independent output rows, which changes no arithmetic.
 *
 * Pins (tests/test_oracle_pins.py): numpy float64 mean(|W|); threshold invariants and crafted
 * +-gamma/2 ties; pack/unpack round trips; int8 invariants, crafted rounding ties; brute-force
 * integer matmul on tiny shapes and numpy int64 matmul; gate = 0 reduces to the pure ternary
 * layer; hand-worked 2x2 correction; SiLU-off equals (x A) B; the fake-quant float restatement;
 * the paper's T_max worked example (7B, FP16, 500 GB/s -> 35.7 tokens/s); for the LayerNorm
 * front end: numpy float64 statistics, a constant row, rows that are already normalised (the
 * front end then reduces to the plain quantiser), sign and power-of-two invariances, the listing's
 * rounding of the tie 76/152 (-> 63), the library layer_norm routine, and the equivalence of a
 * grouped gate with its expanded per-channel vector; for the differential attention: the library
 * scaled_dot_product_attention routine, lambda = 0, identical streams, a single token, constant V,
 * causality, and the lambda_0 formula's value; for the backward pass: automatic differentiation
 * (a library routine) of a float64 restatement whose quantisers are made straight-through with the
 * value-plus-detached-difference construction, gate = 0, and linearity in dY.
 * No function here is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_FLAG_NO_SILU 1u /* correction is (x A) B instead of SiLU(x A) B */

/* ---- exact decoding of the 16-bit input encodings ------------------------------------------ */

/* bfloat16: the upper 16 bits of an IEEE-754 binary32. */
static double bf16_to_double(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* IEEE-754 binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static double fp16_to_double(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int f = h & 0x3ff;
    double v;
    if (e == 0)
        v = ldexp((double)f, -24); /* zero and subnormals: f * 2^-10 * 2^-14 */
    else if (e == 31)
        v = f ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)f / 1024.0, e - 15);
    return sign ? -v : v;
}

int oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- Section 2.2, weight scale: gamma_W = (1/(m n)) sum_ij |W_ij| ---------------------------- */
/* Summed in double in index order, rounded once to binary32 (the stored scale is one fp32). */
float oracle_gamma_w(const float *W, int64_t d_out, int64_t d_in) {
    double acc = 0.0;
    for (int64_t i = 0; i < d_out * d_in; ++i) acc += fabs((double)W[i]);
    return (float)(acc / (double)(d_out * d_in));
}

/* ---- Section 2.2, ternary codes: Clip(Round(W / gamma_W), -1, 1) ------------------------------ */
/* Round-to-nearest of W/gamma followed by the clip has decision boundaries at +-gamma/2 (the
 * paper states these boundaries); a value exactly on a boundary is a tie between 0 and +-1 and
 * round-half-to-even sends it to 0.  gamma/2 is exact in binary32, so the comparison is exact. */
void oracle_ternarise(const float *W, int64_t d_out, int64_t d_in, float gamma, int8_t *T) {
    double half = (double)gamma / 2.0;
    for (int64_t i = 0; i < d_out * d_in; ++i) {
        double w = (double)W[i];
        T[i] = (w > half) ? 1 : (w < -half) ? -1 : 0;
    }
}

/* ---- packed layout (the paper only says "1.58-bit"; two bits per weight are used) ------------ */
/* The matrix is cut into tiles of 16 output rows by 256 input columns; d_out is padded up to a
 * multiple of 16 and d_in up to a multiple of 256 with zero weights.  A tile is 1024 bytes: its 16
 * rows one after the other, 64 bytes per row.  Tiles are stored with the column-tile index
 * running fastest: tile (R, C) starts at byte (R * (d_in_padded / 256) + C) * 1024.  The 64 bytes
 * of a row are 16 little-endian 32-bit words; word i holds the 16 weights whose column inside
 * the tile is 16 i .. 16 i + 15.  Writing that column as 16 i + 4 j + b with j, b in 0..3, the
 * weight's code c = t + 1 (0, 1 or 2; 3 is never written) sits in bits 8 b + 2 j and 8 b + 2 j + 1
 * of word i. */
static int64_t padded_cols(int64_t d_in) { return (d_in + 255) / 256 * 256; }
static int64_t padded_rows(int64_t d_out) { return (d_out + 15) / 16 * 16; }

int64_t oracle_packed_bytes(int64_t d_out, int64_t d_in) { return padded_rows(d_out) * padded_cols(d_in) / 4; }

/* Byte offset of the word that holds weight (n, k), and the bit position of its code in it. */
static int64_t word_offset(int64_t n, int64_t k, int64_t d_in, int *shift) {
    int64_t col_tiles = padded_cols(d_in) / 256;
    int64_t R = n / 16, row = n % 16, C = k / 256, col = k % 256;
    int64_t i = col / 16, j = (col % 16) / 4, b = col % 4;
    *shift = (int)(8 * b + 2 * j);
    return (R * col_tiles + C) * 1024 + row * 64 + i * 4;
}

void oracle_pack(const int8_t *T, int64_t d_out, int64_t d_in, uint8_t *packed) {
    int64_t rows = padded_rows(d_out), cols = padded_cols(d_in);
    memset(packed, 0, (size_t)(rows * cols / 4));
    for (int64_t n = 0; n < rows; ++n)
        for (int64_t k = 0; k < cols; ++k) {
            int t = (n < d_out && k < d_in) ? T[n * d_in + k] : 0; /* padding is weight 0 */
            int shift;
            int64_t off = word_offset(n, k, d_in, &shift);
            uint32_t c = (uint32_t)(t + 1) << shift;
            packed[off + 0] |= (uint8_t)(c & 0xff);
            packed[off + 1] |= (uint8_t)((c >> 8) & 0xff);
            packed[off + 2] |= (uint8_t)((c >> 16) & 0xff);
            packed[off + 3] |= (uint8_t)((c >> 24) & 0xff);
        }
}

/* Returns the number of invalid codes (value 3) met inside the matrix; those decode to 0. */
int64_t oracle_unpack(const uint8_t *packed, int64_t d_out, int64_t d_in, int8_t *T) {
    int64_t bad = 0;
    for (int64_t n = 0; n < d_out; ++n)
        for (int64_t k = 0; k < d_in; ++k) {
            int shift;
            int64_t off = word_offset(n, k, d_in, &shift);
            uint32_t word = (uint32_t)packed[off] | ((uint32_t)packed[off + 1] << 8) |
                            ((uint32_t)packed[off + 2] << 16) | ((uint32_t)packed[off + 3] << 24);
            uint32_t c = (word >> shift) & 3u;
            if (c == 3u) { ++bad; c = 1u; }
            T[n * d_in + k] = (int8_t)((int)c - 1);
        }
    return bad;
}

/* ---- base-3 packed layout: five ternary codes per byte, 1.6 bits per weight ------------------- */
/* The paper counts log2(3) = 1.58 bits per weight; five codes c = t + 1 in {0,1,2} fit one byte as
 * the base-3 number c0 + 3 c1 + 9 c2 + 27 c3 + 81 c4 (0..242).  The matrix is cut into tiles of 16
 * output rows by 320 input columns (d_out padded to 16, d_in to 320, with zero weights); a tile is
 * 1024 bytes, its 16 rows one after the other, 64 bytes per row; tiles are stored with the column
 * tile running fastest: tile (R, C) starts at byte (R * (d_in_padded / 320) + C) * 1024.
 * Which five columns of its row a byte holds: write the byte's index in the row as q = 16 t + j
 * (t in 0..3, j in 0..15) and let col(p, t) = 32 (p / 2) + 16 (p % 2) + 4 t for p in 0..19.  Then
 * digit e < 4 of the byte is the code of tile column col(j, t) + e, and digit 4 is the code of tile
 * column col(16 + j / 4, t) + j % 4. */
static int64_t padded_cols_b3(int64_t d_in) { return (d_in + 319) / 320 * 320; }

int64_t oracle_packed_bytes_b3(int64_t d_out, int64_t d_in) { return padded_rows(d_out) * padded_cols_b3(d_in) / 5; }

/* Byte offset of the byte that holds weight (n, k), and the power of three its code is scaled by. */
static int64_t byte_offset_b3(int64_t n, int64_t k, int64_t d_in, int *power) {
    static const int pow3[5] = {1, 3, 9, 27, 81};
    int64_t col_tiles = padded_cols_b3(d_in) / 320;
    int64_t R = n / 16, row = n % 16, C = k / 320, col = k % 320;
    int64_t p = 2 * (col / 32) + (col % 32) / 16, t = (col % 16) / 4, e = col % 4;
    int64_t j;
    if (p < 16) {
        j = p;
        *power = pow3[e];
    } else {
        j = 4 * (p - 16) + e;
        *power = pow3[4];
    }
    return (R * col_tiles + C) * 1024 + row * 64 + 16 * t + j;
}

void oracle_pack_b3(const int8_t *T, int64_t d_out, int64_t d_in, uint8_t *packed) {
    int64_t rows = padded_rows(d_out), cols = padded_cols_b3(d_in);
    memset(packed, 0, (size_t)(rows * cols / 5));
    for (int64_t n = 0; n < rows; ++n)
        for (int64_t k = 0; k < cols; ++k) {
            int t = (n < d_out && k < d_in) ? T[n * d_in + k] : 0; /* padding is weight 0 */
            int power;
            int64_t off = byte_offset_b3(n, k, d_in, &power);
            packed[off] = (uint8_t)(packed[off] + (t + 1) * power);
        }
}

/* Returns the number of invalid bytes (value above 242) met; their codes decode to 0. */
int64_t oracle_unpack_b3(const uint8_t *packed, int64_t d_out, int64_t d_in, int8_t *T) {
    int64_t bad = 0;
    for (int64_t n = 0; n < d_out; ++n)
        for (int64_t k = 0; k < d_in; ++k) {
            int power;
            int64_t off = byte_offset_b3(n, k, d_in, &power);
            int v = packed[off];
            if (v > 242) {
                bad += (power == 1); /* count each bad byte once per column group that starts in it */
                T[n * d_in + k] = 0;
                continue;
            }
            T[n * d_in + k] = (int8_t)((v / power) % 3 - 1);
        }
    return bad;
}

/* ---- Section 2.2.1 / Algorithm 1 steps 1-2: per-token absmax int8 quantisation --------------- */
/* gamma_x = max_k |x_k| (floored at 1e-5 so that an all-zero token does not divide by zero; the
 * floored value is used for both quantisation and dequantisation);
 * x~_k = Clip(Round(x_k / gamma_x * 127), -127, 127), Round = nearest, ties to even, of the
 * exact quotient.  127*x is exact in double for a bf16 x, so one correctly rounded division
 * followed by rint() yields the exact result. */
void oracle_act_quant(const uint16_t *x_bf16, int64_t M, int64_t d_in, int8_t *xq, float *gamma_x) {
    for (int64_t m = 0; m < M; ++m) {
        double amax = 0.0;
        for (int64_t k = 0; k < d_in; ++k) {
            double a = fabs(bf16_to_double(x_bf16[m * d_in + k]));
            if (a > amax) amax = a;
        }
        float g = (float)amax; /* exact: a bf16 value is a binary32 value */
        if (g < 1e-5f) g = 1e-5f;
        gamma_x[m] = g;
        for (int64_t k = 0; k < d_in; ++k) {
            double q = rint(127.0 * bf16_to_double(x_bf16[m * d_in + k]) / (double)g);
            if (q > 127.0) q = 127.0;
            if (q < -127.0) q = -127.0;
            xq[m * d_in + k] = (int8_t)q;
        }
    }
}

/* ---- Algorithm 1 step 3: Y_int = X~ (int8)  x  W~^T (ternary), integer arithmetic ------------- */
/* Returns 0, or 1 if any sum left the int32 range (it cannot for d_in < 2^24). */
int oracle_int_gemm(const int8_t *xq, const int8_t *T, int64_t M, int64_t d_out, int64_t d_in,
                    int32_t *y_int) {
    int overflow = 0;
#pragma omp parallel for schedule(static) reduction(| : overflow)
    for (int64_t n = 0; n < d_out; ++n)
        for (int64_t m = 0; m < M; ++m) {
            int64_t acc = 0;
            for (int64_t k = 0; k < d_in; ++k)
                acc += (int64_t)xq[m * d_in + k] * (int64_t)T[n * d_in + k];
            if (acc > INT32_MAX || acc < INT32_MIN) overflow |= 1;
            y_int[m * d_out + n] = (int32_t)acc;
        }
    return overflow;
}

static double silu(double z) { return z / (1.0 + exp(-z)); } /* z * sigmoid(z) */

/* ---- Algorithm 1, whole layer ----------------------------------------------------------------- */
/* y[m][n] = Y_int[m][n] * gamma_x[m] * gamma_W / 127  +  g[n] * sum_j SiLU(sum_k x[m][k] A[k][j]) B[j][n]
 *
 * Storage: x [M][d_in] bf16 bits; T [d_out][d_in] int8 ternary codes; At [r][d_in] fp16 bits
 * (the transpose of the paper's A); Bt [d_out][r] fp16 bits (the transpose of the paper's B);
 * gate [d_out] fp32 (the evaluated g = tanh(alpha), one value per output channel; the paper's
 * scalar gate is the constant vector); y [M][d_out] double.  r = 0 or a null gate gives the pure
 * ternary layer.  Optional outputs (nullable): xq_out [M][d_in], gamma_x_out [M],
 * y_int_out [M][d_out], h_out [M][r] double (after the activation). */
int oracle_forward(const uint16_t *x_bf16, int64_t M, const int8_t *T, float gamma_w, int64_t d_in,
                   int64_t d_out, const uint16_t *At_fp16, const uint16_t *Bt_fp16, int32_t r,
                   const float *gate, uint32_t flags, double *y, int8_t *xq_out, float *gamma_x_out,
                   int32_t *y_int_out, double *h_out, int8_t *xq_scratch, float *gx_scratch,
                   int32_t *yint_scratch, double *h_scratch) {
    int8_t *xq = xq_out ? xq_out : xq_scratch;
    float *gx = gamma_x_out ? gamma_x_out : gx_scratch;
    int32_t *yi = y_int_out ? y_int_out : yint_scratch;
    double *H = h_out ? h_out : h_scratch;
    int have_corr = (r > 0 && At_fp16 && Bt_fp16 && gate);

    /* Path 1: structural backbone. */
    oracle_act_quant(x_bf16, M, d_in, xq, gx);
    int overflow = oracle_int_gemm(xq, T, M, d_out, d_in, yi);

    /* Path 2: H = SiLU(X A). */
    if (have_corr) {
#pragma omp parallel for schedule(static)
        for (int64_t m = 0; m < M; ++m)
            for (int32_t j = 0; j < r; ++j) {
                double z = 0.0;
                for (int64_t k = 0; k < d_in; ++k)
                    z += bf16_to_double(x_bf16[m * d_in + k]) * fp16_to_double(At_fp16[(int64_t)j * d_in + k]);
                H[m * r + j] = (flags & ORACLE_FLAG_NO_SILU) ? z : silu(z);
            }
    }

    /* Dequantise, Y_corr = H B, gated fusion. */
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < d_out; ++n)
        for (int64_t m = 0; m < M; ++m) {
            double y_tern = (double)yi[m * d_out + n] * ((double)gx[m] * (double)gamma_w / 127.0);
            double y_corr = 0.0;
            if (have_corr) {
                for (int32_t j = 0; j < r; ++j)
                    y_corr += H[m * r + j] * fp16_to_double(Bt_fp16[n * r + j]);
                y_corr *= (double)gate[n];
            }
            y[m * d_out + n] = y_tern + y_corr;
        }
    return overflow;
}

/* ---- Appendix E, ScientificBitLinear.forward: the LayerNorm in front of the quantiser -------- */
/* The listing normalises each token before it is quantised (LayerNorm over d_in with a learned
 * weight and bias, biased variance, eps inside the square root), while the correction path of
 * AdaptiveDualPathLinear.forward reads the raw x.
 *
 * Statistics of each token, in double: mean = sum x / d_in, var = sum (x - mean)^2 / d_in,
 * rstd = 1 / sqrt(var + eps). */
void oracle_ln_stats(const uint16_t *x_bf16, int64_t M, int64_t d_in, double eps, double *mean, double *rstd) {
    for (int64_t m = 0; m < M; ++m) {
        double sum = 0.0;
        for (int64_t k = 0; k < d_in; ++k) sum += bf16_to_double(x_bf16[m * d_in + k]);
        double mu = sum / (double)d_in;
        double ss = 0.0;
        for (int64_t k = 0; k < d_in; ++k) {
            double d = bf16_to_double(x_bf16[m * d_in + k]) - mu;
            ss += d * d;
        }
        mean[m] = mu;
        rstd[m] = 1.0 / sqrt(ss / (double)d_in + eps);
    }
}

/* Normalisation and quantisation of the normalised token.  The listing does both in binary32
 * (x.float(), autocast disabled), so the precision is the paper's: every operation below is one
 * correctly rounded binary32 operation, in this order (the reading this library fixes, since the
 * rounded value decides the int8 code):
 *     d = x - mean;  n = d * rstd;  s = n * w[k];  xn = s + b[k];
 *     gamma_x = max(max_k |xn|, 1e-5);  scale = 127 / gamma_x;  q = rint(xn * scale), clipped to
 *     [-127, 127] (Algorithm 1's range; the product never reaches -127.5).
 * mean and rstd are given as binary32 values (per token).  Compiled with -ffp-contract=off, so no
 * operation is fused. */
void oracle_ln_quant(const uint16_t *x_bf16, int64_t M, int64_t d_in, const float *mean, const float *rstd,
                     const float *ln_w, const float *ln_b, float *xn_out, int8_t *xq, float *gamma_x) {
    for (int64_t m = 0; m < M; ++m) {
        float amax = 0.0f;
        for (int64_t k = 0; k < d_in; ++k) {
            float xf = (float)bf16_to_double(x_bf16[m * d_in + k]); /* exact */
            float d = xf - mean[m];
            float n = d * rstd[m];
            float s = n * ln_w[k];
            float xn = s + ln_b[k];
            if (xn_out) xn_out[m * d_in + k] = xn;
            float a = fabsf(xn);
            if (a > amax) amax = a;
        }
        float g = amax < 1e-5f ? 1e-5f : amax;
        gamma_x[m] = g;
        float scale = 127.0f / g;
        for (int64_t k = 0; k < d_in; ++k) {
            float xf = (float)bf16_to_double(x_bf16[m * d_in + k]);
            float d = xf - mean[m];
            float n = d * rstd[m];
            float s = n * ln_w[k];
            float xn = s + ln_b[k];
            float p = xn * scale;
            float q = rintf(p);
            if (q > 127.0f) q = 127.0f;
            if (q < -127.0f) q = -127.0f;
            xq[m * d_in + k] = (int8_t)q;
        }
    }
}

/* The layer with the LayerNorm front end and a grouped gate:
 *   y[m][n] = Y_int[m][n] * gamma_x[m] * gamma_W / 127 + g[n / gate_group] * sum_j SiLU(sum_k x[m][k] A[k][j]) B[j][n]
 * with X~, gamma_x from the NORMALISED token (above) and the correction from the RAW token.
 * gate holds ceil(d_out / gate_group) values: gate_group = 1 is one value per channel, d_out / n_heads
 * the listing's per-head gate (HeadAdaptiveDiffAttention), d_out the scalar gate.
 * mean_in / rstd_in (nullable): binary32 statistics to use instead of the double ones rounded to
 * binary32 (the tests pass the CUDA library's own, as they do for gamma_W). */
int oracle_forward_ln(const uint16_t *x_bf16, int64_t M, const int8_t *T, float gamma_w, int64_t d_in, int64_t d_out,
                      const float *ln_w, const float *ln_b, double eps, const float *mean_in, const float *rstd_in,
                      const uint16_t *At_fp16, const uint16_t *Bt_fp16, int32_t r, const float *gate, int64_t gate_group,
                      uint32_t flags, double *y, int8_t *xq, float *gamma_x, int32_t *y_int, double *H,
                      float *mean_out, float *rstd_out, double *stat_scratch /* 2 M doubles */) {
    int have_corr = (r > 0 && At_fp16 && Bt_fp16 && gate);
    oracle_ln_stats(x_bf16, M, d_in, eps, stat_scratch, stat_scratch + M);
    for (int64_t m = 0; m < M; ++m) {
        mean_out[m] = mean_in ? mean_in[m] : (float)stat_scratch[m];
        rstd_out[m] = rstd_in ? rstd_in[m] : (float)stat_scratch[M + m];
    }
    oracle_ln_quant(x_bf16, M, d_in, mean_out, rstd_out, ln_w, ln_b, NULL, xq, gamma_x);
    int overflow = oracle_int_gemm(xq, T, M, d_out, d_in, y_int);
    if (have_corr) {
#pragma omp parallel for schedule(static)
        for (int64_t m = 0; m < M; ++m)
            for (int32_t j = 0; j < r; ++j) {
                double z = 0.0;
                for (int64_t k = 0; k < d_in; ++k)
                    z += bf16_to_double(x_bf16[m * d_in + k]) * fp16_to_double(At_fp16[(int64_t)j * d_in + k]);
                H[m * r + j] = (flags & ORACLE_FLAG_NO_SILU) ? z : silu(z);
            }
    }
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < d_out; ++n)
        for (int64_t m = 0; m < M; ++m) {
            double y_tern = (double)y_int[m * d_out + n] * ((double)gamma_x[m] * (double)gamma_w / 127.0);
            double y_corr = 0.0;
            if (have_corr) {
                for (int32_t j = 0; j < r; ++j) y_corr += H[m * r + j] * fp16_to_double(Bt_fp16[n * r + j]);
                y_corr *= (double)gate[n / gate_group];
            }
            y[m * d_out + n] = y_tern + y_corr;
        }
    return overflow;
}

/* ---- Section 2.2, Definition "Straight-Through Estimator": backward pass of the layer ----------- */
/* Forward, as differentiated: y = Xd Wd^T + g (.) (SiLU(x A) B), with Xd = x~ gamma_x / 127 the
 * dequantised activations and Wd = gamma_W t the dequantised weights.  The estimator treats both
 * quantisers as the identity in the backward pass (every activation lies inside its clipping range,
 * and the reference module passes the weight gradient unchanged), everything else is differentiated
 * exactly.  With dY the gradient of the loss with respect to y:
 *     dW[n][k]   = sum_m dY[m][n] Xd[m][k]                      (gradient for the latent weights)
 *     dX[m][k]   = sum_n dY[m][n] Wd[n][k]  +  sum_j dZ[m][j] A[k][j]
 *     Z = x A,  H = SiLU(Z),  dH[m][j] = sum_n dY[m][n] g[n] B[j][n],  dZ = dH (.) SiLU'(Z)
 *     dA[k][j]   = sum_m x[m][k] dZ[m][j],   dB[j][n] = g[n] sum_m H[m][j] dY[m][n]
 *     dg[n]      = sum_m dY[m][n] (H B)[m][n]   (with respect to the evaluated gate g = tanh(alpha))
 * Storage as in the forward pass: At [r][d_in], Bt [d_out][r] fp16 bits; dAt, dBt in the same shapes.
 * dy [M][d_out] bf16 bits.  All sums in double.  Outputs nullable. */
void oracle_backward(const uint16_t *x_bf16, int64_t M, const int8_t *T, float gamma_w, int64_t d_in, int64_t d_out,
                     const uint16_t *At_fp16, const uint16_t *Bt_fp16, int32_t r, const float *gate, const uint16_t *dy_bf16,
                     uint32_t flags, double *dx, double *dW, double *dAt, double *dBt, double *dgate, int8_t *xq_scratch,
                     float *gx_scratch, double *zh_scratch /* 3 M r doubles: Z, H, dZ */) {
    int have_corr = (r > 0 && At_fp16 && Bt_fp16 && gate);
    oracle_act_quant(x_bf16, M, d_in, xq_scratch, gx_scratch);
    double *Z = zh_scratch, *H = zh_scratch + M * (have_corr ? r : 0), *dZ = zh_scratch + 2 * M * (have_corr ? r : 0);
    if (have_corr) {
#pragma omp parallel for schedule(static)
        for (int64_t m = 0; m < M; ++m)
            for (int32_t j = 0; j < r; ++j) {
                double z = 0.0;
                for (int64_t k = 0; k < d_in; ++k)
                    z += bf16_to_double(x_bf16[m * d_in + k]) * fp16_to_double(At_fp16[(int64_t)j * d_in + k]);
                double dh = 0.0;
                for (int64_t n = 0; n < d_out; ++n)
                    dh += bf16_to_double(dy_bf16[m * d_out + n]) * (double)gate[n] * fp16_to_double(Bt_fp16[n * r + j]);
                double sg = 1.0 / (1.0 + exp(-z));
                Z[m * r + j] = z;
                H[m * r + j] = (flags & ORACLE_FLAG_NO_SILU) ? z : z * sg;
                dZ[m * r + j] = (flags & ORACLE_FLAG_NO_SILU) ? dh : dh * (sg * (1.0 + z * (1.0 - sg)));
            }
    }
    if (dx) {
#pragma omp parallel for schedule(static)
        for (int64_t m = 0; m < M; ++m)
            for (int64_t k = 0; k < d_in; ++k) {
                double a = 0.0;
                for (int64_t n = 0; n < d_out; ++n) a += bf16_to_double(dy_bf16[m * d_out + n]) * (double)T[n * d_in + k];
                a *= (double)gamma_w;
                if (have_corr)
                    for (int32_t j = 0; j < r; ++j) a += dZ[m * r + j] * fp16_to_double(At_fp16[(int64_t)j * d_in + k]);
                dx[m * d_in + k] = a;
            }
    }
    if (dW) {
#pragma omp parallel for schedule(static)
        for (int64_t n = 0; n < d_out; ++n)
            for (int64_t k = 0; k < d_in; ++k) {
                double a = 0.0;
                for (int64_t m = 0; m < M; ++m)
                    a += bf16_to_double(dy_bf16[m * d_out + n]) * ((double)xq_scratch[m * d_in + k] * (double)gx_scratch[m] / 127.0);
                dW[n * d_in + k] = a;
            }
    }
    if (have_corr && dAt) {
#pragma omp parallel for schedule(static)
        for (int64_t k = 0; k < d_in; ++k)
            for (int32_t j = 0; j < r; ++j) {
                double a = 0.0;
                for (int64_t m = 0; m < M; ++m) a += dZ[m * r + j] * bf16_to_double(x_bf16[m * d_in + k]);
                dAt[(int64_t)j * d_in + k] = a;
            }
    }
    if (have_corr && (dBt || dgate)) {
#pragma omp parallel for schedule(static)
        for (int64_t n = 0; n < d_out; ++n) {
            double dg = 0.0;
            for (int32_t j = 0; j < r; ++j) {
                double a = 0.0;
                for (int64_t m = 0; m < M; ++m) a += bf16_to_double(dy_bf16[m * d_out + n]) * H[m * r + j];
                if (dBt) dBt[n * r + j] = (double)gate[n] * a;
                dg += a * fp16_to_double(Bt_fp16[n * r + j]);
            }
            if (dgate) dgate[n] = dg;
        }
    }
}

/* ---- Section 2.4, Definition "Differential Attention" ------------------------------------------ */
/* O = ( Softmax(Q1 K1^T / sqrt(d_h)) - lambda * Softmax(Q2 K2^T / sqrt(d_h)) ) V, per batch element and
 * head, causal (token i attends to tokens j <= i: the model is a language model; the listing passes
 * is_causal), times out_scale (1 in the Definition; the listing multiplies by 0.5).
 * Storage, token-major as the projections write it: q, k [B*L][2*h*d_h] bf16 bits, where the first
 * h*d_h columns are the h heads of stream 1 and the last h*d_h those of stream 2 (the Definition's
 * [Q1; Q2], the listing's chunk over 2h heads); v [B*L][h*d_h] bf16 bits; out [B*L][h*d_h] double.
 * Everything in double from the exact bf16 values; the softmax subtracts the row maximum. */
void oracle_diff_attention(const uint16_t *q, const uint16_t *k, const uint16_t *v, int64_t B, int64_t L, int64_t h,
                           int64_t dh, double lambda, double out_scale, double *out) {
    const int64_t dq = 2 * h * dh, dv = h * dh;
    const double inv = 1.0 / sqrt((double)dh);
#pragma omp parallel for schedule(dynamic) collapse(2)
    for (int64_t b = 0; b < B; ++b)
        for (int64_t hd = 0; hd < h; ++hd) {
            double *p = (double *)malloc(sizeof(double) * (size_t)L);
            for (int64_t i = 0; i < L; ++i) {
                double *o = out + ((b * L + i) * dv + hd * dh);
                for (int64_t c = 0; c < dh; ++c) o[c] = 0.0;
                for (int s = 0; s < 2; ++s) {
                    const uint16_t *qi = q + (b * L + i) * dq + (s * h + hd) * dh;
                    double mx = -INFINITY;
                    for (int64_t j = 0; j <= i; ++j) {
                        const uint16_t *kj = k + (b * L + j) * dq + (s * h + hd) * dh;
                        double dot = 0.0;
                        for (int64_t c = 0; c < dh; ++c) dot += bf16_to_double(qi[c]) * bf16_to_double(kj[c]);
                        p[j] = dot * inv;
                        if (p[j] > mx) mx = p[j];
                    }
                    double sum = 0.0;
                    for (int64_t j = 0; j <= i; ++j) {
                        p[j] = exp(p[j] - mx);
                        sum += p[j];
                    }
                    const double w = (s == 0 ? 1.0 : -lambda) / sum;
                    for (int64_t j = 0; j <= i; ++j) {
                        const uint16_t *vj = v + (b * L + j) * dv + hd * dh;
                        const double pj = p[j] * w;
                        for (int64_t c = 0; c < dh; ++c) o[c] += pj * bf16_to_double(vj[c]);
                    }
                }
                for (int64_t c = 0; c < dh; ++c) o[c] *= out_scale;
            }
            free(p);
        }
}

/* lambda_0 = 0.8 - 0.6 exp(-0.3 d_h) (same Definition). */
double oracle_lambda0(double dh) { return 0.8 - 0.6 * exp(-0.3 * dh); }

/* ---- Introduction, memory-wall bound: T_max = B_mem / (P * b / 8) tokens per second ----------- */
double oracle_tmax(double bmem_bytes_per_s, double params, double bits_per_param) {
    return bmem_bytes_per_s / (params * bits_per_param / 8.0);
}

/* ---- Section 4.2, effective bit-width: b_eff = log2(3) + g * b_corr * r / d -------------------- */
double oracle_effective_bits(double g, double b_corr, double r, double d) {
    return log2(3.0) + g * b_corr * r / d;
}
