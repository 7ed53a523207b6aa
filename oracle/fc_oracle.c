/*
 * CPU oracle for fused operator chains.  TEST INFRASTRUCTURE ONLY: it is called by the tests, by
 * the smoke check and by the benchmark's cpu_baseline leg, never by the library's product path,
 * and it shares no code with the CUDA path.
 *
 * Everything is the plain definition, written out in double precision with one accumulator per
 * output and no blocking, fusion or reordering.  Threads (OpenMP) only split independent rows or
 * images.  No BLAS, no SIMD intrinsics, no fast-math.
 *
 * What each routine follows:
 *   orc_gemm_nt        Y = X * W^T with the weight stored [out_features x in_features] row-major,
 *                      i.e. both operands contiguous along the contracted index (the operand
 *                      convention of the paper's appendix GEMM and linear-layer listings).
 *   orc_gemm_nt_mx     the same contraction with block-scaled ("microscaling", MX) operands: along the
 *                      contracted index every 32 consecutive elements of a row share one power-of-two
 *                      scale, stored as an 8-bit exponent (E8M0: 2^(e - 127), e = 255 is NaN), so
 *                      Y[m][n] = sum_j 2^(sa[m][j] - 127) 2^(sb[n][j] - 127) sum_{k in block j} X[m][k] W[n][k].
 *                      The paper only mentions 8-bit floats in passing; the format is the open
 *                      microscaling one that the B200 tensor cores implement (MXFP8: E4M3 elements).
 *   orc_conv2d_nhwc    cross-correlation, zero padding, floor output size
 *                      OH = (H + 2*pad - R)/stride + 1, input row = oh*stride - pad + r, taps that
 *                      fall outside the image contribute nothing (the indexing convention of the
 *                      paper's appendix convolution listing, restated for NHWC / [Cout][R][S][Cin]).
 *   orc_conv2d_nchw    the same operation on the listing's own layouts, image [NB][Cin][H][W] and
 *                      weights [Cout][Cin][R][S]; the output keeps channels last.
 *   orc_bias_n, orc_relu, orc_scale   bias broadcast over the output-feature / channel index, ReLU
 *                      as "negative -> 0", scaling by a scalar (the appendix epilogue: bias, ReLU,
 *                      multiply).
 *   orc_row_logsumexp  max + log(sum exp(v - max)); over a row of length one this is the identity,
 *                      the closed form the paper's appendix (Level-2 Q18 analysis) relies on.
 *   orc_round_bf16, orc_round_f16   round to nearest even onto the 16-bit grid: what a chain of linear
 *                      layers does to an activation that it hands to the next contraction (the paper's
 *                      appendix network keeps activations in the tensor dtype between layers).
 *   orc_maxpool_2x2    maximum over non-overlapping 2 x 2 windows, floor output size (the window
 *                      arithmetic of the paper's appendix max-pool listing with kernel 2, stride 2,
 *                      no padding, restated for NHWC).
 *   orc_gelu_tanh, orc_clamp, orc_affine_n, orc_add_tensor, orc_row_softmax, orc_global_avgpool,
 *   orc_row_sum, orc_row_max (row mean = row sum / N)
 *                      textbook definitions; the paper does not print them, the benchmark
 *                      configurations of this repository name them.
 *
 * Pins (tests, CPU only): identity / zero / rank-1 weights, exact small-integer contractions,
 * exact-rational brute force with a different loop order on tiny shapes, centre and shifted delta
 * kernels, all-ones tap counts (both layouts; the channel-first form also against the library's
 * convolution and against the channel-last form on permuted arrays), high-precision (mpmath) values of GELU / logsumexp / softmax,
 * shift invariance, constant rows, rows summing to one, pooling linearity; max-pool against a
 * reshape-and-max in numpy, a single planted maximum per window, and dropped odd edges; the 16-bit
 * rounding against every stored pattern (identity), exact ties, and numpy's own conversions; the scale
 * bytes against the library's own E8M0 type over all 256 patterns, the block-scaled contraction against
 * the plain one (unit scales), against diag(scales) products for a single block, on operands that are
 * one-hot on either side of a block boundary, and against exact rationals.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* exact widening of stored values */
void orc_widen_bf16(const uint16_t* src, int64_t n, double* dst) {
    for (int64_t i = 0; i < n; ++i) {
        uint32_t u = ((uint32_t)src[i]) << 16;
        float f;
        memcpy(&f, &u, 4);
        dst[i] = (double)f;
    }
}

/* IEEE binary16 -> double, exactly (sign, 5-bit exponent, 10-bit fraction; subnormals, inf, nan) */
void orc_widen_f16(const uint16_t* src, int64_t n, double* dst) {
    for (int64_t i = 0; i < n; ++i) {
        const uint16_t h = src[i];
        const int sign = h >> 15, e = (h >> 10) & 31, f = h & 1023;
        double v;
        if (e == 0) v = ldexp((double)f, -24);
        else if (e == 31) v = f ? NAN : INFINITY;
        else v = ldexp((double)(1024 + f), e - 25);
        dst[i] = sign ? -v : v;
    }
}

/* 8-bit float E4M3 (finite-only variant: 1 sign, 4 exponent bits with bias 7, 3 fraction bits; exponent 0 is
 * subnormal; the all-ones pattern of each sign is NaN, there are no infinities) -> double, exactly */
void orc_widen_f8e4m3(const uint8_t* src, int64_t n, double* dst) {
    for (int64_t i = 0; i < n; ++i) {
        const uint8_t b = src[i];
        const int sign = b >> 7, e = (b >> 3) & 15, f = b & 7;
        double v;
        if (e == 15 && f == 7) v = NAN;
        else if (e == 0) v = ldexp((double) f, -9);           /* f/8 * 2^-6 */
        else v = ldexp((double) (8 + f), e - 10);              /* (1 + f/8) * 2^(e-7) */
        dst[i] = sign ? -v : v;
    }
}

void orc_widen_f32(const float* src, int64_t n, double* dst) {
    for (int64_t i = 0; i < n; ++i) dst[i] = (double)src[i];
}

/* Round to nearest, ties to even, onto the grid of a binary floating-point format with `sig` significant
 * bits, minimum (subnormal) exponent `emin_ulp` for the unit in the last place, and largest finite value
 * `maxv` (values that round beyond it become infinite).  Used where a chain feeds a contraction with
 * the output of a previous one: the tensor-core operand is the value as stored in the 16-bit type. */
static double round_to_grid(double v, int sig, int emin_ulp, double maxv) {
    if (v == 0.0 || isnan(v) || isinf(v)) return v;
    int e;
    (void) frexp(v, &e);                  /* |v| = f * 2^e, f in [0.5, 1)  ->  leading bit has weight 2^(e-1) */
    int ulp_e = e - sig;                  /* weight of the last kept bit */
    if (ulp_e < emin_ulp) ulp_e = emin_ulp;
    const double q = nearbyint(ldexp(v, -ulp_e));   /* default rounding mode: to nearest, ties to even */
    const double r = ldexp(q, ulp_e);
    if (fabs(r) > maxv) return v < 0 ? -INFINITY : INFINITY;
    return r;
}

/* bfloat16: 8 significant bits, smallest subnormal 2^-133, largest finite (2 - 2^-7) * 2^127 */
void orc_round_bf16(double* V, int64_t count) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) V[i] = round_to_grid(V[i], 8, -133, 3.3895313892515355e38);
}

/* IEEE binary16: 11 significant bits, smallest subnormal 2^-24, largest finite 65504 */
void orc_round_f16(double* V, int64_t count) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) V[i] = round_to_grid(V[i], 11, -24, 65504.0);
}

/* V[m][n] = sum_{k ascending} A[m][k] * B[n][k] */
void orc_gemm_nt(const double* A, const double* B, int64_t M, int64_t N, int64_t K, double* V) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) acc += A[m * K + k] * B[n * K + k];
            V[m * N + n] = acc;
        }
    }
}

/* E8M0 scale bytes -> double: 2^(e - 127); the pattern 255 is NaN (the format has no zero, sign or infinity) */
void orc_widen_e8m0(const uint8_t* src, int64_t n, double* dst) {
    for (int64_t i = 0; i < n; ++i) dst[i] = src[i] == 255 ? NAN : ldexp(1.0, (int) src[i] - 127);
}

/* Block-scaled contraction: V[m][n] = sum_{j ascending} SA[m][j] * SB[n][j] * (sum_{k = 32 j .. 32 j + 31} A[m][k] * B[n][k]),
 * SA [M][K/32] and SB [N][K/32] the widened scales.  K must be a multiple of 32. */
void orc_gemm_nt_mx(const double* A, const double* B, const double* SA, const double* SB, int64_t M, int64_t N,
                    int64_t K, double* V) {
    const int64_t blocks = K / 32;
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t j = 0; j < blocks; ++j) {
                double blk = 0.0;
                for (int64_t k = 32 * j; k < 32 * j + 32; ++k) blk += A[m * K + k] * B[n * K + k];
                acc += SA[m * blocks + j] * SB[n * blocks + j] * blk;
            }
            V[m * N + n] = acc;
        }
    }
}

/* V[b][oh][ow][co] = sum_{r,s,ci} in[b][oh*stride-pad+r][ow*stride-pad+s][ci] * Wt[co][r][s][ci] */
void orc_conv2d_nhwc(const double* in, const double* Wt, int64_t NB, int64_t H, int64_t W,
                     int64_t Cin, int64_t Cout, int64_t R, int64_t S, int64_t stride, int64_t pad,
                     double* V) {
    const int64_t OH = (H + 2 * pad - R) / stride + 1;
    const int64_t OW = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < NB; ++b) {
        for (int64_t oh = 0; oh < OH; ++oh) {
            for (int64_t ow = 0; ow < OW; ++ow) {
                for (int64_t co = 0; co < Cout; ++co) {
                    double acc = 0.0;
                    for (int64_t r = 0; r < R; ++r) {
                        const int64_t ih = oh * stride - pad + r;
                        if (ih < 0 || ih >= H) continue;
                        for (int64_t s = 0; s < S; ++s) {
                            const int64_t iw = ow * stride - pad + s;
                            if (iw < 0 || iw >= W) continue;
                            const double* px = in + ((b * H + ih) * W + iw) * Cin;
                            const double* wt = Wt + ((co * R + r) * S + s) * Cin;
                            for (int64_t ci = 0; ci < Cin; ++ci) acc += px[ci] * wt[ci];
                        }
                    }
                    V[((b * OH + oh) * OW + ow) * Cout + co] = acc;
                }
            }
        }
    }
}

/* The same cross-correlation on the layouts the paper's appendix listing itself uses: image
 * [NB][Cin][H][W], weights [Cout][Cin][R][S].  The result keeps the channel index last,
 * V[NB][OH][OW][Cout], so that the epilogue ops and the pooling that follow see one layout. */
void orc_conv2d_nchw(const double* in, const double* Wt, int64_t NB, int64_t H, int64_t W,
                     int64_t Cin, int64_t Cout, int64_t R, int64_t S, int64_t stride, int64_t pad,
                     double* V) {
    const int64_t OH = (H + 2 * pad - R) / stride + 1;
    const int64_t OW = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < NB; ++b) {
        for (int64_t co = 0; co < Cout; ++co) {
            for (int64_t oh = 0; oh < OH; ++oh) {
                for (int64_t ow = 0; ow < OW; ++ow) {
                    double acc = 0.0;
                    for (int64_t ci = 0; ci < Cin; ++ci) {
                        for (int64_t r = 0; r < R; ++r) {
                            const int64_t ih = oh * stride - pad + r;
                            if (ih < 0 || ih >= H) continue;
                            for (int64_t s = 0; s < S; ++s) {
                                const int64_t iw = ow * stride - pad + s;
                                if (iw < 0 || iw >= W) continue;
                                acc += in[((b * Cin + ci) * H + ih) * W + iw] * Wt[((co * Cin + ci) * R + r) * S + s];
                            }
                        }
                    }
                    V[((b * OH + oh) * OW + ow) * Cout + co] = acc;
                }
            }
        }
    }
}

/* elementwise ops on V viewed as [rows][N], in place */
void orc_bias_n(double* V, int64_t rows, int64_t N, const double* b) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < rows; ++m)
        for (int64_t n = 0; n < N; ++n) V[m * N + n] += b[n];
}

void orc_affine_n(double* V, int64_t rows, int64_t N, const double* gamma, const double* beta) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < rows; ++m)
        for (int64_t n = 0; n < N; ++n) V[m * N + n] = V[m * N + n] * gamma[n] + beta[n];
}

void orc_relu(double* V, int64_t count) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) V[i] = V[i] < 0.0 ? 0.0 : V[i];
}

/* GELU, tanh form: 0.5 v (1 + tanh( sqrt(2/pi) (v + 0.044715 v^3) )) */
void orc_gelu_tanh(double* V, int64_t count) {
    const double c = 0.7978845608028654; /* sqrt(2/pi) */
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) {
        const double v = V[i];
        V[i] = 0.5 * v * (1.0 + tanh(c * (v + 0.044715 * v * v * v)));
    }
}

void orc_scale(double* V, int64_t count, double f) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) V[i] *= f;
}

void orc_clamp(double* V, int64_t count, double lo, double hi) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) {
        double v = V[i];
        v = v < lo ? lo : v;
        v = v > hi ? hi : v;
        V[i] = v;
    }
}

void orc_add_tensor(double* V, int64_t count, const double* T) {
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < count; ++i) V[i] += T[i];
}

/* out[m] = max_n V[m][n] + log( sum_n exp(V[m][n] - max) ) */
void orc_row_logsumexp(const double* V, int64_t rows, int64_t N, double* out) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < rows; ++m) {
        const double* v = V + m * N;
        double mx = v[0];
        for (int64_t n = 1; n < N; ++n) mx = v[n] > mx ? v[n] : mx;
        double s = 0.0;
        for (int64_t n = 0; n < N; ++n) s += exp(v[n] - mx);
        out[m] = mx + log(s);
    }
}

/* P[m][n] = exp(V[m][n] - max) / sum_n exp(V[m][n] - max) */
void orc_row_softmax(const double* V, int64_t rows, int64_t N, double* P) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < rows; ++m) {
        const double* v = V + m * N;
        double* p = P + m * N;
        double mx = v[0];
        for (int64_t n = 1; n < N; ++n) mx = v[n] > mx ? v[n] : mx;
        double s = 0.0;
        for (int64_t n = 0; n < N; ++n) s += exp(v[n] - mx);
        for (int64_t n = 0; n < N; ++n) p[n] = exp(v[n] - mx) / s;
    }
}

/* out[b][c] = (1/HW) sum_{p} V[b][p][c] */
void orc_global_avgpool(const double* V, int64_t NB, int64_t HW, int64_t C, double* out) {
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < NB; ++b) {
        for (int64_t c = 0; c < C; ++c) {
            double s = 0.0;
            for (int64_t p = 0; p < HW; ++p) s += V[(b * HW + p) * C + c];
            out[b * C + c] = s / (double)HW;
        }
    }
}

/* out[b][i][j][c] = max over the 2 x 2 window (rows 2i, 2i+1; columns 2j, 2j+1) of V[b][.][.][c];
 * output size floor(OH/2) x floor(OW/2): a last odd row or column belongs to no window */
void orc_maxpool_2x2(const double* V, int64_t NB, int64_t OH, int64_t OW, int64_t C, double* out) {
    const int64_t PH = OH / 2, PW = OW / 2;
#pragma omp parallel for collapse(2) schedule(static)
    for (int64_t b = 0; b < NB; ++b) {
        for (int64_t i = 0; i < PH; ++i) {
            for (int64_t j = 0; j < PW; ++j) {
                for (int64_t c = 0; c < C; ++c) {
                    double mx = V[((b * OH + 2 * i) * OW + 2 * j) * C + c];
                    for (int64_t di = 0; di < 2; ++di)
                        for (int64_t dj = 0; dj < 2; ++dj) {
                            const double v = V[((b * OH + 2 * i + di) * OW + 2 * j + dj) * C + c];
                            mx = v > mx ? v : mx;
                        }
                    out[((b * PH + i) * PW + j) * C + c] = mx;
                }
            }
        }
    }
}

/* out[m] = sum_n V[m][n], n ascending, one accumulator */
void orc_row_sum(const double* V, int64_t rows, int64_t N, double* out) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < rows; ++m) {
        double s = 0.0;
        for (int64_t n = 0; n < N; ++n) s += V[m * N + n];
        out[m] = s;
    }
}

/* out[m] = max_n V[m][n] */
void orc_row_max(const double* V, int64_t rows, int64_t N, double* out) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < rows; ++m) {
        double mx = V[m * N];
        for (int64_t n = 1; n < N; ++n) mx = V[m * N + n] > mx ? V[m * N + n] : mx;
        out[m] = mx;
    }
}
