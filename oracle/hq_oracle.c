/*
 * hq_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, CPU-only statement of what the Hadamard-quantized layer forward of
 * HQ-DM computes, used to check the CUDA library and as the reported CPU baseline.
 * Only the test-suite, the smoke check and the benchmark's CPU-baseline legs may call it;
 * the CUDA library never does, and the two share no source, header, table or helper.
 *
 * Everything is written the way the paper states it: a dense Hadamard matrix built by the
 * Sylvester recurrence and applied as a matrix product, per-row absmax quantization,
 * triple-loop integer GEMM, seven-loop direct convolution, dequantization in fp64.
 * Floating point is fp64 except where the method stores a value (scales are fp32);
 * integer sums are int64.  No blocking, fusion or reordering.  OpenMP only splits the
 * outermost row loop; every row's arithmetic is sequential in index order.
 *
 * Pins (tests/test_oracle_pins.py): H_raw*H_raw^T = n*I and the closed form
 * (-1)^popcount(i&j); the worked vectors of Eq. 15-16; |u - s*q| <= s/2; involution and
 * Parseval; brute-force integer products; conv == im2col GEMM; exact recovery of X*W_hat
 * when activations are not rounded; the network's unquantized operations (GroupNorm, SiLU,
 * attention core, nearest up-sampling, step embedding, float convolution) against torch's CPU
 * routines in fp64 and closed forms (tests/test_oracle_network_pins.py).  Parity unpinned:
 * nothing in this file (trained scales, LoRA values and image-quality metrics are outside it).
 *
 * Layout conventions: activations [rows][cols] row-major; weights [N][RS][C] (output
 * channel, filter tap, input channel), i.e. the transpose of the paper's W in R^{Ci x Co};
 * conv activations NHWC.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef long long i64;

static int is_pow2(i64 n) { return n > 0 && (n & (n - 1)) == 0; }
static int ilog2(i64 n) { int k = 0; while ((1LL << k) < n) ++k; return k; }
static int qmax_of(int bits) { return (1 << (bits - 1)) - 1; }
static int qmin_of(int bits) { return -(1 << (bits - 1)); }

int hqo_version(void) { return 1; }

/* Eq. 5 with the 1/sqrt(2) left out (Eq. 7): H_0 = [1], H_k = [[H, H], [H, -H]], entries +-1.
 * H is n x n, row-major.  Returns 0, or -1 if n is not a power of two. */
int hqo_hadamard_raw(int n, int8_t* H) {
    if (!is_pow2(n)) return -1;
    H[0] = 1;
    for (int size = 1; size < n; size *= 2) {
        for (int i = 0; i < size; ++i) {
            for (int j = 0; j < size; ++j) {
                int8_t v = H[(i64)i * n + j];
                H[(i64)i * n + (j + size)] = v;
                H[(i64)(i + size) * n + j] = v;
                H[(i64)(i + size) * n + (j + size)] = (int8_t)-v;
            }
        }
    }
    return 0;
}

/* Eq. 10 with Eq. 7: u = x * BlockDiag(H_k, ..., H_k), H_k = 2^(-k/2) H_raw, n = 2^k = had_block,
 * cols = m*n.  had_block <= 1 means H = I (the bypass of the paragraph after Eq. 10).
 * Returns 0, -1 on a bad block size. */
int hqo_transform(const double* x, i64 rows, i64 cols, int had_block, double* u) {
    if (had_block <= 1) {
        memcpy(u, x, sizeof(double) * (size_t)(rows * cols));
        return 0;
    }
    const int n = had_block;
    if (!is_pow2(n) || cols % n != 0) return -1;
    int8_t* H = (int8_t*)malloc((size_t)n * n);
    if (!H) return -2;
    hqo_hadamard_raw(n, H);
    const double norm = pow(2.0, -0.5 * (double)ilog2(n));
    const i64 m = cols / n;
#pragma omp parallel for schedule(static)
    for (i64 r = 0; r < rows; ++r) {
        for (i64 b = 0; b < m; ++b) {
            const double* xb = x + r * cols + b * n;
            double* ub = u + r * cols + b * n;
            for (int j = 0; j < n; ++j) {
                double t = 0.0;
                for (int i = 0; i < n; ++i) t += xb[i] * (double)H[(i64)i * n + j];
                ub[j] = t * norm;
            }
        }
    }
    free(H);
    return 0;
}

/* Eq. 3, symmetric: q = clamp(round(u / S), qmin, qmax), round = half-to-even.
 * mode 0: one S per row, S = max_j|u_j| / qmax stored as fp32 (an all-zero row gets S = 1);
 * mode 1: the given scalar S for every row (scales[0] = S).
 * v_out (optional) receives u / S before rounding.  Returns 0, -1 on bad bits. */
int hqo_quantize(const double* u, i64 rows, i64 cols, int bits, int mode, float static_scale,
                 int8_t* q, float* scales, double* v_out) {
    if (bits < 2 || bits > 8) return -1;
    const int qmax = qmax_of(bits), qmin = qmin_of(bits);
    if (mode == 1) scales[0] = static_scale;
#pragma omp parallel for schedule(static)
    for (i64 r = 0; r < rows; ++r) {
        const double* ur = u + r * cols;
        float s;
        if (mode == 0) {
            double amax = 0.0;
            for (i64 j = 0; j < cols; ++j) { double a = fabs(ur[j]); if (a > amax) amax = a; }
            s = (amax > 0.0) ? (float)(amax / (double)qmax) : 1.0f;
            if (!(s > 0.0f)) s = 1.0f;   /* amax so small that the fp32 scale underflows */
            scales[r] = s;
        } else {
            s = static_scale;
        }
        for (i64 j = 0; j < cols; ++j) {
            double v = ur[j] / (double)s;
            if (v_out) v_out[r * cols + j] = v;
            double c = rint(v);
            if (c > qmax) c = qmax;
            if (c < qmin) c = qmin;
            q[r * cols + j] = (int8_t)c;
        }
    }
    return 0;
}

/* Storage of 4-bit (and sign-extended 3-bit) codes: two per byte, element 2j in the low
 * nibble, 2j+1 in the high nibble, two's complement.  count must be even. */
int hqo_pack_nibbles(const int8_t* q, i64 count, uint8_t* out) {
    if (count % 2) return -1;
    for (i64 j = 0; j < count / 2; ++j)
        out[j] = (uint8_t)(((uint8_t)q[2 * j] & 0xF) | (((uint8_t)q[2 * j + 1] & 0xF) << 4));
    return 0;
}

int hqo_unpack_nibbles(const uint8_t* in, i64 count, int8_t* q) {
    if (count % 2) return -1;
    for (i64 j = 0; j < count / 2; ++j) {
        int lo = in[j] & 0xF, hi = (in[j] >> 4) & 0xF;
        q[2 * j] = (int8_t)(lo >= 8 ? lo - 16 : lo);
        q[2 * j + 1] = (int8_t)(hi >= 8 ? hi - 16 : hi);
    }
    return 0;
}

/* Eq. 3 on the weights, one scale per output channel (row o of w [N][KK], KK = RS*C):
 * S_w[o] = max|w[o,:]| / qmax (fp32; 0 -> 1), W_int = clamp(round(w / S_w)). */
int hqo_weight_quantize(const double* w, i64 N, i64 KK, int w_bits, int32_t* w_int, float* s_w) {
    if (w_bits < 2 || w_bits > 8) return -1;
    const int qmax = qmax_of(w_bits), qmin = qmin_of(w_bits);
#pragma omp parallel for schedule(static)
    for (i64 o = 0; o < N; ++o) {
        double amax = 0.0;
        for (i64 k = 0; k < KK; ++k) { double a = fabs(w[o * KK + k]); if (a > amax) amax = a; }
        float s = (amax > 0.0) ? (float)(amax / (double)qmax) : 1.0f;
        if (!(s > 0.0f)) s = 1.0f;
        s_w[o] = s;
        for (i64 k = 0; k < KK; ++k) {
            double c = rint(w[o * KK + k] / (double)s);
            if (c > qmax) c = qmax;
            if (c < qmin) c = qmin;
            w_int[o * KK + k] = (int32_t)c;
        }
    }
    return 0;
}

/* The inner product H * W_int of Eq. 12 / Eq. 14 (channel axis), exact integers:
 * B[o][tap][b*n + i] = sum_j H_raw[i][j] * W_int[o][tap][b*n + j].   w_int, B: [N][RS][C]. */
int hqo_weight_fold(const int32_t* w_int, i64 N, i64 RS, i64 C, int had_block, int32_t* B) {
    if (had_block <= 1) { memcpy(B, w_int, sizeof(int32_t) * (size_t)(N * RS * C)); return 0; }
    const int n = had_block;
    if (!is_pow2(n) || C % n != 0) return -1;
    int8_t* H = (int8_t*)malloc((size_t)n * n);
    if (!H) return -2;
    hqo_hadamard_raw(n, H);
#pragma omp parallel for schedule(static)
    for (i64 row = 0; row < N * RS; ++row) {
        for (i64 b = 0; b < C / n; ++b) {
            const int32_t* wb = w_int + row * C + b * n;
            int32_t* Bb = B + row * C + b * n;
            for (int i = 0; i < n; ++i) {
                i64 t = 0;
                for (int j = 0; j < n; ++j) t += (i64)H[(i64)i * n + j] * wb[j];
                Bb[i] = (int32_t)t;
            }
        }
    }
    free(H);
    return 0;
}

/* The Double-Hadamard weights the paper compares against: W' = H^T W with the orthonormal H
 * (so X H * H^T W = X W), then Eq. 3 per output channel.  w [N][RS][C] -> B [N][RS][C]. */
int hqo_weight_double(const double* w, i64 N, i64 RS, i64 C, int w_bits, int had_block,
                      int32_t* B, float* s_w) {
    double* wt = (double*)malloc(sizeof(double) * (size_t)(N * RS * C));
    if (!wt) return -2;
    /* row (o,tap) of w is a row vector over input channels: (H^T W)[c,o] = sum_j H[j][c] w[o][j] */
    int rc = hqo_transform(w, N * RS, C, had_block, wt);   /* H symmetric: row * H == H^T * column */
    if (rc == 0) rc = hqo_weight_quantize(wt, N, RS * C, w_bits, B, s_w);
    free(wt);
    return rc;
}

/* B = 256*hi + lo with lo in [-128,127] ("balanced" low limb).  Returns 0, or -1 if some hi
 * does not fit a signed byte. */
int hqo_limb_split(const int32_t* B, i64 count, int8_t* hi, int8_t* lo) {
    for (i64 i = 0; i < count; ++i) {
        int32_t v = B[i];
        int32_t l = ((v + 128) & 255) - 128;        /* v + 128 mod 256, two's complement & is a true mod */
        int32_t h = (v - l) / 256;
        if (h < -128 || h > 127) return -1;
        hi[i] = (int8_t)h;
        lo[i] = (int8_t)l;
    }
    return 0;
}

/* The integer product of Eq. 12: acc[m][o] = sum_k q[m][k] * B[o][k].  Returns the number of
 * accumulators that do not fit int32 (0 = all fit). */
i64 hqo_gemm_int(const int8_t* q, const int32_t* B, i64 M, i64 N, i64 K, i64* acc) {
    i64 bad = 0;
#pragma omp parallel for schedule(static) reduction(+ : bad)
    for (i64 m = 0; m < M; ++m) {
        for (i64 o = 0; o < N; ++o) {
            i64 t = 0;
            for (i64 k = 0; k < K; ++k) t += (i64)q[m * K + k] * (i64)B[o * K + k];
            acc[m * N + o] = t;
            if (t > 2147483647LL || t < -2147483648LL) ++bad;
        }
    }
    return bad;
}

/* The integer convolution of Eq. 14 with the transform on the channel axis:
 * acc[n][ho][wo][co] = sum_{r,s,ci} q[n][ho*st + r - p][wo*st + s - p][ci] * B[co][r][s][ci], zero outside.
 * q NHWC [Nb][H][W][C], B [Cout][R][S][C], acc [Nb][Ho][Wo][Cout], Ho = (H + 2p - R)/st + 1. */
i64 hqo_conv2d_int(const int8_t* q, const int32_t* B, i64 Nb, i64 H, i64 W, i64 C, i64 Cout,
                   int R, int S, int stride, int pad, i64* acc) {
    const i64 Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - S) / stride + 1;
    i64 bad = 0;
#pragma omp parallel for schedule(static) reduction(+ : bad)
    for (i64 nho = 0; nho < Nb * Ho; ++nho) {
        const i64 n = nho / Ho, ho = nho % Ho;
        for (i64 wo = 0; wo < Wo; ++wo) {
            for (i64 co = 0; co < Cout; ++co) {
                i64 t = 0;
                for (int r = 0; r < R; ++r) {
                    for (int s = 0; s < S; ++s) {
                        const i64 hi = ho * stride + r - pad, wi = wo * stride + s - pad;
                        if (hi < 0 || hi >= H || wi < 0 || wi >= W) continue;
                        for (i64 ci = 0; ci < C; ++ci)
                            t += (i64)q[((n * H + hi) * W + wi) * C + ci] * (i64)B[((co * R + r) * S + s) * C + ci];
                    }
                }
                acc[((n * Ho + ho) * Wo + wo) * Cout + co] = t;
                if (t > 2147483647LL || t < -2147483648LL) ++bad;
            }
        }
    }
    return bad;
}

/* The rescale in front of the integer product in Eq. 12 / Eq. 14, plus a bias:
 * y[m][o] = alpha * S_a[m] * S_w[o] * acc[m][o] + bias[o]   (S_a one scalar if sa_is_scalar). */
int hqo_dequant(const i64* acc, i64 M, i64 N, const float* s_a, int sa_is_scalar, const float* s_w,
                const float* bias, double alpha, double* y) {
#pragma omp parallel for schedule(static)
    for (i64 m = 0; m < M; ++m) {
        const double sa = (double)(sa_is_scalar ? s_a[0] : s_a[m]);
        for (i64 o = 0; o < N; ++o)
            y[m * N + o] = alpha * sa * (double)s_w[o] * (double)acc[m * N + o] + (bias ? (double)bias[o] : 0.0);
    }
    return 0;
}

/* Convolution whose input pixels each carry their own scale.  The scale of the pixel a tap
 * reads does not factor out of the sum over taps, so each tap's integer sum is rescaled by
 * the scale of the pixel it read:
 * y[n][ho][wo][co] = alpha * S_w[co] * sum_{r,s} S_a[pix(r,s)] * (sum_ci q[pix][ci] * B[co][r][s][ci]) + bias[co]. */
int hqo_conv2d_dequant_perpixel(const int8_t* q, const float* s_a, const int32_t* B, i64 Nb, i64 H, i64 W,
                                i64 C, i64 Cout, int R, int S, int stride, int pad, const float* s_w,
                                const float* bias, double alpha, double* y) {
    const i64 Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - S) / stride + 1;
#pragma omp parallel for schedule(static)
    for (i64 nho = 0; nho < Nb * Ho; ++nho) {
        const i64 n = nho / Ho, ho = nho % Ho;
        for (i64 wo = 0; wo < Wo; ++wo) {
            for (i64 co = 0; co < Cout; ++co) {
                double sum = 0.0;
                for (int r = 0; r < R; ++r) {
                    for (int s = 0; s < S; ++s) {
                        const i64 hi = ho * stride + r - pad, wi = wo * stride + s - pad;
                        if (hi < 0 || hi >= H || wi < 0 || wi >= W) continue;
                        const i64 pix = (n * H + hi) * W + wi;
                        i64 t = 0;
                        for (i64 ci = 0; ci < C; ++ci)
                            t += (i64)q[pix * C + ci] * (i64)B[((co * R + r) * S + s) * C + ci];
                        sum += (double)s_a[pix] * (double)t;
                    }
                }
                y[((n * Ho + ho) * Wo + wo) * Cout + co] =
                    alpha * (double)s_w[co] * sum + (bias ? (double)bias[co] : 0.0);
            }
        }
    }
    return 0;
}

/* ---- Convolution with the transform on the WIDTH axis, as Eq. 13-14 state it ------------------------------
 * The paper reshapes X_c [B][Cin][h][w] to (B*Cin*h) x w and multiplies by the block-diagonal H_c (w x w) from
 * the right, i.e. every image row of every channel is transformed along w.  Here tensors are NHWC, so the w
 * axis has stride C; the arithmetic is the same.
 *
 * u[n][h][b*nb + j][c] = 2^(-k/2) * sum_i x[n][h][b*nb + i][c] * H_raw[i][j]      (nb = 2^k = had_block) */
int hqo_transform_width(const double* x, i64 Nb, i64 H, i64 W, i64 C, int had_block, double* u) {
    if (had_block <= 1) { memcpy(u, x, sizeof(double) * (size_t)(Nb * H * W * C)); return 0; }
    const int n = had_block;
    if (!is_pow2(n) || W % n != 0) return -1;
    int8_t* Hm = (int8_t*)malloc((size_t)n * n);
    if (!Hm) return -2;
    hqo_hadamard_raw(n, Hm);
    const double norm = pow(2.0, -0.5 * (double)ilog2(n));
#pragma omp parallel for schedule(static)
    for (i64 nh = 0; nh < Nb * H; ++nh) {
        for (i64 b = 0; b < W / n; ++b) {
            for (i64 c = 0; c < C; ++c) {
                for (int j = 0; j < n; ++j) {
                    double t = 0.0;
                    for (int i = 0; i < n; ++i) t += x[(nh * W + b * n + i) * C + c] * (double)Hm[(i64)i * n + j];
                    u[(nh * W + b * n + j) * C + c] = t * norm;
                }
            }
        }
    }
    free(Hm);
    return 0;
}

/* The integer factor "(X H_c)_int * H_c" of Eq. 14 with the raw +-1 matrix (its 2^(-k/2) goes to the scale):
 * z[n][h][b*nb + j][c] = sum_i q[n][h][b*nb + i][c] * H_raw[i][j], exact integers, |z| <= nb * max|q|. */
int hqo_codes_inverse_width(const int8_t* q, i64 Nb, i64 H, i64 W, i64 C, int had_block, int32_t* z) {
    const int n = had_block > 1 ? had_block : 1;
    if (!is_pow2(n) || W % n != 0) return -1;
    int8_t* Hm = (int8_t*)malloc((size_t)n * n);
    if (!Hm) return -2;
    hqo_hadamard_raw(n, Hm);
#pragma omp parallel for schedule(static)
    for (i64 nh = 0; nh < Nb * H; ++nh) {
        for (i64 b = 0; b < W / n; ++b) {
            for (i64 c = 0; c < C; ++c) {
                for (int j = 0; j < n; ++j) {
                    i64 t = 0;
                    for (int i = 0; i < n; ++i) t += (i64)q[(nh * W + b * n + i) * C + c] * (i64)Hm[(i64)i * n + j];
                    z[(nh * W + b * n + j) * C + c] = (int32_t)t;
                }
            }
        }
    }
    free(Hm);
    return 0;
}

/* The integer convolution of Eq. 14 on 32-bit integer activations z (NHWC) and integer weights B [Cout][R][S][C]:
 * same sum as hqo_conv2d_int.  Returns the number of accumulators that do not fit int32. */
i64 hqo_conv2d_int_z(const int32_t* z, const int32_t* B, i64 Nb, i64 H, i64 W, i64 C, i64 Cout,
                     int R, int S, int stride, int pad, i64* acc) {
    const i64 Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - S) / stride + 1;
    i64 bad = 0;
#pragma omp parallel for schedule(static) reduction(+ : bad)
    for (i64 nho = 0; nho < Nb * Ho; ++nho) {
        const i64 n = nho / Ho, ho = nho % Ho;
        for (i64 wo = 0; wo < Wo; ++wo) {
            for (i64 co = 0; co < Cout; ++co) {
                i64 t = 0;
                for (int r = 0; r < R; ++r) {
                    for (int s = 0; s < S; ++s) {
                        const i64 hi = ho * stride + r - pad, wi = wo * stride + s - pad;
                        if (hi < 0 || hi >= H || wi < 0 || wi >= W) continue;
                        for (i64 ci = 0; ci < C; ++ci)
                            t += (i64)z[((n * H + hi) * W + wi) * C + ci] * (i64)B[((co * R + r) * S + s) * C + ci];
                    }
                }
                acc[((n * Ho + ho) * Wo + wo) * Cout + co] = t;
                if (t > 2147483647LL || t < -2147483648LL) ++bad;
            }
        }
    }
    return bad;
}

/* ---- LayerNorm with a per-sample affine in front of a quantized linear (the "modulate(norm(x), shift, scale)" of a
 * diffusion-transformer block) ---------------------------------------------------------------------------------
 * Not part of the paper's equations: the usual definition, written out.  x [rows][cols]; per row: mean and biased
 * variance over the cols values; y = (x - mean) / sqrt(var + eps) * w[g][c] + b[g][c], where g = row / rows_per_group
 * selects the affine vectors of the row's sample (rows_per_group <= 0: one vector pair for all rows).
 * w == NULL means 1, b == NULL means 0. */
int hqo_layernorm_affine(const double* x, i64 rows, i64 cols, const double* w, const double* b, i64 rows_per_group,
                         double eps, double* out) {
    if (rows < 0 || cols <= 0) return -1;
#pragma omp parallel for schedule(static)
    for (i64 r = 0; r < rows; ++r) {
        const double* xr = x + r * cols;
        double sum = 0.0;
        for (i64 c = 0; c < cols; ++c) sum += xr[c];
        const double mean = sum / (double)cols;
        double var = 0.0;
        for (i64 c = 0; c < cols; ++c) { const double d = xr[c] - mean; var += d * d; }
        var /= (double)cols;
        const double rstd = 1.0 / sqrt(var + eps);
        const i64 g = rows_per_group > 0 ? r / rows_per_group : 0;
        for (i64 c = 0; c < cols; ++c) {
            const double wc = w ? w[g * cols + c] : 1.0, bc = b ? b[g * cols + c] : 0.0;
            out[r * cols + c] = (xr[c] - mean) * rstd * wc + bc;
        }
    }
    return 0;
}

/* ---- GroupNorm + SiLU in front of a quantized convolution (the "in_layers" of a ResBlock) -------------------
 * Not part of the paper's equations: the usual definitions, written out.  x NHWC [Nb][H][W][C], `groups` groups of
 * C/groups consecutive channels; per sample and group: mean and biased variance over H*W*(C/groups) values;
 * y = (x - mean) / sqrt(var + eps) * gamma[c] + beta[c];   out = y * sigmoid(y) = y / (1 + exp(-y)). */
int hqo_groupnorm_silu(const double* x, i64 Nb, i64 H, i64 W, i64 C, int groups, const double* gamma,
                       const double* beta, double eps, double* out) {
    if (groups <= 0 || C % groups != 0) return -1;
    const i64 cg = C / groups, HW = H * W;
#pragma omp parallel for schedule(static)
    for (i64 ng = 0; ng < Nb * groups; ++ng) {
        const i64 n = ng / groups, g = ng % groups;
        double sum = 0.0;
        for (i64 p = 0; p < HW; ++p)
            for (i64 c = 0; c < cg; ++c) sum += x[(n * HW + p) * C + g * cg + c];
        const double mean = sum / (double)(HW * cg);
        double var = 0.0;
        for (i64 p = 0; p < HW; ++p)
            for (i64 c = 0; c < cg; ++c) { const double d = x[(n * HW + p) * C + g * cg + c] - mean; var += d * d; }
        var /= (double)(HW * cg);
        const double rstd = 1.0 / sqrt(var + eps);
        for (i64 p = 0; p < HW; ++p)
            for (i64 c = 0; c < cg; ++c) {
                const i64 ch = g * cg + c, idx = (n * HW + p) * C + ch;
                const double y = (x[idx] - mean) * rstd * gamma[ch] + beta[ch];
                out[idx] = y / (1.0 + exp(-y));
            }
    }
    return 0;
}

/* ==== The operations around the quantized layers of the noise-prediction network =================================
 * The method replaces every linear and convolution of the network (overview figure of the framework); what sits
 * between them is the network's own, unquantized arithmetic.  None of it is in the paper's equations: each function
 * below is the usual definition written out in fp64, pinned against torch's CPU routines and closed forms. */

/* GroupNorm as above with the activation selectable: act = 0 none (the normalisation in front of an attention
 * block's QKV projection), act = 1 SiLU. */
int hqo_groupnorm(const double* x, i64 Nb, i64 H, i64 W, i64 C, int groups, const double* gamma, const double* beta,
                  double eps, int act, double* out) {
    if (groups <= 0 || C % groups != 0 || (act != 0 && act != 1)) return -1;
    const i64 cg = C / groups, HW = H * W;
#pragma omp parallel for schedule(static)
    for (i64 ng = 0; ng < Nb * groups; ++ng) {
        const i64 n = ng / groups, g = ng % groups;
        double sum = 0.0;
        for (i64 p = 0; p < HW; ++p)
            for (i64 c = 0; c < cg; ++c) sum += x[(n * HW + p) * C + g * cg + c];
        const double mean = sum / (double)(HW * cg);
        double var = 0.0;
        for (i64 p = 0; p < HW; ++p)
            for (i64 c = 0; c < cg; ++c) { const double d = x[(n * HW + p) * C + g * cg + c] - mean; var += d * d; }
        var /= (double)(HW * cg);
        const double rstd = 1.0 / sqrt(var + eps);
        for (i64 p = 0; p < HW; ++p)
            for (i64 c = 0; c < cg; ++c) {
                const i64 ch = g * cg + c, idx = (n * HW + p) * C + ch;
                const double y = (x[idx] - mean) * rstd * gamma[ch] + beta[ch];
                out[idx] = act ? y / (1.0 + exp(-y)) : y;
            }
    }
    return 0;
}

/* Multi-head self-attention core.  qkv [Nb][L][3*C]: for token t the query, key and value vectors of head h are
 * qkv[t][h*dh .. ], qkv[t][C + h*dh ..], qkv[t][2C + h*dh ..], dh = C / heads.  Per sample and head:
 * out[i] = sum_j softmax_j(q_i . k_j / sqrt(dh)) v_j,  written to out [Nb][L][C] at columns h*dh .. */
int hqo_attention(const double* qkv, i64 Nb, i64 L, i64 C, int heads, double* out) {
    if (heads <= 0 || C % heads != 0 || L <= 0) return -1;
    const i64 dh = C / heads;
    const double scale = 1.0 / sqrt((double)dh);
#pragma omp parallel for schedule(static)
    for (i64 nh = 0; nh < Nb * heads; ++nh) {
        const i64 n = nh / heads, h = nh % heads;
        double* s = (double*)malloc((size_t)L * sizeof(double));
        for (i64 i = 0; i < L; ++i) {
            const double* q = qkv + (n * L + i) * 3 * C + h * dh;
            double mx = -INFINITY;
            for (i64 j = 0; j < L; ++j) {
                const double* k = qkv + (n * L + j) * 3 * C + C + h * dh;
                double dot = 0.0;
                for (i64 d = 0; d < dh; ++d) dot += q[d] * k[d];
                s[j] = dot * scale;
                if (s[j] > mx) mx = s[j];
            }
            double den = 0.0;
            for (i64 j = 0; j < L; ++j) { s[j] = exp(s[j] - mx); den += s[j]; }
            double* o = out + (n * L + i) * C + h * dh;
            for (i64 d = 0; d < dh; ++d) {
                double acc = 0.0;
                for (i64 j = 0; j < L; ++j) acc += s[j] * qkv[(n * L + j) * 3 * C + 2 * C + h * dh + d];
                o[d] = acc / den;
            }
        }
        free(s);
    }
    return 0;
}

/* Nearest-neighbour up-sampling by two: out[n][2h+i][2w+j][c] = x[n][h][w][c], i, j in {0, 1}. */
int hqo_upsample_nearest2x(const double* x, i64 Nb, i64 H, i64 W, i64 C, double* out) {
    for (i64 n = 0; n < Nb; ++n)
        for (i64 ho = 0; ho < 2 * H; ++ho)
            for (i64 wo = 0; wo < 2 * W; ++wo)
                for (i64 c = 0; c < C; ++c)
                    out[((n * 2 * H + ho) * 2 * W + wo) * C + c] = x[((n * H + ho / 2) * W + wo / 2) * C + c];
    return 0;
}

/* Sinusoidal embedding of the denoising step: for i < dim/2, f_i = exp(-ln(max_period) * i / (dim/2));
 * out[n][i] = cos(t[n] * f_i), out[n][dim/2 + i] = sin(t[n] * f_i).  dim even. */
int hqo_timestep_embedding(const double* t, i64 Nb, i64 dim, double max_period, double* out) {
    if (dim <= 0 || (dim & 1)) return -1;
    const i64 half = dim / 2;
    for (i64 n = 0; n < Nb; ++n)
        for (i64 i = 0; i < half; ++i) {
            const double f = exp(-log(max_period) * (double)i / (double)half);
            out[n * dim + i] = cos(t[n] * f);
            out[n * dim + half + i] = sin(t[n] * f);
        }
    return 0;
}

/* Floating-point convolution (the network's first and last convolution, which the method leaves unquantized):
 * x NHWC, w [Cout][R][S][C], zero padding; out[n][ho][wo][co] = bias[co] + sum x[n][ho*st+r-p][wo*st+s-p][c] w[co][r][s][c]. */
int hqo_conv2d_float(const double* x, const double* w, const double* bias, i64 Nb, i64 H, i64 W, i64 C, i64 Cout,
                     int R, int S, int stride, int pad, double* out) {
    const i64 Ho = (H + 2 * pad - R) / stride + 1, Wo = (W + 2 * pad - S) / stride + 1;
    if (Ho <= 0 || Wo <= 0) return -1;
#pragma omp parallel for schedule(static)
    for (i64 nho = 0; nho < Nb * Ho; ++nho) {
        const i64 n = nho / Ho, ho = nho % Ho;
        for (i64 wo = 0; wo < Wo; ++wo)
            for (i64 co = 0; co < Cout; ++co) {
                double t = bias ? bias[co] : 0.0;
                for (int r = 0; r < R; ++r) {
                    const i64 hi = ho * stride + r - pad;
                    if (hi < 0 || hi >= H) continue;
                    for (int s = 0; s < S; ++s) {
                        const i64 wi = wo * stride + s - pad;
                        if (wi < 0 || wi >= W) continue;
                        for (i64 c = 0; c < C; ++c)
                            t += x[((n * H + hi) * W + wi) * C + c] * w[((co * R + r) * S + s) * C + c];
                    }
                }
                out[((n * Ho + ho) * Wo + wo) * Cout + co] = t;
            }
    }
    return 0;
}
