/*
 * CPU oracle for the fully binary CNN-style 2D convolution.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * operator computes.  It shares no code, header, table or helper with the CUDA
 * library and must never be called from the product path; only the tests, the
 * smoke check and the CPU-baseline leg of the benchmark may execute it.
 *
 * Everything works on UNPACKED tensors: one int8 per element holding -1 or +1.
 * There are no bit tricks here on purpose, so that each loop can be checked by
 * eye against the paper:
 *   - Section 1: the CNN-style 2D convolution takes a 3D input tensor and a 4D
 *     weight tensor and yields a 3D output tensor, and lowers to a matrix-matrix
 *     product.
 *   - Section 4.2.1: activations pass through a learnable bias and a sign, every
 *     feature is +1 or -1 and every weight is +1 or -1.
 *   - Section 5.2 / Figure 5: the weights used in the forward pass are the sign
 *     of the real weights.
 *   - Section 4.2.1: the convolution is followed by a per-channel scale and bias
 *     (batch norm) and the next module's bias + sign; with integer accumulators
 *     that chain is one integer comparison per output channel (threshold).
 *
 * Readings taken where the paper is silent:
 *   - sign(v) = +1 when v >= 0 (so -0.0 -> +1, NaN -> -1), else -1;
 *   - out-of-image taps read the value -1 (a +-1 tensor has no zero);
 *   - weights are laid out [C_out][kh][kw][C_in], activations [B][H][W][C];
 *   - output extent floor((H + 2*pad - kh)/stride) + 1;
 *   - channel replication by R: output channel c reads input channel c mod C_in;
 *   - threshold compare is acc >= thr -> +1.
 *
 * The only parallelism is an OpenMP loop over independent outputs; the order of
 * the additions inside one output is the textual one (integers: order is moot).
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* sign with bias, Section 4.2.1 (bias then sign); fp32 add, then compare. */
static inline int8_t sign_pm1(float v)
{
    return (v >= 0.0f) ? (int8_t)1 : (int8_t)-1;
}

/*
 * Binarize activations: out[b][h][w][c] = sign(x[b][h][w][c mod C_in] + bias[c]),
 * c in [0, R*C_in).  bias may be NULL (treated as 0).  x is real NHWC fp32.
 */
void oracle_binarize(const float *x, const float *bias, int8_t *out,
                     int B, int H, int W, int C_in, int R)
{
    const int C = C_in * R;
    const long npix = (long)B * H * W;
#pragma omp parallel for schedule(static)
    for (long p = 0; p < npix; ++p) {
        for (int c = 0; c < C; ++c) {
            volatile float s = x[p * C_in + (c % C_in)];
            if (bias) s = s + bias[c];
            out[p * C + c] = sign_pm1(s);
        }
    }
}

/* Section 5.2: binary weights are the sign of the real weights. */
void oracle_sign_weights(const float *w, int8_t *out, long n)
{
    for (long i = 0; i < n; ++i) out[i] = sign_pm1(w[i]);
}

/*
 * One output of the direct +-1 convolution (Section 1 operator with the
 * Section 4.2.1 operands): the sum over the kh*kw taps and the C_in channels of
 * activation * weight, where an out-of-image tap has activation -1.
 *   x : int8 [B][H][W][C_in]        values in {-1,+1}
 *   w : int8 [C_out][kh][kw][C_in]  values in {-1,+1}
 */
static int32_t conv_one_output(const int8_t *x, const int8_t *w,
                               int b, int oh, int ow, int co,
                               int H, int W, int C_in,
                               int kh, int kw, int stride, int pad)
{
    int32_t acc = 0;
    for (int r = 0; r < kh; ++r) {
        for (int t = 0; t < kw; ++t) {
            const int ih = oh * stride - pad + r;
            const int iw = ow * stride - pad + t;
            const int inside = (ih >= 0 && ih < H && iw >= 0 && iw < W);
            for (int ci = 0; ci < C_in; ++ci) {
                const int v = inside
                    ? x[(((long)b * H + ih) * W + iw) * C_in + ci]
                    : -1;
                const int g = w[(((long)co * kh + r) * kw + t) * C_in + ci];
                acc += v * g;
            }
        }
    }
    return acc;
}

/* Whole output tensor y : int32 [B][OH][OW][C_out]. */
void oracle_conv2d(const int8_t *x, const int8_t *w, int32_t *y,
                   int B, int H, int W, int C_in, int C_out,
                   int kh, int kw, int stride, int pad)
{
    const int OH = (H + 2 * pad - kh) / stride + 1;
    const int OW = (W + 2 * pad - kw) / stride + 1;
    const long nout = (long)B * OH * OW;
#pragma omp parallel for schedule(static)
    for (long o = 0; o < nout; ++o) {
        const int b = (int)(o / ((long)OH * OW));
        const int oh = (int)((o / OW) % OH);
        const int ow = (int)(o % OW);
        for (int co = 0; co < C_out; ++co)
            y[o * C_out + co] = conv_one_output(x, w, b, oh, ow, co, H, W, C_in,
                                                kh, kw, stride, pad);
    }
}

/*
 * The same outputs, but only for the listed output pixels: pix[i] is a flat
 * index into [B][OH][OW]; y : int32 [npix][C_out].  Used to check sampled
 * outputs of workloads too large to compute in full.
 */
void oracle_conv2d_pixels(const int8_t *x, const int8_t *w, const int64_t *pix,
                          long npix, int32_t *y,
                          int B, int H, int W, int C_in, int C_out,
                          int kh, int kw, int stride, int pad)
{
    const int OH = (H + 2 * pad - kh) / stride + 1;
    const int OW = (W + 2 * pad - kw) / stride + 1;
    (void)B;
#pragma omp parallel for schedule(static)
    for (long i = 0; i < npix; ++i) {
        const long o = pix[i];
        const int b = (int)(o / ((long)OH * OW));
        const int oh = (int)((o / OW) % OH);
        const int ow = (int)(o % OW);
        for (int co = 0; co < C_out; ++co)
            y[i * C_out + co] = conv_one_output(x, w, b, oh, ow, co, H, W, C_in,
                                                kh, kw, stride, pad);
    }
}

/*
 * Matrix-matrix product the convolution lowers to (Section 1):
 *   C[m][n] = sum_k A[m][k] * Wt[n][k],  A int8 [M][K], Wt int8 [N][K] (+-1).
 */
void oracle_gemm(const int8_t *A, const int8_t *Wt, int32_t *C,
                 long M, long N, long K)
{
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        for (long n = 0; n < N; ++n) {
            int32_t acc = 0;
            for (long k = 0; k < K; ++k)
                acc += (int)A[m * K + k] * (int)Wt[n * K + k];
            C[m * N + n] = acc;
        }
    }
}

/*
 * Per-output-channel integer threshold (batch norm + next bias + sign folded to
 * one comparison, Section 4.2.1): out[i][n] = (acc[i][n] >= thr[n]) ? +1 : -1.
 */
void oracle_threshold(const int32_t *acc, const int32_t *thr, int8_t *out,
                      long rows, long N)
{
#pragma omp parallel for schedule(static)
    for (long i = 0; i < rows; ++i)
        for (long n = 0; n < N; ++n)
            out[i * N + n] = (acc[i * N + n] >= thr[n]) ? (int8_t)1 : (int8_t)-1;
}

/*
 * The convolution module around a binary convolution (Section 4.2.1, Figure 4 top), applied to the
 * convolution's integer result acc:
 *   t = acc * scale[n] + shift[n]          batch norm as a per-channel scale and bias
 *   u = t + identity                       the module's real input, carried around the binary conv
 *   r = (u >= 0) ? u : slope[n] * u        PReLU with a per-channel slope
 *   y = fp16(r)                            the real feature map as it is stored
 *   s = (y + next_bias[n] >= 0) ? +1 : -1  the next module's bias + sign, taken of the STORED value
 * Every step is one fp32 operation rounded to nearest even (no fused multiply-add: this file is
 * compiled with -ffp-contract=off); the conversion to fp16 rounds to nearest even.  identity (fp16
 * bit patterns, may be NULL = no identity path) and y are [rows][N]; s may be NULL.
 */
void oracle_conv_module(const int32_t *acc, const float *scale, const float *shift,
                        const uint16_t *identity, const float *slope, const float *next_bias,
                        uint16_t *y, int8_t *s, long rows, long N)
{
#pragma omp parallel for schedule(static)
    for (long i = 0; i < rows; ++i)
        for (long n = 0; n < N; ++n) {
            const long k = i * N + n;
            float t = (float)acc[k] * scale[n];
            t = t + shift[n];
            float u = t;
            if (identity) {
                _Float16 hi;
                memcpy(&hi, &identity[k], sizeof hi);
                u = t + (float)hi;
            }
            const float r = (u >= 0.0f) ? u : slope[n] * u;
            const _Float16 h = (_Float16)r;
            memcpy(&y[k], &h, sizeof h);
            if (s) {
                const float v = (float)h + (next_bias ? next_bias[n] : 0.0f);
                s[k] = (v >= 0.0f) ? (int8_t)1 : (int8_t)-1;
            }
        }
}
