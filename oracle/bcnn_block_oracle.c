/*
 * CPU oracle for the rest of the paper's building block around the binary convolutions.
 *
 * TEST INFRASTRUCTURE ONLY (see bcnn_oracle.c): plain loops, no code shared with the CUDA library, never called
 * from the product path.
 *
 *   - Section 4.2.1, Figure 4 bottom: P parallel binary residual branches inside a convolution module, each with
 *     its own learned bias (its own binarization), binary weights and batch norm; the branches are summed before
 *     the module's identity addition and PReLU.  The same structure with P = F*F branches, each looking at a
 *     shifted, zero-padded copy of the real map, stands for a binary F x F convolution (last paragraph of 4.2.1).
 *   - Section 4.2.1, "3x3 convolution module": real 3x3 depth-wise convolution (stride S), batch norm, PReLU.
 *   - Section 4.2.2: channel replication by an integer factor R is bookkeeping: channel c reads channel c mod C_in.
 *   - Section 4.2.3: S x S / S average pooling on the identity path of a down-sampling block.
 *   - Section 4.1, Figure 2, Table 1 (last rows): global average pooling and a fully connected layer.
 *
 * Precision.  The branch module extends oracle_conv_module and keeps its convention: one fp32 operation per step,
 * rounded to nearest, in the stated order, fp16 storage (bit-exact parity).  The real-valued vector operations
 * (depth-wise convolution, pooling, fully connected layer) are written in fp64, results rounded once to the
 * storage type; parity for those is within a stated tolerance.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>

static inline double h2d(uint16_t bits)
{
    _Float16 h;
    memcpy(&h, &bits, sizeof h);
    return (double)h;
}

static inline uint16_t d2h(double v)
{
    const _Float16 h = (_Float16)v;          /* one rounding, to nearest even */
    uint16_t bits;
    memcpy(&bits, &h, sizeof bits);
    return bits;
}

/*
 * Convolution module with P parallel binary branches (Figure 4 bottom), applied to the branches' integer
 * convolution results acc[p] (each [rows][N]):
 *   t_p = acc_p * scale_p[n] + shift_p[n]           batch norm of branch p          (two fp32 operations)
 *   t   = ((t_0 + t_1) + t_2) + ...                 branches summed in branch order (fp32, left to right)
 *   u   = t + identity;  r = (u >= 0) ? u : slope[n] * u;  y = fp16(r);  s = (y + next_bias[n] >= 0) ? +1 : -1
 * exactly as oracle_conv_module from there on (P = 1 is that function).
 */
void oracle_conv_module_branches(const int32_t *acc, const float *scale, const float *shift,
                                 const uint16_t *identity, const float *slope, const float *next_bias,
                                 uint16_t *y, int8_t *s, long rows, long N, int P)
{
#pragma omp parallel for schedule(static)
    for (long i = 0; i < rows; ++i)
        for (long n = 0; n < N; ++n) {
            const long k = i * N + n;
            float t = 0.0f;
            for (int p = 0; p < P; ++p) {
                float tp = (float)acc[(long)p * rows * N + k] * scale[(long)p * N + n];
                tp = tp + shift[(long)p * N + n];
                t = (p == 0) ? tp : t + tp;
            }
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

/*
 * 3x3 convolution module: real depth-wise 3x3 convolution with stride S and zero padding 1, batch norm, PReLU.
 *   x : fp16 [B][H][W][C_in];  output channel c (of C = R * C_in) reads input channel c mod C_in (replication)
 *   w : fp32 [C][3][3];  scale, shift, slope : fp32 [C]
 *   y : fp16 [B][OH][OW][C],  OH = (H + 2 - 3) / S + 1
 *   conv = sum_{r,t} xpad[oh*S - 1 + r][ow*S - 1 + t][c mod C_in] * w[c][r][t]     (xpad = 0 outside)
 *   t = conv * scale[c] + shift[c];  y = fp16(t >= 0 ? t : slope[c] * t)            all in fp64, one rounding
 */
void oracle_dwconv3x3_module(const uint16_t *x, const float *w, const float *scale, const float *shift,
                             const float *slope, uint16_t *y, int B, int H, int W, int C_in, int R, int S)
{
    const int C = C_in * R;
    const int OH = (H + 2 - 3) / S + 1, OW = (W + 2 - 3) / S + 1;
    const long nout = (long)B * OH * OW;
#pragma omp parallel for schedule(static)
    for (long o = 0; o < nout; ++o) {
        const int b = (int)(o / ((long)OH * OW));
        const int oh = (int)((o / OW) % OH), ow = (int)(o % OW);
        for (int c = 0; c < C; ++c) {
            double conv = 0.0;
            for (int r = 0; r < 3; ++r)
                for (int t = 0; t < 3; ++t) {
                    const int ih = oh * S - 1 + r, iw = ow * S - 1 + t;
                    if (ih < 0 || ih >= H || iw < 0 || iw >= W) continue;
                    conv += h2d(x[(((long)b * H + ih) * W + iw) * C_in + (c % C_in)]) * (double)w[(c * 3 + r) * 3 + t];
                }
            const double tt = conv * (double)scale[c] + (double)shift[c];
            y[o * C + c] = d2h(tt >= 0.0 ? tt : (double)slope[c] * tt);
        }
    }
}

/*
 * S x S average pooling with stride S (H and W multiples of S), with channel replication:
 *   y[b][oh][ow][c] = fp16( mean over the S x S window of x[..][c mod C_in] )        fp64 mean, one rounding
 */
void oracle_avgpool(const uint16_t *x, uint16_t *y, int B, int H, int W, int C_in, int R, int S)
{
    const int C = C_in * R, OH = H / S, OW = W / S;
    const long nout = (long)B * OH * OW;
#pragma omp parallel for schedule(static)
    for (long o = 0; o < nout; ++o) {
        const int b = (int)(o / ((long)OH * OW));
        const int oh = (int)((o / OW) % OH), ow = (int)(o % OW);
        for (int c = 0; c < C; ++c) {
            double sum = 0.0;
            for (int r = 0; r < S; ++r)
                for (int t = 0; t < S; ++t)
                    sum += h2d(x[(((long)b * H + oh * S + r) * W + ow * S + t) * C_in + (c % C_in)]);
            y[o * C + c] = d2h(sum / (double)(S * S));
        }
    }
}

/* Global average pooling: out[b][c] = mean over the HW pixels of x[b][.][c]   (fp16 in, fp64 out). */
void oracle_gap(const uint16_t *x, double *out, int B, long HW, int C)
{
    for (int b = 0; b < B; ++b)
        for (int c = 0; c < C; ++c) {
            double sum = 0.0;
            for (long i = 0; i < HW; ++i) sum += h2d(x[((long)b * HW + i) * C + c]);
            out[(long)b * C + c] = sum / (double)HW;
        }
}

/* Fully connected layer: logits[b][n] = sum_c pooled[b][c] * w[n][c] + bias[n]   (fp64). */
void oracle_fc(const double *pooled, const float *w, const float *bias, double *logits, int B, int C, int N)
{
#pragma omp parallel for schedule(static)
    for (int b = 0; b < B; ++b)
        for (int n = 0; n < N; ++n) {
            double sum = 0.0;
            for (int c = 0; c < C; ++c) sum += pooled[(long)b * C + c] * (double)w[(long)n * C + c];
            logits[(long)b * N + n] = sum + (bias ? (double)bias[n] : 0.0);
        }
}
