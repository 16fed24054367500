/*
 * Bit-packed CPU checker (TEST INFRASTRUCTURE ONLY; not the oracle).
 *
 * The oracle in bcnn_oracle.c is the definition and is authoritative, but it is
 * O(M*N*K) scalar work and cannot cover every output of the largest workloads.
 * This second CPU program computes the same integers from packed sign bits
 * (bit 1 = +1, bit 0 = -1) so that full-size GPU outputs can be compared in
 * seconds.  It is trusted only because the CPU tests prove it equal to the
 * oracle on shapes the oracle finishes.  It shares no code with the CUDA
 * library.
 *
 * For +-1 vectors a, g of length n with sign-bit strings A, G:
 * products equal to -1 are exactly the positions where the bits differ, so
 * sum a*g = n - 2*popcount(A xor G).  An out-of-image tap is the all -1 vector,
 * i.e. the all-zero bit string.
 */
#include <stdint.h>
#include <stddef.h>

/* x : uint32 words, [B][H][W][C_in/32]; w : [C_out][kh][kw][C_in/32]. */
void checker_conv2d(const uint32_t *x, const uint32_t *w, int32_t *y,
                    int B, int H, int W, int C_in, int C_out,
                    int kh, int kw, int stride, int pad)
{
    const int OH = (H + 2 * pad - kh) / stride + 1;
    const int OW = (W + 2 * pad - kw) / stride + 1;
    const int cw = C_in / 32;
    const long nout = (long)B * OH * OW;
#pragma omp parallel for schedule(static)
    for (long o = 0; o < nout; ++o) {
        const int b = (int)(o / ((long)OH * OW));
        const int oh = (int)((o / OW) % OH);
        const int ow = (int)(o % OW);
        for (int co = 0; co < C_out; ++co) {
            int differ = 0;
            for (int r = 0; r < kh; ++r)
                for (int t = 0; t < kw; ++t) {
                    const int ih = oh * stride - pad + r;
                    const int iw = ow * stride - pad + t;
                    const uint32_t *g = w + (((long)co * kh + r) * kw + t) * cw;
                    if (ih >= 0 && ih < H && iw >= 0 && iw < W) {
                        const uint32_t *a = x + (((long)b * H + ih) * W + iw) * cw;
                        for (int j = 0; j < cw; ++j)
                            differ += __builtin_popcount(a[j] ^ g[j]);
                    } else {
                        for (int j = 0; j < cw; ++j)
                            differ += __builtin_popcount(g[j]);
                    }
                }
            y[o * C_out + co] = kh * kw * C_in - 2 * differ;
        }
    }
}

/* A : [M][K/32] words, Wt : [N][K/32] words, C : int32 [M][N]. */
void checker_gemm(const uint32_t *A, const uint32_t *Wt, int32_t *C,
                  long M, long N, long K)
{
    const long kw = K / 32;
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m)
        for (long n = 0; n < N; ++n) {
            int differ = 0;
            for (long j = 0; j < kw; ++j)
                differ += __builtin_popcount(A[m * kw + j] ^ Wt[n * kw + j]);
            C[m * N + n] = (int32_t)(K - 2 * differ);
        }
}

/* Rows [m0, m1) of the product only: C : int32 [m1-m0][N]. */
void checker_gemm_rows(const uint32_t *A, const uint32_t *Wt, int32_t *C,
                       long m0, long m1, long N, long K)
{
    const long kw = K / 32;
#pragma omp parallel for schedule(static)
    for (long m = m0; m < m1; ++m)
        for (long n = 0; n < N; ++n) {
            int differ = 0;
            for (long j = 0; j < kw; ++j)
                differ += __builtin_popcount(A[m * kw + j] ^ Wt[n * kw + j]);
            C[(m - m0) * N + n] = (int32_t)(K - 2 * differ);
        }
}
