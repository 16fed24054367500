// Shared declarations of the CUDA side: problem description handed to every kernel
// launcher, and small device helpers.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>
#include "bcnn.h"

namespace bcnn {

// One binary convolution seen as an implicit GEMM: M = B*OH*OW rows, N = C_out
// columns, K = kh*kw*C_in bits.  A plain GEMM is the 1x1 case with H = M, W = 1.
struct ConvProblem {
    const uint32_t *x;   // packed NHWC activations, C_in/32 words per pixel
    const uint32_t *w;   // packed [C_out][kh][kw][C_in] weights, K/32 words per row
    const int32_t *thr;  // per-output-channel thresholds, or nullptr for int32 output
    void *out;           // int32 [M][C_out] or packed bits [M][C_out/32 words]
    int B, H, W, C_in, C_out, kh, kw, stride, pad, OH, OW;
    int cw;              // C_in / 32: words per pixel
    int kwords;          // K / 32
    int K;               // kh*kw*C_in
    int M;               // B*OH*OW
    uint32_t cw_magic;   // floor(2^32 / cw) + 1 (0 when cw == 1): n / cw == umulhi(n, magic) for n*cw < 2^32
    uint32_t kw_magic;   // same for the kernel width kw
    int *err;            // device error word (bounded waits report here)
    // convolution-module epilogue (mode == 2): batch norm scale / shift, fp16 identity, PReLU slope, next bias
    int mode;            // 0: int32 output, 1: integer threshold -> packed bits, 2: module epilogue
    const float *bn_scale, *bn_shift, *slope, *next_bias;   // [C_out]; next_bias may be nullptr (0)
    const uint16_t *identity;                               // fp16 [M][C_out] or nullptr
    uint16_t *y_real;                                       // fp16 [M][C_out]; the packed next signs go to `out` (may be nullptr)
    uint32_t ow_mul, ow_shift;    // exact division of any 32-bit value by OW      (see exact_div)
    uint32_t ohw_mul, ohw_shift;  // exact division of any 32-bit value by OH * OW
};

// Convolution module with P parallel binary branches (optionally shifted: P = kh * kw taps of an F x F convolution).
struct BranchProblem {
    const uint32_t *x;       // packed [B][H][W][P * C_in]: the P binarizations of the module's real input side by side
    const uint32_t *w;       // packed [P][C_out][C_in]
    const float *bn_scale, *bn_shift;   // [P][C_out]
    const int32_t *pad_dot;  // [P][C_out] or nullptr (0): a branch's result where its shifted pixel lies outside the image
    const uint16_t *identity;           // fp16 [M][C_out] or nullptr
    const float *slope, *next_bias;     // [C_out]; next_bias may be nullptr (0)
    uint16_t *y_real;        // fp16 [M][C_out]
    uint8_t *y_bits;         // packed [M][C_out / 8] or nullptr
    int B, H, W, C_in, C_out, P, kh, kw;
    int cw;                  // C_in / 32
    long M;                  // B * H * W
};

// Exact n / d for every 32-bit n with a precomputed (mul, shift) pair: with s = ceil(log2 d) and
// mul = floor(2^32 * (2^s - d) / d) + 1,  n / d = (t + ((n - t) >> 1)) >> (s - 1),  t = umulhi(n, mul).
// d == 1 is encoded as shift == 0.
__device__ __forceinline__ uint32_t exact_div(uint32_t n, uint32_t mul, uint32_t shift)
{
    if (shift == 0) return n;
    const uint32_t t = __umulhi(n, mul);
    return (t + ((n - t) >> 1)) >> (shift - 1);
}

// n / d through a precomputed multiplier (exact while n * d < 2^32); magic == 0 encodes d == 1.
__device__ __forceinline__ int fast_div(int n, uint32_t magic)
{
    return magic ? (int)__umulhi((uint32_t)n, magic) : n;
}

// Row m of the implicit patch matrix -> (image, top-left input coordinate).
struct RowCoord {
    int b, ih0, iw0;
};

__device__ __forceinline__ RowCoord row_coord(const ConvProblem &p, int m)
{
    RowCoord rc;
    const int ohw = p.OH * p.OW;
    rc.b = (int)exact_div((uint32_t)m, p.ohw_mul, p.ohw_shift);
    const int rem = m - rc.b * ohw;
    const int oh = (int)exact_div((uint32_t)rem, p.ow_mul, p.ow_shift);
    const int ow = rem - oh * p.OW;
    rc.ih0 = oh * p.stride - p.pad;
    rc.iw0 = ow * p.stride - p.pad;
    return rc;
}

int launch_pack(const float *x, const float *bias, uint32_t *out, long npix, int C_in, int R,
                cudaStream_t stream);
int launch_stem_c4r8_k32(const float *x, const float *bias, const uint32_t *w, const int32_t *thr, uint32_t *out,
                         long npix, cudaStream_t stream);
int launch_conv_lop3(const ConvProblem &p, cudaStream_t stream);
bool conv_lop3_pointwise_k32(const ConvProblem &p);   // the shape runs the one-word pointwise kernel
int launch_conv_mma_b1(const ConvProblem &p, cudaStream_t stream);
bool conv_mma_b1_supports(const ConvProblem &p);
int launch_conv_mma_s8(const ConvProblem &p, cudaStream_t stream);
bool conv_mma_s8_supports(const ConvProblem &p);
int launch_conv_tc_ws(const ConvProblem &p, cudaStream_t stream);
bool conv_tc_ws_supports(const ConvProblem &p);
int launch_conv_tc_pw(const ConvProblem &p, cudaStream_t stream);
bool conv_tc_pw_supports(const ConvProblem &p);
int launch_conv_tc_c3(const ConvProblem &p, cudaStream_t stream);
bool conv_tc_c3_supports(const ConvProblem &p);
int launch_conv_tc_pn(const ConvProblem &p, cudaStream_t stream);
bool conv_tc_pn_supports(const ConvProblem &p);
int launch_conv_tc_i8(const ConvProblem &p, cudaStream_t stream);
// weights expanded once per layer by launch_prepare_weights (conv_tc_pre.cu): [n_pad][k_pad] signed bytes, then
// K - 2 popc(W_n) per row
struct PreparedWeights {
    const uint8_t *wexp;
    const int32_t *cst;
    int n_pad, k_pad;
};
void prepared_layout(int C_out, int K, PreparedWeights &pw, size_t &bytes);
int launch_prepare_weights(const uint32_t *w, void *prepared, int C_out, int K, cudaStream_t stream);
int launch_conv_tc_pre(const ConvProblem &p, const void *prepared, cudaStream_t stream);
bool conv_tc_pre_supports(const ConvProblem &p);
int launch_conv_tc_pre_static(const ConvProblem &p, cudaStream_t stream);   // prepared weights in the library's static array
size_t static_prepared_capacity();
bool conv_tc_i8_supports(const ConvProblem &p);
int launch_selftest_wait_timeout(int polls, cudaStream_t stream);
int launch_conv_branches(const BranchProblem &p, cudaStream_t stream);
int launch_dwconv3x3_module(const uint16_t *x, const float *w, const float *scale, const float *shift, const float *slope,
                            const float *next_bias, uint16_t *y, uint8_t *y_bits, int B, int H, int W, int C_in, int R, int S,
                            cudaStream_t stream);
int launch_avgpool(const uint16_t *x, uint16_t *y, int B, int H, int W, int C_in, int R, int S, cudaStream_t stream);
int launch_gap(const uint16_t *x, float *pooled, int B, int HW, int C, cudaStream_t stream);
int launch_fc(const float *pooled, const float *w, const float *bias, float *logits, int B, int C, int N, cudaStream_t stream);
int *device_error_word();   // device address of the error word of the current device (nullptr on failure)

}  // namespace bcnn
