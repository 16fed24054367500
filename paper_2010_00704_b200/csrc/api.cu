// C ABI: argument validation, problem set-up and engine dispatch.  No allocation,
// no synchronisation: every entry point only enqueues kernels on the caller's stream.
#include "bcnn_common.cuh"

namespace bcnn {

__device__ int g_device_error = 0;

int *device_error_word()
{
    static int *cache[64] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cache[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_error) != cudaSuccess) return nullptr;
        cache[dev] = static_cast<int *>(p);
    }
    return cache[dev];
}

namespace {

// (mul, shift) of exact_div for the divisor d >= 1
void exact_div_params(uint32_t d, uint32_t &mul, uint32_t &shift)
{
    if (d <= 1) { mul = 0; shift = 0; return; }
    uint32_t s = 0;
    while ((1ULL << s) < d) ++s;
    mul = (uint32_t)(((1ULL << 32) * ((1ULL << s) - d)) / d + 1);
    shift = s;
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int make_conv_problem(ConvProblem &p, const void *x, const void *w, const int32_t *thr, void *out,
                      int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad,
                      bool fused)
{
    if (!x || !w || !out || (fused && !thr)) return BCNN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || W <= 0 || C_in <= 0 || C_out <= 0 || kh <= 0 || kw <= 0 || stride <= 0 || pad < 0)
        return BCNN_ERR_INVALID_ARG;
    if (H + 2 * (long)pad < kh || W + 2 * (long)pad < kw) return BCNN_ERR_INVALID_ARG;
    if (C_in % 32 != 0) return BCNN_ERR_UNSUPPORTED;
    if (fused && C_out % 32 != 0) return BCNN_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(w) || !aligned16(out) || (thr && !aligned16(thr))) return BCNN_ERR_ALIGNMENT;
    const long OH = (H + 2L * pad - kh) / stride + 1;
    const long OW = (W + 2L * pad - kw) / stride + 1;
    const long M = (long)B * OH * OW;
    const long K = (long)kh * kw * C_in;
    if (M >= (1L << 31) || K >= (1L << 30)) return BCNN_ERR_UNSUPPORTED;
    if ((long)B * H * W * (C_in / 32) >= (1L << 40)) return BCNN_ERR_UNSUPPORTED;
    p.x = static_cast<const uint32_t *>(x);
    p.w = static_cast<const uint32_t *>(w);
    p.thr = fused ? thr : nullptr;
    p.out = out;
    p.B = B; p.H = H; p.W = W; p.C_in = C_in; p.C_out = C_out;
    p.kh = kh; p.kw = kw; p.stride = stride; p.pad = pad;
    p.OH = (int)OH; p.OW = (int)OW;
    p.cw = C_in / 32;
    p.K = (int)K;
    p.kwords = (int)(K / 32);
    p.M = (int)M;
    p.cw_magic = p.cw == 1 ? 0u : (uint32_t)((1ULL << 32) / (uint64_t)p.cw) + 1u;
    p.err = nullptr;
    p.mode = fused ? 1 : 0;
    p.bn_scale = p.bn_shift = p.slope = p.next_bias = nullptr;
    p.identity = nullptr;
    p.y_real = nullptr;
    exact_div_params((uint32_t)OW, p.ow_mul, p.ow_shift);
    exact_div_params((uint32_t)(OH * OW), p.ohw_mul, p.ohw_shift);
    p.kw_magic = kw == 1 ? 0u : (uint32_t)((1ULL << 32) / (uint64_t)kw) + 1u;
    return BCNN_OK;
}

// Measured on B200 (bench.py --mode sweep):
//   * pointwise layers (1x1, stride 1, no padding; GEMMs) with K <= 128 and C_out <= 128, packed output: pointwise
//     tcgen05 engine (memory-bound shapes: rows bulk-copied in chunks, one hand-over per chunk);
//   * pointwise layers with K = 256 or 512 and 128, 256 or 512 output channels, packed output: wide pointwise tcgen05
//     engine (a row tile expanded once for all resident weight slices; 1.2 - 2x the weight-stationary engine);
//   * 3x3 layers (stride 1 or 2) on 32 or 64 input channels with C_out <= 64, packed output, whose 8 x 16 output tiles
//     are at least three quarters full: halo-tile tcgen05 engine (input tiles by tiled TMA copies);
//   * C_out >= 256, or weights too large to keep expanded in shared memory: streaming tcgen05 engine;
//   * 1x1 layer with C_in = 32 and C_out <= 32 (one XOR + popcount per output): CUDA-core pointwise kernel;
//   * C_out <= 128 with K >= 64, and wider layers with K <= 1152 and M >= 32768 (in 128-channel slices):
//     weight-stationary tcgen05 engine;
//   * other K = 32 layers: register-fed warp-level int8 engine;
//   * the single-bit mma.sync and CUDA-core engines never win and serve as fallbacks.
int auto_engine(const ConvProblem &p)
{
    if (conv_tc_pw_supports(p)) return BCNN_ENGINE_TC_PW;
    if (conv_tc_pn_supports(p)) return BCNN_ENGINE_TC_PN;
    if (p.C_out <= 64 && conv_tc_c3_supports(p)) {
        const long covered = (long)((p.OH + 7) / 8 * 8) * ((p.OW + 15) / 16 * 16);
        if (4L * p.OH * p.OW >= 3L * covered) return BCNN_ENGINE_TC_C3;
    }
    if (conv_lop3_pointwise_k32(p)) return BCNN_ENGINE_LOP3;
    if (p.C_out <= 128 && p.K >= 64 && conv_tc_ws_supports(p)) return BCNN_ENGINE_TC_WS;
    // wider layers in slices of 128 output channels: ahead of the streaming engine while K is short and there are
    // enough rows to share one slice's weights among many CTAs (K = 2304 ties, K = 512 at M = 12544 loses)
    if (p.C_out > 128 && p.K <= 1152 && p.M >= 32768 && conv_tc_ws_supports(p)) return BCNN_ENGINE_TC_WS;
    if (p.C_out <= 64 && conv_mma_s8_supports(p)) return BCNN_ENGINE_MMA_S8;
    if (conv_tc_i8_supports(p)) return BCNN_ENGINE_TC_I8;
    if (conv_mma_b1_supports(p)) return BCNN_ENGINE_MMA_B1;
    return BCNN_ENGINE_LOP3;
}

int dispatch(int engine, const ConvProblem &p, cudaStream_t stream)
{
    if (engine == BCNN_ENGINE_AUTO) engine = auto_engine(p);
    switch (engine) {
    case BCNN_ENGINE_LOP3:
        return launch_conv_lop3(p, stream);
    case BCNN_ENGINE_MMA_B1:
        return launch_conv_mma_b1(p, stream);
    case BCNN_ENGINE_TC_I8:
        return launch_conv_tc_i8(p, stream);
    case BCNN_ENGINE_MMA_S8:
        return launch_conv_mma_s8(p, stream);
    case BCNN_ENGINE_TC_WS:
        return launch_conv_tc_ws(p, stream);
    case BCNN_ENGINE_TC_PW:
        return launch_conv_tc_pw(p, stream);
    case BCNN_ENGINE_TC_C3:
        return launch_conv_tc_c3(p, stream);
    case BCNN_ENGINE_TC_PN:
        return launch_conv_tc_pn(p, stream);
    default:
        return BCNN_ERR_UNSUPPORTED;
    }
}

int gemm_problem(ConvProblem &p, const void *A, const void *Wb, const int32_t *thr, void *out,
                 int64_t M, int N, int K, bool fused)
{
    if (M <= 0 || N <= 0 || K <= 0) return BCNN_ERR_INVALID_ARG;
    if (M >= (1LL << 31)) return BCNN_ERR_UNSUPPORTED;
    if (K % 32 != 0) return BCNN_ERR_UNSUPPORTED;
    // a GEMM is the 1x1 convolution over an M x 1 image with K channels
    return make_conv_problem(p, A, Wb, thr, out, 1, (int)M, 1, K, N, 1, 1, 1, 0, fused);
}

}  // namespace
}  // namespace bcnn

using namespace bcnn;

extern "C" {

int bcnn_pack(const float *x, const float *bias, void *out_bits,
              int B, int H, int W, int C_in, int R, void *stream)
{
    if (!x || !out_bits) return BCNN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || W <= 0 || C_in <= 0 || R <= 0) return BCNN_ERR_INVALID_ARG;
    const long C = (long)C_in * R;
    if (C % 32 != 0 || C >= (1L << 24)) return BCNN_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(out_bits) || (bias && !aligned16(bias))) return BCNN_ERR_ALIGNMENT;
    const long npix = (long)B * H * W;
    if (npix * C >= (1L << 46)) return BCNN_ERR_UNSUPPORTED;
    return launch_pack(x, bias, static_cast<uint32_t *>(out_bits), npix, C_in, R,
                       static_cast<cudaStream_t>(stream));
}

int bcnn_stem_fused(const float *x, const float *bias, const void *w_bits, const int32_t *thr, void *y_bits,
                    int B, int H, int W, int C_in, int R, int C_out, void *stream)
{
    if (!x || !w_bits || !thr || !y_bits) return BCNN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || W <= 0 || C_in <= 0 || R <= 0 || C_out <= 0) return BCNN_ERR_INVALID_ARG;
    if (C_in != 4 || R != 8 || C_out != 32) return BCNN_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(w_bits) || !aligned16(thr) || !aligned16(y_bits) || (bias && !aligned16(bias)))
        return BCNN_ERR_ALIGNMENT;
    const long npix = (long)B * H * W;
    if (npix >= (1L << 40)) return BCNN_ERR_UNSUPPORTED;
    return launch_stem_c4r8_k32(x, bias, static_cast<const uint32_t *>(w_bits), thr, static_cast<uint32_t *>(y_bits),
                                npix, static_cast<cudaStream_t>(stream));
}

int bcnn_gemm_b1(const void *A_bits, const void *W_bits, int32_t *C, int64_t M, int N, int K, void *stream)
{
    return bcnn_gemm_b1_engine(BCNN_ENGINE_AUTO, A_bits, W_bits, nullptr, C, M, N, K, stream);
}

int bcnn_gemm_b1_fused(const void *A_bits, const void *W_bits, const int32_t *thr, void *out_bits,
                       int64_t M, int N, int K, void *stream)
{
    if (!thr) return BCNN_ERR_INVALID_ARG;
    return bcnn_gemm_b1_engine(BCNN_ENGINE_AUTO, A_bits, W_bits, thr, out_bits, M, N, K, stream);
}

int bcnn_conv2d_b1(const void *x_bits, const void *w_bits, int32_t *y, int B, int H, int W, int C_in,
                   int C_out, int kh, int kw, int stride, int pad, void *stream)
{
    return bcnn_conv2d_b1_engine(BCNN_ENGINE_AUTO, x_bits, w_bits, nullptr, y, B, H, W, C_in, C_out,
                                 kh, kw, stride, pad, stream);
}

int bcnn_conv2d_b1_fused(const void *x_bits, const void *w_bits, const int32_t *thr, void *y_bits,
                         int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad,
                         void *stream)
{
    if (!thr) return BCNN_ERR_INVALID_ARG;
    return bcnn_conv2d_b1_engine(BCNN_ENGINE_AUTO, x_bits, w_bits, thr, y_bits, B, H, W, C_in, C_out,
                                 kh, kw, stride, pad, stream);
}

int bcnn_conv2d_b1_module(const void *x_bits, const void *w_bits, const float *bn_scale, const float *bn_shift,
                          const void *identity, const float *prelu_slope, const float *next_bias,
                          void *y_real, void *y_bits, int B, int H, int W, int C_in, int C_out,
                          int kh, int kw, int stride, int pad, void *stream)
{
    if (!bn_scale || !bn_shift || !prelu_slope || !y_real) return BCNN_ERR_INVALID_ARG;
    ConvProblem p;
    // validated like the int32 convolution whose result it post-processes (y_real stands in for the output)
    const int st = make_conv_problem(p, x_bits, w_bits, nullptr, y_real, B, H, W, C_in, C_out, kh, kw, stride, pad, false);
    if (st != BCNN_OK) return st;
    if (C_out % 32 != 0) return BCNN_ERR_UNSUPPORTED;
    if (!aligned16(bn_scale) || !aligned16(bn_shift) || !aligned16(prelu_slope) || (next_bias && !aligned16(next_bias)) ||
        (identity && !aligned16(identity)) || (y_bits && !aligned16(y_bits)))
        return BCNN_ERR_ALIGNMENT;
    p.mode = 2;
    p.bn_scale = bn_scale;
    p.bn_shift = bn_shift;
    p.slope = prelu_slope;
    p.next_bias = next_bias;
    p.identity = static_cast<const uint16_t *>(identity);
    p.y_real = static_cast<uint16_t *>(y_real);
    p.out = y_bits;
    // the two tcgen05 engines carry this epilogue; it is bound by the epilogue warps, of which the weight-stationary
    // engine has twice as many per SM whenever two of its CTAs fit (wider layers run as 128-channel slices)
    if (conv_tc_ws_supports(p)) return launch_conv_tc_ws(p, static_cast<cudaStream_t>(stream));
    return launch_conv_tc_i8(p, static_cast<cudaStream_t>(stream));
}

int bcnn_conv2d_b1_branches(const void *x_bits, const void *w_bits, const float *bn_scale, const float *bn_shift,
                            const int32_t *pad_dot, const void *identity, const float *prelu_slope, const float *next_bias,
                            void *y_real, void *y_bits, int B, int H, int W, int C_in, int C_out, int P, int kh, int kw,
                            void *stream)
{
    if (!x_bits || !w_bits || !bn_scale || !bn_shift || !prelu_slope || !y_real) return BCNN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || W <= 0 || C_in <= 0 || C_out <= 0 || P <= 0 || kh <= 0 || kw <= 0) return BCNN_ERR_INVALID_ARG;
    if (kh * kw > 1 && P != kh * kw) return BCNN_ERR_INVALID_ARG;
    if (C_in % 32 != 0 || C_out % 32 != 0 || P > 64 || (kh % 2 == 0) || (kw % 2 == 0)) return BCNN_ERR_UNSUPPORTED;
    if (!aligned16(x_bits) || !aligned16(w_bits) || !aligned16(bn_scale) || !aligned16(bn_shift) || !aligned16(prelu_slope) ||
        !aligned16(y_real) || (pad_dot && !aligned16(pad_dot)) || (identity && !aligned16(identity)) ||
        (next_bias && !aligned16(next_bias)) || (y_bits && !aligned16(y_bits)))
        return BCNN_ERR_ALIGNMENT;
    BranchProblem p;
    p.x = static_cast<const uint32_t *>(x_bits);
    p.w = static_cast<const uint32_t *>(w_bits);
    p.bn_scale = bn_scale; p.bn_shift = bn_shift; p.pad_dot = pad_dot;
    p.identity = static_cast<const uint16_t *>(identity);
    p.slope = prelu_slope; p.next_bias = next_bias;
    p.y_real = static_cast<uint16_t *>(y_real);
    p.y_bits = static_cast<uint8_t *>(y_bits);
    p.B = B; p.H = H; p.W = W; p.C_in = C_in; p.C_out = C_out; p.P = P; p.kh = kh; p.kw = kw;
    p.cw = C_in / 32;
    p.M = (long)B * H * W;
    if (p.M >= (1L << 40)) return BCNN_ERR_UNSUPPORTED;
    return launch_conv_branches(p, static_cast<cudaStream_t>(stream));
}

int bcnn_dwconv3x3_module(const void *x, const float *w, const float *bn_scale, const float *bn_shift, const float *prelu_slope,
                          const float *next_bias, void *y_real, void *y_bits, int B, int H, int W, int C_in, int R, int S,
                          void *stream)
{
    if (!x || !w || !bn_scale || !bn_shift || !prelu_slope || !y_real) return BCNN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || W <= 0 || C_in <= 0 || R <= 0 || S <= 0) return BCNN_ERR_INVALID_ARG;
    const long C = (long)C_in * R;
    if (C_in % 8 != 0 || C >= (1L << 20) || (y_bits && C % 32 != 0)) return BCNN_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(w) || !aligned16(bn_scale) || !aligned16(bn_shift) || !aligned16(prelu_slope) ||
        !aligned16(y_real) || (next_bias && !aligned16(next_bias)) || (y_bits && !aligned16(y_bits)))
        return BCNN_ERR_ALIGNMENT;
    if ((long)B * H * W * C >= (1L << 46)) return BCNN_ERR_UNSUPPORTED;
    return launch_dwconv3x3_module(static_cast<const uint16_t *>(x), w, bn_scale, bn_shift, prelu_slope, next_bias,
                                   static_cast<uint16_t *>(y_real), static_cast<uint8_t *>(y_bits), B, H, W, C_in, R, S,
                                   static_cast<cudaStream_t>(stream));
}

int bcnn_avgpool(const void *x, void *y, int B, int H, int W, int C_in, int R, int S, void *stream)
{
    if (!x || !y) return BCNN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || W <= 0 || C_in <= 0 || R <= 0 || S <= 0) return BCNN_ERR_INVALID_ARG;
    if (H % S != 0 || W % S != 0) return BCNN_ERR_INVALID_ARG;
    if (C_in % 8 != 0 || (long)C_in * R >= (1L << 20) || (long)B * H * W * C_in * R >= (1L << 46)) return BCNN_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(y)) return BCNN_ERR_ALIGNMENT;
    return launch_avgpool(static_cast<const uint16_t *>(x), static_cast<uint16_t *>(y), B, H, W, C_in, R, S,
                          static_cast<cudaStream_t>(stream));
}

int bcnn_gap(const void *x, float *pooled, int B, int H, int W, int C, void *stream)
{
    if (!x || !pooled) return BCNN_ERR_INVALID_ARG;
    if (B <= 0 || H <= 0 || W <= 0 || C <= 0) return BCNN_ERR_INVALID_ARG;
    if (C % 8 != 0 || (long)H * W >= (1L << 24) || (long)B * H * W * C >= (1L << 46)) return BCNN_ERR_UNSUPPORTED;
    if (!aligned16(x) || !aligned16(pooled)) return BCNN_ERR_ALIGNMENT;
    return launch_gap(static_cast<const uint16_t *>(x), pooled, B, H * W, C, static_cast<cudaStream_t>(stream));
}

int bcnn_fc(const float *pooled, const float *w, const float *bias, float *logits, int B, int C, int N, void *stream)
{
    if (!pooled || !w || !logits) return BCNN_ERR_INVALID_ARG;
    if (B <= 0 || C <= 0 || N <= 0) return BCNN_ERR_INVALID_ARG;
    if (C % 4 != 0) return BCNN_ERR_UNSUPPORTED;
    if (!aligned16(pooled) || !aligned16(w) || !aligned16(logits) || (bias && !aligned16(bias))) return BCNN_ERR_ALIGNMENT;
    return launch_fc(pooled, w, bias, logits, B, C, N, static_cast<cudaStream_t>(stream));
}

int bcnn_conv2d_b1_engine(int engine, const void *x_bits, const void *w_bits, const int32_t *thr, void *out,
                          int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad,
                          void *stream)
{
    ConvProblem p;
    const int st = make_conv_problem(p, x_bits, w_bits, thr, out, B, H, W, C_in, C_out, kh, kw, stride, pad,
                                     thr != nullptr);
    if (st != BCNN_OK) return st;
    return dispatch(engine, p, static_cast<cudaStream_t>(stream));
}

int bcnn_gemm_b1_engine(int engine, const void *A_bits, const void *W_bits, const int32_t *thr, void *out,
                        int64_t M, int N, int K, void *stream)
{
    ConvProblem p;
    const int st = gemm_problem(p, A_bits, W_bits, thr, out, M, N, K, thr != nullptr);
    if (st != BCNN_OK) return st;
    return dispatch(engine, p, static_cast<cudaStream_t>(stream));
}

size_t bcnn_prepared_weights_bytes(int C_out, int K)
{
    if (C_out <= 0 || K <= 0 || K % 32 != 0 || K >= (1 << 30)) return 0;
    PreparedWeights pw;
    size_t bytes = 0;
    prepared_layout(C_out, K, pw, bytes);
    return bytes;
}

int bcnn_prepare_weights(const void *w_bits, void *prepared, int C_out, int K, void *stream)
{
    if (!w_bits || !prepared || C_out <= 0 || K <= 0) return BCNN_ERR_INVALID_ARG;
    if (K % 32 != 0 || K >= (1 << 30)) return BCNN_ERR_UNSUPPORTED;
    if (!aligned16(w_bits) || (reinterpret_cast<uintptr_t>(prepared) & 255u) != 0) return BCNN_ERR_ALIGNMENT;
    return launch_prepare_weights(static_cast<const uint32_t *>(w_bits), prepared, C_out, K, static_cast<cudaStream_t>(stream));
}

int bcnn_conv2d_b1_prepared(const void *x_bits, const void *prepared, const int32_t *thr, void *out,
                            int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad, void *stream)
{
    ConvProblem p;
    const int st = make_conv_problem(p, x_bits, prepared, thr, out, B, H, W, C_in, C_out, kh, kw, stride, pad, thr != nullptr);
    if (st != BCNN_OK) return st;
    if ((reinterpret_cast<uintptr_t>(prepared) & 255u) != 0) return BCNN_ERR_ALIGNMENT;
    return launch_conv_tc_pre(p, prepared, static_cast<cudaStream_t>(stream));
}

int bcnn_gemm_b1_prepared(const void *A_bits, const void *prepared, const int32_t *thr, void *out,
                          int64_t M, int N, int K, void *stream)
{
    ConvProblem p;
    const int st = gemm_problem(p, A_bits, prepared, thr, out, M, N, K, thr != nullptr);
    if (st != BCNN_OK) return st;
    if ((reinterpret_cast<uintptr_t>(prepared) & 255u) != 0) return BCNN_ERR_ALIGNMENT;
    return launch_conv_tc_pre(p, prepared, static_cast<cudaStream_t>(stream));
}

int bcnn_conv2d_b1_fused_noalloc(const void *x_bits, const void *w_bits, const int32_t *thr, void *y_bits,
                                 int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad,
                                 void *stream)
{
    if (!thr) return BCNN_ERR_INVALID_ARG;
    ConvProblem p;
    const int st = make_conv_problem(p, x_bits, w_bits, thr, y_bits, B, H, W, C_in, C_out, kh, kw, stride, pad, true);
    if (st != BCNN_OK) return st;
    static_assert(BCNN_STATIC_SCRATCH_BYTES == (4u << 20), "header and kernel file agree on the array's size");
    if (static_prepared_capacity() != BCNN_STATIC_SCRATCH_BYTES) return BCNN_ERR_CUDA;
    return launch_conv_tc_pre_static(p, static_cast<cudaStream_t>(stream));
}

int bcnn_prepared_preferred(int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad, int fused)
{
    ConvProblem p;
    void *dummy = reinterpret_cast<void *>(uintptr_t(4096));
    const int st = make_conv_problem(p, dummy, dummy, fused ? static_cast<const int32_t *>(dummy) : nullptr, dummy,
                                     B, H, W, C_in, C_out, kh, kw, stride, pad, fused != 0);
    if (st != BCNN_OK) return 0;
    // measured (bench.py --mode sweep): streaming prepared weights wins wherever AUTO would run the streaming engine
    // (wide layers, long K) and on every K >= 2048; the weight-stationary and pointwise engines keep the short-K layers
    if (!conv_tc_pre_supports(p)) return 0;
    return (auto_engine(p) == BCNN_ENGINE_TC_I8 || p.K >= 2048) ? 1 : 0;
}

int bcnn_auto_engine(int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad, int fused)
{
    ConvProblem p;
    // validation only looks at pointer alignment and nullness: hand it aligned dummies
    void *dummy = reinterpret_cast<void *>(uintptr_t(4096));
    const int st = make_conv_problem(p, dummy, dummy, fused ? static_cast<const int32_t *>(dummy) : nullptr, dummy,
                                     B, H, W, C_in, C_out, kh, kw, stride, pad, fused != 0);
    if (st != BCNN_OK) return st;
    return auto_engine(p);
}

int bcnn_device_error(void)
{
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_device_error, sizeof(int)) != cudaSuccess) return BCNN_ERR_CUDA;
    if (v != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_device_error, &zero, sizeof(int)) != cudaSuccess) return BCNN_ERR_CUDA;
    }
    return v;
}

int bcnn_device_status(int *code)
{
    const int v = bcnn_device_error();
    if (code) *code = v > 0 ? v : 0;
    if (v < 0) return v;
    return v == 0 ? BCNN_OK : BCNN_ERR_TIMEOUT;
}

size_t bcnn_workspace_bytes(int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad, int fused)
{
    // no kernel uses global memory beyond its inputs and outputs, whatever the shape
    (void)B; (void)H; (void)W; (void)C_in; (void)C_out; (void)kh; (void)kw; (void)stride; (void)pad; (void)fused;
    return 0;
}

int bcnn_selftest_wait_timeout(int polls, void *stream)
{
    if (polls < 1 || polls > 65536) return BCNN_ERR_INVALID_ARG;
    return launch_selftest_wait_timeout(polls, static_cast<cudaStream_t>(stream));
}

const char *bcnn_status_string(int status)
{
    switch (status) {
    case BCNN_OK: return "ok";
    case BCNN_ERR_INVALID_ARG: return "invalid argument";
    case BCNN_ERR_UNSUPPORTED: return "unsupported shape or engine";
    case BCNN_ERR_ALIGNMENT: return "pointer not 16-byte aligned";
    case BCNN_ERR_CUDA: return "CUDA runtime error";
    case BCNN_ERR_WORKSPACE: return "workspace too small (the layer's prepared weights exceed the library's static scratch array)";
    case BCNN_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    // device error word: which bounded wait gave up
    case 101: return "device wait timed out: streaming tcgen05 engine, producer waiting for a free ring slot";
    case 102: return "device wait timed out: streaming tcgen05 engine, control warp waiting for a full slot or a free accumulator";
    case 103: return "device wait timed out: streaming tcgen05 engine, epilogue waiting for an accumulator";
    case 111: return "device wait timed out: weight-stationary tcgen05 engine, producer waiting for a free ring slot";
    case 112: return "device wait timed out: weight-stationary tcgen05 engine, control warp waiting for a full slot or a free accumulator";
    case 113: return "device wait timed out: weight-stationary tcgen05 engine, epilogue waiting for an accumulator";
    case 121: return "device wait timed out: pointwise tcgen05 engine, loader waiting for a free ring stage";
    case 122: return "device wait timed out: pointwise tcgen05 engine, producer waiting for a chunk's rows";
    case 123: return "device wait timed out: pointwise tcgen05 engine, issuer waiting for a slot's expanded rows";
    case 124: return "device wait timed out: pointwise tcgen05 engine, epilogue waiting for a chunk's accumulators";
    case 131: return "device wait timed out: prepared-weights tcgen05 engine, producer waiting for a free ring slot";
    case 132: return "device wait timed out: prepared-weights tcgen05 engine, control warp waiting for a full slot or a free accumulator";
    case 133: return "device wait timed out: prepared-weights tcgen05 engine, epilogue waiting for an accumulator";
    case 134: return "device wait timed out: prepared-weights tcgen05 engine, loader waiting for a free ring slot";
    case 125: return "device wait timed out: pointwise tcgen05 engine, producer waiting for a slot's previous MMAs";
    case 126: return "device wait timed out: pointwise tcgen05 engine, issuer waiting for a slot's accumulators";
    case 141: return "device wait timed out: 3x3 halo-tile tcgen05 engine, loader waiting for a free ring stage";
    case 142: return "device wait timed out: 3x3 halo-tile tcgen05 engine, producer waiting for a tile's halo";
    case 143: return "device wait timed out: 3x3 halo-tile tcgen05 engine, issuer waiting for a tile's expanded rows";
    case 144: return "device wait timed out: 3x3 halo-tile tcgen05 engine, epilogue waiting for a tile's accumulator";
    case 145: return "device wait timed out: 3x3 halo-tile tcgen05 engine, producer waiting for an activation stage's previous MMAs";
    case 146: return "device wait timed out: 3x3 halo-tile tcgen05 engine, issuer waiting for an accumulator";
    case 151: return "device wait timed out: wide pointwise tcgen05 engine, loader waiting for a free ring stage";
    case 152: return "device wait timed out: wide pointwise tcgen05 engine, producer waiting for a tile's rows";
    case 153: return "device wait timed out: wide pointwise tcgen05 engine, issuer waiting for a tile's expanded rows";
    case 154: return "device wait timed out: wide pointwise tcgen05 engine, epilogue waiting for an accumulator";
    case 155: return "device wait timed out: wide pointwise tcgen05 engine, producer waiting for an activation unit's previous MMAs";
    case 156: return "device wait timed out: wide pointwise tcgen05 engine, issuer waiting for an accumulator";
    case BCNN_SELFTEST_TIMEOUT_CODE: return "device wait timed out: self-test (expected)";
    default: return status > 0 ? "device-side error code" : "unknown status";
    }
}

int bcnn_version(void) { return 100; }

}  // extern "C"
