/*
 * bcnn.h - C ABI of the binary (+-1 x +-1) convolution library for NVIDIA B200 (sm_100a).
 *
 * The operator is the CNN-style 2D convolution of the paper (Section 1: 3D input
 * tensor, 4D weight tensor, 3D output tensor, lowered to a matrix-matrix product)
 * with both operands binarized (Section 4.2.1: every feature is +1 or -1 and every
 * weight is +1 or -1; Section 5.2 / Figure 5: forward weights are the sign of the
 * real weights).  For +-1 vectors the inner product over K elements equals
 * K - 2*popcount(a XOR w) on their sign bits; the library computes exactly that
 * integer.
 *
 * Conventions shared by every call
 *   - Sign-bit encoding: bit 1 = +1, bit 0 = -1.
 *   - Packed activations are NHWC; the C channels of one pixel occupy C/8 consecutive
 *     bytes, channel c in byte c/8, bit c%8 (LSB first).  Read as little-endian 32- or
 *     64-bit words this is the same memory.  C must be a multiple of 32.
 *   - Packed weights are [C_out][kh][kw][C_in] with C_in packed the same way, i.e.
 *     N = C_out rows of K = kh*kw*C_in bits.  A GEMM "B" operand is likewise N rows
 *     of K bits (the K x N matrix stored column by column).
 *   - Out-of-image taps of a convolution read the value -1 (a +-1 tensor has no
 *     zero); BCNN_PAD_VALUE documents it.  K in "K - 2*popcount" is always the full
 *     kh*kw*C_in.
 *   - Output extent: OH = floor((H + 2*pad - kh)/stride) + 1, same for OW.
 *   - All data pointers are DEVICE pointers owned by the caller, 16-byte aligned.
 *     The library never allocates, frees or synchronises: every call only enqueues
 *     kernels on `stream` (a cudaStream_t passed as void*, NULL = default stream)
 *     and returns.  Buffers may be reused as soon as the stream has passed the call.
 *   - Every call validates its arguments first and launches nothing on error.
 *     Return value: BCNN_OK or a negative bcnn_status.
 */
#ifndef BCNN_H
#define BCNN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BCNN_PAD_VALUE (-1)

typedef enum bcnn_status {
    BCNN_OK = 0,
    BCNN_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, empty output */
    BCNN_ERR_UNSUPPORTED = -2, /* channel count not a multiple of 32, size limits */
    BCNN_ERR_ALIGNMENT = -3,   /* a data pointer is not 16-byte aligned */
    BCNN_ERR_CUDA = -4,        /* the CUDA runtime refused a launch */
    BCNN_ERR_WORKSPACE = -5,   /* a caller-provided scratch buffer is too small (no call takes one today:
                                  bcnn_workspace_bytes() is 0 for every shape; the value is reserved) */
    BCNN_ERR_TIMEOUT = -6      /* a bounded device-side wait gave up (see bcnn_device_status) */
} bcnn_status;

/* Engines of the inner product; BCNN_ENGINE_AUTO picks per shape. */
typedef enum bcnn_engine {
    BCNN_ENGINE_AUTO = 0,
    BCNN_ENGINE_LOP3 = 1,   /* CUDA cores: XOR + popcount                              */
    BCNN_ENGINE_MMA_B1 = 2, /* warp-level mma.sync m16n8k256 .b1 AND + popcount         */
    BCNN_ENGINE_TC_I8 = 3,  /* sign bits expanded to bytes in shared memory, tcgen05 kind::i8, TMEM accumulators */
    BCNN_ENGINE_MMA_S8 = 4, /* sign bits expanded to bytes in registers, warp-level mma.sync 8-bit (narrow layers) */
    BCNN_ENGINE_TC_WS = 5,  /* tcgen05 kind::i8 with the expanded weight tile resident in shared memory (C_out <= 128) */
    BCNN_ENGINE_TC_PW = 6,  /* tcgen05 kind::i8 for pointwise layers (1x1, stride 1, no padding; GEMMs) with K <= 128 and
                               C_out <= 128, packed output: rows bulk-copied in chunks, one hand-over per chunk */
    BCNN_ENGINE_TC_C3 = 7,  /* tcgen05 kind::i8 for 3x3 layers (stride 1 or 2, padding 0 or 1) on 32 or 64 input channels
                               with C_out <= 128 and W * C_in a multiple of 128, packed output: the input halo of an
                               8 x 16 tile of output pixels arrives by one tiled TMA copy, padding is the copy's zero fill */
    BCNN_ENGINE_TC_PN = 8   /* tcgen05 kind::i8 for pointwise layers (1x1, stride 1, no padding; GEMMs) with K = 256 or 512 and
                               128, 256 or 512 output channels, packed output: a row tile is expanded once and multiplied
                               against all the weight slices a CTA keeps in shared memory */
} bcnn_engine;

/*
 * Binarize and pack (Section 4.2.1: learnable bias, then sign; Section 4.2.2: channel
 * replication by an integer factor R is bookkeeping, not a copy).
 *   out bit[b][h][w][c] = (x[b][h][w][c mod C_in] + bias[c] >= 0),  c in [0, R*C_in)
 * The add is an fp32 add, the compare is >= 0 (so -0.0 -> +1, NaN -> -1).
 *   x        device, fp32 NHWC [B][H][W][C_in]
 *   bias     device, fp32 [R*C_in], or NULL for no bias
 *   out_bits device, B*H*W*(R*C_in)/8 bytes, layout above; R*C_in % 32 == 0
 * With B = C_out, H = kh, W = kw the same call packs real weights into the weight
 * layout (Section 5.2).
 */
int bcnn_pack(const float *x, const float *bias, void *out_bits,
              int B, int H, int W, int C_in, int R, void *stream);

/*
 * Binary matrix product (Section 1 lowering):
 *   C[m][n] = sum_k a[m][k]*w[n][k] = K - 2*popcount(A_m XOR W_n),  a, w in {-1,+1}
 *   A_bits device, M rows of K bits;  W_bits device, N rows of K bits;  K % 32 == 0
 *   C      device, int32 [M][N] row-major
 */
int bcnn_gemm_b1(const void *A_bits, const void *W_bits, int32_t *C,
                 int64_t M, int N, int K, void *stream);

/*
 * The same product followed by a per-column integer threshold that emits packed sign
 * bits (Section 4.2.1: batch norm scale/bias and the next module's bias + sign, folded
 * into one integer comparison):
 *   out bit[m][n] = (C[m][n] >= thr[n])
 *   thr      device, int32 [N];  out_bits device, M rows of N bits;  N % 32 == 0
 * A batch norm with negative scale is folded by the caller: flip that channel's weight
 * bits and negate its threshold.
 */
int bcnn_gemm_b1_fused(const void *A_bits, const void *W_bits, const int32_t *thr,
                       void *out_bits, int64_t M, int N, int K, void *stream);

/*
 * Binary convolution as an implicit GEMM (the patch matrix is never materialised):
 *   y[b][oh][ow][co] = sum_{r,t,ci} xpad[b][oh*stride-pad+r][ow*stride-pad+t][ci] * w[co][r][t][ci]
 * with xpad = x inside the image and -1 outside.
 *   x_bits device, packed NHWC [B][H][W][C_in];  w_bits device, packed [C_out][kh][kw][C_in]
 *   y      device, int32 NHWC [B][OH][OW][C_out]
 *   C_in % 32 == 0; kh, kw >= 1; stride >= 1; pad >= 0; OH, OW >= 1; B*OH*OW < 2^31
 */
int bcnn_conv2d_b1(const void *x_bits, const void *w_bits, int32_t *y,
                   int B, int H, int W, int C_in, int C_out,
                   int kh, int kw, int stride, int pad, void *stream);

/*
 * Convolution with the fused threshold / re-pack epilogue: the output is the next
 * layer's packed input, y bit[b][oh][ow][co] = (acc >= thr[co]).
 *   thr device int32 [C_out];  y_bits device, packed NHWC [B][OH][OW][C_out];  C_out % 32 == 0
 */
int bcnn_conv2d_b1_fused(const void *x_bits, const void *w_bits, const int32_t *thr,
                         void *y_bits, int B, int H, int W, int C_in, int C_out,
                         int kh, int kw, int stride, int pad, void *stream);

/*
 * Binary convolution followed by the rest of the paper's convolution module (Section 4.2.1, Figure 4: learnable
 * bias -> sign -> binary conv -> batch norm -> + module identity -> PReLU; the bias + sign at the front is the
 * producer of x_bits, the bias + sign of the NEXT module is emitted here), in one pass:
 *   acc = the convolution's integer result (as bcnn_conv2d_b1)
 *   t = acc * bn_scale[co] + bn_shift[co];  u = t + identity;  r = (u >= 0) ? u : prelu_slope[co] * u
 *   y_real = fp16(r);   y bit = (y_real + next_bias[co] >= 0)
 * Every step is one fp32 operation rounded to nearest even (no fused multiply-add); the sign is taken of the
 * stored fp16 value, so it equals bcnn_pack applied to y_real.
 *   bn_scale, bn_shift, prelu_slope  device fp32 [C_out];  next_bias device fp32 [C_out] or NULL (= 0)
 *   identity  device fp16 NHWC [B][OH][OW][C_out] (the module's real input; needs the output's shape), or NULL
 *   y_real    device fp16 NHWC [B][OH][OW][C_out];  y_bits device packed NHWC [B][OH][OW][C_out], or NULL
 *   C_out % 32 == 0.  identity and y_real may be the same buffer (each element is read before it is written).
 */
int bcnn_conv2d_b1_module(const void *x_bits, const void *w_bits, const float *bn_scale, const float *bn_shift,
                          const void *identity, const float *prelu_slope, const float *next_bias,
                          void *y_real, void *y_bits, int B, int H, int W, int C_in, int C_out,
                          int kh, int kw, int stride, int pad, void *stream);

/*
 * Convolution module with P parallel binary residual branches (Section 4.2.1, Figure 4 bottom: each branch has its own
 * learned bias - hence its own binarization -, its own binary weights and its own batch norm; the branches are summed
 * before the identity addition and PReLU), in one pass:
 *   dot_p = binary 1x1 convolution of branch p's sign channels with branch p's weights
 *   t_p = dot_p * bn_scale[p][co] + bn_shift[p][co];   t = ((t_0 + t_1) + t_2) + ...        (branch order, fp32)
 *   u = t + identity;  r = (u >= 0) ? u : prelu_slope[co] * u;  y_real = fp16(r);  y bit = (y_real + next_bias[co] >= 0)
 * one fp32 operation per step as in bcnn_conv2d_b1_module (which this call equals for P = 1, kh = kw = 1).
 *   x_bits   device, packed NHWC [B][H][W][P * C_in]: branch p's signs are channels [p*C_in, (p+1)*C_in) of a pixel,
 *            i.e. the output of ONE bcnn_pack call with R = P and the P branch biases concatenated
 *   w_bits   device, packed [P][C_out][C_in];   bn_scale, bn_shift  device fp32 [P][C_out]
 * With kh * kw > 1 the branches are the taps of a binary kh x kw convolution (last paragraph of Section 4.2.1: P = kh*kw
 * branches, each on the real map shifted to its tap with zero padding applied BEFORE the branch's bias and sign); then
 * P must equal kh * kw, branch p = (r, t) reads pixel (h + r - (kh-1)/2, w + t - (kw-1)/2), and where that pixel lies
 * outside the image its dot_p is pad_dot[p][co] - the caller passes sum_ci sign(0 + bias_p[ci]) * w_p[co][ci] for the
 * paper's padding, or NULL (0) for a tap that contributes nothing.  Stride 1, output H x W.
 *   pad_dot  device int32 [P][C_out] or NULL;  identity, prelu_slope, next_bias, y_real, y_bits as in
 *   bcnn_conv2d_b1_module (identity and y_real may be the same buffer).  C_in % 32 == 0, C_out % 32 == 0.
 */
int bcnn_conv2d_b1_branches(const void *x_bits, const void *w_bits, const float *bn_scale, const float *bn_shift,
                            const int32_t *pad_dot, const void *identity, const float *prelu_slope, const float *next_bias,
                            void *y_real, void *y_bits, int B, int H, int W, int C_in, int C_out, int P, int kh, int kw,
                            void *stream);

/*
 * The 3x3 convolution module (Section 4.2.1: real depth-wise 3x3 convolution for spatial mixing, batch norm, PReLU), with
 * stride S (Section 4.2.3) and channel replication by bookkeeping (Section 4.2.2: output channel c reads input channel
 * c mod C_in; nothing is copied):
 *   conv = sum_{r,t} xpad[oh*S - 1 + r][ow*S - 1 + t][c mod C_in] * w[c][r][t],  xpad = 0 outside the image
 *   y_real = fp16(PReLU(conv * bn_scale[c] + bn_shift[c]));   y bit = (y_real + next_bias[c] >= 0)   (optional)
 * fp32 arithmetic on fp16 storage.  x device fp16 NHWC [B][H][W][C_in]; w device fp32 [C][3][3], C = R * C_in;
 * y_real device fp16 [B][OH][OW][C], OH = (H - 1) / S + 1; y_bits device packed [B][OH][OW][C] or NULL (then next_bias
 * is ignored); next_bias may be NULL (0).  C_in % 8 == 0; C % 32 == 0 when y_bits is given.
 */
int bcnn_dwconv3x3_module(const void *x, const float *w, const float *bn_scale, const float *bn_shift, const float *prelu_slope,
                          const float *next_bias, void *y_real, void *y_bits, int B, int H, int W, int C_in, int R, int S,
                          void *stream);

/*
 * S x S average pooling with stride S on the identity path of a down-sampling block (Section 4.2.3), with the same
 * channel replication: y[b][oh][ow][c] = fp16(mean of the S x S window of x[..][c mod C_in]).  H % S == 0, W % S == 0,
 * C_in % 8 == 0.  S = 1 with R > 1 is plain replication of a map that a consumer needs materialised.
 */
int bcnn_avgpool(const void *x, void *y, int B, int H, int W, int C_in, int R, int S, void *stream);

/*
 * Head (Section 4.1, Figure 2; last rows of Table 1): global average pooling, pooled[b][c] = mean over the H*W pixels of
 * x (fp16 NHWC) as fp32 [B][C], and the fully connected layer logits[b][n] = sum_c pooled[b][c] * w[n][c] + bias[n]
 * (w fp32 [N][C], bias fp32 [N] or NULL, logits fp32 [B][N]).  C % 8 == 0.
 */
int bcnn_gap(const void *x, float *pooled, int B, int H, int W, int C, void *stream);
int bcnn_fc(const float *pooled, const float *w, const float *bias, float *logits, int B, int C, int N, void *stream);

/*
 * Fused stem: bcnn_pack followed by the first binary 1x1 convolution with its threshold epilogue, without
 * writing the packed sign tensor in between (Section 4.1: the stem uses the same block, so even the first
 * convolution is binary; Table 1 "stem replicate": 4 real channels replicated 8x to 32 sign channels;
 * Section 4.2.1: bias + sign, binary 1x1 convolution, batch norm + next sign folded into a threshold):
 *   s bit[b][h][w][c]  = (x[b][h][w][c mod C_in] + bias[c] >= 0),                c in [0, R*C_in)
 *   y bit[b][h][w][co] = (sum_c s[b][h][w][c] * w[co][c] >= thr[co])             s, w in {-1,+1}
 * The result is bit-identical to the two separate calls.
 *   x device fp32 NHWC [B][H][W][C_in];  bias device fp32 [R*C_in] or NULL;
 *   w_bits device, packed [C_out][R*C_in];  thr device int32 [C_out];  y_bits device, packed NHWC [B][H][W][C_out]
 * Supported shape: C_in = 4, R = 8, C_out = 32 (the paper's stem); anything else returns BCNN_ERR_UNSUPPORTED
 * and the caller issues the two calls.
 */
int bcnn_stem_fused(const float *x, const float *bias, const void *w_bits, const int32_t *thr, void *y_bits,
                    int B, int H, int W, int C_in, int R, int C_out, void *stream);

/*
 * The same four products with the inner-product engine chosen by the caller (used to
 * compare engines; BCNN_ENGINE_AUTO behaves like the calls above).  thr == NULL selects
 * the int32 output (`out` is int32), otherwise the packed output.  Returns
 * BCNN_ERR_UNSUPPORTED when the engine cannot run the shape.
 */
int bcnn_conv2d_b1_engine(int engine, const void *x_bits, const void *w_bits, const int32_t *thr,
                          void *out, int B, int H, int W, int C_in, int C_out,
                          int kh, int kw, int stride, int pad, void *stream);
int bcnn_gemm_b1_engine(int engine, const void *A_bits, const void *W_bits, const int32_t *thr,
                        void *out, int64_t M, int N, int K, void *stream);

/*
 * Prepared weights.  A layer's weights do not change between calls; expanding their sign bits to the signed bytes the
 * tensor cores multiply is done once, into a buffer the CALLER owns (the library never allocates), and the *_prepared
 * calls then stream that buffer by TMA instead of expanding the weight bits again for every tile of every call.
 * Worth it for wide layers and long K (C_out > 128: bcnn_prepared_preferred tells); results are bit-identical to the
 * plain calls.
 *   bcnn_prepared_weights_bytes(C_out, K)   size of the buffer for C_out rows of K = kh*kw*C_in bits (0 if invalid)
 *   bcnn_prepare_weights(w_bits, prepared, C_out, K, stream)   w_bits as in bcnn_conv2d_b1; prepared: device, 256-byte
 *                                           aligned, at least that many bytes; enqueues one small kernel
 *   bcnn_conv2d_b1_prepared / bcnn_gemm_b1_prepared   as bcnn_conv2d_b1_engine / bcnn_gemm_b1_engine with `prepared` in
 *                                           place of w_bits: thr == NULL selects the int32 output, else packed bits
 *   bcnn_prepared_preferred(...)            1 if the prepared call is expected to be the faster one for this shape
 * BCNN_ERR_UNSUPPORTED for shapes the engine does not take (the caller then uses the plain call).
 */
size_t bcnn_prepared_weights_bytes(int C_out, int K);
int bcnn_prepare_weights(const void *w_bits, void *prepared, int C_out, int K, void *stream);
int bcnn_conv2d_b1_prepared(const void *x_bits, const void *prepared, const int32_t *thr, void *out,
                            int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad, void *stream);
int bcnn_gemm_b1_prepared(const void *A_bits, const void *prepared, const int32_t *thr, void *out,
                          int64_t M, int N, int K, void *stream);
int bcnn_prepared_preferred(int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad, int fused);

/*
 * bcnn_conv2d_b1_fused for callers that can neither allocate device memory nor pass a buffer for prepared weights
 * (the paper has no counterpart: this is a property of the library, not of the method).  Think of code that runs
 * inside a memory plan it does not own - an inference runtime whose arena was sized before this layer existed, a
 * plug-in that is handed only its input and output tensors - or at a point where an allocation is not allowed or
 * would synchronise the device.  The call is bcnn_prepare_weights + bcnn_conv2d_b1_prepared with the prepared form
 * kept in a static device array inside the library: BCNN_STATIC_SCRATCH_BYTES (4 MiB) that every GPU which loads the
 * library holds until the process ends.  Arguments and result are exactly those of bcnn_conv2d_b1_fused (bit-identical
 * output; thr must not be NULL); it allocates and frees nothing.
 *   - BCNN_ERR_WORKSPACE when bcnn_prepared_weights_bytes(C_out, kh*kw*C_in) exceeds BCNN_STATIC_SCRATCH_BYTES
 *     (e.g. 512 output channels x 4608 bits fit, 1024 x 9216 do not), BCNN_ERR_UNSUPPORTED as for the prepared call.
 *   - The first call on a device looks up the array's device address; make that first call outside any stream capture.
 *   - All calls share the one array and each call overwrites all of it that it uses, so nothing needs clearing; but
 *     two calls that overlap on the GPU (different streams, or the same call from two threads) race on it.  Calls on
 *     one stream are ordered and safe.
 */
#define BCNN_STATIC_SCRATCH_BYTES (4u << 20)
int bcnn_conv2d_b1_fused_noalloc(const void *x_bits, const void *w_bits, const int32_t *thr, void *y_bits,
                                 int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad,
                                 void *stream);

/*
 * Which engine BCNN_ENGINE_AUTO runs for a convolution of this shape (fused != 0: the packed
 * output).  Returns a bcnn_engine value, or a negative bcnn_status for an invalid shape.
 * No pointers, no launch.  A GEMM is the shape (1, M, 1, K, N, 1, 1, 1, 0).
 */
int bcnn_auto_engine(int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad, int fused);

/*
 * Scratch memory (global memory beyond the inputs and outputs) a convolution of this shape needs, in bytes
 * (fused != 0: the packed output).  Every kernel of the library works out of its inputs, outputs, shared and
 * tensor memory, so this is 0 for every valid shape and no call takes a workspace argument; an invalid shape
 * also gives 0 (the call itself reports the error).  A GEMM is the shape (1, M, 1, K, N, 1, 1, 1, 0).
 */
size_t bcnn_workspace_bytes(int B, int H, int W, int C_in, int C_out, int kh, int kw, int stride, int pad, int fused);

/*
 * Device-side error word.  Kernels that wait on hardware barriers give up after a
 * bounded number of polls and record a non-zero code here instead of hanging.
 * Reads the word of the current device (synchronises that device) and clears it.
 * Returns the code (0 = no error) or a negative bcnn_status.  bcnn_status_string names the codes
 * (which engine, which of its roles gave up).
 */
int bcnn_device_error(void);

/*
 * The same check as a status: synchronises the current device, reads and clears the error word and returns
 * BCNN_OK, BCNN_ERR_TIMEOUT when a bounded wait had given up (the results of the calls since the last check
 * are then undefined; the context stays usable), or BCNN_ERR_CUDA.  *code, when not NULL, receives the raw
 * code (0 = none).
 */
int bcnn_device_status(int *code);

/*
 * Self-test of the bounded waits: launches one small kernel that allocates tensor memory and lets one warp
 * wait, with the library's wait helper and a limit of `polls` polls (1 <= polls <= 65536), on a barrier that
 * nothing ever arrives on.  The wait gives up, raises the CTA's abort flag (which the other warps of the CTA,
 * parked on a second barrier, notice), records BCNN_SELFTEST_TIMEOUT_CODE in the device error word, the kernel
 * frees its tensor memory and ends normally.  Enqueues only; bcnn_device_error() / bcnn_device_status() then
 * report the code.  Nothing else in the library calls it.
 */
#define BCNN_SELFTEST_TIMEOUT_CODE 120
int bcnn_selftest_wait_timeout(int polls, void *stream);

const char *bcnn_status_string(int status);
int bcnn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BCNN_H */
