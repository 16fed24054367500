// The real-valued vector operations of the paper's building block and head: the 3x3 convolution module (real depth-
// wise 3x3 convolution, batch norm, PReLU; Section 4.2.1), S x S / S average pooling on the identity path of a down-
// sampling block (Section 4.2.3), channel replication as indexing (Section 4.2.2: channel c reads channel c mod C_in,
// no copy), global average pooling and the fully connected layer (Section 4.1).  All of them are bound by the memory
// traffic of the fp16 NHWC maps: a thread handles 8 consecutive channels (16 bytes) of one output pixel, arithmetic in
// fp32.  The depth-wise module can also emit the next binary module's sign bits (bias + sign of the stored value), so
// that the map is not read again by a pack pass.
#include "bcnn_common.cuh"
#include <cuda_fp16.h>

namespace bcnn {

namespace {

__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8])
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&w[q]));
        f[2 * q] = a.x;
        f[2 * q + 1] = a.y;
    }
}

// x fp16 [B][H][W][C_in] -> y fp16 [B][OH][OW][C], C = R * C_in; w fp32 [C][3][3].
// The block's thread count is a multiple of the 8-channel groups, so a thread keeps its group; weights (tap-major, so
// that a warp's groups read consecutive 32-byte pieces) and per-channel values sit in shared memory.  A block walks a
// CONTIGUOUS range of output pixels, row after row, so that the input rows shared by vertically adjacent outputs are
// still in L1 when they are needed again (with a grid-stride walk every tap came from L2: nine times the input's
// bytes); a thread's pixel coordinates advance by the block's pass size, by carries.
__global__ void __launch_bounds__(256)
dwconv3x3_module_kernel(const uint16_t *x, const float *w, const float *scale, const float *shift, const float *slope,
                        const float *next_bias, uint16_t *y, uint8_t *y_bits,
                        int B, int H, int W, int C_in, int C, int S, int OH, int OW)
{
    // 13 per-channel vectors (nine taps, scale, shift, slope, next bias), each stored as two float4 arrays over the
    // 8-channel groups - channels 8g..8g+3 at [2q][g], 8g+4..8g+7 at [2q+1][g] - so that a warp's groups read
    // consecutive 16-byte pieces (one float per lane, or 32-byte pieces per lane, would conflict 8- and 2-way)
    extern __shared__ __align__(16) float dw_smem[];
    const int groups = C / 8;
    const float4 *vec = reinterpret_cast<const float4 *>(dw_smem);
    for (int i = threadIdx.x; i < 13 * C; i += blockDim.x) {
        const int q = i / C, c = i % C;
        float val;
        if (q < 9) val = __ldg(w + c * 9 + q);
        else if (q == 9) val = __ldg(scale + c);
        else if (q == 10) val = __ldg(shift + c);
        else if (q == 11) val = __ldg(slope + c);
        else val = next_bias ? __ldg(next_bias + c) : 0.f;
        dw_smem[((2 * q + ((c & 7) >> 2)) * groups + (c >> 3)) * 4 + (c & 3)] = val;
    }
    __syncthreads();
    const int g = threadIdx.x % groups, ppb = blockDim.x / groups;      // pixels per block and pass
    const int c0 = 8 * g, ci0 = c0 % C_in;                     // replication: channel c reads channel c mod C_in
    const unsigned npix = (unsigned)B * OH * OW;
    const unsigned per_block = ((npix + gridDim.x - 1) / gridDim.x + ppb - 1) / ppb * ppb;     // a multiple of the pass size
    const unsigned stride = (unsigned)ppb;
    unsigned pix = blockIdx.x * per_block + threadIdx.x / groups;
    const unsigned pix_end = min(npix, (blockIdx.x + 1) * per_block);
    int b = (int)(pix / ((unsigned)OH * OW)), oh = (int)((pix / OW) % OH), ow = (int)(pix % OW);
    const int db = (int)(stride / ((unsigned)OH * OW)), doh = (int)((stride / OW) % OH), dow = (int)(stride % OW);
    for (; pix < pix_end; pix += stride) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        // all nine taps are requested before the first is used (predicated loads, zero outside the image)
        uint4 v[9];
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const int ih = oh * S - 1 + r;
#pragma unroll
            for (int t = 0; t < 3; ++t) {
                const int iw = ow * S - 1 + t;
                const bool ok = ih >= 0 && ih < H && iw >= 0 && iw < W;
                v[r * 3 + t] = ok ? __ldg(reinterpret_cast<const uint4 *>(x + (((long)b * H + ih) * W + iw) * C_in + ci0)) : make_uint4(0u, 0u, 0u, 0u);
            }
        }
#pragma unroll
        for (int r = 0; r < 3; ++r) {
#pragma unroll
            for (int t = 0; t < 3; ++t) {
                float xv[8];
                unpack8(v[r * 3 + t], xv);
                const float4 w0 = vec[(2 * (r * 3 + t)) * groups + g], w1 = vec[(2 * (r * 3 + t) + 1) * groups + g];
                acc[0] = fmaf(xv[0], w0.x, acc[0]); acc[1] = fmaf(xv[1], w0.y, acc[1]);
                acc[2] = fmaf(xv[2], w0.z, acc[2]); acc[3] = fmaf(xv[3], w0.w, acc[3]);
                acc[4] = fmaf(xv[4], w1.x, acc[4]); acc[5] = fmaf(xv[5], w1.y, acc[5]);
                acc[6] = fmaf(xv[6], w1.z, acc[6]); acc[7] = fmaf(xv[7], w1.w, acc[7]);
            }
        }
        uint32_t ow4[4];
        uint32_t bits = 0;
        float sc8[8], sh8[8], sl8[8], nb8[8];
        {
            const float4 a0 = vec[18 * groups + g], a1 = vec[19 * groups + g], b0 = vec[20 * groups + g], b1 = vec[21 * groups + g];
            const float4 d0 = vec[22 * groups + g], d1 = vec[23 * groups + g], e0 = vec[24 * groups + g], e1 = vec[25 * groups + g];
            sc8[0] = a0.x; sc8[1] = a0.y; sc8[2] = a0.z; sc8[3] = a0.w; sc8[4] = a1.x; sc8[5] = a1.y; sc8[6] = a1.z; sc8[7] = a1.w;
            sh8[0] = b0.x; sh8[1] = b0.y; sh8[2] = b0.z; sh8[3] = b0.w; sh8[4] = b1.x; sh8[5] = b1.y; sh8[6] = b1.z; sh8[7] = b1.w;
            sl8[0] = d0.x; sl8[1] = d0.y; sl8[2] = d0.z; sl8[3] = d0.w; sl8[4] = d1.x; sl8[5] = d1.y; sl8[6] = d1.z; sl8[7] = d1.w;
            nb8[0] = e0.x; nb8[1] = e0.y; nb8[2] = e0.z; nb8[3] = e0.w; nb8[4] = e1.x; nb8[5] = e1.y; nb8[6] = e1.z; nb8[7] = e1.w;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float r2[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const float tt = fmaf(acc[2 * q + e], sc8[2 * q + e], sh8[2 * q + e]);
                r2[e] = tt >= 0.f ? tt : sl8[2 * q + e] * tt;
            }
            const __half2 y2 = __floats2half2_rn(r2[0], r2[1]);
            ow4[q] = *reinterpret_cast<const uint32_t *>(&y2);
            if (y_bits) {
                const float2 yf = __half22float2(y2);
                bits |= (__fadd_rn(yf.x, nb8[2 * q]) >= 0.f ? 1u : 0u) << (2 * q);
                bits |= (__fadd_rn(yf.y, nb8[2 * q + 1]) >= 0.f ? 1u : 0u) << (2 * q + 1);
            }
        }
        *reinterpret_cast<uint4 *>(y + (long)pix * C + c0) = make_uint4(ow4[0], ow4[1], ow4[2], ow4[3]);
        if (y_bits) y_bits[((long)pix * C + c0) >> 3] = (uint8_t)bits;
        // next pixel of this thread: + stride, by carries
        ow += dow;
        if (ow >= OW) { ow -= OW; ++oh; }
        oh += doh;
        if (oh >= OH) { oh -= OH; ++b; }
        b += db;
    }
}

__global__ void __launch_bounds__(256)
avgpool_kernel(const uint16_t *x, uint16_t *y, int B, int H, int W, int C_in, int C, int S)
{
    const int OH = H / S, OW = W / S, groups = C / 8;
    const long total = (long)B * OH * OW * groups;
    const float inv = 1.0f / (float)(S * S);
    for (long i = (long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
        const int g = (int)(i % groups);
        const long pix = i / groups;
        const int ow = (int)(pix % OW), oh = (int)((pix / OW) % OH), b = (int)(pix / ((long)OW * OH));
        const int c0 = 8 * g, ci0 = c0 % C_in;
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int r = 0; r < S; ++r)
            for (int t = 0; t < S; ++t) {
                float xv[8];
                unpack8(__ldg(reinterpret_cast<const uint4 *>(x + (((long)b * H + oh * S + r) * W + ow * S + t) * C_in + ci0)), xv);
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[c] += xv[c];
            }
        uint32_t o[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const __half2 y2 = __floats2half2_rn(acc[2 * q] * inv, acc[2 * q + 1] * inv);
            o[q] = *reinterpret_cast<const uint32_t *>(&y2);
        }
        *reinterpret_cast<uint4 *>(y + pix * C + c0) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// pooled[b][c] = mean over HW pixels; thread = (image, 8 channels); 4 partial sums in flight per channel
__global__ void __launch_bounds__(256)
gap_kernel(const uint16_t *x, float *pooled, int B, int HW, int C)
{
    const int groups = C / 8;
    const long total = (long)B * groups;
    for (long i = (long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long)gridDim.x * blockDim.x) {
        const int g = (int)(i % groups), b = (int)(i / groups);
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        const uint16_t *src = x + (long)b * HW * C + 8 * g;
        for (int q = 0; q < HW; ++q) {
            float xv[8];
            unpack8(__ldg(reinterpret_cast<const uint4 *>(src + (long)q * C)), xv);
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[c] += xv[c];
        }
        const float inv = 1.0f / (float)HW;
        float4 *dst = reinterpret_cast<float4 *>(pooled + (long)b * C + 8 * g);
        dst[0] = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
        dst[1] = make_float4(acc[4] * inv, acc[5] * inv, acc[6] * inv, acc[7] * inv);
    }
}

// logits[b][n] = sum_c pooled[b][c] * w[n][c] + bias[n].  A CTA takes FC_IMAGES images (their pooled rows in shared
// memory) and all outputs; a warp takes outputs warp, warp + 8, ...: lanes stride over c with 16-byte weight loads
// (each weight row is read once per CTA), then a shuffle reduction.
constexpr int FC_IMAGES = 4;
__global__ void __launch_bounds__(256)
fc_kernel(const float *pooled, const float *w, const float *bias, float *logits, int B, int C, int N)
{
    extern __shared__ __align__(16) float fc_smem[];           // [FC_IMAGES][C]
    const int b0 = blockIdx.x * FC_IMAGES;
    const int nb = min(FC_IMAGES, B - b0);
    for (int i = threadIdx.x; i < FC_IMAGES * C; i += blockDim.x)
        fc_smem[i] = (i / C) < nb ? __ldg(pooled + (long)b0 * C + i) : 0.f;
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // blockIdx.y takes every gridDim.y-th group of eight outputs
    for (int n = blockIdx.y * 8 + warp; n < N; n += 8 * gridDim.y) {
        float acc[FC_IMAGES] = {0.f, 0.f, 0.f, 0.f};
        const float4 *wr = reinterpret_cast<const float4 *>(w + (long)n * C);
        for (int c4 = lane; c4 < C / 4; c4 += 32) {
            const float4 wv = __ldg(wr + c4);
#pragma unroll
            for (int im = 0; im < FC_IMAGES; ++im) {
                const float4 pv = reinterpret_cast<const float4 *>(fc_smem + im * C)[c4];
                acc[im] = fmaf(pv.x, wv.x, fmaf(pv.y, wv.y, fmaf(pv.z, wv.z, fmaf(pv.w, wv.w, acc[im]))));
            }
        }
#pragma unroll
        for (int im = 0; im < FC_IMAGES; ++im) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc[im] += __shfl_xor_sync(0xffffffffu, acc[im], off);
        }
        float v = acc[0];
        if (lane == 1) v = acc[1];
        if (lane == 2) v = acc[2];
        if (lane == 3) v = acc[3];
        if (lane < nb) logits[(long)(b0 + lane) * N + n] = v + (bias ? __ldg(bias + n) : 0.f);
    }
}

int grid_for(long total_threads)
{
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long blocks = (total_threads + 255) / 256;
    const long cap = (long)sms * 16;
    return (int)(blocks < cap ? (blocks < 1 ? 1 : blocks) : cap);
}

}  // namespace

int launch_dwconv3x3_module(const uint16_t *x, const float *w, const float *scale, const float *shift, const float *slope,
                            const float *next_bias, uint16_t *y, uint8_t *y_bits, int B, int H, int W, int C_in, int R, int S,
                            cudaStream_t stream)
{
    const int C = C_in * R, OH = (H + 2 - 3) / S + 1, OW = (W + 2 - 3) / S + 1;
    const int groups = C / 8;
    const int smem = 13 * C * 4;
    if (groups > 256 || smem > 200 * 1024) return BCNN_ERR_UNSUPPORTED;      // more than 2048 channels
    if ((long)B * OH * OW >= (1L << 31)) return BCNN_ERR_UNSUPPORTED;         // pixel indices are 32-bit
    const int threads = (256 / groups) * groups;                            // <= 256, a multiple of groups
    const long passes = ((long)B * OH * OW + threads / groups - 1) / (threads / groups);
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long cap = (long)sms * 8;
    const unsigned blocks = (unsigned)(passes < cap ? passes : cap);
    if (cudaFuncSetAttribute(dwconv3x3_module_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) return BCNN_ERR_CUDA;
    dwconv3x3_module_kernel<<<blocks, threads, smem, stream>>>(x, w, scale, shift, slope, next_bias, y, y_bits,
                                                               B, H, W, C_in, C, S, OH, OW);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

int launch_avgpool(const uint16_t *x, uint16_t *y, int B, int H, int W, int C_in, int R, int S, cudaStream_t stream)
{
    const int C = C_in * R;
    avgpool_kernel<<<grid_for((long)B * (H / S) * (W / S) * (C / 8)), 256, 0, stream>>>(x, y, B, H, W, C_in, C, S);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

int launch_gap(const uint16_t *x, float *pooled, int B, int HW, int C, cudaStream_t stream)
{
    gap_kernel<<<grid_for((long)B * (C / 8)), 256, 0, stream>>>(x, pooled, B, HW, C);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

int launch_fc(const float *pooled, const float *w, const float *bias, float *logits, int B, int C, int N, cudaStream_t stream)
{
    const int smem = FC_IMAGES * C * 4;
    if (smem > 200 * 1024) return BCNN_ERR_UNSUPPORTED;
    if (cudaFuncSetAttribute(fc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess) return BCNN_ERR_CUDA;
    const int images = (B + FC_IMAGES - 1) / FC_IMAGES;
    int ny = 1;                                     // enough CTAs to fill the GPU a few times over
    while (images * ny < 592 && ny * 8 < N) ny *= 2;
    fc_kernel<<<dim3(images, ny), 256, smem, stream>>>(pooled, w, bias, logits, B, C, N);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace bcnn
