// Convolution module with P parallel binary branches (Section 4.2.1, Figure 4 bottom) and, with P = kh * kw shifted
// branches, the paper's stand-in for a binary F x F convolution (last paragraph of Section 4.2.1).
//
// Per output element the module moves 2 bytes of identity and 2 bytes of real map (plus one bit), and every branch
// adds only C_in / 32 xor + popcount word operations: for the channel counts of the large feature maps (32 .. 128) the
// layer is bound by the real map's memory traffic, not by the inner product, so the branches run on the CUDA cores
// and the module arithmetic follows in the same thread, with no intermediate in global memory.
//
//   thread = one output pixel x 8 consecutive output channels (16 bytes of the fp16 maps, one byte of sign bits);
//   a CTA keeps the weights, batch-norm parameters and pad values of one slice of output channels (all branches) in
//   shared memory and walks row tiles with a grid stride.
// Arithmetic (bit-exact against the oracle): per branch  t_p = dot_p * scale_p + shift_p,  summed in branch order,
// then + identity, PReLU, fp16, sign of (stored value + next bias): one fp32 operation per step, no contraction.
#include "bcnn_common.cuh"
#include <cuda_fp16.h>

namespace bcnn {

namespace {

constexpr int THREADS = 256;
constexpr int MAX_SMEM = 200 * 1024;

__global__ void __launch_bounds__(THREADS)
conv_branches_kernel(const BranchProblem p, const int NS /* channels per slice */, const int tile_rows)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // [P][NS][cw] weight words, then [P][NS] scale, [P][NS] shift, [P][NS] pad dot, [NS] slope, [NS] next bias
    uint32_t *w_s = reinterpret_cast<uint32_t *>(smem_raw);
    float *scale_s = reinterpret_cast<float *>(w_s + (size_t)p.P * NS * p.cw);
    float *shift_s = scale_s + p.P * NS;
    int *pad_s = reinterpret_cast<int *>(shift_s + p.P * NS);
    float *slope_s = reinterpret_cast<float *>(pad_s + p.P * NS);
    float *nb_s = slope_s + NS;

    const int n0 = blockIdx.y * NS;                            // first channel of this CTA's slice
    const int cn = min(NS, p.C_out - n0);
    for (int i = threadIdx.x; i < p.P * NS * p.cw; i += THREADS) {
        const int k = i % p.cw, c = (i / p.cw) % NS, br = i / (p.cw * NS);
        w_s[i] = c < cn ? __ldg(p.w + ((long)br * p.C_out + n0 + c) * p.cw + k) : 0u;
    }
    for (int i = threadIdx.x; i < p.P * NS; i += THREADS) {
        const int c = i % NS, br = i / NS;
        const bool have = c < cn;
        scale_s[i] = have ? __ldg(p.bn_scale + (long)br * p.C_out + n0 + c) : 0.f;
        shift_s[i] = have ? __ldg(p.bn_shift + (long)br * p.C_out + n0 + c) : 0.f;
        pad_s[i] = (have && p.pad_dot) ? __ldg(p.pad_dot + (long)br * p.C_out + n0 + c) : 0;
    }
    for (int i = threadIdx.x; i < NS; i += THREADS) {
        slope_s[i] = i < cn ? __ldg(p.slope + n0 + i) : 0.f;
        nb_s[i] = (i < cn && p.next_bias) ? __ldg(p.next_bias + n0 + i) : 0.f;
    }
    __syncthreads();

    const int groups = NS / 8;                                 // 8-channel groups of the slice
    const int rpp = THREADS / groups;                          // rows per pass
    const int g = threadIdx.x % groups, rsub = threadIdx.x / groups;
    if (rsub >= rpp || 8 * g >= cn) return;
    const int ch = 8 * g;                                      // first channel (within the slice) of this thread
    const int pw = p.P * p.cw;                                 // words per input pixel
    const int K = p.C_in;
    const bool shifted = p.kh * p.kw > 1;
    const long HW = (long)p.H * p.W;

    for (long tile = blockIdx.x; tile * tile_rows < p.M; tile += gridDim.x) {
        const long row_end = min(p.M, (tile + 1) * (long)tile_rows);
        for (long m = tile * tile_rows + rsub; m < row_end; m += rpp) {
            int h = 0, w = 0;
            if (shifted) {
                const long rem = m % HW;
                h = (int)(rem / p.W);
                w = (int)(rem - (long)h * p.W);
            }
            float t[8];
#pragma unroll 1
            for (int br = 0; br < p.P; ++br) {
                int dot[8];
                long pix = m;
                bool inside = true;
                if (shifted) {
                    const int r = br / p.kw, tt = br - r * p.kw;
                    const int dy = r - (p.kh - 1) / 2, dx = tt - (p.kw - 1) / 2;
                    inside = h + dy >= 0 && h + dy < p.H && w + dx >= 0 && w + dx < p.W;
                    pix = m + (long)dy * p.W + dx;
                }
                if (inside) {
                    int pc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
                    const uint32_t *xa = p.x + pix * pw + (long)br * p.cw;
                    const uint32_t *wb = w_s + ((size_t)br * NS + ch) * p.cw;
                    for (int k = 0; k < p.cw; ++k) {
                        const uint32_t a = __ldg(xa + k);
#pragma unroll
                        for (int c = 0; c < 8; ++c) pc[c] += __popc(a ^ wb[c * p.cw + k]);
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c) dot[c] = K - 2 * pc[c];
                } else {
#pragma unroll
                    for (int c = 0; c < 8; ++c) dot[c] = pad_s[br * NS + ch + c];
                }
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    float tp = __fmul_rn(__int2float_rn(dot[c]), scale_s[br * NS + ch + c]);
                    tp = __fadd_rn(tp, shift_s[br * NS + ch + c]);
                    t[c] = br == 0 ? tp : __fadd_rn(t[c], tp);
                }
            }
            const long e0 = m * p.C_out + n0 + ch;                 // first element of this thread's 8 channels
            uint4 idv = make_uint4(0u, 0u, 0u, 0u);
            if (p.identity) idv = __ldg(reinterpret_cast<const uint4 *>(p.identity + e0));
            const uint32_t idw[4] = {idv.x, idv.y, idv.z, idv.w};
            uint32_t ow[4];
            uint32_t bits = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float2 idf = __half22float2(*reinterpret_cast<const __half2 *>(&idw[q]));
                float r[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float u = p.identity ? __fadd_rn(t[2 * q + e], e ? idf.y : idf.x) : t[2 * q + e];
                    r[e] = (u >= 0.0f) ? u : __fmul_rn(slope_s[ch + 2 * q + e], u);
                }
                const __half2 y2 = __floats2half2_rn(r[0], r[1]);
                ow[q] = *reinterpret_cast<const uint32_t *>(&y2);
                const float2 yf = __half22float2(y2);
                bits |= (__fadd_rn(yf.x, nb_s[ch + 2 * q]) >= 0.0f ? 1u : 0u) << (2 * q);
                bits |= (__fadd_rn(yf.y, nb_s[ch + 2 * q + 1]) >= 0.0f ? 1u : 0u) << (2 * q + 1);
            }
            *reinterpret_cast<uint4 *>(p.y_real + e0) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
            if (p.y_bits) p.y_bits[e0 >> 3] = (uint8_t)bits;
        }
    }
}

}  // namespace

int launch_conv_branches(const BranchProblem &p, cudaStream_t stream)
{
    // slice of output channels whose weights and parameters fit in shared memory (a multiple of 32, a divisor of the
    // thread count in 8-channel groups)
    const long per_channel = (long)p.P * (p.cw * 4 + 12) + 8;
    int NS = 256;
    while (NS > 32 && (NS * per_channel > MAX_SMEM || NS / 2 >= p.C_out)) NS /= 2;
    if (NS * per_channel > MAX_SMEM) return BCNN_ERR_UNSUPPORTED;
    const int slices = (p.C_out + NS - 1) / NS;
    const int smem = (int)(NS * per_channel);
    int dev = 0, sms = 148;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int tile_rows = 8 * (THREADS / (NS / 8));            // eight passes per tile
    const long tiles = (p.M + tile_rows - 1) / tile_rows;
    long gx = (long)sms * 4 / slices;
    if (gx < 1) gx = 1;
    if (gx > tiles) gx = tiles;
    if (cudaFuncSetAttribute(conv_branches_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MAX_SMEM) != cudaSuccess) return BCNN_ERR_CUDA;
    conv_branches_kernel<<<dim3((unsigned)gx, (unsigned)slices), THREADS, smem, stream>>>(p, NS, tile_rows);
    return cudaGetLastError() == cudaSuccess ? BCNN_OK : BCNN_ERR_CUDA;
}

}  // namespace bcnn
