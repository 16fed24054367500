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
    // Per-channel vectors of the slice, each stored as two 16-byte arrays over its 8-channel groups (channels 8g..8g+3
    // at [2q][g], 8g+4..8g+7 at [2q+1][g]) so that a warp's groups read consecutive 16-byte pieces without bank
    // conflicts: vectors q = br * cw + k are the weight words, then per branch scale, shift, pad dot, then slope and
    // next bias.
    uint32_t *sm = reinterpret_cast<uint32_t *>(smem_raw);
    const int groups = NS / 8;                                 // 8-channel groups of the slice
    const int n0 = blockIdx.y * NS;                            // first channel of this CTA's slice
    const int cn = min(NS, p.C_out - n0);
    const int nw = p.P * p.cw;                                 // weight vectors
    const int nvec = nw + 3 * p.P + 2;
    auto slot = [&](int q, int c) { return ((2 * q + ((c & 7) >> 2)) * groups + (c >> 3)) * 4 + (c & 3); };
    for (int i = threadIdx.x; i < nvec * NS; i += THREADS) {
        const int q = i / NS, c = i % NS;
        const bool have = c < cn;
        uint32_t val = 0;
        if (q < nw) {
            const int br = q / p.cw, k = q - br * p.cw;
            if (have) val = __ldg(p.w + ((long)br * p.C_out + n0 + c) * p.cw + k);
        } else if (q < nw + 3 * p.P) {
            const int br = (q - nw) / 3, kind = (q - nw) % 3;
            if (have) {
                if (kind == 0) val = __float_as_uint(__ldg(p.bn_scale + (long)br * p.C_out + n0 + c));
                else if (kind == 1) val = __float_as_uint(__ldg(p.bn_shift + (long)br * p.C_out + n0 + c));
                else val = p.pad_dot ? (uint32_t)__ldg(p.pad_dot + (long)br * p.C_out + n0 + c) : 0u;
            }
        } else if (q == nw + 3 * p.P) {
            if (have) val = __float_as_uint(__ldg(p.slope + n0 + c));
        } else {
            if (have && p.next_bias) val = __float_as_uint(__ldg(p.next_bias + n0 + c));
        }
        sm[slot(q, c)] = val;
    }
    __syncthreads();
    const uint4 *vec = reinterpret_cast<const uint4 *>(smem_raw);

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
                    for (int k = 0; k < p.cw; ++k) {
                        const uint32_t a = __ldg(xa + k);
                        const uint4 w0 = vec[(2 * (br * p.cw + k)) * groups + g], w1 = vec[(2 * (br * p.cw + k) + 1) * groups + g];
                        pc[0] += __popc(a ^ w0.x); pc[1] += __popc(a ^ w0.y); pc[2] += __popc(a ^ w0.z); pc[3] += __popc(a ^ w0.w);
                        pc[4] += __popc(a ^ w1.x); pc[5] += __popc(a ^ w1.y); pc[6] += __popc(a ^ w1.z); pc[7] += __popc(a ^ w1.w);
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c) dot[c] = K - 2 * pc[c];
                } else {
                    const uint4 d0 = vec[(2 * (nw + 3 * br + 2)) * groups + g], d1 = vec[(2 * (nw + 3 * br + 2) + 1) * groups + g];
                    dot[0] = (int)d0.x; dot[1] = (int)d0.y; dot[2] = (int)d0.z; dot[3] = (int)d0.w;
                    dot[4] = (int)d1.x; dot[5] = (int)d1.y; dot[6] = (int)d1.z; dot[7] = (int)d1.w;
                }
                const uint4 s0 = vec[(2 * (nw + 3 * br)) * groups + g], s1 = vec[(2 * (nw + 3 * br) + 1) * groups + g];
                const uint4 h0 = vec[(2 * (nw + 3 * br + 1)) * groups + g], h1 = vec[(2 * (nw + 3 * br + 1) + 1) * groups + g];
                const uint32_t sc8[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w}, sh8[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    float tp = __fmul_rn(__int2float_rn(dot[c]), __uint_as_float(sc8[c]));
                    tp = __fadd_rn(tp, __uint_as_float(sh8[c]));
                    t[c] = br == 0 ? tp : __fadd_rn(t[c], tp);
                }
            }
            const long e0 = m * p.C_out + n0 + ch;                 // first element of this thread's 8 channels
            uint4 idv = make_uint4(0u, 0u, 0u, 0u);
            if (p.identity) idv = __ldg(reinterpret_cast<const uint4 *>(p.identity + e0));
            const uint32_t idw[4] = {idv.x, idv.y, idv.z, idv.w};
            uint32_t ow[4];
            uint32_t bits = 0;
            const uint4 l0 = vec[(2 * (nw + 3 * p.P)) * groups + g], l1 = vec[(2 * (nw + 3 * p.P) + 1) * groups + g];
            const uint4 b0 = vec[(2 * (nw + 3 * p.P + 1)) * groups + g], b1 = vec[(2 * (nw + 3 * p.P + 1) + 1) * groups + g];
            const uint32_t sl8[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w}, nb8[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float2 idf = __half22float2(*reinterpret_cast<const __half2 *>(&idw[q]));
                float r[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const float u = p.identity ? __fadd_rn(t[2 * q + e], e ? idf.y : idf.x) : t[2 * q + e];
                    r[e] = (u >= 0.0f) ? u : __fmul_rn(__uint_as_float(sl8[2 * q + e]), u);
                }
                const __half2 y2 = __floats2half2_rn(r[0], r[1]);
                ow[q] = *reinterpret_cast<const uint32_t *>(&y2);
                const float2 yf = __half22float2(y2);
                bits |= (__fadd_rn(yf.x, __uint_as_float(nb8[2 * q])) >= 0.0f ? 1u : 0u) << (2 * q);
                bits |= (__fadd_rn(yf.y, __uint_as_float(nb8[2 * q + 1])) >= 0.0f ? 1u : 0u) << (2 * q + 1);
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
