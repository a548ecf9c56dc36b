// First-layer kernel of a stack: few input channels (C <= 4, e.g. RGB) and at most 64 filters on the FP32 pipes, writing
// its result directly as the split, channels-innermost operand tensor of the tensor-core layer that follows.
//
// Why a kernel of its own: such a layer is bound by its output (Section 6.2's first VGG layer moves 21x more bytes out
// than in), and in a stack the output is needed as [S][N][H][W][Cp] hi/lo planes, not as NCHW.  Here one thread owns one
// output pixel and all filters: the 3x3xC neighbourhood sits in registers, the weights -- the pattern-sparse kernels
// written out as 9*C taps with zeros where the pattern has none -- are kernel parameters, so every FFMA takes its
// weight straight from the constant bank and the filter loop is straight-line code.  The 64 results of a pixel are one
// 128-byte row per operand plane; a warp's 32 consecutive pixels are 4 KB of contiguous memory per plane, written
// through a swizzled shared-memory transpose as fully coalesced 16-byte stores.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "kernels.hpp"

namespace patdnn {
namespace {

constexpr int kWarps = 8;

template <int C, typename T>
__global__ void __launch_bounds__(kWarps * 32, 2)
conv_smallc_split_kernel(const __grid_constant__ SmallCWeights wt, const T *__restrict__ in, uint16_t *__restrict__ dst,
                         int N, int H, int W, int F, int relu, int Cp, int S) {
    __shared__ __align__(16) unsigned char stage[kWarps][32 * 128];
    pdl_trigger();
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long P = static_cast<long long>(N) * H * W;
    const long long plane_out = P * Cp;                          // elements per operand plane
    unsigned char *st = stage[warp];
    for (long long p0 = (static_cast<long long>(blockIdx.x) * kWarps + warp) * 32; p0 < P;
         p0 += static_cast<long long>(gridDim.x) * kWarps * 32) {
        const long long pix = p0 + lane;
        const bool ok = pix < P;
        float v[9 * C];
        {
            // 32-bit index arithmetic (the launcher checks N*H*W and N*C*H*W < 2^31): 64-bit divisions are subroutines
            const unsigned q = ok ? static_cast<unsigned>(pix) : 0u;
            const unsigned uw = static_cast<unsigned>(W), uh = static_cast<unsigned>(H);
            const unsigned r = q / uw;
            const int x = static_cast<int>(q - r * uw);
            const unsigned n = r / uh;
            const int y = static_cast<int>(r - n * uh);
            const bool rok[3] = {ok && y >= 1, ok, ok && y + 1 < H};
            const bool cok[3] = {x >= 1, true, x + 1 < W};
            const T *base = in + (static_cast<size_t>(n) * C * H + y) * W + x;     // channel 0, centre tap
            const int plane = H * W;
#pragma unroll
            for (int c = 0; c < C; ++c)
#pragma unroll
                for (int dy = 0; dy < 3; ++dy)
#pragma unroll
                    for (int dx = 0; dx < 3; ++dx) {
                        float t = 0.f;
                        if (rok[dy] && cok[dx]) t = static_cast<float>(base[c * plane + (dy - 1) * W + (dx - 1)]);
                        v[9 * c + 3 * dy + dx] = t;
                    }
        }
        // 64 filters, straight-line: weights are immediate constant-bank operands
        uint32_t hi[32], lo[32];
#pragma unroll
        for (int f = 0; f < 64; f += 8) {                        // eight independent accumulation chains at a time
            float a[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) a[j] = wt.bias[f + j];
#pragma unroll
            for (int k = 0; k < 9 * C; ++k)
#pragma unroll
                for (int j = 0; j < 8; ++j) a[j] = fmaf(wt.w[(f + j) * kSmallCTaps + k], v[k], a[j]);
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                float a0 = a[j], a1 = a[j + 1];
                if (relu) { a0 = fmaxf(a0, 0.f); a1 = fmaxf(a1, 0.f); }
                if (S == 2) {
                    const __nv_bfloat162 h2 = __floats2bfloat162_rn(a0, a1);
                    const float2 hf = __bfloat1622float2(h2);
                    const __nv_bfloat162 l2 = __floats2bfloat162_rn(a0 - hf.x, a1 - hf.y);
                    hi[(f + j) >> 1] = *reinterpret_cast<const uint32_t *>(&h2);
                    lo[(f + j) >> 1] = *reinterpret_cast<const uint32_t *>(&l2);
                } else {
                    const __half2 h2 = __floats2half2_rn(a0, a1);
                    hi[(f + j) >> 1] = *reinterpret_cast<const uint32_t *>(&h2);
                    lo[(f + j) >> 1] = 0u;
                }
            }
        }
        // transpose through shared memory, one plane at a time: row = lane's pixel (128 bytes), chunk index XOR (lane & 7)
        const int rows = static_cast<int>(P - p0 < 32 ? P - p0 : 32);
#pragma unroll
        for (int sp = 0; sp < 2; ++sp) {
            if (sp >= S) break;
            __syncwarp();
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                const uint32_t *s4 = (sp == 0 ? hi : lo) + 4 * ch;
                *reinterpret_cast<uint4 *>(st + lane * 128 + ((ch ^ (lane & 7)) << 4)) = make_uint4(s4[0], s4[1], s4[2], s4[3]);
            }
            __syncwarp();
            unsigned char *g = reinterpret_cast<unsigned char *>(dst + sp * plane_out + p0 * Cp);
            if (Cp == 64) {                                      // the 32 rows are one contiguous 4 KB block
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int idx = k * 32 + lane, row = idx >> 3, ch = idx & 7;
                    if (row < rows)
                        *reinterpret_cast<uint4 *>(g + idx * 16) = *reinterpret_cast<const uint4 *>(st + row * 128 + ((ch ^ (row & 7)) << 4));
                }
            } else {                                             // wider channel pitch: 128-byte rows at a pitch of 2*Cp bytes
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int idx = k * 32 + lane, row = idx >> 3, ch = idx & 7;
                    if (row < rows)
                        *reinterpret_cast<uint4 *>(g + static_cast<size_t>(row) * Cp * 2 + ch * 16) =
                            *reinterpret_cast<const uint4 *>(st + row * 128 + ((ch ^ (row & 7)) << 4));
                }
            }
        }
    }
    (void)F;
}

template <int C>
cudaError_t launch_c(const SmallCWeights &wt, const void *in, int in_is_half, void *dst, int N, int H, int W, int F, int relu,
                     int Cp, int S, cudaStream_t st) {
    const long long P = static_cast<long long>(N) * H * W;
    if (P * C >= (1ll << 31)) return cudaErrorInvalidValue;      // the kernel indexes pixels with 32 bits
    const long long blocks_needed = (P + kWarps * 32 - 1) / (kWarps * 32);
    const int grid = static_cast<int>(blocks_needed < sm_count() * 8 ? blocks_needed : sm_count() * 8);
    if (in_is_half)
        return launch_pdl(conv_smallc_split_kernel<C, __half>, dim3(grid), dim3(kWarps * 32), 0, st, 1, wt,
                          static_cast<const __half *>(in), static_cast<uint16_t *>(dst), N, H, W, F, relu, Cp, S);
    return launch_pdl(conv_smallc_split_kernel<C, float>, dim3(grid), dim3(kWarps * 32), 0, st, 1, wt,
                      static_cast<const float *>(in), static_cast<uint16_t *>(dst), N, H, W, F, relu, Cp, S);
}

}  // namespace

bool smallc_split_supported(int F, int C) { return C >= 1 && C <= 4 && F >= 1 && F <= 64; }

void build_smallc_weights(const Fkw &fkw, const std::vector<float> &bias, SmallCWeights &wt) {
    for (float &x : wt.w) x = 0.f;
    for (float &x : wt.bias) x = 0.f;
    for (int i = 0; i < fkw.F; ++i) {
        const int f = fkw.reorder[i];
        wt.bias[f] = bias[f];
        for (int32_t k = fkw.offset[i]; k < fkw.offset[i + 1]; ++k) {
            const int c = fkw.index[k];
            const uint32_t mask = fkw.patterns[fkw.kernel_pid[k]];
            int j = 0;
            for (int t = 0; t < 9; ++t)
                if ((mask >> t) & 1u) wt.w[f * kSmallCTaps + 9 * c + t] = fkw.weight_f32[static_cast<size_t>(k) * 4 + j++];
        }
    }
}

cudaError_t launch_smallc_split(const SmallCWeights &wt, const void *in, int in_is_half, void *dst, int N, int C, int H, int W,
                                int F, int relu, int Cp, int S, cudaStream_t st) {
    if (N == 0) return cudaSuccess;
    switch (C) {
        case 1: return launch_c<1>(wt, in, in_is_half, dst, N, H, W, F, relu, Cp, S, st);
        case 2: return launch_c<2>(wt, in, in_is_half, dst, N, H, W, F, relu, Cp, S, st);
        case 3: return launch_c<3>(wt, in, in_is_half, dst, N, H, W, F, relu, Cp, S, st);
        case 4: return launch_c<4>(wt, in, in_is_half, dst, N, H, W, F, relu, Cp, S, st);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace patdnn
