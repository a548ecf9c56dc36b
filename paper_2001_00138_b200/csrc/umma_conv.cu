// Dense tensor-core reformulation of the pattern-sparse convolution for sm_100a (tcgen05 + TMEM + TMA).
//
// The layer is out = act(bias + sum_{tap} X_tap * W_tap): nine shifted views X_tap of the input times nine F x C
// weight slices W_tap in which the pruned taps and kernels are zero.  As an implicit GEMM per tap this is a plain
// dense contraction (M = pixels, N = filters, K = channels), which the 5th-generation tensor cores run far above the
// FP32 FMA rate -- enough to pay for the zeros when the layer is not too sparse.  The planner uses this path only
// where it beats the CUDA-core kernel.
//
// Precision.  fp32 layers must stay within 1e-4 of the fp64 oracle, which a single bf16/tf32 product cannot give.
// Every fp32 operand is split x = hi + lo with hi = bf16(x), lo = bf16(x - hi) (16 significand bits together) and the
// product is taken as hi*hi + hi*lo + lo*hi, three bf16 MMAs into one fp32 TMEM accumulator; the dropped lo*lo term
// and the split rounding are below 2^-16 relative.  fp16 layers (2e-3) use one fp16 MMA on the stored values.
//
// Data flow.
//   transition_* kernels  : NCHW activations -> [S][N][H][W][Cp] (channels innermost, padded to a multiple of 64 with
//                           zeros; S = 2 planes hi/lo for fp32 layers, 1 for fp16 layers); inside a stack the previous
//                           layer's epilogue writes this tensor instead;
//   encode (host)         : weights -> [S][9][Fp][Cp] in the same split, zeros where pruned;
//   conv_umma_kernel      : one CTA = 128 output pixels (a TW x TH x TN box of the image batch) x BN filters; small grids
//                           split the channel/tap loop over a thread-block cluster;
//   conv_umma_halo_kernel : persistent CTAs, three halo boxes per channel block instead of nine, double-buffered TMEM.
//       warp 0     TMA producer: per (channel block of 64, tap) the shifted pixel box (zero fill outside the image gives
//                  the padding) and the weight tile, 128-byte swizzle, mbarrier rings;
//       warp 1     one thread issues tcgen05.mma (M=128, K=16, 4 k-steps per stage, the split products) into TMEM and
//                  releases the stage with tcgen05.commit;
//       warps 2-9  epilogue: tcgen05.ld the accumulator, bias + ReLU (+ 2x2 maximum), store NCHW or the next layer's
//                  operands.
// Every mbarrier wait is bounded; on expiry the kernel records a status word and leaves through the normal exit
// (TMEM is always deallocated).  Every TMA load is issued by, and lands in, one CTA only.
#include <cuda.h>
#include <type_traits>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstdlib>
#include <cstring>

#include "../../include/patdnn.h"
#include "kernels.hpp"
#include "umma_ptx.cuh"

namespace patdnn {


namespace {

constexpr int kThreads = 320;                // general kernel: TMA warp, MMA warp, eight epilogue warps
constexpr int kHaloThreads = 320;            // persistent kernel: TMA warp, MMA warp, eight epilogue warps
constexpr int kGatherThreads = 256;          // plus eight gather warps for layers whose operand rows are built in the kernel
// ---- transition into a tensor-core layer: finish the producer, change layout, split operands ---------------------
// src is NCHW with Hs x Ws pixels: the caller's input (float or half), or the raw fp32 sums of the previous
// tensor-core layer, in which case that layer's bias + ReLU are applied here and (clear) the sums are zeroed after
// reading so that a K-split GEMM can accumulate into them again.  pool = 1 takes the 2x2/stride-2 maximum on the way
// (max commutes with the per-channel bias and ReLU).  dst is [S][N][H][W][Cp], channels padded with zeros.
// grid = (ceil(W/32), H, N * Cp/64), block = (32, 8).
template <typename T>
__global__ void __launch_bounds__(256) transition_kernel(T *__restrict__ src, uint16_t *__restrict__ dst,
                                                         const float *__restrict__ bias, int relu, int pool, int clear,
                                                         int N, int C, int Hs, int Ws, int Cp, int S) {
    pdl_trigger();
    pdl_wait();
    __shared__ float tile[64][33];
    const int H = pool ? Hs / 2 : Hs, W = pool ? Ws / 2 : Ws;
    const int cblocks = Cp / 64;
    const int n = blockIdx.z / cblocks, c0 = (blockIdx.z - n * cblocks) * 64;
    const int x0 = blockIdx.x * 32, y = blockIdx.y;
    const int tx = threadIdx.x, tyq = threadIdx.y;
    const size_t plane_out = static_cast<size_t>(N) * H * W * Cp;
    {
        for (int cc = tyq; cc < 64; cc += 8) {
            const int c = c0 + cc, x = x0 + tx;
            float v = 0.f;
            if (c < C && x < W) {
                T *sp = src + ((static_cast<size_t>(n) * C + c) * Hs + (pool ? 2 * y : y)) * Ws + (pool ? 2 * x : x);
                if constexpr (sizeof(T) == 2) {
                    v = __half2float(sp[0]);
                    if (pool) v = fmaxf(fmaxf(v, __half2float(sp[1])), fmaxf(__half2float(sp[Ws]), __half2float(sp[Ws + 1])));
                } else {
                    if (pool && (Ws & 1) == 0 && (reinterpret_cast<uintptr_t>(src) & 7) == 0) {   // 8-byte aligned pairs
                        const float2 a = *reinterpret_cast<const float2 *>(sp), b = *reinterpret_cast<const float2 *>(sp + Ws);
                        v = fmaxf(fmaxf(a.x, a.y), fmaxf(b.x, b.y));
                        if (clear) {
                            *reinterpret_cast<float2 *>(sp) = make_float2(0.f, 0.f);
                            *reinterpret_cast<float2 *>(sp + Ws) = make_float2(0.f, 0.f);
                        }
                    } else if (pool) {                       // odd row pitch: the pairs are not 8-byte aligned
                        v = fmaxf(fmaxf(sp[0], sp[1]), fmaxf(sp[Ws], sp[Ws + 1]));
                        if (clear) { sp[0] = 0.f; sp[1] = 0.f; sp[Ws] = 0.f; sp[Ws + 1] = 0.f; }
                    } else {
                        v = sp[0];
                        if (clear) sp[0] = 0.f;
                    }
                }
                if (bias) v += __ldg(bias + c);
                if (relu) v = fmaxf(v, 0.f);
            }
            tile[cc][tx] = v;
        }
        __syncthreads();
        for (int px = tyq; px < 32; px += 8) {           // a warp writes one pixel's 64 channels (2 per lane)
            const int x = x0 + px;
            if (x < W) {
                const float a = tile[2 * tx][px], b = tile[2 * tx + 1][px];
                const size_t o = ((static_cast<size_t>(n) * H + y) * W + x) * Cp + c0 + 2 * tx;
                if (S == 2) {
                    const __nv_bfloat16 ah = __float2bfloat16_rn(a), bh = __float2bfloat16_rn(b);
                    const __nv_bfloat16 al = __float2bfloat16_rn(a - __bfloat162float(ah));
                    const __nv_bfloat16 bl = __float2bfloat16_rn(b - __bfloat162float(bh));
                    *reinterpret_cast<uint32_t *>(dst + o) = static_cast<uint32_t>(__bfloat16_as_ushort(ah)) |
                                                             (static_cast<uint32_t>(__bfloat16_as_ushort(bh)) << 16);
                    *reinterpret_cast<uint32_t *>(dst + plane_out + o) = static_cast<uint32_t>(__bfloat16_as_ushort(al)) |
                                                                         (static_cast<uint32_t>(__bfloat16_as_ushort(bl)) << 16);
                } else {
                    *reinterpret_cast<uint32_t *>(dst + o) = static_cast<uint32_t>(__half_as_ushort(__float2half_rn(a))) |
                                                             (static_cast<uint32_t>(__half_as_ushort(__float2half_rn(b))) << 16);
                }
            }
        }
        __syncthreads();
    }
}

// Same operation for fp32 sources whose rows are 16-byte aligned (Ws % 4 == 0): float4 loads, 16-byte stores.
// A block moves 64 channels x XT output pixels of one row (XT = 64, or 32 when pooling); grid = (ceil(W/XT), H, N*Cp/64).
template <bool POOL>
__global__ void __launch_bounds__(256) transition_vec_kernel(float *__restrict__ src, uint16_t *__restrict__ dst,
                                                             const float *__restrict__ bias, int relu, int clear,
                                                             int N, int C, int Hs, int Ws, int Cp, int S) {
    pdl_trigger();
    pdl_wait();
    constexpr int XT = POOL ? 32 : 64;
    __shared__ float tile[64][XT + 1];
    const int H = POOL ? Hs / 2 : Hs, W = POOL ? Ws / 2 : Ws;
    const int cblocks = Cp / 64;
    const int n = blockIdx.z / cblocks, c0 = (blockIdx.z - n * cblocks) * 64;
    const int x0 = blockIdx.x * XT, y = blockIdx.y;
    const int tid = threadIdx.x;
    const int q = tid & 15, crow = tid >> 4;                    // 16 float4 lanes per channel row, 16 rows per pass
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int cc = crow + 16 * k, c = c0 + cc;
        float v[4] = {0.f, 0.f, 0.f, 0.f};
        const int xs = (POOL ? 2 * x0 : x0) + 4 * q;             // first source column of this lane
        if (c < C && xs < Ws) {
            float *sp = src + ((static_cast<size_t>(n) * C + c) * Hs + (POOL ? 2 * y : y)) * Ws + xs;
            const float4 a = *reinterpret_cast<const float4 *>(sp);
            if (clear) *reinterpret_cast<float4 *>(sp) = make_float4(0.f, 0.f, 0.f, 0.f);
            if (POOL) {
                const float4 b = *reinterpret_cast<const float4 *>(sp + Ws);
                if (clear) *reinterpret_cast<float4 *>(sp + Ws) = make_float4(0.f, 0.f, 0.f, 0.f);
                v[0] = fmaxf(fmaxf(a.x, a.y), fmaxf(b.x, b.y));
                v[1] = fmaxf(fmaxf(a.z, a.w), fmaxf(b.z, b.w));
            } else {
                v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
            }
            const float bb = bias ? __ldg(bias + c) : 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[j] += bb;
                if (relu) v[j] = fmaxf(v[j], 0.f);
            }
        }
        if (POOL) { tile[cc][2 * q] = v[0]; tile[cc][2 * q + 1] = v[1]; }
        else { tile[cc][4 * q] = v[0]; tile[cc][4 * q + 1] = v[1]; tile[cc][4 * q + 2] = v[2]; tile[cc][4 * q + 3] = v[3]; }
    }
    __syncthreads();
    // 4 lanes per pixel, 16 channels (32 bytes) per lane per plane
    const size_t plane_out = static_cast<size_t>(N) * H * W * Cp;
    const int sub = tid & 3;
#pragma unroll
    for (int pass = 0; pass < XT / 64 + (XT < 64 ? 1 : 0); ++pass) {
        const int px = (tid >> 2) + 64 * pass;
        const int x = x0 + px;
        if (px < XT && x < W) {
            uint32_t hi[8], lo[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float a = tile[16 * sub + 2 * j][px], b = tile[16 * sub + 2 * j + 1][px];
                if (S == 2) {
                    const __nv_bfloat16 ah = __float2bfloat16_rn(a), bh = __float2bfloat16_rn(b);
                    const __nv_bfloat16 al = __float2bfloat16_rn(a - __bfloat162float(ah));
                    const __nv_bfloat16 bl = __float2bfloat16_rn(b - __bfloat162float(bh));
                    hi[j] = static_cast<uint32_t>(__bfloat16_as_ushort(ah)) | (static_cast<uint32_t>(__bfloat16_as_ushort(bh)) << 16);
                    lo[j] = static_cast<uint32_t>(__bfloat16_as_ushort(al)) | (static_cast<uint32_t>(__bfloat16_as_ushort(bl)) << 16);
                } else {
                    hi[j] = static_cast<uint32_t>(__half_as_ushort(__float2half_rn(a))) |
                            (static_cast<uint32_t>(__half_as_ushort(__float2half_rn(b))) << 16);
                }
            }
            const size_t o = ((static_cast<size_t>(n) * H + y) * W + x) * Cp + c0 + 16 * sub;
            uint4 *d0 = reinterpret_cast<uint4 *>(dst + o);
            d0[0] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            d0[1] = make_uint4(hi[4], hi[5], hi[6], hi[7]);
            if (S == 2) {
                uint4 *d1 = reinterpret_cast<uint4 *>(dst + plane_out + o);
                d1[0] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                d1[1] = make_uint4(lo[4], lo[5], lo[6], lo[7]);
            }
        }
    }
}

// The same operation without pooling for ANY image size and both source types: a channel's H*W pixels are contiguous in
// NCHW, so the image is treated as a flat [C][H*W] matrix and transposed in 64 x 64 tiles through shared memory --
// loads run along the pixels (a warp reads 32 consecutive elements of one channel), stores along the channels (four
// lanes write the 64 channels of one pixel, 32 bytes each per plane).  grid = (ceil(HW/64), Cp/64, N), block = 256.
template <typename T>
__global__ void __launch_bounds__(256) transition_flat_kernel(const T *__restrict__ src, uint16_t *__restrict__ dst, int N, int C,
                                                              int HW, int Cp, int S) {
    pdl_trigger();
    pdl_wait();
    __shared__ float tile[64][65];                               // [channel][pixel]
    const int p0 = blockIdx.x * 64, c0 = blockIdx.y * 64, n = blockIdx.z;
    const int tid = threadIdx.x;
    {
        const int px = tid & 63, p = p0 + px;
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const int cc = 4 * k + (tid >> 6), c = c0 + cc;
            float v = 0.f;
            if (c < C && p < HW) {
                const T raw = src[(static_cast<size_t>(n) * C + c) * HW + p];
                if constexpr (sizeof(T) == 2) v = __half2float(raw); else v = raw;
            }
            tile[cc][px] = v;
        }
    }
    __syncthreads();
    const int px = tid >> 2, sub = tid & 3, p = p0 + px;
    if (p >= HW) return;
    uint32_t hi[8], lo[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float a = tile[16 * sub + 2 * j][px], b = tile[16 * sub + 2 * j + 1][px];
        if (S == 2) {
            const __nv_bfloat16 ah = __float2bfloat16_rn(a), bh = __float2bfloat16_rn(b);
            const __nv_bfloat16 al = __float2bfloat16_rn(a - __bfloat162float(ah));
            const __nv_bfloat16 bl = __float2bfloat16_rn(b - __bfloat162float(bh));
            hi[j] = static_cast<uint32_t>(__bfloat16_as_ushort(ah)) | (static_cast<uint32_t>(__bfloat16_as_ushort(bh)) << 16);
            lo[j] = static_cast<uint32_t>(__bfloat16_as_ushort(al)) | (static_cast<uint32_t>(__bfloat16_as_ushort(bl)) << 16);
        } else {
            hi[j] = static_cast<uint32_t>(__half_as_ushort(__float2half_rn(a))) |
                    (static_cast<uint32_t>(__half_as_ushort(__float2half_rn(b))) << 16);
        }
    }
    const size_t o = (static_cast<size_t>(n) * HW + p) * Cp + c0 + 16 * sub;
    uint4 *d0 = reinterpret_cast<uint4 *>(dst + o);
    d0[0] = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    d0[1] = make_uint4(hi[4], hi[5], hi[6], hi[7]);
    if (S == 2) {
        uint4 *d1 = reinterpret_cast<uint4 *>(dst + static_cast<size_t>(N) * HW * Cp + o);
        d1[0] = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        d1[1] = make_uint4(lo[4], lo[5], lo[6], lo[7]);
    }
}

// Layers with very few input channels (9*C <= 64, e.g. an RGB first layer): gather the 3x3 neighbourhood into the
// channel dimension, k = 9*c + tap, so that the whole layer is ONE 64-deep GEMM step instead of nine mostly-padding ones.
// dst is [S][N][H][W][64].  A block stages the three input rows of a 32-pixel row segment for all channels in shared
// memory; then 8 threads per pixel each build 8 consecutive k and store 16 bytes per operand plane.
// grid = (ceil(W/32), H, N), block = 256.
template <typename T>
__global__ void __launch_bounds__(256) im2col_kernel(const T *__restrict__ src, uint16_t *__restrict__ dst, int N, int C,
                                                      int H, int W, int S) {
    pdl_trigger();
    pdl_wait();
    __shared__ float rows[7][3][36];                             // [channel][row -1..1][column -1..32 (+pad)]
    const int x0 = blockIdx.x * 32, y = blockIdx.y, n = blockIdx.z;
    for (int i = threadIdx.x; i < C * 3 * 34; i += 256) {
        const int c = i / 102, rem = i - c * 102, r = rem / 34, j = rem - r * 34;
        const int yy = y + r - 1, xx = x0 + j - 1;
        float v = 0.f;
        if (yy >= 0 && yy < H && xx >= 0 && xx < W) {
            const T raw = src[((static_cast<size_t>(n) * C + c) * H + yy) * W + xx];
            if constexpr (sizeof(T) == 2) v = __half2float(raw); else v = raw;
        }
        rows[c][r][j] = v;
    }
    __syncthreads();
    const int px = threadIdx.x >> 3, part = threadIdx.x & 7;
    const int x = x0 + px;
    if (x >= W) return;
    uint32_t hi[4], lo[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        float v[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int k = 8 * part + 2 * e + h;
            const int c = k / 9, t = k - 9 * c;
            v[h] = (c < C) ? rows[c][t / 3][px + t % 3] : 0.f;
        }
        if (S == 2) {
            const __nv_bfloat16 ah = __float2bfloat16_rn(v[0]), bh = __float2bfloat16_rn(v[1]);
            const __nv_bfloat16 al = __float2bfloat16_rn(v[0] - __bfloat162float(ah));
            const __nv_bfloat16 bl = __float2bfloat16_rn(v[1] - __bfloat162float(bh));
            hi[e] = static_cast<uint32_t>(__bfloat16_as_ushort(ah)) | (static_cast<uint32_t>(__bfloat16_as_ushort(bh)) << 16);
            lo[e] = static_cast<uint32_t>(__bfloat16_as_ushort(al)) | (static_cast<uint32_t>(__bfloat16_as_ushort(bl)) << 16);
        } else {
            hi[e] = static_cast<uint32_t>(__half_as_ushort(__float2half_rn(v[0]))) |
                    (static_cast<uint32_t>(__half_as_ushort(__float2half_rn(v[1]))) << 16);
        }
    }
    const size_t pix = (static_cast<size_t>(n) * H + y) * W + x;
    const size_t o = pix * 64 + 8 * part;
    *reinterpret_cast<uint4 *>(dst + o) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
    if (S == 2)
        *reinterpret_cast<uint4 *>(dst + static_cast<size_t>(N) * H * W * 64 + o) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
}

// Finish CNT consecutive filters (f_lo ..) of one output pixel: bias + ReLU, then either the caller's NCHW tensor
// (mode 0) or the next tensor-core layer's split channels-innermost activations (mode 3: [S][N][H][W][out_cp];
// mode 4: the same after a fused 2x2 max-pool, [S][N][H/2][W/2][out_cp]).
template <int CNT, typename T>
__device__ __forceinline__ void emit_chunk(const DenseParams &p, float (&a)[CNT], const float *s_bias, int f_lo, int n, int y,
                                           int x, bool pix_ok) {   // called by whole warps (mode 4 exchanges between lanes)
    // s_bias: this CTA's bias slice in shared memory, indexed from f_lo (zero beyond the layer's last filter)
#pragma unroll
    for (int j = 0; j < CNT; ++j) {
        const int f = f_lo + j;
        float v = a[j] + s_bias[j];
        if (p.relu) v = fmaxf(v, 0.f);
        a[j] = (f < p.F) ? v : 0.f;
    }
    if (p.mode == 4) {
        // Fused 2x2/stride-2 max-pool (bias and ReLU commute with the maximum): the four pixels of a window sit in one
        // warp -- x and x+1 in neighbouring lanes, y and y+1 TW lanes apart (TW is 2, 4, 8 or 16 and boxes start on even
        // coordinates in this mode) -- so two butterfly exchanges leave the window maximum in all four lanes, and the
        // lane of the even/even pixel stores it at the pooled position.
#pragma unroll
        for (int j = 0; j < CNT; ++j) {
            float v = a[j];
            v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
            v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, p.TW));
            a[j] = v;
        }
        pix_ok = pix_ok && !(x & 1) && !(y & 1) && x + 1 < p.W && y + 1 < p.H;
    }
    if (!pix_ok) return;
    if (p.mode == 0) {
        T *out = static_cast<T *>(p.out);
        const size_t plane = static_cast<size_t>(p.H) * p.W;
        const size_t obase = static_cast<size_t>(n) * p.F * plane + static_cast<size_t>(y) * p.W + x;
#pragma unroll
        for (int j = 0; j < CNT; ++j) {
            const int f = f_lo + j;
            if (f < p.F) {
                if constexpr (sizeof(T) == 2) out[obase + f * plane] = __float2half_rn(a[j]);
                else out[obase + f * plane] = a[j];
            }
        }
    } else {
        if (f_lo >= p.out_cp) return;                    // filter tiles may be padded beyond the next layer's channels
        uint16_t *dst = static_cast<uint16_t *>(p.out);
        const int oh = p.mode == 4 ? p.H / 2 : p.H, ow = p.mode == 4 ? p.W / 2 : p.W;
        const int oy = p.mode == 4 ? y >> 1 : y, ox = p.mode == 4 ? x >> 1 : x;
        const size_t o = ((static_cast<size_t>(n) * oh + oy) * ow + ox) * p.out_cp + f_lo;
        const size_t plane_out = static_cast<size_t>(p.N) * oh * ow * p.out_cp;
#pragma unroll
        for (int g = 0; g < CNT / 8; ++g) {
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float u = a[8 * g + 2 * j], w = a[8 * g + 2 * j + 1];
                if constexpr (sizeof(T) == 2) {
                    hi[j] = static_cast<uint32_t>(__half_as_ushort(__float2half_rn(u))) |
                            (static_cast<uint32_t>(__half_as_ushort(__float2half_rn(w))) << 16);
                    lo[j] = 0;
                } else {
                    const __nv_bfloat16 uh = __float2bfloat16_rn(u), wh = __float2bfloat16_rn(w);
                    const __nv_bfloat16 ul = __float2bfloat16_rn(u - __bfloat162float(uh));
                    const __nv_bfloat16 wl = __float2bfloat16_rn(w - __bfloat162float(wh));
                    hi[j] = static_cast<uint32_t>(__bfloat16_as_ushort(uh)) | (static_cast<uint32_t>(__bfloat16_as_ushort(wh)) << 16);
                    lo[j] = static_cast<uint32_t>(__bfloat16_as_ushort(ul)) | (static_cast<uint32_t>(__bfloat16_as_ushort(wl)) << 16);
                }
            }
            *reinterpret_cast<uint4 *>(dst + o + 8 * g) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            if constexpr (sizeof(T) != 2) *reinterpret_cast<uint4 *>(dst + plane_out + o + 8 * g) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
    }
}

// ---- the implicit-GEMM kernel -------------------------------------------------------------------------------------
template <int BN, int TERMS, typename T>
__global__ void __launch_bounds__(kThreads, 1)
conv_umma_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, const DenseParams p) {
    constexpr int S = (TERMS == 3) ? 2 : 1;                     // operand planes (hi, lo)
    constexpr int A_BYTES = kTileM * 128;
    constexpr int B_BYTES = BN * 128;
    constexpr int STAGE_BYTES = S * (A_BYTES + B_BYTES);
    // Narrow filter tiles: the hi and lo weight planes lie back to back in shared memory, so ONE MMA of width 2*BN
    // forms x_hi*w_hi (columns 0..BN) and x_hi*w_lo (columns BN..2BN); the epilogue adds the two column groups.
    constexpr bool MERGE = (TERMS == 3) && (BN <= 128);
    constexpr int ACC_COLS = MERGE ? 2 * BN : BN;
    constexpr int TMEM_COLS = ACC_COLS < 32 ? 32 : ACC_COLS;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) uint64_t bars[2 * 8 + 1];          // full[stages], empty[stages], accumulator ready
    __shared__ uint32_t tmem_slot;
    __shared__ float s_bias[BN];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_trigger();
    const int stages = p.stages;
    const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[8]), bar_acc = smem_u32(&bars[16]);
    const WaitCtx status{p.status, p.spin_limit ? p.spin_limit : kSpinLimit};

    // The ks CTAs of a cluster share one (pixel box, filter tile) and split its K loop -- the (channel block, tap)
    // iterations -- into ks ranges; then the filter tile index is fastest so that CTAs sharing a pixel box run together.
    const int ks = p.ksplit;
    const int rank = blockIdx.x % ks;
    int pt = blockIdx.x / ks + p.tile_base;
    const int ft = pt % p.n_ftiles; pt /= p.n_ftiles;
    const int tix = pt % p.tiles_x; pt /= p.tiles_x;
    const int tiy = pt % p.tiles_y; pt /= p.tiles_y;
    const int tin = pt;
    const int x0 = tix * p.TW, y0 = tiy * p.TH, n0 = tin * p.TN, f0 = ft * BN;
    const int total_iters = p.taps * p.KB;                      // taps = 9, or 1 for gathered (im2col) activations
    const int it0 = rank * total_iters / ks;                    // even split: every range holds at least one iteration
    const int iters = (rank + 1) * total_iters / ks - it0;
    // output pixel of this thread when it acts as an epilogue thread (warps 2..5 and 6..9 each cover the 128 accumulator rows)
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;                           // epilogue warps 2..5 take the lower columns, 6..9 the upper
    constexpr int HC = BN >= 64 ? BN / 2 : BN;                  // columns per half (narrow tiles: half 0 takes them all)
    const int col_lo = (BN >= 64) ? half * HC : 0, col_hi = (BN >= 64) ? col_lo + HC : (half == 0 ? BN : 0);
    const int m = q * 32 + lane;
    const int per_img = p.TW * p.TH;
    const int tn = m / per_img, rem = m - tn * per_img;
    const int ty = rem / p.TW, txx = rem - ty * p.TW;
    const int n = n0 + tn, y = y0 + ty, x = x0 + txx;
    const bool pix_ok = tn < p.TN && n < p.N && y < p.H && x < p.W;

    for (int i = threadIdx.x; i < BN; i += kThreads) s_bias[i] = (f0 + i < p.F) ? p.bias[f0 + i] : 0.f;
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {   // TMEM allocation by one full warp; the same warp frees it at the end
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    // The weights do not depend on the previous kernel: the producer thread fetches the weight tiles of the first ring
    // slots before it waits for that kernel, so they travel (from HBM, when the L2 is cold) while it drains.
    const int npre = iters < stages ? iters : stages;
    if (threadIdx.x == 0) {
        for (int it = 0; it < npre; ++it) {
            const int cb = (it0 + it) / p.taps, tap = (it0 + it) - cb * p.taps;
            const uint32_t base = smem_u32(smem + static_cast<size_t>(it) * STAGE_BYTES);
            mbar_expect_tx(bar_full + 8 * it, S * (p.box_bytes + B_BYTES));
#pragma unroll
            for (int sp = 0; sp < S; ++sp)
                tma_load_4d(base + S * A_BYTES + sp * B_BYTES, &mapB, bar_full + 8 * it, cb * kKBlock, f0, tap, sp);
        }
    }
    pdl_wait();                                                 // set-up done; from here on the previous kernel's data is read
    bool acc_ready = false;                                     // epilogue thread holding a finished K-range partial

    if (warp == 0) {
        if (lane == 0) {
            const uint32_t tx_bytes = S * (p.box_bytes + B_BYTES);
            // ring slot, its use count and the (channel block, tap) of the iteration advance without divisions: this one
            // thread's instruction stream is what a short channel/tap loop waits for
            int s = 0, use = 0, cb = it0 / p.taps, tap = it0 - cb * p.taps;
            const uint32_t smem_base = smem_u32(smem);
            for (int it = 0; it < iters; ++it) {
                if (use > 0 && !mbar_wait(bar_empty + 8 * s, (use - 1) & 1, status, 1)) break;
                if (it + 1 != p.test_skip_load) {                // test hook: that iteration's loads never arrive
                    const int r = p.taps == 9 ? tap / 3 : 1, sx = p.taps == 9 ? tap - 3 * r : 1;
                    const uint32_t base = smem_base + s * STAGE_BYTES;
                    if (it >= npre) mbar_expect_tx(bar_full + 8 * s, tx_bytes);   // the first slots were armed with their weights
#pragma unroll
                    for (int sp = 0; sp < S; ++sp) {
                        tma_load_5d(base + sp * A_BYTES, &mapA, bar_full + 8 * s, cb * kKBlock, x0 + sx - 1, y0 + r - 1, n0, sp);
                        if (it >= npre) tma_load_4d(base + S * A_BYTES + sp * B_BYTES, &mapB, bar_full + 8 * s, cb * kKBlock, f0, tap, sp);
                    }
                }
                if (++s == stages) { s = 0; ++use; }
                if (++tap == p.taps) { tap = 0; ++cb; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(TERMS == 3 ? 1 : 0, BN);
            constexpr uint32_t idesc2 = instr_desc(1, MERGE ? 2 * BN : BN);
            bool ok = true;
            int s = 0, use = 0;
            const uint32_t smem_base = smem_u32(smem);
            for (int it = 0; it < iters && ok; ++it) {
                ok = mbar_wait(bar_full + 8 * s, use & 1, status, 2);
                if (!ok) break;
                tc_fence_after();
                const uint32_t base = smem_base + s * STAGE_BYTES;
                const uint64_t a_hi = smem_desc_sw128(base), a_lo = smem_desc_sw128(base + A_BYTES);
                const uint64_t b_hi = smem_desc_sw128(base + S * A_BYTES), b_lo = smem_desc_sw128(base + S * A_BYTES + B_BYTES);
#pragma unroll
                for (int k = 0; k < 4; ++k) {                   // 4 x K=16 inside the 128-byte swizzle row: +32 bytes
                    const uint64_t koff = static_cast<uint64_t>(2 * k);
                    if constexpr (MERGE) {
                        umma_f16(tmem_base, a_hi + koff, b_hi + koff, idesc2, (it > 0 || k > 0) ? 1u : 0u);
                        umma_f16(tmem_base, a_lo + koff, b_hi + koff, idesc, 1u);
                    } else {
                        umma_f16(tmem_base, a_hi + koff, b_hi + koff, idesc, (it > 0 || k > 0) ? 1u : 0u);
                        if constexpr (TERMS == 3) {
                            umma_f16(tmem_base, a_hi + koff, b_lo + koff, idesc, 1u);
                            umma_f16(tmem_base, a_lo + koff, b_hi + koff, idesc, 1u);
                        }
                    }
                }
                umma_commit(bar_empty + 8 * s);                 // frees the stage once these MMAs have read it
                if (++s == stages) { s = 0; ++use; }
            }
            if (ok) umma_commit(bar_acc);
        }
    } else {
        // epilogue warps: warp w owns TMEM lanes 32*(w%4) .. +31; lane = output pixel m of the box
        if (mbar_wait(bar_acc, 0, status, 3)) {
            tc_fence_after();
            if (ks == 1) {
#pragma unroll 1
                for (int c0 = col_lo; c0 < col_hi; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + c0, v);
                    float a[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) a[j] = __uint_as_float(v[j]);
                    if constexpr (MERGE) {
                        tmem_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + BN + c0, v);
#pragma unroll
                        for (int j = 0; j < 32; ++j) a[j] += __uint_as_float(v[j]);
                    }
                    emit_chunk<32, T>(p, a, s_bias + c0, f0 + c0, n, y, x, pix_ok);
                }
            } else {
                acc_ready = true;                                // partial sums stay in TMEM until the cluster is ready
            }
        }
    }
    if (ks > 1) {
        // Sum the K ranges across the cluster through distributed shared memory.  CTA r finishes the columns
        // [r*BN/ks, (r+1)*BN/ks): every CTA PUSHES the matching slice of its partial tile into r's shared memory
        // (remote stores need no answer, remote loads would expose their latency; a warp's 16-byte stores cover 512
        // contiguous bytes -- the same stores scattered at a row pitch measured twice as slow as 4-byte ones), slot =
        // sender's rank, layout [slot][column quad][pixel][4]; then r adds
        // the ks slots in rank order from its own memory.  Barrier 1: every CTA's MMAs have read their pipeline
        // buffers, which the slots reuse.  Barrier 2: all slots have landed.  Every thread of every CTA takes part in
        // both barriers, also after a timed-out wait, so nobody is left waiting.
        const int cols = BN / ks;
        const uint32_t rbase = smem_u32(smem);
        __syncwarp();                                           // lane 0 of the two role warps rejoins its warp: the
                                                                // cluster barriers below are warp-aligned instructions
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        if (acc_ready) {
#pragma unroll 1
            for (int c0 = col_lo; c0 < col_hi; c0 += 32) {
                uint32_t v[32], v2[32];
                tmem_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + c0, v);
                if constexpr (MERGE) tmem_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + BN + c0, v2);
#pragma unroll
                for (int j0 = 0; j0 < 32; j0 += 8) {             // cols is a multiple of 8: one owner per 8 columns
                    const int owner = (c0 + j0) / cols, cl = (c0 + j0) - owner * cols;
                    uint32_t remote;
                    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(rbase), "r"(owner));
                    // slot layout [sender][column quad][pixel][4 columns]: a warp's 16-byte stores are 512 contiguous bytes
                    remote += (((rank * cols + cl) >> 2) * kTileM + m) * 16;
#pragma unroll
                    for (int h4 = 0; h4 < 2; ++h4) {
                        float w4[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            w4[j] = __uint_as_float(v[j0 + 4 * h4 + j]) + (MERGE ? __uint_as_float(v2[j0 + 4 * h4 + j]) : 0.f);
                        asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(remote + h4 * kTileM * 16), "f"(w4[0]),
                                     "f"(w4[1]), "f"(w4[2]), "f"(w4[3]) : "memory");
                    }
                }
            }
        }
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        if (warp >= 2) {
            const float4 *R4 = reinterpret_cast<const float4 *>(smem);
            const int cbeg = rank * cols;
#pragma unroll 1
            for (int c0 = 8 * half; c0 < cols; c0 += 16) {
                float a[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) a[j] = 0.f;
                for (int qq = 0; qq < ks; ++qq) {
                    const float4 lo4 = R4[((qq * cols + c0) >> 2) * kTileM + m];
                    const float4 hi4 = R4[(((qq * cols + c0) >> 2) + 1) * kTileM + m];
                    a[0] += lo4.x; a[1] += lo4.y; a[2] += lo4.z; a[3] += lo4.w;
                    a[4] += hi4.x; a[5] += hi4.y; a[6] += hi4.z; a[7] += hi4.w;
                }
                emit_chunk<8, T>(p, a, s_bias + cbeg + c0, f0 + cbeg + c0, n, y, x, pix_ok);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- halo-sharing, persistent variant for large batches ------------------------------------------------------------
// The nine taps of a channel block read overlapping pixel windows.  Here a tile is TW x (MT*TH) pixels with TW a
// multiple of 8 and TW*TH = 128, and per channel block only THREE boxes are loaded -- one per horizontal shift s, each
// MT*TH+2 rows tall -- instead of nine: one box row is TW*128 bytes, a whole number of 1024-byte swizzle groups, so
// the operand of vertical tap r is the same buffer entered r rows lower (descriptor start + r*TW*128).
// CTAs are persistent (one per SM, tiles taken round-robin) and the accumulator is double buffered in TMEM: while the
// epilogue warps drain tile i, the MMA thread already works on tile i+1.
// Rings: A (per channel block and shift), B (per channel block and tap), accumulator full/empty (2 buffers).
//
// GATHER (layers with 9*C <= 64, one gathered tap): no activation tensor in memory at all.  Four extra warps read the
// 3x3 neighbourhood of their pixels straight from the caller's NCHW input, split it, and write the [pixel][k] operand
// rows (k = 9*c + tap, zero beyond 9*C) into the A ring in the swizzled layout a TMA load would have produced.
template <int BN, int MT, int TERMS, typename T, bool GATHER>
__global__ void __launch_bounds__(GATHER ? kHaloThreads + kGatherThreads : (MT == 2 ? kHaloThreads + 32 : kHaloThreads), 1)
conv_umma_halo_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, const DenseParams p) {
    constexpr int S = (TERMS == 3) ? 2 : 1;
    constexpr int B_BYTES = BN * 128;
    constexpr bool MERGE = (TERMS == 3) && (BN <= 128);          // see conv_umma_kernel: x_hi * [w_hi | w_lo] in one MMA
    constexpr int ACC_COLS = MERGE ? 2 * BN : BN;
    constexpr int BUF_COLS = MT * ACC_COLS;                      // one accumulator buffer
    // Double tiles of the TMA-fed kernel have one MMA-issuing thread per accumulator (warp 1 and warp 10): narrow MMAs
    // cost their issue, not their arithmetic, and two threads issue twice as many.
    constexpr int ISSUERS = (MT == 2 && !GATHER) ? 2 : 1;
    static_assert(2 * BUF_COLS <= 512, "two accumulator buffers must fit the 512 TMEM columns");
    constexpr int TMEM_COLS = 2 * BUF_COLS < 32 ? 32 : 2 * BUF_COLS;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) uint64_t bars[4 * 8 + 4];          // fullA, emptyA, fullB, emptyB (8 slots each), acc full/empty x2
    __shared__ uint32_t tmem_slot;
    __shared__ float s_bias[2][BN];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NA = p.na, NB = p.stages;
    const int a_plane = p.box_bytes;                            // one box (one operand plane): (MT*TH+2) * TW * 128 bytes
    const int a_stage = S * a_plane;
    const int b_stage = S * B_BYTES;
    unsigned char *smem_b = smem + NA * a_stage;
    const uint32_t bar_fa = smem_u32(&bars[0]), bar_ea = smem_u32(&bars[8]), bar_fb = smem_u32(&bars[16]),
                   bar_eb = smem_u32(&bars[24]), bar_af = smem_u32(&bars[32]), bar_ae = smem_u32(&bars[34]);
    const WaitCtx status{p.status, p.spin_limit ? p.spin_limit : kSpinLimit};
    const int row_bytes = p.TW * 128;
    const int n_tiles = p.tile_limit > 0 ? p.tile_limit : p.n_ftiles * p.tiles_x * p.tiles_y * p.tiles_n;
    const int KB = p.KB;
    const int nshift = p.taps == 9 ? 3 : 1;                     // 3 horizontal shifts x 3 vertical taps, or one gathered tap

    pdl_trigger();
    if (threadIdx.x == 0) {
        for (int s = 0; s < 8; ++s) {
            mbar_init(bar_fa + 8 * s, GATHER ? kGatherThreads / 32 : 1); mbar_init(bar_ea + 8 * s, ISSUERS);
            mbar_init(bar_fb + 8 * s, 1); mbar_init(bar_eb + 8 * s, ISSUERS);
        }
        mbar_init(bar_af, ISSUERS); mbar_init(bar_af + 8, ISSUERS);
        mbar_init(bar_ae, 8); mbar_init(bar_ae + 8, 8);         // one arrival per epilogue warp
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;

    auto decode = [&](int t, int &ft, int &x0, int &y0, int &n) {
        ft = t % p.n_ftiles; t /= p.n_ftiles;
        const int tix = t % p.tiles_x; t /= p.tiles_x;
        const int tiy = t % p.tiles_y; t /= p.tiles_y;
        n = t; x0 = tix * p.TW; y0 = tiy * (MT * p.TH);
    };
    pdl_wait();                                                 // set-up done; from here on the previous kernel's data is read

    if (warp == 0) {
        if (lane == 0) {
            // slots of the two rings and their use counts, advanced without divisions (this thread's instruction stream
            // is what a short channel/tap loop waits for)
            int sa = 0, ua = 0, sb = 0, ub = 0;
            const uint32_t a_ring = smem_u32(smem), b_ring = smem_u32(smem_b);
            bool ok = true;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x) {
                int ft, x0, y0, n;
                decode(t, ft, x0, y0, n);
                const int f0 = ft * BN;
                for (int cb = 0; cb < KB && ok; ++cb) {
                    for (int sx = 0; sx < nshift && ok; ++sx) {
                        if constexpr (!GATHER) {
                            if (ua > 0 && !mbar_wait(bar_ea + 8 * sa, (ua - 1) & 1, status, 1)) { ok = false; break; }
                            const uint32_t abase = a_ring + sa * a_stage;
                            mbar_expect_tx(bar_fa + 8 * sa, S * a_plane);
#pragma unroll
                            for (int sp = 0; sp < S; ++sp)
                                tma_load_5d(abase + sp * a_plane, &mapA, bar_fa + 8 * sa, cb * kKBlock, x0 + sx - (nshift >> 1), y0 - (nshift >> 1), n, sp);
                            if (++sa == NA) { sa = 0; ++ua; }
                        }
                        for (int r = 0; r < nshift; ++r) {
                            if (ub > 0 && !mbar_wait(bar_eb + 8 * sb, (ub - 1) & 1, status, 1)) { ok = false; break; }
                            const uint32_t bbase = b_ring + sb * b_stage;
                            mbar_expect_tx(bar_fb + 8 * sb, S * B_BYTES);
#pragma unroll
                            for (int sp = 0; sp < S; ++sp)
                                tma_load_4d(bbase + sp * B_BYTES, &mapB, bar_fb + 8 * sb, cb * kKBlock, f0, r * nshift + sx, sp);
                            if (++sb == NB) { sb = 0; ++ub; }
                        }
                    }
                }
            }
        }
    } else if (warp == 1 || (ISSUERS == 2 && warp == kHaloThreads / 32)) {
        const int mt_lo = (ISSUERS == 2) ? (warp == 1 ? 0 : 1) : 0, mt_hi = (ISSUERS == 2) ? mt_lo + 1 : MT;
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(TERMS == 3 ? 1 : 0, BN);
            constexpr uint32_t idesc2 = instr_desc(1, MERGE ? 2 * BN : BN);
            int sa = 0, ua = 0, sb = 0, ub = 0, j = 0;
            const uint32_t a_ring = smem_u32(smem), b_ring = smem_u32(smem_b);
            bool ok = true;
            for (int t = blockIdx.x; t < n_tiles && ok; t += gridDim.x, ++j) {
                const int buf = j & 1, ub2 = j >> 1;
                if (ub2 > 0 && !mbar_wait(bar_ae + 8 * buf, (ub2 - 1) & 1, status, 2)) { ok = false; break; }
                tc_fence_after();
                bool first = true;
                for (int cb = 0; cb < KB && ok; ++cb) {
                    for (int sx = 0; sx < nshift && ok; ++sx) {
                        ok = mbar_wait(bar_fa + 8 * sa, ua & 1, status, 2);
                        if (!ok) break;
                        const uint32_t abase = a_ring + sa * a_stage;
                        for (int r = 0; r < nshift && ok; ++r) {
                            ok = mbar_wait(bar_fb + 8 * sb, ub & 1, status, 2);
                            if (!ok) break;
                            tc_fence_after();
                            const uint32_t bbase = b_ring + sb * b_stage;
                            const uint64_t b_hi = smem_desc_sw128(bbase), b_lo = smem_desc_sw128(bbase + B_BYTES);
#pragma unroll
                            for (int mt = 0; mt < MT; ++mt) {
                                if (mt < mt_lo || mt >= mt_hi) continue;                         // the other issuer's tile
                                const uint32_t arow = abase + (mt * p.TH + r) * row_bytes;       // 1024-byte aligned
                                const uint64_t a_hi = smem_desc_sw128(arow), a_lo = smem_desc_sw128(arow + a_plane);
                                const uint32_t acc = tmem_base + buf * BUF_COLS + mt * ACC_COLS;
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    const uint64_t koff = static_cast<uint64_t>(2 * k);
                                    if constexpr (MERGE) {
                                        umma_f16(acc, a_hi + koff, b_hi + koff, idesc2, (first && k == 0) ? 0u : 1u);
                                        umma_f16(acc, a_lo + koff, b_hi + koff, idesc, 1u);
                                    } else {
                                        umma_f16(acc, a_hi + koff, b_hi + koff, idesc, (first && k == 0) ? 0u : 1u);
                                        if constexpr (TERMS == 3) {
                                            umma_f16(acc, a_hi + koff, b_lo + koff, idesc, 1u);
                                            umma_f16(acc, a_lo + koff, b_hi + koff, idesc, 1u);
                                        }
                                    }
                                }
                            }
                            first = false;
                            umma_commit(bar_eb + 8 * sb);
                            if (++sb == NB) { sb = 0; ++ub; }
                        }
                        if (ok) umma_commit(bar_ea + 8 * sa);
                        if (++sa == NA) { sa = 0; ++ua; }
                    }
                }
                if (ok) umma_commit(bar_af + 8 * buf);
            }
        }
    } else if (GATHER && warp >= kHaloThreads / 32) {
        // gather warps: the input patch of a tile (all channels, one-pixel border, zeros outside the image) is staged
        // in shared memory -- double buffered, the next tile's patch is fetched into registers while this tile's rows
        // are built -- and thread g builds the operand rows g, g+256, ... of the tile's A stage (one stage per tile).
        const T *__restrict__ src = static_cast<const T *>(p.gather_src);
        const int g = threadIdx.x - kHaloThreads;
        const int ph = MT * p.TH + 2, pw = p.TW + 2, pplane = ph * pw, pcount = p.C * pplane;
        const int pstride = (pcount + 3) & ~3;
        float *patch0 = reinterpret_cast<float *>(smem_b + NB * b_stage);    // 2 x [C][ph][pw], behind the two rings
        constexpr int PF = 8;                                    // patch elements per thread (planner: pcount <= 8 * 256)
        float pre[PF];
        auto fetch = [&](int t) {
            int ft, x0, y0, n;
            decode(t, ft, x0, y0, n);
#pragma unroll
            for (int u = 0; u < PF; ++u) {
                const int i = g + u * kGatherThreads;
                float v = 0.f;
                if (i < pcount) {
                    const int c = i / pplane, rem = i - c * pplane, py = rem / pw, px = rem - py * pw;
                    const int yy = y0 + py - 1, xx = x0 + px - 1;
                    if (yy >= 0 && yy < p.H && xx >= 0 && xx < p.W)
                        v = static_cast<float>(src[((static_cast<size_t>(n) * p.C + c) * p.H + yy) * p.W + xx]);
                }
                pre[u] = v;
            }
        };
        auto stash = [&](float *dst) {
#pragma unroll
            for (int u = 0; u < PF; ++u) {
                const int i = g + u * kGatherThreads;
                if (i < pcount) dst[i] = pre[u];
            }
        };
        if (static_cast<int>(blockIdx.x) < n_tiles) { fetch(blockIdx.x); stash(patch0); }
        asm volatile("bar.sync 2, %0;" ::"n"(kGatherThreads) : "memory");
        int ia = 0;
        for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++ia) {
            const float *patch = patch0 + (ia & 1) * pstride;
            const bool more = t + static_cast<int>(gridDim.x) < n_tiles;
            if (more) fetch(t + gridDim.x);                      // loads in flight while the rows are built
            const int sa = ia % NA, ua = ia / NA;
            if (ua > 0 && !mbar_wait(bar_ea + 8 * sa, (ua - 1) & 1, status, 4)) break;
            unsigned char *abase = smem + static_cast<size_t>(sa) * a_stage;
            for (int row = g; row < MT * kTileM; row += kGatherThreads) {
                const int ty = row / p.TW, tx = row - ty * p.TW;
                unsigned char *r_hi = abase + row * 128, *r_lo = r_hi + a_plane;
                const int sw = row & 7;                          // 128-byte swizzle: 16-byte chunk index XOR (row mod 8)
                const float *pp = patch + ty * pw + tx;
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    uint32_t hi[4], lo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float v2[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int kk = 8 * ch + 2 * e + u;   // compile-time: the loops are fully unrolled
                            const int c = kk / 9, tap = kk - 9 * c, r = tap / 3, sx = tap - 3 * r;
                            v2[u] = (c < p.C) ? pp[c * pplane + r * pw + sx] : 0.f;
                        }
                        if constexpr (S == 2) {
                            const __nv_bfloat162 h2 = __floats2bfloat162_rn(v2[0], v2[1]);
                            const float2 hf = __bfloat1622float2(h2);
                            const __nv_bfloat162 l2 = __floats2bfloat162_rn(v2[0] - hf.x, v2[1] - hf.y);
                            hi[e] = *reinterpret_cast<const uint32_t *>(&h2);
                            lo[e] = *reinterpret_cast<const uint32_t *>(&l2);
                        } else {
                            const __half2 h2 = __floats2half2_rn(v2[0], v2[1]);
                            hi[e] = *reinterpret_cast<const uint32_t *>(&h2);
                        }
                    }
                    *reinterpret_cast<uint4 *>(r_hi + ((ch ^ sw) << 4)) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    if constexpr (S == 2) *reinterpret_cast<uint4 *>(r_lo + ((ch ^ sw) << 4)) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");    // generic-proxy writes -> visible to the MMA
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_fa + 8 * sa) : "memory");
            if (more) stash(patch0 + ((ia + 1) & 1) * pstride);
            asm volatile("bar.sync 2, %0;" ::"n"(kGatherThreads) : "memory");   // next patch complete, this one free
        }
    } else {
        // eight epilogue warps: warp w reads TMEM lanes 32*(w%4).. and one half of the filter columns
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;
        const int m = q * 32 + lane;
        const int ty = m / p.TW, txx = m - ty * p.TW;
        const int et = threadIdx.x - 64;                         // 0..255 among the epilogue threads
        int j = 0;
        for (int t = blockIdx.x; t < n_tiles; t += gridDim.x, ++j) {
            const int buf = j & 1;
            int ft, x0, y0, n;
            decode(t, ft, x0, y0, n);
            const int f0 = ft * BN;
            for (int i = et; i < BN; i += 256) s_bias[buf][i] = (f0 + i < p.F) ? p.bias[f0 + i] : 0.f;
            asm volatile("bar.sync 1, 256;" ::: "memory");     // the eight epilogue warps only
            if (!mbar_wait(bar_af + 8 * buf, (j >> 1) & 1, status, 3)) break;
            tc_fence_after();
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                const int y = y0 + mt * p.TH + ty, x = x0 + txx;
                const bool pix_ok = y < p.H && x < p.W;
#pragma unroll 1
                for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
                    uint32_t v[32];
                    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * BUF_COLS + mt * ACC_COLS + c0;
                    tmem_ld32(taddr, v);
                    float a[32];
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) a[jj] = __uint_as_float(v[jj]);
                    if constexpr (MERGE) {
                        tmem_ld32(taddr + BN, v);
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) a[jj] += __uint_as_float(v[jj]);
                    }
                    emit_chunk<32, T>(p, a, &s_bias[buf][c0], f0 + c0, n, y, x, pix_ok);
                }
            }
            // this warp is done reading the buffer: hand it back to the MMA thread
            tc_fence_before();
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_ae + 8 * buf) : "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- CTA-pair variant of the persistent kernel for 256-filter tiles ----------------------------------------------------
// Two CTAs of a cluster work on one 256-pixel x 256-filter tile with cta_group::2 MMAs (M = 256): each CTA loads the
// halo boxes of ITS 128 pixels and only HALF of every weight tile (128 of the 256 filters); the tensor cores of both SMs
// read the two halves.  Per SM the weight traffic from L2 -- what the single-CTA kernel waits for on these layers --
// halves.  Protocol (barrier arrays sit at the same shared-memory offsets in both CTAs):
//   full A / full B   live in the leader (cluster rank 0): two arrivals per phase, one arrive.expect_tx from each CTA's
//                     producer thread with that CTA's byte count; both CTAs' TMA loads complete on the leader's barrier
//   empty A / empty B one per CTA, released by the leader's MMA thread with one tcgen05.commit per CTA
//   accumulator full  one per CTA, same; accumulator empty: in the leader, 16 arrivals (8 epilogue warps x 2 CTAs)
// The leader's MMA thread issues for both; every CTA drains its own 128 TMEM lanes.  Each load lands in one CTA only.
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(local_addr), "r"(rank));
    return a;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t cluster_bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.release.cluster.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void tma_load_5d_pair(uint32_t dst, const CUtensorMap *map, uint32_t cluster_bar, int c0, int c1, int c2,
                                                 int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap *map, uint32_t cluster_bar, int c0, int c1, int c2,
                                                 int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(cluster_bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void umma_f16_pair(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8, %9, %10, %11, %12}, p;\n\t}"
        ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u), "r"(0u), "r"(0u),
          "r"(0u), "r"(0u) : "memory");
}
__device__ __forceinline__ void umma_commit_pair(uint32_t cluster_bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(cluster_bar) : "memory");
}
__host__ __device__ constexpr uint32_t instr_desc_m(int fmt, int n, int m) {
    return (1u << 4) | (static_cast<uint32_t>(fmt) << 7) | (static_cast<uint32_t>(fmt) << 10) |
           (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(m >> 4) << 24);
}

template <int TERMS, typename T>
__global__ void __launch_bounds__(kHaloThreads, 1)
conv_umma_pair_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, const DenseParams p) {
    constexpr int BN = 256, BH = 128;                            // filters per tile, filters whose weights this CTA loads
    constexpr int S = (TERMS == 3) ? 2 : 1;
    constexpr int B_BYTES = BH * 128;                            // one weight plane of this CTA's half
    constexpr int TMEM_COLS = 512;                               // two accumulator buffers of 256 columns
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) uint64_t bars[4 * 8 + 4];
    __shared__ uint32_t tmem_slot;
    __shared__ float s_bias[2][BN];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const bool leader = rank == 0;
    const int NA = p.na, NB = p.stages;
    const int a_plane = p.box_bytes;                             // (TH+2) * TW * 128 bytes
    const int a_stage = S * a_plane, b_stage = S * B_BYTES;
    unsigned char *smem_b = smem + NA * a_stage;
    const uint32_t bar_fa = smem_u32(&bars[0]), bar_ea = smem_u32(&bars[8]), bar_fb = smem_u32(&bars[16]),
                   bar_eb = smem_u32(&bars[24]), bar_af = smem_u32(&bars[32]), bar_ae = smem_u32(&bars[34]);
    // the same barriers seen from the cluster: the leader's full/acc-empty barriers, each CTA's empty/acc-full barriers
    const uint32_t L_fa = map_to_cta(bar_fa, 0), L_fb = map_to_cta(bar_fb, 0), L_ae = map_to_cta(bar_ae, 0);
    const WaitCtx status{p.status, p.spin_limit ? p.spin_limit : kSpinLimit};
    const int row_bytes = p.TW * 128;
    const int pix_tiles = p.tiles_x * p.tiles_y * p.tiles_n;
    const int pair_tiles = (pix_tiles + 1) / 2;
    const int n_pairs = p.tile_limit > 0 ? p.tile_limit : p.n_ftiles * pair_tiles;
    const int KB = p.KB;
    const int n_clusters = gridDim.x / 2, cluster_id = blockIdx.x / 2;

    pdl_trigger();
    if (threadIdx.x == 0) {
        for (int s = 0; s < 8; ++s) {
            mbar_init(bar_fa + 8 * s, 2); mbar_init(bar_ea + 8 * s, 1);
            mbar_init(bar_fb + 8 * s, 2); mbar_init(bar_eb + 8 * s, 1);
        }
        mbar_init(bar_af, 1); mbar_init(bar_af + 8, 1);
        mbar_init(bar_ae, 16); mbar_init(bar_ae + 8, 16);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                          // both CTAs' barriers exist before anyone signals them
    tc_fence_after();
    const uint32_t tmem_base = tmem_slot;
    pdl_wait();

    // pair q: filter tile ft (fastest), pixel tiles 2*pp and 2*pp+1; this CTA takes pixel tile 2*pp + rank
    auto decode = [&](int q, int &ft, int &x0, int &y0, int &n) {
        ft = q % p.n_ftiles;
        int t = 2 * (q / p.n_ftiles) + static_cast<int>(rank);
        const int tix = t % p.tiles_x; t /= p.tiles_x;
        const int tiy = t % p.tiles_y; t /= p.tiles_y;
        n = t; x0 = tix * p.TW; y0 = tiy * p.TH;                 // an odd last tile gives n == N: loads read zeros, nothing is stored
    };

    if (warp == 0) {
        if (lane == 0) {
            int ia = 0, ib = 0;
            bool ok = true;
            for (int q = cluster_id; q < n_pairs && ok; q += n_clusters) {
                int ft, x0, y0, n;
                decode(q, ft, x0, y0, n);
                const int f0 = ft * BN + static_cast<int>(rank) * BH;
                for (int cb = 0; cb < KB && ok; ++cb) {
                    for (int sx = 0; sx < 3 && ok; ++sx) {
                        const int sa = ia % NA, ua = ia / NA;
                        if (ua > 0 && !mbar_wait(bar_ea + 8 * sa, (ua - 1) & 1, status, 1)) { ok = false; break; }
                        const uint32_t abase = smem_u32(smem + static_cast<size_t>(sa) * a_stage);
                        mbar_expect_tx_cluster(L_fa + 8 * sa, S * a_plane);
#pragma unroll
                        for (int sp = 0; sp < S; ++sp)
                            tma_load_5d_pair(abase + sp * a_plane, &mapA, L_fa + 8 * sa, cb * kKBlock, x0 + sx - 1, y0 - 1, n, sp);
                        ++ia;
                        for (int r = 0; r < 3; ++r) {
                            const int sb = ib % NB, ub = ib / NB;
                            if (ub > 0 && !mbar_wait(bar_eb + 8 * sb, (ub - 1) & 1, status, 1)) { ok = false; break; }
                            const uint32_t bbase = smem_u32(smem_b + static_cast<size_t>(sb) * b_stage);
                            mbar_expect_tx_cluster(L_fb + 8 * sb, S * B_BYTES);
#pragma unroll
                            for (int sp = 0; sp < S; ++sp)
                                tma_load_4d_pair(bbase + sp * B_BYTES, &mapB, L_fb + 8 * sb, cb * kKBlock, f0, r * 3 + sx, sp);
                            ++ib;
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            constexpr uint32_t idesc = instr_desc_m(TERMS == 3 ? 1 : 0, BN, 256);
            const uint32_t P_ea = map_to_cta(bar_ea, 1), P_eb = map_to_cta(bar_eb, 1), P_af = map_to_cta(bar_af, 1);
            int ia = 0, ib = 0, j = 0;
            bool ok = true;
            for (int q = cluster_id; q < n_pairs && ok; q += n_clusters, ++j) {
                const int buf = j & 1, ub2 = j >> 1;
                if (ub2 > 0 && !mbar_wait(bar_ae + 8 * buf, (ub2 - 1) & 1, status, 2)) { ok = false; break; }
                tc_fence_after();
                bool first = true;
                for (int cb = 0; cb < KB && ok; ++cb) {
                    for (int sx = 0; sx < 3 && ok; ++sx) {
                        const int sa = ia % NA, ua = ia / NA;
                        ok = mbar_wait(bar_fa + 8 * sa, ua & 1, status, 2);
                        if (!ok) break;
                        const uint32_t abase = smem_u32(smem + static_cast<size_t>(sa) * a_stage);
                        for (int r = 0; r < 3 && ok; ++r) {
                            const int sb = ib % NB, ub = ib / NB;
                            ok = mbar_wait(bar_fb + 8 * sb, ub & 1, status, 2);
                            if (!ok) break;
                            tc_fence_after();
                            const uint32_t bbase = smem_u32(smem_b + static_cast<size_t>(sb) * b_stage);
                            const uint64_t b_hi = smem_desc_sw128(bbase), b_lo = smem_desc_sw128(bbase + B_BYTES);
                            const uint32_t arow = abase + r * row_bytes;
                            const uint64_t a_hi = smem_desc_sw128(arow), a_lo = smem_desc_sw128(arow + a_plane);
                            const uint32_t acc = tmem_base + buf * BN;
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const uint64_t koff = static_cast<uint64_t>(2 * k);
                                umma_f16_pair(acc, a_hi + koff, b_hi + koff, idesc, (first && k == 0) ? 0u : 1u);
                                if constexpr (TERMS == 3) {
                                    umma_f16_pair(acc, a_hi + koff, b_lo + koff, idesc, 1u);
                                    umma_f16_pair(acc, a_lo + koff, b_hi + koff, idesc, 1u);
                                }
                            }
                            first = false;
                            umma_commit_pair(bar_eb + 8 * sb);
                            umma_commit_pair(P_eb + 8 * sb);
                            ++ib;
                        }
                        if (ok) { umma_commit_pair(bar_ea + 8 * sa); umma_commit_pair(P_ea + 8 * sa); }
                        ++ia;
                    }
                }
                if (ok) { umma_commit_pair(bar_af + 8 * buf); umma_commit_pair(P_af + 8 * buf); }
            }
        }
    } else {
        const int q4 = warp & 3;
        const int half = (warp - 2) >> 2;
        const int m = q4 * 32 + lane;
        const int ty = m / p.TW, txx = m - ty * p.TW;
        const int et = threadIdx.x - 64;
        int j = 0;
        for (int q = cluster_id; q < n_pairs; q += n_clusters, ++j) {
            const int buf = j & 1;
            int ft, x0, y0, n;
            decode(q, ft, x0, y0, n);
            const int f0 = ft * BN;
            for (int i = et; i < BN; i += 256) s_bias[buf][i] = (f0 + i < p.F) ? p.bias[f0 + i] : 0.f;
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (!mbar_wait(bar_af + 8 * buf, (j >> 1) & 1, status, 3)) break;
            tc_fence_after();
            const int y = y0 + ty, x = x0 + txx;
            const bool pix_ok = n < p.N && y < p.H && x < p.W;
#pragma unroll 1
            for (int c0 = half * (BN / 2); c0 < (half + 1) * (BN / 2); c0 += 32) {
                uint32_t v[32];
                tmem_ld32(tmem_base + (static_cast<uint32_t>(q4 * 32) << 16) + buf * BN + c0, v);
                float a[32];
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) a[jj] = __uint_as_float(v[jj]);
                emit_chunk<32, T>(p, a, &s_bias[buf][c0], f0 + c0, n, y, x, pix_ok);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(L_ae + 8 * buf);
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                          // nobody's shared memory or TMEM goes away under its peer
    if (warp == 2) {
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// The tail launch of a plan: its last tail_tiles tiles on the one-tile-per-CTA kernel, K loop split over clusters.
template <int BN, int TERMS, typename T>
cudaError_t launch_tail(const DensePlan &pl, const DenseParams &p, cudaStream_t st, int first_tile) {
    DenseParams q = p;
    q.tile_base = first_tile; q.tile_limit = 0;
    q.ksplit = pl.tail_ks; q.stages = pl.tail_stages; q.box_bytes = pl.tail_box_bytes;
    q.iters_per_split = (pl.taps * pl.KB + pl.tail_ks - 1) / pl.tail_ks;
    return launch_pdl(conv_umma_kernel<BN, TERMS, T>, dim3(pl.tail_tiles * pl.tail_ks), dim3(kThreads), pl.tail_smem, st,
                      pl.tail_ks, pl.mapA_tail, pl.mapB, q);
}

template <int BN, int TERMS, typename T>
cudaError_t launch_umma(const DensePlan &pl, const DenseParams &p, cudaStream_t st, bool prep) {
    auto kern = conv_umma_kernel<BN, TERMS, T>;
    if (prep) return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
    cudaError_t e = launch_pdl(kern, dim3(pl.grid), dim3(kThreads), pl.smem_bytes, st, pl.ksplit, pl.mapA, pl.mapB, p);
    if (e == cudaSuccess && pl.tail_tiles) e = launch_tail<BN, TERMS, T>(pl, p, st, pl.grid);
    return e;
}

template <int BN, int MT, int TERMS, typename T>
cudaError_t launch_halo(const DensePlan &pl, const DenseParams &p, cudaStream_t st, bool prep) {
    if (pl.gather) {
        auto kern = conv_umma_halo_kernel<BN, MT, TERMS, T, true>;
        if (prep) return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 222 * 1024);
        return launch_pdl(kern, dim3(pl.grid), dim3(kHaloThreads + kGatherThreads), pl.smem_bytes, st, 1, pl.mapA, pl.mapB, p);
    }
    auto kern = conv_umma_halo_kernel<BN, MT, TERMS, T, false>;
    if (prep) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 222 * 1024);
        if (e == cudaSuccess && pl.tail_tiles)
            e = cudaFuncSetAttribute(conv_umma_kernel<BN, TERMS, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
        return e;
    }
    DenseParams q = p;
    q.tile_limit = pl.tail_tiles ? pl.n_tiles - pl.tail_tiles : 0;
    cudaError_t e = launch_pdl(kern, dim3(pl.grid), dim3(MT == 2 ? kHaloThreads + 32 : kHaloThreads), pl.smem_bytes, st, 1, pl.mapA,
                               pl.mapB, q);
    if (e == cudaSuccess && pl.tail_tiles) e = launch_tail<BN, TERMS, T>(pl, p, st, pl.n_tiles - pl.tail_tiles);
    return e;
}

template <int TERMS, typename T>
cudaError_t launch_pair(const DensePlan &pl, const DenseParams &p, cudaStream_t st, bool prep) {
    auto kern = conv_umma_pair_kernel<TERMS, T>;
    if (prep) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 222 * 1024);
        if (e == cudaSuccess && pl.tail_tiles)
            e = cudaFuncSetAttribute(conv_umma_kernel<256, TERMS, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
        return e;
    }
    DenseParams q = p;
    q.tile_limit = pl.tail_tiles ? pl.n_tiles - pl.tail_tiles : 0;      // in pair tiles
    return launch_pdl(kern, dim3(pl.grid), dim3(kHaloThreads), pl.smem_bytes, st, 2, pl.mapA, pl.mapB_pair, q);
}

cudaError_t route(const DensePlan &pl, const DenseParams &p, int dtype, cudaStream_t st, bool prep) {
    if (pl.pair)
        return dtype == PATDNN_F16 ? launch_pair<1, __half>(pl, p, st, prep) : launch_pair<3, float>(pl, p, st, prep);
    if (pl.halo) {
#define PATDNN_HALO(bn, mt)                                                                                        \
    if (pl.BN == bn && pl.MT == mt)                                                                                \
        return dtype == PATDNN_F16 ? launch_halo<bn, mt, 1, __half>(pl, p, st, prep) : launch_halo<bn, mt, 3, float>(pl, p, st, prep);
        PATDNN_HALO(256, 1) PATDNN_HALO(128, 1) PATDNN_HALO(64, 1) PATDNN_HALO(64, 2)
#undef PATDNN_HALO
        return cudaErrorInvalidConfiguration;
    }
#define PATDNN_UMMA(bn)                                                                          \
    if (pl.BN == bn)                                                                             \
        return dtype == PATDNN_F16 ? launch_umma<bn, 1, __half>(pl, p, st, prep) : launch_umma<bn, 3, float>(pl, p, st, prep);
    PATDNN_UMMA(256) PATDNN_UMMA(128) PATDNN_UMMA(64) PATDNN_UMMA(32)
#undef PATDNN_UMMA
    return cudaErrorInvalidConfiguration;
}

// CTAs of the one-tile-per-CTA kernel that are resident at the same time when launched as clusters of `ks`
// (cudaOccupancyMaxActiveClusters; cached; the figures measured on B200 serve where the query is unavailable).
template <int BN, int TERMS, typename T>
int query_cluster_capacity(int ks, int smem) {
    auto kern = conv_umma_kernel<BN, TERMS, T>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024) != cudaSuccess) { cudaGetLastError(); return 0; }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(ks) * 64); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = ks; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    return n * ks;
}

int cluster_capacity(int bn, int dtype, int ks, int smem) {
    static int cache[4][2][4] = {};                                // [BN 32..256][dtype][ks 1, 2, 4, 8], current device of first use
    const int bi = bn == 256 ? 3 : (bn == 128 ? 2 : (bn == 64 ? 1 : 0)), ki = ks == 8 ? 3 : (ks == 4 ? 2 : (ks == 2 ? 1 : 0));
    const int di = dtype == PATDNN_F16 ? 1 : 0;
    if (ks <= 1) return sm_count();
    if (cache[bi][di][ki] == 0) {
        int n = 0;
#define PATDNN_CAP(b)                                                                                              \
    if (bn == b) n = di ? query_cluster_capacity<b, 1, __half>(ks, smem) : query_cluster_capacity<b, 3, float>(ks, smem);
        PATDNN_CAP(256) PATDNN_CAP(128) PATDNN_CAP(64) PATDNN_CAP(32)
#undef PATDNN_CAP
        if (n <= 0) n = ks == 2 ? 148 : (ks == 4 ? 132 : 120);
        cache[bi][di][ki] = n;
    }
    return cache[bi][di][ki];
}

}  // namespace

bool dense_supported(int F, int C, int N, int H, int W) {
    // the layout kernels in front of the GEMM put (image, 64-channel block) on a grid dimension of at most 65535
    const long long cblocks = (C + kKBlock - 1) / kKBlock;
    return encode_fn() != nullptr && F >= 1 && C >= 1 && N >= 1 && H >= 1 && W >= 1 && W <= 4096 && H <= 4096 &&
           N * cblocks <= 65535;
}

// Pixel box (TW x TH x TN <= 128) that wastes the fewest MMA rows for this image size.
void plan_dense(int F, int C, int N, int H, int W, int dtype, DensePlan &pl, bool pool_tiles, int force_bn) {
    pl = DensePlan();
    pl.S = dtype == PATDNN_F16 ? 1 : 2;
    pl.im2col = (9 * C <= kKBlock) ? 1 : 0;                        // tiny C: taps gathered into the channel dimension
    pl.taps = pl.im2col ? 1 : 9;
    pl.Cp = pl.im2col ? kKBlock : (C + kKBlock - 1) / kKBlock * kKBlock;
    pl.KB = pl.Cp / kKBlock;
    pl.BN = F > 128 ? 256 : (F > 64 ? 128 : (F > 32 ? 64 : 32));
    {
        const int want = debug_option("bn", 0);                   // tuning override
        if (want == 32 || want == 64 || want == 128 || want == 256) pl.BN = std::min(pl.BN, want);
    }
    pl.Fp = (F + pl.BN - 1) / pl.BN * pl.BN;
    pl.n_ftiles = pl.Fp / pl.BN;
    double best = -1;
    for (int tw = 1; tw <= std::min(W, kTileM); ++tw) {
        const int th = std::min(H, kTileM / tw);
        int tn = (th == H) ? std::max(1, std::min(N, kTileM / (tw * th))) : 1;
        if (tw > 256 || th > 256 || tn > 256) continue;
        if (pool_tiles) {                                           // see emit_chunk, mode 4
            if (!(tw == 2 || tw == 4 || tw == 8 || tw == 16) || ((th & 1) && th != H)) continue;
            tn = 1;
        }
        const int64_t tx = (W + tw - 1) / tw, ty = (H + th - 1) / th, tz = (N + tn - 1) / tn;
        const double util = static_cast<double>(N) * H * W / (static_cast<double>(tx * ty * tz) * kTileM);
        const double score = util + 1e-6 * tw;                      // prefer wide boxes (coalesced stores) on ties
        if (score > best) { best = score; pl.TW = tw; pl.TH = th; pl.TN = tn; pl.tiles_x = (int)tx; pl.tiles_y = (int)ty; pl.tiles_n = (int)tz; }
    }
    // Few pixel tiles (small batch): cut the K loop into ks ranges, one CTA each, ks CTAs forming a cluster that sums
    // its partial tiles through distributed shared memory (measured: 4 ranges beat 8, whose reduction and cluster
    // scheduling cost more than the shorter loop saves); if that still leaves most SMs idle, narrow the filter tile.
    const int ptiles = pl.tiles_x * pl.tiles_y * pl.tiles_n;
    const int total_iters = pl.taps * pl.KB;
    // a 2-way split of a 128-wide tile exchanges a quarter of what a 4-way split of a 256-wide tile does (measured faster)
    const bool keep_bn = debug_option("bn_keep", 0) != 0;        // tuning override: no narrowing
    const int n_sm0 = sm_count();
    while (!keep_bn && pl.BN > 128 && ptiles * ((F + pl.BN - 1) / pl.BN) * 2 * 37 < n_sm0 * 25) pl.BN /= 2;
    while (!keep_bn && pl.BN > 64 && ptiles * ((F + pl.BN - 1) / pl.BN) * 8 * 37 < n_sm0 * 15) pl.BN /= 2;   // 8-way split still too few CTAs
    if (force_bn) pl.BN = force_bn;
    pl.poolable = (pool_tiles && best > 0) ? 1 : 0;
    pl.Fp = (F + pl.BN - 1) / pl.BN * pl.BN;
    pl.n_ftiles = pl.Fp / pl.BN;
    const int base_grid = ptiles * pl.n_ftiles;
    const int stage = pl.S * (kTileM * 128 + pl.BN * 128);
    pl.stages = std::max(2, std::min(8, (220 * 1024) / stage));
    pl.smem_bytes = pl.stages * stage + 1024;
    const int n_sm = sm_count();
    int ks = 1;
    // one wave only: a second wave costs more than the shorter loop saves.  How many CTAs of this kernel are resident
    // at once as clusters of 2, 4 or 8 comes from the occupancy query (B200, ~200 KB of shared memory per CTA: 148 / 132 / 120)
    if (base_grid * 37 < n_sm * 25)                            // fewer CTAs than about two thirds of the SMs
        while (ks < 8 && base_grid * ks * 2 <= cluster_capacity(pl.BN, dtype, ks * 2, pl.smem_bytes) && ks * 2 <= total_iters &&
               pl.BN / (ks * 2) >= 8)
            ks *= 2;
    {
        const int want = debug_option("ksplit", 0);
        if ((want == 1 || want == 2 || want == 4 || want == 8) && want <= total_iters && pl.BN / want >= 8) ks = want;
    }
    pl.ksplit = ks;
    pl.iters_per_split = (total_iters + ks - 1) / ks;
    pl.box_bytes = pl.TW * pl.TH * pl.TN * 128;
    pl.grid = pl.tiles_x * pl.tiles_y * pl.tiles_n * pl.n_ftiles * pl.ksplit;

    // Large grids: the halo-sharing kernel (three boxes per channel block instead of nine) if a TW x TH = 128 box
    // with TW a multiple of 8 wastes no more pixels than the free-form box does.
    const bool halo_ok = debug_option("halo", 1) != 0;
    if (pl.ksplit == 1 && pl.BN >= 64 && halo_ok) {
        const double util_now = static_cast<double>(N) * H * W / (static_cast<double>(ptiles) * kTileM);
        int btw = 0; double butil = 0;
        for (int tw : {32, 16, 8, 64, 128}) {                      // ties: 32-wide boxes first (128-byte store rows, 1.5x halo)
            if (pool_tiles && tw != 16 && tw != 8) continue;
            const int th = kTileM / tw;
            const double u = static_cast<double>(H) * W /
                             (static_cast<double>((W + tw - 1) / tw) * tw * static_cast<double>((H + th - 1) / th) * th);
            const int mt_try = (pl.BN == 64 && ((H + th - 1) / th) % 2 == 0) ? 2 : 1;
            const int hr = pl.im2col ? 0 : 2;                       // halo rows
            const bool fits = 2 * pl.S * (mt_try * th + hr) * tw * 128 + 2 * pl.S * pl.BN * 128 <= 218 * 1024;
            if (fits && u > butil + 1e-9) { butil = u; btw = tw; }
        }
        // gathered layers: the MMA work is tiny and the kernel-side gather saves a whole tensor, so padding matters less
        const double slack = debug_option("halo_slack", 2) / 100.0;   // MMA rows a halo box may waste beyond the free-form box
        if (btw && butil >= util_now - (pl.im2col ? 0.30 : slack)) {
            const int th = kTileM / btw;
            int mt = (pl.BN == 64 && ((H + th - 1) / th) % 2 == 0) ? 2 : 1;
            if (mt == 2) {
                // a double tile costs ~1/0.65 single tiles (measured); with few rounds the finer granularity can win
                const long long t1 = static_cast<long long>((W + btw - 1) / btw) * ((H + th - 1) / th) * N * pl.n_ftiles;
                const long long r1 = (t1 + n_sm - 1) / n_sm, r2 = (t1 / 2 + n_sm - 1) / n_sm;
                if (0.65 * static_cast<double>(r1) < static_cast<double>(r2)) mt = 1;
            }
            if (const int mv = debug_option("mt", 0)) mt = (mv == 2 && pl.BN == 64) ? 2 : 1;
            const int hr = pl.im2col ? 0 : 2;
            const int a_stage = pl.S * (mt * th + hr) * btw * 128;
            const int b_stage = pl.S * pl.BN * 128;
            int na = 2, nb = 2;
            // gathered layers stage their fp32 input patch (tile plus border, all channels) behind the rings
            const int pcount = C * (mt * th + 2) * (btw + 2);
            const int patch = pl.im2col ? ((2 * ((pcount + 3) & ~3) * 4 + 1023) / 1024) * 1024 : 0;   // double buffered
            const int budget = 218 * 1024 - patch;
            while (nb < 6 && na * a_stage + (nb + 1) * b_stage <= budget) ++nb;
            if (na * a_stage + nb * b_stage <= budget) {
                while (na < 3 && (na + 1) * a_stage + nb * b_stage <= budget) ++na;
                pl.halo = 1; pl.MT = mt; pl.TW = btw; pl.TH = th; pl.TN = 1;
                pl.gather = pl.im2col && pcount <= 8 * 256;      // operand rows built in the kernel, no gathered tensor
                pl.tiles_x = (W + btw - 1) / btw; pl.tiles_y = (H + mt * th - 1) / (mt * th); pl.tiles_n = N;
                pl.box_bytes = (mt * th + hr) * btw * 128;
                pl.na = na; pl.stages = nb;
                pl.smem_bytes = na * a_stage + nb * b_stage + patch + 1024;
                pl.n_tiles = pl.tiles_x * pl.tiles_y * pl.tiles_n * pl.n_ftiles;
                pl.grid = std::min(pl.n_tiles, n_sm);            // persistent CTAs, one per SM
            }
        }
    }
    // 256-filter tiles with enough pixel tiles: CTA pairs (cta_group::2), each CTA loading half of every weight tile.
    // Half-size weight stages also let the 28-pixel-wide halo boxes fit.  Opt-in (PATDNN_DEBUG=pair=1): correct, but measured
    // 8-12 % slower than the single-CTA kernels on the 56x56 and 28x28 layers at batch 32 -- those are not bound by the
    // weight traffic this halves.
    if (pl.BN == 256 && pl.ksplit == 1 && !pl.im2col && !pool_tiles && debug_option("pair", 0) == 1 && halo_ok) {
        const double util_free = static_cast<double>(N) * H * W / (static_cast<double>(ptiles) * kTileM);
        int btw = 0; double butil = 0;
        for (int tw : {32, 16, 8}) {
            const int th = kTileM / tw;
            const double u = static_cast<double>(H) * W /
                             (static_cast<double>((W + tw - 1) / tw) * tw * static_cast<double>((H + th - 1) / th) * th);
            const bool fits = 2 * pl.S * (th + 2) * tw * 128 + 2 * pl.S * 128 * 128 <= 218 * 1024;
            if (fits && u > butil + 1e-9) { butil = u; btw = tw; }
        }
        if (btw && butil >= util_free - 0.02) {
            const int th = kTileM / btw;
            const int tx = (W + btw - 1) / btw, ty = (H + th - 1) / th;
            const int pix_tiles = tx * ty * N;
            const int n_pairs = ((pix_tiles + 1) / 2) * pl.n_ftiles;
            if (n_pairs >= n_sm / 2) {
                const int a_stage = pl.S * (th + 2) * btw * 128, b_stage = pl.S * 128 * 128;
                int na = 2, nb = 2;
                const int budget = 218 * 1024;
                while (nb < 6 && na * a_stage + (nb + 1) * b_stage <= budget) ++nb;
                while (na < 3 && (na + 1) * a_stage + nb * b_stage <= budget) ++na;
                pl.pair = 1; pl.halo = 0; pl.MT = 1; pl.gather = 0;
                pl.TW = btw; pl.TH = th; pl.TN = 1; pl.tiles_x = tx; pl.tiles_y = ty; pl.tiles_n = N;
                pl.box_bytes = (th + 2) * btw * 128;
                pl.na = na; pl.stages = nb;
                pl.smem_bytes = na * a_stage + nb * b_stage + 1024;
                pl.n_tiles = n_pairs;                            // pair tiles
                pl.grid = 2 * std::min(n_pairs, n_sm / 2);
                pl.tail_tiles = 0;
                return;
            }
        }
    }
    // Round quantisation: T equal tiles on n_sm SMs take ceil(T/n_sm) rounds.  When the last round is nearly empty its
    // tiles go to a second launch whose K loop is split over clusters (largest split that still fits one wave).
    const int T = pl.halo ? pl.n_tiles : pl.grid;
    if (debug_option("tail", 1) != 0 && pl.ksplit == 1 && pl.MT == 1 && !pl.gather && T > n_sm && T % n_sm != 0) {
        const int tail = T % n_sm;
        const int tstage = pl.S * (kTileM * 128 + pl.BN * 128);
        const int tstages = std::max(2, std::min(8, (220 * 1024) / tstage));
        const int tsmem = tstages * tstage + 1024;
        int tks = 0;
        for (int cand : {8, 4, 2})
            if (tail * cand <= cluster_capacity(pl.BN, dtype, cand, tsmem) && total_iters / cand >= 2 && pl.BN / cand >= 8) { tks = cand; break; }
        if (tks) {
            pl.tail_tiles = tail; pl.tail_ks = tks;
            pl.tail_stages = tstages;
            pl.tail_smem = tsmem;
            pl.tail_box_bytes = pl.TW * pl.TH * pl.TN * 128;
            if (pl.halo) pl.grid = std::min(T - tail, n_sm);
            else pl.grid = T - tail;
        }
    }
}

// Dense split weights [S][9][Fp][Cp] (16-bit words) from the canonical FKW arrays.
void build_dense_weights(const Fkw &fkw, const DensePlan &pl, std::vector<uint16_t> &w) {
    const size_t plane = static_cast<size_t>(pl.taps) * pl.Fp * pl.Cp;
    w.assign(plane * pl.S, 0);
    for (int i = 0; i < fkw.F; ++i) {
        const int f = fkw.reorder[i];
        for (int32_t k = fkw.offset[i]; k < fkw.offset[i + 1]; ++k) {
            const int c = fkw.index[k];
            const uint32_t mask = fkw.patterns[fkw.kernel_pid[k]];
            int j = 0;
            for (int t = 0; t < 9; ++t) {
                if (!((mask >> t) & 1u)) continue;
                const float v = fkw.weight_f32[static_cast<size_t>(k) * 4 + j++];
                const size_t o = pl.im2col ? static_cast<size_t>(f) * pl.Cp + 9 * c + t
                                           : (static_cast<size_t>(t) * pl.Fp + f) * pl.Cp + c;
                if (pl.S == 2) {
                    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
                    const __nv_bfloat16 lo = __float2bfloat16_rn(v - __bfloat162float(hi));
                    uint16_t hb, lb;
                    std::memcpy(&hb, &hi, 2); std::memcpy(&lb, &lo, 2);
                    w[o] = hb; w[plane + o] = lb;
                } else {
                    w[o] = float_to_half_rne(v);
                }
            }
        }
    }
}

// Tensor maps over the handle-owned split activations and weights.  Returns a PATDNN_* status.
int make_dense_maps(DensePlan &pl, void *d_act, void *d_w, int N, int H, int W, int dtype) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return PATDNN_E_CUDA;
    const CUtensorMapDataType dt = dtype == PATDNN_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    {
        cuuint64_t dims[5] = {(cuuint64_t)pl.Cp, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N, (cuuint64_t)pl.S};
        cuuint64_t strides[4] = {(cuuint64_t)pl.Cp * 2, (cuuint64_t)W * pl.Cp * 2, (cuuint64_t)H * W * pl.Cp * 2,
                                 (cuuint64_t)N * H * W * pl.Cp * 2};
        cuuint32_t box[5] = {(cuuint32_t)kKBlock, (cuuint32_t)pl.TW, (cuuint32_t)(pl.pair ? pl.TH + 2 : (pl.halo ? pl.MT * pl.TH + (pl.im2col ? 0 : 2) : pl.TH)),
                             (cuuint32_t)pl.TN, 1};
        cuuint32_t es[5] = {1, 1, 1, 1, 1};
        if (enc(&pl.mapA, dt, 5, d_act, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PATDNN_E_CUDA;
    }
    if (pl.pair) {
        cuuint64_t dims[4] = {(cuuint64_t)pl.Cp, (cuuint64_t)pl.Fp, (cuuint64_t)pl.taps, (cuuint64_t)pl.S};
        cuuint64_t strides[3] = {(cuuint64_t)pl.Cp * 2, (cuuint64_t)pl.Fp * pl.Cp * 2, (cuuint64_t)pl.taps * pl.Fp * pl.Cp * 2};
        cuuint32_t box[4] = {(cuuint32_t)kKBlock, 128u, 1, 1};
        cuuint32_t es[4] = {1, 1, 1, 1};
        if (enc(&pl.mapB_pair, dt, 4, d_w, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PATDNN_E_CUDA;
    }
    if (pl.tail_tiles) {
        cuuint64_t dims[5] = {(cuuint64_t)pl.Cp, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N, (cuuint64_t)pl.S};
        cuuint64_t strides[4] = {(cuuint64_t)pl.Cp * 2, (cuuint64_t)W * pl.Cp * 2, (cuuint64_t)H * W * pl.Cp * 2,
                                 (cuuint64_t)N * H * W * pl.Cp * 2};
        cuuint32_t box[5] = {(cuuint32_t)kKBlock, (cuuint32_t)pl.TW, (cuuint32_t)pl.TH, (cuuint32_t)pl.TN, 1};
        cuuint32_t es[5] = {1, 1, 1, 1, 1};
        if (enc(&pl.mapA_tail, dt, 5, d_act, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PATDNN_E_CUDA;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)pl.Cp, (cuuint64_t)pl.Fp, (cuuint64_t)pl.taps, (cuuint64_t)pl.S};
        cuuint64_t strides[3] = {(cuuint64_t)pl.Cp * 2, (cuuint64_t)pl.Fp * pl.Cp * 2, (cuuint64_t)pl.taps * pl.Fp * pl.Cp * 2};
        cuuint32_t box[4] = {(cuuint32_t)kKBlock, (cuuint32_t)pl.BN, 1, 1};
        cuuint32_t es[4] = {1, 1, 1, 1};
        if (enc(&pl.mapB, dt, 4, d_w, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PATDNN_E_CUDA;
    }
    return PATDNN_OK;
}

int make_chain_maps(CUtensorMap &mapA, CUtensorMap &mapB, const ChainLayer &L, const DensePlan &pl, void *d_act, void *d_w, int dtype) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return PATDNN_E_CUDA;
    const CUtensorMapDataType dt = dtype == PATDNN_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    {
        cuuint64_t dims[5] = {(cuuint64_t)pl.Cp, (cuuint64_t)L.W, (cuuint64_t)L.H, (cuuint64_t)L.N, (cuuint64_t)pl.S};
        cuuint64_t strides[4] = {(cuuint64_t)pl.Cp * 2, (cuuint64_t)L.W * pl.Cp * 2, (cuuint64_t)L.H * L.W * pl.Cp * 2,
                                 (cuuint64_t)L.N * L.H * L.W * pl.Cp * 2};
        cuuint32_t box[5] = {(cuuint32_t)kKBlock, (cuuint32_t)L.TW, (cuuint32_t)L.TH, (cuuint32_t)L.TN, 1};
        cuuint32_t es[5] = {1, 1, 1, 1, 1};
        if (enc(&mapA, dt, 5, d_act, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PATDNN_E_CUDA;
    }
    {
        // filter tiles of 128 whatever tile width the handle's weight image was padded for: rows past Fp read as zero
        cuuint64_t dims[4] = {(cuuint64_t)pl.Cp, (cuuint64_t)pl.Fp, (cuuint64_t)pl.taps, (cuuint64_t)pl.S};
        cuuint64_t strides[3] = {(cuuint64_t)pl.Cp * 2, (cuuint64_t)pl.Fp * pl.Cp * 2, (cuuint64_t)pl.taps * pl.Fp * pl.Cp * 2};
        cuuint32_t box[4] = {(cuuint32_t)kKBlock, 128u, 1, 1};
        cuuint32_t es[4] = {1, 1, 1, 1};
        if (enc(&mapB, dt, 4, d_w, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PATDNN_E_CUDA;
    }
    return PATDNN_OK;
}

// ---- allocation-free variant: split activations go to a fixed device array ----------------------------------------
// Scratch for callers that must not allocate device memory at run time.  Every context that loads the library holds
// these 16 MiB until it exits.  All calls share the array: two calls that overlap on the GPU race on it.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of g_static_scratch for the current device.  In host code the symbol is only a handle, not an
// address a kernel can use: the address comes from cudaGetSymbolAddress, once per device (the caller serialises).
cudaError_t static_scratch_address(void **ptr) {
    static void *addr[64] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!addr[dev]) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (!p) return cudaErrorInvalidSymbol;
        addr[dev] = p;
    }
    *ptr = addr[dev];
    return cudaSuccess;
}

cudaError_t prepare_dense(const DensePlan &pl, int dtype) {
    DenseParams dummy{};
    return route(pl, dummy, dtype, nullptr, true);
}

cudaError_t launch_transition(const void *src, int src_is_half, void *dst, const float *bias, int relu, int pool, int clear,
                              int N, int C, int Hs, int Ws, int Cp, int S, cudaStream_t st) {
    const int H = pool ? Hs / 2 : Hs, W = pool ? Ws / 2 : Ws;
    if (N == 0 || H == 0 || W == 0) return cudaSuccess;
    const int gz = N * (Cp / 64);
    // no pool, nothing to finish: the flat transpose, unless float4 rows are available (same traffic, fewer instructions)
    if (!pool && !bias && !relu && !clear && N <= 65535 && Cp / 64 <= 65535 &&
        (src_is_half || Ws % 4 != 0 || (reinterpret_cast<uintptr_t>(src) & 15) != 0)) {
        const int HW = Hs * Ws;
        dim3 grid((HW + 63) / 64, Cp / 64, N);
        if (src_is_half)
            return launch_pdl(transition_flat_kernel<__half>, grid, dim3(256), 0, st, 1, static_cast<const __half *>(src),
                              static_cast<uint16_t *>(dst), N, C, HW, Cp, S);
        return launch_pdl(transition_flat_kernel<float>, grid, dim3(256), 0, st, 1, static_cast<const float *>(src),
                          static_cast<uint16_t *>(dst), N, C, HW, Cp, S);
    }
    if (!src_is_half && Ws % 4 == 0 && (reinterpret_cast<uintptr_t>(src) & 15) == 0) {
        float *fs = static_cast<float *>(const_cast<void *>(src));
        uint16_t *d16 = static_cast<uint16_t *>(dst);
        if (pool)
            return launch_pdl(transition_vec_kernel<true>, dim3((W + 31) / 32, H, gz), dim3(256), 0, st, 1, fs, d16, bias, relu, clear,
                              N, C, Hs, Ws, Cp, S);
        return launch_pdl(transition_vec_kernel<false>, dim3((W + 63) / 64, H, gz), dim3(256), 0, st, 1, fs, d16, bias, relu, clear,
                          N, C, Hs, Ws, Cp, S);
    }
    dim3 grid((W + 31) / 32, H, gz), block(32, 8);
    if (src_is_half)
        return launch_pdl(transition_kernel<__half>, grid, block, 0, st, 1, static_cast<__half *>(const_cast<void *>(src)),
                          static_cast<uint16_t *>(dst), bias, relu, pool, 0, N, C, Hs, Ws, Cp, S);
    return launch_pdl(transition_kernel<float>, grid, block, 0, st, 1, static_cast<float *>(const_cast<void *>(src)),
                      static_cast<uint16_t *>(dst), bias, relu, pool, clear, N, C, Hs, Ws, Cp, S);
}

cudaError_t launch_im2col(const void *src, int src_is_half, void *dst, int N, int C, int H, int W, int S, cudaStream_t st) {
    if (N == 0) return cudaSuccess;
    dim3 grid((W + 31) / 32, H, N);
    if (src_is_half)
        return launch_pdl(im2col_kernel<__half>, grid, dim3(256), 0, st, 1, static_cast<const __half *>(src),
                          static_cast<uint16_t *>(dst), N, C, H, W, S);
    return launch_pdl(im2col_kernel<float>, grid, dim3(256), 0, st, 1, static_cast<const float *>(src), static_cast<uint16_t *>(dst),
                      N, C, H, W, S);
}

cudaError_t launch_dense_gemm(const DensePlan &pl, const DenseParams &p, int dtype, cudaStream_t st) {
    return route(pl, p, dtype, st, false);
}

}  // namespace patdnn
