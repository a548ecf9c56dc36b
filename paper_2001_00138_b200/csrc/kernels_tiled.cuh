#pragma once
// Tiled pattern-sparse 3x3 convolution for sm_100a (kernel template; instantiated per blocking in tiled_inst_*.cu).
//
// Mapping of the paper's execution scheme (Sections 5.2 and 5.4) to the GPU:
//   * a thread owns a TY x 4 block of output pixels for FR filters: FR*TY*4 fp32 accumulators in registers;
//   * the 32 lanes of a warp own 32 consecutive thread tiles (row-major over image, tile row, tile column), the
//     FR filters are FR consecutive positions of the filter reorder, so every lane of a warp executes the same
//     kernel with the same pattern: the pattern is warp-uniform and nothing diverges;
//   * a CTA is PW pixel warps x FW filter warps.  It stages, per chunk of CC input channels, the full-width input
//     rows its tiles touch (with zero rows above/below every image and a zero lead/tail column group) into shared
//     memory with asynchronous copies, double buffered ("conventional input tiling", Section 5.4);
//   * per input channel a lane loads its (TY+2) x 6 input patch into registers ONCE: one 16-byte shared load per
//     row, the two halo columns come from the neighbouring lanes by shuffle (from shared memory on the first/last
//     lane and at the image border).  The patch is then reused by all four taps of a kernel (kernel-level load
//     redundancy elimination) and by every kernel of the warp's FR filters that reads this channel (filter-level
//     elimination);
//   * the kernels of a (filter block, channel chunk) arrive as a stream of 32-byte records; a threaded interpreter
//     written in PTX (generated/tiled_cases.inc) reaches, with one warp-uniform indirect branch per record, the
//     straight-line code specialised for (accumulator slot, pattern): 4*TY*4 FFMAs with compile-time register
//     numbers and no control flow inside;
//   * epilogue: bias + ReLU, store to output channel reorder[i] (Section 5.3's reorder array).
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/patdnn.h"
#include "kernels.hpp"
#include "generated/tiled_cases.inc"

namespace patdnn {

namespace {

constexpr int NPAT = kBuiltinPatterns;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

template <int BYTES>
__device__ __forceinline__ void cp_async_zfill(uint32_t dst, const void *src, int src_bytes) {
    if constexpr (BYTES == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
    else if constexpr (BYTES == 8)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

template <typename T> struct Elem;
template <> struct Elem<float> {
    static __device__ __forceinline__ void store4(float *o, const float (&v)[4]) {
        *reinterpret_cast<float4 *>(o) = make_float4(v[0], v[1], v[2], v[3]);
    }
    static __device__ __forceinline__ void store1(float *o, float v) { *o = v; }
};
template <> struct Elem<__half> {
    static __device__ __forceinline__ void store4(__half *o, const float (&v)[4]) {
        const __half2 a = __floats2half2_rn(v[0], v[1]), b = __floats2half2_rn(v[2], v[3]);
        uint2 raw;
        raw.x = *reinterpret_cast<const uint32_t *>(&a);
        raw.y = *reinterpret_cast<const uint32_t *>(&b);
        *reinterpret_cast<uint2 *>(o) = raw;
    }
    static __device__ __forceinline__ void store1(__half *o, float v) { *o = __float2half_rn(v); }
};

template <int TY, int FR, bool HALF> struct Interp;
#define PATDNN_DEF_INTERP(ty, fr)                                                                              \
    template <> struct Interp<ty, fr, false> {                                                                 \
        static __device__ __forceinline__ void run(float (&acc)[fr][ty][4], uint32_t ep, uint32_t pbase,       \
                                                   uint32_t pitch_b, uint32_t pl, uint32_t pr) {               \
            PATDNN_INTERP_##ty##_##fr##_F32(acc, ep, pbase, pitch_b, pl, pr);                                  \
        }                                                                                                      \
    };                                                                                                         \
    template <> struct Interp<ty, fr, true> {                                                                  \
        static __device__ __forceinline__ void run(float (&acc)[fr][ty][4], uint32_t ep, uint32_t pbase,       \
                                                   uint32_t pitch_b, uint32_t pl, uint32_t pr) {               \
            PATDNN_INTERP_##ty##_##fr##_F16(acc, ep, pbase, pitch_b, pl, pr);                                  \
        }                                                                                                      \
    };
PATDNN_DEF_INTERP(4, 8)
PATDNN_DEF_INTERP(4, 4)
PATDNN_DEF_INTERP(2, 8)
#undef PATDNN_DEF_INTERP

constexpr int kRecordBytes = 32;   // {w0, w1, w2, w3, descriptor, pad, pad, pad}

template <int TY, int FR, int PW, int FW, int MINB, typename T>
__global__ void __launch_bounds__(PW *FW * 32, MINB) conv_tiled_kernel(const TiledParams p) {
    constexpr int NS = 2;
    constexpr int NT = PW * FW * 32;
    constexpr int ES = sizeof(T);
    extern __shared__ __align__(16) unsigned char smem[];
    pdl_trigger();
    pdl_wait();                                  // the input may be the previous kernel's output

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int fw = warp % FW, pw = warp / FW;
    const int grid_fg = (p.nblk + FW - 1) / FW;
    const int fg = blockIdx.x % grid_fg, pixcta = blockIdx.x / grid_fg;
    const int blk = fg * FW + fw;                        // this warp's filter block
    const bool blk_ok = blk < p.nblk;

    // ---- geometry of this CTA's tile range --------------------------------------------------------------
    const int tpi = p.TYn * p.TXn;
    const int t_first = pixcta * (PW * 32);
    const int vr_lo = (t_first / tpi) * (p.H + 2) + ((t_first % tpi) / p.TXn) * TY;
    const int t = t_first + pw * 32 + lane;
    const bool tile_ok = t < p.tiles_total;
    const int tc = tile_ok ? t : p.tiles_total - 1;
    const int n = tc / tpi;
    const int trem = tc - n * tpi;
    const int ty = trem / p.TXn, lx = trem - ty * p.TXn;
    const int r0 = n * (p.H + 2) + ty * TY - vr_lo;
    const uint32_t pL = (lx == 0) || (lane == 0);
    const uint32_t pR = (lx == p.TXn - 1) || (lane == 31);

    const int pitch_b = p.pitch * ES;
    const int ch_stride_b = p.rows_max * pitch_b;
    const int in_stage_b = p.CC * ch_stride_b + 16;
    const int seg_stage_b = FW * p.seg_cap * kRecordBytes + kRecordBytes;
    const int stage_b = in_stage_b + seg_stage_b;
    const int lane_off_b = r0 * pitch_b + (p.lead + 4 * lx) * ES;
    const int gpr = pitch_b / p.copy_bytes;               // copy groups per row
    const int nitems = p.rows_max * gpr;
    int2 *s_items = reinterpret_cast<int2 *>(smem + NS * stage_b);

    // Copy plan of one channel, built once: for every copy group of every staged row, the source element offset
    // inside a channel plane (counted from the first image this CTA stages, so that it fits 32 bits whatever the
    // batch; -1 = zero fill) and the destination byte offset.
    const int n_base = vr_lo / (p.H + 2);
    {
        const int epg = p.copy_bytes / ES;
        for (int i = tid; i < nitems; i += NT) {
            const int row = i / gpr, g = i - row * gpr;
            const int vr = vr_lo + row;
            const int nn = vr / (p.H + 2), yy = vr - nn * (p.H + 2) - 1;
            const int col = g * epg - p.lead;
            const bool ok = nn < p.N && yy >= 0 && yy < p.H && col >= 0 && col < p.W;
            s_items[i] = make_int2(ok ? ((nn - n_base) * p.C * p.H + yy) * p.W + col : -1, row * pitch_b + g * p.copy_bytes);
        }
    }
    if (tid < NS * 4)   // the zero group behind each stage's input rows (read as "column W" of the very last row)
        *reinterpret_cast<uint32_t *>(smem + (tid >> 2) * stage_b + in_stage_b - 16 + (tid & 3) * 4) = 0u;
    __syncthreads();

    const T *gin = static_cast<const T *>(p.in);
    const int plane = p.H * p.W;
    const unsigned char *grec = reinterpret_cast<const unsigned char *>(p.rec);

    auto stage_chunk = [&](int q, int s) {
        const uint32_t sin = smem_u32(smem + s * stage_b);
        const int c0 = q * p.CC;
        const int ccn = min(p.CC, p.C - c0);
        const T *gchunk = gin + (static_cast<size_t>(n_base) * p.C + c0) * plane;
        for (int i = tid; i < nitems; i += NT) {
            const int2 it = s_items[i];
            const bool ok = it.x >= 0;
            const T *sp = ok ? gchunk + it.x : gin;
            const int step = ok ? plane : 0;
            uint32_t d = sin + it.y;
            for (int cc = 0; cc < ccn; ++cc) {
                if (p.copy_bytes == 16) cp_async_zfill<16>(d, sp, ok ? 16 : 0);
                else if (p.copy_bytes == 8) cp_async_zfill<8>(d, sp, ok ? 8 : 0);
                else cp_async_zfill<4>(d, sp, ok ? 4 : 0);
                d += ch_stride_b;
                sp += step;
            }
        }
        // "column W" of the last staged channel's last row is the lead group of the following channel slot: keep it
        // zero when the chunk is short (for a full chunk it is the zero group behind the stage, written once)
        if (ccn < p.CC && tid == 0) cp_async_zfill<16>(sin + ccn * ch_stride_b, gin, 0);
        // entry segments of this CTA's filter blocks for the chunk (each warp copies a share of its block's)
        if (blk_ok) {
            const int sidx = blk * p.nchunk + q;
            const int start = p.seg[sidx], len2 = p.seglen[sidx] * 2;     // 16-byte copies
            const uint32_t sd = sin + in_stage_b + fw * p.seg_cap * kRecordBytes;
            const unsigned char *src = grec + static_cast<size_t>(start) * kRecordBytes;
            for (int e = pw * 32 + lane; e < len2; e += PW * 32) cp_async_zfill<16>(sd + e * 16, src + e * 16, 16);
        }
    };

    float acc[FR][TY][4];
#pragma unroll
    for (int j = 0; j < FR; ++j)
#pragma unroll
        for (int y = 0; y < TY; ++y)
#pragma unroll
            for (int x = 0; x < 4; ++x) acc[j][y][x] = 0.f;

    // ---- pipeline over channel chunks ---------------------------------------------------------------------
    stage_chunk(0, 0);
    cp_async_commit();
    for (int q = 0; q < p.nchunk; ++q) {
        cp_async_wait<0>();
        __syncthreads();
        if (q + 1 < p.nchunk) stage_chunk(q + 1, (q + 1) & 1);
        cp_async_commit();
        if (blk_ok) {
            const uint32_t sbase = smem_u32(smem + (q & 1) * stage_b);
            Interp<TY, FR, (ES == 2)>::run(acc, sbase + in_stage_b + fw * p.seg_cap * kRecordBytes,
                                          sbase + lane_off_b, pitch_b, pL, pR);
        }
    }
    cp_async_wait<0>();

    // ---- epilogue: bias + ReLU, scatter to the original output channel -----------------------------------------
    if (!blk_ok || !tile_ok) return;
    T *gout = static_cast<T *>(p.out);
    const int x0 = 4 * lx;
    const bool vec_ok = (p.W % 4 == 0);
#pragma unroll
    for (int j = 0; j < FR; ++j) {
        const int i = blk * FR + j;
        if (i >= p.F) break;
        const int f = __ldg(p.reorder + i);
        const float b = __ldg(p.bias + f);
#pragma unroll
        for (int y = 0; y < TY; ++y) {
            const int yy = ty * TY + y;
            if (yy >= p.H) break;
            float v[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                v[x] = acc[j][y][x] + b;
                if (p.relu) v[x] = fmaxf(v[x], 0.f);
            }
            T *o = gout + ((static_cast<size_t>(n) * p.F + f) * p.H + yy) * p.W + x0;
            if (vec_ok) {
                Elem<T>::store4(o, v);
            } else {
#pragma unroll
                for (int x = 0; x < 4; ++x)
                    if (x0 + x < p.W) Elem<T>::store1(o + x, v[x]);
            }
        }
    }
}

template <int TY, int FR, int PW, int FW, int MINB, typename T>
cudaError_t launch_instance(const TiledPlan &plan, const TiledParams &p, cudaStream_t stream, bool prepare_only) {
    auto kern = conv_tiled_kernel<TY, FR, PW, FW, MINB, T>;
    if (prepare_only)   // per kernel instance, not per layer: the largest opt-in size
        return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
    const int grid = plan.grid_pix * plan.grid_fg;
    return launch_pdl(kern, dim3(grid), dim3(PW * FW * 32), plan.smem_bytes, stream, 1, p);
}


}  // namespace

}  // namespace patdnn
