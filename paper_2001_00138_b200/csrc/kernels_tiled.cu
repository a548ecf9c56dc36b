// Tiled pattern-sparse 3x3 convolution for sm_100a.
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
//   * the kernels of a (filter block, channel chunk) arrive as a descriptor stream; each descriptor selects, by one
//     warp-uniform indirect branch, the straight-line code specialised for (accumulator slot, pattern): 4*TY*4
//     FFMAs with compile-time register indices and no control flow inside;
//   * epilogue: bias + ReLU, store to output channel reorder[i] (Section 5.3's reorder array).
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/patdnn.h"
#include "kernels.hpp"

namespace patdnn {

namespace {

constexpr int NPAT = kBuiltinPatterns;
constexpr int kMaxRows = 320;

__host__ __device__ constexpr uint32_t builtin_mask(int p) {
    constexpr uint32_t m[NPAT] = {0x01B, 0x036, 0x0D8, 0x1B0, 0x03A, 0x0B8, 0x09A, 0x0B2, 0x017, 0x1D0, 0x059, 0x134};
    return m[p];
}
__host__ __device__ constexpr int nth_tap(uint32_t mask, int n) {
    int seen = 0;
    for (int t = 0; t < 9; ++t)
        if ((mask >> t) & 1u) {
            if (seen == n) return t;
            ++seen;
        }
    return 0;
}

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

// One kernel (accumulator slot J, builtin pattern PID): 4 taps x TY x 4 pixels of FFMA on registers only.
template <int TY, int FR, int J, int PID>
__device__ __forceinline__ void fma_kernel(float (&acc)[FR][TY][4], const float (&patch)[TY + 2][6], const float4 &w) {
    constexpr uint32_t m = builtin_mask(PID);
    constexpr int t0 = nth_tap(m, 0), t1 = nth_tap(m, 1), t2 = nth_tap(m, 2), t3 = nth_tap(m, 3);
#pragma unroll
    for (int y = 0; y < TY; ++y)
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            float a = acc[J][y][x];
            a = fmaf(w.x, patch[y + t0 / 3][x + t0 % 3], a);
            a = fmaf(w.y, patch[y + t1 / 3][x + t1 % 3], a);
            a = fmaf(w.z, patch[y + t2 / 3][x + t2 % 3], a);
            a = fmaf(w.w, patch[y + t3 / 3][x + t3 % 3], a);
            acc[J][y][x] = a;
        }
}

template <typename T> struct Elem;
template <> struct Elem<float> {
    static __device__ __forceinline__ void load_row(const unsigned char *a, float (&row)[6], bool pL, bool pR) {
        const float4 v = *reinterpret_cast<const float4 *>(a);
        row[1] = v.x; row[2] = v.y; row[3] = v.z; row[4] = v.w;
        float l = __shfl_up_sync(0xffffffffu, v.w, 1);
        float r = __shfl_down_sync(0xffffffffu, v.x, 1);
        if (pL) l = *reinterpret_cast<const float *>(a - 4);
        if (pR) r = *reinterpret_cast<const float *>(a + 16);
        row[0] = l; row[5] = r;
    }
    static __device__ __forceinline__ void store4(float *o, const float (&v)[4]) {
        *reinterpret_cast<float4 *>(o) = make_float4(v[0], v[1], v[2], v[3]);
    }
    static __device__ __forceinline__ void store1(float *o, float v) { *o = v; }
};
template <> struct Elem<__half> {
    static __device__ __forceinline__ void load_row(const unsigned char *a, float (&row)[6], bool pL, bool pR) {
        const uint2 raw = *reinterpret_cast<const uint2 *>(a);
        const float2 lo = __half22float2(*reinterpret_cast<const __half2 *>(&raw.x));
        const float2 hi = __half22float2(*reinterpret_cast<const __half2 *>(&raw.y));
        row[1] = lo.x; row[2] = lo.y; row[3] = hi.x; row[4] = hi.y;
        float l = __shfl_up_sync(0xffffffffu, hi.y, 1);
        float r = __shfl_down_sync(0xffffffffu, lo.x, 1);
        if (pL) l = __half2float(*reinterpret_cast<const __half *>(a - 2));
        if (pR) r = __half2float(*reinterpret_cast<const __half *>(a + 8));
        row[0] = l; row[5] = r;
    }
    static __device__ __forceinline__ void store4(__half *o, const float (&v)[4]) {
        const __half2 a = __floats2half2_rn(v[0], v[1]), b = __floats2half2_rn(v[2], v[3]);
        uint2 raw;
        raw.x = *reinterpret_cast<const uint32_t *>(&a);
        raw.y = *reinterpret_cast<const uint32_t *>(&b);
        *reinterpret_cast<uint2 *>(o) = raw;
    }
    static __device__ __forceinline__ void store1(__half *o, float v) { *o = __float2half_rn(v); }
};

#define PATDNN_CASE(J, P)                                                                   \
    case ((J) < FR ? (J) * NPAT + (P) : 4096 + (J) * NPAT + (P)):                            \
        if constexpr ((J) < FR) fma_kernel<TY, FR, ((J) < FR ? (J) : 0), (P)>(acc, patch, w); \
        break;
#define PATDNN_CASES_J(J)                                                                        \
    PATDNN_CASE(J, 0) PATDNN_CASE(J, 1) PATDNN_CASE(J, 2) PATDNN_CASE(J, 3) PATDNN_CASE(J, 4)    \
    PATDNN_CASE(J, 5) PATDNN_CASE(J, 6) PATDNN_CASE(J, 7) PATDNN_CASE(J, 8) PATDNN_CASE(J, 9)    \
    PATDNN_CASE(J, 10) PATDNN_CASE(J, 11)
#define PATDNN_CASES_ALL                                                                              \
    PATDNN_CASES_J(0) PATDNN_CASES_J(1) PATDNN_CASES_J(2) PATDNN_CASES_J(3) PATDNN_CASES_J(4)         \
    PATDNN_CASES_J(5) PATDNN_CASES_J(6) PATDNN_CASES_J(7) PATDNN_CASES_J(8) PATDNN_CASES_J(9)         \
    PATDNN_CASES_J(10) PATDNN_CASES_J(11) PATDNN_CASES_J(12) PATDNN_CASES_J(13) PATDNN_CASES_J(14)    \
    PATDNN_CASES_J(15)

template <int TY, int FR, int PW, int FW, int NS, typename T>
__global__ void __launch_bounds__(PW *FW * 32, 1) conv_tiled_kernel(const TiledParams p) {
    static_assert(FR <= 16, "case table covers 16 accumulator slots");
    constexpr int NT = PW * FW * 32;
    constexpr int NWARP = PW * FW;
    constexpr int ES = sizeof(T);
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ int32_t s_rowsrc[kMaxRows];

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
    const bool pL = (lx == 0) || (lane == 0);
    const bool pR = (lx == p.TXn - 1) || (lane == 31);

    const int pitch_b = p.pitch * ES;
    const int ch_stride_b = p.rows_max * pitch_b;
    const int in_stage_b = p.CC * ch_stride_b + 16;
    const int stage_b = in_stage_b + FW * p.seg_cap * 20;
    const int lane_off_b = r0 * pitch_b + (p.lead + 4 * lx) * ES;

    // row table: element offset of each staged row inside a channel plane (plus the image offset), -1 = zero row
    for (int r = tid; r < p.rows_max; r += NT) {
        const int vr = vr_lo + r;
        const int nn = vr / (p.H + 2), yy = vr - nn * (p.H + 2) - 1;
        s_rowsrc[r] = (nn < p.N && yy >= 0 && yy < p.H) ? (nn * p.C * p.H + yy) * p.W : -1;
    }
    if (tid < NS * 4)   // the zero group behind each stage's input rows (read as "column W" of the very last row)
        *reinterpret_cast<uint32_t *>(smem + (tid >> 2) * stage_b + in_stage_b - 16 + (tid & 3) * 4) = 0u;
    __syncthreads();

    const T *gin = static_cast<const T *>(p.in);
    const int plane = p.H * p.W;

    auto stage_chunk = [&](int q, int s) {
        unsigned char *sbase = smem + s * stage_b;
        const uint32_t sin = smem_u32(sbase);
        const int c0 = q * p.CC;
        const int ccn = min(p.CC, p.C - c0);
        const int gpr = pitch_b / p.copy_bytes;           // copy groups per row
        const int epg = p.copy_bytes / ES;                // elements per group
        for (int cc = 0; cc < ccn; ++cc) {
            const T *gplane = gin + static_cast<size_t>(c0 + cc) * plane;
            for (int row = warp; row < p.rows_max; row += NWARP) {
                const int src = s_rowsrc[row];
                const uint32_t drow = sin + cc * ch_stride_b + row * pitch_b;
                for (int g = lane; g < gpr; g += 32) {
                    const int col = g * epg - p.lead;
                    const bool ok = src >= 0 && col >= 0 && col < p.W;
                    const T *sp = ok ? gplane + src + col : gin;
                    const uint32_t d = drow + g * p.copy_bytes;
                    if (p.copy_bytes == 16) cp_async_zfill<16>(d, sp, ok ? 16 : 0);
                    else if (p.copy_bytes == 8) cp_async_zfill<8>(d, sp, ok ? 8 : 0);
                    else cp_async_zfill<4>(d, sp, ok ? 4 : 0);
                }
            }
        }
        if (pw == 0 && blk_ok) {                          // this filter block's entry segment for the chunk
            const int sidx = blk * p.nchunk + q;
            const int start = p.seg[sidx], len = p.seglen[sidx];
            const uint32_t sd = sin + in_stage_b + fw * p.seg_cap * 4;
            const uint32_t sw = sin + in_stage_b + FW * p.seg_cap * 4 + fw * p.seg_cap * 16;
            for (int e = lane; e < len; e += 32) cp_async_zfill<16>(sw + e * 16, p.wts + start + e, 16);
            for (int e = lane; e < (len >> 2); e += 32) cp_async_zfill<16>(sd + e * 16, p.desc + start + e * 4, 16);
        }
    };

    float acc[FR][TY][4];
#pragma unroll
    for (int j = 0; j < FR; ++j)
#pragma unroll
        for (int y = 0; y < TY; ++y)
#pragma unroll
            for (int x = 0; x < 4; ++x) acc[j][y][x] = 0.f;
    float patch[TY + 2][6];
#pragma unroll
    for (int r = 0; r < TY + 2; ++r)
#pragma unroll
        for (int x = 0; x < 6; ++x) patch[r][x] = 0.f;

    // ---- pipeline over channel chunks ---------------------------------------------------------------------
#pragma unroll
    for (int s = 0; s < NS - 1; ++s) {
        if (s < p.nchunk) stage_chunk(s, s);
        cp_async_commit();
    }
    for (int q = 0; q < p.nchunk; ++q) {
        cp_async_wait<NS - 2>();
        __syncthreads();
        if (q + NS - 1 < p.nchunk) stage_chunk(q + NS - 1, (q + NS - 1) % NS);
        cp_async_commit();

        if (blk_ok) {
            const unsigned char *sbase = smem + (q % NS) * stage_b;
            const uint32_t *dp = reinterpret_cast<const uint32_t *>(sbase + in_stage_b) + fw * p.seg_cap;
            const float4 *wp = reinterpret_cast<const float4 *>(sbase + in_stage_b + FW * p.seg_cap * 4) + fw * p.seg_cap;
            const unsigned char *pbase = sbase + lane_off_b;
            bool more = true;
#pragma unroll 1
            while (more) {
                const uint32_t d = *dp++;
                const float4 w = *wp++;
                switch (d & 1023u) {
                    PATDNN_CASES_ALL
                    case FR * NPAT: {
                        const unsigned char *a = pbase + (d >> 10);
#pragma unroll
                        for (int r = 0; r < TY + 2; ++r) Elem<T>::load_row(a + r * pitch_b, patch[r], pL, pR);
                        break;
                    }
                    default:
                        more = false;
                        break;
                }
            }
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

template <int TY, int FR, int PW, int FW, int NS, typename T>
cudaError_t launch_instance(const TiledPlan &plan, const TiledParams &p, cudaStream_t stream, bool prepare_only) {
    auto kern = conv_tiled_kernel<TY, FR, PW, FW, NS, T>;
    if (prepare_only)
        return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);  // per instance, not per layer
    const int grid = plan.grid_pix * plan.grid_fg;
    kern<<<grid, PW * FW * 32, plan.smem_bytes, stream>>>(p);
    return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch(const TiledPlan &plan, const TiledParams &p, cudaStream_t stream, bool prep) {
    const TiledConfig &c = plan.cfg;
#define PATDNN_INST(ty, fr, pw, fw, ns)                                                  \
    if (c.TY == ty && c.FR == fr && c.PW == pw && c.FW == fw && c.NS == ns)              \
        return launch_instance<ty, fr, pw, fw, ns, T>(plan, p, stream, prep);
    PATDNN_INST(2, 16, 2, 4, 2)
    PATDNN_INST(2, 16, 2, 2, 2)
    PATDNN_INST(2, 16, 2, 1, 2)
    PATDNN_INST(2, 16, 1, 4, 2)
    PATDNN_INST(2, 16, 1, 2, 2)
    PATDNN_INST(2, 16, 1, 1, 2)
    PATDNN_INST(4, 8, 2, 4, 2)
    PATDNN_INST(4, 8, 2, 2, 2)
    PATDNN_INST(4, 8, 2, 1, 2)
    PATDNN_INST(4, 8, 1, 4, 2)
    PATDNN_INST(4, 8, 1, 2, 2)
    PATDNN_INST(4, 8, 1, 1, 2)
#undef PATDNN_INST
    return cudaErrorInvalidConfiguration;
}

}  // namespace

cudaError_t launch_tiled(const TiledPlan &plan, const TiledParams &p, int dtype, cudaStream_t stream) {
    if (plan.tiles_total == 0) return cudaSuccess;
    return dtype == PATDNN_F16 ? dispatch<__half>(plan, p, stream, false) : dispatch<float>(plan, p, stream, false);
}

cudaError_t prepare_tiled(const TiledPlan &plan, int dtype) {
    TiledParams dummy{};
    return dtype == PATDNN_F16 ? dispatch<__half>(plan, dummy, nullptr, true) : dispatch<float>(plan, dummy, nullptr, true);
}

}  // namespace patdnn
