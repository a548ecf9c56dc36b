// Pattern-run kernel: the paper's scheme on the FP32 pipes with one FILTER per lane (Sections 5.2 to 5.4).
//
// A thread owns one filter (a position of the filter-kernel reorder) and a tile of 7 x 7 output pixels of one image:
// 49 accumulators in registers.  A warp is 32 consecutive FKR positions, a CTA up to 16 such warps; all of them read one
// input tile -- every channel's 9 x 9 patch (tile plus halo, zeros outside the image) -- staged once in shared memory.
// The work of a thread is its filter's FKW kernel list, pattern run after pattern run (the stride[] runs of Section 5.3):
// per kept kernel one channel index and four weights; the channel selects the patch in shared memory (an address, not a
// branch), the pattern selects the code -- one fully unrolled body per pattern, which streams the patch rows the
// pattern touches through nine registers and reuses each loaded word for up to four taps (load-redundancy
// elimination: 64 to 72 loads for 196 FMAs).  The pattern of a step is the same for all lanes of a warp, so nothing
// diverges; what the filter-kernel reorder buys here is lane balance: a warp needs as many steps per pattern as its
// longest lane, and filters of similar length and pattern mix sit in the same warp.
//
// Device layout (prun_plan.cpp): per warp group and pattern a range of STEPS; per step 32 lanes x {channel patch offset,
// 4 weights}, padded with zero-weight entries that read the patch of a lane with work (a broadcast).  Within a step the
// lanes' channels differ modulo 32 (or are equal), so the per-lane patch reads are free of shared-memory bank conflicts
// (patch pitch 81 words).  Like the dense path, a zero weight still multiplies its input: inputs must be finite.
//
// The kernel's time follows the kept kernels (steps), unlike the dense tensor-core path; its bound is the shared-memory
// load pipe: 2.7 to 3.1 FMAs per loaded word against the 4 the FP32 pipes could take.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/patdnn.h"
#include "kernels.hpp"

namespace patdnn {

namespace {

constexpr int kT = kPrunTile;                // 7 x 7 output pixels per thread
constexpr int kPatch = (kT + 2) * (kT + 2);  // 81 words per channel: odd, so channel c starts at bank 17 * c mod 32

template <typename T> __device__ __forceinline__ float load_f32(const T *p);
template <> __device__ __forceinline__ float load_f32<float>(const float *p) { return __ldg(p); }
template <> __device__ __forceinline__ float load_f32<__half>(const __half *p) { return __half2float(__ldg(p)); }
template <typename T> __device__ __forceinline__ void store_f32(T *p, float v);
template <> __device__ __forceinline__ void store_f32<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void store_f32<__half>(__half *p, float v) { *p = __float2half_rn(v); }

__host__ __device__ constexpr int tap_of(int mask, int k) {      // k-th set bit of a 9-bit pattern mask (ascending tap order = FKW weight order)
    int seen = 0;
    for (int t = 0; t < 9; ++t)
        if ((mask >> t) & 1) {
            if (seen == k) return t;
            ++seen;
        }
    return 0;
}
__host__ __device__ constexpr int min4(int a, int b, int c, int d) { return (a < b ? a : b) < (c < d ? c : d) ? (a < b ? a : b) : (c < d ? c : d); }
__host__ __device__ constexpr int max4(int a, int b, int c, int d) { return (a > b ? a : b) > (c > d ? c : d) ? (a > b ? a : b) : (c > d ? c : d); }

// All steps [s0, s1) of one pattern run of this warp.
struct Entry { uint32_t cb; float w0, w1, w2, w3; };
__device__ __forceinline__ Entry load_entry(const uint32_t *__restrict__ chan, const float *__restrict__ wts, int s, int lane) {
    Entry e;
    e.cb = __ldg(chan + static_cast<size_t>(s) * 32 + lane);
    e.w0 = __ldg(wts + (static_cast<size_t>(s) * 4 + 0) * 32 + lane); e.w1 = __ldg(wts + (static_cast<size_t>(s) * 4 + 1) * 32 + lane);
    e.w2 = __ldg(wts + (static_cast<size_t>(s) * 4 + 2) * 32 + lane); e.w3 = __ldg(wts + (static_cast<size_t>(s) * 4 + 3) * 32 + lane);
    return e;
}

// `first` is the entry of step s0 (fetched by the caller during the previous run); returns the entry of step s1, the first
// of the warp's next non-empty run (s_last = the warp's last step: nothing is read beyond it).
template <int MASK>
__device__ __forceinline__ Entry run_pattern(float (&acc)[kT * kT], const float *__restrict__ xs, const uint32_t *__restrict__ chan,
                                             const float *__restrict__ wts, int s0, int s1, int s_last, int lane, Entry first) {
    constexpr int T0 = tap_of(MASK, 0), T1 = tap_of(MASK, 1), T2 = tap_of(MASK, 2), T3 = tap_of(MASK, 3);
    constexpr int R0 = T0 / 3, R1 = T1 / 3, R2 = T2 / 3, R3 = T3 / 3;
    constexpr int S0 = T0 % 3, S1 = T1 % 3, S2 = T2 % 3, S3 = T3 % 3;
    constexpr int RMIN = min4(R0, R1, R2, R3), RMAX = max4(R0, R1, R2, R3);
    constexpr int CMIN = min4(S0, S1, S2, S3), CMAX = max4(S0, S1, S2, S3);
    // the next step's entry is fetched while this step computes
    uint32_t cb = first.cb;
    float w0 = first.w0, w1 = first.w1, w2 = first.w2, w3 = first.w3;
    Entry nx = first;
#pragma unroll 1
    for (int s = s0; s < s1; ++s) {
        nx = load_entry(chan, wts, (s + 1 <= s_last) ? s + 1 : s_last, lane);
        const float *xp = xs + cb;
#pragma unroll
        for (int ry = RMIN; ry <= RMAX + kT - 1; ++ry) {           // patch rows the pattern touches
            float row[kT + 2];
#pragma unroll
            for (int cx = CMIN; cx <= CMAX + kT - 1; ++cx) row[cx] = xp[ry * (kT + 2) + cx];
#pragma unroll
            for (int x = 0; x < kT; ++x) {
                if (ry - R0 >= 0 && ry - R0 < kT) acc[(ry - R0) * kT + x] = fmaf(w0, row[x + S0], acc[(ry - R0) * kT + x]);
                if (ry - R1 >= 0 && ry - R1 < kT) acc[(ry - R1) * kT + x] = fmaf(w1, row[x + S1], acc[(ry - R1) * kT + x]);
                if (ry - R2 >= 0 && ry - R2 < kT) acc[(ry - R2) * kT + x] = fmaf(w2, row[x + S2], acc[(ry - R2) * kT + x]);
                if (ry - R3 >= 0 && ry - R3 < kT) acc[(ry - R3) * kT + x] = fmaf(w3, row[x + S3], acc[(ry - R3) * kT + x]);
            }
        }
        cb = nx.cb; w0 = nx.w0; w1 = nx.w1; w2 = nx.w2; w3 = nx.w3;
    }
    return nx;
}

// grid = (N * tiles_y * tiles_x, filter groups of up to 512 positions), block = one warp per warp group (up to 16).
template <typename T>
__global__ void __launch_bounds__(kPrunWarps * 32, 1) conv_prun_kernel(const PrunParams p) {
    pdl_trigger();
    extern __shared__ float xs[];                                 // [C + 1][81]; plane C is all zero (padding entries read it)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int t = blockIdx.x;
    const int txi = t % p.tiles_x; t /= p.tiles_x;
    const int tyi = t % p.tiles_y; t /= p.tiles_y;
    const int n = t, y0 = tyi * kT, x0 = txi * kT;
    const T *in = static_cast<const T *>(p.in);
    pdl_wait();
    // stage the input tile: every channel's 9 x 9 patch, zeros outside the image.  Consecutive threads take consecutive
    // words of a patch row (nine pixels of one image row), so that a warp's requests fall into a few sectors; fp32 words
    // go straight to shared memory with 4-byte asynchronous copies (zero fill outside the image), fp16 words through
    // registers (they are converted on the way).
    const int words = p.C * kPatch;
    for (int i = tid; i < words; i += blockDim.x) {
        const int c = i / kPatch, r = i - c * kPatch, py = r / (kT + 2), px = r - py * (kT + 2);
        const int y = y0 - 1 + py, x = x0 - 1 + px;
        const bool ok = y >= 0 && y < p.H && x >= 0 && x < p.W;
        const T *src = in + ((static_cast<size_t>(n) * p.C + c) * p.H + (ok ? y : 0)) * p.W + (ok ? x : 0);
        if constexpr (sizeof(T) == 4) {
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(xs + i))), "l"(src),
                         "r"(ok ? 4 : 0) : "memory");
        } else {
            xs[i] = ok ? load_f32<T>(src) : 0.f;
        }
    }
    for (int i = tid; i < kPatch; i += blockDim.x) xs[p.C * kPatch + i] = 0.f;   // the zero patch of the padding entries
    if constexpr (sizeof(T) == 4) asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();
    // one warp per warp group (32 consecutive FKR positions); the CTA's up to 16 warps share the staged tile
    float acc[kT * kT];
#pragma unroll
    for (int i = 0; i < kT * kT; ++i) acc[i] = 0.f;
    const int g_cta = p.groups_per_cta;                           // warp groups of this CTA's 512 positions that exist
    if (warp < g_cta) {
        const int group = blockIdx.y * kPrunWarps + warp;
        const int *runs = p.run_ofs + static_cast<size_t>(group) * (p.P + 1);
        const int s_first = __ldg(runs), s_end = __ldg(runs + p.P);   // the group's steps are consecutive over its runs
        Entry e{};
        if (s_end > s_first) e = load_entry(p.chan, p.wts, s_first, lane);
        for (int q = 0; q < p.P; ++q) {
            const int s0 = __ldg(runs + q), s1 = __ldg(runs + q + 1);
            if (s0 == s1) continue;                               // warp-uniform
            switch (p.builtin[q]) {                               // one unrolled body per pattern of the built-in table
#define PATDNN_PRUN_CASE(id, mask) case id: e = run_pattern<mask>(acc, xs, p.chan, p.wts, s0, s1, s_end - 1, lane, e); break;
                PATDNN_PRUN_CASE(0, 0x01B) PATDNN_PRUN_CASE(1, 0x036) PATDNN_PRUN_CASE(2, 0x0D8) PATDNN_PRUN_CASE(3, 0x1B0)
                PATDNN_PRUN_CASE(4, 0x03A) PATDNN_PRUN_CASE(5, 0x0B8) PATDNN_PRUN_CASE(6, 0x09A) PATDNN_PRUN_CASE(7, 0x0B2)
                PATDNN_PRUN_CASE(8, 0x017) PATDNN_PRUN_CASE(9, 0x1D0) PATDNN_PRUN_CASE(10, 0x059) PATDNN_PRUN_CASE(11, 0x134)
#undef PATDNN_PRUN_CASE
                default: break;
            }
        }
    }
    // epilogue: bias + ReLU, then through shared memory so that the stores run along the pixels of a filter
    __syncthreads();                                              // every warp is done with the input tile
    float *os = xs;                                               // [positions of the CTA][49], pitch 49: conflict-free by lane
    __shared__ int s_f[kPrunWarps * 32];
    {
        const int pos = blockIdx.y * (kPrunWarps * 32) + tid;
        const int f = (warp < g_cta && pos < p.F) ? __ldg(p.reorder + pos) : -1;
        const float b = f >= 0 ? __ldg(p.bias + f) : 0.f;
        s_f[tid] = f;
        if (warp < g_cta) {
#pragma unroll
            for (int i = 0; i < kT * kT; ++i) {
                float v = acc[i] + b;
                if (p.relu) v = fmaxf(v, 0.f);
                os[tid * (kT * kT) + i] = v;
            }
        }
    }
    __syncthreads();
    T *out = static_cast<T *>(p.out);
    const int rows = g_cta * 32 * kT;                             // (filter, tile row) pairs: seven consecutive pixels each
    for (int i = tid; i < rows; i += blockDim.x) {
        const int fl = i / kT, yy = i - fl * kT;
        const int ff = s_f[fl], y = y0 + yy;
        if (ff < 0 || y >= p.H) continue;
        T *dst = out + ((static_cast<size_t>(n) * p.F + ff) * p.H + y) * p.W + x0;
        const float *src = os + fl * (kT * kT) + yy * kT;
#pragma unroll
        for (int xx = 0; xx < kT; ++xx)
            if (x0 + xx < p.W) store_f32<T>(dst + xx, src[xx]);
    }
}

}  // namespace

cudaError_t prepare_prun(const PrunPlan &pl, int dtype) {
    if (dtype == PATDNN_F16)
        return cudaFuncSetAttribute(conv_prun_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem_bytes);
    return cudaFuncSetAttribute(conv_prun_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem_bytes);
}

cudaError_t launch_prun(const PrunPlan &pl, const PrunParams &p, int dtype, cudaStream_t st) {
    if (p.N == 0) return cudaSuccess;
    const dim3 grid(static_cast<unsigned>(p.N) * pl.tiles_y * pl.tiles_x, pl.groups), block(pl.threads);
    if (dtype == PATDNN_F16) return launch_pdl(conv_prun_kernel<__half>, grid, block, pl.smem_bytes, st, 1, p);
    return launch_pdl(conv_prun_kernel<float>, grid, block, pl.smem_bytes, st, 1, p);
}

}  // namespace patdnn
