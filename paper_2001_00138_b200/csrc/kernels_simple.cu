// Generic (untiled) kernels: they take any pattern set and any shape, read the input straight from global memory and
// serve as the lower rungs of the ablation ladder of Section 6.3 and as the path for pattern sets the tiled kernel has
// no specialised code for.
//   noopt   : original filter order; one branch on the pattern per kernel inside the channel loop (the "No-opt"
//             code skeleton of Section 5.1).
//   reorder : walks the FKW arrays of Section 5.3 -- for the filter at position i, pattern run after pattern run
//             (stride[i][p] .. stride[i][p+1]), so the tap offsets are loop-invariant inside a run and no branch
//             on the pattern remains in the inner loop (the "+Reorder" skeleton); the result is written to output
//             channel reorder[i].
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstdlib>
#include <cstring>

#include "kernels.hpp"

namespace patdnn {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__half>(__half v) { return __half2float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __half from_f32<__half>(float v) { return __float2half_rn(v); }

// One thread = one output pixel of one filter position.  grid = (ceil(H*W/256), F, N).
template <typename T>
__global__ void __launch_bounds__(256) conv_fkw_reorder_kernel(SimpleParams p) {
    const int pix = blockIdx.x * blockDim.x + threadIdx.x;
    const int i = blockIdx.y;                  // filter position after FKR
    const int n = blockIdx.z;
    if (pix >= p.H * p.W) return;
    const int y = pix / p.W, x = pix - y * p.W;
    const T *in = static_cast<const T *>(p.in) + static_cast<size_t>(n) * p.C * p.H * p.W;
    const int32_t base = p.offset[i];
    const int32_t *srow = p.stride + static_cast<size_t>(i) * (p.P + 1);
    float acc = 0.f;
    for (int pat = 0; pat < p.P; ++pat) {
        const int32_t k0 = base + srow[pat], k1 = base + srow[pat + 1];
        if (k0 == k1) continue;
        // The four taps of this pattern: offsets and in-image predicates are fixed for the whole run.
        int off[4];
        bool ok[4];
        const uint32_t m = p.patterns[pat];
        int j = 0;
        for (int t = 0; t < 9; ++t) {
            if (!((m >> t) & 1u)) continue;
            const int r = t / 3, s = t - 3 * r;
            const int yy = y + r - 1, xx = x + s - 1;
            ok[j] = yy >= 0 && yy < p.H && xx >= 0 && xx < p.W;
            off[j] = yy * p.W + xx;
            ++j;
        }
        for (int32_t k = k0; k < k1; ++k) {
            const T *plane = in + static_cast<size_t>(p.index[k]) * p.H * p.W;
            const float4 w = p.weight[k];
            if (ok[0]) acc = fmaf(w.x, to_f32<T>(plane[off[0]]), acc);
            if (ok[1]) acc = fmaf(w.y, to_f32<T>(plane[off[1]]), acc);
            if (ok[2]) acc = fmaf(w.z, to_f32<T>(plane[off[2]]), acc);
            if (ok[3]) acc = fmaf(w.w, to_f32<T>(plane[off[3]]), acc);
        }
    }
    const int f = p.reorder[i];
    acc += p.bias[f];
    if (p.relu) acc = fmaxf(acc, 0.f);
    static_cast<T *>(p.out)[((static_cast<size_t>(n) * p.F + f) * p.H + y) * p.W + x] = from_f32<T>(acc);
}

// No-opt: filter f in original order, loop over all C channels, look the kernel's pattern up and branch on it.
template <typename T>
__global__ void __launch_bounds__(256) conv_noopt_kernel(SimpleParams p) {
    const int pix = blockIdx.x * blockDim.x + threadIdx.x;
    const int f = blockIdx.y;
    const int n = blockIdx.z;
    if (pix >= p.H * p.W) return;
    const int y = pix / p.W, x = pix - y * p.W;
    const T *in = static_cast<const T *>(p.in) + static_cast<size_t>(n) * p.C * p.H * p.W;
    float acc = 0.f;
    for (int c = 0; c < p.C; ++c) {
        const int32_t slot = p.dense_slot[static_cast<size_t>(f) * p.C + c];   // stored kernel id or -1
        if (slot < 0) continue;
        const uint32_t m = p.patterns[p.kernel_pid[slot]];
        const float4 w4 = p.weight[slot];
        const float w[4] = {w4.x, w4.y, w4.z, w4.w};
        const T *plane = in + static_cast<size_t>(c) * p.H * p.W;
        int j = 0;
        for (int t = 0; t < 9; ++t) {
            if (!((m >> t) & 1u)) continue;                       // the per-kernel branch on the pattern
            const int r = t / 3, s = t - 3 * r;
            const int yy = y + r - 1, xx = x + s - 1;
            if (yy >= 0 && yy < p.H && xx >= 0 && xx < p.W) acc = fmaf(w[j], to_f32<T>(plane[yy * p.W + xx]), acc);
            ++j;
        }
    }
    acc += p.bias[f];
    if (p.relu) acc = fmaxf(acc, 0.f);
    static_cast<T *>(p.out)[((static_cast<size_t>(n) * p.F + f) * p.H + y) * p.W + x] = from_f32<T>(acc);
}

template <typename T>
__global__ void __launch_bounds__(256) maxpool2x2_kernel(const T *in, T *out, int NC, int H, int W) {
    pdl_trigger();
    pdl_wait();
    const int Ho = H / 2, Wo = W / 2;
    const size_t total = static_cast<size_t>(NC) * Ho * Wo;
    for (size_t idx = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; idx < total;
         idx += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const int x = static_cast<int>(idx % Wo);
        const size_t t = idx / Wo;
        const int y = static_cast<int>(t % Ho);
        const size_t nc = t / Ho;
        const T *p = in + (nc * H + 2 * y) * W + 2 * x;
        const float a = fmaxf(to_f32<T>(p[0]), to_f32<T>(p[1]));
        const float b = fmaxf(to_f32<T>(p[W]), to_f32<T>(p[W + 1]));
        out[idx] = from_f32<T>(fmaxf(a, b));
    }
}

bool debug_option_text(const char *key, char *buf, size_t cap) {
    const char *env = std::getenv("PATDNN_DEBUG");
    if (!env || !key || cap == 0) return false;
    const size_t klen = std::strlen(key);
    for (const char *q = env; *q;) {
        const char *end = std::strchr(q, ',');
        const size_t len = end ? static_cast<size_t>(end - q) : std::strlen(q);
        if (len > klen && std::strncmp(q, key, klen) == 0 && q[klen] == '=') {
            const size_t n = std::min(len - klen - 1, cap - 1);
            std::memcpy(buf, q + klen + 1, n);
            buf[n] = 0;
            return true;
        }
        q += len + (end ? 1 : 0);
    }
    return false;
}

int debug_option(const char *key, int dflt) {
    char buf[32];
    return debug_option_text(key, buf, sizeof buf) ? std::atoi(buf) : dflt;
}

bool pdl_enabled() {
    static const bool on = debug_option("pdl", 1) != 0;
    return on;
}

int sm_count() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return 148; }
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) { cudaGetLastError(); n = 148; }
        cached[dev] = n;
    }
    return cached[dev];
}

cudaError_t launch_simple(const SimpleParams &p, int variant, int dtype, cudaStream_t stream) {
    if (p.N == 0) return cudaSuccess;
    dim3 grid((p.H * p.W + 255) / 256, p.F, p.N), block(256);
    if (variant == 1) {
        if (dtype == 1) conv_noopt_kernel<__half><<<grid, block, 0, stream>>>(p);
        else conv_noopt_kernel<float><<<grid, block, 0, stream>>>(p);
    } else {
        if (dtype == 1) conv_fkw_reorder_kernel<__half><<<grid, block, 0, stream>>>(p);
        else conv_fkw_reorder_kernel<float><<<grid, block, 0, stream>>>(p);
    }
    return cudaGetLastError();
}

cudaError_t launch_maxpool2x2(const void *in, void *out, int N, int C, int H, int W, int dtype, cudaStream_t stream) {
    const size_t total = static_cast<size_t>(N) * C * (H / 2) * (W / 2);
    if (total == 0) return cudaSuccess;
    const int blocks = static_cast<int>(std::min<size_t>((total + 255) / 256, sm_count() * 16));
    if (dtype == 1)
        return launch_pdl(maxpool2x2_kernel<__half>, dim3(blocks), dim3(256), 0, stream, 1, static_cast<const __half *>(in),
                          static_cast<__half *>(out), N * C, H, W);
    else
        return launch_pdl(maxpool2x2_kernel<float>, dim3(blocks), dim3(256), 0, stream, 1, static_cast<const float *>(in),
                          static_cast<float *>(out), N * C, H, W);
}

}  // namespace patdnn
