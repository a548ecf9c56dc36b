// Layer-specific code for the few-channel first layer of a stack, generated and compiled at run time.
//
// The paper's compiler emits, per model, branch-free code in which every kept weight is a constant of the instruction
// stream (Sections 5.1 and 5.4: pattern-based code generation, load redundancy elimination at compile time).  The static
// kernel in smallc_split.cu cannot do that -- it multiplies all 9*C taps of every filter, zeros included, with weights
// fetched as operands.  Here the same kernel body is written out for ONE layer: for each filter only the FFMAs of its
// kept weights, the weights as immediate operands, bias/ReLU/storage type folded in.  NVRTC (looked up with dlopen, no
// link-time dependency) compiles it for sm_100a when a stack is created; if NVRTC is not available the stack keeps the
// static kernel.  Everything else -- one pixel and all filters per thread, the swizzled shared-memory transpose, the
// split [S][N][H][W][64] output, programmatic dependent launch -- is as in smallc_split.cu.
#include <cuda.h>
#include <cuda_runtime.h>
#include <dlfcn.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <sstream>
#include <string>
#include <vector>

#include "kernels.hpp"

namespace patdnn {
namespace {

// ---- NVRTC through dlopen ------------------------------------------------------------------------------------------
typedef struct _nvrtcProgram *nvrtcProgram;
struct Nvrtc {
    int (*CreateProgram)(nvrtcProgram *, const char *, const char *, int, const char *const *, const char *const *) = nullptr;
    int (*CompileProgram)(nvrtcProgram, int, const char *const *) = nullptr;
    int (*GetCUBINSize)(nvrtcProgram, size_t *) = nullptr;
    int (*GetCUBIN)(nvrtcProgram, char *) = nullptr;
    int (*GetProgramLogSize)(nvrtcProgram, size_t *) = nullptr;
    int (*GetProgramLog)(nvrtcProgram, char *) = nullptr;
    int (*DestroyProgram)(nvrtcProgram *) = nullptr;
    bool ok = false;
};

const Nvrtc &nvrtc() {
    static Nvrtc n = [] {
        Nvrtc r;
        void *h = nullptr;
        for (const char *name : {"libnvrtc.so.12", "libnvrtc.so", "/usr/local/cuda/lib64/libnvrtc.so.12",
                                 "/usr/local/cuda/lib64/libnvrtc.so"}) {
            h = dlopen(name, RTLD_NOW | RTLD_LOCAL);
            if (h) break;
        }
        if (!h) return r;
#define PATDNN_SYM(field, sym) r.field = reinterpret_cast<decltype(r.field)>(dlsym(h, sym))
        PATDNN_SYM(CreateProgram, "nvrtcCreateProgram");
        PATDNN_SYM(CompileProgram, "nvrtcCompileProgram");
        PATDNN_SYM(GetCUBINSize, "nvrtcGetCUBINSize");
        PATDNN_SYM(GetCUBIN, "nvrtcGetCUBIN");
        PATDNN_SYM(GetProgramLogSize, "nvrtcGetProgramLogSize");
        PATDNN_SYM(GetProgramLog, "nvrtcGetProgramLog");
        PATDNN_SYM(DestroyProgram, "nvrtcDestroyProgram");
#undef PATDNN_SYM
        r.ok = r.CreateProgram && r.CompileProgram && r.GetCUBINSize && r.GetCUBIN && r.DestroyProgram;
        return r;
    }();
    return n;
}

// ---- driver entry points (module load, launch) ---------------------------------------------------------------------
struct Driver {
    CUresult (*ModuleLoadData)(CUmodule *, const void *) = nullptr;
    CUresult (*ModuleGetFunction)(CUfunction *, CUmodule, const char *) = nullptr;
    CUresult (*ModuleUnload)(CUmodule) = nullptr;
    CUresult (*LaunchKernelEx)(const CUlaunchConfig *, CUfunction, void **, void **) = nullptr;
    bool ok = false;
};

const Driver &driver() {
    static Driver d = [] {
        Driver r;
        auto get = [](const char *name) -> void * {
            void *sym = nullptr;
            cudaDriverEntryPointQueryResult q;
            if (cudaGetDriverEntryPoint(name, &sym, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
                return nullptr;
            return sym;
        };
        r.ModuleLoadData = reinterpret_cast<decltype(r.ModuleLoadData)>(get("cuModuleLoadData"));
        r.ModuleGetFunction = reinterpret_cast<decltype(r.ModuleGetFunction)>(get("cuModuleGetFunction"));
        r.ModuleUnload = reinterpret_cast<decltype(r.ModuleUnload)>(get("cuModuleUnload"));
        r.LaunchKernelEx = reinterpret_cast<decltype(r.LaunchKernelEx)>(get("cuLaunchKernelEx"));
        r.ok = r.ModuleLoadData && r.ModuleGetFunction && r.ModuleUnload && r.LaunchKernelEx;
        return r;
    }();
    return d;
}

std::string hexfloat(float v) {
    char buf[64];
    std::snprintf(buf, sizeof buf, "%af", static_cast<double>(v));
    return buf;
}

constexpr int kSplitWarps = 4;                                   // warps per CTA of the split-operand form

// The CUDA C++ source of the layer's kernel.
// nchw_out: write the caller's NCHW tensor (a layer run on its own) instead of the next layer's split operands.
std::string generate_source(const Fkw &fkw, const std::vector<float> &bias, int C, bool relu, bool half_in, bool nchw_out) {
    // kept weights per original filter: (k = 9*c + tap, value)
    std::vector<std::vector<std::pair<int, float>>> taps(64);
    std::vector<float> b(64, 0.f);
    for (int i = 0; i < fkw.F; ++i) {
        const int f = fkw.reorder[i];
        b[f] = bias[f];
        for (int32_t k = fkw.offset[i]; k < fkw.offset[i + 1]; ++k) {
            const int c = fkw.index[k];
            const uint32_t mask = fkw.patterns[fkw.kernel_pid[k]];
            int j = 0;
            for (int t = 0; t < 9; ++t)
                if ((mask >> t) & 1u) taps[f].push_back({9 * c + t, fkw.weight_f32[static_cast<size_t>(k) * 4 + j++]});
        }
    }
    std::ostringstream o;
    const int S = half_in ? 1 : 2;
    // Split-operand form: 4 warps per CTA and the finished 16-byte chunks go to the warp's shared-memory stage group by
    // group, so that a thread holds only its 3x3xC inputs and eight accumulators (six CTAs per SM); the NCHW form
    // stores straight from registers.
    const int warps = nchw_out ? 8 : kSplitWarps;
    o << "typedef unsigned int u32;\n";
    o << "extern \"C\" __global__ void __launch_bounds__(" << warps * 32 << ", " << (nchw_out ? 2 : 6) << ") patdnn_first_layer(const "
      << (half_in ? "unsigned short" : "float") << " *__restrict__ in, "
      << (nchw_out && !half_in ? "float" : "unsigned short") << " *__restrict__ dst, int N, int H, int W) {\n";
    if (!nchw_out) o << "  __shared__ __align__(16) unsigned char stage[" << warps << "][" << S << "][32 * 128];\n";
    o << "  asm volatile(\"griddepcontrol.launch_dependents;\" ::: \"memory\");\n";
    o << "  asm volatile(\"griddepcontrol.wait;\" ::: \"memory\");\n";
    o << "  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;\n";
    o << "  const unsigned P = (unsigned)N * H * W;\n";
    o << "  const size_t plane_out = (size_t)P * 64;\n";
    if (!nchw_out) o << "  unsigned char *st = stage[warp][0];\n";
    else o << "  (void)warp;\n";
    o << "  for (unsigned p0 = (blockIdx.x * " << warps << " + warp) * 32; p0 < P; p0 += gridDim.x * " << warps << " * 32) {\n";
    o << "    const unsigned pix = p0 + lane; const bool ok = pix < P;\n";
    o << "    const unsigned q = ok ? pix : 0u, r_ = q / (unsigned)W; const int x = (int)(q - r_ * W);\n";
    o << "    const unsigned n = r_ / (unsigned)H; const int y = (int)(r_ - n * H);\n";
    o << "    const bool rok[3] = {ok && y >= 1, ok, ok && y + 1 < H}; const bool cok[3] = {x >= 1, true, x + 1 < W};\n";
    o << "    const " << (half_in ? "unsigned short" : "float") << " *base = in + ((size_t)n * " << C << " * H + y) * W + x;\n";
    o << "    const int plane = H * W;\n";
    o << "    float v[" << 9 * C << "];\n";
    o << "#pragma unroll\n    for (int c = 0; c < " << C << "; ++c)\n#pragma unroll\n      for (int dy = 0; dy < 3; ++dy)\n#pragma unroll\n"
         "        for (int dx = 0; dx < 3; ++dx) {\n          float t = 0.f;\n          if (rok[dy] && cok[dx]) {\n";
    if (half_in)
        o << "            const unsigned short raw = base[c * plane + (dy - 1) * W + (dx - 1)];\n"
             "            asm(\"cvt.f32.f16 %0, %1;\" : \"=f\"(t) : \"h\"(raw));\n";
    else
        o << "            t = base[c * plane + (dy - 1) * W + (dx - 1)];\n";
    o << "          }\n          v[9 * c + 3 * dy + dx] = t;\n        }\n";
    if (nchw_out) o << "    const size_t obase = (size_t)n * " << fkw.F << " * plane + (size_t)y * W + x;\n";
    for (int g = 0; g < 8; ++g) {
        o << "    {\n";
        for (int j = 0; j < 8; ++j) o << "      float a" << j << " = " << hexfloat(b[8 * g + j]) << ";\n";
        size_t longest = 0;
        for (int j = 0; j < 8; ++j) longest = std::max(longest, taps[8 * g + j].size());
        for (size_t t = 0; t < longest; ++t)                     // round-robin over the eight chains
            for (int j = 0; j < 8; ++j)
                if (t < taps[8 * g + j].size())
                    o << "      a" << j << " = fmaf(" << hexfloat(taps[8 * g + j][t].second) << ", v[" << taps[8 * g + j][t].first
                      << "], a" << j << ");\n";
        if (relu)
            for (int j = 0; j < 8; ++j) o << "      a" << j << " = fmaxf(a" << j << ", 0.f);\n";
        if (nchw_out) {                                          // a warp stores 32 consecutive pixels of one filter plane
            for (int j = 0; j < 8; ++j) {
                const int f = 8 * g + j;
                if (f >= fkw.F) break;
                if (half_in)
                    o << "      if (ok) { unsigned short hv; asm(\"cvt.rn.f16.f32 %0, %1;\" : \"=h\"(hv) : \"f\"(a" << j << ")); dst[obase + (size_t)"
                      << f << " * plane] = hv; }\n";
                else
                    o << "      if (ok) dst[obase + (size_t)" << f << " * plane] = a" << j << ";\n";
            }
            o << "    }\n";
            continue;
        }
        o << "      u32 h0, h1, h2, h3" << (S == 2 ? ", l0, l1, l2, l3" : "") << ";\n";
        for (int j = 0; j < 8; j += 2) {
            const int w = j / 2;
            if (S == 2) {
                o << "      asm(\"cvt.rn.bf16x2.f32 %0, %1, %2;\" : \"=r\"(h" << w << ") : \"f\"(a" << j + 1 << "), \"f\"(a" << j << "));\n"
                  << "      { const float e0 = a" << j << " - __uint_as_float(h" << w << " << 16), e1 = a" << j + 1 << " - __uint_as_float(h" << w
                  << " & 0xffff0000u);\n"
                  << "        asm(\"cvt.rn.bf16x2.f32 %0, %1, %2;\" : \"=r\"(l" << w << ") : \"f\"(e1), \"f\"(e0)); }\n";
            } else {
                o << "      asm(\"cvt.rn.f16x2.f32 %0, %1, %2;\" : \"=r\"(h" << w << ") : \"f\"(a" << j + 1 << "), \"f\"(a" << j << "));\n";
            }
        }
        // this group's eight filters are 16-byte chunk g of the pixel's 128-byte row (chunk index swizzled by the row)
        o << "      *reinterpret_cast<uint4 *>(st + lane * 128 + ((" << g << " ^ (lane & 7)) << 4)) = make_uint4(h0, h1, h2, h3);\n";
        if (S == 2)
            o << "      *reinterpret_cast<uint4 *>(st + 4096 + lane * 128 + ((" << g << " ^ (lane & 7)) << 4)) = make_uint4(l0, l1, l2, l3);\n";
        o << "    }\n";
    }
    if (!nchw_out) o << "    const int rows = (int)(P - p0 < 32u ? P - p0 : 32u);\n";
    if (!nchw_out) o << "    __syncwarp();\n";
    for (int sp = 0; sp < (nchw_out ? 0 : S); ++sp) {
        o << "    {\n      unsigned char *g = reinterpret_cast<unsigned char *>(dst + " << sp
          << " * plane_out + (size_t)p0 * 64);\n#pragma unroll\n      for (int k = 0; k < 8; ++k) {\n"
          << "        const int idx = k * 32 + lane, row = idx >> 3, ch = idx & 7;\n"
          << "        if (row < rows) *reinterpret_cast<uint4 *>(g + idx * 16) = *reinterpret_cast<const uint4 *>(st + " << sp * 4096
          << " + row * 128 + ((ch ^ (row & 7)) << 4));\n"
          << "      }\n    }\n";
    }
    if (!nchw_out) o << "    __syncwarp();\n";                  // the stage is free again before the next pixels' chunks

    o << "  }\n}\n";
    return o.str();
}

}  // namespace

struct SmallCJit {
    CUmodule mod = nullptr;
    CUfunction fn = nullptr;
    int warps = 8;                                               // warps per CTA the source was generated for
};

SmallCJit *smallc_jit_build(const Fkw &fkw, const std::vector<float> &bias, int C, int relu, int is_half, std::string *log,
                            int nchw_out) {
    if (debug_option("jit", 1) == 0) return nullptr;
    const Nvrtc &rt = nvrtc();
    const Driver &dr = driver();
    if (!rt.ok || !dr.ok) { if (log) *log = "NVRTC or the driver entry points are not available"; return nullptr; }
    const std::string src = generate_source(fkw, bias, C, relu != 0, is_half != 0, nchw_out != 0);
    nvrtcProgram prog = nullptr;
    if (rt.CreateProgram(&prog, src.c_str(), "patdnn_first_layer.cu", 0, nullptr, nullptr) != 0) return nullptr;
    const char *opts[] = {"--gpu-architecture=sm_100a", "--std=c++17"};
    const int rc = rt.CompileProgram(prog, 2, opts);
    if (rc != 0) {
        if (log && rt.GetProgramLogSize && rt.GetProgramLog) {
            size_t n = 0;
            rt.GetProgramLogSize(prog, &n);
            log->resize(n);
            if (n) rt.GetProgramLog(prog, &(*log)[0]);
        }
        rt.DestroyProgram(&prog);
        return nullptr;
    }
    size_t n = 0;
    std::vector<char> cubin;
    if (rt.GetCUBINSize(prog, &n) != 0 || n == 0) { rt.DestroyProgram(&prog); return nullptr; }
    cubin.resize(n);
    const bool got = rt.GetCUBIN(prog, cubin.data()) == 0;
    rt.DestroyProgram(&prog);
    if (!got) return nullptr;
    cudaFree(nullptr);                                           // make sure the primary context is current
    SmallCJit *j = new SmallCJit();
    if (dr.ModuleLoadData(&j->mod, cubin.data()) != CUDA_SUCCESS ||
        dr.ModuleGetFunction(&j->fn, j->mod, "patdnn_first_layer") != CUDA_SUCCESS) {
        if (j->mod) dr.ModuleUnload(j->mod);
        delete j;
        if (log) *log = "cuModuleLoadData failed";
        return nullptr;
    }
    j->warps = nchw_out ? 8 : kSplitWarps;
    return j;
}

cudaError_t smallc_jit_launch(SmallCJit *j, const void *in, void *dst, int N, int H, int W, cudaStream_t st) {
    const long long P = static_cast<long long>(N) * H * W;
    if (P == 0) return cudaSuccess;
    const int per_cta = j->warps * 32;
    const long long blocks_needed = (P + per_cta - 1) / per_cta;
    const long long cap = static_cast<long long>(sm_count()) * (2048 / per_cta);   // a few rounds of resident CTAs
    const unsigned grid = static_cast<unsigned>(blocks_needed < cap ? blocks_needed : cap);
    CUlaunchConfig cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.gridDimX = grid; cfg.gridDimY = 1; cfg.gridDimZ = 1;
    cfg.blockDimX = static_cast<unsigned>(per_cta); cfg.blockDimY = 1; cfg.blockDimZ = 1;
    cfg.sharedMemBytes = 0;
    cfg.hStream = st;
    CUlaunchAttribute attr[1];
    std::memset(attr, 0, sizeof attr);
    unsigned na = 0;
    if (pdl_enabled()) {
        attr[0].id = CU_LAUNCH_ATTRIBUTE_PROGRAMMATIC_STREAM_SERIALIZATION;
        attr[0].value.programmaticStreamSerializationAllowed = 1;
        na = 1;
    }
    cfg.attrs = attr; cfg.numAttrs = na;
    void *args[] = {&in, &dst, &N, &H, &W};
    return driver().LaunchKernelEx(&cfg, j->fn, args, nullptr) == CUDA_SUCCESS ? cudaSuccess : cudaErrorLaunchFailure;
}

void smallc_jit_free(SmallCJit *j) {
    if (!j) return;
    if (j->mod && driver().ok) driver().ModuleUnload(j->mod);
    delete j;
}

}  // namespace patdnn
