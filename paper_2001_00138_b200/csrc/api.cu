// C ABI of the library (declared in include/patdnn.h): handles, uploads, launches.  No torch types anywhere.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#include "../../include/patdnn.h"
#include "fkw_encoder.hpp"
#include "kernels.hpp"

using namespace patdnn;

namespace {

thread_local std::string g_cuda_error;
std::atomic<int64_t> g_launches{0};
std::mutex g_static_mutex;                    // serialises the host-side set-up of patdnn_conv_static

int cuda_fail(cudaError_t e, const char *what) {
    g_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
    cudaGetLastError();                       // clear the sticky-free error state
    return PATDNN_E_CUDA;
}
#define CU(call)                                             \
    do {                                                     \
        cudaError_t e_ = (call);                             \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call);  \
    } while (0)

template <typename T>
int upload(const std::vector<T> &v, T **dptr, std::vector<void *> &owned) {
    *dptr = nullptr;
    const size_t bytes = std::max<size_t>(v.size() * sizeof(T), 16);
    void *d = nullptr;
    CU(cudaMalloc(&d, bytes));
    owned.push_back(d);
    if (!v.empty()) CU(cudaMemcpy(d, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice));
    *dptr = static_cast<T *>(d);
    return PATDNN_OK;
}

}  // namespace

struct patdnn_layer {
    patdnn_desc desc{};
    Fkw fkw;
    std::vector<float> bias;                 // [F], zeros if the caller gave none
    int variant = PATDNN_VARIANT_REORDER;    // resolved
    bool on_device = false;
    int device = -1;
    std::vector<void *> owned;               // device allocations
    // canonical arrays on the device
    int32_t *d_offset = nullptr, *d_reorder = nullptr, *d_index = nullptr, *d_stride = nullptr;
    int32_t *d_kernel_pid = nullptr, *d_dense_slot = nullptr;
    float *d_weight = nullptr, *d_bias = nullptr;
    uint16_t *d_patterns = nullptr;
    // tiled kernel
    TiledPlan plan;
    uint32_t *d_rec = nullptr;
    int32_t *d_seg = nullptr, *d_seglen = nullptr;
    int64_t device_bytes = 0;
    // pattern-run kernel
    PrunPlan prun;
    uint32_t *d_prun_chan = nullptr;
    float *d_prun_wts = nullptr;
    int32_t *d_prun_runs = nullptr;
    // dense tensor-core path
    DensePlan dense;
    uint16_t *d_wdense = nullptr;
    void *d_act = nullptr;
    int *d_status = nullptr;
    DensePlan dense_static;                  // same plan with its activation map over the fixed scratch array
    bool dense_static_ready = false;         // guarded by g_static_mutex
    uint32_t spin_limit = 0;                 // patdnn_debug_wait: polls per bounded device-side wait (0 = default)
    int test_skip_load = 0;                  // patdnn_debug_wait: see DenseParams::test_skip_load
    SmallCJit *jit_nchw = nullptr;           // few-channel layer on the FP32 pipes: code generated for it (nullptr: tiled/generic kernel)
    DensePlan dense_pool;                    // plan over the same buffers whose epilogue can max-pool (built by a stack)
    int dense_pool_state = 0;                // 0 = not tried, 1 = ready, -1 = this layer's shape has no such plan
    // staging buffers of patdnn_conv_host
    void *d_in_stage = nullptr, *d_out_stage = nullptr;
    unsigned long long *chain_bar = nullptr;           // grid-barrier words of a stack's chained launch that reports to this handle's status
};

struct patdnn_stack_s {
    std::vector<patdnn_handle> layers;
    std::vector<int32_t> pool;
    // pipelined host entry point: two input/output slots, one stream per copy direction
    void *p_in[2] = {nullptr, nullptr}, *p_out[2] = {nullptr, nullptr};
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_run[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
    int64_t submitted = 0, waited = 0;
    std::vector<int> smallc;                  // per layer: index into smallc_w, or -1
    std::vector<SmallCWeights> smallc_w;      // few-channel layers fused with the layout of the tensor-core layer after them
    std::vector<SmallCJit *> smallc_jit;      // the same layers as run-time generated code (nullptr: static kernel)
    // runs of small tensor-core layers executed by one persistent cooperative kernel
    struct ChainRun {
        int first = 0, count = 0, grid = 0;
        ChainParams params{};
    };
    std::vector<ChainRun> chains;
    std::vector<int> chain_at;                // per layer: index into chains of the run that starts here, or -1
    float *d_partial = nullptr;               // partial-tile scratch shared by the runs
    unsigned long long *d_bar = nullptr;      // grid-barrier arrival counter
    void *buf[2] = {nullptr, nullptr};
    void *d_in = nullptr, *d_out = nullptr;   // staging buffers of patdnn_stack_run_host
    size_t buf_bytes = 0, in_bytes = 0, out_bytes = 0;
    int32_t oN = 0, oF = 0, oH = 0, oW = 0;
};

static size_t esize_of(int dtype) { return dtype == PATDNN_F16 ? 2 : 4; }

static DenseParams dense_params(const patdnn_layer *h, const DensePlan &pl) {
    const patdnn_desc &d = h->desc;
    DenseParams p{};
    p.bias = h->d_bias; p.status = h->d_status;
    p.N = d.N; p.C = d.C; p.H = d.H; p.W = d.W; p.F = d.F;
    p.TW = pl.TW; p.TH = pl.TH; p.TN = pl.TN; p.tiles_x = pl.tiles_x; p.tiles_y = pl.tiles_y; p.tiles_n = pl.tiles_n;
    p.n_ftiles = pl.n_ftiles; p.KB = pl.KB; p.stages = pl.stages; p.box_bytes = pl.box_bytes; p.relu = d.relu;
    p.iters_per_split = pl.iters_per_split; p.ksplit = pl.ksplit; p.na = pl.na; p.taps = pl.taps;
    p.spin_limit = h->spin_limit; p.test_skip_load = h->test_skip_load;
    return p;
}

// GEMM of a tensor-core layer whose split activations already sit in the buffer its activation map points to.
// next == nullptr: finished NCHW result into `out`; else the result goes, already split and channels-innermost, straight
// into the activation buffer of the tensor-core layer `next` (same spatial size; or, with `pooled` and a poolable
// plan, after a 2x2 max-pool taken in the epilogue).
static int dense_gemm(patdnn_layer *h, const DensePlan &pl, void *out, const patdnn_layer *next, cudaStream_t st,
                      bool pooled = false, const void *gather_src = nullptr) {
    DenseParams p = dense_params(h, pl);
    p.gather_src = gather_src;                               // gather plans read the layer's NCHW input themselves
    if (next) {
        p.mode = pooled ? 4 : 3; p.out = next->d_act; p.out_cp = next->dense.Cp;
    } else {
        p.mode = 0; p.out = out;
    }
    cudaError_t e = launch_dense_gemm(pl, p, h->desc.dtype, st);
    if (e != cudaSuccess) return cuda_fail(e, "tensor-core kernel launch");
    g_launches.fetch_add(pl.tail_tiles ? 2 : 1, std::memory_order_relaxed);
    return PATDNN_OK;
}

// One tensor-core layer from an NCHW input to its finished NCHW output.
static int dense_forward(patdnn_layer *h, const DensePlan &pl, const void *in, void *act, void *out, cudaStream_t st) {
    const patdnn_desc &d = h->desc;
    if (pl.gather) return dense_gemm(h, pl, out, nullptr, st, false, in);
    cudaError_t e = pl.im2col ? launch_im2col(in, d.dtype == PATDNN_F16, act, d.N, d.C, d.H, d.W, pl.S, st)
                              : launch_transition(in, d.dtype == PATDNN_F16, act, nullptr, 0, 0, 0, d.N, d.C, d.H, d.W, pl.Cp, pl.S, st);
    if (e != cudaSuccess) return cuda_fail(e, "layout kernel launch");
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return dense_gemm(h, pl, out, nullptr, st);
}

extern "C" {

int patdnn_encode(const float *weights, const uint8_t *mask, const uint16_t *pattern_set, int32_t n_patterns,
                  const patdnn_desc *desc, patdnn_handle *out) {
    if (!weights || !mask || !pattern_set || !desc || !out) return PATDNN_E_NULL;
    if (desc->F < 1 || desc->C < 1 || desc->N < 0 || desc->H < 1 || desc->W < 1) return PATDNN_E_SHAPE;
    if (desc->H > 65535 || desc->W > 65535 || desc->N > 65535 || desc->F > 65535) return PATDNN_E_SHAPE;
    // one image's input and output each stay below 2^31 elements (offsets inside an image are 32-bit; the batch is not
    // limited that way: offsets that include the image index are 64-bit)
    if (static_cast<int64_t>(std::max(desc->C, desc->F)) * desc->H * desc->W > INT32_MAX) return PATDNN_E_SHAPE;
    if (desc->dtype != PATDNN_F32 && desc->dtype != PATDNN_F16) return PATDNN_E_DTYPE;
    if (desc->variant < PATDNN_VARIANT_AUTO || desc->variant > PATDNN_VARIANT_PATTERN_RUN) return PATDNN_E_DTYPE;
    if (desc->filter_order != 0 && desc->filter_order != 1) return PATDNN_E_ORDER;
    if (desc->filter_order == 1 && !desc->order) return PATDNN_E_NULL;
    patdnn_layer *h = new (std::nothrow) patdnn_layer();
    if (!h) return PATDNN_E_ALLOC;
    int rc = PATDNN_OK;
    try {
        rc = build_fkw(weights, mask, pattern_set, n_patterns, desc->F, desc->C, desc->dtype,
                       desc->filter_order == 1 ? desc->order : nullptr, h->fkw);
        if (rc == PATDNN_OK) {
            h->desc = *desc;
            h->desc.order = nullptr;
            h->bias.assign(desc->F, 0.f);
            if (desc->bias) std::memcpy(h->bias.data(), desc->bias, sizeof(float) * desc->F);
            h->desc.bias = nullptr;
            // resolve the variant
            const bool can_tile = tiled_supported(h->fkw, desc->N, desc->H, desc->W, desc->dtype);
            if (desc->variant == PATDNN_VARIANT_AUTO) {
                h->variant = can_tile ? PATDNN_VARIANT_TILED : PATDNN_VARIANT_REORDER;
                // Tensor cores only where the dense reformulation is expected to win: compare a time estimate of the
                // zero-padded per-tap GEMMs with the CUDA-core kernel's rate on the kept weights (both measured on
                // B200: ~1200 TFLOP/s sustained for the 16-bit MMAs of this kernel, ~12 TFLOP/s for the tiled kernel).
                if (!(desc->flags & PATDNN_FLAG_HOST_ONLY) && desc->N > 0 &&
                    dense_supported(desc->F, desc->C, desc->N, desc->H, desc->W)) {
                    DensePlan dp;
                    plan_dense(desc->F, desc->C, desc->N, desc->H, desc->W, desc->dtype, dp);
                    const double terms = desc->dtype == PATDNN_F16 ? 1.0 : 3.0;
                    const double rows = static_cast<double>(dp.tiles_x) * dp.tiles_y * dp.tiles_n * 128.0;
                    const double t_dense = terms * 2.0 * dp.taps * dp.Cp * dp.Fp * rows / 1.2e15 +
                                           static_cast<double>(desc->N) * desc->H * desc->W * (desc->C * 4.0 + dp.Cp * 2.0 * dp.S) / 4.0e12 +
                                           4e-6;
                    // CUDA-core kernel: ~12 TFLOP/s on kept weights for large images, ~4 for 14x14-class layers (measured)
                    const double tiled_rate = (desc->H * desc->W <= 256) ? 4.0e12 : 1.2e13;
                    // (every CTA of the tiled kernel's filter dimension -- 16 filters each -- stages the whole input again)
                    const double t_tiled = 8.0 * h->fkw.K * static_cast<double>(desc->N) * desc->H * desc->W / tiled_rate + 1.5e-5 +
                                           std::ceil(desc->F / 16.0) * desc->N * desc->C * static_cast<double>(desc->H) * desc->W *
                                               (desc->dtype == PATDNN_F16 ? 2.0 : 4.0) / 3.5e12;
                    // layers with 9*C <= 64 (gathered-neighbourhood GEMM) are store-bound there: measured slower than the
                    // CUDA-core kernel on the RGB first layer, so AUTO leaves them on it unless it cannot run the layer
                    // (when the tiled kernel cannot take such a layer -- a pattern outside its builtin table -- fp32 layers
                    // go to the generic FKW kernel, which is exact to fp32: with so few terms per output the hi/lo split's
                    // per-product error is not averaged down)
                    if (t_dense < t_tiled && (!dp.im2col || (!can_tile && desc->dtype == PATDNN_F16))) h->variant = PATDNN_VARIANT_DENSE_TC;
                    // Very sparse layers: the pattern-run kernel's time follows the kept kernels (measured with 16 warps per
                    // CTA: ~0.8 us per step of the slowest warp plus ~20 us per wave of CTAs), the tensor cores' does
                    // not.  Worth planning only where it can win: at most ~1 in 7 kernels kept.
                    if (static_cast<double>(h->fkw.K) <= 0.15 * desc->F * desc->C && prun_supported(h->fkw, desc->N, desc->H, desc->W)) {
                        PrunPlan pp;
                        PrunLayout pl_tmp;
                        if (plan_prun(h->fkw, desc->N, desc->H, desc->W, pp, pl_tmp) == PATDNN_OK) {
                            const double ctas = static_cast<double>(desc->N) * pp.tiles_x * pp.tiles_y * pp.groups;
                            const double waves = std::ceil(ctas / sm_count());
                            const double t_prun = waves * (pp.max_warp_steps * (0.055e-6 * pp.groups_per_cta) + 25e-6);
                            const double t_best = h->variant == PATDNN_VARIANT_DENSE_TC ? t_dense : t_tiled;
                            if (t_prun < 0.8 * t_best) h->variant = PATDNN_VARIANT_PATTERN_RUN;   // clear wins only
                        }
                    }
                }
            } else {
                h->variant = desc->variant;
            }
            if (desc->N == 0) h->variant = PATDNN_VARIANT_REORDER;   // an empty batch launches nothing: no plan to make
            if (h->variant == PATDNN_VARIANT_TILED && !can_tile) rc = PATDNN_E_SHAPE;
            if (h->variant == PATDNN_VARIANT_PATTERN_RUN && !prun_supported(h->fkw, desc->N, desc->H, desc->W)) rc = PATDNN_E_SHAPE;
        }
        TiledLayout lay;
        PrunLayout play;
        if (rc == PATDNN_OK && h->variant == PATDNN_VARIANT_PATTERN_RUN)
            rc = plan_prun(h->fkw, desc->N, desc->H, desc->W, h->prun, play);
        if (rc == PATDNN_OK && h->variant == PATDNN_VARIANT_TILED)
            rc = plan_tiled(h->fkw, desc->N, desc->H, desc->W, desc->dtype, h->plan, lay);
        if (rc == PATDNN_OK && !(desc->flags & PATDNN_FLAG_HOST_ONLY)) {
            int dev = -1;
            cudaError_t e = cudaGetDevice(&dev);
            if (e != cudaSuccess) {
                rc = cuda_fail(e, "cudaGetDevice");
            } else {
                h->device = dev;
                const Fkw &k = h->fkw;
                if (h->variant == PATDNN_VARIANT_DENSE_TC) {
                    if (!dense_supported(k.F, k.C, desc->N, desc->H, desc->W)) rc = PATDNN_E_SHAPE;
                    if (!rc) {
                        plan_dense(k.F, k.C, std::max(desc->N, 1), desc->H, desc->W, desc->dtype, h->dense);
                        std::vector<uint16_t> wd;
                        build_dense_weights(k, h->dense, wd);
                        rc = upload(wd, &h->d_wdense, h->owned);
                        h->device_bytes = static_cast<int64_t>(wd.size()) * 2;
                    }
                    if (!rc) rc = upload(h->bias, &h->d_bias, h->owned);
                    if (!rc && h->dense.gather) {
                        h->d_act = h->d_wdense;                  // never read: the tensor map only needs a valid base
                    } else if (!rc) {
                        const size_t act_bytes = static_cast<size_t>(h->dense.S) * std::max(desc->N, 1) * desc->H *
                                                 desc->W * h->dense.Cp * 2;
                        cudaError_t ce = cudaMalloc(&h->d_act, act_bytes);
                        if (ce != cudaSuccess) rc = cuda_fail(ce, "cudaMalloc(split activations)");
                        else {
                            h->owned.push_back(h->d_act);
                            // padded channels must read as zero even when a producer writes fewer channels than Cp
                            ce = cudaMemset(h->d_act, 0, act_bytes);
                            if (ce != cudaSuccess) rc = cuda_fail(ce, "cudaMemset(split activations)");
                        }
                    }
                    if (!rc) {
                        std::vector<int> zero(4, 0);
                        rc = upload(zero, &h->d_status, h->owned);
                    }
                    if (!rc) rc = make_dense_maps(h->dense, h->d_act, h->d_wdense, std::max(desc->N, 1), desc->H, desc->W, desc->dtype);
                    if (rc == PATDNN_E_CUDA && g_cuda_error.empty()) g_cuda_error = "cuTensorMapEncodeTiled failed";
                    if (!rc) {
                        cudaError_t pe = prepare_dense(h->dense, desc->dtype);
                        if (pe != cudaSuccess) rc = cuda_fail(pe, "cudaFuncSetAttribute(dense kernel)");
                    }
                } else if (h->variant == PATDNN_VARIANT_PATTERN_RUN) {
                    rc = upload(play.chan, &h->d_prun_chan, h->owned);
                    if (!rc) rc = upload(play.wts, &h->d_prun_wts, h->owned);
                    if (!rc) rc = upload(play.run_ofs, &h->d_prun_runs, h->owned);
                    if (!rc) rc = upload(k.reorder, &h->d_reorder, h->owned);
                    if (!rc) rc = upload(h->bias, &h->d_bias, h->owned);
                    h->device_bytes = static_cast<int64_t>(play.chan.size()) * 4 + play.wts.size() * 4 + play.run_ofs.size() * 4 + k.F * 8;
                    if (!rc) {
                        cudaError_t pe = prepare_prun(h->prun, desc->dtype);
                        if (pe != cudaSuccess) rc = cuda_fail(pe, "cudaFuncSetAttribute(shared memory)");
                    }
                } else if (h->variant == PATDNN_VARIANT_TILED) {
                    rc = upload(lay.rec, &h->d_rec, h->owned);
                    if (!rc) rc = upload(lay.seg, &h->d_seg, h->owned);
                    if (!rc) rc = upload(lay.seglen, &h->d_seglen, h->owned);
                    if (!rc) rc = upload(k.reorder, &h->d_reorder, h->owned);
                    if (!rc) rc = upload(h->bias, &h->d_bias, h->owned);
                    h->device_bytes = static_cast<int64_t>(lay.rec.size()) * 4 + lay.seg.size() * 8 + k.F * 8;
                    if (!rc) {
                        cudaError_t pe = prepare_tiled(h->plan, desc->dtype);
                        if (pe != cudaSuccess) rc = cuda_fail(pe, "cudaFuncSetAttribute(shared memory)");
                    }
                } else {
                    rc = upload(k.offset, &h->d_offset, h->owned);
                    if (!rc) rc = upload(k.reorder, &h->d_reorder, h->owned);
                    if (!rc) rc = upload(k.index, &h->d_index, h->owned);
                    if (!rc) rc = upload(k.stride, &h->d_stride, h->owned);
                    if (!rc) rc = upload(k.weight_f32, &h->d_weight, h->owned);
                    if (!rc) rc = upload(k.patterns, &h->d_patterns, h->owned);
                    if (!rc) rc = upload(k.kernel_pid, &h->d_kernel_pid, h->owned);
                    if (!rc) rc = upload(h->bias, &h->d_bias, h->owned);
                    h->device_bytes = static_cast<int64_t>(k.K) * 24 + k.F * (4 * (k.P + 1) + 12);
                    if (!rc && h->variant == PATDNN_VARIANT_NOOPT) {
                        std::vector<int32_t> slot(static_cast<size_t>(k.F) * k.C, -1);
                        for (int i = 0; i < k.F; ++i)
                            for (int32_t kk = k.offset[i]; kk < k.offset[i + 1]; ++kk)
                                slot[static_cast<size_t>(k.reorder[i]) * k.C + k.index[kk]] = kk;
                        rc = upload(slot, &h->d_dense_slot, h->owned);
                        h->device_bytes += static_cast<int64_t>(slot.size()) * 4;
                    }
                }
                if (!rc) h->on_device = true;
                // AUTO on a few-channel layer that stays on the FP32 pipes: code generated for this layer (kept weights as
                // immediates) replaces the tiled kernel where the run-time compiler is available
                if (!rc && desc->variant == PATDNN_VARIANT_AUTO && h->variant != PATDNN_VARIANT_DENSE_TC && desc->N > 0 &&
                    smallc_split_supported(k.F, k.C) &&
                    static_cast<int64_t>(desc->N) * std::max(k.C, k.F) * desc->H * desc->W < (int64_t(1) << 31))
                    h->jit_nchw = smallc_jit_build(k, h->bias, k.C, desc->relu, desc->dtype == PATDNN_F16, nullptr, 1);
            }
        }
    } catch (const std::bad_alloc &) {
        rc = PATDNN_E_ALLOC;
    }
    if (rc != PATDNN_OK) {
        patdnn_free(h);
        return rc;
    }
    *out = h;
    return PATDNN_OK;
}

int patdnn_conv(patdnn_handle h, const void *in, void *out, void *stream) {
    if (!h) return PATDNN_E_NULL;
    if (!h->on_device) return PATDNN_E_NO_DEVICE;
    const patdnn_desc &d = h->desc;
    if (d.N == 0) return PATDNN_OK;                          // an empty batch has no tensors to point at
    if (!in || !out) return PATDNN_E_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (h->jit_nchw) {
        e = smallc_jit_launch(h->jit_nchw, in, out, d.N, d.H, d.W, st);
    } else if (h->variant == PATDNN_VARIANT_DENSE_TC) {
        return dense_forward(h, h->dense, in, h->d_act, out, st);
    } else if (h->variant == PATDNN_VARIANT_PATTERN_RUN) {
        PrunParams p{};
        p.in = in; p.out = out;
        p.chan = h->d_prun_chan; p.wts = h->d_prun_wts; p.run_ofs = h->d_prun_runs; p.reorder = h->d_reorder; p.bias = h->d_bias;
        p.N = d.N; p.C = d.C; p.H = d.H; p.W = d.W; p.F = d.F; p.P = h->fkw.P;
        p.tiles_x = h->prun.tiles_x; p.tiles_y = h->prun.tiles_y; p.relu = d.relu; p.groups_per_cta = h->prun.groups_per_cta;
        std::memcpy(p.builtin, h->prun.builtin, sizeof p.builtin);
        e = launch_prun(h->prun, p, d.dtype, st);
    } else if (h->variant == PATDNN_VARIANT_TILED) {
        TiledParams p{};
        p.in = in; p.out = out;
        p.rec = h->d_rec;
        p.seg = h->d_seg; p.seglen = h->d_seglen; p.reorder = h->d_reorder; p.bias = h->d_bias;
        p.N = d.N; p.C = d.C; p.H = d.H; p.W = d.W; p.F = d.F;
        p.TXn = h->plan.TXn; p.TYn = h->plan.TYn; p.tiles_total = h->plan.tiles_total;
        p.pitch = h->plan.pitch; p.lead = h->plan.lead; p.rows_max = h->plan.rows_max;
        p.nchunk = h->plan.nchunk; p.CC = h->plan.cfg.CC; p.nblk = h->plan.nblk; p.seg_cap = h->plan.seg_cap;
        p.copy_bytes = h->plan.copy_bytes; p.relu = d.relu;
        e = launch_tiled(h->plan, p, d.dtype, st);
    } else {
        SimpleParams p{};
        p.in = in; p.out = out;
        p.offset = h->d_offset; p.reorder = h->d_reorder; p.index = h->d_index; p.stride = h->d_stride;
        p.weight = reinterpret_cast<const float4 *>(h->d_weight); p.patterns = h->d_patterns;
        p.kernel_pid = h->d_kernel_pid; p.dense_slot = h->d_dense_slot; p.bias = h->d_bias;
        p.N = d.N; p.C = d.C; p.H = d.H; p.W = d.W; p.F = d.F; p.P = h->fkw.P; p.relu = d.relu;
        e = launch_simple(p, h->variant, d.dtype, st);
    }
    if (e != cudaSuccess) return cuda_fail(e, "kernel launch");
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return PATDNN_OK;
}

int patdnn_conv_static(patdnn_handle h, const void *in, void *out, void *stream) {
    if (!h) return PATDNN_E_NULL;
    if (!h->on_device) return PATDNN_E_NO_DEVICE;
    const patdnn_desc &d = h->desc;
    if (d.N == 0) return PATDNN_OK;                          // as patdnn_conv: an empty batch has no tensors to point at
    if (!in || !out) return PATDNN_E_NULL;
    if (h->variant != PATDNN_VARIANT_DENSE_TC) return patdnn_conv(h, in, out, stream);   // no scratch on those paths
    if (h->dense.gather) return dense_forward(h, h->dense, in, nullptr, out, static_cast<cudaStream_t>(stream));   // no scratch
    const size_t need = static_cast<size_t>(h->dense.S) * d.N * d.H * d.W * h->dense.Cp * 2;
    if (need > kStaticScratchBytes) return PATDNN_E_SCRATCH;
    // The array lives once per device and its address is baked into the handle's tensor map: the call must run on
    // the device the handle was encoded on.
    int dev = -1;
    CU(cudaGetDevice(&dev));
    if (dev != h->device) {
        g_cuda_error = "patdnn_conv_static: the current device is not the device the handle was encoded on";
        return PATDNN_E_CUDA;
    }
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        const cudaError_t e = static_scratch_address(&scratch);   // first call on this device: cudaGetSymbolAddress
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
        if (!h->dense_static_ready) {                         // first call for this handle: tensor map over the array
            h->dense_static = h->dense;
            const int rc = make_dense_maps(h->dense_static, scratch, h->d_wdense, d.N, d.H, d.W, d.dtype);
            if (rc) {
                if (rc == PATDNN_E_CUDA) g_cuda_error = "cuTensorMapEncodeTiled failed";
                return rc;
            }
            h->dense_static_ready = true;
        }
    }
    return dense_forward(h, h->dense_static, in, scratch, out, static_cast<cudaStream_t>(stream));
}

int patdnn_debug_wait(patdnn_handle h, uint32_t polls, int32_t skip_load_iteration) {
    if (!h) return PATDNN_E_NULL;
    if (skip_load_iteration < 0) return PATDNN_E_SHAPE;
    h->spin_limit = polls;
    h->test_skip_load = skip_load_iteration;
    return PATDNN_OK;
}

int patdnn_conv_host(patdnn_handle h, const void *in_host, void *out_host, void *stream) {
    if (!h || !in_host || !out_host) return PATDNN_E_NULL;
    if (!h->on_device) return PATDNN_E_NO_DEVICE;
    const patdnn_desc &d = h->desc;
    const size_t es = esize_of(d.dtype);
    const size_t in_b = static_cast<size_t>(d.N) * d.C * d.H * d.W * es;
    const size_t out_b = static_cast<size_t>(d.N) * d.F * d.H * d.W * es;
    if (in_b == 0) return PATDNN_OK;
    if (!h->d_in_stage) {
        CU(cudaMalloc(&h->d_in_stage, in_b));
        h->owned.push_back(h->d_in_stage);
        CU(cudaMalloc(&h->d_out_stage, out_b));
        h->owned.push_back(h->d_out_stage);
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CU(cudaMemcpyAsync(h->d_in_stage, in_host, in_b, cudaMemcpyHostToDevice, st));
    const int rc = patdnn_conv(h, h->d_in_stage, h->d_out_stage, stream);
    if (rc) return rc;
    CU(cudaMemcpyAsync(out_host, h->d_out_stage, out_b, cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    return PATDNN_OK;
}

int patdnn_check(patdnn_handle h) {
    if (!h) return PATDNN_E_NULL;
    if (!h->on_device) return PATDNN_E_NO_DEVICE;
    CU(cudaDeviceSynchronize());
    if (h->d_status) {
        int st = 0;
        CU(cudaMemcpy(&st, h->d_status, sizeof(int), cudaMemcpyDeviceToHost));
        if (st != 0) {
            cudaMemset(h->d_status, 0, sizeof(int));
            if (h->chain_bar) cudaMemset(h->chain_bar, 0, 16);   // the grid barrier may have been left half-way
            return PATDNN_E_DEVICE_TIMEOUT;
        }
    }
    return PATDNN_OK;
}

int patdnn_free(patdnn_handle h) {
    if (!h) return PATDNN_OK;
    for (void *p : h->owned) cudaFree(p);
    smallc_jit_free(h->jit_nchw);
    delete h;
    return PATDNN_OK;
}

int patdnn_export(patdnn_handle h, patdnn_fkw_view *v) {
    if (!h || !v) return PATDNN_E_NULL;
    const Fkw &k = h->fkw;
    v->F = k.F; v->C = k.C; v->P = k.P; v->K = k.K;
    v->offset = k.offset.data();
    v->reorder = k.reorder.data();
    v->index = k.index.data();
    v->stride = k.stride.data();
    v->weight = k.dtype == PATDNN_F16 ? static_cast<const void *>(k.weight_f16.data())
                                      : static_cast<const void *>(k.weight_f32.data());
    return PATDNN_OK;
}

int patdnn_decode(patdnn_handle h, float *dense_out) {
    if (!h || !dense_out) return PATDNN_E_NULL;
    decode_fkw(h->fkw, dense_out);
    return PATDNN_OK;
}

int patdnn_plan(patdnn_handle h, patdnn_plan_info *info) {
    if (!h || !info) return PATDNN_E_NULL;
    std::memset(info, 0, sizeof(*info));
    info->variant = h->variant;
    info->device_bytes = h->device_bytes;
    info->generated = h->jit_nchw ? 1 : 0;
    if (h->variant == PATDNN_VARIANT_TILED) {
        const TiledPlan &p = h->plan;
        info->tile_rows = p.cfg.TY; info->tile_cols = kTileCols;
        info->filters_per_warp = p.cfg.FR;
        info->warps_per_cta = p.cfg.PW * p.cfg.FW;
        info->channels_per_stage = p.cfg.CC;
        info->channel_splits = 1;
        info->grid_x = p.grid_pix * p.grid_fg; info->grid_y = 1; info->grid_z = 1;
        info->smem_bytes = p.smem_bytes;
        info->entries = p.entries;
    } else if (h->variant == PATDNN_VARIANT_PATTERN_RUN) {
        const PrunPlan &p = h->prun;
        info->tile_rows = kPrunTile; info->tile_cols = kPrunTile; info->filters_per_warp = 32;
        info->warps_per_cta = p.threads / 32; info->channels_per_stage = h->desc.C; info->channel_splits = 1;
        info->grid_x = h->desc.N * p.tiles_y * p.tiles_x; info->grid_y = p.groups; info->grid_z = 1;
        info->smem_bytes = p.smem_bytes;
        info->entries = p.entries;                               // lane entries, padding included: kept kernels / entries = lane use
    } else if (h->variant == PATDNN_VARIANT_DENSE_TC) {
        const DensePlan &p = h->dense;
        info->tile_rows = p.TH * p.MT; info->tile_cols = p.TW; info->filters_per_warp = p.BN; info->warps_per_cta = 10;
        info->channels_per_stage = 64; info->channel_splits = p.ksplit;
        // grid_x: CTAs of the main launch (plus, for the one-tile-per-CTA kernel, the tiles of a K-split tail launch, so
        // that it stays the tile count); grid_y: tiles shared by the persistent CTAs; grid_z: tiles given to a tail launch
        info->grid_x = (p.halo || p.pair) ? p.grid : p.grid + p.tail_tiles;
        info->grid_y = p.pair ? 2 * p.n_tiles : (p.halo ? p.n_tiles : 1);     // CTA pairs: in single-tile units
        info->grid_z = 1 + p.tail_tiles; info->smem_bytes = p.smem_bytes;
        info->entries = static_cast<int64_t>(p.taps) * p.Fp * p.Cp;
    } else {
        info->tile_rows = 1; info->tile_cols = 1; info->filters_per_warp = 1; info->warps_per_cta = 8;
        info->channels_per_stage = 0; info->channel_splits = 1;
        info->grid_x = (h->desc.H * h->desc.W + 255) / 256; info->grid_y = h->desc.F; info->grid_z = h->desc.N;
        info->entries = h->fkw.K;
    }
    return PATDNN_OK;
}

int patdnn_maxpool2x2(const void *in, void *out, int32_t N, int32_t C, int32_t H, int32_t W, int32_t dtype,
                      void *stream) {
    if (!in || !out) return PATDNN_E_NULL;
    if (N < 0 || C < 1 || H < 2 || W < 2) return PATDNN_E_SHAPE;
    if (dtype != PATDNN_F32 && dtype != PATDNN_F16) return PATDNN_E_DTYPE;
    cudaError_t e = launch_maxpool2x2(in, out, N, C, H, W, dtype, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail(e, "maxpool launch");
    if (N > 0) g_launches.fetch_add(1, std::memory_order_relaxed);
    return PATDNN_OK;
}

int patdnn_stack_create(const patdnn_handle *handles, const int32_t *pool_after, int32_t n, patdnn_stack *out) {
    if (!handles || !out) return PATDNN_E_NULL;
    if (n < 1) return PATDNN_E_SHAPE;
    patdnn_stack_s *s = new (std::nothrow) patdnn_stack_s();
    if (!s) return PATDNN_E_ALLOC;
    size_t max_bytes = 0;
    int32_t N = 0, C = 0, H = 0, W = 0, dtype = 0;
    for (int i = 0; i < n; ++i) {
        patdnn_handle h = handles[i];
        if (!h) { delete s; return PATDNN_E_NULL; }
        if (!h->on_device) { delete s; return PATDNN_E_NO_DEVICE; }
        const patdnn_desc &d = h->desc;
        if (i == 0) { N = d.N; C = d.C; H = d.H; W = d.W; dtype = d.dtype; }
        if (d.N != N || d.C != C || d.H != H || d.W != W || d.dtype != dtype) { delete s; return PATDNN_E_STACK; }
        C = d.F;
        max_bytes = std::max(max_bytes, static_cast<size_t>(N) * C * H * W * esize_of(dtype));
        const int pool = pool_after ? pool_after[i] : 0;
        if (pool) {
            if (H < 2 || W < 2) { delete s; return PATDNN_E_STACK; }
            H /= 2; W /= 2;
        }
        s->layers.push_back(h);
        s->pool.push_back(pool);
    }
    // tensor-core layer -> pool -> tensor-core layer: a second plan of the first layer whose epilogue pools in registers
    for (int i = 0; i + 1 < n; ++i) {
        patdnn_layer *h = s->layers[i], *nx = s->layers[i + 1];
        if (!s->pool[i] || h->variant != PATDNN_VARIANT_DENSE_TC || nx->variant != PATDNN_VARIANT_DENSE_TC || nx->dense.im2col ||
            h->dense_pool_state != 0)
            continue;
        const patdnn_desc &d = h->desc;
        h->dense_pool_state = -1;
        if (d.N < 1) continue;
        DensePlan pp;
        plan_dense(d.F, d.C, d.N, d.H, d.W, d.dtype, pp, true, h->dense.BN);
        if (!pp.poolable || pp.Fp != h->dense.Fp || pp.Cp != h->dense.Cp || pp.taps != h->dense.taps || (h->dense.gather && !pp.gather)) continue;   // a gather layer owns no activation buffer
        if (make_dense_maps(pp, h->d_act, h->d_wdense, d.N, d.H, d.W, d.dtype) != PATDNN_OK) continue;
        if (prepare_dense(pp, d.dtype) != cudaSuccess) { cudaGetLastError(); continue; }
        h->dense_pool = pp;
        h->dense_pool_state = 1;
    }
    // CUDA-core layer with few input channels -> tensor-core layer (no pool between): one kernel that writes the second
    // layer's operands instead of an NCHW tensor plus a layout pass
    s->smallc.assign(n, -1);
    for (int i = 0; i + 1 < n; ++i) {
        patdnn_layer *h = s->layers[i], *nx = s->layers[i + 1];
        const patdnn_desc &d = h->desc;
        if (h->variant == PATDNN_VARIANT_DENSE_TC || s->pool[i] || nx->variant != PATDNN_VARIANT_DENSE_TC || nx->dense.im2col ||
            nx->dense.Cp != 64 || !smallc_split_supported(d.F, d.C) || debug_option("smallc", 1) == 0 ||
            static_cast<int64_t>(d.N) * d.C * d.H * d.W >= (int64_t(1) << 31))
            continue;
        s->smallc_w.emplace_back();
        build_smallc_weights(h->fkw, h->bias, s->smallc_w.back());
        s->smallc_jit.push_back(smallc_jit_build(h->fkw, h->bias, d.C, d.relu, d.dtype == PATDNN_F16, nullptr));
        s->smallc[i] = static_cast<int>(s->smallc_w.size()) - 1;
    }
    // Runs of consecutive tensor-core layers with at most one tile per SM (small batches) as one persistent kernel per
    // run.  Opt-in (PATDNN_DEBUG=chain=1): correct, but measured no faster than one kernel per layer -- VGG-shaped stack
    // at batch 1: 205 us against 200 us; its layers are bound by the L2 -> SM traffic of their operand tiles (about
    // 14 TB/s in both forms), and the exchange of partial tiles through global memory with two grid barriers costs as
    // much per layer (about 8 us) as the launch, set-up and cluster exchange it replaces.
    s->chain_at.assign(n, -1);
    const int cgrid = debug_option("chain", 0) == 1 ? chain_grid(dtype) : 0;
    if (cgrid > 0) {
        auto eligible = [&](int i, ChainLayer &L) {
            patdnn_layer *h = s->layers[i];
            const patdnn_desc &d = h->desc;
            if (h->variant != PATDNN_VARIANT_DENSE_TC || h->dense.im2col || h->dense.gather || h->dense.taps != 9 || d.N < 1) return false;
            L = ChainLayer();
            if (!chain_box(d.N, d.H, d.W, s->pool[i] != 0, L)) return false;
            L.N = d.N; L.C = d.C; L.H = d.H; L.W = d.W; L.F = d.F;
            L.n_ftiles = (d.F + 127) / 128;
            L.KB = h->dense.KB; L.ipt = 9 * L.KB;
            L.n_tiles = L.tiles_x * L.tiles_y * L.tiles_n * L.n_ftiles;
            L.total = L.n_tiles * L.ipt;
            L.gw = std::min(cgrid, L.total);
            if (static_cast<long long>(L.total) * cgrid >= (1ll << 31)) return false;
            L.box_bytes = L.TW * L.TH * L.TN * 128;
            L.relu = d.relu; L.pool = s->pool[i] != 0;
            L.bias = h->d_bias;
            return L.n_tiles <= cgrid;                            // a chunk then touches at most two tiles
        };
        int i = 0;
        while (i < n) {
            ChainLayer L;
            if (!eligible(i, L)) { ++i; continue; }
            patdnn_stack_s::ChainRun run;
            run.first = i; run.grid = cgrid;
            bool good = true;
            while (i < n && run.count < kChainMaxLayers && eligible(i, L)) {
                patdnn_layer *h = s->layers[i];
                const bool more = i + 1 < n && run.count + 1 < kChainMaxLayers;
                ChainLayer nextL;
                const bool next_in = more && eligible(i + 1, nextL);
                const bool next_dense = i + 1 < n && s->layers[i + 1]->variant == PATDNN_VARIANT_DENSE_TC && !s->layers[i + 1]->dense.im2col;
                if (next_in || next_dense) { L.out_mode = 3; L.out = s->layers[i + 1]->d_act; L.out_cp = s->layers[i + 1]->dense.Cp; }
                else { L.out_mode = 0; L.out = nullptr; L.out_cp = 0; }          // NCHW destination patched in at run time
                if (make_chain_maps(run.params.mapA[run.count], run.params.mapB[run.count], L, h->dense, h->d_act, h->d_wdense, dtype) != PATDNN_OK) {
                    good = false;
                    break;
                }
                run.params.layer[run.count++] = L;
                ++i;
            }
            if (!good || run.count < 2) { if (run.count == 0) ++i; continue; }   // single layers stay on their own kernels
            run.params.n_layers = run.count;
            run.params.stages = chain_stages(dtype);
            run.params.status = s->layers[run.first]->d_status;
            s->chain_at[run.first] = static_cast<int>(s->chains.size());
            s->chains.push_back(run);
        }
        if (!s->chains.empty()) {
            cudaError_t e = cudaMalloc(reinterpret_cast<void **>(&s->d_partial), chain_partial_bytes(cgrid));
            if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void **>(&s->d_bar), 16);
            if (e == cudaSuccess) e = cudaMemset(s->d_bar, 0, 16);
            if (e != cudaSuccess) { patdnn_stack_free(s); return cuda_fail(e, "cudaMalloc(chain scratch)"); }
            for (auto &run : s->chains) {
                run.params.partial = s->d_partial;
                run.params.bar = s->d_bar;
                s->layers[run.first]->chain_bar = s->d_bar;
            }
        }
    }
    s->oN = N; s->oF = C; s->oH = H; s->oW = W;
    s->buf_bytes = std::max<size_t>(max_bytes, 16);
    const patdnn_desc &d0 = handles[0]->desc;
    s->in_bytes = static_cast<size_t>(d0.N) * d0.C * d0.H * d0.W * esize_of(dtype);
    s->out_bytes = static_cast<size_t>(N) * C * H * W * esize_of(dtype);
    for (int b = 0; b < 2; ++b) {
        cudaError_t e = cudaMalloc(&s->buf[b], s->buf_bytes);
        if (e != cudaSuccess) { patdnn_stack_free(s); return cuda_fail(e, "cudaMalloc(stack buffer)"); }
    }
    *out = s;
    return PATDNN_OK;
}

// Chained execution.  Where two tensor-core layers follow each other without a pool, the first one's epilogue writes
// the second one's input directly (bias + ReLU applied, channels innermost, operands split): no tensor in NCHW form and
// no layout kernel in between.  A pool between them is taken in the first one's epilogue where its shape allows a
// poolable plan, else folded into the layout kernel of the second.
static int stack_run_impl(patdnn_stack s, const void *in, void *out, void *stream, cudaEvent_t *ev);

int patdnn_stack_run(patdnn_stack s, const void *in, void *out, void *stream) {
    return stack_run_impl(s, in, out, stream, nullptr);
}

int patdnn_stack_run_timed(patdnn_stack s, const void *in, void *out, void *stream, float *layer_ms) {
    if (!s || !layer_ms) return PATDNN_E_NULL;
    const int n = static_cast<int>(s->layers.size());
    std::vector<cudaEvent_t> ev(n + 1, nullptr);
    int rc = PATDNN_OK;
    for (int i = 0; i <= n && !rc; ++i)
        if (cudaEventCreate(&ev[i]) != cudaSuccess) rc = cuda_fail(cudaGetLastError(), "cudaEventCreate");
    if (!rc) rc = stack_run_impl(s, in, out, stream, ev.data());
    if (!rc) {
        cudaError_t e = cudaEventSynchronize(ev[n]);
        if (e != cudaSuccess) rc = cuda_fail(e, "cudaEventSynchronize");
    }
    for (int i = 0; i < n && !rc; ++i)
        if (cudaEventElapsedTime(&layer_ms[i], ev[i], ev[i + 1]) != cudaSuccess) rc = cuda_fail(cudaGetLastError(), "cudaEventElapsedTime");
    for (cudaEvent_t e : ev)
        if (e) cudaEventDestroy(e);
    return rc;
}

// ev (optional, n + 1 events): ev[i] is recorded in front of layer i's launches, ev[n] behind the last launch.
static int stack_run_impl(patdnn_stack s, const void *in, void *out, void *stream, cudaEvent_t *ev) {
    if (!s || !in || !out) return PATDNN_E_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int n = static_cast<int>(s->layers.size());
    const void *cur = in;            // finished NCHW activations feeding the next layer (unless `direct`)
    bool cur_pool = false;           // a 2x2 max-pool still has to be applied to `cur`
    bool direct = false;             // the next layer's split input was already written by the previous epilogue
    int which = 0;
    int curH = s->layers[0]->desc.H, curW = s->layers[0]->desc.W;   // spatial size of `cur` (before a pending pool)
    for (int i = 0; i < n; ++i) {
        patdnn_layer *h = s->layers[i];
        const patdnn_desc &d = h->desc;
        if (d.N == 0) {
            if (ev) for (int j = i; j <= n; ++j) CU(cudaEventRecord(ev[j], st));
            return PATDNN_OK;
        }
        if (ev) CU(cudaEventRecord(ev[i], st));
        const bool last = (i == n - 1);
        const bool is_dense = h->variant == PATDNN_VARIANT_DENSE_TC;
        if (is_dense) {
            const bool next_dense = !last && s->layers[i + 1]->variant == PATDNN_VARIANT_DENSE_TC && !s->layers[i + 1]->dense.im2col;
            const bool fuse_pool = next_dense && s->pool[i] && h->dense_pool_state == 1;
            const DensePlan &use = fuse_pool ? h->dense_pool : h->dense;
            if (!direct && h->dense.im2col) {
                if (cur_pool) {
                    const int rc = patdnn_maxpool2x2(cur, s->buf[which], d.N, d.C, curH, curW, d.dtype, stream);
                    if (rc) return rc;
                    cur = s->buf[which];
                    which ^= 1;
                }
                if (!use.gather) {
                    cudaError_t e = launch_im2col(cur, d.dtype == PATDNN_F16, h->d_act, d.N, d.C, d.H, d.W, h->dense.S, st);
                    if (e != cudaSuccess) return cuda_fail(e, "layout kernel launch");
                    g_launches.fetch_add(1, std::memory_order_relaxed);
                }
            } else if (!direct) {
                cudaError_t e = launch_transition(cur, d.dtype == PATDNN_F16, h->d_act, nullptr, 0, cur_pool, 0, d.N, d.C,
                                                  curH, curW, h->dense.Cp, h->dense.S, st);
                if (e != cudaSuccess) return cuda_fail(e, "layout kernel launch");
                g_launches.fetch_add(1, std::memory_order_relaxed);
            }
            if (s->chain_at[i] >= 0) {
                // this layer's operands are in place: one persistent kernel runs it and the layers chained behind it
                const patdnn_stack_s::ChainRun &run = s->chains[s->chain_at[i]];
                const int e_idx = run.first + run.count - 1;
                ChainParams cp = run.params;
                cp.spin_limit = h->spin_limit; cp.test_skip_load = h->test_skip_load;
                const patdnn_desc &ld = s->layers[e_idx]->desc;
                if (cp.layer[run.count - 1].out_mode == 0) {
                    void *dst = (e_idx == n - 1) ? out : s->buf[which];
                    cp.layer[run.count - 1].out = dst;
                    cur = dst; which ^= 1; direct = false;
                } else {
                    direct = true;
                }
                if (ev) for (int j = i + 1; j <= e_idx; ++j) CU(cudaEventRecord(ev[j], st));
                cudaError_t ce = chain_launch(cp, run.grid, d.dtype, st);
                if (ce != cudaSuccess) return cuda_fail(ce, "chained tensor-core kernel launch");
                g_launches.fetch_add(1, std::memory_order_relaxed);
                cur_pool = false;                                 // pools inside and behind the run are taken while reducing
                curH = s->pool[e_idx] ? ld.H / 2 : ld.H; curW = s->pool[e_idx] ? ld.W / 2 : ld.W;
                i = e_idx;
                continue;
            }
            patdnn_layer *next = (next_dense && (!s->pool[i] || fuse_pool)) ? s->layers[i + 1] : nullptr;
            void *dst = next ? nullptr : ((last && !s->pool[i]) ? out : s->buf[which]);
            const int rc = dense_gemm(h, use, dst, next, st, fuse_pool, (use.gather && !direct) ? cur : nullptr);
            if (rc) return rc;
            direct = next != nullptr;
            if (!direct) { cur = dst; which ^= 1; }
            cur_pool = s->pool[i] != 0 && !fuse_pool;
            curH = d.H; curW = d.W;
        } else {
            if (cur_pool) {
                const int rc = patdnn_maxpool2x2(cur, s->buf[which], d.N, d.C, curH, curW, d.dtype, stream);
                if (rc) return rc;
                cur = s->buf[which];
                which ^= 1;
            }
            if (s->smallc[i] >= 0) {
                patdnn_layer *nx = s->layers[i + 1];
                SmallCJit *jit = s->smallc_jit[s->smallc[i]];
                cudaError_t e = jit ? smallc_jit_launch(jit, cur, nx->d_act, d.N, d.H, d.W, st)
                                    : launch_smallc_split(s->smallc_w[s->smallc[i]], cur, d.dtype == PATDNN_F16, nx->d_act, d.N, d.C,
                                                          d.H, d.W, d.F, d.relu, nx->dense.Cp, nx->dense.S, st);
                if (e != cudaSuccess) return cuda_fail(e, "few-channel kernel launch");
                g_launches.fetch_add(1, std::memory_order_relaxed);
                direct = true;
                cur_pool = false;
                curH = d.H; curW = d.W;
                continue;
            }
            void *dst = (last && !s->pool[i]) ? out : s->buf[which];
            const int rc = patdnn_conv(h, cur, dst, stream);
            if (rc) return rc;
            cur = dst;
            which ^= 1;
            cur_pool = s->pool[i] != 0;
            curH = d.H; curW = d.W;
            direct = false;
        }
    }
    if (cur_pool) {
        const patdnn_desc &ld = s->layers[n - 1]->desc;
        const int rc = patdnn_maxpool2x2(cur, out, ld.N, ld.F, ld.H, ld.W, ld.dtype, stream);
        if (rc) return rc;
    }
    if (ev) CU(cudaEventRecord(ev[n], st));
    return PATDNN_OK;
}

int patdnn_stack_run_host(patdnn_stack s, const void *in_host, void *out_host, void *stream) {
    if (!s || !in_host || !out_host) return PATDNN_E_NULL;
    if (!s->d_in) {
        CU(cudaMalloc(&s->d_in, std::max<size_t>(s->in_bytes, 16)));
        CU(cudaMalloc(&s->d_out, std::max<size_t>(s->out_bytes, 16)));
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    CU(cudaMemcpyAsync(s->d_in, in_host, s->in_bytes, cudaMemcpyHostToDevice, st));
    const int rc = patdnn_stack_run(s, s->d_in, s->d_out, stream);
    if (rc) return rc;
    CU(cudaMemcpyAsync(out_host, s->d_out, s->out_bytes, cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    return PATDNN_OK;
}

// Pipelined variant of patdnn_stack_run_host: the copies of call i+1 overlap the kernels of call i.
int patdnn_stack_submit_host(patdnn_stack s, const void *in_host, void *out_host, void *stream) {
    if (!s || !in_host || !out_host) return PATDNN_E_NULL;
    if (s->submitted - s->waited >= 2) return PATDNN_E_STACK;            // both slots in flight: wait for one first
    if (!s->h2d) {
        CU(cudaStreamCreateWithFlags(&s->h2d, cudaStreamNonBlocking));
        CU(cudaStreamCreateWithFlags(&s->d2h, cudaStreamNonBlocking));
        for (int b = 0; b < 2; ++b) {
            CU(cudaMalloc(&s->p_in[b], std::max<size_t>(s->in_bytes, 16)));
            CU(cudaMalloc(&s->p_out[b], std::max<size_t>(s->out_bytes, 16)));
            CU(cudaEventCreateWithFlags(&s->ev_in[b], cudaEventDisableTiming));
            CU(cudaEventCreateWithFlags(&s->ev_run[b], cudaEventDisableTiming));
            CU(cudaEventCreateWithFlags(&s->ev_out[b], cudaEventDisableTiming));
        }
    }
    const int b = static_cast<int>(s->submitted & 1);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // slot b was last used two submissions ago and has been waited for (checked above), so its buffers are free
    CU(cudaMemcpyAsync(s->p_in[b], in_host, s->in_bytes, cudaMemcpyHostToDevice, s->h2d));
    CU(cudaEventRecord(s->ev_in[b], s->h2d));
    CU(cudaStreamWaitEvent(st, s->ev_in[b], 0));
    const int rc = patdnn_stack_run(s, s->p_in[b], s->p_out[b], stream);
    if (rc) return rc;
    CU(cudaEventRecord(s->ev_run[b], st));
    CU(cudaStreamWaitEvent(s->d2h, s->ev_run[b], 0));
    CU(cudaMemcpyAsync(out_host, s->p_out[b], s->out_bytes, cudaMemcpyDeviceToHost, s->d2h));
    CU(cudaEventRecord(s->ev_out[b], s->d2h));
    ++s->submitted;
    return PATDNN_OK;
}

int patdnn_stack_wait_host(patdnn_stack s) {
    if (!s) return PATDNN_E_NULL;
    if (s->waited >= s->submitted) return PATDNN_OK;
    CU(cudaEventSynchronize(s->ev_out[s->waited & 1]));
    ++s->waited;
    return PATDNN_OK;
}

int patdnn_stack_out_shape(patdnn_stack s, int32_t *N, int32_t *F, int32_t *H, int32_t *W) {
    if (!s || !N || !F || !H || !W) return PATDNN_E_NULL;
    *N = s->oN; *F = s->oF; *H = s->oH; *W = s->oW;
    return PATDNN_OK;
}

int patdnn_stack_generated(patdnn_stack s, int32_t *count) {
    if (!s || !count) return PATDNN_E_NULL;
    int32_t n = 0;
    for (const SmallCJit *j : s->smallc_jit) n += j ? 1 : 0;
    *count = n;
    return PATDNN_OK;
}

int patdnn_stack_free(patdnn_stack s) {
    if (!s) return PATDNN_OK;
    for (int b = 0; b < 2; ++b)
        if (s->buf[b]) cudaFree(s->buf[b]);
    if (s->d_in) cudaFree(s->d_in);
    if (s->d_out) cudaFree(s->d_out);
    for (int b = 0; b < 2; ++b) {
        if (s->p_in[b]) cudaFree(s->p_in[b]);
        if (s->p_out[b]) cudaFree(s->p_out[b]);
        if (s->ev_in[b]) cudaEventDestroy(s->ev_in[b]);
        if (s->ev_run[b]) cudaEventDestroy(s->ev_run[b]);
        if (s->ev_out[b]) cudaEventDestroy(s->ev_out[b]);
    }
    for (SmallCJit *j : s->smallc_jit) smallc_jit_free(j);
    if (s->d_partial) cudaFree(s->d_partial);
    if (s->d_bar) cudaFree(s->d_bar);
    for (patdnn_layer *h : s->layers)
        if (h && h->chain_bar == s->d_bar) h->chain_bar = nullptr;
    if (s->h2d) cudaStreamDestroy(s->h2d);
    if (s->d2h) cudaStreamDestroy(s->d2h);
    delete s;
    return PATDNN_OK;
}

int64_t patdnn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }
void patdnn_reset_launch_count(void) { g_launches.store(0, std::memory_order_relaxed); }

const char *patdnn_strerror(int status) {
    switch (status) {
        case PATDNN_OK: return "ok";
        case PATDNN_E_NULL: return "a required pointer is NULL";
        case PATDNN_E_SHAPE: return "unsupported or inconsistent shape";
        case PATDNN_E_PATTERN_SET: return "pattern set is not a list of distinct 4-of-9 patterns (1..32 entries)";
        case PATDNN_E_MASK: return "a kernel mask is neither empty nor a pattern of the set";
        case PATDNN_E_ORDER: return "filter order is not a permutation";
        case PATDNN_E_CUDA: return "CUDA call failed";
        case PATDNN_E_NO_DEVICE: return "handle has no device image (host-only encode or no CUDA device)";
        case PATDNN_E_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
        case PATDNN_E_DTYPE: return "unknown dtype or variant";
        case PATDNN_E_ALLOC: return "host allocation failed";
        case PATDNN_E_STACK: return "stack layers do not chain";
        case PATDNN_E_SCRATCH: return "layer needs more scratch than the fixed 16 MiB device buffer holds";
        default: return "unknown status";
    }
}

const char *patdnn_last_cuda_error(void) { return g_cuda_error.c_str(); }
const char *patdnn_version(void) { return "patdnn-b200 0.1 (sm_100a)"; }

}  // extern "C"
