// Internal interfaces between the C ABI, the host planners and the CUDA kernels.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdlib>
#include <string>
#include <vector>

#include "fkw_encoder.hpp"

namespace patdnn {

// ---- programmatic dependent launch ---------------------------------------------------------------------------------
// Every kernel of the library is launched with the programmatic-stream-serialization attribute: its CTAs may become
// resident while the previous kernel of the stream is still draining, run their set-up (barriers, TMEM allocation,
// bias slice), and block in pdl_wait() until the previous kernel has completed and its writes are visible.  No global
// data that an earlier kernel may produce is touched before pdl_wait().  PATDNN_PDL=0 turns the attribute off.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif
bool pdl_enabled();

// ---- debugging / tuning overrides and device facts ----------------------------------------------------------------
// ONE environment variable steers every override: PATDNN_DEBUG="key=value,key=value,...".  Keys (all optional):
//   pdl=0      launch without programmatic dependent launch        jit=0     no run-time generated first-layer kernel
//   smallc=0   no fused few-channel first layer in stacks          tile=TYxFR blocking of the CUDA-core tiled kernel
//   bn=N       cap of the tensor-core filter tile                  bn_keep=1 no narrowing of the filter tile
//   ksplit=N   cluster split of the channel loop (1, 2, 4, 8)      halo=0    no persistent halo-sharing kernel
//   mt=N       accumulator tiles per persistent CTA                pair=1    CTA-pair (cta_group::2) kernel
//   tail=0     no K-split tail launch                              halo_slack=N  MMA rows (%) a halo box may waste more than a free box
//   chain=1    persistent multi-layer kernel in stacks (opt-in)    chain_stages=N  its ring depth
// debug_option returns the integer after "key=", or dflt when the key (or the variable) is absent.
int debug_option(const char *key, int dflt);
bool debug_option_text(const char *key, char *buf, size_t cap);   // raw text after "key=" (false when absent)
int sm_count();                                                   // multiprocessors of the current device (148 if unknown)

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, int cluster, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (cluster > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = cluster; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (pdl_enabled()) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr; cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// ---- generic kernels (kernels_simple.cu) -------------------------------------------------------------------
struct SimpleParams {
    const void *in;
    void *out;
    const int32_t *offset;      // [F+1]
    const int32_t *reorder;     // [F]
    const int32_t *index;       // [K]
    const int32_t *stride;      // [F][P+1]
    const float4 *weight;       // [K] four kept weights (fp32 values; half-rounded for fp16 layers)
    const uint16_t *patterns;   // [P]
    const int32_t *kernel_pid;  // [K]
    const int32_t *dense_slot;  // [F][C] stored kernel id of (original filter, channel) or -1 (no-opt variant only)
    const float *bias;          // [F] original numbering
    int N, C, H, W, F, P, relu;
};

cudaError_t launch_simple(const SimpleParams &p, int variant, int dtype, cudaStream_t stream);
cudaError_t launch_maxpool2x2(const void *in, void *out, int N, int C, int H, int W, int dtype, cudaStream_t stream);

// ---- tiled kernel (kernels_tiled.cu) -----------------------------------------------------------------------
// Patterns the tiled kernel has straight-line code for.  A layer whose pattern set is a subset (in any order) runs
// on the tiled kernel; any other set runs on the generic FKW kernel.
constexpr int kBuiltinPatterns = 12;
extern const uint16_t kBuiltinPatternMasks[kBuiltinPatterns];

constexpr int kTileCols = 4;          // output columns per thread

struct TiledConfig {
    int TY;          // output rows per thread
    int FR;          // filters register-blocked per warp
    int PW;          // pixel warps per CTA (each covers 32 consecutive thread tiles)
    int FW;          // filter warps per CTA (each covers FR consecutive filter positions)
    int CC;          // input channels per shared-memory stage
    int NS;          // stages (2)
    int MINB;        // CTAs per SM the instance is compiled for (register cap)
};

struct TiledPlan {
    TiledConfig cfg{};
    int TXn = 0, TYn = 0;       // thread tiles per image row / tile rows per image
    int tiles_total = 0;        // N * TYn * TXn
    int pitch = 0;              // shared-memory row pitch in elements
    int lead = 0;               // zero elements in front of column 0 of every row
    int rows_max = 0;           // rows staged per CTA
    int nchunk = 0;             // ceil(C / CC)
    int nblk = 0;               // filter blocks, ceil(F / FR)
    int seg_cap = 0;            // largest (block, chunk) record segment, records
    int copy_bytes = 0;         // bytes per asynchronous copy when staging rows: 16, 8 or 4
    int grid_pix = 0, grid_fg = 0;
    int smem_bytes = 0;
    int64_t entries = 0;
};

struct TiledLayout {            // host image of the private device layout
    std::vector<uint32_t> rec;  // 8 words per record: {w0, w1, w2, w3 (float bits), descriptor, 0, 0, 0}
    std::vector<int32_t> seg;   // [nblk*nchunk] first record of each segment
    std::vector<int32_t> seglen;// [nblk*nchunk] records in the segment (END included)
};

struct TiledParams {
    const void *in;
    void *out;
    const uint32_t *rec;
    const int32_t *seg;
    const int32_t *seglen;
    const int32_t *reorder;
    const float *bias;
    int N, C, H, W, F;
    int TXn, TYn, tiles_total;
    int pitch, lead, rows_max;
    int nchunk, CC, nblk, seg_cap, copy_bytes;
    int relu;
};

// Can the tiled kernel run this layer (pattern set inside the builtin table, supported shape and dtype)?
bool tiled_supported(const Fkw &fkw, int N, int H, int W, int dtype);
// Pick a configuration for the shape and lay the kernels out for it.
int plan_tiled(const Fkw &fkw, int N, int H, int W, int dtype, TiledPlan &plan, TiledLayout &layout);
cudaError_t launch_tiled(const TiledPlan &plan, const TiledParams &p, int dtype, cudaStream_t stream);
cudaError_t prepare_tiled(const TiledPlan &plan, int dtype);   // opt in to the dynamic shared memory size

// ---- pattern-run kernel: one filter per lane, FKW pattern runs as step lists (prun_conv.cu, prun_plan.cpp) ---------------
constexpr int kPrunTile = 7;          // output pixels per thread: 7 x 7
constexpr int kPrunWarps = 16;        // warps per CTA, one per warp group of 32 filters
struct PrunPlan {
    int tiles_x = 0, tiles_y = 0;     // 7 x 7 tiles per image
    int groups = 0, threads = 0;      // filter groups of up to 512 positions (grid.y); threads per CTA
    int groups_per_cta = 0;           // warp groups a CTA holds (at most 16)
    int smem_bytes = 0;
    int builtin[32] = {};             // per pattern of the layer: its index in the built-in pattern table
    int64_t steps = 0, entries = 0;   // warp steps over all groups; lane entries (32 per step, padding included)
    int max_warp_steps = 0;           // steps of the slowest warp (two groups each): what a CTA waits for
};
struct PrunLayout {                   // host image of the private device layout
    std::vector<int32_t> run_ofs;     // [warp groups][P + 1] first step of each pattern run
    std::vector<uint32_t> chan;       // [steps][32] word offset of the lane's channel patch in shared memory
    std::vector<float> wts;           // [steps][4][32] the kernel's four kept weights (ascending tap order)
};
struct PrunParams {
    const void *in;
    void *out;
    const uint32_t *chan;
    const float *wts;
    const int32_t *run_ofs;
    const int32_t *reorder;
    const float *bias;
    int N, C, H, W, F, P;
    int tiles_x, tiles_y, relu;
    int groups_per_cta;               // warp groups (of the 16 a CTA can hold) that exist: ceil(min(F, 512) / 32)
    int builtin[32];
};
bool prun_supported(const Fkw &fkw, int N, int H, int W);
int plan_prun(const Fkw &fkw, int N, int H, int W, PrunPlan &plan, PrunLayout &layout);
cudaError_t prepare_prun(const PrunPlan &plan, int dtype);
cudaError_t launch_prun(const PrunPlan &plan, const PrunParams &p, int dtype, cudaStream_t stream);

// ---- dense tensor-core reformulation (umma_conv.cu) -----------------------------------------------------------
struct DensePlan {
    int S = 0;                  // operand planes: 2 (bf16 hi + lo, fp32 layers) or 1 (fp16 layers)
    int Cp = 0, KB = 0;         // channels padded to a multiple of 64; channel blocks
    int BN = 0, Fp = 0, n_ftiles = 0;
    int TW = 0, TH = 0, TN = 0; // pixel box (columns, rows, images), TW*TH*TN <= 128
    int tiles_x = 0, tiles_y = 0, tiles_n = 0;
    int box_bytes = 0, stages = 0, smem_bytes = 0, grid = 0;
    int im2col = 0, taps = 9;              // tiny C: 3x3 neighbourhood gathered into the channel dimension (one tap)
    int n_tiles = 0;                       // halo kernel: tiles shared by the persistent CTAs
    int halo = 0, MT = 1, na = 0;          // halo-sharing kernel: accumulator tiles per CTA, A-ring depth (stages = B ring)
    int ksplit = 1, iters_per_split = 0;   // the (channel block, tap) loop cut into ksplit ranges = CTAs of one cluster
    int pair = 0;                          // CTA-pair kernel (cta_group::2): tiles of 256 pixels x 256 filters, grid = 2 * clusters
    CUtensorMap mapB_pair{};               // weight box of one CTA of a pair: 128 of the 256 filters
    int gather = 0;                        // im2col layer on the persistent kernel: operand rows gathered in the kernel
    // Tail of a grid that is not a whole number of 148-CTA rounds: the last tail_tiles tiles run as a second launch of
    // the one-tile-per-CTA kernel with the K loop split tail_ks ways (clusters), instead of costing a whole extra round.
    int tail_tiles = 0, tail_ks = 1, tail_stages = 0, tail_smem = 0, tail_box_bytes = 0;
    CUtensorMap mapA_tail{};               // per-tap box of the tail launch (no halo rows)
    int poolable = 0;                      // boxes meet the conditions of the fused max-pool epilogue (mode 4)
    CUtensorMap mapA{}, mapB{};
};

struct DenseParams {
    void *out;
    const float *bias;
    int *status;                // device word: 0 = ok, else the role whose bounded wait expired
    int N, C, H, W, F;
    int TW, TH, TN, tiles_x, tiles_y, n_ftiles;
    int KB, stages, box_bytes, relu;
    int tiles_n, iters_per_split, ksplit, na, taps;
    int mode;                   // 0: out = caller's NCHW tensor; 3: out = next layer's split [S][N][H][W][out_cp] buffer;
                                // 4: as 3 after a fused 2x2 max-pool, [S][N][H/2][W/2][out_cp] (needs a pool_tiles plan)
    int out_cp;                 // channel pitch of the mode-3/4 destination
    int tile_base;              // one-tile-per-CTA kernel: index of the first tile this launch covers
    int tile_limit;             // persistent kernel: tiles [0, tile_limit) only (0 = all)
    const void *gather_src;     // gather plans: the layer's NCHW input (fp32 or fp16 as the layer's dtype)
    uint32_t spin_limit;        // polls a bounded device-side wait may take before it gives up (0 = the default, ~2 s)
    int test_skip_load;         // test hook of the one-tile-per-CTA kernel: the producer leaves out the loads of its
                                // (1-based) iteration test_skip_load, so that a bounded wait runs out (0 = off)
};

constexpr size_t kStaticScratchBytes = size_t(16) << 20;   // fixed device array behind patdnn_conv_static
cudaError_t static_scratch_address(void **ptr);            // first call per device looks the address up; not thread-safe

// ---- first-layer kernel writing a tensor-core layer's operands (smallc_split.cu) ----------------------------------
constexpr int kSmallCTaps = 36;            // 9 taps x at most 4 input channels
struct SmallCWeights {                     // passed by value as a kernel parameter: weights become constant-bank operands
    float w[64 * kSmallCTaps];             // [filter][9*c + tap], zeros where the pattern keeps nothing
    float bias[64];
};
bool smallc_split_supported(int F, int C);
void build_smallc_weights(const Fkw &fkw, const std::vector<float> &bias, SmallCWeights &wt);
// in: NCHW (fp32 or fp16); dst: [S][N][H][W][Cp] split operands of the next layer (Cp = 64), bias + ReLU applied.
cudaError_t launch_smallc_split(const SmallCWeights &wt, const void *in, int in_is_half, void *dst, int N, int C, int H, int W,
                                int F, int relu, int Cp, int S, cudaStream_t st);

// The same layer as code generated for it and compiled at run time (smallc_jit.cu): only the kept weights, as immediates.
// smallc_jit_build returns nullptr where NVRTC is not available (the caller keeps the static kernel).
struct SmallCJit;
// nchw_out = 1: the kernel writes the layer's NCHW output (dst = the caller's tensor) instead of split operands.
SmallCJit *smallc_jit_build(const Fkw &fkw, const std::vector<float> &bias, int C, int relu, int is_half, std::string *log,
                            int nchw_out = 0);
cudaError_t smallc_jit_launch(SmallCJit *j, const void *in, void *dst, int N, int H, int W, cudaStream_t st);
void smallc_jit_free(SmallCJit *j);

// ---- several tensor-core layers in one persistent cooperative kernel (umma_chain.cu) -----------------------------------
constexpr int kChainMaxLayers = 12;
struct ChainLayer {
    int N, C, H, W, F;
    int TW, TH, TN, tiles_x, tiles_y, tiles_n, n_ftiles;   // pixel box, boxes per image axis / batch, filter tiles of 128
    int KB, ipt;                // channel blocks of 64; iterations per tile = 9 * KB
    int n_tiles, total;         // tiles of the layer; total = n_tiles * ipt, cut into equal chunks over the working CTAs
    int gw;                     // working CTAs of this layer = min(grid, total)
    int box_bytes;              // TW * TH * TN * 128
    int relu, pool;             // pool: 2x2 max-pool taken while reducing
    int out_mode, out_cp;       // 0: NCHW tensor of the layer's dtype; 3: the next layer's split operands [S][N][h][w][out_cp]
    const float *bias;          // DEVICE [F]
    void *out;
};
struct ChainParams {
    CUtensorMap mapA[kChainMaxLayers], mapB[kChainMaxLayers];
    ChainLayer layer[kChainMaxLayers];
    int n_layers, stages;
    float *partial;             // DEVICE scratch: 2 * CTAs slots of 128 x 128 fp32; CTA c's partial of tile t is slot c + t
    unsigned long long *bar;    // DEVICE: arrivals at the grid barrier; only grows, a multiple of the grid size between launches
    int *status;                // DEVICE word: 0 = ok, else the role whose bounded wait expired
    uint32_t spin_limit;        // polls per bounded wait (0 = default)
    int test_skip_load;         // test hook: producers leave out the activation loads of this (1-based) iteration of their
                                // first layer's chunk, so that a bounded wait runs out (0 = off)
};
bool chain_box(int N, int H, int W, bool pool, ChainLayer &L);
int chain_stages(int dtype);
size_t chain_partial_bytes(int grid);
int chain_grid(int dtype);                                 // CTAs of the cooperative launch (0: not available here)
cudaError_t chain_launch(const ChainParams &p, int grid, int dtype, cudaStream_t st);
// tensor maps of one chained layer over its split activations and dense weights (PATDNN_* status)
int make_chain_maps(CUtensorMap &mapA, CUtensorMap &mapB, const ChainLayer &L, const DensePlan &pl, void *d_act, void *d_w, int dtype);

bool dense_supported(int F, int C, int N, int H, int W);
// pool_tiles: only pixel boxes whose epilogue can max-pool in registers (one image per box, 2/4/8/16 pixels wide, starting
// on even rows); sets pl.poolable.  force_bn pins the filter tile width, so that a second plan of a layer shares the
// weight layout of the first.
void plan_dense(int F, int C, int N, int H, int W, int dtype, DensePlan &pl, bool pool_tiles = false, int force_bn = 0);
void build_dense_weights(const Fkw &fkw, const DensePlan &pl, std::vector<uint16_t> &w);
int make_dense_maps(DensePlan &pl, void *d_act, void *d_w, int N, int H, int W, int dtype);
cudaError_t prepare_dense(const DensePlan &pl, int dtype);
cudaError_t launch_transition(const void *src, int src_is_half, void *dst, const float *bias, int relu, int pool, int clear,
                              int N, int C, int Hs, int Ws, int Cp, int S, cudaStream_t st);
cudaError_t launch_im2col(const void *src, int src_is_half, void *dst, int N, int C, int H, int W, int S, cudaStream_t st);
cudaError_t launch_dense_gemm(const DensePlan &pl, const DenseParams &p, int dtype, cudaStream_t st);

}  // namespace patdnn
