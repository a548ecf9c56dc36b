/*
 * patdnn.h -- C ABI of the pattern-sparse 3x3 convolution library (NVIDIA B200, sm_100a).
 *
 * The operation is the inference hot path of PatDNN (Niu et al., ASPLOS 2020): a 3x3, stride-1, pad-1
 * convolution whose weights satisfy the two constraint sets of Section 4.2 (Eq. 1) --
 *   kernel pattern pruning : every kept (filter, channel) kernel keeps exactly 4 of its 9 weights, at the
 *                            positions of one pattern out of a small fixed set;
 *   connectivity pruning   : whole (filter, channel) kernels are removed.
 * The host side builds the compressed weight storage of Section 5.3 (FKW: offset, reorder, index, stride and
 * weight arrays) after the filter-kernel reorder of Section 5.2 (FKR).  The device side has several kernels for the
 * same layer (PATDNN_VARIANT_* below): the paper's scheme on the FP32 pipes -- branch-free, pattern-specialised,
 * register-reusing loops (Sections 5.2 and 5.4) -- and a dense per-tap reformulation on the tensor cores, which on
 * this GPU is faster for all but very sparse or very thin layers and is what PATDNN_VARIANT_AUTO normally runs.
 * Every kernel fuses bias + ReLU.
 *
 * The three calls of the paper's problem statement are patdnn_encode, patdnn_conv and patdnn_free, with
 * patdnn_export / patdnn_decode / patdnn_strerror as inspection helpers.  Everything else declared here
 * (patdnn_conv_host, patdnn_conv_static, patdnn_check, patdnn_plan, patdnn_stack_*, patdnn_maxpool2x2, the launch
 * counter, patdnn_debug_wait, and the `variant` and `flags` fields of patdnn_desc) is an addition of this library
 * with no counterpart in the paper; each says so where it is declared.
 *
 * Conventions used by every call
 *   - tap t = 3*r + s (r = kernel row, s = kernel column); a pattern is a 9-bit mask, bit t set = tap t kept,
 *     exactly four bits set; the pattern id of a kernel is the 0-based position of its mask in `pattern_set`.
 *   - tensors are dense, row-major, NCHW / OIHW; the output has the input's spatial size.
 *   - out[n,f,y,x] = act(bias[f] + sum_{c,r,s} (weights*mask)[f,c,r,s] * in[n,c,y+r-1,x+s-1]), input = 0 outside
 *     the image, act = max(0,.) when `relu` is set (cross-correlation, no kernel flip).
 *   - every function returns a status code (0 = PATDNN_OK); nothing aborts, throws or prints.
 *   - pointers are marked HOST or DEVICE; the library never frees or keeps a caller pointer after the call
 *     returns, except where a stack keeps the handles it was built from.
 *   - there is no CPU fallback: the compute entry points fail with PATDNN_E_CUDA / PATDNN_E_NO_DEVICE when no
 *     usable device is present.
 */
#ifndef PATDNN_H
#define PATDNN_H

#include <stdint.h>

#if defined(__GNUC__)
#define PATDNN_API __attribute__((visibility("default")))
#else
#define PATDNN_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
    PATDNN_OK = 0,
    PATDNN_E_NULL = 1,          /* a required pointer is NULL */
    PATDNN_E_SHAPE = 2,         /* a size is non-positive, too large, or unsupported */
    PATDNN_E_PATTERN_SET = 3,   /* a pattern does not have exactly 4 of 9 bits, is duplicated, or P is not in 1..32 */
    PATDNN_E_MASK = 4,          /* a kernel's mask is neither empty nor a pattern of the set (Section 4.2) */
    PATDNN_E_ORDER = 5,         /* caller-supplied filter order is not a permutation */
    PATDNN_E_CUDA = 6,          /* a CUDA call failed; patdnn_last_cuda_error() has the text */
    PATDNN_E_NO_DEVICE = 7,     /* handle was encoded host-only, or no CUDA device is usable */
    PATDNN_E_DEVICE_TIMEOUT = 8,/* a bounded device-side wait expired */
    PATDNN_E_DTYPE = 9,         /* unknown dtype / variant value */
    PATDNN_E_ALLOC = 10,        /* host allocation failed */
    PATDNN_E_STACK = 11,        /* layers of a stack do not chain (shape or dtype mismatch) */
    PATDNN_E_SCRATCH = 12       /* the layer needs more scratch than the fixed device buffer of patdnn_conv_static */
};

enum { PATDNN_F32 = 0, PATDNN_F16 = 1 };   /* storage type of weights and activations; accumulation is fp32 */

/* Kernel variants (an addition: the paper generates one code version per layer and tunes it offline).
 * AUTO compares, at encode time, an estimate of the tensor-core variant's time (the zero-padded dense work of nine
 * per-tap GEMMs, three bf16 products per fp32 product) with the CUDA-core tiled kernel's rate on the kept weights and
 * takes the faster: DENSE_TC for every layer with more than 7 input channels that is not extremely sparse -- all but
 * the first layer of the VGG-16 and ResNet-50 shaped workloads -- and, for layers with at most 4 input channels and 64
 * filters, FP32 code generated for the layer at run time (kept weights as immediates; the tiled kernel where no
 * run-time compiler is present).  Other few-channel fp32 layers stay on TILED, or on REORDER when their pattern set
 * is not among the tiled kernel's twelve built-in patterns.  Layers that keep at most ~1 kernel in 7 are also planned
 * for PATTERN_RUN, whose time follows the kept kernels, and take it where its estimate clearly beats the others (on the
 * 512 -> 512 @ 14x14 sweep layer: from ~96 % connectivity pruning on).  The explicit values run the kernel they name and
 * exist for the ablation ladder of Section 6.3 (no optimisation -> +reorder -> +load-redundancy elimination -> tensor
 * cores). */
enum {
    PATDNN_VARIANT_AUTO = 0,
    PATDNN_VARIANT_NOOPT = 1,     /* original filter order, per-kernel branch on the pattern, global loads */
    PATDNN_VARIANT_REORDER = 2,   /* walks the FKW arrays in pattern order (branch-free per run), global loads */
    PATDNN_VARIANT_TILED = 3,     /* shared-memory tile + halo, register patch reuse across taps and filters */
    PATDNN_VARIANT_DENSE_TC = 4,  /* per-tap dense implicit GEMM on the tensor cores (tcgen05); fp32 layers use three
                                     bf16 products of operands split into hi + lo; chosen where it beats TILED */
    PATDNN_VARIANT_PATTERN_RUN = 5 /* one filter per lane, the FKW pattern runs of Section 5.3 as warp-uniform step lists,
                                     the whole input tile (all channels) in shared memory; its time follows the number
                                     of kept kernels; AUTO takes it for very sparse layers on small images */
};

enum { PATDNN_FLAG_HOST_ONLY = 1 };   /* encode on the host only: no device is touched, patdnn_conv is refused */

typedef struct patdnn_layer *patdnn_handle;   /* opaque; owned by the library until patdnn_free */
typedef struct patdnn_stack_s *patdnn_stack;  /* opaque; owned by the library until patdnn_stack_free */

typedef struct {
    int32_t F, C;            /* filters (output channels), input channels; kernel 3x3, stride 1, pad 1 */
    int32_t N, H, W;         /* batch and spatial size the handle is planned for */
    int32_t dtype;           /* PATDNN_F32 or PATDNN_F16 */
    int32_t relu;            /* 1 = fuse ReLU after the bias add */
    int32_t filter_order;    /* 0 = filter reorder of Section 5.2; 1 = caller-supplied order (kernel reorder still applies) */
    const int32_t *order;    /* HOST [F] permutation (position -> original filter) when filter_order == 1, else NULL */
    const float *bias;       /* HOST [F] in original filter numbering, or NULL for zeros */
    int32_t variant;         /* PATDNN_VARIANT_* (addition; 0 = AUTO) */
    int32_t flags;           /* PATDNN_FLAG_* (addition; 0 = none) */
} patdnn_desc;

/*
 * patdnn_encode -- validate a pruned layer against its pattern set (Section 4.2), run the filter-kernel reorder
 * (Section 5.2), build the FKW arrays (Section 5.3), derive the private device layout and upload it.
 *   weights      HOST float  [F][C][3][3]; values where mask == 0 are ignored; a kept weight may be 0.0
 *   mask         HOST uint8  [F][C][3][3], entries 0 or 1
 *   pattern_set  HOST uint16 [n_patterns] 9-bit masks, 1 <= n_patterns <= 32
 *   desc         HOST; copied
 *   out          receives the handle on success (untouched on failure)
 * Size limits (E_SHAPE beyond them): F, N, H, W <= 65535; max(C, F) * H * W < 2^31 (one image's input and output; the
 * whole batch may hold more than 2^31 elements); PATDNN_VARIANT_DENSE_TC additionally H, W <= 4096 and
 * N * ceil(C / 64) <= 65535 (AUTO falls back to a CUDA-core variant beyond that).
 * Errors: E_NULL, E_SHAPE, E_PATTERN_SET, E_MASK, E_ORDER, E_DTYPE, E_ALLOC, E_CUDA.
 * The call is synchronous (it returns after the upload completed) and uses the current CUDA device.
 */
PATDNN_API int patdnn_encode(const float *weights, const uint8_t *mask, const uint16_t *pattern_set, int32_t n_patterns,
                  const patdnn_desc *desc, patdnn_handle *out);

/*
 * patdnn_conv -- run the layer of Section 2.1 / Section 4.2 (formula at the top of this file) asynchronously on
 * `stream`, with the kernel the handle was planned for:
 *   TILED     shared-memory tile + halo staging, pattern-ordered branch-free FMA bodies, register patch reused by the
 *             four taps of a kernel and by the filters of a warp (Sections 5.2 and 5.4), output scattered through reorder[];
 *   PATTERN_RUN  one filter per lane: the filter's FKW pattern runs (stride[], Section 5.3) as warp-uniform step lists, the
 *             channel of a kernel an indirect shared-memory address, one unrolled body per pattern that streams the
 *             patch rows through registers; the whole input tile (all channels) in shared memory: needs built-in
 *             patterns and (C + 1) * 324 bytes <= 200 KB;
 *   REORDER / NOOPT  the generic kernels of the ablation ladder (any pattern set);
 *   DENSE_TC  one layout kernel (NCHW -> channels-innermost, operands split into bf16 hi + lo for fp32 layers) into a
 *             handle-owned scratch buffer, then the tcgen05 implicit GEMM over nine shifted TMA boxes (one launch, plus a
 *             second launch for the last partial round of tiles where the plan has one);
 *   generated FP32 code (AUTO, few-channel layers): one kernel.
 *   in   DEVICE [N][C][H][W] of the handle's dtype (float or IEEE half), 16-byte aligned
 *   out  DEVICE [N][F][H][W] of the same dtype, 16-byte aligned; must not overlap `in`
 *   stream  a cudaStream_t (NULL = default stream).  No synchronisation happens inside.
 * Errors: E_NULL, E_NO_DEVICE, E_CUDA (launch failure).
 */
PATDNN_API int patdnn_conv(patdnn_handle h, const void *in, void *out, void *stream);

/*
 * patdnn_conv_host (addition, used by end-to-end measurements) -- the same operation with HOST buffers: copies `in` to a handle-owned device buffer, runs the
 * layer, copies the result back, all on `stream`, and waits for the stream before returning.  Pinned host memory
 * makes the copies asynchronous with respect to other streams.  The device buffers are allocated on first use and
 * live until patdnn_free.
 */
PATDNN_API int patdnn_conv_host(patdnn_handle h, const void *in_host, void *out_host, void *stream);

/*
 * patdnn_conv_static -- patdnn_conv for callers that cannot allocate device memory when they run a layer: code inside
 * a CUDA-graph replay loop or a real-time control loop, a plug-in that runs under a host whose memory pool it must
 * not touch, or a process whose allocator is locked down after start-up.  The paper has no counterpart; this is an
 * addition of this library.
 *
 * The tensor-core variant of a layer needs scratch for the re-laid-out, hi/lo-split activations.  patdnn_conv keeps
 * that scratch in a buffer allocated by patdnn_encode; this entry point uses a fixed 16 MiB device array that is part
 * of the library image instead, and calls no cudaMalloc, cudaFree or allocating library routine.
 *   - in, out, stream: as for patdnn_conv (DEVICE pointers supplied by the caller).
 *   - limit: S * N * H * W * roundup(C, 64) * 2 bytes <= 16 MiB (S = 2 for fp32 layers, 1 for fp16 layers); a larger
 *     layer is refused with PATDNN_E_SCRATCH.  Layers that run on a CUDA-core variant need no scratch and are simply
 *     forwarded to patdnn_conv.
 *   - the first call on a device (and the first call for a handle) does set-up work on the host: it looks up the
 *     device address of the array and encodes a tensor map over it.  Make that first call before starting any stream
 *     capture.  The call must be made with the device current on which the handle was encoded (PATDNN_E_CUDA
 *     otherwise); the set-up is serialised between host threads.
 *   - all calls, from every handle, share the one array, which keeps whatever the last call left in it; the kernels
 *     overwrite everything they read, so nothing needs clearing, but two calls that can overlap on the GPU (different
 *     streams without an ordering between them) race on the array and must be serialised by the caller.
 */
PATDNN_API int patdnn_conv_static(patdnn_handle h, const void *in, void *out, void *stream);

/*
 * patdnn_check (addition) -- wait for the device and report whether any kernel launched for this handle gave up on a bounded
 * device-side wait (PATDNN_E_DEVICE_TIMEOUT) or a CUDA error is pending (PATDNN_E_CUDA).  Synchronous.
 */
PATDNN_API int patdnn_check(patdnn_handle h);

/* patdnn_free -- release the handle and everything it owns (device and host).  NULL is accepted. */
PATDNN_API int patdnn_free(patdnn_handle h);

/* Canonical FKW arrays (Section 5.3), HOST memory owned by the handle and valid until patdnn_free.
 *   offset  [F+1] kernels stored before filter position i; offset[F] = K
 *   reorder [F]   original output channel of the filter at position i
 *   index   [K]   input channel of stored kernel k
 *   stride  [F][P+1] per filter, cumulative kernel counts per pattern (stride[i][0] = 0, stride[i][P] = length)
 *   weight  [K][4] the kept weights in ascending tap order: float (F32) or IEEE half bit patterns (F16, uint16)
 * Order inside a filter: ascending pattern id, then ascending input channel.  Filter order: ascending length; inside
 * one length a greedy chain from the smallest original id to the most similar unplaced filter (ties: smallest id).
 */
typedef struct {
    int32_t F, C, P, K;
    const int32_t *offset;
    const int32_t *reorder;
    const int32_t *index;
    const int32_t *stride;
    const void *weight;
} patdnn_fkw_view;

/* patdnn_export -- fill `v` with pointers to the handle's canonical FKW arrays (no copy). */
PATDNN_API int patdnn_export(patdnn_handle h, patdnn_fkw_view *v);

/* patdnn_decode -- rebuild dense HOST float [F][C][3][3] weights from the FKW arrays; equals weights*mask bit for
 * bit for F32 handles and the half-rounded values for F16 handles. */
PATDNN_API int patdnn_decode(patdnn_handle h, float *dense_out);

/* Planned launch geometry of a handle, for reports and tests (addition). */
typedef struct {
    int32_t variant;            /* resolved PATDNN_VARIANT_* */
    int32_t tile_rows, tile_cols;   /* output pixels per thread (rows x columns) */
    int32_t filters_per_warp;   /* register-blocked filters sharing one input patch */
    int32_t warps_per_cta;
    int32_t channels_per_stage; /* input channels staged per shared-memory buffer */
    int32_t channel_splits;     /* >1: the channel range is split across a thread-block cluster */
    int32_t grid_x, grid_y, grid_z; /* CUDA-core kernels: the launch grid.  Tensor-core path: grid_x = CTAs of the main
                                     * launch (= tiles for the one-tile-per-CTA kernel), grid_y = tiles shared by the
                                     * persistent CTAs (1 otherwise), grid_z = 1 + tiles handed to a second, K-split
                                     * launch when the tile count is not a whole number of rounds of one CTA per SM */
    int32_t smem_bytes;
    int64_t device_bytes;       /* bytes of the private device layout */
    int64_t entries;            /* kernel entries in the device layout (kept kernels plus padding) */
    int32_t generated;          /* 1: patdnn_conv runs code generated for this layer at encode time (few input channels
                                 * under PATDNN_VARIANT_AUTO, run-time compiler present); the fields above then describe
                                 * the kernel it replaces */
    int32_t reserved;
} patdnn_plan_info;

PATDNN_API int patdnn_plan(patdnn_handle h, patdnn_plan_info *info);

/*
 * Stacks (addition; the paper's framework fuses and chains layers in its graph optimiser, which is out of scope here).
 * A stack chains layers on the device: layer i's output is layer i+1's input, optionally through a 2x2/stride-2
 * max-pool (the VGG-16 arrangement).  The stack owns two ping-pong activation buffers; the handles stay owned by
 * the caller and must outlive the stack.  Between two tensor-core layers no NCHW tensor is formed: the first one's
 * kernel writes the second one's operands (after the pool, where one follows, for which patdnn_stack_create may add a
 * second launch plan to the first layer's handle); a first layer with at most 4 input channels and 64 filters that is
 * followed by a tensor-core layer runs as one FP32 kernel that writes that layer's operands.  A handle may serve
 * several stacks, but not two calls that overlap
 * on the GPU: its operand buffer is shared.
 *   patdnn_stack_create   handles HOST [n]; pool_after HOST [n] (1 = max-pool after that layer) or NULL
 *   patdnn_stack_run      in DEVICE [N][C0][H0][W0]; out DEVICE, the last layer's (pooled) output; asynchronous
 *   patdnn_stack_run_host the same with HOST buffers; copies in, runs, copies out, waits for the stream
 *   patdnn_stack_submit_host / patdnn_stack_wait_host  the pipelined form of run_host for a stream of batches: submit
 *                         enqueues copy-in (library-owned copy stream), the kernels (caller's stream) and copy-out
 *                         (second copy stream) and returns; wait blocks until the OLDEST submitted batch has landed in
 *                         its out_host.  At most two batches may be in flight (a third submit returns E_STACK);
 *                         in_host must stay untouched until the kernels of its batch ran, i.e. until its wait;
 *                         pinned host memory is needed for the copies to overlap.  All submits of a stack must use
 *                         the same stream.
 *   patdnn_stack_run_timed  patdnn_stack_run with a CUDA event recorded on `stream` in front of every layer's launches
 *                         and one behind the last; waits for the stack and writes the elapsed milliseconds of each
 *                         layer (its kernels as launched inside the stack) to layer_ms, HOST [n].  For reports; the
 *                         events between the launches switch off their overlap, so time whole steps with
 *                         patdnn_stack_run
 *   patdnn_stack_out_shape  N, F, H, W of the stack's output
 *   patdnn_stack_generated  writes to *count how many layers of the stack run code generated for them when the stack
 *                         was created (few-channel first layers; 0 where the run-time compiler is missing or switched
 *                         off, in which case the static kernel runs)
 * Errors: E_NULL, E_STACK, E_CUDA, E_NO_DEVICE.
 */
PATDNN_API int patdnn_stack_create(const patdnn_handle *handles, const int32_t *pool_after, int32_t n, patdnn_stack *out);
PATDNN_API int patdnn_stack_run(patdnn_stack s, const void *in, void *out, void *stream);
PATDNN_API int patdnn_stack_run_timed(patdnn_stack s, const void *in, void *out, void *stream, float *layer_ms);
PATDNN_API int patdnn_stack_run_host(patdnn_stack s, const void *in_host, void *out_host, void *stream);
PATDNN_API int patdnn_stack_submit_host(patdnn_stack s, const void *in_host, void *out_host, void *stream);
PATDNN_API int patdnn_stack_wait_host(patdnn_stack s);
PATDNN_API int patdnn_stack_out_shape(patdnn_stack s, int32_t *N, int32_t *F, int32_t *H, int32_t *W);
PATDNN_API int patdnn_stack_generated(patdnn_stack s, int32_t *count);
PATDNN_API int patdnn_stack_free(patdnn_stack s);

/* patdnn_maxpool2x2 -- 2x2 / stride-2 max-pool (floor) on DEVICE NCHW tensors of the given dtype; asynchronous.
 * Not part of the paper's method; provided so that the VGG-shaped stack runs without any other library. */
PATDNN_API int patdnn_maxpool2x2(const void *in, void *out, int32_t N, int32_t C, int32_t H, int32_t W, int32_t dtype,
                      void *stream);

/* Number of this library's kernels launched by the process since the last reset (addition, for reports). */
PATDNN_API int64_t patdnn_launch_count(void);
PATDNN_API void patdnn_reset_launch_count(void);

/*
 * patdnn_debug_wait (addition; test hook of the failure-detection path) -- every device-side wait of the tensor-core
 * kernels is bounded: after `polls` unsuccessful polls of a barrier (0 = the default, about two seconds) a kernel
 * records a status word, lets all its roles fall through to the common exit, frees its tensor memory and returns;
 * patdnn_check then reports PATDNN_E_DEVICE_TIMEOUT and clears the word.  `skip_load_iteration` > 0 makes the
 * producer of the one-tile-per-CTA kernel leave out the loads of that (1-based) iteration of its channel/tap loop, so
 * that a test can watch a wait run out; 0 restores normal operation.  Applies to later launches of this handle.
 * Errors: E_NULL, E_SHAPE (negative iteration).
 */
PATDNN_API int patdnn_debug_wait(patdnn_handle h, uint32_t polls, int32_t skip_load_iteration);

PATDNN_API const char *patdnn_strerror(int status);
PATDNN_API const char *patdnn_last_cuda_error(void);   /* text of the last CUDA failure seen by this thread ("" if none) */
PATDNN_API const char *patdnn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PATDNN_H */
