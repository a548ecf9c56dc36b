// Several consecutive tensor-core layers of a stack in ONE persistent kernel, for small batches.
//
// At batch 1 a VGG-shaped layer has a handful of 128-pixel tiles: as one kernel per layer every layer pays a launch,
// a pipeline fill, a cluster exchange and a drain, and thread-block clusters cap the split of the channel/tap loop at
// eight CTAs, which leaves most SMs idle on the deepest layers.  Here one cooperative launch keeps one CTA per SM
// resident for the whole run of layers.  (Opt-in: measured no faster than one kernel per layer, see patdnn_stack_create.)
// Per layer:
//   phase A  the (tile, iteration) space of the layer -- tiles of 128 pixels x 128 filters, 9 * C/64 iterations each -- is
//            cut into gridDim.x equal contiguous chunks, one per CTA, whatever the tile boundaries (a chunk touches at
//            most two tiles); a CTA multiplies its chunk exactly like the one-tile-per-CTA kernel (TMA producer warp, one
//            MMA-issuing thread, TMEM accumulator, double buffered) and writes each partial tile as fp32 to a scratch
//            slot in global memory (L2-resident);
//   grid barrier
//   phase B  all CTAs share the reduction: a thread sums the partial tiles of one pixel and eight filters in CTA
//            order (deterministic), adds bias, applies ReLU and the 2x2 max-pool where one follows, and writes either the
//            next layer's split, channels-innermost operands or the final NCHW tensor;
//   grid barrier (then the producer warps may read what phase B wrote).
// The weights of the next layer do not depend on the barrier: a producer warp fetches the first ring slots' weight
// tiles of its next chunk while its CTA is still reducing.
//
// Every wait is bounded -- mbarrier waits as in the other kernels, the grid barrier by the same polling budget -- and a
// wait that runs out records a status word, after which every role of every CTA falls through to the common exit.
// The launch is cooperative, so all CTAs are resident together; no clusters, every CTA loads its own operands.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>

#include "../../include/patdnn.h"
#include "kernels.hpp"
#include "umma_ptx.cuh"

namespace patdnn {

namespace {

constexpr int kChainThreads = 320;           // TMA warp, MMA warp, eight epilogue / reduction warps
constexpr int kBN = 128;                     // filters per tile
constexpr int kSlotFloats = kTileM * kBN;    // one partial tile

__device__ __forceinline__ unsigned long long ld_acquire_gpu(const unsigned long long *p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float4 ld_cg_f4(const float *p) {     // L2 only: the line may be stale in this SM's L1
    float4 v;
    asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
    return v;
}

// Barrier over all CTAs of a cooperative launch; called by ONE thread per CTA.  *bar counts arrivals and only ever
// grows: between launches it is a multiple of the grid size, so the value a CTA reads before its own first arrival,
// rounded down to that multiple, is the same base for every CTA; barrier k of a launch is passed once the count
// reaches base + k * nblocks.  One release-add to arrive, bounded acquire-polling to wait.
__device__ bool grid_barrier(unsigned long long *bar, unsigned long long &target, unsigned nblocks, const WaitCtx &w, int code) {
    target += nblocks;
    asm volatile("red.release.gpu.global.add.u64 [%0], 1;" ::"l"(bar) : "memory");
    for (uint32_t i = 0; i < w.limit; ++i) {
        if (ld_acquire_gpu(bar) >= target) return true;
        if ((i & 15u) == 15u && *reinterpret_cast<volatile int *>(w.word) != 0) return false;
    }
    atomicCAS(w.word, 0, code);
    return false;
}

struct TilePos { int ft, x0, y0, n0; };

__device__ __forceinline__ TilePos decode_tile(const ChainLayer &L, int tile) {
    TilePos t;
    t.ft = tile % L.n_ftiles; tile /= L.n_ftiles;
    const int tix = tile % L.tiles_x; tile /= L.tiles_x;
    const int tiy = tile % L.tiles_y; tile /= L.tiles_y;
    t.x0 = tix * L.TW; t.y0 = tiy * L.TH; t.n0 = tile * L.TN;
    return t;
}

// First iteration of CTA `cta`'s chunk of a layer: the layer's `total` iterations are cut into L.gw equal contiguous
// chunks (gw = min(grid, total): no chunk is empty); CTAs from gw on have no work in this layer.  cta * total < 2^31.
__device__ __forceinline__ int chunk_begin(const ChainLayer &L, int cta) {
    return cta >= L.gw ? L.total : cta * L.total / L.gw;
}

// Phase B for one layer: see the file header.
// The partial tile of CTA c for tile t sits in slot c + t (chunks are contiguous and ordered, so the slots of one tile
// are consecutive): a plain strided loop over the tile's K contributors, unrolled so that several loads are in flight.
template <int ROWS>
__device__ __forceinline__ void sum_partials(const float *base, int K, const int (&rows)[4], int g, float (&acc)[ROWS][8]) {
#pragma unroll
    for (int a = 0; a < ROWS; ++a)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[a][j] = 0.f;
    constexpr int UB = 8 / ROWS;                                  // contributors whose loads are issued together
    for (int k0 = 0; k0 < K; k0 += UB) {
        float4 lo4[UB][ROWS], hi4[UB][ROWS];
#pragma unroll
        for (int k = 0; k < UB; ++k) {
            const float *slot = base + static_cast<size_t>(k0 + k) * kSlotFloats;
#pragma unroll
            for (int a = 0; a < ROWS; ++a) {
                if (k0 + k < K) {
                    lo4[k][a] = ld_cg_f4(slot + (static_cast<size_t>(2 * g) * kTileM + rows[a]) * 4);
                    hi4[k][a] = ld_cg_f4(slot + (static_cast<size_t>(2 * g + 1) * kTileM + rows[a]) * 4);
                } else {
                    lo4[k][a] = make_float4(0.f, 0.f, 0.f, 0.f);
                    hi4[k][a] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
#pragma unroll
        for (int k = 0; k < UB; ++k)                              // in contributor order: the sum is deterministic
#pragma unroll
            for (int a = 0; a < ROWS; ++a) {
                acc[a][0] += lo4[k][a].x; acc[a][1] += lo4[k][a].y; acc[a][2] += lo4[k][a].z; acc[a][3] += lo4[k][a].w;
                acc[a][4] += hi4[k][a].x; acc[a][5] += hi4[k][a].y; acc[a][6] += hi4[k][a].z; acc[a][7] += hi4[k][a].w;
            }
    }
}

// Finish eight consecutive filters (f_lo ..) of one output pixel (n, y, x of the oh x ow output): bias, ReLU, store.
template <typename T>
__device__ __forceinline__ void chain_emit(const ChainLayer &L, float (&v)[8], int f_lo, int n, int y, int x, int oh, int ow) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int f = f_lo + j;
        float sv = v[j] + ((f < L.F) ? __ldg(L.bias + f) : 0.f);
        if (L.relu) sv = fmaxf(sv, 0.f);
        v[j] = (f < L.F) ? sv : 0.f;
    }
    if (L.out_mode == 0) {
        T *out = static_cast<T *>(L.out);
        const size_t plane = static_cast<size_t>(oh) * ow;
        const size_t obase = static_cast<size_t>(n) * L.F * plane + static_cast<size_t>(y) * ow + x;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int f = f_lo + j;
            if (f < L.F) {
                if constexpr (sizeof(T) == 2) out[obase + f * plane] = __float2half_rn(v[j]);
                else out[obase + f * plane] = v[j];
            }
        }
    } else {
        if (f_lo >= L.out_cp) return;                             // filter tiles may be padded beyond the next layer's channels
        uint16_t *dst = static_cast<uint16_t *>(L.out);
        const size_t o = ((static_cast<size_t>(n) * oh + y) * ow + x) * L.out_cp + f_lo;
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float a = v[2 * j], b = v[2 * j + 1];
            if constexpr (sizeof(T) == 2) {
                hi[j] = static_cast<uint32_t>(__half_as_ushort(__float2half_rn(a))) |
                        (static_cast<uint32_t>(__half_as_ushort(__float2half_rn(b))) << 16);
                lo[j] = 0;
            } else {
                const __nv_bfloat16 ah = __float2bfloat16_rn(a), bh = __float2bfloat16_rn(b);
                const __nv_bfloat16 al = __float2bfloat16_rn(a - __bfloat162float(ah));
                const __nv_bfloat16 bl = __float2bfloat16_rn(b - __bfloat162float(bh));
                hi[j] = static_cast<uint32_t>(__bfloat16_as_ushort(ah)) | (static_cast<uint32_t>(__bfloat16_as_ushort(bh)) << 16);
                lo[j] = static_cast<uint32_t>(__bfloat16_as_ushort(al)) | (static_cast<uint32_t>(__bfloat16_as_ushort(bl)) << 16);
            }
        }
        *reinterpret_cast<uint4 *>(dst + o) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        if constexpr (sizeof(T) != 2) {
            const size_t plane_out = static_cast<size_t>(L.N) * oh * ow * L.out_cp;
            *reinterpret_cast<uint4 *>(dst + plane_out + o) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
    }
}

// A job is one warp's work: one tile, one group of eight filters and a block of 32 or 64 pixel rows, one or two rows per
// lane (the finer split where the layer has few jobs); behind a pool, all pooled pixels of the tile (at most 32), one
// per lane.  Job j belongs to CTA j % grid, so that every CTA gets work before any gets a second job.  et = 0..255.
template <int ROWS, typename T>
__device__ __forceinline__ void reduce_rows(const ChainLayer &L, const TilePos &tp, const float *base, int K, int g, int f_lo,
                                            int row0, int oh, int ow) {
    const int rows[4] = {row0, row0 + 32, row0, row0};
    float acc[ROWS][8];
    sum_partials<ROWS>(base, K, rows, g, acc);                    // rows beyond the box hold stale sums: never stored
    const int rows_img = L.TW * L.TH;
#pragma unroll
    for (int a = 0; a < ROWS; ++a) {
        const int r = rows[a];
        const int tn = r / rows_img, rem = r - tn * rows_img, ty = rem / L.TW, tx = rem - ty * L.TW;
        const int n = tp.n0 + tn, y = tp.y0 + ty, x = tp.x0 + tx;
        if (tn >= L.TN || n >= L.N || y >= L.H || x >= L.W) continue;
        chain_emit<T>(L, acc[a], f_lo, n, y, x, oh, ow);
    }
}

template <int TERMS, typename T>
__device__ void chain_reduce(const ChainParams &p, const ChainLayer &L, int cta, int G, int et) {
    const int lane = et & 31, wslot = et >> 5;                   // eight reduction warps per CTA
    const int oh = L.pool ? L.H / 2 : L.H, ow = L.pool ? L.W / 2 : L.W;
    const int cg_jobs = L.n_tiles * (kBN / 8);                    // (tile, filter group) pairs
    const int two_rows = !L.pool && cg_jobs * 2 >= G * 8;         // enough jobs for every warp with 64-row blocks?
    const int blocks = L.pool ? 1 : (two_rows ? 2 : 4);           // row blocks per (tile, filter group)
    const int njobs = cg_jobs * blocks;
    for (int job = cta + G * wslot; job < njobs; job += G * 8) {
        const int rb = job % blocks, cgj = job / blocks;
        const int g = cgj % (kBN / 8), tile = cgj / (kBN / 8);
        const TilePos tp = decode_tile(L, tile);
        // CTAs c0 .. c1 hold the chunks that meet this tile's iterations [t0, t0 + ipt)
        const int t0 = tile * L.ipt, tl = t0 + L.ipt - 1;
        int c0 = t0 * L.gw / L.total;                             // t0 * gw < total * grid < 2^31
        while (c0 + 1 < L.gw && chunk_begin(L, c0 + 1) <= t0) ++c0;
        while (c0 > 0 && chunk_begin(L, c0) > t0) --c0;
        int c1 = tl * L.gw / L.total;
        while (c1 + 1 < L.gw && chunk_begin(L, c1 + 1) <= tl) ++c1;
        while (c1 > 0 && chunk_begin(L, c1) > tl) --c1;
        const float *base = p.partial + static_cast<size_t>(c0 + tile) * kSlotFloats;
        const int K = c1 - c0 + 1;
        const int f_lo = tp.ft * kBN + 8 * g;
        if (L.pool) {
            const int pw = L.TW / 2, per = pw * (L.TH / 2), R = per * L.TN;
            for (int r = lane; r < R; r += 32) {
                const int tn = r / per, rem = r - tn * per, py = rem / pw, px = rem - py * pw;
                const int m00 = (tn * L.TH + 2 * py) * L.TW + 2 * px;
                const int rows[4] = {m00, m00 + 1, m00 + L.TW, m00 + L.TW + 1};
                const int n = tp.n0 + tn, y = tp.y0 + 2 * py, x = tp.x0 + 2 * px;
                if (n >= L.N || y + 1 >= L.H || x + 1 >= L.W) continue;
                float acc[4][8], v[8];
                sum_partials<4>(base, K, rows, g, acc);
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = fmaxf(fmaxf(acc[0][j], acc[1][j]), fmaxf(acc[2][j], acc[3][j]));   // max commutes with bias + ReLU
                chain_emit<T>(L, v, f_lo, n, y >> 1, x >> 1, oh, ow);
            }
        } else if (two_rows) {
            reduce_rows<2, T>(L, tp, base, K, g, f_lo, rb * 64 + lane, oh, ow);
        } else {
            reduce_rows<1, T>(L, tp, base, K, g, f_lo, rb * 32 + lane, oh, ow);
        }
    }
}

template <int TERMS, typename T>
__global__ void __launch_bounds__(kChainThreads, 1) conv_chain_kernel(const __grid_constant__ ChainParams p) {
    constexpr int S = (TERMS == 3) ? 2 : 1;
    constexpr int A_BYTES = kTileM * 128;
    constexpr int B_BYTES = kBN * 128;
    constexpr int STAGE_BYTES = S * (A_BYTES + B_BYTES);
    constexpr bool MERGE = (TERMS == 3);                          // x_hi * [w_hi | w_lo] as one MMA of width 2 * kBN
    constexpr int ACC_COLS = MERGE ? 2 * kBN : kBN;
    constexpr int TMEM_COLS = 2 * ACC_COLS;                       // two accumulator buffers
    extern __shared__ unsigned char smem_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ __align__(8) uint64_t bars[8 + 8 + 2 + 2 + 1];     // full, empty (ring); accumulator full, empty; layer ready
    __shared__ uint32_t tmem_slot;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = gridDim.x, cta = blockIdx.x;
    const int stages = p.stages;
    const uint32_t bar_full = smem_u32(&bars[0]), bar_empty = smem_u32(&bars[8]), bar_af = smem_u32(&bars[16]),
                   bar_ae = smem_u32(&bars[18]), bar_ready = smem_u32(&bars[20]);
    const WaitCtx status{p.status, p.spin_limit ? p.spin_limit : kSpinLimit};

    if (threadIdx.x == 0) {
        for (int s = 0; s < 8; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_af, 1); mbar_init(bar_af + 8, 1);
        mbar_init(bar_ae, 8); mbar_init(bar_ae + 8, 8);           // one arrival per epilogue warp
        mbar_init(bar_ready, 1);
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
    pdl_wait();

    if (warp == 0) {
        if (lane == 0) {
            uint32_t cnt = 0;                                     // ring uses so far, over all layers
            bool ok = true;
            for (int l = 0; l < p.n_layers && ok; ++l) {
                const ChainLayer &L = p.layer[l];
                const int beg = chunk_begin(L, cta), n = chunk_begin(L, cta + 1) - beg;
                const uint32_t tx_bytes = S * (L.box_bytes + B_BYTES);
                const int npre = n < stages ? n : stages;
                // (tile, channel block, tap) of an iteration and its tile's coordinates, advanced without divisions
                struct Cursor { int cb, tap, f0, x0, y0, n0; uint32_t s, use; };
                auto cursor_at = [&](int it, uint32_t c) {
                    Cursor q;
                    const int tile = it / L.ipt, k = it - tile * L.ipt;
                    q.cb = k / 9; q.tap = k - 9 * q.cb;
                    const TilePos tp = decode_tile(L, tile);
                    q.f0 = tp.ft * kBN; q.x0 = tp.x0; q.y0 = tp.y0; q.n0 = tp.n0;
                    q.s = c % stages; q.use = c / stages;
                    return q;
                };
                auto advance = [&](Cursor &q) {
                    if (++q.s == static_cast<uint32_t>(stages)) { q.s = 0; ++q.use; }
                    if (++q.tap < 9) return;
                    q.tap = 0;
                    if (++q.cb < L.KB) return;
                    q.cb = 0;                                      // next tile: filter tile fastest, then x, y, images
                    q.f0 += kBN;
                    if (q.f0 < L.n_ftiles * kBN) return;
                    q.f0 = 0; q.x0 += L.TW;
                    if (q.x0 < L.tiles_x * L.TW) return;
                    q.x0 = 0; q.y0 += L.TH;
                    if (q.y0 < L.tiles_y * L.TH) return;
                    q.y0 = 0; q.n0 += L.TN;
                };
                auto load_b = [&](const Cursor &q) {              // waits for the slot, arms it and fetches its weight tile
                    if (q.use > 0 && !mbar_wait(bar_empty + 8 * q.s, (q.use - 1) & 1, status, 1)) return false;
                    const uint32_t base = smem_u32(smem + static_cast<size_t>(q.s) * STAGE_BYTES);
                    mbar_expect_tx(bar_full + 8 * q.s, tx_bytes);
#pragma unroll
                    for (int sp = 0; sp < S; ++sp)
                        tma_load_4d(base + S * A_BYTES + sp * B_BYTES, &p.mapB[l], bar_full + 8 * q.s, q.cb * kKBlock, q.f0, q.tap, sp);
                    return true;
                };
                auto load_a = [&](const Cursor &q) {
                    const int r = q.tap / 3, sx = q.tap - 3 * r;
                    const uint32_t base = smem_u32(smem + static_cast<size_t>(q.s) * STAGE_BYTES);
#pragma unroll
                    for (int sp = 0; sp < S; ++sp)
                        tma_load_5d(base + sp * A_BYTES, &p.mapA[l], bar_full + 8 * q.s, q.cb * kKBlock, q.x0 + sx - 1, q.y0 + r - 1, q.n0, sp);
                };
                Cursor qb = cursor_at(beg, cnt), qa = qb;
                // the weights do not depend on the previous layer: first ring slots before the layer barrier
                for (int j = 0; j < npre && ok; ++j) {
                    ok = load_b(qb);
                    advance(qb);
                }
                if (!ok) break;
                if (l > 0) {
                    ok = mbar_wait(bar_ready, (l - 1) & 1, status, 1);
                    if (!ok) break;
                    asm volatile("fence.proxy.async.global;" ::: "memory");   // phase-B stores (generic proxy) -> TMA reads
                }
                for (int j = 0; j < n && ok; ++j) {
                    if (j >= npre) {
                        ok = load_b(qb);
                        if (!ok) break;
                        advance(qb);
                    }
                    if (!(l == 0 && j + 1 == p.test_skip_load)) load_a(qa);   // test hook: those loads never arrive
                    advance(qa);
                }
                cnt += n;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(TERMS == 3 ? 1 : 0, kBN);
            constexpr uint32_t idesc2 = instr_desc(1, MERGE ? 2 * kBN : kBN);
            uint32_t cnt = 0, seg = 0;
            bool ok = true;
            for (int l = 0; l < p.n_layers && ok; ++l) {
                const ChainLayer &L = p.layer[l];
                int it = chunk_begin(L, cta);
                const int end = chunk_begin(L, cta + 1);
                while (it < end && ok) {
                    const int tile = it / L.ipt;
                    const int seg_end = min(end, (tile + 1) * L.ipt);
                    const uint32_t buf = seg & 1u;
                    if (seg >= 2 && !mbar_wait(bar_ae + 8 * buf, ((seg >> 1) - 1) & 1, status, 2)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t acc = tmem_base + buf * ACC_COLS;
                    bool first = true;
                    for (; it < seg_end; ++it, ++cnt) {
                        const uint32_t s = cnt % stages;
                        ok = mbar_wait(bar_full + 8 * s, (cnt / stages) & 1, status, 2);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t base = smem_u32(smem + static_cast<size_t>(s) * STAGE_BYTES);
                        const uint64_t a_hi = smem_desc_sw128(base), a_lo = smem_desc_sw128(base + A_BYTES);
                        const uint64_t b_hi = smem_desc_sw128(base + S * A_BYTES);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {             // 4 x K=16 inside the 128-byte swizzle row: +32 bytes
                            const uint64_t koff = static_cast<uint64_t>(2 * k);
                            if constexpr (MERGE) {
                                umma_f16(acc, a_hi + koff, b_hi + koff, idesc2, (first && k == 0) ? 0u : 1u);
                                umma_f16(acc, a_lo + koff, b_hi + koff, idesc, 1u);
                            } else {
                                umma_f16(acc, a_hi + koff, b_hi + koff, idesc, (first && k == 0) ? 0u : 1u);
                            }
                        }
                        first = false;
                        umma_commit(bar_empty + 8 * s);
                    }
                    if (ok) umma_commit(bar_af + 8 * buf);
                    ++seg;
                }
            }
        }
    } else {
        // epilogue / reduction warps: warp w owns TMEM lanes 32*(w%4) .. +31 and one half of the filter columns
        const int q = warp & 3, half = (warp - 2) >> 2;
        const int m = q * 32 + lane;
        const int et = threadIdx.x - 64;
        unsigned long long target = 0;                           // arrivals that complete this CTA's next barrier
        if (et == 0) target = ld_acquire_gpu(p.bar) / G * G;      // read before this CTA's first arrival: see grid_barrier
        uint32_t seg = 0;
        bool dead = false;                                        // a wait ran out somewhere: keep meeting the barriers, skip the work
        for (int l = 0; l < p.n_layers; ++l) {
            const ChainLayer &L = p.layer[l];
            int it = chunk_begin(L, cta);
            const int end = chunk_begin(L, cta + 1);
            while (it < end) {
                const int tile = it / L.ipt;
                const int seg_end = min(end, (tile + 1) * L.ipt);
                const uint32_t buf = seg & 1u;
                if (!dead && !mbar_wait(bar_af + 8 * buf, (seg >> 1) & 1, status, 3)) dead = true;
                dead = __any_sync(0xffffffffu, dead);            // warp-uniform: the TMEM loads below are warp-wide
                if (!dead) {
                    tc_fence_after();
                    float *slot = p.partial + static_cast<size_t>(cta + tile) * kSlotFloats;
#pragma unroll 1
                    for (int c0 = half * (kBN / 2); c0 < (half + 1) * (kBN / 2); c0 += 32) {
                        uint32_t v[32];
                        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * ACC_COLS + c0;
                        tmem_ld32(taddr, v);
                        float a[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) a[j] = __uint_as_float(v[j]);
                        if constexpr (MERGE) {
                            tmem_ld32(taddr + kBN, v);
#pragma unroll
                            for (int j = 0; j < 32; ++j) a[j] += __uint_as_float(v[j]);
                        }
                        // slot layout [column quad][pixel][4 columns]: a warp's 16-byte stores are 512 contiguous bytes
#pragma unroll
                        for (int j4 = 0; j4 < 8; ++j4)
                            *reinterpret_cast<float4 *>(slot + (static_cast<size_t>(c0 / 4 + j4) * kTileM + m) * 4) =
                                make_float4(a[4 * j4], a[4 * j4 + 1], a[4 * j4 + 2], a[4 * j4 + 3]);
                    }
                    tc_fence_before();
                }
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_ae + 8 * buf) : "memory");
                ++seg;
                it = seg_end;
            }
            // every partial tile of the layer is in memory before anyone reduces
            __threadfence();
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (et == 0) grid_barrier(p.bar, target, G, status, 4);
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (*reinterpret_cast<volatile int *>(p.status) != 0) dead = true;
            if (!dead) chain_reduce<TERMS, T>(p, L, cta, G, et);
            if (l + 1 < p.n_layers) {
                asm volatile("fence.proxy.async.global;" ::: "memory");   // these stores are read through TMA next
                __threadfence();
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (et == 0) {
                    grid_barrier(p.bar, target, G, status, 5);
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_ready) : "memory");   // wakes the producer warp
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

template <int TERMS, typename T>
cudaError_t chain_launch_t(const ChainParams &p, int grid, int smem, cudaStream_t st, bool prep, int *max_blocks) {
    auto kern = conv_chain_kernel<TERMS, T>;
    if (prep) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        return cudaOccupancyMaxActiveBlocksPerMultiprocessor(max_blocks, kern, kChainThreads, smem);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kChainThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;                  // all CTAs resident together, or the launch fails
    attr[0].val.cooperative = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, p);
}

}  // namespace

// Pixel box (TW x TH x TN <= 128 pixels) that wastes the fewest MMA rows; with a pool behind the layer the 2x2 windows
// must not straddle boxes (even extents, even box sizes).
bool chain_box(int N, int H, int W, bool pool, ChainLayer &L) {
    if (pool && ((H & 1) || (W & 1))) return false;
    double best = -1;
    for (int tw = 1; tw <= std::min(W, kTileM); ++tw) {
        const int th = std::min(H, kTileM / tw);
        const int tn = (th == H) ? std::max(1, std::min(N, kTileM / (tw * th))) : 1;
        if (tw > 256 || th > 256 || tn > 256) continue;
        if (pool && ((tw & 1) || (th & 1))) continue;
        const int64_t tx = (W + tw - 1) / tw, ty = (H + th - 1) / th, tz = (N + tn - 1) / tn;
        const double util = static_cast<double>(N) * H * W / (static_cast<double>(tx * ty * tz) * kTileM);
        const double score = util + 1e-6 * tw;
        if (score > best) {
            best = score;
            L.TW = tw; L.TH = th; L.TN = tn; L.tiles_x = static_cast<int>(tx); L.tiles_y = static_cast<int>(ty); L.tiles_n = static_cast<int>(tz);
        }
    }
    return best > 0;
}

int chain_stages(int dtype) {
    const int S = dtype == PATDNN_F16 ? 1 : 2;
    const int stage = S * (kTileM * 128 + kBN * 128);
    const int want = debug_option("chain_stages", 0);
    if (want >= 2 && want <= 8 && want * stage <= 200 * 1024) return want;
    return std::max(2, std::min(8, (200 * 1024) / stage));
}

int chain_smem_bytes(int dtype) {
    const int S = dtype == PATDNN_F16 ? 1 : 2;
    return chain_stages(dtype) * S * (kTileM * 128 + kBN * 128) + 1024;
}

size_t chain_partial_bytes(int grid) { return static_cast<size_t>(grid) * 2 * kSlotFloats * sizeof(float); }

// CTAs of the cooperative launch: one per SM, if the kernel fits an SM and the device launches cooperatively; else 0.
int chain_grid(int dtype) {
    int dev = 0, coop = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) {
        cudaGetLastError();
        return 0;
    }
    int nb = 0;
    ChainParams dummy{};
    const cudaError_t e = dtype == PATDNN_F16 ? chain_launch_t<1, __half>(dummy, 0, chain_smem_bytes(dtype), nullptr, true, &nb)
                                              : chain_launch_t<3, float>(dummy, 0, chain_smem_bytes(dtype), nullptr, true, &nb);
    if (e != cudaSuccess || nb < 1) { cudaGetLastError(); return 0; }
    return sm_count();
}

cudaError_t chain_launch(const ChainParams &p, int grid, int dtype, cudaStream_t st) {
    return dtype == PATDNN_F16 ? chain_launch_t<1, __half>(p, grid, chain_smem_bytes(dtype), st, false, nullptr)
                               : chain_launch_t<3, float>(p, grid, chain_smem_bytes(dtype), st, false, nullptr);
}

}  // namespace patdnn
