// Host planner for the tiled kernel: picks the thread/warp blocking for a layer shape and turns the canonical FKW
// arrays (Section 5.3) into the kernel's private, channel-major entry stream.
//
// Private layout.  Filters are taken in FKR order (Section 5.2) in blocks of FR consecutive positions, so the
// filters one warp register-blocks have (nearly) equal length -- the load-balance use of the filter reorder -- and
// input channels are taken in chunks of CC.  For every (filter block, channel chunk) there is one segment of 32-bit
// records (descriptor plus four weights), sorted by input channel:
//     LOAD(channel)                       fetch that channel's input patch into registers, once for all the
//                                         block's kernels on the channel (filter-level load redundancy elimination,
//                                         Section 5.4)
//     FMA(slot j, pattern p), w0..w3      accumulate kernel (filter slot j, this channel) with the straight-line
//                                         code of pattern p (kernel-level elimination: the patch registers are
//                                         reused by the four taps)
//     END
// Each record is 32 bytes: {w0, w1, w2, w3, descriptor, 0, 0, 0}.
#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include "../../include/patdnn.h"
#include "kernels.hpp"

namespace patdnn {

const uint16_t kBuiltinPatternMasks[kBuiltinPatterns] = {0x01B, 0x036, 0x0D8, 0x1B0, 0x03A, 0x0B8,
                                                         0x09A, 0x0B2, 0x017, 0x1D0, 0x059, 0x134};

static int builtin_id(uint16_t mask) {
    for (int i = 0; i < kBuiltinPatterns; ++i)
        if (kBuiltinPatternMasks[i] == mask) return i;
    return -1;
}

static int row_copy_bytes(int W, int dtype) {
    const int esize = dtype == PATDNN_F16 ? 2 : 4;
    const int row_bytes = W * esize;
    if (row_bytes % 16 == 0) return 16;
    if (row_bytes % 8 == 0) return 8;
    if (row_bytes % 4 == 0) return 4;
    return 0;
}

bool tiled_supported(const Fkw &fkw, int N, int H, int W, int dtype) {
    if (N < 1 || H < 1 || W < 1) return false;
    for (uint16_t m : fkw.patterns)
        if (builtin_id(m) < 0) return false;
    if (row_copy_bytes(W, dtype) == 0) return false;
    if (static_cast<int64_t>(std::max(fkw.C, fkw.F)) * H * W >= (int64_t(1) << 31)) return false;   // 32-bit offsets inside one image
    if (static_cast<int64_t>(N) * (H + 2) >= (int64_t(1) << 31) || static_cast<int64_t>(N) * H * W >= (int64_t(1) << 33)) return false;
    if (W > 1024) return false;
    return true;
}

static void fill_geometry(TiledPlan &pl, const Fkw &fkw, int N, int H, int W, int dtype) {
    const TiledConfig &c = pl.cfg;
    const int esize = dtype == PATDNN_F16 ? 2 : 4;
    pl.TXn = (W + kTileCols - 1) / kTileCols;
    pl.TYn = (H + c.TY - 1) / c.TY;
    pl.tiles_total = N * pl.TYn * pl.TXn;
    pl.lead = 16 / esize;
    const int pitch_bytes = ((pl.lead + kTileCols * pl.TXn) * esize + 15) / 16 * 16;
    pl.pitch = pitch_bytes / esize;
    pl.copy_bytes = row_copy_bytes(W, dtype);
    pl.nchunk = (fkw.C + c.CC - 1) / c.CC;
    pl.nblk = (fkw.F + c.FR - 1) / c.FR;
    const int per_cta = c.PW * 32;
    pl.grid_pix = (pl.tiles_total + per_cta - 1) / per_cta;
    pl.grid_fg = (pl.nblk + c.FW - 1) / c.FW;
    const int tpi = pl.TYn * pl.TXn;
    auto first_row = [&](int t) { return (t / tpi) * (H + 2) + ((t % tpi) / pl.TXn) * c.TY; };
    int rows = 0;
    for (int b = 0; b < pl.grid_pix; ++b) {
        const int t0 = b * per_cta, t1 = std::min(t0 + per_cta, pl.tiles_total) - 1;
        rows = std::max(rows, first_row(t1) + c.TY + 2 - first_row(t0));
    }
    pl.rows_max = rows;
}

static int smem_bytes_for(const TiledPlan &pl, int dtype) {
    const int esize = dtype == PATDNN_F16 ? 2 : 4;
    const int in_stage = pl.cfg.CC * pl.rows_max * pl.pitch * esize + 16;
    const int seg_stage = pl.cfg.FW * pl.seg_cap * 32 + 32;
    const int items = pl.rows_max * (pl.pitch * esize / pl.copy_bytes) * 8;     // per-CTA copy plan
    return pl.cfg.NS * (in_stage + seg_stage) + items;
}

static void build_layout(const Fkw &fkw, TiledPlan &pl, TiledLayout &lay, int dtype) {
    const TiledConfig &c = pl.cfg;
    const int esize = dtype == PATDNN_F16 ? 2 : 4;
    const int nseg = pl.nblk * pl.nchunk;
    struct E { int cc, j, pid; int32_t k; };
    std::vector<std::vector<E>> bucket(nseg);
    std::vector<int> bid(fkw.P);
    for (int p = 0; p < fkw.P; ++p) bid[p] = builtin_id(fkw.patterns[p]);
    for (int i = 0; i < fkw.F; ++i) {
        const int b = i / c.FR, j = i % c.FR;
        for (int32_t k = fkw.offset[i]; k < fkw.offset[i + 1]; ++k) {
            const int ch = fkw.index[k];
            bucket[static_cast<size_t>(b) * pl.nchunk + ch / c.CC].push_back({ch % c.CC, j, bid[fkw.kernel_pid[k]], k});
        }
    }
    const uint32_t code_load = static_cast<uint32_t>(c.FR * kBuiltinPatterns);
    const uint32_t code_end = code_load + 1;
    const uint32_t ch_stride_bytes = static_cast<uint32_t>(pl.rows_max) * pl.pitch * esize;
    lay.rec.clear();
    lay.seg.assign(nseg, 0); lay.seglen.assign(nseg, 0);
    int cap = 0;
    auto push = [&](uint32_t desc, const float *w) {
        uint32_t r[8] = {0, 0, 0, 0, desc, 0, 0, 0};
        if (w) std::memcpy(r, w, 16);
        lay.rec.insert(lay.rec.end(), r, r + 8);
    };
    for (int s = 0; s < nseg; ++s) {
        std::vector<E> &v = bucket[s];
        std::sort(v.begin(), v.end(), [](const E &a, const E &b) { return a.cc != b.cc ? a.cc < b.cc : a.j < b.j; });
        const size_t start = lay.rec.size() / 8;
        lay.seg[s] = static_cast<int32_t>(start);
        int cur = -1;
        for (const E &e : v) {
            if (e.cc != cur) {
                cur = e.cc;
                push(code_load | ((static_cast<uint32_t>(cur) * ch_stride_bytes) << 10), nullptr);
            }
            push(static_cast<uint32_t>(e.j * kBuiltinPatterns + e.pid), &fkw.weight_f32[static_cast<size_t>(e.k) * 4]);
        }
        push(code_end, nullptr);
        lay.seglen[s] = static_cast<int32_t>(lay.rec.size() / 8 - start);
        cap = std::max(cap, lay.seglen[s]);
    }
    pl.seg_cap = cap;
    pl.entries = static_cast<int64_t>(lay.rec.size() / 8);
}

int plan_tiled(const Fkw &fkw, int N, int H, int W, int dtype, TiledPlan &plan, TiledLayout &layout) {
    if (!tiled_supported(fkw, N, H, W, dtype)) return PATDNN_E_SHAPE;
    // Blocking choice: (rows per thread, filters per warp).  The override is for tuning runs and tests.
    TiledConfig cfg{};
    int ty = 4, fr = 4;
    if (H < 4 || (H % 4 != 0 && H < 16)) { ty = 2; fr = 8; }
    char ov[16];
    if (debug_option_text("tile", ov, sizeof ov)) {            // "TYxFR", e.g. 4x4
        int a = 0, b = 0;
        if (std::sscanf(ov, "%dx%d", &a, &b) == 2 &&
            ((a == 4 && b == 8) || (a == 4 && b == 4) || (a == 2 && b == 8))) {
            ty = a; fr = b;
        }
    }
    cfg.TY = ty; cfg.FR = fr;
    cfg.MINB = (ty * fr * 4 <= 64) ? 2 : 1;
    cfg.PW = 2;
    cfg.FW = 4;
    cfg.NS = 2;
    const int64_t tiles = static_cast<int64_t>(N) * ((H + cfg.TY - 1) / cfg.TY) * ((W + 3) / 4);
    if (tiles <= 32) cfg.PW = 1;
    const int nblk0 = (fkw.F + cfg.FR - 1) / cfg.FR;
    cfg.FW = nblk0 >= 3 ? 4 : (nblk0 == 2 ? 2 : 1);
    const int kMaxSmem = (cfg.MINB == 2 ? 100 : 200) * 1024;
    for (int cc : {8, 4, 2, 1}) {
        cfg.CC = std::min(cc, fkw.C);
        plan = TiledPlan();
        plan.cfg = cfg;
        fill_geometry(plan, fkw, N, H, W, dtype);
        plan.seg_cap = (cfg.FR + 1) * cfg.CC + 1;                    // upper bound before the layout exists
        if (smem_bytes_for(plan, dtype) <= kMaxSmem || cc == 1) break;
    }
    build_layout(fkw, plan, layout, dtype);
    plan.smem_bytes = smem_bytes_for(plan, dtype);
    if (plan.smem_bytes > 224 * 1024) return PATDNN_E_SHAPE;
    return PATDNN_OK;
}

}  // namespace patdnn
