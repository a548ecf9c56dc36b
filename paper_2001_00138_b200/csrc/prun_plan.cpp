// Host side of the pattern-run kernel (prun_conv.cu): turns the FKW arrays into per-warp STEP lists.
//
// A warp group is 32 consecutive positions of the filter-kernel reorder (Section 5.2); lane l runs the filter at position
// 32 * group + l.  For every pattern p the group gets a range of steps; in one step every lane processes one of its
// kernels of pattern p (FKW stride[] run, Section 5.3) or a zero-weight padding entry.  A group needs as many steps for
// a pattern as its longest lane -- which is why filters of similar length and pattern mix belong in one warp.  Within a
// step the channels of the lanes are made pairwise different modulo 32 (or equal), so that the per-lane reads of the
// channels' patches in shared memory hit 32 different banks: a greedy assignment, longest remaining lane first.
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <vector>

#include "../../include/patdnn.h"
#include "kernels.hpp"

namespace patdnn {

static int prun_builtin_id(uint16_t mask) {
    for (int i = 0; i < kBuiltinPatterns; ++i)
        if (kBuiltinPatternMasks[i] == mask) return i;
    return -1;
}

bool prun_supported(const Fkw &fkw, int N, int H, int W) {
    if (N < 1 || H < 1 || W < 1 || fkw.P > 32) return false;
    for (uint16_t m : fkw.patterns)
        if (prun_builtin_id(m) < 0) return false;
    const int64_t patch_words = static_cast<int64_t>(fkw.C + 1) * (kPrunTile + 2) * (kPrunTile + 2);
    if (patch_words * 4 > 200 * 1024) return false;               // the whole input tile, all channels, stays in shared memory
    const int64_t tiles = static_cast<int64_t>(N) * ((H + kPrunTile - 1) / kPrunTile) * ((W + kPrunTile - 1) / kPrunTile);
    if (tiles >= (int64_t(1) << 31) || (fkw.F + 511) / 512 > 65535) return false;
    if (static_cast<int64_t>(N) * std::max(fkw.C, fkw.F) * H * W >= (int64_t(1) << 40)) return false;
    return true;
}

int plan_prun(const Fkw &fkw, int N, int H, int W, PrunPlan &pl, PrunLayout &lay) {
    if (!prun_supported(fkw, N, H, W)) return PATDNN_E_SHAPE;
    const int P = fkw.P, F = fkw.F, C = fkw.C;
    constexpr int kPatch = (kPrunTile + 2) * (kPrunTile + 2);
    pl = PrunPlan();
    pl.tiles_x = (W + kPrunTile - 1) / kPrunTile;
    pl.tiles_y = (H + kPrunTile - 1) / kPrunTile;
    pl.groups = (F + 511) / 512;
    pl.groups_per_cta = std::min(kPrunWarps, (F + 31) / 32);
    pl.threads = pl.groups_per_cta * 32;
    pl.smem_bytes = 4 * std::max((C + 1) * kPatch, pl.groups_per_cta * 32 * kPrunTile * kPrunTile);
    const int warp_groups = pl.groups * 16;
    lay.run_ofs.assign(static_cast<size_t>(warp_groups) * (P + 1), 0);
    lay.chan.clear();
    lay.wts.clear();
    int64_t steps = 0;
    std::vector<int> group_steps(warp_groups, 0);
    struct Item { int32_t k, c; };
    std::vector<Item> lists[32];
    for (int g = 0; g < warp_groups; ++g) {
        const int64_t g_first = steps;
        for (int p = 0; p <= P; ++p) {
            lay.run_ofs[static_cast<size_t>(g) * (P + 1) + p] = static_cast<int32_t>(steps);
            if (p == P) break;
            size_t remaining = 0;
            for (int l = 0; l < 32; ++l) {
                lists[l].clear();
                const int pos = g * 32 + l;
                if (pos >= F) continue;
                const int32_t base = fkw.offset[pos];
                const int32_t *st = &fkw.stride[static_cast<size_t>(pos) * (P + 1)];
                for (int32_t k = base + st[p]; k < base + st[p + 1]; ++k) lists[l].push_back({k, fkw.index[k]});
                remaining += lists[l].size();
            }
            while (remaining > 0) {
                // one step: lanes with the most kernels left choose first; a residue class (channel mod 32) may be taken
                // by one channel only
                int order[32];
                for (int l = 0; l < 32; ++l) order[l] = l;
                std::stable_sort(order, order + 32, [&](int a, int b) { return lists[a].size() > lists[b].size(); });
                int32_t owner[32];
                std::fill(owner, owner + 32, -1);
                const size_t at = lay.chan.size();
                constexpr uint32_t kUnset = 0xFFFFFFFFu;
                lay.chan.resize(at + 32, kUnset);
                lay.wts.resize(lay.wts.size() + 4 * 32, 0.f);
                float *w = &lay.wts[(at / 32) * 4 * 32];
                for (int oi = 0; oi < 32; ++oi) {
                    const int l = order[oi];
                    std::vector<Item> &L = lists[l];
                    for (size_t i = 0; i < L.size(); ++i) {
                        const int r = L[i].c & 31;
                        if (owner[r] != -1 && owner[r] != L[i].c) continue;
                        owner[r] = L[i].c;
                        lay.chan[at + l] = static_cast<uint32_t>(L[i].c) * kPatch;
                        for (int j = 0; j < 4; ++j) w[j * 32 + l] = fkw.weight_f32[static_cast<size_t>(L[i].k) * 4 + j];
                        L.erase(L.begin() + static_cast<std::ptrdiff_t>(i));
                        --remaining;
                        break;
                    }
                }
                // padding entries (weights 0) read the patch of a lane that has work in this step: the same address is a
                // broadcast, so they cost no shared-memory bank conflict
                uint32_t any = static_cast<uint32_t>(C) * kPatch;                  // (the zero patch, if a step were empty)
                for (int l = 0; l < 32; ++l)
                    if (lay.chan[at + l] != kUnset) { any = lay.chan[at + l]; break; }
                for (int l = 0; l < 32; ++l)
                    if (lay.chan[at + l] == kUnset) lay.chan[at + l] = any;
                ++steps;
                if (steps >= (int64_t(1) << 30)) return PATDNN_E_SHAPE;
            }
        }
        group_steps[g] = static_cast<int>(steps - g_first);
    }
    // the slowest warp sets the CTA's time
    for (int g = 0; g < warp_groups; ++g) pl.max_warp_steps = std::max(pl.max_warp_steps, group_steps[g]);
    pl.steps = steps;
    pl.entries = steps * 32;
    for (int p = 0; p < P; ++p) pl.builtin[p] = prun_builtin_id(fkw.patterns[p]);
    return PATDNN_OK;
}

}  // namespace patdnn
