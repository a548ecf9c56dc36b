// Host-side filter-kernel reorder (Section 5.2) and FKW compressed weight storage (Section 5.3).
//
// Input contract (Section 4.2, Eq. 1): every kernel's 3x3 mask is either empty (connectivity-pruned) or equal to
// one pattern of the set.  Output: the five arrays offset / reorder / index / stride / weight.
//   kernel reorder : inside a filter, kept kernels sorted by (pattern id, input channel);
//   filter reorder : filters grouped by ascending length (number of kept kernels); inside a group a greedy chain
//                    that starts at the smallest original id and appends the unplaced filter with the largest
//                    similarity to the last one (ties: smallest id).  Similarity of two equal-length filters is the
//                    number of positions with the same pattern id once both are sorted by pattern id.
#include "fkw_encoder.hpp"

#include <algorithm>
#include <cstring>
#include <map>
#include <numeric>

#include "../../include/patdnn.h"

namespace patdnn {

uint16_t float_to_half_rne(float f) {
    uint32_t x;
    std::memcpy(&x, &f, 4);
    const uint32_t sign = (x >> 16) & 0x8000u;
    const uint32_t absx = x & 0x7fffffffu;
    if (absx >= 0x7f800000u) {                                   // inf / nan
        return static_cast<uint16_t>(sign | 0x7c00u | ((absx > 0x7f800000u) ? (0x200u | ((absx >> 13) & 0x3ffu)) : 0u));
    }
    if (absx >= 0x477ff000u) return static_cast<uint16_t>(sign | 0x7c00u);   // rounds to >= 65520 -> inf
    if (absx < 0x33000001u) return static_cast<uint16_t>(sign);               // below half of the smallest subnormal
    int32_t exp = static_cast<int32_t>(absx >> 23) - 127;
    uint32_t man = (absx & 0x7fffffu) | 0x800000u;                            // 24-bit significand
    int shift;
    uint32_t base;
    if (exp < -14) {                                                          // subnormal half
        shift = 13 + (-14 - exp);
        base = 0;
    } else {
        shift = 13;
        base = static_cast<uint32_t>(exp + 15) << 10;
        man &= 0x7fffffu;
    }
    uint32_t q = man >> shift;
    const uint32_t rem = man & ((1u << shift) - 1u);
    const uint32_t half = 1u << (shift - 1);
    if (rem > half || (rem == half && (q & 1u))) ++q;                         // round to nearest even
    return static_cast<uint16_t>(sign | (base + q));                          // a carry out of q bumps the exponent
}

float half_to_float(uint16_t h) {
    const uint32_t sign = static_cast<uint32_t>(h & 0x8000u) << 16;
    uint32_t exp = (h >> 10) & 0x1fu;
    uint32_t man = h & 0x3ffu;
    uint32_t x;
    if (exp == 0) {
        if (man == 0) {
            x = sign;
        } else {
            int e = -1;
            do { ++e; man <<= 1; } while (!(man & 0x400u));
            x = sign | (static_cast<uint32_t>(127 - 15 - e) << 23) | ((man & 0x3ffu) << 13);
        }
    } else if (exp == 31) {
        x = sign | 0x7f800000u | (man << 13);
    } else {
        x = sign | ((exp + 127 - 15) << 23) | (man << 13);
    }
    float f;
    std::memcpy(&f, &x, 4);
    return f;
}

int validate_pattern_set(const uint16_t *pattern_set, int32_t n_patterns) {
    if (!pattern_set) return PATDNN_E_NULL;
    if (n_patterns < 1 || n_patterns > 32) return PATDNN_E_PATTERN_SET;
    for (int i = 0; i < n_patterns; ++i) {
        const uint32_t m = pattern_set[i];
        if (m >= 512u || __builtin_popcount(m) != 4) return PATDNN_E_PATTERN_SET;
        for (int j = 0; j < i; ++j)
            if (pattern_set[j] == m) return PATDNN_E_PATTERN_SET;
    }
    return PATDNN_OK;
}

int classify_kernels(const uint8_t *mask, const uint16_t *pattern_set, int32_t P, int32_t F, int32_t C,
                     std::vector<int32_t> &pid) {
    int16_t id_of_mask[512];
    std::fill(id_of_mask, id_of_mask + 512, int16_t(-1));
    for (int p = 0; p < P; ++p) id_of_mask[pattern_set[p]] = static_cast<int16_t>(p);
    pid.assign(static_cast<size_t>(F) * C, -1);
    for (size_t k = 0; k < static_cast<size_t>(F) * C; ++k) {
        uint32_t bits = 0;
        for (int t = 0; t < 9; ++t) {
            const uint8_t v = mask[k * 9 + t];
            if (v > 1) return PATDNN_E_MASK;
            bits |= static_cast<uint32_t>(v) << t;
        }
        if (bits == 0) continue;
        if (id_of_mask[bits] < 0) return PATDNN_E_MASK;
        pid[k] = id_of_mask[bits];
    }
    return PATDNN_OK;
}

void filter_reorder(const std::vector<int32_t> &pid, int32_t P, int32_t F, int32_t C, std::vector<int32_t> &order) {
    // cum[f][p] = number of kept kernels of filter f with pattern id < p (exclusive prefix sums of the histogram).
    std::vector<int32_t> cum(static_cast<size_t>(F) * (P + 1), 0);
    for (int f = 0; f < F; ++f) {
        int32_t *row = &cum[static_cast<size_t>(f) * (P + 1)];
        for (int c = 0; c < C; ++c) {
            const int32_t p = pid[static_cast<size_t>(f) * C + c];
            if (p >= 0) ++row[p + 1];
        }
        for (int p = 0; p < P; ++p) row[p + 1] += row[p];
    }
    std::map<int32_t, std::vector<int32_t>> groups;               // length -> filters in ascending id
    for (int f = 0; f < F; ++f) groups[cum[static_cast<size_t>(f) * (P + 1) + P]].push_back(f);
    order.clear();
    order.reserve(F);
    for (auto &kv : groups) {
        std::vector<int32_t> &g = kv.second;
        std::vector<char> placed(g.size(), 0);
        size_t last = 0;
        placed[0] = 1;
        order.push_back(g[0]);
        for (size_t step = 1; step < g.size(); ++step) {
            const int32_t *a = &cum[static_cast<size_t>(g[last]) * (P + 1)];
            int64_t best_sim = -1;
            size_t best = 0;
            for (size_t j = 0; j < g.size(); ++j) {
                if (placed[j]) continue;
                const int32_t *b = &cum[static_cast<size_t>(g[j]) * (P + 1)];
                int64_t sim = 0;                                  // overlap of the two sorted runs of each pattern
                for (int p = 0; p < P; ++p) {
                    const int32_t lo = std::max(a[p], b[p]), hi = std::min(a[p + 1], b[p + 1]);
                    if (hi > lo) sim += hi - lo;
                }
                if (sim > best_sim) { best_sim = sim; best = j; }
            }
            placed[best] = 1;
            order.push_back(g[best]);
            last = best;
        }
    }
}

int build_fkw(const float *weights, const uint8_t *mask, const uint16_t *pattern_set, int32_t P, int32_t F,
              int32_t C, int32_t dtype, const int32_t *caller_order, Fkw &out) {
    if (!weights || !mask) return PATDNN_E_NULL;
    if (F < 1 || C < 1 || C > 65535 || static_cast<int64_t>(F) * C > (int64_t(1) << 28)) return PATDNN_E_SHAPE;
    if (dtype != PATDNN_F32 && dtype != PATDNN_F16) return PATDNN_E_DTYPE;
    int rc = validate_pattern_set(pattern_set, P);
    if (rc) return rc;
    std::vector<int32_t> pid;
    rc = classify_kernels(mask, pattern_set, P, F, C, pid);
    if (rc) return rc;

    out = Fkw();
    out.F = F; out.C = C; out.P = P; out.dtype = dtype;
    out.patterns.assign(pattern_set, pattern_set + P);
    if (caller_order) {
        std::vector<char> seen(F, 0);
        for (int i = 0; i < F; ++i) {
            const int32_t f = caller_order[i];
            if (f < 0 || f >= F || seen[f]) return PATDNN_E_ORDER;
            seen[f] = 1;
        }
        out.reorder.assign(caller_order, caller_order + F);
    } else {
        filter_reorder(pid, P, F, C, out.reorder);
    }

    int tap_of[32][4];
    for (int p = 0; p < P; ++p) {
        int n = 0;
        for (int t = 0; t < 9; ++t)
            if ((pattern_set[p] >> t) & 1) tap_of[p][n++] = t;
    }
    out.offset.assign(F + 1, 0);
    out.stride.assign(static_cast<size_t>(F) * (P + 1), 0);
    for (int i = 0; i < F; ++i) {
        const int32_t f = out.reorder[i];
        int32_t *row = &out.stride[static_cast<size_t>(i) * (P + 1)];
        for (int c = 0; c < C; ++c) {
            const int32_t p = pid[static_cast<size_t>(f) * C + c];
            if (p >= 0) ++row[p + 1];
        }
        for (int p = 0; p < P; ++p) row[p + 1] += row[p];
        out.offset[i + 1] = out.offset[i] + row[P];
    }
    const int32_t K = out.offset[F];
    out.K = K;
    out.index.resize(K);
    out.kernel_pid.resize(K);
    out.weight_f32.resize(static_cast<size_t>(K) * 4);
    if (dtype == PATDNN_F16) out.weight_f16.resize(static_cast<size_t>(K) * 4);
    std::vector<int32_t> cursor(P);
    for (int i = 0; i < F; ++i) {
        const int32_t f = out.reorder[i];
        const int32_t *row = &out.stride[static_cast<size_t>(i) * (P + 1)];
        for (int p = 0; p < P; ++p) cursor[p] = out.offset[i] + row[p];
        for (int c = 0; c < C; ++c) {                             // ascending channel inside every pattern run
            const int32_t p = pid[static_cast<size_t>(f) * C + c];
            if (p < 0) continue;
            const int32_t k = cursor[p]++;
            out.index[k] = c;
            out.kernel_pid[k] = p;
            const float *w9 = weights + (static_cast<size_t>(f) * C + c) * 9;
            for (int j = 0; j < 4; ++j) {
                const float w = w9[tap_of[p][j]];
                if (dtype == PATDNN_F16) {
                    const uint16_t h = float_to_half_rne(w);
                    out.weight_f16[static_cast<size_t>(k) * 4 + j] = h;
                    out.weight_f32[static_cast<size_t>(k) * 4 + j] = half_to_float(h);
                } else {
                    out.weight_f32[static_cast<size_t>(k) * 4 + j] = w;
                }
            }
        }
    }
    return PATDNN_OK;
}

void decode_fkw(const Fkw &fkw, float *dense) {
    std::memset(dense, 0, sizeof(float) * static_cast<size_t>(fkw.F) * fkw.C * 9);
    for (int i = 0; i < fkw.F; ++i) {
        const int32_t f = fkw.reorder[i];
        const int32_t *row = &fkw.stride[static_cast<size_t>(i) * (fkw.P + 1)];
        for (int p = 0; p < fkw.P; ++p) {
            for (int32_t j = row[p]; j < row[p + 1]; ++j) {
                const int32_t k = fkw.offset[i] + j;
                float *d9 = dense + (static_cast<size_t>(f) * fkw.C + fkw.index[k]) * 9;
                int n = 0;
                for (int t = 0; t < 9; ++t)
                    if ((fkw.patterns[p] >> t) & 1) d9[t] = fkw.weight_f32[static_cast<size_t>(k) * 4 + n++];
            }
        }
    }
}

}  // namespace patdnn
