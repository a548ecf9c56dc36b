// Host-side filter-kernel reorder (Section 5.2) and FKW compressed weight storage (Section 5.3).
#pragma once
#include <cstdint>
#include <vector>

namespace patdnn {

struct Fkw {
    int32_t F = 0, C = 0, P = 0, K = 0;
    int32_t dtype = 0;                         // PATDNN_F32 / PATDNN_F16
    std::vector<uint16_t> patterns;            // [P] 9-bit masks
    std::vector<int32_t> offset;               // [F+1]
    std::vector<int32_t> reorder;              // [F] position -> original filter
    std::vector<int32_t> index;                // [K]
    std::vector<int32_t> stride;               // [F][P+1]
    std::vector<float> weight_f32;             // [K][4] (always filled; half-rounded values for F16)
    std::vector<uint16_t> weight_f16;          // [K][4] half bit patterns (F16 only)
    std::vector<int32_t> kernel_pid;           // [K] pattern id of stored kernel k (implied by stride; kept for layouts)
};

// Status codes are the PATDNN_* values of patdnn.h.
int validate_pattern_set(const uint16_t *pattern_set, int32_t n_patterns);

// pid[f*C+c] = pattern id or -1 for an empty kernel.
int classify_kernels(const uint8_t *mask, const uint16_t *pattern_set, int32_t P, int32_t F, int32_t C,
                     std::vector<int32_t> &pid);

// Filter reorder: ascending length groups, greedy most-similar chain inside a group.
void filter_reorder(const std::vector<int32_t> &pid, int32_t P, int32_t F, int32_t C, std::vector<int32_t> &order);

int build_fkw(const float *weights, const uint8_t *mask, const uint16_t *pattern_set, int32_t P, int32_t F,
              int32_t C, int32_t dtype, const int32_t *caller_order, Fkw &out);

void decode_fkw(const Fkw &fkw, float *dense);   // [F][C][3][3]

uint16_t float_to_half_rne(float f);
float half_to_float(uint16_t h);

}  // namespace patdnn
