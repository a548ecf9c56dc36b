// Dispatch from a planned blocking to the compiled instances of the tiled kernel.
#include <cuda_runtime.h>

#include "../../include/patdnn.h"
#include "kernels.hpp"

namespace patdnn {

#define PATDNN_DECL(name) \
    cudaError_t name(const TiledPlan &plan, const TiledParams &p, int dtype, cudaStream_t stream, bool prep);
PATDNN_DECL(launch_tiled_4x8)
PATDNN_DECL(launch_tiled_4x4)
PATDNN_DECL(launch_tiled_2x8)
#undef PATDNN_DECL

static cudaError_t route(const TiledPlan &plan, const TiledParams &p, int dtype, cudaStream_t stream, bool prep) {
    const TiledConfig &c = plan.cfg;
    if (c.TY == 4 && c.FR == 8) return launch_tiled_4x8(plan, p, dtype, stream, prep);
    if (c.TY == 4 && c.FR == 4) return launch_tiled_4x4(plan, p, dtype, stream, prep);
    if (c.TY == 2 && c.FR == 8) return launch_tiled_2x8(plan, p, dtype, stream, prep);
    return cudaErrorInvalidConfiguration;
}

cudaError_t launch_tiled(const TiledPlan &plan, const TiledParams &p, int dtype, cudaStream_t stream) {
    if (plan.tiles_total == 0) return cudaSuccess;
    return route(plan, p, dtype, stream, false);
}

cudaError_t prepare_tiled(const TiledPlan &plan, int dtype) {
    TiledParams dummy{};
    return route(plan, dummy, dtype, nullptr, true);
}

}  // namespace patdnn
