// Instances of the tiled kernel for 2 output rows per thread and 8 filters per warp.
#include "kernels_tiled.cuh"

namespace patdnn {

cudaError_t launch_tiled_2x8(const TiledPlan &plan, const TiledParams &p, int dtype, cudaStream_t stream, bool prep) {
    const TiledConfig &c = plan.cfg;
#define PATDNN_INST(pw, fw)                                                                                   \
    if (c.PW == pw && c.FW == fw)                                                                             \
        return dtype == PATDNN_F16 ? launch_instance<2, 8, pw, fw, 2, __half>(plan, p, stream, prep)      \
                                   : launch_instance<2, 8, pw, fw, 2, float>(plan, p, stream, prep);
    PATDNN_INST(2, 4) PATDNN_INST(2, 2) PATDNN_INST(2, 1) PATDNN_INST(1, 4) PATDNN_INST(1, 2) PATDNN_INST(1, 1)
#undef PATDNN_INST
    return cudaErrorInvalidConfiguration;
}

}  // namespace patdnn
