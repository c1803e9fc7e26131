// tcgen05 kernel variants for activation = FGR_ACT_SILU (one translation unit per activation).
#include "fgr_umma_kernel.cuh"

namespace fgr {

cudaError_t umma_launch_act_silu(bool sc, int red, bool wy, const Params& p, const void* tx, const void* tw, int grid,
                               int smem, cudaStream_t s) {
  return umma::launch_act<FGR_ACT_SILU>(sc, red, wy, p, *static_cast<const CUtensorMap*>(tx), *static_cast<const CUtensorMap*>(tw),
                              grid, smem, s);
}

cudaError_t umma_prepare_act_silu() { return umma::prepare_act<FGR_ACT_SILU>(); }

}  // namespace fgr
