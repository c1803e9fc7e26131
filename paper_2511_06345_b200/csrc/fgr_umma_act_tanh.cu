// tcgen05 kernel variants for activation = FGR_ACT_TANH (one translation unit per activation).
#include "fgr_umma_kernel.cuh"

namespace fgr {

cudaError_t umma_launch_act_tanh(bool sc, int red, bool wy, const Params& p, const void* tx, const void* tw, int grid,
                               int smem, cudaStream_t s) {
  return umma::launch_act<FGR_ACT_TANH>(sc, red, wy, p, *static_cast<const CUtensorMap*>(tx), *static_cast<const CUtensorMap*>(tw),
                              grid, smem, s);
}

cudaError_t umma_prepare_act_tanh() { return umma::prepare_act<FGR_ACT_TANH>(); }

}  // namespace fgr
