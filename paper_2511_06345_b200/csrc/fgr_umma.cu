// Dispatch of the tcgen05 path: picks the compiled kernel variant for a problem's activation,
// scaling, reduction kind and Y store.  The kernel itself is in fgr_umma_kernel.cuh.
#include <mutex>

#include "fgr_umma_kernel.cuh"

namespace fgr {

// Raises the dynamic shared-memory limit of every kernel variant on the current device.  The attribute
// belongs to (device, kernel), so the several hundred calls are made once per device ordinal; later
// handles on that device find it done.
cudaError_t umma_prepare(int device) {
  constexpr int kMaxDevices = 64;
  static std::mutex mu;
  static bool done[kMaxDevices] = {};
  std::lock_guard<std::mutex> lock(mu);
  if (device >= 0 && device < kMaxDevices && done[device]) return cudaSuccess;
  cudaError_t e = umma_prepare_act_none();
  if (e == cudaSuccess) e = umma_prepare_act_relu();
  if (e == cudaSuccess) e = umma_prepare_act_gelu();
  if (e == cudaSuccess) e = umma_prepare_act_sigmoid();
  if (e == cudaSuccess) e = umma_prepare_act_tanh();
  if (e == cudaSuccess) e = umma_prepare_act_silu();
  if (e == cudaSuccess && device >= 0 && device < kMaxDevices) done[device] = true;
  return e;
}

cudaError_t launch_umma(const Params& p, const void* tmap_x, const void* tmap_w, int grid, int smem_bytes,
                        cudaStream_t stream) {
  const bool softmax = p.reduce == FGR_RED_SOFTMAX;
  const bool exp_kind = p.reduce == FGR_RED_LSE || p.reduce == FGR_RED_SOFTMAX || p.reduce == FGR_RED_MAX_SUMEXP;
  const bool wy = softmax ? p.R != nullptr : p.write_y != 0;   // softmax: the variant compiled with the residual add
  // exp kinds that do not store y fold log2(e) into the staged scale vector, so they always multiply
  const bool sc = (exp_kind && (softmax || !wy)) || p.scale_kind != FGR_SCALE_NONE;
  switch (p.act) {
    case FGR_ACT_NONE: return umma_launch_act_none(sc, p.reduce, wy, p, tmap_x, tmap_w, grid, smem_bytes, stream);
    case FGR_ACT_RELU: return umma_launch_act_relu(sc, p.reduce, wy, p, tmap_x, tmap_w, grid, smem_bytes, stream);
    case FGR_ACT_GELU_TANH: return umma_launch_act_gelu(sc, p.reduce, wy, p, tmap_x, tmap_w, grid, smem_bytes, stream);
    case FGR_ACT_SIGMOID: return umma_launch_act_sigmoid(sc, p.reduce, wy, p, tmap_x, tmap_w, grid, smem_bytes, stream);
    case FGR_ACT_TANH: return umma_launch_act_tanh(sc, p.reduce, wy, p, tmap_x, tmap_w, grid, smem_bytes, stream);
    case FGR_ACT_SILU: return umma_launch_act_silu(sc, p.reduce, wy, p, tmap_x, tmap_w, grid, smem_bytes, stream);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace fgr
