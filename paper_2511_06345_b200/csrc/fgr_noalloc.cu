// fgr_run_static: the operator for callers that cannot allocate device memory.
//
// Some code that wants this operator runs where cudaMalloc is off limits: inside a framework whose
// allocator owns the whole device and hands nothing out, in a real-time loop that must not take the
// allocator's locks, or in an embedding that receives buffers but no allocator.  fgr_run asks
// such a caller for a workspace it has no way to obtain.  This entry point keeps the split-N
// partial pairs in a fixed array that is part of the library image instead, so the caller passes
// only inputs and outputs.
//
// The array below lives in every CUDA context that loads the library, from load until exit.  Its
// name is usable directly in device code of this file only; host code must first translate it
// into a device address with cudaGetSymbolAddress (per device, with that device current) - passing
// the bare name to a kernel would hand it a host-side stand-in, not device memory.
#include <cuda_runtime.h>

#include <cstring>
#include <mutex>

#include "fgr_internal.h"

namespace {

constexpr size_t kScratchBytes = 4u << 20;   // FGR_STATIC_SCRATCH_BYTES
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

// Device address of g_scratch per device ordinal; filled by the first call on that device.
float* g_scratch_addr[kMaxDevices] = {};
std::mutex g_setup_mutex;

}  // namespace

extern "C" {

int fgr_run_static(const fgr_desc* desc, const void* X, const void* W, const float* bias, const float* scale_vec,
                   void* Y, float* out, void* cuda_stream) {
  if (!desc || !X || !W) return FGR_ERR_INVALID_ARG;
  // the size field first: a shorter struct from an older caller must not be read past its end
  if (desc->struct_bytes != sizeof(fgr_desc)) return FGR_ERR_INVALID_ARG;
  if (desc->force_path != FGR_PATH_AUTO && desc->force_path != FGR_PATH_SIMT) return FGR_ERR_UNSUPPORTED;
  if (desc->device < 0 || desc->device >= kMaxDevices) return FGR_ERR_INVALID_ARG;
  // validation and tiling come from the public planner, with the CUDA-core path selected
  fgr_desc d = *desc;
  d.force_path = FGR_PATH_SIMT;
  fgr_plan_info plan;
  int rc = fgr_plan(&d, 0, &plan);
  if (rc != FGR_OK) return rc;
  if (d.conv_taps > 1 || d.conv_rows > 1) return FGR_ERR_UNSUPPORTED;   // plain GEMMs only
  const unsigned long long need = (unsigned long long)d.batch * d.M * plan.parts_per_row * 8ull;
  if (need > kScratchBytes) return FGR_ERR_WORKSPACE;   // the fixed scratch cannot hold this problem's partial pairs

  const bool softmax = d.reduce == FGR_RED_SOFTMAX;
  if ((reinterpret_cast<uintptr_t>(X) & 15u) || (reinterpret_cast<uintptr_t>(W) & 15u) ||
      (Y && (reinterpret_cast<uintptr_t>(Y) & 15u)) || (out && (reinterpret_cast<uintptr_t>(out) & 7u)) ||
      (bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) || (scale_vec && (reinterpret_cast<uintptr_t>(scale_vec) & 3u)))
    return FGR_ERR_INVALID_ARG;
  if ((d.write_y || softmax) && !Y) return FGR_ERR_INVALID_ARG;
  if (!softmax && !out) return FGR_ERR_INVALID_ARG;
  if (d.scale_kind == FGR_SCALE_PER_COLUMN && !scale_vec) return FGR_ERR_INVALID_ARG;

  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != d.device && cudaSetDevice(d.device) != cudaSuccess) { cudaGetLastError(); return FGR_ERR_CUDA; }
  rc = FGR_OK;
  float* scratch = nullptr;
  {
    // one-time set-up on this device (two host threads may make their first call together): architecture
    // check and the device address of the scratch array.  With the CUDA runtime's lazy module loading this
    // look-up is also what loads the module that holds the array, i.e. when the device reserves its bytes.
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[d.device]) {
      int major = 0;
      void* addr = nullptr;
      if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, d.device) != cudaSuccess) rc = FGR_ERR_CUDA;
      else if (major != 10) rc = FGR_ERR_ARCH;
      else if (cudaGetSymbolAddress(&addr, g_scratch) != cudaSuccess || !addr) { cudaGetLastError(); rc = FGR_ERR_CUDA; }
      else g_scratch_addr[d.device] = static_cast<float*>(addr);
    }
    scratch = g_scratch_addr[d.device];
  }
  if (rc == FGR_OK) {
    fgr::Params p;
    std::memset(&p, 0, sizeof p);
    p.batch = d.batch; p.M = d.M; p.N = d.N; p.K = d.K;
    p.dtype = d.dtype; p.act = d.act; p.scale_kind = d.scale_kind; p.reduce = d.reduce;
    p.write_y = d.write_y; p.bias_per_batch = d.bias_per_batch; p.scale = d.scale;
    p.ldx = d.ldx ? d.ldx : d.K;
    p.ldw = d.ldw ? d.ldw : d.K;
    p.ldy = d.ldy ? d.ldy : d.N;
    p.bsx = d.bsx ? d.bsx : (long long)d.M * p.ldx;
    p.bsw = d.w_shared ? 0 : (d.bsw ? d.bsw : (long long)d.N * p.ldw);
    p.w_shared = d.w_shared;
    p.bsy = d.bsy ? d.bsy : (long long)d.M * p.ldy;
    p.X = X; p.W = W; p.bias = bias; p.scale_vec = scale_vec; p.Y = Y; p.out = out;
    p.parts = scratch;   // every pair the second kernel reads is written by the first
    p.status = nullptr;                   // the CUDA-core kernels have no waits and report no status
    p.tile_n = plan.tile_n;
    p.half_n = plan.tile_n;
    p.slots_per_tile = 1;
    p.tiles_m = (d.M + plan.tile_m - 1) / plan.tile_m;
    p.tiles_n = (d.N + plan.tile_n - 1) / plan.tile_n;
    p.num_tiles = plan.num_tiles;
    p.parts_per_row = plan.parts_per_row;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = fgr::launch_simt(p, stream);
    if (e == cudaSuccess) e = softmax ? fgr::launch_normalise(p, stream) : fgr::launch_merge(p, stream);
    if (e != cudaSuccess) { cudaGetLastError(); rc = FGR_ERR_CUDA; }
  }
  if (prev != d.device && prev >= 0) cudaSetDevice(prev);
  return rc;
}

}  // extern "C"
