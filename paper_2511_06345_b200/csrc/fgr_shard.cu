// Combine step of the operator when its N dimension is sharded over several GPUs.
//
// Every shard (one per GPU) owns a contiguous slice of W's rows (= columns of Y) and computes, for
// each output row, the row statistics of its slice: (max, sum of exp(y - max)) or (max, sum).  After
// an all-gather of those pairs, every GPU holds pairs[shard][row] and runs the kernels below:
//   - combine_rows_kernel: merges the pairs of a row in ascending shard order -> out
//     (LSE, (max, sum), (max, sum-exp)); one thread per row;
//   - combine_softmax_kernel: the same merge, then rescales this GPU's slice of P, which the local
//     softmax had normalised by its own (max, sum-exp), to the statistics of the whole row.
// The merge order is the shard index, so all GPUs get bit-identical results.
#include <cuda_bf16.h>
#include <math_constants.h>

#include "fgr_internal.h"

namespace fgr {
namespace {

struct ShardParams {
  long long rows;
  int shards, reduce, shard, n_local;
  int groups, align;     // MEANVAR: N / align column groups dealt to the shards, the first groups % shards get one more
  long long ldp;
  const float2* pairs;   // [shards][rows]
  float* out;
  void* P;
};

// (a, b) <- (a, b) merged with v, in this order
__device__ __forceinline__ void merge_exp(float& a, float& b, float2 v) {
  const float mn = fmaxf(a, v.x);
  if (mn > -CUDART_INF_F) b = b * expf(a - mn) + v.y * expf(v.x - mn);
  a = mn;
}

__global__ void __launch_bounds__(256) combine_rows_kernel(const ShardParams p) {
  const long long row = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= p.rows) return;
  if (p.reduce == FGR_RED_MEANVAR) {
    // pairs are (mean, population variance) of a shard's columns; the shard widths follow the partition rule
    const int base = p.groups / p.shards, extra = p.groups % p.shards;
    float n = 0.0f, mean = 0.0f, m2 = 0.0f;
    for (int g = 0; g < p.shards; ++g) {
      const float nb = (float)((base + (g < extra ? 1 : 0)) * p.align);
      const float2 v = p.pairs[(long long)g * p.rows + row];
      const float tot = n + nb, delta = v.x - mean;
      mean += delta * (nb / tot);
      m2 += v.y * nb + delta * delta * (n * nb / tot);
      n = tot;
    }
    reinterpret_cast<float2*>(p.out)[row] = make_float2(mean, m2 / n);
    return;
  }
  float a = -CUDART_INF_F, b = 0.0f;
  for (int g = 0; g < p.shards; ++g) {
    const float2 v = p.pairs[(long long)g * p.rows + row];
    if (p.reduce == FGR_RED_MAXSUM) { a = fmaxf(a, v.x); b += v.y; }
    else merge_exp(a, b, v);
  }
  if (p.reduce == FGR_RED_LSE) p.out[row] = a + logf(b);
  else reinterpret_cast<float2*>(p.out)[row] = make_float2(a, b);
}

// One CTA per row (a warp per row when the slice is short).  P_local[row, :] *= l_g exp(m_g - m) / l.
template <typename T, int G>
__global__ void __launch_bounds__(256) combine_softmax_kernel(const ShardParams p) {
  const int sub = threadIdx.x % G;
  const long long row = (long long)blockIdx.x * (blockDim.x / G) + threadIdx.x / G;
  if (row >= p.rows) return;
  float a = -CUDART_INF_F, b = 0.0f;
  for (int g = 0; g < p.shards; ++g) merge_exp(a, b, p.pairs[(long long)g * p.rows + row]);
  const float2 mine = p.pairs[(long long)p.shard * p.rows + row];
  const float f = mine.y * expf(mine.x - a) / b;
  if (sub == 0 && p.out) reinterpret_cast<float2*>(p.out)[row] = make_float2(a, b);
  T* y = static_cast<T*>(p.P) + row * p.ldp;
  constexpr int V = 16 / (int)sizeof(T);
  for (int c = sub * V; c < p.n_local; c += G * V) {
    uint4 raw = *reinterpret_cast<const uint4*>(y + c);
    if constexpr (sizeof(T) == 4) {
      float* v = reinterpret_cast<float*>(&raw);
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] *= f;
    } else {
      uint32_t* w = reinterpret_cast<uint32_t*>(&raw);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        __nv_bfloat162 r = __floats2bfloat162_rn(__uint_as_float(w[j] << 16) * f, __uint_as_float(w[j] & 0xffff0000u) * f);
        w[j] = *reinterpret_cast<uint32_t*>(&r);
      }
    }
    *reinterpret_cast<uint4*>(y + c) = raw;
  }
}

template <typename T>
cudaError_t launch_softmax(const ShardParams& p, cudaStream_t s) {
  constexpr int V = 16 / (int)sizeof(T);
  if (p.n_local <= 32 * V * 4) {
    combine_softmax_kernel<T, 32><<<(unsigned)((p.rows + 7) / 8), 256, 0, s>>>(p);
  } else {
    combine_softmax_kernel<T, 256><<<(unsigned)p.rows, 256, 0, s>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace
}  // namespace fgr

extern "C" int fgr_combine_shards(const fgr_shard_desc* d, const float* pairs, float* out, void* P_local, void* cuda_stream) {
  using namespace fgr;
  if (!d || d->struct_bytes != sizeof(fgr_shard_desc) || !pairs) return FGR_ERR_INVALID_ARG;
  if (d->rows < 1 || d->shards < 1 || d->device < 0) return FGR_ERR_INVALID_ARG;
  const bool meanvar = d->reduce == FGR_RED_MEANVAR;
  if ((d->reduce < FGR_RED_LSE || d->reduce > FGR_RED_MAX_SUMEXP) && !meanvar) return FGR_ERR_INVALID_ARG;
  int groups = 0, align = 0;
  if (meanvar) {
    // the column partition of the shards: n_total columns in groups of 8 (bf16) / 4 (fp32), contiguous slices in
    // shard order, the first (groups % shards) shards one group wider
    if (d->dtype != FGR_F32 && d->dtype != FGR_BF16) return FGR_ERR_INVALID_ARG;
    align = d->dtype == FGR_F32 ? 4 : 8;
    if (d->n_total < 1 || d->n_total % align) return FGR_ERR_INVALID_ARG;
    groups = d->n_total / align;
    if (groups < d->shards) return FGR_ERR_INVALID_ARG;
  }
  if ((reinterpret_cast<uintptr_t>(pairs) & 7u) || (out && (reinterpret_cast<uintptr_t>(out) & 7u))) return FGR_ERR_INVALID_ARG;
  const bool softmax = d->reduce == FGR_RED_SOFTMAX;
  long long ldp = 0;
  if (softmax) {
    if (d->dtype != FGR_F32 && d->dtype != FGR_BF16) return FGR_ERR_INVALID_ARG;
    if (!P_local || d->shard < 0 || d->shard >= d->shards || d->n_local < 1 || d->ldp < 0) return FGR_ERR_INVALID_ARG;
    const int g = d->dtype == FGR_F32 ? 4 : 8;
    ldp = d->ldp ? d->ldp : d->n_local;
    if (ldp < d->n_local) return FGR_ERR_INVALID_ARG;
    if (d->n_local % g || ldp % g) return FGR_ERR_UNSUPPORTED;
    if (reinterpret_cast<uintptr_t>(P_local) & 15u) return FGR_ERR_INVALID_ARG;
    if ((long long)d->rows > 0x7fffffffLL) return FGR_ERR_UNSUPPORTED;
  } else if (!out) {
    return FGR_ERR_INVALID_ARG;
  }
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != d->device && cudaSetDevice(d->device) != cudaSuccess) { cudaGetLastError(); return FGR_ERR_CUDA; }
  ShardParams p = {d->rows, d->shards, d->reduce, d->shard, d->n_local, groups, align, ldp, reinterpret_cast<const float2*>(pairs), out, P_local};
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e;
  if (!softmax) {
    combine_rows_kernel<<<(unsigned)((d->rows + 255) / 256), 256, 0, s>>>(p);
    e = cudaGetLastError();
  } else {
    e = d->dtype == FGR_F32 ? launch_softmax<float>(p, s) : launch_softmax<__nv_bfloat16>(p, s);
  }
  if (prev != d->device && prev >= 0) cudaSetDevice(prev);
  if (e != cudaSuccess) { cudaGetLastError(); return FGR_ERR_CUDA; }
  return FGR_OK;
}
