// Skinny-M path (M <= 16, bf16): the problem is a handful of GEMVs, bound by streaming W from HBM
// once.  No tensor cores: one warp owns R rows of W at a time, its lanes stride over K with 128-bit
// coalesced loads, X (at most 16 rows) sits in shared memory in K chunks, every lane keeps R x M
// fp32 partial dot products, and a xor-shuffle butterfly sums them over the warp.  Lane m then owns
// output row m: it applies bias / activation / scale and keeps the running row reduction over the
// W rows its warp has seen.  One partial pair per (row, CTA) goes to the workspace; the merge kernel
// finishes.  Softmax is not offered on this path (it needs the per-slot maximum before storing).
#include <cuda_bf16.h>
#include <math_constants.h>

#include "fgr_internal.h"

namespace fgr {
namespace {

constexpr int kGemvThreads = 512;
constexpr int kGemvWarps = kGemvThreads / 32;
constexpr int kLaneK = 8;                    // bf16 elements per 128-bit load
constexpr int kWarpK = 32 * kLaneK;          // K covered by one warp-wide load

__device__ __forceinline__ float activation(int act, float u) {
  if (act == FGR_ACT_RELU) return fmaxf(u, 0.0f);
  if (act == FGR_ACT_GELU_TANH) {
    const float c = 0.7978845608028654f;  // sqrt(2 / pi)
    return 0.5f * u * (1.0f + tanhf(c * (u + 0.044715f * u * u * u)));
  }
  if (act == FGR_ACT_SIGMOID) return 1.0f / (1.0f + expf(-u));
  if (act == FGR_ACT_TANH) return tanhf(u);
  if (act == FGR_ACT_SILU) return u / (1.0f + expf(-u));
  return u;
}

// 128-bit streaming load of W: read once, keep it out of L1
__device__ __forceinline__ uint4 load_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ float dot8(const uint4& a, const uint4& b, float acc) {
  const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc = fmaf(__uint_as_float(aw[i] << 16), __uint_as_float(bw[i] << 16), acc);
    acc = fmaf(__uint_as_float(aw[i] & 0xffff0000u), __uint_as_float(bw[i] & 0xffff0000u), acc);
  }
  return acc;
}

// MT: rows of X held per lane (M rounded up to 1, 2, 4, 8 or 16); R: rows of W per warp and pass;
// U: warp-wide K steps whose loads are issued together.
template <int MT, int R, int U>
__global__ void __launch_bounds__(kGemvThreads, 1) gemv_kernel(const Params p, int rows_per_cta, int kc) {
  extern __shared__ __align__(16) unsigned char gemv_smem[];
  __nv_bfloat16* Xs = reinterpret_cast<__nv_bfloat16*>(gemv_smem);                      // [MT][kc]
  float2* red = reinterpret_cast<float2*>(gemv_smem + (size_t)MT * kc * 2);             // [warps][MT]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bt = blockIdx.y;
  const int n_begin = blockIdx.x * rows_per_cta;
  const int n_end = min(p.N, n_begin + rows_per_cta);
  const __nv_bfloat16* X = static_cast<const __nv_bfloat16*>(p.X) + (long long)bt * p.bsx;
  const __nv_bfloat16* W = static_cast<const __nv_bfloat16*>(p.W) + (long long)bt * p.bsw;
  __nv_bfloat16* Y = static_cast<__nv_bfloat16*>(p.Y) + (long long)bt * p.bsy;
  const float* bias = p.bias ? p.bias + (p.bias_per_batch ? (long long)bt * p.N : 0) : nullptr;
  const bool meanvar = p.reduce == FGR_RED_MEANVAR;
  const bool exp_kind = p.reduce != FGR_RED_MAXSUM && !meanvar;

  // lane m < M: running (max, sum) or (max, sum of exp(y - max)) of row m; for mean / variance the sums of
  // (y - shift) and (y - shift)^2 against the first y this lane saw, and their count
  float s0 = meanvar ? 0.0f : -CUDART_INF_F, s1 = 0.0f, shift = 0.0f;
  int cnt = 0;

  for (int pass0 = n_begin; pass0 < n_end; pass0 += kGemvWarps * R) {
    const int n0 = pass0 + warp * R;
    float acc[R][MT];
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int m = 0; m < MT; ++m) acc[r][m] = 0.0f;

    for (int k0 = 0; k0 < p.K; k0 += kc) {
      const int kcur = min(kc, p.K - k0);              // a multiple of 8
      const int kpad = (kcur + kWarpK - 1) / kWarpK * kWarpK;
      __syncthreads();                                 // the previous chunk is no longer read
      for (int i = threadIdx.x; i < MT * (kpad / kLaneK); i += kGemvThreads) {
        const int m = i / (kpad / kLaneK), k = (i - m * (kpad / kLaneK)) * kLaneK;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);          // rows beyond M and columns beyond K count as zero
        if (m < p.M && k < kcur) v = *reinterpret_cast<const uint4*>(X + (long long)m * p.ldx + k0 + k);
        *reinterpret_cast<uint4*>(Xs + (size_t)m * kc + k) = v;
      }
      __syncthreads();
      if (n0 < n_end) {
        // U warp-wide steps per iteration: R * U 128-bit loads of W in flight per lane
        for (int k = lane * kLaneK; k < kpad; k += kWarpK * U) {
          uint4 wv[U][R];
#pragma unroll
          for (int u = 0; u < U; ++u)
#pragma unroll
            for (int r = 0; r < R; ++r) {
              const int kk = k + u * kWarpK;
              wv[u][r] = make_uint4(0u, 0u, 0u, 0u);
              if (n0 + r < n_end && kk < kcur) wv[u][r] = load_stream(W + (long long)(n0 + r) * p.ldw + k0 + kk);
            }
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const int kk = k + u * kWarpK;
            if (kk >= kpad) break;                     // (warp-uniform: kpad is a multiple of a warp-wide step)
#pragma unroll
            for (int m = 0; m < MT; ++m) {
              const uint4 xv = *reinterpret_cast<const uint4*>(Xs + (size_t)m * kc + kk);
#pragma unroll
              for (int r = 0; r < R; ++r) acc[r][m] = dot8(wv[u][r], xv, acc[r][m]);
            }
          }
        }
      }
    }
    if (n0 >= n_end) continue;   // (warp-uniform) no rows left for this warp in the last pass

    // warp-shuffle butterfly: afterwards every lane holds the full dot products
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
      for (int m = 0; m < MT; ++m) {
        float v = acc[r][m];
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        acc[r][m] = v;
      }
    // lane m finishes output row m for the R columns n0 .. n0 + R - 1
#pragma unroll
    for (int r = 0; r < R; ++r) {
      const int n = n0 + r;
      if (n >= n_end) break;
      float z = 0.0f;
#pragma unroll
      for (int m = 0; m < MT; ++m) if (lane == m) z = acc[r][m];
      if (lane < p.M) {
        float s = 1.0f;
        if (p.scale_kind == FGR_SCALE_PER_COLUMN) s = p.scale_vec[n];
        else if (p.scale_kind == FGR_SCALE_SCALAR) s = p.scale;
        float y = activation(p.act, z + (bias ? bias[n] : 0.0f)) * s;
        if (p.R) y += __bfloat162float(static_cast<const __nv_bfloat16*>(p.R)[(long long)bt * p.bsr + (long long)lane * p.ldr + n]);
        if (p.write_y) Y[(long long)lane * p.ldy + n] = __float2bfloat16_rn(y);
        if (meanvar) {
          if (cnt == 0) shift = y;
          const float d = y - shift;
          s0 += d;
          s1 = fmaf(d, d, s1);
          ++cnt;
        } else if (exp_kind) {
          const float mn = fmaxf(s0, y);
          s1 = s1 * expf(s0 - mn) + expf(y - mn);
          s0 = mn;
        } else {
          s0 = fmaxf(s0, y);
          s1 += y;
        }
      }
    }
  }
  if (meanvar && cnt > 0) {   // -> (mean, sum of squared deviations) of this warp's columns of row `lane`
    const float md = s0 / (float)cnt;
    s1 = fmaxf(s1 - s0 * md, 0.0f);
    s0 = shift + md;
  }

  // combine the warps of this CTA in warp order (fixed, so results repeat bit for bit)
  __syncthreads();
  if (lane < MT) red[warp * MT + lane] = make_float2(s0, s1);
  __syncthreads();
  if (warp == 0 && lane < p.M) {
    float a = -CUDART_INF_F, b = 0.0f;
    float n = 0.0f;
    if (meanvar) { a = 0.0f; }
    for (int w = 0; w < kGemvWarps; ++w) {
      const float2 v = red[w * MT + lane];
      if (meanvar) {
        // columns warp w finished: R per pass of kGemvWarps * R columns, clipped at the end of this CTA's range
        int cw = 0;
        for (int pass0 = n_begin; pass0 < n_end; pass0 += kGemvWarps * R) {
          const int left = n_end - (pass0 + w * R);
          cw += left <= 0 ? 0 : (left < R ? left : R);
        }
        if (cw > 0) {
          const float nb = (float)cw, tot = n + nb, delta = v.x - a;
          a += delta * (nb / tot);
          b += v.y + delta * delta * (n * nb / tot);
          n = tot;
        }
      } else if (exp_kind) {
        const float mn = fmaxf(a, v.x);
        if (mn > -CUDART_INF_F) b = b * expf(a - mn) + v.y * expf(v.x - mn);
        a = mn;
      } else {
        a = fmaxf(a, v.x);
        b += v.y;
      }
    }
    reinterpret_cast<float2*>(p.parts)[((long long)bt * p.M + lane) * p.parts_per_row + blockIdx.x] = make_float2(a, b);
  }
}

template <int MT, int R, int U>
cudaError_t launch_variant(const Params& p, int grid, int rows_per_cta, int kc, cudaStream_t stream) {
  const size_t smem = (size_t)MT * kc * 2 + (size_t)kGemvWarps * MT * sizeof(float2);
  cudaError_t e = cudaFuncSetAttribute(gemv_kernel<MT, R, U>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  gemv_kernel<MT, R, U><<<dim3((unsigned)grid, (unsigned)p.batch), kGemvThreads, smem, stream>>>(p, rows_per_cta, kc);
  return cudaGetLastError();
}

}  // namespace

int gemv_rows_per_warp(int M) { return M > 8 ? 2 : 4; }

// K chunk of X kept in shared memory: as much as fits in about 192 KB, a multiple of one warp-wide load.
int gemv_k_chunk(int M, int K) {
  const int mt = M > 8 ? 16 : M > 4 ? 8 : M > 2 ? 4 : M > 1 ? 2 : 1;
  int kc = (192 * 1024 / (2 * mt)) / kWarpK * kWarpK;
  const int kpad = (K + kWarpK - 1) / kWarpK * kWarpK;
  return kc < kpad ? kc : kpad;
}

cudaError_t launch_gemv(const Params& p, int grid, int rows_per_cta, cudaStream_t stream) {
  const int kc = gemv_k_chunk(p.M, p.K);
  if (p.M > 8) return launch_variant<16, 2, 2>(p, grid, rows_per_cta, kc, stream);
  if (p.M > 4) return launch_variant<8, 4, 2>(p, grid, rows_per_cta, kc, stream);
  if (p.M > 2) return launch_variant<4, 4, 3>(p, grid, rows_per_cta, kc, stream);
  if (p.M > 1) return launch_variant<2, 4, 4>(p, grid, rows_per_cta, kc, stream);
  return launch_variant<1, 4, 4>(p, grid, rows_per_cta, kc, stream);
}

}  // namespace fgr
