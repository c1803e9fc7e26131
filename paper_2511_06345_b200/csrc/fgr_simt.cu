// CUDA-core kernels of the fgr library:
//   - simt_gemm_kernel: 64 x 64 output tiles, fp32 FMA, fused epilogue and per-tile row reduction
//     (the fp32 path; also a valid path for bf16 inputs),
//   - merge_kernel: combines the split-N partial pairs of every row in a fixed order,
//   - normalise_kernel: second pass of the softmax (rescales the stored exponentials).
// Accurate expf / logf / tanhf throughout: fp32 outputs are held to 1e-4 * (1 + |ref|).
#include <cuda_bf16.h>
#include <math_constants.h>

#include "fgr_internal.h"

namespace fgr {
namespace {

constexpr int BK = 32;
constexpr int PAD = 4;

__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  uint2 r = *reinterpret_cast<const uint2*>(p);
  float4 f;
  f.x = __uint_as_float(r.x << 16);
  f.y = __uint_as_float(r.x & 0xffff0000u);
  f.z = __uint_as_float(r.y << 16);
  f.w = __uint_as_float(r.y & 0xffff0000u);
  return f;
}
__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void store4(float* p, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
__device__ __forceinline__ void store4(__nv_bfloat16* p, float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 r;
  r.x = *reinterpret_cast<uint32_t*>(&lo);
  r.y = *reinterpret_cast<uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = r;
}

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

__device__ __forceinline__ float group16_max(float v) {
#pragma unroll
  for (int o = 8; o >= 1; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float group16_sum(float v) {
#pragma unroll
  for (int o = 8; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Programmatic dependent launch: the kernels below may be made resident while the kernel before
// them in the stream is still running; this wait returns once that kernel has completed and its
// writes are visible.  (A no-op for a kernel launched the ordinary way.)
__device__ __forceinline__ void wait_for_prior_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel in the stream (if it was launched as a programmatic dependent) become
// resident now and run its set-up; it still waits for this grid to finish before touching memory.
__device__ __forceinline__ void let_next_kernel_start() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// G lanes per row (32 / G rows per warp): lane t of a group takes partials t, t + G, ... in ascending
// order, then a fixed xor-shuffle tree combines the G lanes.  The order never depends on timing:
// bit-identical results from run to run.
// Every thread of the warp calls this (the shuffles are warp-wide); `row` is the lane group's row, `row_ok`
// whether it exists.  FROM_L2: the pairs may have been written by other SMs during this same kernel, so they
// are read past L1 (in the merge kernel, a launch of its own, ordinary loads are 1.8 us faster on 128 rows x
// 256 pairs: 55.0 against 56.9 us for the weight-streaming workload's whole step).
template <int G, bool FROM_L2>
__device__ __forceinline__ float2 load_pair(const float2* p) {
  if constexpr (FROM_L2) return __ldcg(p);
  else return *p;
}
template <int G, bool FROM_L2>
__device__ __forceinline__ void merge_rows(const Params& p, long long row, bool row_ok) {
  const int lane = threadIdx.x & 31, sub = lane % G;
  const float2* src = reinterpret_cast<const float2*>(p.parts) + (row_ok ? row : 0) * p.parts_per_row;
  if (p.reduce == FGR_RED_MEANVAR) {
    // pairs are (mean, sum of squared deviations) of a slot; the slot's column count follows from the
    // tiling.  Pairwise update: delta = mean_b - mean_a; mean += delta n_b / n; M2 += M2_b + delta^2 n_a n_b / n
    float n = 0.0f, mean = 0.0f, m2 = 0.0f;
    for (int t = sub; t < p.parts_per_row; t += G) {
      const float nb = (float)slot_columns(t, p.N, p.tile_n, p.half_n, p.slots_per_tile);
      if (nb > 0.0f) {
        const float2 v = load_pair<G, FROM_L2>(src + t);
        const float tot = n + nb, delta = v.x - mean;
        mean += delta * (nb / tot);
        m2 += v.y + delta * delta * (n * nb / tot);
        n = tot;
      }
    }
#pragma unroll
    for (int o = G / 2; o >= 1; o >>= 1) {
      const float on = __shfl_xor_sync(0xffffffffu, n, o), om = __shfl_xor_sync(0xffffffffu, mean, o),
                  o2 = __shfl_xor_sync(0xffffffffu, m2, o);
      // the lower lane's triple is always the left operand, so both lanes compute the same bits
      const bool hi = (lane & o) != 0;
      const float na = hi ? on : n, ma = hi ? om : mean, qa = hi ? o2 : m2;
      const float nb = hi ? n : on, mb = hi ? mean : om, qb = hi ? m2 : o2;
      const float tot = na + nb;
      if (tot > 0.0f) {
        const float delta = mb - ma;
        mean = ma + delta * (nb / tot);
        m2 = qa + qb + delta * delta * (na * nb / tot);
      }
      n = tot;
    }
    if (sub == 0 && row_ok) reinterpret_cast<float2*>(p.out)[row] = make_float2(mean, m2 / (float)p.N);
    return;
  }
  const bool exp_kind = p.reduce != FGR_RED_MAXSUM;
  float a = -CUDART_INF_F, b = 0.0f;
#pragma unroll 4
  for (int t = sub; t < p.parts_per_row; t += G) {
    float2 v = load_pair<G, FROM_L2>(src + t);
    if (exp_kind) {
      float mn = fmaxf(a, v.x);
      if (mn > -CUDART_INF_F) b = b * expf(a - mn) + v.y * expf(v.x - mn);
      a = mn;
    } else {
      a = fmaxf(a, v.x);
      b += v.y;
    }
  }
#pragma unroll
  for (int o = G / 2; o >= 1; o >>= 1) {
    float oa = __shfl_xor_sync(0xffffffffu, a, o), ob = __shfl_xor_sync(0xffffffffu, b, o);
    if (exp_kind) {
      float mn = fmaxf(a, oa);
      // both operands of the sum are evaluated in the same (lower lane first) order on both lanes
      float lo_a = (lane & o) ? oa : a, lo_b = (lane & o) ? ob : b;
      float hi_a = (lane & o) ? a : oa, hi_b = (lane & o) ? b : ob;
      b = (mn > -CUDART_INF_F) ? lo_b * expf(lo_a - mn) + hi_b * expf(hi_a - mn) : 0.0f;
      a = mn;
    } else {
      float lo_b = (lane & o) ? ob : b, hi_b = (lane & o) ? b : ob;
      a = fmaxf(a, oa);
      b = lo_b + hi_b;
    }
  }
  if (sub == 0 && row_ok) {
    if (p.reduce == FGR_RED_LSE) p.out[row] = a + logf(b);
    else if (p.reduce != FGR_RED_SOFTMAX) reinterpret_cast<float2*>(p.out)[row] = make_float2(a, b);
  }
}

// Lanes per row of the merge: few, each folding up to eight pairs (its loads are independent and go out together).
__host__ __device__ inline int merge_lanes(int parts_per_row) { return parts_per_row <= 8 ? 2 : parts_per_row <= 64 ? 8 : 32; }

template <typename T>
__global__ void __launch_bounds__(256) simt_gemm_kernel(const Params p) {
  __shared__ __align__(16) float Xs[BK][kSimtTile + PAD];
  __shared__ __align__(16) float Ws[BK][kSimtTile + PAD];

  const int bt = blockIdx.z;
  const int m0 = blockIdx.y * kSimtTile;
  const int n0 = blockIdx.x * kSimtTile;
  const int t = threadIdx.x;
  const int tx = t & 15, ty = t >> 4;
  const int lr = t >> 2, lk = (t & 3) * 4;

  const T* X = static_cast<const T*>(p.X) + (long long)bt * p.bsx;
  const T* W = static_cast<const T*>(p.W) + (long long)bt * p.bsw;

  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

  // the loads of k-block i + 1 are issued before the FMAs of k-block i, so their latency is hidden; a k-block
  // is 32 wide (two 16-byte loads per thread and matrix), which halves the number of load -> barrier -> FMA
  // rounds a short problem is bound by
  auto fetch = [&](int k0, float4 (&xv)[2], float4 (&wv)[2]) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      xv[h] = make_float4(0.f, 0.f, 0.f, 0.f);
      wv[h] = xv[h];
      if (k0 + 16 * h + lk < p.K) {   // K is a multiple of 4: the four elements are in range together
        // 2-D convolution: element k of the row lies in filter row k / (S C), which reads the image conv_width
        // pixels further down (S C is a multiple of 4, so the four elements stay in one filter row)
        const int kk = k0 + 16 * h + lk, fr = p.conv_rows > 1 ? kk / p.conv_kseg : 0;
        const long long xoff = p.conv_rows > 1 ? (long long)fr * p.conv_width * p.ldx + (kk - fr * p.conv_kseg) : kk;
        if (m0 + lr < p.M) xv[h] = load4(X + (long long)(m0 + lr) * p.ldx + xoff);
        if (n0 + lr < p.N) wv[h] = load4(W + (long long)(n0 + lr) * p.ldw + k0 + 16 * h + lk);
      }
    }
  };
  float4 xv[2], wv[2];
  fetch(0, xv, wv);
  for (int k0 = 0; k0 < p.K; k0 += BK) {
    __syncthreads();
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int kk = 16 * h + lk;
      Xs[kk + 0][lr] = xv[h].x; Xs[kk + 1][lr] = xv[h].y; Xs[kk + 2][lr] = xv[h].z; Xs[kk + 3][lr] = xv[h].w;
      Ws[kk + 0][lr] = wv[h].x; Ws[kk + 1][lr] = wv[h].y; Ws[kk + 2][lr] = wv[h].z; Ws[kk + 3][lr] = wv[h].w;
    }
    __syncthreads();
    if (k0 + BK < p.K) fetch(k0 + BK, xv, wv);
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float4 a = *reinterpret_cast<const float4*>(&Xs[k][ty * 4]);
      float4 b = *reinterpret_cast<const float4*>(&Ws[k][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
  }

  // ---- fused epilogue: y = act(z + b) * s, in registers
  const int nc = n0 + tx * 4;
  const bool cols_ok = nc < p.N;   // N is a multiple of 4: the four columns are in range together
  float bj[4] = {0.f, 0.f, 0.f, 0.f}, sj[4] = {1.f, 1.f, 1.f, 1.f};
  if (cols_ok) {
    if (p.bias) {
      const float* b = p.bias + (p.bias_per_batch ? (long long)bt * p.N : 0);
#pragma unroll
      for (int j = 0; j < 4; ++j) bj[j] = b[nc + j];
    }
    if (p.scale_kind == FGR_SCALE_PER_COLUMN) {
#pragma unroll
      for (int j = 0; j < 4; ++j) sj[j] = p.scale_vec[nc + j];
    } else if (p.scale_kind == FGR_SCALE_SCALAR) {
#pragma unroll
      for (int j = 0; j < 4; ++j) sj[j] = p.scale;
    }
  }
  T* Y = static_cast<T*>(p.Y) + (long long)bt * p.bsy;
  const T* Rres = p.R ? static_cast<const T*>(p.R) + (long long)bt * p.bsr : nullptr;
  const bool meanvar = p.reduce == FGR_RED_MEANVAR;
  const bool exp_kind = p.reduce != FGR_RED_MAXSUM && !meanvar;
  const bool store_y = p.write_y && p.reduce != FGR_RED_SOFTMAX;
  const int tile_cols = p.N - n0 < kSimtTile ? p.N - n0 : kSimtTile;   // columns of this tile inside the matrix

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    float y[4];
    float mx = -CUDART_INF_F, sm = 0.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      y[j] = activation(p.act, acc[i][j] + bj[j]) * sj[j];
      if (Rres && cols_ok && m < p.M) y[j] += to_float(Rres[(long long)m * p.ldr + nc + j]);
      if (cols_ok) { mx = fmaxf(mx, y[j]); sm += y[j]; }
    }
    if (store_y && cols_ok && m < p.M) store4(Y + (long long)m * p.ldy + nc, y[0], y[1], y[2], y[3]);
    // ---- per-tile row reduction across the 16 threads that share this row
    mx = group16_max(mx);
    float second;
    if (meanvar) {
      // two passes over the tile's columns of this row: mean, then squared deviations from it
      const float mean = group16_sum(sm) / (float)tile_cols;
      float dev = 0.0f;
#pragma unroll
      for (int j = 0; j < 4; ++j) if (cols_ok) dev += (y[j] - mean) * (y[j] - mean);
      mx = mean;
      second = group16_sum(dev);
    } else if (exp_kind) {
      float e[4], l = 0.0f;
#pragma unroll
      for (int j = 0; j < 4; ++j) { e[j] = cols_ok ? expf(y[j] - mx) : 0.0f; l += e[j]; }
      if (p.reduce == FGR_RED_SOFTMAX && cols_ok && m < p.M)
        store4(Y + (long long)m * p.ldy + nc, e[0], e[1], e[2], e[3]);
      second = group16_sum(l);
    } else {
      second = group16_sum(sm);
    }
    if (tx == 0 && m < p.M) {
      float2* dst = reinterpret_cast<float2*>(p.parts) +
                    ((long long)bt * p.M + m) * p.parts_per_row + blockIdx.x;
      *dst = make_float2(mx, second);
    }
  }
  // ---- split-N merge without a second launch (p.done != null: every reduction but softmax, whose second
  // pass rewrites P).  The CTAs of a block of 64 rows count themselves; the one that brings the count to the
  // number of column tiles knows that all partial pairs of those rows are in memory and merges them, exactly
  // as the merge kernel would (same lanes per row, same order: the same bits), then zeroes the count for the
  // next run.  No CTA waits for another.  Small problems are bound by launch latency: this halves it.
  if (p.done) {
    __shared__ int last;
    __threadfence();                       // this thread's pairs before the count
    __syncthreads();
    unsigned int* count = p.done + (long long)bt * gridDim.y + blockIdx.y;
    if (t == 0) last = atomicAdd(count, 1u) + 1 == gridDim.x ? 1 : 0;
    __syncthreads();
    if (last) {
      if (t == 0) *count = 0u;
      __threadfence();                     // the other CTAs' pairs, ordered after the count that revealed them
      const int g = merge_lanes(p.parts_per_row);
      for (int first = 0; first < kSimtTile; first += 256 / g) {
        const int li = first + t / g;      // row of the tile this lane group takes in this pass
        const bool ok = li < kSimtTile && m0 + li < p.M;
        const long long row = (long long)bt * p.M + m0 + li;
        if (g == 2) merge_rows<2, true>(p, row, ok);
        else if (g == 8) merge_rows<8, true>(p, row, ok);
        else merge_rows<32, true>(p, row, ok);
      }
    }
  }
}

template <int G>
__global__ void __launch_bounds__(256) merge_kernel(const Params p) {
  let_next_kernel_start();
  wait_for_prior_kernel();
  const long long row = ((long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * (32 / G) + (threadIdx.x & 31) / G;
  merge_rows<G, false>(p, row, row < (long long)p.batch * p.M);
}

// Softmax, second pass.  The GEMM pass stored E[m, n] = exp(y - m_slot) per partial slot together
// with (m_slot, l_slot).  One CTA per row: the first warp merges the slots into (m_row, l_row) and
// leaves the factor exp(m_slot - m_row) / l_row of every slot in shared memory; then the CTA
// rescales the row with 16-byte accesses.
template <typename T>
__device__ __forceinline__ void normalise_row(const Params& p, long long row, float* factor) {
  const int bt = (int)(row / p.M), m = (int)(row % p.M);
  const float2* src = reinterpret_cast<const float2*>(p.parts) + row * p.parts_per_row;
  if (threadIdx.x < 32) {
    const int lane = threadIdx.x;
    float a = -CUDART_INF_F;
    for (int t = lane; t < p.parts_per_row; t += 32) a = fmaxf(a, src[t].x);
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
    float l = 0.0f;
    for (int t = lane; t < p.parts_per_row; t += 32) {
      float2 v = src[t];
      float f = (v.x > -CUDART_INF_F) ? expf(v.x - a) : 0.0f;
      factor[t] = f;
      l += v.y * f;
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
      float ol = __shfl_xor_sync(0xffffffffu, l, o);
      l = (lane & o) ? ol + l : l + ol;
    }
    const float inv = 1.0f / l;
    for (int t = lane; t < p.parts_per_row; t += 32) factor[t] *= inv;
    // optional row statistics (row max, sum of exp(y - max)): what a combine over column shards needs
    if (lane == 0 && p.out) reinterpret_cast<float2*>(p.out)[row] = make_float2(a, l);
  }
  __syncthreads();
  T* y = static_cast<T*>(p.Y) + (long long)bt * p.bsy + (long long)m * p.ldy;
  constexpr int V = 16 / (int)sizeof(T);   // elements per 16-byte access; N is a multiple of V
  // Slot boundaries are multiples of 16 columns, so the V elements of one access share a factor.
  auto scale_vec = [&](uint4 raw, float f) {
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
    return raw;
  };
  if constexpr (sizeof(T) == 2) {
    // bf16 rows that start on a 32-byte boundary: 256-bit accesses (16 elements, still inside one slot)
    if ((reinterpret_cast<uintptr_t>(y) & 31u) == 0 && p.N % 16 == 0) {
      for (int c = threadIdx.x * 16; c < p.N; c += blockDim.x * 16) {
        uint32_t w[8];
        asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                     : "l"(y + c)
                     : "memory");
        const float f = factor[part_slot(c, p.tile_n, p.half_n, p.slots_per_tile)];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          __nv_bfloat162 r = __floats2bfloat162_rn(__uint_as_float(w[j] << 16) * f, __uint_as_float(w[j] & 0xffff0000u) * f);
          w[j] = *reinterpret_cast<uint32_t*>(&r);
        }
        asm volatile("st.global.cs.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(y + c), "r"(w[0]), "r"(w[1]), "r"(w[2]),
                     "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                     : "memory");
      }
      return;
    }
  }
  const int stride = blockDim.x * V;
  int c = threadIdx.x * V;
  for (; c + stride < p.N; c += 2 * stride) {   // two independent 16-byte accesses in flight per thread
    const uint4 a0 = *reinterpret_cast<const uint4*>(y + c);
    const uint4 a1 = *reinterpret_cast<const uint4*>(y + c + stride);
    const float f0 = factor[part_slot(c, p.tile_n, p.half_n, p.slots_per_tile)];
    const float f1 = factor[part_slot(c + stride, p.tile_n, p.half_n, p.slots_per_tile)];
    *reinterpret_cast<uint4*>(y + c) = scale_vec(a0, f0);
    *reinterpret_cast<uint4*>(y + c + stride) = scale_vec(a1, f1);
  }
  if (c < p.N) {
    const uint4 a0 = *reinterpret_cast<const uint4*>(y + c);
    *reinterpret_cast<uint4*>(y + c) = scale_vec(a0, factor[part_slot(c, p.tile_n, p.half_n, p.slots_per_tile)]);
  }
}

// Softmax, second pass after the CUDA-core main kernel: waits for that kernel to end, then one CTA per row,
// last rows first (the main kernel writes rows in ascending order, so the rows written last are the ones
// still in L2).
template <typename T>
__global__ void __launch_bounds__(256) normalise_kernel(const Params p) {
  extern __shared__ float factor[];   // [parts_per_row]
  let_next_kernel_start();
  wait_for_prior_kernel();
  normalise_row<T>(p, (long long)gridDim.x - 1 - blockIdx.x, factor);
}

// Softmax, second pass beside the tcgen05 main kernel.  This kernel is launched as the main kernel's
// programmatic dependent and does not wait for it to end: its CTAs start once every CTA of the main kernel
// has started (or ended), find room next to them on the SMs (40 registers a thread, 16 bytes of shared
// memory: two CTAs fit beside a main-kernel CTA), and rescale each block of rows as soon as the main kernel
// has published it (p.done), while the stored exponentials are still in L2.  The second pass then costs no
// DRAM read and hides behind the main kernel, except for the rows of the main kernel's last tiles.  The
// main kernel never waits for this one, so the wait below always ends; it is bounded all the same (about a
// second, or as soon as the status word shows that something gave up), after which the CTA leaves its row
// untouched.
//
// A CTA per row, rows in ascending order (the order in which the main kernel finishes them).  Thread 0 polls
// the row block's counter with acquire loads.  Then every thread issues the loads of its part of the row
// BEFORE the row's statistics exist (they do not depend on them), warp 0 merges the row's partial pairs
// (lanes stride over them, fixed shuffle tree: bit-identical from run to run) and broadcasts (m_row, 1 / l_row),
// and each thread rescales what it loaded by exp(m_slot - m_row) / l_row, the slot's pair coming from L1.
// The next kernel in the stream is let in only when a CTA is done: until then the rows of the main kernel's
// last tiles have the SMs to themselves (that tail is the one part of this pass that nothing hides).
// The last CTA to finish zeroes the counters for the next run.
constexpr long long kChaseWaitCycles = 2000000000LL;   // about one second at ~2 GHz
constexpr int kChaseThreads = 256;

__device__ __forceinline__ unsigned int load_acquire(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t scale_bf16x2(uint32_t w, float f) {
  __nv_bfloat162 r = __floats2bfloat162_rn(__uint_as_float(w << 16) * f, __uint_as_float(w & 0xffff0000u) * f);
  return *reinterpret_cast<uint32_t*>(&r);
}

template <typename T>
__global__ void __launch_bounds__(kChaseThreads) normalise_chase_kernel(const Params p) {
  __shared__ int flag;
  __shared__ float stat[2];   // (m_row, 1 / l_row)
  const int lane = threadIdx.x & 31;
  const long long row = blockIdx.x;
  if (threadIdx.x == 0) {
    const long long unit = (row / p.M) * p.tiles_m + (row % p.M) / (kUmmaTileM * p.cta_pair);
    int ok = 1;
    if (load_acquire(p.done + unit) < p.done_target) {
      const long long t0 = clock64();
      for (unsigned int ns = 128;; ns = ns < 1024 ? 2 * ns : ns) {
        __nanosleep(ns);
        if (load_acquire(p.done + unit) >= p.done_target) break;
        if (*reinterpret_cast<volatile int*>(p.status) != 0) { ok = 0; break; }   // the main kernel (or another CTA) gave up
        if (clock64() - t0 > kChaseWaitCycles) { atomicExch(p.status, (int)FGR_ERR_DEVICE_TIMEOUT); ok = 0; break; }
      }
    }
    flag = ok;
  }
  __syncthreads();
  if (flag) {
    const float2* src = reinterpret_cast<const float2*>(p.parts) + row * p.parts_per_row;
    const int bt = (int)(row / p.M), m = (int)(row % p.M);
    T* y = static_cast<T*>(p.Y) + (long long)bt * p.bsy + (long long)m * p.ldy;
    auto stats = [&]() {   // warp 0: (m_row, l_row) from the partial pairs
      float a = -CUDART_INF_F;
      for (int t = lane; t < p.parts_per_row; t += 32) a = fmaxf(a, src[t].x);
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
      float l = 0.0f;
      for (int t = lane; t < p.parts_per_row; t += 32) {
        const float2 v = src[t];
        if (v.x > -CUDART_INF_F) l += v.y * expf(v.x - a);
      }
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) {
        const float ol = __shfl_xor_sync(0xffffffffu, l, o);
        l = (lane & o) ? ol + l : l + ol;
      }
      if (lane == 0) {
        stat[0] = a;
        stat[1] = 1.0f / l;
        // optional row statistics (row max, sum of exp(y - max)): what a combine over column shards needs
        if (p.out) reinterpret_cast<float2*>(p.out)[row] = make_float2(a, l);
      }
    };
    auto factor_at = [&](int c) {
      const float ms = src[part_slot(c, p.tile_n, p.half_n, p.slots_per_tile)].x;
      return ms > -CUDART_INF_F ? expf(ms - stat[0]) * stat[1] : 0.0f;
    };
    constexpr int U = 2;                       // accesses in flight per thread
    bool wide = false;
    if constexpr (sizeof(T) == 2) wide = (reinterpret_cast<uintptr_t>(y) & 31u) == 0 && p.N % 16 == 0;
    bool have_stats = false;
    if (wide) {
      // bf16 rows that start on a 32-byte boundary: 256-bit accesses (16 elements, inside one slot)
      for (int c0 = threadIdx.x * 16; c0 < p.N || !have_stats; c0 += U * kChaseThreads * 16) {
        uint32_t w[U][8];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int c = c0 + u * kChaseThreads * 16;
          if (c < p.N)
            asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                         : "=r"(w[u][0]), "=r"(w[u][1]), "=r"(w[u][2]), "=r"(w[u][3]), "=r"(w[u][4]), "=r"(w[u][5]), "=r"(w[u][6]),
                           "=r"(w[u][7])
                         : "l"(y + c)
                         : "memory");
        }
        if (!have_stats) {                     // uniform across the CTA: the first trip of every thread
          if (threadIdx.x < 32) stats();
          __syncthreads();
          have_stats = true;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int c = c0 + u * kChaseThreads * 16;
          if (c < p.N) {
            const float f = factor_at(c);
#pragma unroll
            for (int j = 0; j < 8; ++j) w[u][j] = scale_bf16x2(w[u][j], f);
            asm volatile("st.global.cs.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(y + c), "r"(w[u][0]), "r"(w[u][1]),
                         "r"(w[u][2]), "r"(w[u][3]), "r"(w[u][4]), "r"(w[u][5]), "r"(w[u][6]), "r"(w[u][7])
                         : "memory");
          }
        }
      }
    } else {
      constexpr int V = 16 / (int)sizeof(T);   // elements per 16-byte access; N is a multiple of V, slot edges of 16
      for (int c0 = threadIdx.x * V; c0 < p.N || !have_stats; c0 += U * kChaseThreads * V) {
        uint4 w[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int c = c0 + u * kChaseThreads * V;
          if (c < p.N) w[u] = *reinterpret_cast<const uint4*>(y + c);
        }
        if (!have_stats) {
          if (threadIdx.x < 32) stats();
          __syncthreads();
          have_stats = true;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int c = c0 + u * kChaseThreads * V;
          if (c < p.N) {
            const float f = factor_at(c);
            if constexpr (sizeof(T) == 4) {
              float* v = reinterpret_cast<float*>(&w[u]);
#pragma unroll
              for (int j = 0; j < 4; ++j) v[j] *= f;
            } else {
              w[u].x = scale_bf16x2(w[u].x, f); w[u].y = scale_bf16x2(w[u].y, f);
              w[u].z = scale_bf16x2(w[u].z, f); w[u].w = scale_bf16x2(w[u].w, f);
            }
            *reinterpret_cast<uint4*>(y + c) = w[u];
          }
        }
      }
    }
  }
  __syncthreads();
  let_next_kernel_start();
  // finish ticket: whoever draws the last one knows that no CTA will read a counter again
  const long long units = (long long)p.batch * p.tiles_m;
  if (threadIdx.x == 0) flag = atomicAdd(p.done + units, 1u) == gridDim.x - 1 ? 1 : 0;
  __syncthreads();
  if (flag)
    for (long long u = threadIdx.x; u <= units; u += blockDim.x) p.done[u] = 0u;
}

}  // namespace

cudaError_t launch_simt(const Params& p, cudaStream_t stream) {
  dim3 grid((unsigned)p.tiles_n, (unsigned)p.tiles_m, (unsigned)p.batch);
  if (p.dtype == FGR_F32) simt_gemm_kernel<float><<<grid, 256, 0, stream>>>(p);
  else simt_gemm_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(p);
  return cudaGetLastError();
}

// Launch with programmatic stream serialization: the kernel may become resident before the kernel
// ahead of it in the stream has finished (hiding its launch latency); it calls
// wait_for_prior_kernel() before touching memory.
template <typename Kernel>
cudaError_t launch_dependent(Kernel kernel, unsigned grid, unsigned block, size_t smem, cudaStream_t stream, const Params& p) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, p);
}

cudaError_t launch_merge(const Params& p, cudaStream_t stream) {
  const long long rows = (long long)p.batch * p.M;
  // Lanes per row: few, each folding up to eight pairs (its loads are independent and go out together), so that
  // the grid stays small.  The next run's main kernel, a programmatic dependent of this one, may move in only
  // once every CTA here has started; a grid that fits beside the main kernel in one wave (two CTAs per SM) lets
  // it do so while the main kernel's CTAs are still leaving.
  const int g = merge_lanes(p.parts_per_row);
  if (g == 2) return launch_dependent(merge_kernel<2>, (unsigned)((rows + 127) / 128), 256, 0, stream, p);
  if (g == 8) return launch_dependent(merge_kernel<8>, (unsigned)((rows + 31) / 32), 256, 0, stream, p);
  return launch_dependent(merge_kernel<32>, (unsigned)((rows + 7) / 8), 256, 0, stream, p);
}

cudaError_t launch_normalise(const Params& p, cudaStream_t stream) {
  const long long rows = (long long)p.batch * p.M;
  if (p.done) {   // beside the tcgen05 main kernel
    if (p.dtype == FGR_F32) return launch_dependent(normalise_chase_kernel<float>, (unsigned)rows, kChaseThreads, 0, stream, p);
    return launch_dependent(normalise_chase_kernel<__nv_bfloat16>, (unsigned)rows, kChaseThreads, 0, stream, p);
  }
  const size_t smem = (size_t)p.parts_per_row * sizeof(float);
  if (p.dtype == FGR_F32) return launch_dependent(normalise_kernel<float>, (unsigned)rows, 256, smem, stream, p);
  return launch_dependent(normalise_kernel<__nv_bfloat16>, (unsigned)rows, 256, smem, stream, p);
}

}  // namespace fgr
