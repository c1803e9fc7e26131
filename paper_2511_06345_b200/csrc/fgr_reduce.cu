// Stand-alone reduction over the last dimension of a matrix A[M, N]: max, sum, (max, sum),
// LogSumExp, (max, sum-exp) and softmax.  HBM-bound: every element is read once with 128-bit loads
// (softmax reads the row a second time, normally from L2, and writes P once).  G threads share a
// row (a warp for short rows, a whole CTA for long ones); each thread keeps an online
// (max, sum of 2^((v - max) log2 e)) pair and a plain sum, and a fixed shuffle / shared-memory tree
// combines them, so results repeat bit for bit.
#include <cuda_bf16.h>
#include <map>
#include <mutex>
#include <utility>
#include <math_constants.h>

#include "fgr.h"

namespace {

constexpr int kThreads = 256;
constexpr int kMaxCluster = 16;         // 8 is the portable limit; larger clusters are asked for where they pay
constexpr int kClusterThreads = 1024;   // CTAs of the cluster kernel: few CTAs, so each keeps many loads in flight
constexpr float kLog2e = 1.4426950408889634f;

struct ReduceParams {
  int M, N, kind;
  long long lda, ldp;
  const void* A;
  void* P;
  float* out;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int kElems = 4;
  __device__ static void unpack(const uint4& r, float* v) {
    v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y); v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
  }
  __device__ static void store(float* p, const float* v) { *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]); }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int kElems = 8;
  __device__ static void unpack(const uint4& r, float* v) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(w[i] << 16); v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
  }
  __device__ static void store(__nv_bfloat16* p, const float* v) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

struct State { float m, l, s; };   // max, sum of 2^((v - max) log2 e), plain sum

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {   // x + y on one lane, y + x on its partner: the same bits
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// All lanes of a warp end up with the warp's (max, sum-exp relative to that max, sum).
template <bool EXP, bool SUM>
__device__ __forceinline__ State warp_combine(State st) {
  const float m = warp_max(st.m);
  if (EXP) st.l = warp_sum(st.m > -CUDART_INF_F ? st.l * ex2((st.m - m) * kLog2e) : 0.0f);
  st.m = m;
  if (SUM) st.s = warp_sum(st.s);
  return st;
}

// One thread's share of the columns [c_lo, c_hi) of a row: four vectors per iteration, i.e. four
// independent 128-bit loads in flight.  The raw 16-byte words are kept and unpacked where they are used
// (twice for the exp kinds): that keeps the register count low enough for eight CTAs per SM, i.e. for
// enough bytes in flight.
template <typename T, int G, bool EXP, bool SUM>
__device__ __forceinline__ void accumulate(const T* a, int c_lo, int c_hi, int sub, State& st) {
  constexpr int V = Vec<T>::kElems;
  constexpr int U = 4;
  for (int c0 = c_lo + sub * V; c0 < c_hi; c0 += U * G * V) {
    uint4 raw[U];
    int nv = 0;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int c = c0 + u * G * V;
      if (c < c_hi) { raw[u] = *reinterpret_cast<const uint4*>(a + c); nv = u + 1; }
    }
    float vm = -CUDART_INF_F;
    if constexpr (sizeof(T) == 2 && !SUM) {
      // maximum of the packed pairs first (one instruction per two elements), unpacked once at the end
      __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162*>(&raw[0].x);
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (u < nv) {
          const uint32_t w[4] = {raw[u].x, raw[u].y, raw[u].z, raw[u].w};
#pragma unroll
          for (int i = 0; i < 4; ++i) m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&w[i]));
        }
      const uint32_t mb = *reinterpret_cast<const uint32_t*>(&m2);
      vm = fmaxf(__uint_as_float(mb << 16), __uint_as_float(mb & 0xffff0000u));
    } else {
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (u < nv) {
          float v[V];
          Vec<T>::unpack(raw[u], v);
#pragma unroll
          for (int j = 0; j < V; ++j) { vm = fmaxf(vm, v[j]); if (SUM) st.s += v[j]; }
        }
    }
    if (EXP) {
      const float mn = fmaxf(st.m, vm);
      const float off = mn * kLog2e;
      float l = 0.0f;
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (u < nv) {
          float v[V];
          Vec<T>::unpack(raw[u], v);
#pragma unroll
          for (int j = 0; j < V; ++j) l += ex2(fmaf(v[j], kLog2e, -off));
        }
      st.l = st.l * ex2((st.m - mn) * kLog2e) + l;
      st.m = mn;
    } else {
      st.m = fmaxf(st.m, vm);
    }
  }
}

// G = threads per row: 32 (a warp, kThreads / 32 rows per CTA) or kThreads (one row per CTA).
// EXP: the kind needs sum-exp; SUM: it needs the plain sum.
template <typename T, int G, bool EXP, bool SUM>
__global__ void __launch_bounds__(kThreads, 8) reduce_rows_kernel(const ReduceParams p) {
  constexpr int V = Vec<T>::kElems;
  constexpr int kRowsPerCta = kThreads / G;
  __shared__ State red[kThreads / 32];
  const int sub = threadIdx.x % G;
  const long long row = (long long)blockIdx.x * kRowsPerCta + threadIdx.x / G;
  const bool row_ok = row < p.M;
  const T* a = static_cast<const T*>(p.A) + (row_ok ? row : 0) * p.lda;

  State st = {-CUDART_INF_F, 0.0f, 0.0f};
  if (row_ok) accumulate<T, G, EXP, SUM>(a, 0, p.N, sub, st);
  // combine the threads of a row: inside the warp by shuffles ...
  st = warp_combine<EXP, SUM>(st);
  // ... then, for a row spread over the whole CTA, the warps in warp order
  if (G == kThreads) {
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = st;
    __syncthreads();
    if (p.kind != FGR_RED_SOFTMAX && threadIdx.x != 0) return;   // only softmax needs the row's pair in every thread
    float m = red[0].m;
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) m = fmaxf(m, red[w].m);
    float l = 0.0f, sum = 0.0f;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) {
      if (EXP) l += red[w].m > -CUDART_INF_F ? red[w].l * ex2((red[w].m - m) * kLog2e) : 0.0f;
      sum += red[w].s;
    }
    st.m = m; st.l = l; st.s = sum;
  }
  if (!row_ok) return;
  if (sub == 0) {
    switch (p.kind) {
      case FGR_RED_LSE: p.out[row] = st.m + logf(st.l); break;
      case FGR_RED_MAXSUM: reinterpret_cast<float2*>(p.out)[row] = make_float2(st.m, st.s); break;
      case FGR_RED_MAX_SUMEXP: reinterpret_cast<float2*>(p.out)[row] = make_float2(st.m, st.l); break;
      case FGR_REDUCE_MAX: p.out[row] = st.m; break;
      case FGR_REDUCE_SUM: p.out[row] = st.s; break;
      default: break;
    }
  }
  if (p.kind == FGR_RED_SOFTMAX) {
    // second pass: the row was read a moment ago, so it normally comes from L2
    T* dst = static_cast<T*>(p.P) + row * p.ldp;
    const float inv = 1.0f / st.l;
    for (int c = sub * V; c < p.N; c += G * V) {
      float v[V];
      Vec<T>::unpack(*reinterpret_cast<const uint4*>(a + c), v);
#pragma unroll
      for (int j = 0; j < V; ++j) v[j] = ex2((v[j] - st.m) * kLog2e) * inv;
      Vec<T>::store(dst + c, v);
    }
  }
}

// Few, long rows: a row per CTA would leave most SMs idle, so a thread-block cluster of CL CTAs shares a
// row.  CTA r reduces the r-th segment of the columns as above, then the CL per-CTA states are exchanged
// through distributed shared memory: every CTA stores its state into slot r of the array in each CTA
// that needs it (all of them for softmax, the first otherwise), a cluster barrier orders the stores
// before the reads, and the states are folded in rank order (bit-identical from run to run).  No
// global scratch memory, one launch.
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void store_remote(const float* local, uint32_t cta, float v) {
  uint32_t laddr = (uint32_t)__cvta_generic_to_shared(local), raddr;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(laddr), "r"(cta));
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(raddr), "f"(v) : "memory");
}
__device__ __forceinline__ int cluster_ctas() {
  uint32_t n;
  asm("mov.u32 %0, %%cluster_nctaid.x;" : "=r"(n));
  return (int)n;
}
template <typename T, bool EXP, bool SUM>
__global__ void __launch_bounds__(kClusterThreads, 2) reduce_rows_cluster_kernel(const ReduceParams p) {
  constexpr int V = Vec<T>::kElems;
  __shared__ State red[kClusterThreads / 32];
  __shared__ State peers[kMaxCluster];
  const int CL = cluster_ctas();                       // CTAs per row: any size from 1 to kMaxCluster
  const int rank = (int)(blockIdx.x % CL);            // = the CTA's rank in its cluster (cluster dims CL x 1 x 1)
  const long long row = blockIdx.x / CL;              // the grid is exactly M * CL CTAs
  const T* a = static_cast<const T*>(p.A) + row * p.lda;
  const int seg = ((p.N / V + CL - 1) / CL) * V;      // columns per CTA, a multiple of the vector width
  const int c_lo = rank * seg < p.N ? rank * seg : p.N;
  const int c_hi = c_lo + seg < p.N ? c_lo + seg : p.N;

  State st = {-CUDART_INF_F, 0.0f, 0.0f};
  accumulate<T, kClusterThreads, EXP, SUM>(a, c_lo, c_hi, threadIdx.x, st);
  st = warp_combine<EXP, SUM>(st);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = st;
  __syncthreads();
  const bool softmax = p.kind == FGR_RED_SOFTMAX;
  if (threadIdx.x == 0) {
    float m = red[0].m;
#pragma unroll
    for (int w = 1; w < kClusterThreads / 32; ++w) m = fmaxf(m, red[w].m);
    float l = 0.0f, sum = 0.0f;
#pragma unroll
    for (int w = 0; w < kClusterThreads / 32; ++w) {
      if (EXP) l += red[w].m > -CUDART_INF_F ? red[w].l * ex2((red[w].m - m) * kLog2e) : 0.0f;
      sum += red[w].s;
    }
    for (int r = 0; r < (softmax ? CL : 1); ++r) {
      store_remote(&peers[rank].m, (uint32_t)r, m);
      store_remote(&peers[rank].l, (uint32_t)r, l);
      store_remote(&peers[rank].s, (uint32_t)r, sum);
    }
  }
  cluster_barrier();                                   // every thread of every CTA of the cluster
  if (!softmax && (rank != 0 || threadIdx.x != 0)) return;
  float m = peers[0].m;
  for (int r = 1; r < CL; ++r) m = fmaxf(m, peers[r].m);
  float l = 0.0f, sum = 0.0f;
  for (int r = 0; r < CL; ++r) {
    if (EXP) l += peers[r].m > -CUDART_INF_F ? peers[r].l * ex2((peers[r].m - m) * kLog2e) : 0.0f;
    sum += peers[r].s;
  }
  switch (p.kind) {
    case FGR_RED_LSE: p.out[row] = m + logf(l); break;
    case FGR_RED_MAXSUM: reinterpret_cast<float2*>(p.out)[row] = make_float2(m, sum); break;
    case FGR_RED_MAX_SUMEXP: reinterpret_cast<float2*>(p.out)[row] = make_float2(m, l); break;
    case FGR_REDUCE_MAX: p.out[row] = m; break;
    case FGR_REDUCE_SUM: p.out[row] = sum; break;
    default: break;
  }
  if (softmax) {
    // second pass over this CTA's own segment, from its end to its start: what was read last is the most
    // likely to be in L2 still (the matrix as a whole may exceed it); four vectors per iteration in flight
    T* dst = static_cast<T*>(p.P) + row * p.ldp;
    const float inv = 1.0f / l;
    constexpr int kStep = kClusterThreads * V;
    const int iters = (c_hi - c_lo + 4 * kStep - 1) / (4 * kStep);
    for (int it = iters - 1; it >= 0; --it) {
      const int c0 = c_lo + it * 4 * kStep + threadIdx.x * V;
      uint4 raw[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (c0 + u * kStep < c_hi) raw[u] = *reinterpret_cast<const uint4*>(a + c0 + u * kStep);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (c0 + u * kStep < c_hi) {
          float v[V];
          Vec<T>::unpack(raw[u], v);
#pragma unroll
          for (int j = 0; j < V; ++j) v[j] = ex2((v[j] - m) * kLog2e) * inv;
          Vec<T>::store(dst + c0 + u * kStep, v);
        }
    }
  }
}

template <typename Kernel>
cudaError_t launch_cluster(Kernel kernel, unsigned grid, int cl, const ReduceParams& p, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kClusterThreads);
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)cl;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, p);
}

// How many clusters of cl CTAs of this kernel the current device can hold at once (0 if it cannot place
// one).  Sizes above 8 are beyond the portable limit: the kernel opts in first.  Both the opt-in and the
// occupancy answer belong to one device, so they are asked once per (device, kernel) and size, with that
// device current (the caller has made it so).
int max_active_clusters(void (*kernel)(ReduceParams), int cl) {
  struct Entry { bool opted_in; int n[kMaxCluster + 1]; };   // n: 0 = not asked yet, -1 = none
  static std::map<std::pair<int, void (*)(ReduceParams)>, Entry> table;
  static std::mutex mu;
  if (cl < 1 || cl > kMaxCluster) return 0;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return 0; }
  std::lock_guard<std::mutex> lock(mu);
  Entry& e = table[std::make_pair(device, kernel)];            // value-initialised on first use
  if (!e.opted_in) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
      cudaGetLastError();
      return 0;
    }
    e.opted_in = true;
  }
  if (e.n[cl] == 0) {
    e.n[cl] = -1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)cl);
    cfg.blockDim = dim3(kClusterThreads);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cl;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) == cudaSuccess && n >= 1) e.n[cl] = n;
    cudaGetLastError();
  }
  return e.n[cl] > 0 ? e.n[cl] : 0;
}

// Whether the cluster kernels (CTAs of 1024 threads, one or several per row) take a matrix of M rows of N
// elements of V per 16 bytes: the rows are too few to fill the machine with a 256-thread CTA each (fewer
// than two per SM) and long enough to give every thread of two such CTAs a full iteration (four vectors).
// Softmax, which walks its row twice, keeps the 1024-thread CTA (one per row) up to 1024 rows: on rows of
// 64 Ki to 900 Ki bf16 elements it took 70 us against 114 at 296 rows, 69 against 82 at 560, 65 against 70
// at 900, while the one-pass kinds are level with the 256-thread kernel from about 300 rows on.
bool few_long_rows(int M, int N, int V, bool softmax) {
  return M < (softmax ? 1024 : 2 * 148) && (long long)N >= 2LL * kClusterThreads * V * 4;
}

// CTAs per row for those kernels: as many as keep the grid at about 256 CTAs in one wave, every thread with
// a full iteration, and all M clusters resident together.  Measured on 64 Mi bf16 elements in 1 to 295 rows
// (LogSumExp and max + sum; the plain maximum is flat): the time falls with the cluster size up to exactly
// these limits and jumps by 20 to 40 % past them; 8 CTAs per row throughout took up to 1.8 times as long
// (256 rows), 16 wherever the device allows it up to 1.3 times (16 rows).
int cluster_size(void (*kernel)(ReduceParams), int M, int N, int V) {
  int cl = 256 / M < kMaxCluster ? 256 / M : kMaxCluster;
  if (cl < 1) cl = 1;
  while (cl > 2 && (long long)N < (long long)cl * kClusterThreads * V * 4) --cl;
  while (cl > 8 && max_active_clusters(kernel, cl) < M) --cl;   // 8 is the portable limit, always placeable
  return cl;
}

// (mean, population variance) of every row.  Each thread accumulates sum (v - c) and sum (v - c)^2
// over its elements, c being the first element it sees (a shift inside the data's range, so the
// final  M2 = sum d^2 - (sum d)^2 / n  cancels only mildly; E[v^2] - E[v]^2 of the raw values is never
// formed and a large common offset costs no accuracy).  Four instructions per element and no
// division in the loop.  The threads of a row are then combined by fixed shuffle / shared-memory sums.
struct Moments { float n, mean, m2; };
template <typename T, int G>
__global__ void __launch_bounds__(kThreads, 8) meanvar_rows_kernel(const ReduceParams p) {
  constexpr int V = Vec<T>::kElems;
  constexpr int kRowsPerCta = kThreads / G;
  __shared__ Moments red[kThreads / 32];
  const int sub = threadIdx.x % G, lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * kRowsPerCta + threadIdx.x / G;
  const bool row_ok = row < p.M;
  const T* a = static_cast<const T*>(p.A) + (row_ok ? row : 0) * p.lda;
  Moments st = {0.0f, 0.0f, 0.0f};
  if (row_ok && sub * V < p.N) {
    float shift = 0.0f, s1 = 0.0f, s2 = 0.0f;
    int cnt = 0;
    for (int c0 = sub * V; c0 < p.N; c0 += 4 * G * V) {
      uint4 raw[4];
      int nv = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = c0 + u * G * V;
        if (c < p.N) { raw[u] = *reinterpret_cast<const uint4*>(a + c); nv = u + 1; }
      }
      if (cnt == 0) shift = __uint_as_float(sizeof(T) == 4 ? raw[0].x : raw[0].x << 16);   // the thread's first element
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (u < nv) {
          float v[V];
          Vec<T>::unpack(raw[u], v);
#pragma unroll
          for (int j = 0; j < V; ++j) { const float d = v[j] - shift; s1 += d; s2 = fmaf(d, d, s2); }
        }
      cnt += nv * V;
    }
    st.n = (float)cnt;
    const float md = s1 / st.n;
    st.mean = shift + md;
    st.m2 = fmaxf(s2 - s1 * md, 0.0f);
  }
  // Combine the threads of a warp without a chain of pairwise updates: the warp mean is the count-
  // weighted mean of the thread means, and by the parallel-axis identity
  //   M2 = sum_i [ M2_i + n_i (mean_i - mean)^2 ]   (all terms non-negative: nothing cancels).
  const float cn = warp_sum(st.n), cs = warp_sum(st.n * st.mean);
  const float wmean = cn > 0.0f ? cs / cn : 0.0f;
  const float dm = st.mean - wmean;
  const float q = warp_sum(fmaf(st.n * dm, dm, st.m2));
  Moments row_m = {cn, wmean, q};
  if (G == kThreads) {
    // a row spread over the CTA: thread 0 folds the eight warp triples, in warp order, with the pairwise update
    //   delta = mean_b - mean_a;  mean = mean_a + delta n_b / n;  M2 = M2_a + M2_b + delta^2 n_a n_b / n
    if (lane == 0) red[threadIdx.x >> 5] = row_m;
    __syncthreads();
    if (threadIdx.x != 0) return;
    row_m = red[0];
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) {
      const Moments b = red[w];
      const float tot = row_m.n + b.n;
      if (tot > 0.0f) {
        const float delta = b.mean - row_m.mean, wb = b.n / tot;
        row_m.m2 = row_m.m2 + b.m2 + delta * delta * (row_m.n * wb);
        row_m.mean = fmaf(delta, wb, row_m.mean);
        row_m.n = tot;
      }
    }
  }
  if (row_ok && sub == 0) reinterpret_cast<float2*>(p.out)[row] = make_float2(row_m.mean, row_m.m2 / (float)p.N);
}

// Mean / variance of few, long rows: the cluster form of the kernel above.  CTA r of a cluster of CL
// reduces the r-th column segment to (count, mean, M2), stores the triple into slot r of the first
// CTA's shared memory, and after the cluster barrier the first CTA folds the CL triples in rank order.
__device__ __forceinline__ Moments fold(Moments a, Moments b) {
  const float tot = a.n + b.n;
  if (tot <= 0.0f) return a;
  const float delta = b.mean - a.mean, wb = b.n / tot;
  return {tot, fmaf(delta, wb, a.mean), a.m2 + b.m2 + delta * delta * (a.n * wb)};
}
template <typename T>
__global__ void __launch_bounds__(kClusterThreads, 2) meanvar_rows_cluster_kernel(const ReduceParams p) {
  constexpr int V = Vec<T>::kElems;
  constexpr int G = kClusterThreads;
  __shared__ Moments red[kClusterThreads / 32];
  __shared__ Moments peers[kMaxCluster];
  const int CL = cluster_ctas();                       // CTAs per row: any size from 1 to kMaxCluster
  const int rank = (int)(blockIdx.x % CL), lane = threadIdx.x & 31, sub = threadIdx.x;
  const long long row = blockIdx.x / CL;
  const T* a = static_cast<const T*>(p.A) + row * p.lda;
  const int seg = ((p.N / V + CL - 1) / CL) * V;
  const int c_lo = rank * seg < p.N ? rank * seg : p.N;
  const int c_hi = c_lo + seg < p.N ? c_lo + seg : p.N;
  Moments st = {0.0f, 0.0f, 0.0f};
  if (c_lo + sub * V < c_hi) {
    float shift = 0.0f, s1 = 0.0f, s2 = 0.0f;
    int cnt = 0;
    for (int c0 = c_lo + sub * V; c0 < c_hi; c0 += 4 * G * V) {
      uint4 raw[4];
      int nv = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int c = c0 + u * G * V;
        if (c < c_hi) { raw[u] = *reinterpret_cast<const uint4*>(a + c); nv = u + 1; }
      }
      if (cnt == 0) shift = __uint_as_float(sizeof(T) == 4 ? raw[0].x : raw[0].x << 16);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (u < nv) {
          float v[V];
          Vec<T>::unpack(raw[u], v);
#pragma unroll
          for (int j = 0; j < V; ++j) { const float d = v[j] - shift; s1 += d; s2 = fmaf(d, d, s2); }
        }
      cnt += nv * V;
    }
    st.n = (float)cnt;
    const float md = s1 / st.n;
    st.mean = shift + md;
    st.m2 = fmaxf(s2 - s1 * md, 0.0f);
  }
  const float cn = warp_sum(st.n), cs = warp_sum(st.n * st.mean);
  const float wmean = cn > 0.0f ? cs / cn : 0.0f;
  const float dm = st.mean - wmean;
  const float q = warp_sum(fmaf(st.n * dm, dm, st.m2));
  if (lane == 0) red[threadIdx.x >> 5] = {cn, wmean, q};
  __syncthreads();
  if (threadIdx.x == 0) {
    Moments m = red[0];
#pragma unroll
    for (int w = 1; w < kClusterThreads / 32; ++w) m = fold(m, red[w]);
    store_remote(&peers[rank].n, 0u, m.n);
    store_remote(&peers[rank].mean, 0u, m.mean);
    store_remote(&peers[rank].m2, 0u, m.m2);
  }
  cluster_barrier();                                   // every thread of every CTA of the cluster
  if (rank != 0 || threadIdx.x != 0) return;
  Moments m = peers[0];
  for (int r = 1; r < CL; ++r) m = fold(m, peers[r]);
  reinterpret_cast<float2*>(p.out)[row] = make_float2(m.mean, m.m2 / (float)p.N);
}

template <typename T>
cudaError_t launch(const ReduceParams& p, cudaStream_t s) {
  const bool exp_kind = p.kind == FGR_RED_LSE || p.kind == FGR_RED_SOFTMAX || p.kind == FGR_RED_MAX_SUMEXP;
  const bool warp_rows = p.N <= 32 * Vec<T>::kElems * 8;   // a warp covers the row in at most two iterations
  const unsigned grid = warp_rows ? (unsigned)((p.M + kThreads / 32 - 1) / (kThreads / 32)) : (unsigned)p.M;
  const bool sum_kind = p.kind == FGR_RED_MAXSUM || p.kind == FGR_REDUCE_SUM;
  if (p.kind == FGR_RED_MEANVAR) {
    if (few_long_rows(p.M, p.N, Vec<T>::kElems, false)) {
      const int mcl = cluster_size(meanvar_rows_cluster_kernel<T>, p.M, p.N, Vec<T>::kElems);
      return launch_cluster(meanvar_rows_cluster_kernel<T>, (unsigned)p.M * (unsigned)mcl, mcl, p, s);
    }
    if (warp_rows) meanvar_rows_kernel<T, 32><<<grid, kThreads, 0, s>>>(p);
    else meanvar_rows_kernel<T, kThreads><<<grid, kThreads, 0, s>>>(p);
    return cudaGetLastError();
  }
  if (few_long_rows(p.M, p.N, Vec<T>::kElems, p.kind == FGR_RED_SOFTMAX)) {
    void (*kernel)(ReduceParams) = exp_kind   ? reduce_rows_cluster_kernel<T, true, false>
                                   : sum_kind ? reduce_rows_cluster_kernel<T, false, true>
                                              : reduce_rows_cluster_kernel<T, false, false>;
    const int want = cluster_size(kernel, p.M, p.N, Vec<T>::kElems);
    return launch_cluster(kernel, (unsigned)p.M * (unsigned)want, want, p, s);
  }
#define FGR_REDUCE_LAUNCH(Gv) \
  do { \
    if (exp_kind) reduce_rows_kernel<T, Gv, true, false><<<grid, kThreads, 0, s>>>(p); \
    else if (sum_kind) reduce_rows_kernel<T, Gv, false, true><<<grid, kThreads, 0, s>>>(p); \
    else reduce_rows_kernel<T, Gv, false, false><<<grid, kThreads, 0, s>>>(p); \
  } while (0)
  if (warp_rows) FGR_REDUCE_LAUNCH(32);
  else FGR_REDUCE_LAUNCH(kThreads);
#undef FGR_REDUCE_LAUNCH
  return cudaGetLastError();
}

}  // namespace

extern "C" int fgr_reduce_rows(const fgr_reduce_desc* d, const void* A, void* P, float* out, void* cuda_stream) {
  if (!d || d->struct_bytes != sizeof(fgr_reduce_desc) || !A) return FGR_ERR_INVALID_ARG;
  if (d->dtype != FGR_F32 && d->dtype != FGR_BF16) return FGR_ERR_INVALID_ARG;
  if (d->reduce < FGR_RED_LSE || d->reduce > FGR_RED_MEANVAR) return FGR_ERR_INVALID_ARG;
  if (d->M < 1 || d->N < 1 || d->device < 0 || d->lda < 0 || d->ldp < 0) return FGR_ERR_INVALID_ARG;
  const int g = d->dtype == FGR_F32 ? 4 : 8;   // elements per 16 bytes
  const long long lda = d->lda ? d->lda : d->N, ldp = d->ldp ? d->ldp : d->N;
  if (lda < d->N || ldp < d->N) return FGR_ERR_INVALID_ARG;
  if (d->N % g || lda % g || ldp % g) return FGR_ERR_UNSUPPORTED;
  const bool softmax = d->reduce == FGR_RED_SOFTMAX;
  if (softmax ? !P : !out) return FGR_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(A) & 15u) || (softmax && (reinterpret_cast<uintptr_t>(P) & 15u)) ||
      (out && (reinterpret_cast<uintptr_t>(out) & 7u)))
    return FGR_ERR_INVALID_ARG;
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != d->device && cudaSetDevice(d->device) != cudaSuccess) { cudaGetLastError(); return FGR_ERR_CUDA; }
  ReduceParams p = {d->M, d->N, d->reduce, lda, ldp, A, P, out};
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e = d->dtype == FGR_F32 ? launch<float>(p, s) : launch<__nv_bfloat16>(p, s);
  if (prev != d->device && prev >= 0) cudaSetDevice(prev);
  if (e != cudaSuccess) { cudaGetLastError(); return FGR_ERR_CUDA; }
  return FGR_OK;
}
