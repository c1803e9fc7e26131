// tcgen05 path of the fgr library (bf16 inputs, fp32 accumulation in tensor memory): the kernel
// template.  Activation, scaling, reduction kind and the Y store are compile-time parameters, so
// the epilogue of each variant is a straight line of a few instructions per element.
//
// One persistent CTA per SM, 10 warps with fixed roles:
//   warp 0      TMA producer: X and W k-blocks (64 bf16 = one 128-byte swizzled row per matrix row)
//               into a ring of shared-memory stages, completion on "full" mbarriers;
//   warp 1      MMA issuer: one thread issues tcgen05.mma (128 x tile_n x 16 per instruction) into
//               one of two TMEM accumulator buffers; tcgen05.commit releases ring stages ("empty")
//               and publishes finished accumulators ("tmem_full");
//   warps 2..9  epilogue: tcgen05.ld of the accumulator (thread = one output row, 32 TMEM lanes per
//               warp, two warps share a lane quadrant and split the tile's columns), bias +
//               activation + scale in registers, running row reduction, optional bf16 store, one
//               partial pair per (row, tile half) to the workspace, then "tmem_empty".
// The epilogue of tile i overlaps the mainloop of tile i + 1 through the two accumulator buffers.
//
// Every mbarrier wait is bounded: after about a second it records FGR_ERR_DEVICE_TIMEOUT in the
// device status word, raises a CTA-wide abort flag that all other waits observe, and the CTA drains
// (waits, bounded, for TMA copies still in flight), frees its tensor memory and returns.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include <type_traits>

#include "fgr_internal.h"

namespace fgr {
namespace umma {

constexpr uint32_t kTmemCols = 512;
constexpr int kChunk = 16;                       // accumulator columns per tcgen05.ld
constexpr long long kWaitCycles = 2000000000LL;  // about one second at ~2 GHz
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false if the CTA is aborting (this wait or another one timed out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 63u) == 0u) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) {
        *abort_flag = 1;
        atomicExch(status, (int)FGR_ERR_DEVICE_TIMEOUT);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tcgen05_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tcgen05_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tcgen05_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate; `accumulate` = 0 overwrites D.
__device__ __forceinline__ void tcgen05_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same with tf32 operands (fp32 words whose low 13 mantissa bits the tensor core ignores), K = 8.
__device__ __forceinline__ void tcgen05_mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp gets lane (base + i), register j =
// column j.  The load is asynchronous: tcgen05_wait_ld() must precede the first use of r.
__device__ __forceinline__ void tcgen05_ld16_issue(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tcgen05_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// ---- CTA pairs (cluster of two CTAs driving one tcgen05.mma.cta_group::2).  Within a cluster of
// two, a shared-memory address of the odd CTA differs from the same offset in the even CTA by
// bit 24; clearing it names the even (leader) CTA's copy.
constexpr uint32_t kPeerBitMask = 0xFEFFFFFFu;
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// TMA load whose completion bytes are counted on the LEADER CTA's mbarrier (same offset as `bar`).
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar & kPeerBitMask)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar & kPeerBitMask) : "memory");
}
__device__ __forceinline__ void tcgen05_alloc_pair(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tcgen05_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tcgen05_dealloc_pair(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// Arrives (once all MMAs issued so far have completed) on the barrier at this offset in BOTH CTAs.
__device__ __forceinline__ void tcgen05_commit_pair(uint32_t bar) {
  asm volatile(
      "{\n\t.reg .b16 m;\n\tmov.b16 m, 3;\n\t"
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], m;\n\t}"
      ::"r"(bar)
      : "memory");
}
// D (256 rows: 128 in each CTA's tensor memory) (+)= A (128 rows from each CTA) * B^T (tile_n / 2 rows from each CTA)
__device__ __forceinline__ void tcgen05_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                      uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tcgen05_mma_tf32_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                      uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Release / acquire fence at device scope (lighter than __threadfence(), the sequentially consistent one).
__device__ __forceinline__ void fence_acq_rel_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// Shared-memory matrix descriptor of a K-major bf16 tile whose rows are 128 bytes, stored with the
// 128-byte swizzle (what a TMA load with the 128B swizzle mode leaves in shared memory): groups of
// 8 rows are 1024 bytes apart (stride byte offset); the leading byte offset is unused for this
// layout; descriptor version 1; layout type 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);   // start address, 16-byte units
  d |= (uint64_t)1 << 16;                     // leading byte offset (ignored for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;           // stride byte offset
  d |= (uint64_t)1 << 46;                     // version
  d |= (uint64_t)2 << 61;                     // 128-byte swizzle
  return d;
}
// Instruction descriptor: D fp32; A and B both bf16 (kind::f16, format code 1) or both tf32
// (kind::tf32, format code 2), both K-major; M = 128 (256 for a CTA pair), N = tile_n.
__device__ __forceinline__ uint32_t make_idesc(int tile_m, int tile_n, bool tf32) {
  const uint32_t fmt = tf32 ? 2u : 1u;
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(tile_n >> 3) << 17) | ((uint32_t)(tile_m >> 4) << 24);
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
template <int ACT>
__device__ __forceinline__ float activation(float u) {
  if constexpr (ACT == FGR_ACT_RELU) {
    return fmaxf(u, 0.0f);
  } else if constexpr (ACT == FGR_ACT_GELU_TANH) {
    // 0.5 u (1 + tanh t) = u / (1 + exp(-2 t)),  t = sqrt(2/pi) (u + 0.044715 u^3)
    constexpr float k = -2.0f * 0.7978845608028654f * 1.4426950408889634f;   // -2 sqrt(2/pi) log2(e)
    const float w = fmaf(k * 0.044715f, u * u, k);
    return __fdividef(u, 1.0f + ex2(u * w));
  } else if constexpr (ACT == FGR_ACT_SIGMOID) {
    return __fdividef(1.0f, 1.0f + ex2(-1.4426950408889634f * u));
  } else if constexpr (ACT == FGR_ACT_TANH) {
    // tanh u = 1 - 2 / (1 + e^(2u)); for large u the quotient underflows to 0, for very negative u it is 2
    return 1.0f - __fdividef(2.0f, 1.0f + ex2(2.0f * 1.4426950408889634f * u));
  } else if constexpr (ACT == FGR_ACT_SILU) {
    return __fdividef(u, 1.0f + ex2(-1.4426950408889634f * u));
  } else {
    return u;
  }
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 r = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&r);
}

// 16 fp32 -> 16 bf16 to global memory; the first 8 (16 bytes) always, the second 8 if `both`.  A
// 32-byte aligned pair goes out as one 256-bit store: a whole 32-byte sector per lane, which the L2
// takes as one full-sector write instead of two partial ones.
__device__ __forceinline__ void store_bf16x16(__nv_bfloat16* dst, const float* y, bool both) {
  const uint32_t w0 = pack_bf16(y[0], y[1]), w1 = pack_bf16(y[2], y[3]), w2 = pack_bf16(y[4], y[5]), w3 = pack_bf16(y[6], y[7]);
  if (both) {
    const uint32_t w4 = pack_bf16(y[8], y[9]), w5 = pack_bf16(y[10], y[11]), w6 = pack_bf16(y[12], y[13]),
                   w7 = pack_bf16(y[14], y[15]);
    if ((reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
      asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(w0), "r"(w1), "r"(w2), "r"(w3),
                   "r"(w4), "r"(w5), "r"(w6), "r"(w7)
                   : "memory");
    } else {
      *reinterpret_cast<uint4*>(dst) = make_uint4(w0, w1, w2, w3);
      *reinterpret_cast<uint4*>(dst + 8) = make_uint4(w4, w5, w6, w7);
    }
  } else {
    *reinterpret_cast<uint4*>(dst) = make_uint4(w0, w1, w2, w3);
  }
}

// 16 fp32 to global memory, the first `nv` of them (a multiple of 4) if fewer than 16 are real.
__device__ __forceinline__ void store_f32x16(float* dst, const float* y, int nv) {
#pragma unroll
  for (int q = 0; q < 4; ++q)
    if (4 * q < nv) *reinterpret_cast<float4*>(dst + 4 * q) = make_float4(y[4 * q], y[4 * q + 1], y[4 * q + 2], y[4 * q + 3]);
}

// y[0..16) += f * R[0..16): the residual tensor's elements for 16 columns of one row, of which the first nv
// (bf16: 8 or 16; fp32: a multiple of 4) are inside the matrix.
__device__ __forceinline__ void add_residual16(float* y, const __nv_bfloat16* r, int nv, float f) {
#pragma unroll
  for (int h = 0; h < 2; ++h)
    if (h == 0 || nv >= kChunk) {
      const uint4 v = *reinterpret_cast<const uint4*>(r + 8 * h);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        y[8 * h + 2 * i] = fmaf(f, __uint_as_float(w[i] << 16), y[8 * h + 2 * i]);
        y[8 * h + 2 * i + 1] = fmaf(f, __uint_as_float(w[i] & 0xffff0000u), y[8 * h + 2 * i + 1]);
      }
    }
}
__device__ __forceinline__ void add_residual16(float* y, const float* r, int nv, float f) {
#pragma unroll
  for (int q = 0; q < 4; ++q)
    if (4 * q < nv) {
      const float4 v = *reinterpret_cast<const float4*>(r + 4 * q);
      y[4 * q] = fmaf(f, v.x, y[4 * q]); y[4 * q + 1] = fmaf(f, v.y, y[4 * q + 1]);
      y[4 * q + 2] = fmaf(f, v.z, y[4 * q + 2]); y[4 * q + 3] = fmaf(f, v.w, y[4 * q + 3]);
    }
}

// Work unit t -> (batch, first row of this CTA, first column).  A unit is one 128-row tile, or for
// a CTA pair a 256-row tile of which CTA `rank` owns rows [128 rank, 128 rank + 128).
struct TileCoord { int bt, m0, n0; };
__device__ __forceinline__ TileCoord tile_coord(long long t, const Params& p, int rank) {
  TileCoord c;
  const int per_batch = p.tiles_m * p.tiles_n;
  c.bt = (int)(t / per_batch);
  const int r = (int)(t - (long long)c.bt * per_batch);
  c.m0 = (r / p.tiles_n) * (kUmmaTileM * p.cta_pair) + rank * kUmmaTileM;   // N fastest
  c.n0 = (r % p.tiles_n) * p.tile_n;
  return c;
}

// Compile-time description of one epilogue variant.
//   ACT : fgr_act          SC : multiply by the staged scale vector
//   RED : fgr_reduce       WY : store y as bf16 (softmax always stores; there WY selects the variant with a residual)
template <int ACT, bool SC, int RED, bool WY>
struct Variant {
  static constexpr bool kExp = RED == FGR_RED_LSE || RED == FGR_RED_SOFTMAX || RED == FGR_RED_MAX_SUMEXP;
  static constexpr bool kMeanVar = RED == FGR_RED_MEANVAR;
  // the residual add is compiled into every variant but plain softmax, whose WY = true twin carries it
  // (its two passes over the accumulator are the most register-hungry epilogue)
  static constexpr bool kResidual = RED != FGR_RED_SOFTMAX || WY;
  static constexpr bool kSoftmax = RED == FGR_RED_SOFTMAX;
  static constexpr bool kStoreY = WY && !kSoftmax;
  // exp kinds work in log2 units; when y itself is not stored the factor log2(e) is folded into
  // the staged scale vector (so SC is set by the host for those variants)
  static constexpr bool kFoldLog2e = kExp && !kStoreY;
};

// y (or y * log2 e when folded) of 16 accumulator columns
template <int ACT, bool SC>
__device__ __forceinline__ void apply16(const uint32_t* r, const float* bias_s, const float* scale_s, float* y) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 b = *reinterpret_cast<const float4*>(bias_s + 4 * q);
    const float bb[4] = {b.x, b.y, b.z, b.w};
    float ss[4] = {1.f, 1.f, 1.f, 1.f};
    if constexpr (SC) {
      const float4 s = *reinterpret_cast<const float4*>(scale_s + 4 * q);
      ss[0] = s.x; ss[1] = s.y; ss[2] = s.z; ss[3] = s.w;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float a = activation<ACT>(__uint_as_float(r[4 * q + j]) + bb[j]);
      y[4 * q + j] = SC ? a * ss[j] : a;
    }
  }
}

// the same from 16 fp32 sums held in registers
template <int ACT, bool SC>
__device__ __forceinline__ void apply16f(const float* z, const float* bias_s, const float* scale_s, float* y) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const float4 b = *reinterpret_cast<const float4*>(bias_s + 4 * q);
    const float bb[4] = {b.x, b.y, b.z, b.w};
    float ss[4] = {1.f, 1.f, 1.f, 1.f};
    if constexpr (SC) {
      const float4 s = *reinterpret_cast<const float4*>(scale_s + 4 * q);
      ss[0] = s.x; ss[1] = s.y; ss[2] = s.z; ss[3] = s.w;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float a = activation<ACT>(z[4 * q + j] + bb[j]);
      y[4 * q + j] = SC ? a * ss[j] : a;
    }
  }
}

// ------------------------------------------------------------------------------------------ kernel
// PAIR = false: every CTA works alone on 128 x tile_n tiles (tcgen05 cta_group::1).
// PAIR = true : the grid is launched in clusters of two CTAs that share 256 x tile_n tiles.  Each
//   CTA loads its own 128 rows of X and half (tile_n / 2 rows) of the W tile; the even CTA (the
//   leader) issues tcgen05.mma.cta_group::2, which reads both CTAs' shared memory and writes rows
//   [0, 128) of the tile to its own tensor memory and rows [128, 256) to its peer's.  Per CTA and
//   k-block that is 32 KB of operands instead of 48 KB for the same tensor work.  Barriers:
//   "full" lives in the leader (both CTAs' TMA loads count their bytes there), "empty" and
//   "tmem_full" are signalled in both CTAs by one multicast tcgen05.commit, "tmem_empty" lives in
//   the leader and collects the epilogue warps of both CTAs.
// TF32 = true: fp32 problem computed as three tf32 products (3xTF32).  The operands arrive already
//   split by split_tf32_kernel into a "hi" plane (x rounded to tf32) and a "lo" plane (x - hi), side
//   by side along K: [rows][2 * k_plane].  A ring stage holds one 32-wide k-block of all four tiles
//   (sub-block 0 = X_hi, W_hi; sub-block 1 = X_lo, W_lo) and the MMA warp accumulates
//   X_hi W_hi + X_hi W_lo + X_lo W_hi into the one fp32 accumulator; Y / P are stored as fp32.
template <int ACT, bool SC, int RED, bool WY, bool PAIR, bool TF32>
__global__ void __launch_bounds__(kUmmaThreads, 1)
umma_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w, const Params p) {
  using V = Variant<ACT, SC, RED, WY>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
  const int w_rows = PAIR ? p.tile_n / 2 : p.tile_n;       // rows of the W tile this CTA loads
  const UmmaSmem L = umma_smem_layout(w_rows, p.stages, p.ksub);

  float* vec_s = reinterpret_cast<float*>(base_ptr + L.vec_off);   // [epilogue warp][bias|scale][128]
  const uint32_t bar_base = base + L.bar_off;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kUmmaMaxStages + s); };
  auto tmem_full_bar = [&](int b) { return bar_base + 8u * (2 * kUmmaMaxStages + b); };
  auto tmem_empty_bar = [&](int b) { return bar_base + 8u * (2 * kUmmaMaxStages + 2 + b); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L.misc_off);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L.misc_off + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kstep = TF32 ? kUmmaBlockK / 2 : kUmmaBlockK * p.ksub;   // K elements per ring stage (128-byte rows)
  // (2-D convolution: conv_rows segments of kseg_blocks 64-wide k-blocks each, zero-filled at each segment's end)
  const int kblocks = p.conv_rows > 1 ? (p.conv_rows * p.kseg_blocks + p.ksub - 1) / p.ksub : (p.K + kstep - 1) / kstep;
  // 3xTF32: the tensor core truncates the fp32 accumulator once per instruction, a bias that grows
  // with the number of instructions in a chain (about 7e-9 K relative).  So a tile's K range is cut
  // into chunks of p.chunk_blocks k-blocks; each chunk is accumulated in tensor memory on its own and
  // the epilogue warps add the chunks up in registers with ordinary rounded fp32 additions.
  const int chunk_blocks = TF32 ? p.chunk_blocks : kblocks;
  const int rank = PAIR ? (int)cluster_ctarank() : 0;      // 0 = leader
  // work units are dealt round-robin to CTAs (PAIR: to clusters)
  const long long unit0 = PAIR ? (long long)(blockIdx.x >> 1) : (long long)blockIdx.x;
  const long long unit_step = PAIR ? (long long)(gridDim.x >> 1) : (long long)gridDim.x;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmap_x);
    prefetch_tensormap(&tmap_w);
    for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tmem_full_bar(b), 1); mbar_init(tmem_empty_bar(b), PAIR ? 16 : 8); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    if constexpr (PAIR) {
      tcgen05_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
      tcgen05_relinquish_pair();
    } else {
      tcgen05_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
      tcgen05_relinquish();
    }
  }
  tcgen05_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();   // the peer's barriers exist before anything signals them
  tcgen05_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Programmatic dependent launch: everything above overlapped the tail of the kernel ahead of this
  // one in the stream; from here on its results (and the workspace it was reading) are needed.  The
  // merge / normalise kernel that follows may become resident now; it waits for this grid to finish.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    // ================================================================ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      // The time from a stage's "empty" signal to its loads going out adds to every refill of the ring, so
      // whatever can be worked out before the wait is: addresses, coordinates, the byte count.  (Measured: a
      // dozen more integer instructions after the wait cost c2 and c5 4 %.)  The 2-D convolution's coordinates
      // get a loop of their own (CONV2D), so that plain GEMMs and 1-D convolutions do not pay for them.
      auto produce = [&](auto conv2d_tag) {
        constexpr bool CONV2D = decltype(conv2d_tag)::value;
        const uint32_t tx = (PAIR ? 2u : 1u) * (uint32_t)L.stage_bytes;
        const int wrow0 = PAIR ? rank * w_rows : 0;
        uint32_t s = 0, ph = 0;              // ring slot and its phase, kept incrementally
        for (long long t = unit0; t < p.num_tiles && ok; t += unit_step) {
          const TileCoord c = tile_coord(t, p, rank);
          const int wbt = p.w_shared ? 0 : c.bt;
          for (int kb = 0; kb < kblocks; ++kb, ++it) {
            const uint32_t xs = base + s * (uint32_t)L.stage_bytes;
            const uint32_t fb = full_bar((int)s);
            int kx[4], xy[4], wy[4], wz[4];  // per sub-block: K coordinate, X row, W's second and third coordinate
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if constexpr (CONV2D) {
                // k-block g of the tile lies in filter row g / kseg_blocks: its X rows are the output rows shifted
                // down by that many image rows, its W rows come from that plane of the filters [S C, R, N]
                const int g = kb * p.ksub + j, fr = g / p.kseg_blocks;
                kx[j] = (g - fr * p.kseg_blocks) * kUmmaBlockK;
                xy[j] = c.m0 + fr * p.conv_width;
                wy[j] = fr;
                wz[j] = c.n0 + wrow0;
              } else {
                kx[j] = kb * kstep + j * (TF32 ? p.k_plane : kUmmaBlockK);
                xy[j] = c.m0;
                wy[j] = c.n0 + wrow0;
                wz[j] = wbt;
              }
            }
            if (!(ok = mbar_wait(empty_bar((int)s), ph ^ 1u, abort_flag, p.status))) break;
            if (!PAIR || rank == 0) mbar_arrive_expect_tx(fb, tx);
            // The sub-blocks of a stage are adjacent in K: consecutive requests for the same matrix
            // rows ask the DRAM for neighbouring 128-byte lines (out-of-range sub-blocks read as zero).
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (j < p.ksub) {
                const uint32_t dst = xs + (uint32_t)(j * L.sub_bytes) + L.x_bytes;
                if constexpr (PAIR) tma_load_3d_pair(dst, &tmap_w, kx[j], wy[j], wz[j], fb);
                else tma_load_3d(dst, &tmap_w, kx[j], wy[j], wz[j], fb);
              }
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (j < p.ksub) {
                const uint32_t dst = xs + (uint32_t)(j * L.sub_bytes);
                if constexpr (PAIR) tma_load_3d_pair(dst, &tmap_x, kx[j], xy[j], c.bt, fb);
                else tma_load_3d(dst, &tmap_x, kx[j], xy[j], c.bt, fb);
              }
            if (++s == (uint32_t)p.stages) { s = 0; ph ^= 1u; }
          }
        }
      };
      if (!TF32 && p.conv_rows > 1) produce(std::true_type{});
      else produce(std::false_type{});
      if (!ok && !PAIR) {
        // Aborting: let the copies already issued land before the CTA gives its shared memory back.
        // (A pair ends with a cluster-wide barrier and its copies are counted in the leader, so
        // there the wait for the peer serves the same purpose.)
        const uint32_t issued = it < (uint32_t)p.stages ? it : (uint32_t)p.stages;
        for (uint32_t j = 0; j < issued; ++j) {
          const uint32_t i2 = it - 1 - j;
          const long long t0 = clock64();
          while (!mbar_try_wait(full_bar(i2 % p.stages), (i2 / p.stages) & 1u))
            if (clock64() - t0 > kWaitCycles / 8) break;
        }
      }
    }
  } else if (warp == 1) {
    // ================================================================ MMA issuer (the leader CTA of a pair)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = make_idesc(PAIR ? 2 * kUmmaTileM : kUmmaTileM, p.tile_n, TF32);
      uint32_t it = 0, tcount = 0;       // tcount counts accumulator hand-overs: tiles, or K chunks of tiles (3xTF32)
      uint32_t slot = 0, sph = 0;        // ring slot and its phase, kept incrementally
      bool ok = true;
      for (long long t = unit0; t < p.num_tiles && ok; t += unit_step)
       for (int kb0 = 0; kb0 < kblocks && ok; kb0 += chunk_blocks, ++tcount) {
        const uint32_t buf = tcount & 1u, aph = (tcount >> 1) & 1u;
        if (!(ok = mbar_wait(tmem_empty_bar(buf), aph ^ 1u, abort_flag, p.status))) break;
        tcgen05_fence_after();
        const uint32_t d = tmem_base + buf * 256u;
        const int kb1 = kb0 + chunk_blocks < kblocks ? kb0 + chunk_blocks : kblocks;
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = (int)slot;
          // descriptors of the stage's tiles before the wait: the MMAs go out the moment the operands are there
          const uint32_t xs = base + slot * (uint32_t)L.stage_bytes;
          uint64_t adesc[4], bdesc[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            adesc[j] = make_smem_desc(xs + (uint32_t)(j * L.sub_bytes));
            bdesc[j] = make_smem_desc(xs + (uint32_t)(j * L.sub_bytes) + L.x_bytes);
          }
          if (!(ok = mbar_wait(full_bar(s), sph, abort_flag, p.status))) break;
          tcgen05_fence_after();
          if (++slot == (uint32_t)p.stages) { slot = 0; sph ^= 1u; }
          if constexpr (TF32) {
            const uint64_t a_hi = adesc[0], b_hi = bdesc[0], a_lo = adesc[1], b_lo = bdesc[1];
#pragma unroll
            for (int pr = 0; pr < 3; ++pr) {               // the two small products first, then hi * hi
              const uint64_t a0 = pr == 0 ? a_lo : a_hi, b0 = pr == 1 ? b_lo : b_hi;
#pragma unroll
              for (int k = 0; k < 4; ++k) {                // 8 tf32 = 32 bytes = 2 descriptor address units
                const uint32_t acc = ((kb - kb0) | pr | k) != 0 ? 1u : 0u;
                if constexpr (PAIR) tcgen05_mma_tf32_pair(d, a0 + 2u * k, b0 + 2u * k, idesc, acc);
                else tcgen05_mma_tf32(d, a0 + 2u * k, b0 + 2u * k, idesc, acc);
              }
            }
          } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              if (j < p.ksub) {
#pragma unroll
                for (int k = 0; k < kUmmaBlockK / 16; ++k) {   // 16 bf16 = 32 bytes = 2 descriptor address units
                  const uint32_t acc = (kb | j | k) != 0 ? 1u : 0u;
                  if constexpr (PAIR) tcgen05_mma_bf16_pair(d, adesc[j] + 2u * k, bdesc[j] + 2u * k, idesc, acc);
                  else tcgen05_mma_bf16(d, adesc[j] + 2u * k, bdesc[j] + 2u * k, idesc, acc);
                }
              }
          }
          if constexpr (PAIR) tcgen05_commit_pair(empty_bar(s)); else tcgen05_commit(empty_bar(s));
        }
        if (ok) {
          if constexpr (PAIR) tcgen05_commit_pair(tmem_full_bar(buf)); else tcgen05_commit(tmem_full_bar(buf));
        }
      }
    }
  } else {
    // ================================================================ epilogue (warps 2..9)
    const int ew = warp - 2;
    const int quad = warp & 3;              // TMEM lanes a warp may read: 32 * (warp id % 4) ...
    const int half = ew >> 2;               // which part of the tile's columns
    float* bias_s = vec_s + ew * 256;       // this warp's staging: [bias | scale][128]
    float* scale_s = bias_s + 128;
    const int c_begin = half ? p.half_n : 0;
    const int c_end = half ? p.tile_n : p.half_n;
    uint32_t tcount = 0;
    bool ok = true;
    // Softmax: the normalise kernel runs beside this one and rescales a block of rows once every tile of it is
    // stored; a warp adds 1 to the count of its tile's row block.  It does so after it has waited for the
    // accumulator of its next tile (or has none left): the fence that must precede the count then finds the
    // tile's stores acknowledged, where a fence right after them stalls the warp until the last has drained.
    long long unpublished = -1;             // row-block unit of the tile this warp has stored but not yet published
    auto publish = [&]() {
      if constexpr (V::kSoftmax) {
        if (unpublished >= 0) {
          fence_acq_rel_gpu();              // every lane: its stores of that tile before the count below
          __syncwarp();
          if (lane == 0) atomicAdd(p.done + unpublished, 1u);
          unpublished = -1;
        }
      }
    };
    for (long long t = unit0; t < p.num_tiles && ok; t += unit_step, ++tcount) {
      const TileCoord c = tile_coord(t, p, rank);
      // stage the bias and scale of this warp's columns in its own slice of shared memory
      for (int i = lane; i < c_end - c_begin; i += 32) {
        const int n = c.n0 + c_begin + i;
        float b = 0.0f, s = 1.0f;
        if (n < p.N) {
          if (p.bias) b = p.bias[(p.bias_per_batch ? (long long)c.bt * p.N : 0) + n];
          if (p.scale_kind == FGR_SCALE_PER_COLUMN) s = p.scale_vec[n];
          else if (p.scale_kind == FGR_SCALE_SCALAR) s = p.scale;
        }
        bias_s[i] = b;
        if constexpr (SC) scale_s[i] = V::kFoldLog2e ? s * kLog2e : s;
      }
      __syncwarp();
      const int m = c.m0 + quad * 32 + lane;
      const bool row_ok = m < p.M;
      const int n_valid = p.N - c.n0;       // columns of this tile inside the matrix (may exceed tile_n)
      const int c_lim = c_end < n_valid ? c_end : n_valid;   // a multiple of 8 (fp32: of 4)
      uint32_t ra[kChunk], rb[kChunk];
      float y[kChunk];
      // 3xTF32: the sums of this thread's (at most 128) columns over the K chunks seen so far
      float S[TF32 ? 8 * kChunk : 1];
      if constexpr (TF32) {
#pragma unroll
        for (int i = 0; i < 8 * kChunk; ++i) S[i] = 0.0f;
        // every chunk but the last: add the chunk's accumulator to S and hand the buffer back
        for (int kb0 = 0; kb0 + chunk_blocks < kblocks; kb0 += chunk_blocks, ++tcount) {
          const uint32_t cbuf = tcount & 1u;
          ok = __all_sync(0xffffffffu, mbar_wait(tmem_full_bar(cbuf), (tcount >> 1) & 1u, abort_flag, p.status));
          if (!ok) break;
          tcgen05_fence_after();
          const uint32_t ca = tmem_base + ((uint32_t)(quad * 32) << 16) + cbuf * 256u;
#pragma unroll
          for (int q = 0; q < 8; q += 2) {
            const int cc = c_begin + kChunk * q;
            if (cc < c_lim) {
              const bool second = cc + kChunk < c_lim;
              tcgen05_ld16_issue(ca + cc, ra);
              if (second) tcgen05_ld16_issue(ca + cc + kChunk, rb);
              tcgen05_wait_ld();
#pragma unroll
              for (int j = 0; j < kChunk; ++j) S[kChunk * q + j] += __uint_as_float(ra[j]);
              if (second) {
#pragma unroll
                for (int j = 0; j < kChunk; ++j) S[kChunk * (q + 1) + j] += __uint_as_float(rb[j]);
              }
            }
          }
          tcgen05_fence_before();
          __syncwarp();
          if (lane == 0) {
            if constexpr (PAIR) mbar_arrive_leader(tmem_empty_bar(cbuf)); else mbar_arrive(tmem_empty_bar(cbuf));
          }
        }
        if (!ok) break;
      }
      const uint32_t buf = tcount & 1u, aph = (tcount >> 1) & 1u;
      ok = __all_sync(0xffffffffu, mbar_wait(tmem_full_bar(buf), aph, abort_flag, p.status));
      if (!ok) break;
      publish();   // the previous tile: its stores went out before the wait above, nothing new has been stored since
      tcgen05_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + buf * 256u;
      using OutT = typename std::conditional<TF32, float, __nv_bfloat16>::type;
      OutT* yrow = static_cast<OutT*>(p.Y) + (long long)c.bt * p.bsy + (long long)m * p.ldy + c.n0;
      // the residual row (added after activation and scale; in log2 units where the epilogue works in them)
      const OutT* rrow = p.R ? static_cast<const OutT*>(p.R) + (long long)c.bt * p.bsr + (long long)m * p.ldr + c.n0 : nullptr;
      const bool use_r = V::kResidual && rrow != nullptr && row_ok;
      constexpr float kResF = V::kFoldLog2e ? kLog2e : 1.0f;
      // is column j of a 16-column chunk with nv real columns inside the matrix?  (bf16: N is a multiple
      // of 8, so a ragged chunk has exactly 8; fp32: a multiple of 4)
      auto real = [](int j, int nv) { return TF32 ? j < nv : (j < 8 || nv >= kChunk); };
      auto store16 = [&](int cc, const float* yy, int nv) {
        if constexpr (TF32) store_f32x16(yrow + cc, yy, nv);
        else store_bf16x16(yrow + cc, yy, nv >= kChunk);
      };

      float r0 = -CUDART_INF_F, r1 = 0.0f;  // (max, sum) or (max in log2 units, sum of 2^(t - max))

      // Walks this warp's columns 32 at a time: both loads are issued before the single wait.
      // f(y, cc, nv): y = epilogue values of columns cc .. cc+15, nv = how many of them are real
      // (16 or more, or exactly 8 in the last chunk of a matrix whose N is not a multiple of 16).
      bool folded = false;                  // 3xTF32: has the last chunk been added to S yet?
      auto sweep = [&](auto&& f) {
        if constexpr (TF32) {
          // fixed trip count and static indices keep S in registers
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const int cc = c_begin + kChunk * q;
            if (cc < c_lim) {
              if (!folded) {
                tcgen05_ld16_issue(taddr + cc, ra);
                tcgen05_wait_ld();
#pragma unroll
                for (int j = 0; j < kChunk; ++j) S[kChunk * q + j] += __uint_as_float(ra[j]);
              }
              apply16f<ACT, SC>(S + kChunk * q, bias_s + kChunk * q, scale_s + kChunk * q, y);
              if (use_r) add_residual16(y, rrow + cc, c_lim - cc, kResF);
              f(y, cc, c_lim - cc);
            }
          }
          folded = true;
        }
        for (int cc = c_begin; !TF32 && cc < c_lim; cc += 2 * kChunk) {
          const bool second = cc + kChunk < c_lim;
          tcgen05_ld16_issue(taddr + cc, ra);
          if (second) tcgen05_ld16_issue(taddr + cc + kChunk, rb);
          tcgen05_wait_ld();
          apply16<ACT, SC>(ra, bias_s + (cc - c_begin), scale_s + (cc - c_begin), y);
          if (use_r) add_residual16(y, rrow + cc, c_lim - cc, kResF);
          f(y, cc, c_lim - cc);
          if (second) {
            apply16<ACT, SC>(rb, bias_s + (cc + kChunk - c_begin), scale_s + (cc + kChunk - c_begin), y);
            if (use_r) add_residual16(y, rrow + cc + kChunk, c_lim - cc - kChunk, kResF);
            f(y, cc + kChunk, c_lim - cc - kChunk);
          }
        }
      };

      if constexpr (V::kSoftmax) {
        // pass A: row maximum over this warp's columns (log2 units)
        sweep([&](float* yy, int, int nv) {
#pragma unroll
          for (int j = 0; j < kChunk; ++j) if (real(j, nv)) r0 = fmaxf(r0, yy[j]);
        });
        // pass B: exponentials relative to that maximum, their sum, and the bf16 store
        sweep([&](float* yy, int cc, int nv) {
#pragma unroll
          for (int j = 0; j < kChunk; ++j) {
            yy[j] = real(j, nv) ? ex2(yy[j] - r0) : 0.0f;
            r1 += yy[j];
          }
          if (row_ok) store16(cc, yy, nv);
        });
      } else if constexpr (V::kMeanVar) {
        // pass A: sum of this warp's columns (and the Y store); pass B: squared deviations from their mean
        sweep([&](float* yy, int cc, int nv) {
          if constexpr (V::kStoreY) {
            if (row_ok) store16(cc, yy, nv);
          }
#pragma unroll
          for (int j = 0; j < kChunk; ++j) if (real(j, nv)) r1 += yy[j];
        });
        const float mean = c_lim > c_begin ? r1 / (float)(c_lim - c_begin) : 0.0f;
        float dev = 0.0f;
        sweep([&](float* yy, int, int nv) {
#pragma unroll
          for (int j = 0; j < kChunk; ++j) if (real(j, nv)) dev = fmaf(yy[j] - mean, yy[j] - mean, dev);
        });
        r0 = mean;
        r1 = dev;
      } else {
        sweep([&](float* yy, int cc, int nv) {
          if constexpr (V::kStoreY) {
            if (row_ok) store16(cc, yy, nv);
          }
          if constexpr (V::kExp) {
            if constexpr (V::kStoreY) {
#pragma unroll
              for (int j = 0; j < kChunk; ++j) yy[j] *= kLog2e;
            }
            float cm = -CUDART_INF_F;
#pragma unroll
            for (int j = 0; j < kChunk; ++j) if (real(j, nv)) cm = fmaxf(cm, yy[j]);
            const float mn = fmaxf(r0, cm);
            float l = 0.0f;
#pragma unroll
            for (int j = 0; j < kChunk; ++j) if (real(j, nv)) l += ex2(yy[j] - mn);
            r1 = fmaf(r1, ex2(r0 - mn), l);
            r0 = mn;
          } else {
#pragma unroll
            for (int j = 0; j < kChunk; ++j) if (real(j, nv)) { r0 = fmaxf(r0, yy[j]); r1 += yy[j]; }
          }
        });
      }
      // accumulator buffer drained: hand it back to the MMA warp
      tcgen05_fence_before();
      __syncwarp();
      if (lane == 0) {
        if constexpr (PAIR) mbar_arrive_leader(tmem_empty_bar(buf)); else mbar_arrive(tmem_empty_bar(buf));
      }

      if (row_ok) {
        if constexpr (V::kExp) r0 *= kLn2;   // back to natural-log units; r1 is unchanged by the change of base
        const int tn = c.n0 / p.tile_n;
        float2* dst = reinterpret_cast<float2*>(p.parts) + ((long long)c.bt * p.M + m) * p.parts_per_row + tn * 2 + half;
        *dst = make_float2(r0, r1);
      }
      if constexpr (V::kSoftmax) {
        if (p.done) unpublished = t / p.tiles_n;                     // row block (of 128 rows, or 256 for a CTA pair)
      }
    }
    if (ok) publish();
  }

  tcgen05_fence_before();
  __syncthreads();
  if constexpr (PAIR) {
    // neither CTA may leave while its peer can still read its shared memory or signal its barriers
    cluster_sync_all();
    if (warp == 1) tcgen05_dealloc_pair(tmem_base, kTmemCols);
  } else {
    if (warp == 1) tcgen05_dealloc(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------------ host
template <int ACT, bool SC, int RED, bool WY>
cudaError_t launch_one(const Params& p, const CUtensorMap& tx, const CUtensorMap& tw, int grid, int smem, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kUmmaThreads);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see griddepcontrol in the kernel
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  const bool tf32 = p.dtype == FGR_F32;
  if (p.cta_pair == 2) {
    cfg.numAttrs = 2;
    if (tf32) return cudaLaunchKernelEx(&cfg, umma_kernel<ACT, SC, RED, WY, true, true>, tx, tw, p);
    return cudaLaunchKernelEx(&cfg, umma_kernel<ACT, SC, RED, WY, true, false>, tx, tw, p);
  }
  cfg.numAttrs = 1;
  if (tf32) return cudaLaunchKernelEx(&cfg, umma_kernel<ACT, SC, RED, WY, false, true>, tx, tw, p);
  return cudaLaunchKernelEx(&cfg, umma_kernel<ACT, SC, RED, WY, false, false>, tx, tw, p);
}
template <int ACT, bool SC, int RED, bool WY>
cudaError_t prepare_one() {
  cudaError_t e = cudaFuncSetAttribute(umma_kernel<ACT, SC, RED, WY, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(umma_kernel<ACT, SC, RED, WY, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(umma_kernel<ACT, SC, RED, WY, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(umma_kernel<ACT, SC, RED, WY, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
  return e;
}

// The variants that exist per activation.  Exp kinds that do not store y always multiply by the
// staged vector (it carries log2 e); softmax has no separate Y store.
#define FGR_UMMA_VARIANTS(X)                                                                      \
  X(false, FGR_RED_MAXSUM, false) X(false, FGR_RED_MAXSUM, true) X(true, FGR_RED_MAXSUM, false)   \
  X(true, FGR_RED_MAXSUM, true) X(true, FGR_RED_LSE, false) X(false, FGR_RED_LSE, true)           \
  X(true, FGR_RED_LSE, true) X(true, FGR_RED_MAX_SUMEXP, false) X(false, FGR_RED_MAX_SUMEXP, true) \
  X(true, FGR_RED_MAX_SUMEXP, true) X(true, FGR_RED_SOFTMAX, false) X(true, FGR_RED_SOFTMAX, true) \
  X(false, FGR_RED_MEANVAR, false) X(false, FGR_RED_MEANVAR, true) X(true, FGR_RED_MEANVAR, false) \
  X(true, FGR_RED_MEANVAR, true)

template <int ACT>
cudaError_t launch_act(bool sc, int red, bool wy, const Params& p, const CUtensorMap& tx, const CUtensorMap& tw, int grid,
                       int smem, cudaStream_t s) {
#define FGR_CASE(SCv, REDv, WYv) \
  if (sc == SCv && red == REDv && wy == WYv) return launch_one<ACT, SCv, REDv, WYv>(p, tx, tw, grid, smem, s);
  FGR_UMMA_VARIANTS(FGR_CASE)
#undef FGR_CASE
  return cudaErrorInvalidValue;
}
template <int ACT>
cudaError_t prepare_act() {
  cudaError_t e = cudaSuccess;
#define FGR_PREP(SCv, REDv, WYv) if (e == cudaSuccess) e = prepare_one<ACT, SCv, REDv, WYv>();
  FGR_UMMA_VARIANTS(FGR_PREP)
#undef FGR_PREP
  return e;
}

}  // namespace umma

// One translation unit per activation (so that they compile in parallel).
cudaError_t umma_launch_act_none(bool sc, int red, bool wy, const Params& p, const void* tx, const void* tw, int grid, int smem, cudaStream_t s);
cudaError_t umma_launch_act_relu(bool sc, int red, bool wy, const Params& p, const void* tx, const void* tw, int grid, int smem, cudaStream_t s);
cudaError_t umma_launch_act_gelu(bool sc, int red, bool wy, const Params& p, const void* tx, const void* tw, int grid, int smem, cudaStream_t s);
cudaError_t umma_launch_act_sigmoid(bool sc, int red, bool wy, const Params& p, const void* tx, const void* tw, int grid, int smem, cudaStream_t s);
cudaError_t umma_prepare_act_sigmoid();
cudaError_t umma_launch_act_tanh(bool sc, int red, bool wy, const Params& p, const void* tx, const void* tw, int grid, int smem, cudaStream_t s);
cudaError_t umma_prepare_act_tanh();
cudaError_t umma_launch_act_silu(bool sc, int red, bool wy, const Params& p, const void* tx, const void* tw, int grid, int smem, cudaStream_t s);
cudaError_t umma_prepare_act_silu();
cudaError_t umma_prepare_act_none();
cudaError_t umma_prepare_act_relu();
cudaError_t umma_prepare_act_gelu();

}  // namespace fgr
