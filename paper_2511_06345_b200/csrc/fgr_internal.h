// Internal declarations shared by the host dispatcher and the kernels of the fgr library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "fgr.h"

namespace fgr {

constexpr int kStatusBytes = 256;     // head of the workspace: device status word + diagnostics
constexpr int kUmmaTileM = 128;       // rows of one tcgen05 accumulator tile (= TMEM lanes)
constexpr int kUmmaBlockK = 64;       // bf16 elements per K block = one 128-byte swizzle row
constexpr int kUmmaThreads = 320;     // warp 0 TMA producer, warp 1 MMA issuer, warps 2..9 epilogue
constexpr int kUmmaMaxStages = 12;
constexpr int kSimtTile = 64;         // SIMT path: 64 x 64 output tile per CTA
constexpr int kSmemLimit = 232448;    // 227 KB: the per-CTA opt-in maximum on sm_100

// Kernel parameters: plain values and device pointers.
struct Params {
  int batch, M, N, K;
  int dtype, act, scale_kind, reduce, write_y, bias_per_batch;
  float scale;
  long long ldx, ldw, ldy, bsx, bsw, bsy;
  const void* X;
  const void* W;
  const float* bias;
  const float* scale_vec;
  void* Y;
  const void* R;       // residual tensor [batch, M, N] in the dtype of Y, added after activation and scale; may be null
  long long ldr, bsr;  // its row and batch strides in elements
  float* out;
  float* parts;        // [batch * M][parts_per_row][2] split-N partial pairs
  int* status;         // device status word (0 = ok)
  int parts_per_row;
  int tile_n;          // N extent of one tile
  int half_n;          // tcgen05 paths: columns [0, half_n) of a tile go to slot 0, the rest to slot 1
  int slots_per_tile;  // partial pairs per (row, tile): 1 (SIMT) or 2 (tcgen05)
  int tiles_m, tiles_n;
  long long num_tiles;
  int stages;
  int ksub;            // tcgen05 paths: 64-wide K sub-blocks per ring stage (1, 2 or 4)
  int cta_pair;        // tcgen05 paths: 1 = each CTA works alone, 2 = clusters of two CTAs share 256-row tiles
  int k_plane;         // 3xTF32 path: K rounded up to 32 = width of the hi plane (the lo plane follows it)
  int w_shared;        // 1: W is one [N, K] matrix used by every batch element (bsw = 0)
  // 2-D convolution (conv_rows > 1): K is conv_rows segments of conv_kseg = S * C contiguous elements; segment r of
  // output row m starts at X row m + r * conv_width (rows of C elements); a segment is kseg_blocks 64-wide k-blocks
  int conv_rows, conv_width, conv_kseg, kseg_blocks;
  int chunk_blocks;    // 3xTF32 path: 32-wide k-blocks accumulated in tensor memory before the epilogue adds them up
  // Softmax on the tcgen05 paths: the normalise kernel runs beside the main kernel and rescales a block of rows
  // as soon as all its tiles are stored.  done[u] (in the workspace head) counts the epilogue warps that have
  // finished and published a tile of row-block unit u = tile index / tiles_n; a unit is complete at
  // done_target.  done[num_units] is the finish ticket of the normalise kernel, whose last CTA zeroes the array
  // for the next run.  Null elsewhere: the second kernel then simply waits for the first to end.
  unsigned int* done;
  unsigned int done_target;
  int head_bytes;      // workspace bytes ahead of the partial pairs: status block (+ the counters above)
};

// Column -> partial-slot mapping shared by the producers of the partials and the normalise pass.
__host__ __device__ inline int part_slot(int col, int tile_n, int half_n, int slots_per_tile) {
  int t = col / tile_n;
  int w = col - t * tile_n;
  return t * slots_per_tile + ((slots_per_tile == 2 && w >= half_n) ? 1 : 0);
}

// Number of matrix columns that partial slot `t` of a row covers (the last tile may be ragged).
__host__ __device__ inline int slot_columns(int t, int N, int tile_n, int half_n, int slots_per_tile) {
  const int tile = t / slots_per_tile, h = t - tile * slots_per_tile;
  const int begin = tile * tile_n + (h ? half_n : 0);
  int end = (slots_per_tile == 2 && h == 0) ? tile * tile_n + half_n : (tile + 1) * tile_n;
  if (end > N) end = N;
  return end > begin ? end - begin : 0;
}

// Shared-memory carve-up of the tcgen05 kernel (offsets from a 1024-byte aligned base).
struct UmmaSmem {
  int stage_bytes, sub_bytes, x_bytes, w_bytes;   // a stage is `ksub` sub-blocks of (X tile, W tile)
  int vec_off;      // bias / scale staging: [8 epilogue warps][2 vectors][128] floats
  int bar_off;      // mbarriers
  int misc_off;     // TMEM base address, abort flag
  int total;        // bytes to request (includes 1024 of alignment slack)
};
// `w_rows`: rows of the W tile one CTA loads per k-block (tile_n, or tile_n / 2 for a CTA pair).
__host__ __device__ inline UmmaSmem umma_smem_layout(int w_rows, int stages, int ksub) {
  UmmaSmem s;
  s.x_bytes = kUmmaTileM * kUmmaBlockK * 2;
  s.w_bytes = w_rows * kUmmaBlockK * 2;
  s.sub_bytes = s.x_bytes + s.w_bytes;
  s.stage_bytes = s.sub_bytes * ksub;
  s.vec_off = s.stage_bytes * stages;
  s.bar_off = s.vec_off + 8 * 2 * 128 * 4;
  s.misc_off = s.bar_off + (2 * kUmmaMaxStages + 4) * 8;
  s.total = s.misc_off + 16 + 1024;
  return s;
}

// Launchers (each enqueues on `stream` and returns the cudaError_t of the launch).
cudaError_t launch_simt(const Params& p, cudaStream_t stream);
cudaError_t launch_merge(const Params& p, cudaStream_t stream);
cudaError_t launch_normalise(const Params& p, cudaStream_t stream);
// 3xTF32 path: splits fp32 src [batch][rows][K] (strides ld, bs) into dst [batch][rows][2 * k_plane]
// = [hi | lo], hi = x rounded to tf32, lo = x - hi rounded to tf32, zero beyond K.
cudaError_t launch_split_tf32(const float* src, float* dst, int batch, int rows, int K, long long ld, long long bs,
                              int k_plane, cudaStream_t stream);
cudaError_t launch_gemv(const Params& p, int grid, int rows_per_cta, cudaStream_t stream);
int gemv_rows_per_warp(int M);
int gemv_k_chunk(int M, int K);
cudaError_t umma_prepare(int device);   // opt-in shared memory attribute, once per device
cudaError_t launch_umma(const Params& p, const void* tmap_x, const void* tmap_w, int grid, int smem_bytes,
                        cudaStream_t stream);

}  // namespace fgr
