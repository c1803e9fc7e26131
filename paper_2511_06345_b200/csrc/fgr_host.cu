// Host side of the fgr library: descriptor validation, shape -> path selection, tiling and
// workspace layout, TMA descriptor encoding, and the extern "C" entry points of include/fgr.h.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "fgr_internal.h"

using namespace fgr;

namespace {
constexpr int kHostChunks = 4;
constexpr int kMapSlots = 8;
struct MapCache {
  const void* key[kMapSlots];
  CUtensorMap map[kMapSlots];
  int next;                  // slot the next new pointer replaces (round robin)
  const CUtensorMap* find(const void* ptr) const {
    for (int i = 0; i < kMapSlots; ++i)
      if (key[i] == ptr && ptr) return &map[i];
    return nullptr;
  }
  CUtensorMap* claim(const void* ptr) {
    const int i = next;
    next = (next + 1) % kMapSlots;
    key[i] = ptr;
    return &map[i];
  }
  void forget(const void* ptr) {
    for (int i = 0; i < kMapSlots; ++i)
      if (key[i] == ptr) key[i] = nullptr;
  }
  void clear() { for (int i = 0; i < kMapSlots; ++i) key[i] = nullptr; }
};
}  // namespace

struct fgr_handle {
  fgr_desc desc;
  fgr_plan_info plan;
  Params base;               // everything but the per-run pointers
  int num_sms;
  // cached TMA descriptors (tcgen05 paths): the last kMapSlots distinct base pointers per operand, so a
  // caller that alternates between a few buffers (double buffering, a rotation) encodes each map once
  MapCache maps_x, maps_w;
  // optional residual tensor (fgr_set_residual)
  const void* residual;
  long long ldr, bsr;
  // status plumbing
  void* last_workspace;
  cudaStream_t last_stream;
  bool ran;
  // staging owned by the handle (fgr_run_host only)
  void* stage[7];
  size_t stage_bytes[7];
  cudaStream_t host_stream;
  // fgr_run_host in chunks: sub-handles for blocks of rows (or of batches), their workspaces (slices of one
  // allocation), a stream for each copy direction and the events that chain copy -> run -> copy
  fgr_handle* sub[kHostChunks];
  long long sub_first[kHostChunks + 1];   // first row (batch == 1) or first batch of each chunk
  int sub_count;                          // 0 = not planned yet, 1 = whole problem in one piece
  bool sub_by_batch;
  void* sub_ws;
  size_t sub_ws_bytes, sub_ws_off[kHostChunks];
  cudaStream_t in_stream, out_stream;
  cudaEvent_t ev_in[kHostChunks], ev_run[kHostChunks], ev_shared;
  // optional timing of the main kernel
  bool profiling;
  std::vector<cudaEvent_t>* events;   // pairs (before, after)
  size_t events_used;
};

namespace {

// Machine balance used by the selector: measured dense bf16 rate over measured HBM bandwidth of a
// B200 (about 1640 TFLOP/s over about 6.5 TB/s), in flop per byte.
constexpr double kRidgeFlopPerByte = 250.0;
constexpr int kDefaultSms = 148;
// 3xTF32: K elements accumulated inside the tensor core per chunk = 32 * kTf32ChunkBlocks.  The tensor
// core truncates its fp32 accumulator once per instruction (measured: a relative bias of about 7e-9 per
// unit of K, towards zero); 128 keeps that below 1e-6, the level of an fp32 FMA loop at K of a few thousand.
constexpr int kTf32ChunkBlocks = 4;
constexpr double kTf32MinFlop = 1.0e9;   // below this the fp32 problem stays on the CUDA-core path (measured: the two cross near 512^3)
size_t align256(size_t x) { return (x + 255u) & ~(size_t)255u; }

int elem_bytes(int dtype) { return dtype == FGR_F32 ? 4 : 2; }
int out_width(int reduce) { return reduce == FGR_RED_LSE ? 1 : reduce == FGR_RED_SOFTMAX ? 0 : 2; }

struct Resolved { long long ldx, ldw, ldy, bsx, bsw, bsy; };

// Elements of X that one batch element's M output rows read, first to last (convolutions: the signal or image).
long long x_span(const fgr_desc& d, long long ldx) {
  if (d.conv_rows > 1) {
    const int s = d.conv_taps > 1 ? d.conv_taps : 1;
    const long long c = d.K / ((long long)d.conv_rows * s);
    return ((long long)(d.M - 1) + (long long)(d.conv_rows - 1) * d.conv_width) * ldx + s * c;
  }
  return (long long)(d.M - 1) * ldx + d.K;
}

Resolved resolve_strides(const fgr_desc& d) {
  Resolved r;
  const int rows2d = d.conv_rows > 1 ? d.conv_rows : 1;   // 2-D convolution: K is rows2d segments of taps * C elements
  const int taps = (d.conv_taps > 1 ? d.conv_taps : 1) * rows2d;   // convolution: rows of the implicit matrix overlap
  r.ldx = d.ldx ? d.ldx : d.K / taps;
  r.ldw = d.ldw ? d.ldw : d.K;
  r.ldy = d.ldy ? d.ldy : d.N;
  // (a strided 1-D convolution has ldx = stride * C: its signal is (M - 1) * stride + taps samples of C channels;
  //  a 2-D one reads, for its last output row, up to filter row R - 1 below it: see x_span)
  r.bsx = d.bsx ? d.bsx : (taps > 1 ? x_span(d, r.ldx) : (long long)d.M * r.ldx);
  r.bsw = d.w_shared ? 0 : (d.bsw ? d.bsw : (long long)d.N * r.ldw);   // shared W: every batch reads the same matrix
  r.bsy = d.bsy ? d.bsy : (long long)d.M * r.ldy;
  return r;
}

int validate(const fgr_desc* d) {
  if (!d) return FGR_ERR_INVALID_ARG;
  if (d->struct_bytes != sizeof(fgr_desc)) return FGR_ERR_INVALID_ARG;
  if (d->dtype != FGR_F32 && d->dtype != FGR_BF16) return FGR_ERR_INVALID_ARG;
  if (d->act < FGR_ACT_NONE || d->act > FGR_ACT_SILU) return FGR_ERR_INVALID_ARG;
  if (d->scale_kind < FGR_SCALE_NONE || d->scale_kind > FGR_SCALE_PER_COLUMN) return FGR_ERR_INVALID_ARG;
  if ((d->reduce < FGR_RED_LSE || d->reduce > FGR_RED_MAX_SUMEXP) && d->reduce != FGR_RED_MEANVAR) return FGR_ERR_INVALID_ARG;
  if (d->force_path < FGR_PATH_AUTO || d->force_path > FGR_PATH_UMMA_TF32X3) return FGR_ERR_INVALID_ARG;
  if (d->batch < 1 || d->M < 1 || d->N < 1 || d->K < 1) return FGR_ERR_INVALID_ARG;
  if (d->write_y != 0 && d->write_y != 1) return FGR_ERR_INVALID_ARG;
  if (d->bias_per_batch != 0 && d->bias_per_batch != 1) return FGR_ERR_INVALID_ARG;
  if (d->device < 0) return FGR_ERR_INVALID_ARG;
  if (d->scale_kind == FGR_SCALE_SCALAR && !std::isfinite(d->scale)) return FGR_ERR_INVALID_ARG;
  if (d->ldx < 0 || d->ldw < 0 || d->ldy < 0 || d->bsx < 0 || d->bsw < 0 || d->bsy < 0) return FGR_ERR_INVALID_ARG;
  const int g = 16 / elem_bytes(d->dtype);   // elements per 16 bytes
  if (d->K % g || d->N % g) return FGR_ERR_UNSUPPORTED;
  if (d->conv_taps < 0 || (d->w_shared != 0 && d->w_shared != 1)) return FGR_ERR_INVALID_ARG;
  if (d->conv_rows < 0 || d->conv_width < 0) return FGR_ERR_INVALID_ARG;
  const bool conv2d = d->conv_rows > 1;
  const int taps = (d->conv_taps > 1 ? d->conv_taps : 1) * (conv2d ? d->conv_rows : 1);
  if (d->K % taps) return FGR_ERR_INVALID_ARG;
  if ((d->K / taps) % g) return FGR_ERR_UNSUPPORTED;
  if (conv2d) {
    if (d->conv_width < (d->conv_taps > 1 ? d->conv_taps : 1)) return FGR_ERR_INVALID_ARG;
    if (d->ldx != 0 && d->ldx != d->K / taps) return FGR_ERR_UNSUPPORTED;   // stride 1 only
    if (!d->w_shared && d->batch > 1) return FGR_ERR_UNSUPPORTED;            // one filter bank (the W tensor map is [S C, R, N])
    if (d->ldw != 0 && d->ldw != d->K) return FGR_ERR_UNSUPPORTED;
  }
  const Resolved r = resolve_strides(*d);
  if (r.ldx < d->K / taps || r.ldw < d->K || r.ldy < d->N) return FGR_ERR_INVALID_ARG;
  // a window must be K contiguous elements: the row stride is the convolution's stride times C, never a padded C
  if (taps > 1 && r.ldx % (d->K / taps) != 0) return FGR_ERR_UNSUPPORTED;
  if (r.ldx % g || r.ldw % g || r.ldy % g || r.bsx % g || r.bsw % g || r.bsy % g) return FGR_ERR_UNSUPPORTED;
  if (d->batch > 1 && (r.bsx < x_span(*d, r.ldx) || (!d->w_shared && r.bsw < (long long)(d->N - 1) * r.ldw + d->K) ||
                       r.bsy < (long long)(d->M - 1) * r.ldy + d->N))
    return FGR_ERR_INVALID_ARG;
  if ((long long)d->batch * d->M > (1LL << 31) - 1) return FGR_ERR_UNSUPPORTED;
  if (d->force_cta_pair < 0 || d->force_cta_pair > 2) return FGR_ERR_INVALID_ARG;
  if (d->force_ksub < 0 || d->force_ksub > 4) return FGR_ERR_INVALID_ARG;
  if (d->force_tile_n && (d->force_tile_n % 16 || d->force_tile_n < 16 || d->force_tile_n > 256)) return FGR_ERR_INVALID_ARG;
  return FGR_OK;
}

double min_bytes(const fgr_desc& d) {
  const double e = elem_bytes(d.dtype);
  const int taps = (d.conv_taps > 1 ? d.conv_taps : 1) * (d.conv_rows > 1 ? d.conv_rows : 1);   // a convolution's input is read once, not once per tap
  const Resolved rs = resolve_strides(d);
  const double x_elems = d.conv_rows > 1 ? (double)x_span(d, rs.ldx)
                         : taps > 1 ? (double)(d.M - 1) * (rs.ldx < d.K ? rs.ldx : d.K) + d.K : (double)d.M * d.K;   // samples actually read
  double b = ((double)d.batch * x_elems + (double)(d.w_shared ? 1 : d.batch) * d.N * d.K) * e;
  b += 4.0 * d.N * (d.bias_per_batch ? d.batch : 1);   // bias (counted whether or not one is passed)
  if (d.scale_kind == FGR_SCALE_PER_COLUMN) b += 4.0 * d.N;
  if (d.write_y || d.reduce == FGR_RED_SOFTMAX) b += (double)d.batch * d.M * d.N * e;
  b += 4.0 * d.batch * d.M * out_width(d.reduce);
  return b;
}

// Narrow-tile choice for the weight-streaming path: every SM should stream an equal share of W
// exactly once.  Cost model per wave: the W tile (tile_n rows) from HBM plus the X tile (128 rows)
// from L2, per k-block.
int pick_stream_tile_n(long long tiles_mb, int N, int sms) {
  int best = 16;
  double best_cost = 1e300;
  for (int tn = 16; tn <= 256; tn += 16) {
    const long long tiles = tiles_mb * ((N + tn - 1) / tn);
    const long long waves = (tiles + sms - 1) / sms;
    // a ragged last tile streams a full X tile for a few real columns: a mild penalty
    const double cost = (double)waves * (tn + 64) * (N % tn ? 1.1 : 1.0);
    if (cost < best_cost - 1e-9 || (std::fabs(cost - best_cost) <= 1e-9 && tn > best)) { best_cost = cost; best = tn; }
  }
  return best;
}

int make_plan(const fgr_desc& d, int num_sms, fgr_plan_info* info, Params* pp) {
  const int sms = num_sms > 0 ? num_sms : kDefaultSms;
  const Resolved r = resolve_strides(d);
  fgr_plan_info pi;
  std::memset(&pi, 0, sizeof pi);
  pi.flop = 2.0 * d.batch * (double)d.M * d.N * d.K;
  pi.min_bytes = min_bytes(d);

  int path = d.force_path;
  if (path == FGR_PATH_AUTO) {
    // fp32: CUDA-core FMA tiles, or for large compute-bound problems three tf32 tensor-core products
    // (the operand split costs one extra pass over X and W, so small or skinny problems stay on FMA)
    if (d.dtype == FGR_F32) path = (d.M >= 128 && d.N >= 128 && d.K >= 128 && pi.flop >= kTf32MinFlop) ? FGR_PATH_UMMA_TF32X3 : FGR_PATH_SIMT;
    else if (d.M <= 4 && d.reduce != FGR_RED_SOFTMAX) path = FGR_PATH_SIMT_GEMV;   // a few GEMVs: CUDA cores keep up with HBM
    else if (d.M <= 128 && pi.flop / pi.min_bytes < kRidgeFlopPerByte) path = FGR_PATH_UMMA_STREAM_W;
    else path = FGR_PATH_UMMA_TILED;
  }
  const bool conv2d = d.conv_rows > 1;
  if (conv2d && d.force_path == FGR_PATH_AUTO) {   // 2-D convolution: the tiled / streaming tensor-core paths (bf16) or CUDA cores
    if (path == FGR_PATH_UMMA_TF32X3) path = FGR_PATH_SIMT;
    if (path == FGR_PATH_SIMT_GEMV) path = FGR_PATH_UMMA_STREAM_W;
  }
  if (conv2d && (path == FGR_PATH_UMMA_TF32X3 || path == FGR_PATH_SIMT_GEMV)) return FGR_ERR_UNSUPPORTED;
  if (path == FGR_PATH_SIMT_GEMV && (d.dtype != FGR_BF16 || d.M > 16 || d.reduce == FGR_RED_SOFTMAX)) return FGR_ERR_UNSUPPORTED;
  if ((path == FGR_PATH_UMMA_TILED || path == FGR_PATH_UMMA_STREAM_W) && d.dtype != FGR_BF16) return FGR_ERR_UNSUPPORTED;
  if (path == FGR_PATH_UMMA_TF32X3 && d.dtype != FGR_F32) return FGR_ERR_UNSUPPORTED;
  const bool tf32 = path == FGR_PATH_UMMA_TF32X3;

  Params p;
  std::memset(&p, 0, sizeof p);
  p.batch = d.batch; p.M = d.M; p.N = d.N; p.K = d.K;
  p.dtype = d.dtype; p.act = d.act; p.scale_kind = d.scale_kind; p.reduce = d.reduce;
  p.write_y = d.write_y; p.bias_per_batch = d.bias_per_batch; p.scale = d.scale;
  p.w_shared = d.w_shared;
  p.conv_rows = conv2d ? d.conv_rows : 0;
  p.conv_width = d.conv_width;
  p.conv_kseg = conv2d ? d.K / d.conv_rows : 0;
  p.kseg_blocks = conv2d ? (p.conv_kseg + kUmmaBlockK - 1) / kUmmaBlockK : 0;
  p.ldx = r.ldx; p.ldw = r.ldw; p.ldy = r.ldy; p.bsx = r.bsx; p.bsw = r.bsw; p.bsy = r.bsy;

  if (path == FGR_PATH_SIMT_GEMV) {
    // every CTA streams a contiguous block of W rows; one partial pair per (row of X, CTA)
    const int r = gemv_rows_per_warp(d.M);
    int rows = (d.N + sms - 1) / sms;
    rows = (rows + r - 1) / r * r;
    p.tile_n = rows;
    p.half_n = rows;
    p.slots_per_tile = 1;
    p.tiles_m = 1;
    p.tiles_n = (d.N + rows - 1) / rows;
    p.stages = 0;
    p.cta_pair = 1;
    pi.tile_m = d.M;
    pi.smem_bytes = 0;
    if (d.batch > 65535) return FGR_ERR_UNSUPPORTED;
  } else if (path == FGR_PATH_SIMT) {
    p.tile_n = kSimtTile;
    p.half_n = kSimtTile;
    p.slots_per_tile = 1;
    p.tiles_m = (d.M + kSimtTile - 1) / kSimtTile;
    p.tiles_n = (d.N + kSimtTile - 1) / kSimtTile;
    p.stages = 0;
    pi.tile_m = kSimtTile;
    pi.smem_bytes = 0;
    if (p.tiles_m > 65535 || d.batch > 65535) return FGR_ERR_UNSUPPORTED;
  } else {
    int tn = d.force_tile_n;
    const int row_blocks = (d.M + kUmmaTileM - 1) / kUmmaTileM;
    if (!tn) {
      if (path == FGR_PATH_UMMA_STREAM_W) tn = pick_stream_tile_n((long long)d.batch * row_blocks, d.N, sms);
      else tn = d.N >= 256 ? 256 : ((d.N + 15) / 16) * 16;
      // Too few 256-wide tiles to give every CTA (pair) one: narrow the tiles until one wave fills the
      // machine (measured: 6 to 17 % faster on mid-size shapes, e.g. bf16 256 x 8192 x 4096 30.5 -> 26.2 us
      // with 64 tiles of 128 instead of 32 of 256; fp32 205 -> 180 us).  Same cost model as the streaming path.
      if (path != FGR_PATH_UMMA_STREAM_W && tn == 256) {
        const int want_pair = (d.force_cta_pair ? d.force_cta_pair : (row_blocks >= 2 && sms >= 2 ? 2 : 1));
        const long long units_m = (long long)d.batch * ((d.M + kUmmaTileM * want_pair - 1) / (kUmmaTileM * want_pair));
        const int groups = sms / want_pair;
        if (units_m * ((d.N + 255) / 256) < groups) {
          int best = 256;
          double best_cost = 1e300;
          for (int t = 32; t <= 256; t += 32) {
            const long long tiles = units_m * ((d.N + t - 1) / t);
            const long long waves = (tiles + groups - 1) / groups;
            const double cost = (double)waves * (t + 64) * (d.N % t ? 1.1 : 1.0);
            if (cost < best_cost - 1e-9 || (std::fabs(cost - best_cost) <= 1e-9 && t > best)) { best_cost = cost; best = t; }
          }
          tn = best;
        }
      }
    }
    // CTA pairs (256-row tiles, one tcgen05.mma.cta_group::2 for two SMs) cut the operand traffic
    // per SM by a third; they need at least two row blocks and a W tile that halves into whole
    // 16-row groups.
    int pair = d.force_cta_pair;
    if (!pair) pair = ((path == FGR_PATH_UMMA_TILED || tf32) && row_blocks >= 2 && tn % 32 == 0 && sms >= 2) ? 2 : 1;
    if (pair == 2 && tn % 32 != 0) return FGR_ERR_UNSUPPORTED;
    p.cta_pair = pair;
    p.tiles_m = (d.M + kUmmaTileM * pair - 1) / (kUmmaTileM * pair);
    p.tile_n = tn;
    p.half_n = ((tn / 2 + 15) / 16) * 16;
    p.slots_per_tile = 2;
    p.tiles_n = (d.N + tn - 1) / tn;
    const int w_rows = tn / pair;
    // Two adjacent 64-wide K sub-blocks per ring stage: the memory system then sees requests for
    // neighbouring 128-byte lines of the same matrix row back to back, which measurably raises the
    // rate at which operands arrive (L2 and DRAM both work in units larger than one line).  Used
    // when at least three such stages fit in shared memory and K is long enough to fill them.
    int ksub = tf32 ? 2 : d.force_ksub;   // 3xTF32: the two sub-blocks of a stage are the hi and lo planes
    if (!ksub) ksub = (d.K > kUmmaBlockK && umma_smem_layout(w_rows, 3, 2).total <= kSmemLimit) ? 2 : 1;
    while (!tf32 && ksub > 1 && umma_smem_layout(w_rows, 2, ksub).total > kSmemLimit) --ksub;
    // (2-D convolution: a stage is ksub whole k-blocks of the R * kseg_blocks the tile has; when that number is not a
    //  multiple of ksub the last stage's surplus sub-blocks lie beyond the last filter row and read as zero)
    p.ksub = ksub;
    p.k_plane = tf32 ? (d.K + 31) / 32 * 32 : 0;
    p.chunk_blocks = kTf32ChunkBlocks;
    int stages = kUmmaMaxStages;
    while (stages > 1 && umma_smem_layout(w_rows, stages, ksub).total > kSmemLimit) --stages;
    p.stages = stages;
    pi.tile_m = kUmmaTileM * pair;
    pi.smem_bytes = umma_smem_layout(w_rows, stages, ksub).total;
  }
  p.num_tiles = (long long)d.batch * p.tiles_m * p.tiles_n;
  p.parts_per_row = p.tiles_n * p.slots_per_tile;
  if (d.reduce == FGR_RED_SOFTMAX && p.parts_per_row > 12288) return FGR_ERR_UNSUPPORTED;

  pi.path = path;
  pi.tile_n = p.tile_n;
  pi.stages = p.stages;
  pi.parts_per_row = p.parts_per_row;
  pi.num_tiles = p.num_tiles;
  if (path == FGR_PATH_SIMT) {
    pi.grid = (int)(p.num_tiles > 0x7fffffff ? 0x7fffffff : p.num_tiles);
  } else if (path == FGR_PATH_SIMT_GEMV) {
    pi.grid = p.tiles_n * d.batch;
  } else {
    const long long groups = sms / p.cta_pair;   // CTAs, or clusters of two
    pi.grid = (int)(p.num_tiles < groups ? p.num_tiles : groups) * p.cta_pair;
  }
  const bool cuda_cores = path == FGR_PATH_SIMT || path == FGR_PATH_SIMT_GEMV;
  pi.cta_pair = cuda_cores ? 1 : p.cta_pair;
  pi.ksub = cuda_cores ? 0 : p.ksub;
  pi.launches = tf32 ? 4 : 2;   // (operand split of X and of W +) main kernel + (merge | softmax normalise)
  // tcgen05 softmax: completion counters per row-block unit (+ one finish ticket) follow the status block
  p.head_bytes = kStatusBytes;
  p.done_target = 0;
  if (!cuda_cores && d.reduce == FGR_RED_SOFTMAX) {
    const long long units = (long long)d.batch * p.tiles_m;
    p.head_bytes += (int)align256((size_t)(units + 1) * sizeof(unsigned int));
    p.done_target = (unsigned int)p.tiles_n * 8u * (unsigned int)p.cta_pair;   // epilogue warps per unit
  } else if (path == FGR_PATH_SIMT && d.reduce != FGR_RED_SOFTMAX) {
    // CUDA-core tiles: one counter per block of 64 rows; the CTA that completes a block merges its rows, so
    // there is no second launch (these are the small problems, bound by launch latency)
    p.head_bytes += (int)align256((size_t)d.batch * p.tiles_m * sizeof(unsigned int));
    p.done_target = (unsigned int)p.tiles_n;
    pi.launches = 1;
  }
  pi.workspace_bytes = (uint64_t)p.head_bytes + (uint64_t)d.batch * d.M * p.parts_per_row * 8ull;
  if (tf32)   // the hi / lo planes of X and W follow the partial pairs, each on a 256-byte boundary
    pi.workspace_bytes = align256(align256((size_t)pi.workspace_bytes) + (size_t)d.batch * d.M * 2 * p.k_plane * 4) +
                         (uint64_t)(d.w_shared ? 1 : d.batch) * d.N * 2 * p.k_plane * 4;
  *info = pi;
  if (pp) *pp = p;
  return FGR_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// bf16 [batch, rows, K] with strides (ld, bs) -> 3-D map, box = 64 (K) x box_rows x 1, 128-byte swizzle,
// out-of-range elements read as zero.
// (fp32 = true: 4-byte elements, box = 32 (K) x box_rows x 1, the same 128-byte rows.)
// (box_in_z = true: the box is 64 x 1 x box_rows - rows of the box come from the third dimension, the middle one
//  selects a plane: the filters of a 2-D convolution as [S C, R, N].)
int encode_operand(CUtensorMap* map, const void* ptr, int K, int rows, int batch, long long ld, long long bs, int box_rows,
                   bool fp32 = false, bool box_in_z = false) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return FGR_ERR_CUDA;
  const unsigned eb = fp32 ? 4 : 2;
  cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)batch};
  cuuint64_t strides[2] = {(cuuint64_t)ld * eb, (cuuint64_t)(batch > 1 || box_in_z ? bs : (long long)rows * ld) * eb};
  cuuint32_t box[3] = {(cuuint32_t)(kUmmaBlockK * 2 / eb), (cuuint32_t)(box_in_z ? 1 : box_rows), (cuuint32_t)(box_in_z ? box_rows : 1)};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult rc = fn(map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? FGR_OK : FGR_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

__global__ void empty_kernel() {}

}  // namespace

extern "C" {

int fgr_plan(const fgr_desc* desc, int num_sms, fgr_plan_info* info) {
  if (!info) return FGR_ERR_INVALID_ARG;
  int rc = validate(desc);
  if (rc != FGR_OK) return rc;
  return make_plan(*desc, num_sms, info, nullptr);
}

int fgr_create(const fgr_desc* desc, fgr_handle** out) {
  if (!out) return FGR_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = validate(desc);
  if (rc != FGR_OK) return rc;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || desc->device >= ndev) { cudaGetLastError(); return FGR_ERR_CUDA; }
  int major = 0, sms = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, desc->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, desc->device) != cudaSuccess)
    return FGR_ERR_CUDA;
  if (major != 10) return FGR_ERR_ARCH;
  fgr_handle* h = new (std::nothrow) fgr_handle;
  if (!h) return FGR_ERR_INVALID_ARG;
  std::memset(h, 0, sizeof *h);
  h->events = new (std::nothrow) std::vector<cudaEvent_t>();
  if (!h->events) { delete h; return FGR_ERR_INVALID_ARG; }
  h->desc = *desc;
  h->num_sms = sms;
  rc = make_plan(*desc, sms, &h->plan, &h->base);
  if (rc != FGR_OK) { delete h->events; delete h; return rc; }
  if (h->plan.path == FGR_PATH_UMMA_TILED || h->plan.path == FGR_PATH_UMMA_STREAM_W || h->plan.path == FGR_PATH_UMMA_TF32X3) {
    int prev = 0;
    cudaGetDevice(&prev);
    cudaError_t e = cudaSetDevice(desc->device);
    if (e == cudaSuccess) e = umma_prepare(desc->device);
    cudaSetDevice(prev);
    if (e != cudaSuccess || !encode_fn()) { cudaGetLastError(); delete h->events; delete h; return FGR_ERR_CUDA; }
  }
  *out = h;
  return FGR_OK;
}

size_t fgr_workspace_bytes(const fgr_handle* h) { return h ? (size_t)h->plan.workspace_bytes : 0; }

int fgr_get_plan(const fgr_handle* h, fgr_plan_info* info) {
  if (!h || !info) return FGR_ERR_INVALID_ARG;
  *info = h->plan;
  return FGR_OK;
}

int fgr_run(fgr_handle* h, const void* X, const void* W, const float* bias, const float* scale_vec, void* Y,
            float* out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!h || !X || !W) return FGR_ERR_INVALID_ARG;
  const fgr_desc& d = h->desc;
  const bool softmax = d.reduce == FGR_RED_SOFTMAX;
  if (!aligned16(X) || !aligned16(W) || (Y && !aligned16(Y))) return FGR_ERR_INVALID_ARG;
  if ((d.write_y || softmax) && !Y) return FGR_ERR_INVALID_ARG;
  if (!softmax && !out) return FGR_ERR_INVALID_ARG;
  if (d.scale_kind == FGR_SCALE_PER_COLUMN && !scale_vec) return FGR_ERR_INVALID_ARG;
  if ((bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) || (scale_vec && (reinterpret_cast<uintptr_t>(scale_vec) & 3u)) ||
      (out && (reinterpret_cast<uintptr_t>(out) & 7u)))
    return FGR_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) || workspace_bytes < h->plan.workspace_bytes)
    return FGR_ERR_WORKSPACE;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != d.device && cudaSetDevice(d.device) != cudaSuccess) { cudaGetLastError(); return FGR_ERR_CUDA; }
  int rc = FGR_OK;
  cudaError_t e = cudaSuccess;

  Params p = h->base;
  p.X = X; p.W = W; p.bias = bias; p.scale_vec = scale_vec; p.Y = Y; p.out = out;
  p.R = h->residual; p.ldr = h->ldr; p.bsr = h->bsr;
  p.status = static_cast<int*>(workspace);
  p.parts = reinterpret_cast<float*>(static_cast<char*>(workspace) + p.head_bytes);
  p.done = p.done_target ? reinterpret_cast<unsigned int*>(static_cast<char*>(workspace) + kStatusBytes) : nullptr;

  if (workspace != h->last_workspace) {   // a workspace seen for the first time: clear its status word (and counters)
    e = cudaMemsetAsync(workspace, 0, (size_t)p.head_bytes, stream);
    h->last_workspace = workspace;
  }
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  if (h->profiling && h->events_used + 2 <= 2 * 4096) {
    if (h->events->size() < h->events_used + 2) {
      cudaEvent_t a = nullptr, b = nullptr;
      if (cudaEventCreate(&a) == cudaSuccess && cudaEventCreate(&b) == cudaSuccess) { h->events->push_back(a); h->events->push_back(b); }
    }
    if (h->events->size() >= h->events_used + 2) { ev0 = (*h->events)[h->events_used]; ev1 = (*h->events)[h->events_used + 1]; }
  }
  const bool tf32 = h->plan.path == FGR_PATH_UMMA_TF32X3;
  float* xp = nullptr;
  float* wp = nullptr;
  if (tf32 && e == cudaSuccess) {
    // split X and W into tf32 hi / lo planes inside the workspace (ahead of the timed main kernel)
    char* wsb = static_cast<char*>(workspace);
    const size_t x_off = align256((size_t)p.head_bytes + (size_t)d.batch * d.M * p.parts_per_row * 8u);
    const size_t w_off = align256(x_off + (size_t)d.batch * d.M * 2 * p.k_plane * 4);
    xp = reinterpret_cast<float*>(wsb + x_off);
    wp = reinterpret_cast<float*>(wsb + w_off);
    e = launch_split_tf32(static_cast<const float*>(X), xp, d.batch, d.M, d.K, p.ldx, p.bsx, p.k_plane, stream);
    if (e == cudaSuccess) e = launch_split_tf32(static_cast<const float*>(W), wp, d.w_shared ? 1 : d.batch, d.N, d.K, p.ldw, p.bsw, p.k_plane, stream);
  }
  if (e == cudaSuccess && ev0) e = cudaEventRecord(ev0, stream);
  if (e == cudaSuccess) {
    if (h->plan.path == FGR_PATH_SIMT) {
      e = launch_simt(p, stream);
    } else if (h->plan.path == FGR_PATH_SIMT_GEMV) {
      e = launch_gemv(p, p.tiles_n, p.tile_n, stream);
    } else if (tf32) {
      // the tensor-core kernel reads the planes, which live in the workspace: both maps are keyed by it
      const CUtensorMap* mx = h->maps_x.find(workspace);
      const CUtensorMap* mw = h->maps_w.find(workspace);
      if (!mx || !mw) {
        const long long ldp = 2LL * p.k_plane;
        h->maps_x.forget(workspace);
        h->maps_w.forget(workspace);
        CUtensorMap* nx = h->maps_x.claim(workspace);
        CUtensorMap* nw = h->maps_w.claim(workspace);
        rc = encode_operand(nx, xp, (int)ldp, d.M, d.batch, ldp, (long long)d.M * ldp, kUmmaTileM, true);
        if (rc == FGR_OK) rc = encode_operand(nw, wp, (int)ldp, d.N, d.w_shared ? 1 : d.batch, ldp, (long long)d.N * ldp, p.tile_n / p.cta_pair, true);
        if (rc != FGR_OK) { h->maps_x.forget(workspace); h->maps_w.forget(workspace); }
        mx = nx; mw = nw;
      }
      if (rc == FGR_OK && e == cudaSuccess) e = launch_umma(p, mx, mw, h->plan.grid, h->plan.smem_bytes, stream);
    } else {
      const CUtensorMap* mx = h->maps_x.find(X);
      if (!mx) {
        CUtensorMap* nx = h->maps_x.claim(X);
        if (p.conv_rows > 1)   // [S C, window rows, batch]: segment r of output row m is window row m + r * conv_width
          rc = encode_operand(nx, X, p.conv_kseg, d.M + (d.conv_rows - 1) * d.conv_width, d.batch, p.ldx, p.bsx, kUmmaTileM);
        else
          rc = encode_operand(nx, X, d.K, d.M, d.batch, p.ldx, p.bsx, kUmmaTileM);
        if (rc != FGR_OK) h->maps_x.forget(X);
        mx = nx;
      }
      const CUtensorMap* mw = rc == FGR_OK ? h->maps_w.find(W) : nullptr;
      if (rc == FGR_OK && !mw) {
        CUtensorMap* nw = h->maps_w.claim(W);
        if (p.conv_rows > 1)   // [S C, R, N]: one filter bank; filter row r of filter n starts at W[n * K + r * S C]
          rc = encode_operand(nw, W, p.conv_kseg, d.conv_rows, d.N, p.conv_kseg, p.ldw, p.tile_n / p.cta_pair, false, true);
        else
          rc = encode_operand(nw, W, d.K, d.N, d.w_shared ? 1 : d.batch, p.ldw, p.bsw, p.tile_n / p.cta_pair);
        if (rc != FGR_OK) h->maps_w.forget(W);
        mw = nw;
      }
      if (rc == FGR_OK) e = launch_umma(p, mx, mw, h->plan.grid, h->plan.smem_bytes, stream);
    }
  }
  if (rc == FGR_OK && e == cudaSuccess && ev1) {
    e = cudaEventRecord(ev1, stream);
    h->events_used += 2;
  }
  if (rc == FGR_OK && e == cudaSuccess) {
    if (softmax) e = launch_normalise(p, stream);
    else if (h->plan.path != FGR_PATH_SIMT) e = launch_merge(p, stream);   // (the CUDA-core GEMM kernel merges its own pairs)
  }
  if (e != cudaSuccess) { cudaGetLastError(); rc = FGR_ERR_CUDA; }
  h->last_stream = stream;
  h->ran = true;
  if (prev != d.device && prev >= 0) cudaSetDevice(prev);
  return rc;
}

int fgr_set_residual(fgr_handle* h, const void* R, int64_t ldr, int64_t bsr) {
  if (!h || ldr < 0 || bsr < 0) return FGR_ERR_INVALID_ARG;
  if (!R) { h->residual = nullptr; return FGR_OK; }
  const fgr_desc& d = h->desc;
  const int g = 16 / elem_bytes(d.dtype);
  const long long l = ldr ? ldr : d.N, b = bsr ? bsr : (long long)d.M * l;
  if (l < d.N || (d.batch > 1 && b < (long long)(d.M - 1) * l + d.N)) return FGR_ERR_INVALID_ARG;
  if (l % g || b % g) return FGR_ERR_UNSUPPORTED;
  if (!aligned16(R)) return FGR_ERR_INVALID_ARG;
  h->residual = R; h->ldr = l; h->bsr = b;
  return FGR_OK;
}

int fgr_get_status(fgr_handle* h) {
  if (!h) return FGR_ERR_INVALID_ARG;
  if (!h->ran) return FGR_OK;
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != h->desc.device) cudaSetDevice(h->desc.device);
  int word = 0;
  int rc = FGR_OK;
  if (cudaStreamSynchronize(h->last_stream) != cudaSuccess ||
      cudaMemcpy(&word, h->last_workspace, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    rc = FGR_ERR_CUDA;
  } else if (word != 0) {
    rc = word;
    // reported once; a run that gave up may also have left its completion counters half counted
    cudaMemset(h->last_workspace, 0, (size_t)h->base.head_bytes);
  }
  if (prev != h->desc.device && prev >= 0) cudaSetDevice(prev);
  return rc;
}

// Plans fgr_run_host's chunks once per handle: kHostChunks blocks of batches when there are at least that
// many, else (one batch, plain GEMM, enough rows) blocks of rows in multiples of 256.  Each chunk gets a
// sub-handle of its own shape with the parent's strides spelled out, so it runs on a slice of the parent's
// staging buffers.  Returns false if the problem stays in one piece.
static bool plan_host_chunks(fgr_handle* h) {
  if (h->sub_count) return h->sub_count > 1;
  h->sub_count = 1;
  const fgr_desc& d = h->desc;
  const Params& b = h->base;
  if (d.conv_taps > 1 || d.conv_rows > 1) return false;   // overlapping rows: the chunks' input copies would overlap too
  long long total, unit;
  if (d.batch >= kHostChunks) { h->sub_by_batch = true; total = d.batch; unit = 1; }
  else if (d.batch == 1 && d.M >= kHostChunks * 256) { h->sub_by_batch = false; total = d.M; unit = 256; }
  else return false;
  const long long per = ((total + kHostChunks - 1) / kHostChunks + unit - 1) / unit * unit;
  // a chunk's slice of `out` must start on an 8-byte boundary
  if ((per * (h->sub_by_batch ? d.M : 1) * out_width(d.reduce)) % 2 != 0) return false;
  int n = 0;
  for (long long first = 0; first < total && n < kHostChunks; first += per) h->sub_first[n++] = first;
  h->sub_first[n] = total;
  size_t ws = 0;
  for (int c = 0; c < n; ++c) {
    fgr_desc sd = d;
    const int count = (int)(h->sub_first[c + 1] - h->sub_first[c]);
    if (h->sub_by_batch) sd.batch = count; else sd.M = count;
    sd.ldx = b.ldx; sd.ldw = b.ldw; sd.ldy = b.ldy;
    sd.bsx = b.bsx; sd.bsw = b.bsw; sd.bsy = b.bsy;
    if (fgr_create(&sd, &h->sub[c]) != FGR_OK) {
      for (int k = 0; k < c; ++k) { fgr_destroy(h->sub[k]); h->sub[k] = nullptr; }
      return false;
    }
    h->sub_ws_off[c] = ws;
    ws += align256((size_t)h->sub[c]->plan.workspace_bytes);
  }
  bool ok = cudaMalloc(&h->sub_ws, ws) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&h->in_stream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaStreamCreateWithFlags(&h->out_stream, cudaStreamNonBlocking) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&h->ev_shared, cudaEventDisableTiming) == cudaSuccess;
  for (int c = 0; c < n && ok; ++c)
    ok = cudaEventCreateWithFlags(&h->ev_in[c], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&h->ev_run[c], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {   // leave what exists to fgr_destroy; run in one piece
    cudaGetLastError();
    for (int c = 0; c < n; ++c) { fgr_destroy(h->sub[c]); h->sub[c] = nullptr; }
    return false;
  }
  h->sub_ws_bytes = ws;
  h->sub_count = n;
  return n > 1;
}

int fgr_run_host(fgr_handle* h, const void* X, const void* W, const float* bias, const float* scale_vec, void* Y,
                 float* out) {
  if (!h || !X || !W) return FGR_ERR_INVALID_ARG;
  const fgr_desc& d = h->desc;
  const Params& b = h->base;
  const bool softmax = d.reduce == FGR_RED_SOFTMAX;
  const bool need_y = d.write_y || softmax;
  if ((need_y && !Y) || (!softmax && !out)) return FGR_ERR_INVALID_ARG;
  if (d.scale_kind == FGR_SCALE_PER_COLUMN && !scale_vec) return FGR_ERR_INVALID_ARG;
  if (h->residual) return FGR_ERR_UNSUPPORTED;   // the residual is a device tensor: use fgr_run
  const size_t e = (size_t)elem_bytes(d.dtype);
  // extents in bytes of each buffer as laid out by the descriptor's strides
  const size_t want[7] = {
      ((size_t)(d.batch - 1) * b.bsx + (size_t)x_span(d, b.ldx)) * e,
      ((size_t)(d.batch - 1) * b.bsw + (size_t)(d.N - 1) * b.ldw + d.K) * e,
      bias ? (size_t)d.N * (d.bias_per_batch ? d.batch : 1) * 4 : 0,
      scale_vec ? (size_t)d.N * 4 : 0,
      need_y ? ((size_t)(d.batch - 1) * b.bsy + (size_t)(d.M - 1) * b.ldy + d.N) * e : 0,
      (size_t)d.batch * d.M * out_width(d.reduce) * 4,
      (size_t)h->plan.workspace_bytes};
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != d.device && cudaSetDevice(d.device) != cudaSuccess) { cudaGetLastError(); return FGR_ERR_CUDA; }
  int rc = FGR_OK;
  if (!h->host_stream && cudaStreamCreateWithFlags(&h->host_stream, cudaStreamNonBlocking) != cudaSuccess) rc = FGR_ERR_CUDA;
  for (int i = 0; i < 7 && rc == FGR_OK; ++i) {
    if (want[i] > h->stage_bytes[i]) {
      if (h->stage[i]) cudaFree(h->stage[i]);
      h->stage[i] = nullptr;
      h->stage_bytes[i] = 0;
      if (cudaMalloc(&h->stage[i], want[i]) != cudaSuccess) rc = FGR_ERR_CUDA;
      else h->stage_bytes[i] = want[i];
      if (i == 0) h->maps_x.clear();   // (the maps are keyed by address; a handle's strides never change, so a
      if (i == 1) h->maps_w.clear();   //  reused address would still be described correctly: this is tidiness)
    }
  }
  if (rc == FGR_OK && plan_host_chunks(h)) {
    // Chunked: the copy in of chunk c + 1, the kernels of chunk c and the copy out of chunk c - 1 overlap
    // (three streams, events in between).  What all chunks share (bias, scale; W unless it is batched) goes first.
    const size_t ex = e;
    const int n = h->sub_count;
    auto fail = [&](cudaError_t ce) { if (ce != cudaSuccess && rc == FGR_OK) rc = FGR_ERR_CUDA; };
    if (want[2]) fail(cudaMemcpyAsync(h->stage[2], bias, want[2], cudaMemcpyHostToDevice, h->in_stream));
    if (want[3]) fail(cudaMemcpyAsync(h->stage[3], scale_vec, want[3], cudaMemcpyHostToDevice, h->in_stream));
    const bool w_chunked = h->sub_by_batch && !d.w_shared;
    if (!w_chunked) fail(cudaMemcpyAsync(h->stage[1], W, want[1], cudaMemcpyHostToDevice, h->in_stream));
    fail(cudaEventRecord(h->ev_shared, h->in_stream));
    fail(cudaStreamWaitEvent(h->host_stream, h->ev_shared, 0));
    for (int c = 0; c < n && rc == FGR_OK; ++c) {
      const long long first = h->sub_first[c], count = h->sub_first[c + 1] - first;
      const size_t x_off = (size_t)first * (h->sub_by_batch ? b.bsx : b.ldx) * ex;
      const size_t y_off = (size_t)first * (h->sub_by_batch ? b.bsy : b.ldy) * ex;
      const size_t w_off = w_chunked ? (size_t)first * b.bsw * ex : 0;
      const size_t rows_before = (size_t)first * (h->sub_by_batch ? d.M : 1);
      const size_t rows_here = (size_t)count * (h->sub_by_batch ? d.M : 1);
      // bytes of this chunk's slices (the last row of a slice ends at its K or N, not at the next stride)
      const size_t x_bytes = h->sub_by_batch ? ((size_t)(count - 1) * b.bsx + (size_t)(d.M - 1) * b.ldx + d.K) * ex
                                             : ((size_t)(count - 1) * b.ldx + d.K) * ex;
      const size_t w_bytes = ((size_t)(count - 1) * b.bsw + (size_t)(d.N - 1) * b.ldw + d.K) * ex;
      const size_t y_bytes = h->sub_by_batch ? ((size_t)(count - 1) * b.bsy + (size_t)(d.M - 1) * b.ldy + d.N) * ex
                                             : ((size_t)(count - 1) * b.ldy + d.N) * ex;
      char* dx = static_cast<char*>(h->stage[0]) + x_off;
      char* dw = static_cast<char*>(h->stage[1]) + w_off;
      char* dy = need_y ? static_cast<char*>(h->stage[4]) + y_off : nullptr;
      float* dout = softmax ? nullptr : static_cast<float*>(h->stage[5]) + rows_before * out_width(d.reduce);
      const float* dbias = bias ? static_cast<const float*>(h->stage[2]) + (d.bias_per_batch && h->sub_by_batch ? (size_t)first * d.N : 0) : nullptr;
      fail(cudaMemcpyAsync(dx, static_cast<const char*>(X) + x_off, x_bytes, cudaMemcpyHostToDevice, h->in_stream));
      if (w_chunked) fail(cudaMemcpyAsync(dw, static_cast<const char*>(W) + w_off, w_bytes, cudaMemcpyHostToDevice, h->in_stream));
      fail(cudaEventRecord(h->ev_in[c], h->in_stream));
      fail(cudaStreamWaitEvent(h->host_stream, h->ev_in[c], 0));
      if (rc == FGR_OK)
        rc = fgr_run(h->sub[c], dx, dw, dbias, scale_vec ? static_cast<float*>(h->stage[3]) : nullptr, dy, dout,
                     static_cast<char*>(h->sub_ws) + h->sub_ws_off[c], (size_t)h->sub[c]->plan.workspace_bytes, h->host_stream);
      fail(cudaEventRecord(h->ev_run[c], h->host_stream));
      fail(cudaStreamWaitEvent(h->out_stream, h->ev_run[c], 0));
      if (need_y) fail(cudaMemcpyAsync(static_cast<char*>(Y) + y_off, dy, y_bytes, cudaMemcpyDeviceToHost, h->out_stream));
      if (!softmax)
        fail(cudaMemcpyAsync(out + rows_before * out_width(d.reduce), dout, rows_here * out_width(d.reduce) * 4, cudaMemcpyDeviceToHost, h->out_stream));
    }
    if (cudaStreamSynchronize(h->out_stream) != cudaSuccess || cudaStreamSynchronize(h->in_stream) != cudaSuccess) { cudaGetLastError(); rc = FGR_ERR_CUDA; }
    for (int c = 0; c < n; ++c) {
      const int st = fgr_get_status(h->sub[c]);
      if (rc == FGR_OK && st != FGR_OK) rc = st;
    }
    if (prev != d.device && prev >= 0) cudaSetDevice(prev);
    return rc;
  }
  cudaStream_t s = h->host_stream;
  const void* src[4] = {X, W, bias, scale_vec};
  for (int i = 0; i < 4 && rc == FGR_OK; ++i)
    if (want[i] && cudaMemcpyAsync(h->stage[i], src[i], want[i], cudaMemcpyHostToDevice, s) != cudaSuccess) rc = FGR_ERR_CUDA;
  if (rc == FGR_OK)
    rc = fgr_run(h, h->stage[0], h->stage[1], bias ? static_cast<float*>(h->stage[2]) : nullptr,
                 scale_vec ? static_cast<float*>(h->stage[3]) : nullptr, need_y ? h->stage[4] : nullptr,
                 softmax ? nullptr : static_cast<float*>(h->stage[5]), h->stage[6], h->stage_bytes[6], s);
  if (rc == FGR_OK && need_y && cudaMemcpyAsync(Y, h->stage[4], want[4], cudaMemcpyDeviceToHost, s) != cudaSuccess) rc = FGR_ERR_CUDA;
  if (rc == FGR_OK && want[5] && !softmax &&
      cudaMemcpyAsync(out, h->stage[5], want[5], cudaMemcpyDeviceToHost, s) != cudaSuccess)
    rc = FGR_ERR_CUDA;
  if (rc == FGR_OK) rc = fgr_get_status(h);
  else cudaGetLastError();
  if (prev != d.device && prev >= 0) cudaSetDevice(prev);
  return rc;
}

int fgr_profile_enable(fgr_handle* h, int enable) {
  if (!h) return FGR_ERR_INVALID_ARG;
  h->profiling = enable != 0;
  return FGR_OK;
}

int fgr_profile_read(fgr_handle* h, double* main_kernel_ms, int* runs) {
  if (!h || !main_kernel_ms || !runs) return FGR_ERR_INVALID_ARG;
  double sum = 0.0;
  int n = 0, rc = FGR_OK;
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != h->desc.device) cudaSetDevice(h->desc.device);
  for (size_t i = 0; i + 1 < h->events_used; i += 2) {
    float ms = 0.0f;
    if (cudaEventSynchronize((*h->events)[i + 1]) != cudaSuccess ||
        cudaEventElapsedTime(&ms, (*h->events)[i], (*h->events)[i + 1]) != cudaSuccess) { cudaGetLastError(); rc = FGR_ERR_CUDA; break; }
    sum += ms;
    ++n;
  }
  if (prev != h->desc.device && prev >= 0) cudaSetDevice(prev);
  h->events_used = 0;
  *main_kernel_ms = sum;
  *runs = n;
  return rc;
}

int fgr_profile_empty_launches(int n, int device, void* cuda_stream) {
  if (n < 0 || device < 0) return FGR_ERR_INVALID_ARG;
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != device && cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return FGR_ERR_CUDA; }
  cudaError_t e = cudaSuccess;
  for (int i = 0; i < n && e == cudaSuccess; ++i) {
    empty_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>();
    e = cudaGetLastError();
  }
  if (prev != device && prev >= 0) cudaSetDevice(prev);
  return e == cudaSuccess ? FGR_OK : FGR_ERR_CUDA;
}

int fgr_destroy(fgr_handle* h) {
  if (!h) return FGR_OK;
  for (int c = 0; c < kHostChunks; ++c) if (h->sub[c]) fgr_destroy(h->sub[c]);
  bool owns = h->host_stream != nullptr || !h->events->empty() || h->sub_ws || h->in_stream || h->out_stream || h->ev_shared;
  for (int i = 0; i < 7; ++i) owns = owns || h->stage[i];
  if (owns) {
    int prev = -1;
    cudaGetDevice(&prev);
    if (prev != h->desc.device) cudaSetDevice(h->desc.device);
    if (h->host_stream) { cudaStreamSynchronize(h->host_stream); cudaStreamDestroy(h->host_stream); }
    for (int i = 0; i < 7; ++i) if (h->stage[i]) cudaFree(h->stage[i]);
    if (h->in_stream) { cudaStreamSynchronize(h->in_stream); cudaStreamDestroy(h->in_stream); }
    if (h->out_stream) { cudaStreamSynchronize(h->out_stream); cudaStreamDestroy(h->out_stream); }
    if (h->sub_ws) cudaFree(h->sub_ws);
    if (h->ev_shared) cudaEventDestroy(h->ev_shared);
    for (int c = 0; c < kHostChunks; ++c) {
      if (h->ev_in[c]) cudaEventDestroy(h->ev_in[c]);
      if (h->ev_run[c]) cudaEventDestroy(h->ev_run[c]);
    }
    for (cudaEvent_t ev : *h->events) cudaEventDestroy(ev);
    if (prev != h->desc.device && prev >= 0) cudaSetDevice(prev);
  }
  delete h->events;
  delete h;
  return FGR_OK;
}

const char* fgr_status_string(int status) {
  switch (status) {
    case FGR_OK: return "ok";
    case FGR_ERR_INVALID_ARG: return "invalid argument";
    case FGR_ERR_UNSUPPORTED: return "unsupported shape or configuration";
    case FGR_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case FGR_ERR_CUDA: return "CUDA call failed";
    case FGR_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case FGR_ERR_ARCH: return "device is not compute capability 10.x";
    default: return "unknown status";
  }
}

const char* fgr_path_name(int path) {
  switch (path) {
    case FGR_PATH_AUTO: return "auto";
    case FGR_PATH_SIMT: return "simt";
    case FGR_PATH_UMMA_TILED: return "umma_tiled";
    case FGR_PATH_UMMA_STREAM_W: return "umma_stream_w";
    case FGR_PATH_SIMT_GEMV: return "simt_gemv";
    case FGR_PATH_UMMA_TF32X3: return "umma_tf32x3";
    default: return "unknown";
  }
}

}  // extern "C"
