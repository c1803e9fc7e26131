/*
 * fgr.h - C ABI of the fused GEMM + epilogue + row-reduce operator for NVIDIA B200 (sm_100a).
 *
 * The operator.  For every batch bt and row m
 *
 *     z[m, n] = sum_k X[bt, m, k] * W[bt, n, k]            (X * W^T, K contiguous in both)
 *     y[m, n] = act(z[m, n] + b[n]) * s[n]                  act in {identity, ReLU, GELU-tanh, sigmoid, tanh, SiLU}
 *
 * followed by a reduction over n of each row:
 *
 *     FGR_RED_LSE        out[m]    = log sum_n exp(y[m, n])
 *     FGR_RED_SOFTMAX    P[m, n]   = exp(y[m, n]) / sum_n exp(y[m, n])      (written in Y's slot)
 *     FGR_RED_MAXSUM     out[m, :] = ( max_n y , sum_n y )
 *     FGR_RED_MAX_SUMEXP out[m, :] = ( max_n y , sum_n exp(y - max_n y) )
 *     FGR_RED_MEANVAR    out[m, :] = ( mean_n y , (1/N) sum_n (y - mean)^2 )
 *
 * Variations of the same operator (each documented where it is declared): a residual tensor added to
 * y (fgr_set_residual), one weight matrix shared by all batch elements (fgr_desc.w_shared), 1-D
 * convolution as an implicit GEMM (fgr_desc.conv_taps), fp32 problems on tensor cores
 * (FGR_PATH_UMMA_TF32X3), N sharded over several GPUs (fgr_combine_shards), and the reductions alone on
 * a given matrix (fgr_reduce_rows).
 *
 * Where this comes from.  The paper's task statement is: given the reference operator's inputs,
 * produce the same outputs, faster (Section 3.1, Verifier; Section 3.3), for operators of the
 * categories "matrix multiplication, convolution, element-wise and reduction" (Section 1; Section 4.1,
 * Datasets).  The paper prints no formula for any operator; the formulas above are the plain
 * definitions of a linear layer, the activation, a scale and a last-dimension reduction.
 *
 * Conventions for every entry point.
 *   - All functions return an fgr_status (0 = success) unless stated; nothing throws or aborts.
 *   - "device pointer" = memory of the CUDA device named in the descriptor; "host pointer" =
 *     ordinary process memory.  The caller owns every buffer it passes; the library owns only
 *     the handle.  fgr_run never allocates and never synchronises.
 *   - Layout: row-major.  X [batch, M, K], W [batch, N, K], Y / P [batch, M, N]; row strides
 *     ldx, ldw, ldy and batch strides bsx, bsw, bsy in elements (0 = packed).
 *   - Element types: X, W, Y/P are `dtype` (fp32, or bf16 as raw 16-bit patterns); bias,
 *     scale_vec and out are always fp32.  Accumulation is fp32.
 *   - Supported shapes: batch, M, N, K >= 1; K and N multiples of 8 (bf16) or 4 (fp32);
 *     X, W, Y base pointers 16-byte aligned; ld* and bs* multiples of 8 (bf16) / 4 (fp32).
 *     Anything else returns FGR_ERR_UNSUPPORTED or FGR_ERR_INVALID_ARG, never a wrong answer.
 *   - Inputs must be finite.  NaN/Inf inputs give unspecified values but never hang or fault.
 *   - One handle may be used by one thread and one stream at a time.
 */
#ifndef FGR_H_
#define FGR_H_

#if defined(__GNUC__)
#define FGR_API __attribute__((visibility("default")))
#else
#define FGR_API
#endif

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FGR_OK = 0,
  FGR_ERR_INVALID_ARG = 1,    /* null / misaligned pointer, bad enum, bad stride, bad struct size */
  FGR_ERR_UNSUPPORTED = 2,    /* a shape the kernels do not cover (see "Supported shapes") */
  FGR_ERR_WORKSPACE = 3,      /* workspace null, misaligned or smaller than fgr_workspace_bytes */
  FGR_ERR_CUDA = 4,           /* a CUDA runtime/driver call failed (no device, launch error, ...) */
  FGR_ERR_DEVICE_TIMEOUT = 5, /* a bounded in-kernel wait ran out; outputs of that run are invalid */
  FGR_ERR_ARCH = 6            /* the device is not compute capability 10.x */
} fgr_status;

typedef enum { FGR_F32 = 0, FGR_BF16 = 1 } fgr_dtype;
typedef enum { FGR_ACT_NONE = 0, FGR_ACT_RELU = 1, FGR_ACT_GELU_TANH = 2, FGR_ACT_SIGMOID = 3, FGR_ACT_TANH = 4,
               FGR_ACT_SILU = 5 } fgr_act;
typedef enum { FGR_SCALE_NONE = 0, FGR_SCALE_SCALAR = 1, FGR_SCALE_PER_COLUMN = 2 } fgr_scale_kind;
typedef enum { FGR_RED_LSE = 0, FGR_RED_SOFTMAX = 1, FGR_RED_MAXSUM = 2, FGR_RED_MAX_SUMEXP = 3,
               /* (mean, population variance) of y over N: the row statistics of a normalisation layer.  Computed
                  per tile in two passes and merged pairwise (mean, sum of squared deviations), never as
                  E[y^2] - E[y]^2. */
               FGR_RED_MEANVAR = 6 } fgr_reduce;

/* Execution paths (fgr_plan_info.path, fgr_desc.force_path). */
typedef enum {
  FGR_PATH_AUTO = 0,
  FGR_PATH_SIMT = 1,          /* CUDA-core tiles, fp32 FMA: the fp32 path, also valid for bf16 */
  FGR_PATH_UMMA_TILED = 2,    /* tcgen05 128 x 256 tiles, TMA ring, compute-bound shapes (bf16) */
  FGR_PATH_UMMA_STREAM_W = 3, /* tcgen05 with narrow N tiles and a deep TMA ring: M <= 128, W streamed once (bf16) */
  FGR_PATH_SIMT_GEMV = 4,     /* M <= 16: warps stream rows of W with 128-bit loads, shuffle reductions (bf16; no softmax;
                                 chosen automatically for M <= 4) */
  FGR_PATH_UMMA_TF32X3 = 5    /* fp32 on tensor cores: X and W are split into tf32 hi + lo planes (in the workspace) and
                                 tcgen05 kind::tf32 accumulates hi*hi + hi*lo + lo*hi in fp32; fp32-level accuracy
                                 (about 2^-21 per product); chosen automatically for large compute-bound fp32 problems */
} fgr_path;

typedef struct fgr_desc {
  uint32_t struct_bytes;   /* = sizeof(fgr_desc) */
  int32_t batch, M, N, K;
  int32_t dtype;           /* fgr_dtype of X, W and Y/P */
  int32_t act;             /* fgr_act */
  int32_t scale_kind;      /* fgr_scale_kind */
  int32_t reduce;          /* fgr_reduce */
  float scale;             /* the scalar s when scale_kind == FGR_SCALE_SCALAR */
  int32_t write_y;         /* 1: also write y to Y (SOFTMAX always writes P to Y) */
  int64_t ldx, ldw, ldy;   /* row strides in elements; 0 = packed (K, K, N) */
  int64_t bsx, bsw, bsy;   /* batch strides in elements; 0 = packed (M*ldx, N*ldw, M*ldy) */
  int32_t bias_per_batch;  /* 0: bias[N] shared by all batches; 1: bias[batch, N] */
  int32_t device;          /* CUDA device ordinal */
  int32_t force_path;      /* fgr_path; FGR_PATH_AUTO lets the shape decide */
  int32_t force_tile_n;    /* 0 = automatic; else the N extent of a tcgen05 tile (multiple of 16, 16..256) */
  int32_t force_cta_pair;  /* 0 = automatic; 1 = every CTA alone (128-row tiles); 2 = clusters of two CTAs
                              sharing 256-row tiles (tcgen05 cta_group::2; needs tile_n % 32 == 0) */
  int32_t force_ksub;      /* 0 = automatic; else 1, 2 or 4: 64-wide K sub-blocks per shared-memory ring stage */
  int32_t conv_taps;       /* 0 or 1: plain GEMM.  R > 1: 1-D convolution as an implicit GEMM (the operator category
                              "convolution", Section 1 and Section 4.1; 1-D is the paper's case study, Section 4.4).
                              X is then the channels-last input [batch, L, C] with L = M + R - 1 and C = K / R,
                              W the filters [batch, N, R * C] (tap-major, channel-minor), stride 1, no padding:
                                z[b, l, n] = sum_r sum_c X[b, l + r, c] * W[n, r * C + c],   l = 0 .. M - 1.
                              Output row l of the GEMM reads the K = R * C contiguous elements that start at
                              X[b, l, 0], so the rows of the implicit matrix overlap: ldx = 0 means C (stride 1); a
                              convolution of stride s has ldx = s * C (then L = (M - 1) * s + R; any multiple of C is
                              taken as such a stride, channel padding is not supported); bsx defaults to the signal
                              length times C; nothing is copied or unfolded.  K % R == 0 and C a multiple of 8 (bf16)
                              / 4 (fp32).  fgr_run_static takes plain GEMMs only. */
  int32_t w_shared;        /* 0: W is [batch, N, K] (one weight matrix per batch element).  1: W is one [N, K] matrix
                              used by every batch element (bsw is ignored) - a filter bank shared by all signals of
                              a convolution, or one linear layer applied to a batch of inputs */
  int32_t conv_rows;       /* 0 or 1: not a 2-D convolution.  R > 1: 2-D convolution as an implicit GEMM (the operator
                              category "convolution", Section 1 and Section 4.1), stride 1, no padding, no dilation:
                              X is the channels-last image [batch, H, conv_width, C], W the filters [N, R, S, C] with
                              S = conv_taps (0 or 1 mean S = 1) and C = K / (R * S),
                                z[b, p, q, n] = sum_r sum_s sum_c X[b, p + r, q + s, c] * W[n, r, s, c].
                              The output keeps the image's row pitch: GEMM row m = p * conv_width + q, so Y is
                              [batch, P, conv_width, N] seen as [batch, M, N] with M = (P - 1) * conv_width + Q rows
                              (P = H - R + 1, Q = conv_width - S + 1), and so is `out`.  Rows with q >= Q are not outputs
                              of the convolution (their windows wrap into the next image row): they hold finite
                              values of no meaning and the caller skips them.  Nothing is copied or unfolded: filter
                              row r of output row m reads the S * C contiguous elements at X[b, (m + r * conv_width), 0].
                              ldx must be 0 (= C); bsx defaults to the smallest image that holds the M windows; the
                              image must hold (M - 1 + (R - 1) * conv_width + S) pixels.  Needs w_shared = 1 or batch = 1;
                              bf16 on the tiled / streaming tensor-core paths, fp32 (and bf16) on the CUDA-core path. */
  int32_t conv_width;      /* image row length in pixels when conv_rows > 1 (>= S) */
} fgr_desc;

/* What fgr_plan / fgr_create decided; plain host data, for callers, tests and benchmarks. */
typedef struct fgr_plan_info {
  int32_t path;            /* fgr_path actually used */
  int32_t tile_m, tile_n;  /* output tile of one CTA, or of one CTA pair (tile_m = 256) */
  int32_t stages;          /* depth of the shared-memory operand ring (0 for SIMT paths) */
  int32_t parts_per_row;   /* number of split-N partial pairs per row in the workspace */
  int32_t grid;            /* CTAs of the main kernel */
  int32_t launches;        /* kernels launched by one fgr_run */
  int32_t smem_bytes;      /* dynamic shared memory of the main kernel */
  int32_t cta_pair;        /* 2 if the main kernel runs as clusters of two CTAs, else 1 */
  int32_t ksub;            /* 64-wide K sub-blocks per ring stage (tcgen05 paths; 0 for SIMT) */
  int64_t num_tiles;       /* output tiles in the problem */
  uint64_t workspace_bytes;/* what fgr_run needs */
  double flop;             /* 2 * batch * M * N * K */
  double min_bytes;        /* operands read once + outputs written once */
} fgr_plan_info;

typedef struct fgr_handle fgr_handle; /* opaque */

/*
 * fgr_plan: validates a descriptor and reports path, tiling and workspace size.  Pure host
 * arithmetic: touches no device, so it works without a GPU.  `num_sms` is the SM count to
 * size the grid for (<= 0: 148).  This is the shape -> path selection: arithmetic intensity
 * 2MNK / bytes against the machine's flop/byte ridge decides between the compute-bound tiled
 * path and the weight-streaming path; dtype and M pick the SIMT paths.  (The paper's
 * counterpart is the Conductor's bottleneck classification from profile metrics, Section 3.1;
 * here it is a deterministic host rule.)
 */
FGR_API int fgr_plan(const fgr_desc* desc /*host*/, int num_sms, fgr_plan_info* info /*host, out*/);

/*
 * fgr_create: fgr_plan + device checks (the device must be compute capability 10.x, else
 * FGR_ERR_ARCH) + kernel attribute set-up.  *out receives a handle that the caller frees with
 * fgr_destroy.  No device memory is allocated.
 */
FGR_API int fgr_create(const fgr_desc* desc /*host*/, fgr_handle** out /*host, out*/);

/* Bytes of device workspace fgr_run needs (>= 256; 0 if h is NULL).  Contents need no initialisation when a
 * workspace address is first given to a handle: fgr_run clears the status word at its head then.  While the
 * same handle keeps being given the same address, the first 256 bytes belong to the library: if other code
 * has written there in between (a caching allocator that recycled the block), zero those 256 bytes before
 * the next fgr_run, or fgr_get_status may report the leftover value as an error code. */
FGR_API size_t fgr_workspace_bytes(const fgr_handle* h);

/* Copies the plan of a handle into *info. */
FGR_API int fgr_get_plan(const fgr_handle* h, fgr_plan_info* info /*host, out*/);

/*
 * fgr_run: enqueues the whole operator (GEMM mainloop, fused epilogue, per-tile row reduction,
 * split-N merge, softmax normalisation) on `cuda_stream` and returns without synchronising.  It launches
 * one to four kernels (fgr_plan_info.launches); on the tensor-core paths the softmax normalisation kernel
 * runs beside the main kernel and follows it block of rows by block of rows (the main kernel never waits for
 * it); all of them are complete, in stream order, before anything enqueued after fgr_run starts.
 *   X, W       device, dtype, read-only
 *   bias       device fp32 [N] (or [batch, N]); NULL = no bias
 *   scale_vec  device fp32 [N]; required iff scale_kind == FGR_SCALE_PER_COLUMN
 *   Y          device, dtype, [batch, M, N]; required iff write_y or SOFTMAX
 *   out        device fp32: [batch*M] (LSE) or [batch*M, 2] (MAXSUM, MAX_SUMEXP, MEANVAR).  SOFTMAX: optional;
 *              if not NULL it receives [batch*M, 2] = (row max, sum of exp(y - max)), the statistics
 *              that P was normalised with (what fgr_combine_shards needs)
 *   workspace  device, 256-byte aligned, at least fgr_workspace_bytes(h); scratch for the
 *              split-N partial pairs and the device status word.  Two runs that overlap in time
 *              must not share a workspace.
 *   cuda_stream  a cudaStream_t passed as void*; NULL = the default stream
 * Results are bit-identical from run to run (the merge order is fixed; no floating atomics).
 * The call only enqueues kernels; after one ordinary call with the same pointers (which clears the
 * workspace's status word and encodes the tensor maps) it can be captured into a CUDA graph.
 */
FGR_API int fgr_run(fgr_handle* h, const void* X, const void* W, const float* bias, const float* scale_vec,
            void* Y, float* out, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * fgr_run_host: the same operator on HOST buffers (same shapes; packed or strided exactly as the
 * descriptor says).  Copies the inputs to device staging buffers owned by the handle (allocated on
 * the first call, freed by fgr_destroy), runs, copies Y / out back and synchronises before
 * returning.  Returns the device status as fgr_get_status would.  Pinned host memory makes the
 * copies asynchronous and faster but is not required.  Problems of at least four batches, or of one batch
 * and at least 1024 rows (plain GEMMs), are run as four chunks - blocks of batches or of rows, which are
 * independent - on three streams, so that the copy in of one chunk, the kernels of the previous one and
 * the copy out of the one before overlap; the results are those of the whole problem.
 */
FGR_API int fgr_run_host(fgr_handle* h, const void* X, const void* W, const float* bias, const float* scale_vec,
                 void* Y, float* out);

/*
 * fgr_set_residual: a further epilogue of the operator class, the skip connection (fused chains of
 * operators are what the paper's method rewrites, Section 1 and Section 4.1):
 *     y = act(z + b) * s + R[batch, M, N]
 * with R in the dtype of X / W / Y.  The residual is added after activation and scale, before the row
 * reduction and before Y is rounded and stored.  R is a device pointer (16-byte aligned) used by every
 * later fgr_run of this handle until it is set again; NULL removes it.  ldr / bsr: row and batch strides
 * in elements, 0 = packed (N, M * ldr); multiples of 8 (bf16) / 4 (fp32).  R may be the same buffer as Y
 * with the same strides (every element is read before it is written, by the same thread), except for
 * SOFTMAX, whose second pass rewrites Y.  fgr_run_host and fgr_run_static take no residual.
 */
FGR_API int fgr_set_residual(fgr_handle* h, const void* R /*device*/, int64_t ldr, int64_t bsr);

/*
 * fgr_get_status: synchronises the stream of the last fgr_run and returns the device status
 * word: FGR_OK, or FGR_ERR_DEVICE_TIMEOUT if a bounded wait inside a kernel gave up (the kernels
 * never trap and never spin without a limit), or FGR_ERR_CUDA if the stream reports an error.
 */
FGR_API int fgr_get_status(fgr_handle* h);

/*
 * fgr_run_static: the same operator for callers that cannot allocate device memory.  (The paper has
 * no counterpart; this is a deployment convenience.)
 *
 * Who needs it: code running where cudaMalloc is not an option - inside a framework whose caching
 * allocator owns the device, in a latency-critical loop that must not take the allocator's locks,
 * or in an embedding that is handed buffers but no allocator.  Such a caller cannot produce the
 * workspace fgr_run asks for, and has no handle.  Here the split-N partial pairs live in a fixed
 * array of FGR_STATIC_SCRATCH_BYTES inside the library image (each GPU that loads the library holds
 * those bytes until the process exits); the caller passes only the descriptor, inputs and outputs.
 * The call makes no allocation call (no cudaMalloc / cudaFree, no allocating library routine) and creates
 * no handle.  One thing to plan for: the CUDA runtime loads a library's device code lazily, so it is the
 * FIRST call on a device that makes the driver load the module holding the array and reserve its
 * FGR_STATIC_SCRATCH_BYTES.  Make that first call at start-up, before the device's memory is handed
 * to whoever owns it; a first call on a device that is already full fails with FGR_ERR_CUDA.  Later
 * calls leave the device's free memory unchanged.
 *
 *   - Always uses the CUDA-core path (FGR_PATH_SIMT; force_path must be AUTO or SIMT), fp32 or bf16.
 *     Results are those of fgr_run on that path.
 *   - Size limit: batch * M * ceil(N / 64) * 8 bytes must fit in FGR_STATIC_SCRATCH_BYTES, else
 *     FGR_ERR_WORKSPACE is returned and nothing is launched.
 *   - X, W, bias, scale_vec, Y, out: device pointers with the meaning and alignment fgr_run requires
 *     (the same checks are applied).
 *   - The first call on a device looks up the device address of the scratch array and checks the
 *     architecture (under a lock: host threads may race to it); make that first call outside any
 *     stream capture.  Later calls only launch.
 *   - All calls on a device share the one array.  It keeps whatever the previous call left, which is
 *     harmless: every pair the merge pass reads is written earlier in the same call, so nothing has
 *     to be cleared.  Two calls whose kernels may overlap on the GPU (different streams, no ordering
 *     between them) race on the array: order them, or use fgr_run with separate workspaces.
 *   - Asynchronous on `cuda_stream`; launch errors come back as FGR_ERR_CUDA.
 */
#define FGR_STATIC_SCRATCH_BYTES (4u << 20)
FGR_API int fgr_run_static(const fgr_desc* desc /*host*/, const void* X, const void* W, const float* bias,
                           const float* scale_vec, void* Y, float* out, void* cuda_stream);

/*
 * fgr_reduce_rows: stand-alone reduction over the last dimension of a given matrix A[M, N] - the
 * operator category "reduction" (Section 4.1, Datasets); the paper's GPU case study is a max
 * reduction over a dimension (Section 4.4.1).  The same row reductions as the fused operator,
 * applied to A itself, plus plain max and plain sum:
 *     FGR_RED_LSE, FGR_RED_MAXSUM, FGR_RED_MAX_SUMEXP, FGR_RED_MEANVAR, FGR_REDUCE_MAX, FGR_REDUCE_SUM -> out
 *     FGR_RED_SOFTMAX -> P[M, N] in A's dtype (P must not overlap A)
 *   A    device, dtype (fp32 or bf16), row stride lda elements (0 = N), 16-byte aligned, read once
 *        (twice for softmax, the second time normally from L2)
 *   P    device, dtype, row stride ldp (0 = N); required iff SOFTMAX
 *   out  device fp32: [M] (LSE, MAX, SUM) or [M, 2] (MAXSUM, MAX_SUMEXP, MEANVAR); required unless SOFTMAX
 * N, lda and ldp must be multiples of 8 (bf16) / 4 (fp32), else FGR_ERR_UNSUPPORTED.  One kernel
 * launch on `cuda_stream`, asynchronous, no workspace, no handle; bit-identical from run to run.
 * A row is reduced by a warp (short rows), a CTA, or - when there are fewer than about 300 rows (softmax: 1024) and they
 * are long - by a thread-block cluster of 1 to 16 CTAs of 1024 threads (sizes above 8 where the device
 * can hold all rows' clusters at once) whose per-CTA results are combined through
 * distributed shared memory (no scratch memory, still one launch).
 */
enum { FGR_REDUCE_MAX = 4, FGR_REDUCE_SUM = 5 };   /* further values of `reduce` for fgr_reduce_rows only */
typedef struct fgr_reduce_desc {
  uint32_t struct_bytes;   /* = sizeof(fgr_reduce_desc) */
  int32_t M, N;
  int32_t dtype;           /* fgr_dtype of A and P */
  int32_t reduce;          /* fgr_reduce, FGR_REDUCE_MAX or FGR_REDUCE_SUM */
  int32_t device;          /* CUDA device ordinal */
  int64_t lda, ldp;        /* row strides in elements; 0 = packed */
} fgr_reduce_desc;
FGR_API int fgr_reduce_rows(const fgr_reduce_desc* desc /*host*/, const void* A, void* P, float* out, void* cuda_stream);

/*
 * fgr_combine_shards: the exchange step's local half when N is sharded over several GPUs (one
 * process per GPU).  The operator's rows are independent, so sharding over rows or batches needs no
 * exchange; sharding over N (the sensible split for a skinny, weight-streaming problem, where W is
 * almost all of the bytes) leaves every GPU with the statistics of its own column slice.  The
 * problem statement is unchanged: the same outputs as the unsharded operator (Section 3.1,
 * Verifier; Section 3.3).  Protocol, per GPU g of G:
 *   1. fgr_run on the slice W[n_g0:n_g1, :] (bias and scale slices alike) with reduce =
 *      FGR_RED_MAX_SUMEXP (for a final LSE or MAX_SUMEXP), FGR_RED_MAXSUM (final MAXSUM),
 *      FGR_RED_MEANVAR (final MEANVAR) or FGR_RED_SOFTMAX with `out` given (final softmax) -> a local
 *      pair per row, [rows, 2] fp32.  (MEANVAR needs the slice widths to weight the pairs: the slices must
 *      be the contiguous partition of N in groups of 8 (bf16) / 4 (fp32) columns, in shard order, the first
 *      (N / group) % G shards one group wider; n_total = N.)
 *   2. all-gather of the pairs (NCCL; rows * 8 bytes per GPU) -> pairs[G][rows][2] on every GPU;
 *   3. fgr_combine_shards merges the G pairs of every row in ascending shard order (so every GPU
 *      computes bit-identical results) and writes `out` as the unsharded operator would; for softmax
 *      it rescales the local slice P_local[rows, n_local] in place by l_g exp(m_g - m) / l.
 *   pairs    device fp32 [shards][rows][2], 8-byte aligned
 *   out      device fp32 [rows] (LSE) or [rows, 2]; required unless SOFTMAX (there optional: (m, l))
 *   P_local  device, dtype, row stride ldp (0 = n_local), 16-byte aligned; SOFTMAX only
 * n_local and ldp must be multiples of 8 (bf16) / 4 (fp32).  One launch on `cuda_stream`,
 * asynchronous, no workspace.
 */
typedef struct fgr_shard_desc {
  uint32_t struct_bytes;   /* = sizeof(fgr_shard_desc) */
  int32_t shards;          /* G >= 1 */
  int32_t reduce;          /* fgr_reduce of the whole operator */
  int32_t dtype;           /* fgr_dtype of P_local (SOFTMAX only) */
  int32_t shard;           /* this GPU's index in [0, G) (SOFTMAX only) */
  int32_t n_local;         /* columns of this GPU's slice (SOFTMAX only) */
  int32_t device;          /* CUDA device ordinal */
  int32_t n_total;         /* MEANVAR only: N of the whole operator (the shard widths follow from it, see above) */
  int64_t rows;            /* batch * M */
  int64_t ldp;             /* row stride of P_local in elements; 0 = n_local */
} fgr_shard_desc;
FGR_API int fgr_combine_shards(const fgr_shard_desc* desc /*host*/, const float* pairs, float* out, void* P_local,
                               void* cuda_stream);

/*
 * Timing of the main kernel (the GEMM + epilogue + per-tile reduction launch), for benchmarks.
 * fgr_profile_enable(h, 1): from now on fgr_run records a CUDA event before and after its main
 * kernel on the run's stream (at most 4096 runs are kept; later runs are not recorded).
 * fgr_profile_read synchronises those events, returns the summed main-kernel time in
 * milliseconds and the number of runs it covers, and forgets them.  Off by default; this follows
 * the timing protocol of Section 4.1 (Metrics): warm-up runs, then repeated timed runs.
 */
FGR_API int fgr_profile_enable(fgr_handle* h, int enable);
FGR_API int fgr_profile_read(fgr_handle* h, double* main_kernel_ms /*host, out*/, int* runs /*host, out*/);

/*
 * fgr_profile_empty_launches: enqueues n launches of a kernel that does nothing (one warp, no memory
 * access) on `cuda_stream` of `device`, asynchronously.  Timed by the caller with events around the call,
 * it gives the cost of a kernel launch in a back-to-back stream on this machine - the floor under a
 * problem so small that launch latency bounds it (the timing protocol of Section 4.1, Metrics, reports
 * such a problem's microseconds beside that floor rather than a roofline fraction).
 */
FGR_API int fgr_profile_empty_launches(int n, int device, void* cuda_stream);

/* Frees the handle and any staging memory it owns.  NULL is a no-op. */
FGR_API int fgr_destroy(fgr_handle* h);

/* Static strings; never NULL. */
FGR_API const char* fgr_status_string(int status);
FGR_API const char* fgr_path_name(int path);

#ifdef __cplusplus
}
#endif
#endif /* FGR_H_ */
