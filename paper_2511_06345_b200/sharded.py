"""The operator with its N dimension sharded over the ranks of a process group (one process per
GPU).  Rows and batches are independent and shard without any exchange; N is the split for skinny,
weight-streaming problems, where W is nearly all of the bytes.  Each rank streams only its slice of
W, computes the row statistics of its slice, and one all-gather of ``rows x 2`` floats per rank
followed by ``fgr_combine_shards`` gives every rank the result of the whole operator.

No arithmetic happens here: the local operator and the combine step are kernels of the library; the
all-gather is torch.distributed (NCCL on GPUs)."""
from __future__ import annotations

import torch

from . import binding as B
from .op import FusedGemmReduce


def shard_range(N: int, world: int, rank: int, align: int = 8):
    """Columns [n0, n1) that ``rank`` owns: contiguous, in rank order, covering [0, N) exactly, every
    boundary a multiple of ``align`` (16-byte rows for the kernels).  The first ``N/align % world``
    ranks hold one more group of ``align`` columns.  N must be a multiple of ``align`` and every rank
    must get at least one group."""
    if N % align:
        raise ValueError("N must be a multiple of %d" % align)
    groups = N // align
    if not 0 <= rank < world or groups < world:
        raise ValueError("cannot give each of %d ranks a non-empty slice of %d columns" % (world, N))
    base, extra = divmod(groups, world)
    g0 = rank * base + min(rank, extra)
    g1 = g0 + base + (1 if rank < extra else 0)
    return g0 * align, g1 * align


def local_reduce_kind(reduce: int) -> int:
    """The reduction each shard runs so that its row statistics can be merged into ``reduce``."""
    if reduce in (B.FGR_RED_LSE, B.FGR_RED_MAX_SUMEXP):
        return B.FGR_RED_MAX_SUMEXP
    if reduce in (B.FGR_RED_MAXSUM, B.FGR_RED_SOFTMAX, B.FGR_RED_MEANVAR):
        return reduce
    raise ValueError("unknown reduction %r" % (reduce,))


def gather_pairs(local_pairs: torch.Tensor, group=None) -> torch.Tensor:
    """All-gathers the per-rank statistics [rows, 2] into [world, rows, 2], index 0 = rank 0.  With no
    initialised process group (a single process) the result is ``local_pairs[None]``."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return local_pairs.unsqueeze(0).contiguous()
    world = dist.get_world_size(group)
    gathered = torch.empty((world,) + tuple(local_pairs.shape), dtype=local_pairs.dtype, device=local_pairs.device)
    dist.all_gather(list(gathered.unbind(0)), local_pairs.contiguous(), group=group)
    return gathered


class NShardedFusedGemmReduce:
    """``Y = act(X W^T + b) s`` + row reduction with W's rows (the columns of Y) split over the ranks
    of ``group``.  Every rank passes all of X and ITS slice of W, bias and scale vector
    (``shard_range(N, world, rank)``); it gets back its slice of Y / P and the full ``out``."""

    def __init__(self, batch, M, N, K, dtype, act, scale_kind, reduce, *, scale=1.0, write_y=0, device=0, group=None,
                 rank=None, world=None):
        import torch.distributed as dist
        on = dist.is_available() and dist.is_initialized()
        self.group = group
        self.world = world if world is not None else (dist.get_world_size(group) if on else 1)
        self.rank = rank if rank is not None else (dist.get_rank(group) if on else 0)
        self.reduce = reduce
        self.dtype = dtype
        self.N = N
        self.n0, self.n1 = shard_range(N, self.world, self.rank, 8 if dtype == B.FGR_BF16 else 4)
        self.rows = batch * M
        self.device_index = device
        self.local = FusedGemmReduce(batch, M, self.n1 - self.n0, K, dtype, act, scale_kind, local_reduce_kind(reduce),
                                     scale=scale, write_y=write_y, device=device)
        self.pairs = torch.empty((self.rows, 2), dtype=torch.float32, device=self.local.device)

    def __call__(self, X, W_local, bias_local=None, scale_local=None):
        Y, _ = self.local(X, W_local, bias_local, scale_local, out=self.pairs)
        gathered = gather_pairs(self.pairs, self.group)
        softmax = self.reduce == B.FGR_RED_SOFTMAX
        out = None
        if not softmax:
            out = torch.empty((self.rows,) if self.reduce == B.FGR_RED_LSE else (self.rows, 2), dtype=torch.float32,
                              device=self.local.device)
        stream = torch.cuda.current_stream(self.local.device).cuda_stream
        B.fgr_combine_shards(self.rows, self.world, self.reduce, gathered, out, Y if softmax else None, dtype=self.dtype,
                             shard=self.rank, n_local=self.n1 - self.n0, device=self.device_index, stream=stream, n_total=self.N)
        return Y, out

    def status(self) -> int:
        return self.local.status()

    def close(self):
        self.local.close()
