"""N-sharded operator: each shard owns a slice of W's rows, computes its row statistics, and a
combine step merges the all-gathered pairs.

CPU (not gpu): the slice arithmetic, the merge identity on the oracle (the statistics of the slices,
merged, are the statistics of the whole row), and the exchange itself with two gloo ranks.
GPU: G shards emulated one after the other on one device, their pairs stacked as an all-gather
would leave them, then fgr_combine_shards through the C ABI, against the oracle of the whole operator.
"""
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np
import pytest

import fgr_inputs as gi
import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _slice_problem(p, n0, n1, reduce):
    """The oracle's view of one shard: rows n0..n1 of W with the matching bias / scale slices."""
    W = p.W[:, n0:n1, :]
    b = None if p.bias is None else p.bias.reshape(-1)[n0:n1]
    s = None if p.scale_vec is None else p.scale_vec[n0:n1]
    return oracle.run(p.X, W, b, s, dtype=p.dtype, act=p.act, scale_kind=p.scale_kind, reduce=reduce, scale=p.scale)


def _merge64(pairs, exp_kind):
    """pairs [G, rows, 2] fp64 -> (max, sum) of the whole row, written from the definition."""
    m = pairs[:, :, 0].max(0)
    if exp_kind:
        return m, (pairs[:, :, 1] * np.exp(pairs[:, :, 0] - m[None, :])).sum(0)
    return m, pairs[:, :, 1].sum(0)


def test_shard_range_partitions_n():
    from paper_2511_06345_b200.sharded import shard_range
    for N, world, align in [(16384, 8, 8), (1000, 3, 8), (520, 5, 8), (36, 4, 4), (8, 1, 8), (64, 8, 8)]:
        edges = [shard_range(N, world, r, align) for r in range(world)]
        assert edges[0][0] == 0 and edges[-1][1] == N
        for (a0, a1), (b0, b1) in zip(edges, edges[1:]):
            assert a1 == b0
        sizes = [b - a for a, b in edges]
        assert all(s > 0 and s % align == 0 for s in sizes)
        assert max(sizes) - min(sizes) <= align
    with pytest.raises(ValueError):
        shard_range(16, 4, 0, 8)      # fewer 8-column groups than ranks
    with pytest.raises(ValueError):
        shard_range(20, 2, 0, 8)      # N not a multiple of the alignment


@pytest.mark.parametrize("world", [1, 2, 3, 5])
def test_oracle_slices_merge_to_whole(world):
    """Merging the per-slice statistics reproduces the whole-row result (every kind), so the protocol
    (local MAX_SUMEXP / MAXSUM / SOFTMAX + stats, then merge) computes the operator's definition."""
    from paper_2511_06345_b200.sharded import shard_range
    # logits a few units apart (scale 9), so that the shift between the slices' maxima matters
    p = gi.make_config("c4", M=6, N=200, K=24, seed=3, scale_kind=gi.SCALE_SCALAR, scale=9.0)
    edges = [shard_range(p.N, world, r) for r in range(world)]
    _, whole_se, _ = oracle.run_problem(gi_with(p, gi.RED_MAX_SUMEXP), want_y=False)
    _, whole_ms, _ = oracle.run_problem(gi_with(p, gi.RED_MAXSUM), want_y=False)
    _, whole_lse, _ = oracle.run_problem(gi_with(p, gi.RED_LSE), want_y=False)
    P_whole, _, _ = oracle.run_problem(gi_with(p, gi.RED_SOFTMAX))
    se = np.stack([_slice_problem(p, a, b, gi.RED_MAX_SUMEXP)[1] for a, b in edges])
    ms = np.stack([_slice_problem(p, a, b, gi.RED_MAXSUM)[1] for a, b in edges])
    m, l = _merge64(se, True)
    np.testing.assert_allclose(m, whole_se[:, 0], rtol=0, atol=0)
    np.testing.assert_allclose(l, whole_se[:, 1], rtol=1e-13)
    np.testing.assert_allclose(m + np.log(l), whole_lse[:, 0], rtol=1e-13)
    mm, ss = _merge64(ms, False)
    np.testing.assert_allclose(mm, whole_ms[:, 0], rtol=0, atol=0)
    np.testing.assert_allclose(ss, whole_ms[:, 1], rtol=1e-12, atol=1e-12)
    # (mean, variance): the slices' pairs weighted by the slice widths give the whole row's pair
    mv = np.stack([_slice_problem(p, a, b, gi.RED_MEANVAR)[1] for a, b in edges])
    widths = np.array([b - a for a, b in edges], dtype=np.float64)
    _, whole_mv, _ = oracle.run_problem(gi_with(p, gi.RED_MEANVAR), want_y=False)
    mean = (mv[:, :, 0] * widths[:, None]).sum(0) / p.N
    var = ((mv[:, :, 1] + (mv[:, :, 0] - mean[None, :]) ** 2) * widths[:, None]).sum(0) / p.N
    np.testing.assert_allclose(mean, whole_mv[:, 0], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(var, whole_mv[:, 1], rtol=1e-11)
    for g, (a, b) in enumerate(edges):
        P_loc = _slice_problem(p, a, b, gi.RED_SOFTMAX)[0]
        f = se[g, :, 1] * np.exp(se[g, :, 0] - m) / l
        np.testing.assert_allclose(P_loc * f[:, None], P_whole[:, a:b], rtol=1e-12, atol=1e-300)


def gi_with(p, reduce):
    import copy
    q = copy.copy(p)
    q.reduce = reduce
    return q


WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    sys.path.insert(0, os.path.join(%r, "tests"))
    import numpy as np
    import torch
    import torch.distributed as dist
    import fgr_inputs as gi
    import oracle
    from paper_2511_06345_b200.sharded import shard_range, gather_pairs, local_reduce_kind
    from test_shard_n import _slice_problem, _merge64, gi_with
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    p = gi.make_config("c4", M=5, N=136, K=16, seed=11)      # every rank builds the same problem
    n0, n1 = shard_range(p.N, world, rank)
    for final in (gi.RED_LSE, gi.RED_MAXSUM, gi.RED_MAX_SUMEXP):
        kind = local_reduce_kind(final)
        local = _slice_problem(p, n0, n1, kind)[1]                      # this rank's [rows, 2]
        gathered = gather_pairs(torch.from_numpy(local)).numpy()          # [world, rows, 2], rank order
        assert gathered.shape == (world, p.M, 2)
        np.testing.assert_array_equal(gathered[rank], local)
        other = 1 - rank
        o0, o1 = shard_range(p.N, world, other)
        np.testing.assert_array_equal(gathered[other], _slice_problem(p, o0, o1, kind)[1])
        m, s = _merge64(gathered, kind == gi.RED_MAX_SUMEXP)
        ref = oracle.run_problem(gi_with(p, final), want_y=False)[1]
        got = (m + np.log(s))[:, None] if final == gi.RED_LSE else np.stack([m, s], 1)
        np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)
    dist.barrier()
    dist.destroy_process_group()
    print("rank %%d ok" %% rank)
""") % (ROOT, ROOT)


def test_exchange_two_ranks_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [pr.communicate(timeout=180)[0] for pr in procs]
    for rank, (pr, out) in enumerate(zip(procs, outs)):
        assert pr.returncode == 0, out
        assert "rank %d ok" % rank in out


# ------------------------------------------------------------------------------------------ GPU
def _run_sharded_on_one_gpu(p, world, final):
    """G shards one after the other on cuda:0 (each its own handle and slice of W), pairs stacked in
    shard order, then the combine step.  Returns (Y/P float64 [rows, N] or None, out float64 or None)."""
    import torch
    import paper_2511_06345_b200 as fgr
    from paper_2511_06345_b200.sharded import shard_range, local_reduce_kind
    from parity import to_device
    X, W, b, s = to_device(p)
    rows = p.batch * p.M
    softmax = final == gi.RED_SOFTMAX
    edges = [shard_range(p.N, world, r, 8 if p.dtype == gi.DTYPE_BF16 else 4) for r in range(world)]
    gathered = torch.empty((world, rows, 2), dtype=torch.float32, device="cuda:0")
    slices = []
    for g, (n0, n1) in enumerate(edges):
        op = fgr.FusedGemmReduce(p.batch, p.M, n1 - n0, p.K, p.dtype, p.act, p.scale_kind, local_reduce_kind(final),
                                 scale=p.scale, write_y=p.write_y, device=0)
        Yg, _ = op(X, W[:, n0:n1, :].contiguous(), None if b is None else b[n0:n1].contiguous(),
                   None if s is None else s[n0:n1].contiguous(), out=gathered[g])
        assert op.status() == fgr.FGR_OK
        op.close()
        slices.append(Yg)
    out = None if softmax else torch.empty((rows,) if final == gi.RED_LSE else (rows, 2), dtype=torch.float32, device="cuda:0")
    stats = []
    for g, (n0, n1) in enumerate(edges):
        st = torch.empty((rows, 2), dtype=torch.float32, device="cuda:0") if softmax else out
        fgr.fgr_combine_shards(rows, world, final, gathered, st, slices[g] if softmax else None, dtype=p.dtype, shard=g,
                               n_local=n1 - n0, device=0, n_total=p.N)
        stats.append(st)
        if not softmax:
            break                   # every shard would compute the same `out`
    torch.cuda.synchronize()
    if softmax:
        for st in stats[1:]:
            assert torch.equal(st, stats[0])      # all shards agree bit for bit on the merged statistics
    Y = None
    if slices[0] is not None:
        Y = torch.cat([y.reshape(rows, -1) for y in slices], 1).float().cpu().numpy().astype(np.float64)
    o = None if out is None else out.cpu().numpy().astype(np.float64).reshape(rows, -1)
    return Y, o


@pytest.mark.gpu
@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("final", [gi.RED_LSE, gi.RED_MAXSUM, gi.RED_MAX_SUMEXP, gi.RED_SOFTMAX, gi.RED_MEANVAR])
def test_sharded_bf16_matches_oracle(cuda_device, world, final):
    from parity import compare
    # skinny, streaming-shaped problem with logits several units apart; ragged slices (N / 8 = 65 groups)
    p = gi.make_config("c4", M=40, N=520, K=136, seed=5, scale_kind=gi.SCALE_SCALAR, scale=6.0, reduce=final,
                       write_y=0 if final == gi.RED_SOFTMAX else 1)
    Y, out = _run_sharded_on_one_gpu(p, world, final)
    compare(p, Y, out, softmax_rel=1.35e-2)     # P is rounded to bf16 a third time by the combine step


@pytest.mark.gpu
@pytest.mark.parametrize("final", [gi.RED_LSE, gi.RED_SOFTMAX, gi.RED_MAXSUM, gi.RED_MEANVAR])
def test_sharded_fp32_matches_oracle(cuda_device, final):
    from parity import compare
    p = gi.make_config("c1", M=24, N=100, K=64, seed=2, scale_kind=gi.SCALE_SCALAR, scale=12.0, reduce=final)
    Y, out = _run_sharded_on_one_gpu(p, 3, final)
    compare(p, Y, out, tcgen05=False)


@pytest.mark.gpu
def test_sharded_one_dominant_shard(cuda_device):
    """One shard holds every row's maximum by a wide margin: the other shards' factors underflow to
    zero without producing NaN, and the result is that shard's alone."""
    from parity import compare
    p = gi.make_config("c4", M=16, N=256, K=64, seed=9, reduce=gi.RED_SOFTMAX, bias_range=None)
    p.bias = np.zeros(p.N, dtype=np.float32)
    p.bias[64:128] = 200.0           # GELU(z + 200) = z + 200 for the second of four shards
    Y, out = _run_sharded_on_one_gpu(p, 4, gi.RED_SOFTMAX)
    assert np.isfinite(Y).all() and (Y[:, :64] == 0).all() and (Y[:, 128:] == 0).all()
    compare(p, Y, out, softmax_rel=1.35e-2)


@pytest.mark.gpu
def test_sharded_wrapper_single_rank(cuda_device):
    """The torch-side wrapper with no process group: one shard, combine still runs."""
    import paper_2511_06345_b200 as fgr
    from parity import to_device, compare
    p = gi.make_config("c4", M=128, N=1024, K=256, seed=1)
    X, W, b, s = to_device(p)
    op = fgr.NShardedFusedGemmReduce(p.batch, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, scale=p.scale, device=0)
    assert (op.n0, op.n1, op.world) == (0, p.N, 1)
    _, out = op(X, W, b, s)
    assert op.status() == fgr.FGR_OK
    compare(p, None, out.cpu().numpy().astype(np.float64).reshape(p.M, 1))
    op.close()


def test_combine_rejects_bad_arguments():
    import ctypes
    import paper_2511_06345_b200 as fgr
    L = fgr.lib()
    d = fgr.fgr_shard_desc(ctypes.sizeof(fgr.fgr_shard_desc), 2, fgr.FGR_RED_LSE, fgr.FGR_BF16, 0, 0, 0, 0, 16, 0)
    assert L.fgr_combine_shards(None, 256, 256, None, None) == fgr.FGR_ERR_INVALID_ARG
    assert L.fgr_combine_shards(ctypes.byref(d), None, 256, None, None) == fgr.FGR_ERR_INVALID_ARG      # no pairs
    assert L.fgr_combine_shards(ctypes.byref(d), 256, None, None, None) == fgr.FGR_ERR_INVALID_ARG      # no out
    assert L.fgr_combine_shards(ctypes.byref(d), 260, 256, None, None) == fgr.FGR_ERR_INVALID_ARG       # misaligned
    d.reduce = fgr.FGR_RED_SOFTMAX
    d.n_local, d.shard = 12, 0
    assert L.fgr_combine_shards(ctypes.byref(d), 256, None, 512, None) == fgr.FGR_ERR_UNSUPPORTED       # n_local % 8
    d.n_local, d.shard = 16, 2
    assert L.fgr_combine_shards(ctypes.byref(d), 256, None, 512, None) == fgr.FGR_ERR_INVALID_ARG       # shard >= shards
    d.struct_bytes = 8
    assert L.fgr_combine_shards(ctypes.byref(d), 256, None, 512, None) == fgr.FGR_ERR_INVALID_ARG
