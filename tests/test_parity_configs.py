"""GPU parity at the full sizes of the five named workloads, in the launch configuration the
benchmark times: EVERY row of every workload is compared element by element with the oracle (all N
columns; the stated tolerance and the tighter derived bounds).  With thread = row, 256-row CTA-pair
tiles and several waves per kernel, a fault confined to one pair, one wave or one TMEM lane quadrant of
a late tile would otherwise hide in rows nobody looked at.  The oracle does a workload in 1 to 10 s on
the 16 cores of a GPU host; rows go through it in blocks so that the fp64 reference of the largest
output (8192 x 8192) never has to exist at once.  FGR_PARITY_ROWS=<n> compares an edge-biased sample
of n rows instead (for a quick look on a small host)."""
import os

import numpy as np
import pytest

import fgr_inputs as gi
import paper_2511_06345_b200 as fgr
from parity import compare, run_gpu, to_device

pytestmark = pytest.mark.gpu


SAMPLE = int(os.environ.get("FGR_PARITY_ROWS", "0"))


def _rows(total, block, count, seed):
    rng = np.random.default_rng(seed)
    edge = [0, 1, block - 1, block, block + 1, total - block, total - 1, total // 2]
    rnd = rng.choice(total, size=count, replace=False).tolist()
    return np.array(sorted(set(r for r in edge + rnd if 0 <= r < total)), dtype=np.int64)


def _blocks(total, block, seed, rows_per_block=1024):
    """The row sets to compare: all rows in consecutive blocks, or (FGR_PARITY_ROWS) one sampled set."""
    if SAMPLE:
        return [_rows(total, block, min(SAMPLE, total), seed)]
    return [np.arange(a, min(a + rows_per_block, total), dtype=np.int64) for a in range(0, total, rows_per_block)]


def compare_all(p, Y, out, block, seed, **kw):
    worst = {}
    for rows in _blocks(p.batch * p.M, block, seed):
        for k, v in compare(p, Y, out, rows=rows, **kw).items():
            worst[k] = max(worst.get(k, 0.0), v)
    return worst


def test_c1_full(cuda_device):
    p = gi.make_config("c1")
    Y, out, plan = run_gpu(p)
    assert plan["path"] == fgr.FGR_PATH_SIMT
    w = compare(p, Y, out, tcgen05=False)
    assert w["out"] <= 1e-4


@pytest.mark.parametrize("reduce", [gi.RED_MAXSUM, gi.RED_MAX_SUMEXP])
def test_c2_every_row(cuda_device, reduce):
    p = gi.make_config("c2", reduce=reduce)
    Y, out, plan = run_gpu(p)
    assert plan["path"] == fgr.FGR_PATH_UMMA_TILED and plan["tile_n"] == 256 and plan["grid"] > 100 and plan["cta_pair"] == 2
    w = compare_all(p, Y, out, 128, 2)
    assert w["Y"] <= 2e-2 and w["out"] <= 2e-2
    # properties that hold for every row: ReLU and positive scales -> max >= 0, sum >= 0, max <= sum
    if reduce == gi.RED_MAXSUM:
        assert (out[:, 0] >= 0).all() and (out[:, 1] >= out[:, 0] - 1e-3).all()
        np.testing.assert_allclose(Y.max(1), out[:, 0], rtol=4e-3, atol=1e-6)     # bf16 Y vs fp32 max
        np.testing.assert_allclose(Y.sum(1), out[:, 1], rtol=2e-3)


def test_c3_softmax_every_row(cuda_device):
    p = gi.make_config("c3")
    Y, out, plan = run_gpu(p)
    assert out is None and plan["parts_per_row"] >= 2          # the split-N merge is exercised
    compare_all(p, Y, out, 128, 3)
    s = Y.sum(1)
    assert np.abs(s - 1).max() <= 1e-2 and Y.min() >= 0 and Y.max() <= 1


def test_c3_shape_with_spread_logits(cuda_device):
    """Same shape, but a scale that spreads the logits over +-25 so that the maximum subtraction and
    the rescaling between tiles matter (at the workload's own scale every P is close to 1/N)."""
    p = gi.make_config("c3", scale=8.0, M=1024)
    Y, out, _ = run_gpu(p)
    compare_all(p, Y, out, 128, 4)
    assert np.abs(Y.sum(1) - 1).max() <= 1e-2


def test_c4_full(cuda_device):
    p = gi.make_config("c4")
    Y, out, plan = run_gpu(p)
    assert plan["path"] == fgr.FGR_PATH_UMMA_STREAM_W and Y is None
    assert plan["num_tiles"] == plan["grid"] <= 148            # every CTA streams its share of W exactly once
    w = compare(p, Y, out)
    assert w["out"] <= 2e-2
    pw = gi.make_config("c4", write_y=1)
    Y, out, _ = run_gpu(pw, tensors=to_device(pw))
    compare(pw, Y, out)


@pytest.mark.parametrize("reduce", [gi.RED_MAXSUM, gi.RED_MAX_SUMEXP])
def test_c5_batched_every_row(cuda_device, reduce):
    p = gi.make_config("c5", reduce=reduce)
    Y, out, plan = run_gpu(p)
    assert Y is None and plan["cta_pair"] == 2
    compare_all(p, Y, out, 1024, 6)
    if reduce == gi.RED_MAXSUM:
        assert (out >= 0).all()
    pw = gi.make_config("c5", write_y=1, batch=4)
    Y, out, _ = run_gpu(pw)
    compare_all(pw, Y, out, 1024, 7)


def test_f2_fp32_tensor_core_every_row(cuda_device):
    """The benchmark's fp32 workload (c2's shapes and epilogue in fp32: the 3xTF32 path) at full size."""
    from test_tf32x3 import _slack
    p = gi.make_config("c2", dtype=gi.DTYPE_F32)
    Y, out, plan = run_gpu(p)
    assert plan["path"] == fgr.FGR_PATH_UMMA_TF32X3 and plan["cta_pair"] == 2 and plan["tile_n"] == 256
    w = {"Y": 0.0, "out": 0.0}
    for rows in _blocks(p.M, 128, 8, rows_per_block=512):
        ys, os_, yr = _slack(p, rows)
        wb = compare(p, Y, out, rows=rows, tcgen05=False, y_slack=ys, out_slack=os_, y_rel_slack=yr)
        w = {k: max(w[k], wb[k]) for k in w}
    assert w["Y"] <= 1e-4 and w["out"] <= 1e-4
    assert (out[:, 0] >= 0).all() and (out[:, 1] >= out[:, 0] - 1e-4).all()


def test_v2_convolution_every_row(cuda_device):
    """The benchmark's convolution workload at full size: 8 signals of 2051 x 512 channels, 4096 shared
    filters of 4 taps, c2's epilogue."""
    p = gi.make_config("c2", batch=8, M=2048, N=4096, K=2048, conv_taps=4, w_shared=1)
    assert p.X.shape == (8, 2051, 512) and p.W.shape == (1, 4096, 2048)
    Y, out, plan = run_gpu(p)
    assert plan["path"] == fgr.FGR_PATH_UMMA_TILED and plan["num_tiles"] == 1024
    import copy
    import oracle
    for rows in _blocks(p.batch * p.M, 2048, 9):
        # the oracle's window matrix for this block of rows only (the full one would be 8 x 2048 x 2048)
        q = copy.copy(p)
        q.conv_taps, q.batch, q.M = 0, 1, len(rows)
        q.X = np.stack([p.X[r // p.M, (r % p.M):(r % p.M) + 4, :].reshape(-1) for r in rows])[None]
        q.W = p.W
        Yr, outr, _ = oracle.run_problem(q)
        got_y, got_o = Y[rows], out[rows]
        assert (np.abs(got_y - Yr) <= 4.5e-3 * np.abs(Yr) + 2e-5 * (1 + np.abs(Yr).max())).all()
        assert (np.abs(got_o - outr) <= 2e-4 * (1 + np.abs(outr)) + 1e-6 * np.abs(Yr).sum(1, keepdims=True)).all()
        assert (np.abs(got_y - Yr) / (1 + np.abs(Yr))).max() <= 2e-2
