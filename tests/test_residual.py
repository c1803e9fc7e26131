"""The residual epilogue  y = act(z + b) * s + R : host-side argument checks and GPU parity of every path
against the oracle, through the C ABI."""
import numpy as np
import pytest

import fgr_inputs as gi
import paper_2511_06345_b200 as fgr

REDS = [gi.RED_LSE, gi.RED_SOFTMAX, gi.RED_MAXSUM, gi.RED_MAX_SUMEXP, gi.RED_MEANVAR]


def _problem(dtype, B, M, N, K, act, sk, red, seed, write_y=1):
    return gi.make_problem("res", B, M, N, K, dtype, act, sk, red, scale=0.7, write_y=write_y, x_std=1.0,
                           w_std=2.0 / np.sqrt(K), bias_range=(-0.5, 0.5), scale_range=(-1.5, 1.5), seed=seed, residual_std=2.0)


CASES = [
    # dtype, B, M, N, K, force_path, tile_n, pair
    (gi.DTYPE_F32, 2, 70, 132, 36, fgr.FGR_PATH_SIMT, 0, 0),
    (gi.DTYPE_BF16, 1, 70, 136, 72, fgr.FGR_PATH_SIMT, 0, 0),
    (gi.DTYPE_BF16, 2, 300, 520, 200, fgr.FGR_PATH_UMMA_TILED, 0, 0),
    (gi.DTYPE_BF16, 1, 257, 1000, 136, fgr.FGR_PATH_UMMA_TILED, 240, 1),
    (gi.DTYPE_BF16, 1, 128, 2048, 320, fgr.FGR_PATH_UMMA_STREAM_W, 0, 0),
    (gi.DTYPE_BF16, 2, 3, 520, 136, fgr.FGR_PATH_SIMT_GEMV, 0, 0),
    (gi.DTYPE_F32, 2, 300, 524, 200, fgr.FGR_PATH_UMMA_TF32X3, 0, 0),
]


@pytest.mark.gpu
@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("red", REDS)
def test_residual_matches_oracle(cuda_device, case, red):
    from parity import compare, run_gpu
    dtype, B, M, N, K, path, tn, pair = case
    if path == fgr.FGR_PATH_SIMT_GEMV and red == gi.RED_SOFTMAX:
        pytest.skip("not on the skinny CUDA-core path")
    for i, act in enumerate([gi.ACT_NONE, gi.ACT_GELU_TANH]):
        for wy in (0, 1):
            p = _problem(dtype, B, M, N, K, act, (i + 1) % 3, red, seed=110 + i, write_y=wy)
            Y, out, plan = run_gpu(p, force_path=path, force_tile_n=tn, force_cta_pair=pair)
            assert plan["path"] == path
            kw = {}
            if path == fgr.FGR_PATH_UMMA_TF32X3:
                from test_tf32x3 import _slack
                if red == gi.RED_MEANVAR:
                    import copy
                    q = copy.copy(p); q.reduce = gi.RED_MAXSUM
                    ys, _, _ = _slack(q)
                    kw = dict(y_slack=ys, out_slack=np.stack([ys.mean(1), 8.0 * ys.max(1)], 1))
                else:
                    ys, os_, yr = _slack(p)
                    kw = dict(y_slack=ys, out_slack=os_, y_rel_slack=yr)
            compare(p, Y, out, tcgen05=dtype == gi.DTYPE_BF16 and path != fgr.FGR_PATH_SIMT, **kw)


@pytest.mark.gpu
def test_residual_set_clear_and_in_place(cuda_device):
    """The residual stays set until it is cleared; R may be the Y buffer itself (y += ...)."""
    import torch
    from parity import to_device
    import oracle
    p = _problem(gi.DTYPE_BF16, 1, 200, 264, 72, gi.ACT_RELU, gi.SCALE_NONE, gi.RED_MAXSUM, seed=5)
    X, W, b, s = to_device(p)
    R = torch.from_numpy(p.residual.copy()).view(torch.int16).view(torch.bfloat16).cuda()
    op = fgr.FusedGemmReduce(1, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, write_y=1, device=0)
    Yr, outr, _ = oracle.run_problem(p)
    buf = R.clone().reshape(1, p.M, p.N)
    Y, out = op(X, W, b, s, Y=buf, residual=buf)                 # in place: Y is the residual buffer
    assert op.status() == fgr.FGR_OK
    got = Y.float().cpu().numpy().astype(np.float64).reshape(p.M, p.N)
    assert (np.abs(got - Yr) <= 4.5e-3 * np.abs(Yr) + 2e-5 * (1 + np.abs(Yr).max())).all()
    assert (np.abs(out.cpu().numpy() - outr) <= 2e-4 * (1 + np.abs(outr)) + 1e-6 * np.abs(Yr).sum(1, keepdims=True)).all()
    Y2, out2 = op(X, W, b, s)                                     # cleared: the plain operator again
    q = gi.make_problem("res", 1, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, write_y=1, seed=5)
    q.X, q.W, q.bias = p.X, p.W, p.bias
    Y0, out0, _ = oracle.run_problem(q)
    assert (np.abs(out2.cpu().numpy() - out0) <= 2e-4 * (1 + np.abs(out0)) + 1e-6 * np.abs(Y0).sum(1, keepdims=True)).all()
    op.close()


def test_residual_argument_checks():
    import ctypes
    L = fgr.lib()
    assert L.fgr_set_residual(None, 256, 0, 0) == fgr.FGR_ERR_INVALID_ARG
