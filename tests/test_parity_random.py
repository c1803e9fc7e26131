"""GPU parity on seeded random problems: shapes, strides of tiling (tile width, CTA pairs, K sub-blocks),
activation, scaling, reduction kind, bias layout and path are all drawn at random; every case is
compared with the CPU oracle on a sample of rows (all columns)."""
import numpy as np
import pytest

import fgr_inputs as gi
import paper_2511_06345_b200 as fgr
from parity import compare, run_gpu

pytestmark = pytest.mark.gpu


def _draw(rng):
    path = int(rng.choice([fgr.FGR_PATH_AUTO, fgr.FGR_PATH_SIMT, fgr.FGR_PATH_UMMA_TILED, fgr.FGR_PATH_UMMA_STREAM_W,
                           fgr.FGR_PATH_SIMT_GEMV]))
    dtype = gi.DTYPE_F32 if path == fgr.FGR_PATH_SIMT and rng.random() < 0.5 else gi.DTYPE_BF16
    g = 4 if dtype == gi.DTYPE_F32 else 8
    B = int(rng.choice([1, 1, 2, 3]))
    M = int(rng.integers(1, 17)) if path == fgr.FGR_PATH_SIMT_GEMV else int(rng.choice([1, 5, 64, 127, 128, 129, 255, 300, 513]))
    N = int(rng.integers(1, 150)) * g
    K = int(rng.integers(1, 90)) * g
    red = int(rng.integers(0, 4))
    if path == fgr.FGR_PATH_SIMT_GEMV and red == gi.RED_SOFTMAX:
        red = gi.RED_LSE
    kw = {}
    if path in (fgr.FGR_PATH_UMMA_TILED, fgr.FGR_PATH_UMMA_STREAM_W):
        kw["force_tile_n"] = int(rng.choice([0, 0, 16, 32, 64, 96, 128, 160, 256]))
        kw["force_ksub"] = int(rng.choice([0, 1, 2, 3, 4]))
        if path == fgr.FGR_PATH_UMMA_TILED and (kw["force_tile_n"] % 32 == 0):
            kw["force_cta_pair"] = int(rng.choice([0, 1, 2]))
            if kw["force_cta_pair"] == 2 and kw["force_tile_n"] == 0 and N < 256 and ((N + 15) // 16 * 16) % 32:
                kw["force_cta_pair"] = 0          # the automatic width would not halve into whole 16-row groups
    p = gi.make_problem("rnd", B, M, N, K, dtype, int(rng.integers(0, 6)), int(rng.integers(0, 3)), red,
                        scale=float(rng.choice([0.5, -1.25, 3.0])), write_y=int(rng.integers(0, 2)), x_std=1.0,
                        w_std=2.0 / np.sqrt(K), bias_range=(-0.5, 0.5) if rng.random() < 0.8 else None,
                        scale_range=(-1.5, 1.5), bias_per_batch=int(rng.integers(0, 2)), seed=int(rng.integers(1, 1 << 30)))
    return p, path, kw


@pytest.mark.parametrize("case", range(48))
def test_random_problem(cuda_device, case):
    rng = np.random.default_rng(7000 + case)
    p, path, kw = _draw(rng)
    Y, out, plan = run_gpu(p, force_path=path, **kw)
    total = p.batch * p.M
    rows = np.unique(rng.integers(0, total, size=min(total, 24)))
    tc = plan["path"] in (fgr.FGR_PATH_UMMA_TILED, fgr.FGR_PATH_UMMA_STREAM_W)
    compare(p, Y, out, rows=rows, tcgen05=tc)


def _draw_extended(rng):
    """The same with the later features in the draw: the fp32 tensor-core path, (mean, variance), a residual
    tensor, shared weights and 1-D convolution windows."""
    path = int(rng.choice([fgr.FGR_PATH_AUTO, fgr.FGR_PATH_SIMT, fgr.FGR_PATH_UMMA_TILED, fgr.FGR_PATH_UMMA_STREAM_W,
                           fgr.FGR_PATH_SIMT_GEMV, fgr.FGR_PATH_UMMA_TF32X3, fgr.FGR_PATH_UMMA_TF32X3]))
    dtype = gi.DTYPE_F32 if path == fgr.FGR_PATH_UMMA_TF32X3 or (path == fgr.FGR_PATH_SIMT and rng.random() < 0.5) else gi.DTYPE_BF16
    g = 4 if dtype == gi.DTYPE_F32 else 8
    B = int(rng.choice([1, 1, 2, 3]))
    M = int(rng.integers(1, 17)) if path == fgr.FGR_PATH_SIMT_GEMV else int(rng.choice([1, 5, 64, 127, 128, 129, 255, 300, 513]))
    N = int(rng.integers(1, 150)) * g
    taps = int(rng.choice([0, 0, 2, 3, 5]))
    C = int(rng.integers(1, 30)) * g
    K = max(taps, 1) * C
    red = int(rng.choice([0, 1, 2, 3, 6]))
    if path == fgr.FGR_PATH_SIMT_GEMV and red == gi.RED_SOFTMAX:
        red = gi.RED_LSE
    kw = {}
    if path in (fgr.FGR_PATH_UMMA_TILED, fgr.FGR_PATH_UMMA_STREAM_W, fgr.FGR_PATH_UMMA_TF32X3):
        kw["force_tile_n"] = int(rng.choice([0, 0, 16, 32, 64, 96, 128, 160, 256]))
        if path != fgr.FGR_PATH_UMMA_TF32X3:
            kw["force_ksub"] = int(rng.choice([0, 1, 2, 3, 4]))
        if path != fgr.FGR_PATH_UMMA_STREAM_W and kw["force_tile_n"] % 32 == 0 and kw["force_tile_n"]:
            kw["force_cta_pair"] = int(rng.choice([0, 1, 2]))
    p = gi.make_problem("rnd", B, M, N, K, dtype, int(rng.integers(0, 6)), int(rng.integers(0, 3)), red,
                        scale=float(rng.choice([0.5, -1.25, 3.0])), write_y=int(rng.integers(0, 2)), x_std=1.0,
                        w_std=2.0 / np.sqrt(K), bias_range=(-0.5, 0.5) if rng.random() < 0.8 else None,
                        scale_range=(-1.5, 1.5), bias_per_batch=int(rng.integers(0, 2)), seed=int(rng.integers(1, 1 << 30)),
                        conv_taps=taps, w_shared=int(rng.integers(0, 2)), residual_std=1.5 if rng.random() < 0.5 else None)
    return p, path, kw


def check_extended(case_seed):
    import copy
    import oracle
    rng = np.random.default_rng(case_seed)
    p, path, kw = _draw_extended(rng)
    Y, out, plan = run_gpu(p, force_path=path, **kw)
    total = p.batch * p.M
    rows = np.unique(rng.integers(0, total, size=min(total, 24)))
    tc = plan["path"] in (fgr.FGR_PATH_UMMA_TILED, fgr.FGR_PATH_UMMA_STREAM_W)
    slack = {}
    if plan["path"] == fgr.FGR_PATH_UMMA_TF32X3:
        from test_tf32x3 import _slack
        q = copy.copy(p)
        if p.conv_taps > 1:
            q.X, q.conv_taps = oracle.conv1d_windows(p.X, p.conv_taps), 0
        q.W = np.broadcast_to(p.W, (p.batch,) + p.W.shape[1:])
        if p.reduce == gi.RED_MEANVAR:
            q.reduce = gi.RED_MAXSUM
            ys, _, _ = _slack(q, rows)
            slack = dict(y_slack=ys, out_slack=np.stack([ys.mean(1), 12.0 * ys.max(1)], 1))
        else:
            ys, os_, yr = _slack(q, rows)
            slack = dict(y_slack=ys, out_slack=os_, y_rel_slack=yr)
    compare(p, Y, out, rows=rows, tcgen05=tc, **slack)


@pytest.mark.parametrize("case", range(64))
def test_random_problem_extended(cuda_device, case):
    check_extended(9000 + case)
