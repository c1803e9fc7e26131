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
