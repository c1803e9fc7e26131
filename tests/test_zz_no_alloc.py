"""fgr_run_static - the entry point for callers that cannot allocate device memory (a framework
whose allocator owns the GPU, a latency-critical loop, an embedding that is handed buffers only).
It keeps its scratch in a fixed array inside the library, so it takes no workspace and no handle.

Checked here through the C ABI against fgr_run on the same path (bit for bit: same kernels, same
tiling) and, independently, against the CPU oracle at the tolerances of the other parity tests, on
calls in a row: each later call uses other shapes and data, so anything an earlier call left in the
shared scratch would show.  Also checked: once the first call on the device has been made, a call
leaves the device's free memory exactly as it found it.  This file is collected last on purpose."""
import numpy as np
import pytest
import torch

import fgr_inputs as gi
import paper_2511_06345_b200 as fgr
from parity import compare, to_device

pytestmark = pytest.mark.gpu


def _both(p):
    """Runs the problem through fgr_run (CUDA-core path) and through fgr_run_static."""
    X, W, b, s = to_device(p)
    rows, dev = p.batch * p.M, "cuda:0"
    tdt = torch.float32 if p.dtype == gi.DTYPE_F32 else torch.bfloat16
    need_y = bool(p.write_y) or p.reduce == gi.RED_SOFTMAX
    desc = fgr.make_desc(p.batch, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, scale=p.scale,
                         write_y=p.write_y, bias_per_batch=p.bias_per_batch, force_path=fgr.FGR_PATH_SIMT)
    stream = torch.cuda.current_stream().cuda_stream
    res = []
    for static in (False, True):
        Y = torch.full((p.batch, p.M, p.N), -7.0, dtype=tdt, device=dev) if need_y else None
        out = torch.full((rows, p.out_width), -7.0, dtype=torch.float32, device=dev) if p.out_width else None
        if static:
            fgr.fgr_run_static(desc, X, W, b, s, Y, out, stream)
        else:
            h = fgr.fgr_create(desc)
            ws = torch.empty(fgr.fgr_workspace_bytes(h), dtype=torch.uint8, device=dev)
            fgr.fgr_run(h, X, W, b, s, Y, out, ws, ws.numel(), stream)
            assert fgr.fgr_get_status(h) == fgr.FGR_OK
            fgr.fgr_destroy(h)
        torch.cuda.synchronize()
        res.append((None if Y is None else Y.float().cpu().numpy(), None if out is None else out.cpu().numpy()))
    return res


def _check(p):
    (y0, o0), (y1, o1) = _both(p)
    rows = p.batch * p.M
    # against fgr_run: the same kernels in the same tiling, so not one bit may differ
    if y0 is not None:
        assert np.array_equal(y1, y0)
    if o0 is not None:
        assert np.array_equal(o1, o0) and not np.any(o1 == -7.0)
    # against the oracle, which shares nothing with either entry point: the stated tolerance and the tight bounds
    Y = None if y1 is None else y1.astype(np.float64).reshape(rows, p.N)
    out = None if o1 is None else o1.astype(np.float64).reshape(rows, -1)
    worst = compare(p, Y, out, tcgen05=False)
    official = 1e-4 if p.dtype == gi.DTYPE_F32 else 2e-2
    assert all(v <= official for v in worst.values())


def test_static_scratch_matches_fgr_run_twice_in_a_row(cuda_device):
    first = gi.make_problem("a", 2, 150, 520, 72, gi.DTYPE_F32, gi.ACT_GELU_TANH, gi.SCALE_PER_COLUMN, gi.RED_LSE,
                            write_y=1, seed=71)
    _check(first)
    second = gi.make_problem("b", 1, 90, 136, 40, gi.DTYPE_BF16, gi.ACT_RELU, gi.SCALE_SCALAR, gi.RED_SOFTMAX,
                             scale=3.0, seed=72)
    _check(second)
    third = gi.make_config("c1")                              # the small named workload, max + sum-exp pairs
    third.reduce = gi.RED_MAX_SUMEXP
    _check(third)


def test_static_scratch_leaves_free_memory_unchanged(cuda_device):
    """After the first call on the device (which loads the module that holds the scratch array), a call
    takes nothing from the device: free memory before == free memory after."""
    p = gi.make_problem("m", 1, 70, 136, 40, gi.DTYPE_BF16, gi.ACT_RELU, gi.SCALE_NONE, gi.RED_MAXSUM, seed=73)
    X, W, b, s = to_device(p)
    out = torch.empty((p.M, 2), dtype=torch.float32, device="cuda:0")
    desc = fgr.make_desc(p.batch, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce)
    fgr.fgr_run_static(desc, X, W, b, s, None, out, None)     # the warm first call
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        fgr.fgr_run_static(desc, X, W, b, s, None, out, None)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0


def test_static_scratch_rejects_what_does_not_fit(cuda_device):
    # 8192 rows x ceil(8192 / 64) pairs x 8 bytes = 8 MiB > the 4 MiB array
    desc = fgr.make_desc(1, 8192, 8192, 64, fgr.FGR_BF16, 0, 0, fgr.FGR_RED_LSE)
    assert 8192 * 128 * 8 > fgr.binding.FGR_STATIC_SCRATCH_BYTES
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda")
    o = torch.zeros(8192, dtype=torch.float32, device="cuda")
    assert fgr.fgr_run_static(desc, x, x, None, None, None, o, None, check=False) == fgr.FGR_ERR_WORKSPACE
    desc = fgr.make_desc(1, 64, 64, 64, fgr.FGR_BF16, 0, 0, fgr.FGR_RED_LSE, force_path=fgr.FGR_PATH_UMMA_TILED)
    assert fgr.fgr_run_static(desc, x, x, None, None, None, o, None, check=False) == fgr.FGR_ERR_UNSUPPORTED
    desc = fgr.make_desc(1, 64, 60, 64, fgr.FGR_BF16, 0, 0, fgr.FGR_RED_LSE)
    assert fgr.fgr_run_static(desc, x, x, None, None, None, o, None, check=False) == fgr.FGR_ERR_UNSUPPORTED
