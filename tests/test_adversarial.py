"""GPU parity on inputs chosen to break a fused epilogue / split-N reduction: logits spread over
+-30, one dominant column placed at tile and half-tile edges, a whole tile far below the rest,
rows that differ in one element, negative per-column scales, ReLU inputs that are all negative,
ragged N tails.  Also the host-buffer entry point."""
import numpy as np
import pytest
import torch

import fgr_inputs as gi
import oracle
import paper_2511_06345_b200 as fgr
from parity import compare, run_gpu, to_device

pytestmark = pytest.mark.gpu

EXP_REDS = [gi.RED_LSE, gi.RED_SOFTMAX, gi.RED_MAX_SUMEXP]


def _base(M, N, K, red, act=gi.ACT_NONE, sk=gi.SCALE_SCALAR, scale=1.0, seed=80, write_y=1, bias=(-0.5, 0.5)):
    return gi.make_problem("adv", 1, M, N, K, gi.DTYPE_BF16, act, sk, red, scale=scale, write_y=write_y, x_std=1.0,
                           w_std=1.0 / np.sqrt(K), bias_range=bias, scale_range=(-1.5, 1.5), seed=seed)


def _set_w_rows(p, rows, value):
    W = gi.bf16_bits_to_f32(p.W).reshape(p.W.shape).copy()
    W[0, rows, :] = value
    p.W = gi.f32_to_bf16_bits(W).reshape(W.shape)


@pytest.mark.parametrize("red", EXP_REDS)
def test_logits_spread_over_sixty(cuda_device, red):
    """Scale 10 turns z ~ N(0,1) into logits of about +-35: exp() of a difference to anything but the
    running maximum would overflow or flush."""
    p = _base(300, 1032, 136, red, scale=10.0)
    Y, out, _ = run_gpu(p)
    compare(p, Y, out)
    Yr, _, _ = oracle.run(p.X, p.W, p.bias, None, dtype=p.dtype, act=p.act, scale_kind=p.scale_kind,
                          reduce=gi.RED_MAXSUM, scale=p.scale)
    assert Yr.max() - Yr.min() > 60


@pytest.mark.parametrize("col", [0, 127, 128, 255, 256, 511, 1031])
def test_dominant_column_at_tile_edges(cuda_device, col):
    """One column 40 above the rest, sitting on a tile edge, a half-tile edge or in the ragged tail."""
    for red in (gi.RED_SOFTMAX, gi.RED_LSE):
        p = _base(140, 1032, 72, red, scale=1.0, bias=None)
        p.bias = np.zeros(p.N, np.float32)
        p.bias[col] = 40.0
        Y, out, _ = run_gpu(p)
        compare(p, Y, out)
        if red == gi.RED_SOFTMAX:
            assert (Y[:, col] > 0.999).all()


@pytest.mark.parametrize("red", EXP_REDS + [gi.RED_MAXSUM])
def test_one_tile_far_below_the_rest(cuda_device, red):
    """Columns 256..511 (one whole tile) sit at -200: their partial pairs must vanish in the merge."""
    p = _base(260, 1024, 72, red, bias=None)
    p.bias = np.zeros(p.N, np.float32)
    p.bias[256:512] = -200.0
    Y, out, _ = run_gpu(p)
    compare(p, Y, out)


def test_rows_identical_but_one_element(cuda_device):
    p = _base(130, 520, 72, gi.RED_LSE, scale=4.0)
    X = gi.bf16_bits_to_f32(p.X).reshape(p.X.shape).copy()
    X[0, :, :] = X[0, 0, :]
    X[0, 77, 13] += 0.5
    p.X = gi.f32_to_bf16_bits(X).reshape(X.shape)
    Y, out, _ = run_gpu(p)
    compare(p, Y, out)
    assert np.ptp(np.delete(out[:, 0], 77)) == 0 and out[77, 0] != out[0, 0]


@pytest.mark.parametrize("red", [gi.RED_MAXSUM, gi.RED_LSE])
def test_negative_per_column_scales(cuda_device, red):
    """All scales negative: the maximum is taken after scaling, so it comes from the smallest act()."""
    p = _base(200, 776, 136, red, act=gi.ACT_GELU_TANH, sk=gi.SCALE_PER_COLUMN)
    p.scale_vec = -np.abs(p.scale_vec) - 0.25
    Y, out, _ = run_gpu(p)
    compare(p, Y, out)


def test_relu_with_all_inputs_negative(cuda_device):
    """Bias -50 makes every ReLU input negative: Y = 0, (max, sum) = (0, 0), LSE = ln N."""
    for red in (gi.RED_MAXSUM, gi.RED_LSE):
        p = _base(150, 520, 72, red, act=gi.ACT_RELU, sk=gi.SCALE_NONE, bias=None)
        p.bias = np.full(p.N, -50.0, np.float32)
        Y, out, _ = run_gpu(p)
        assert (Y == 0).all()
        if red == gi.RED_MAXSUM:
            assert (out == 0).all()
        else:
            np.testing.assert_allclose(out[:, 0], np.log(p.N), rtol=0, atol=2e-6 * np.log(p.N))


@pytest.mark.parametrize("N", [8, 24, 264, 1000, 2056])
def test_ragged_tails_every_reduction(cuda_device, N):
    for red in EXP_REDS + [gi.RED_MAXSUM]:
        p = _base(131, N, 40, red, act=gi.ACT_RELU, sk=gi.SCALE_PER_COLUMN, scale=1.0)
        Y, out, _ = run_gpu(p)
        compare(p, Y, out)
        Y, out, _ = run_gpu(p, force_path=fgr.FGR_PATH_SIMT)
        compare(p, Y, out, tcgen05=False)


def test_host_buffer_entry_point(cuda_device):
    """fgr_run_host: pageable host arrays in, host arrays out, called twice (the staging is reused)."""
    for cfg, kw in [("c2", dict(M=300, N=520, K=136)), ("c3", dict(M=260, N=520, K=72)), ("c1", dict(M=70, N=136, K=64))]:
        p = gi.make_config(cfg, **kw)
        desc = fgr.make_desc(p.batch, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, scale=p.scale,
                             write_y=p.write_y, bias_per_batch=p.bias_per_batch)
        h = fgr.fgr_create(desc)
        rows = p.batch * p.M
        need_y = bool(p.write_y) or p.reduce == gi.RED_SOFTMAX
        ydt = np.float32 if p.dtype == gi.DTYPE_F32 else np.uint16
        for _ in range(2):
            Y = np.zeros((rows, p.N), ydt) if need_y else None
            out = np.full((rows, max(p.out_width, 1)), -7.0, np.float32) if p.out_width else None
            ptr = lambda a: None if a is None else a.ctypes.data
            rc = fgr.fgr_run_host(h, ptr(p.X), ptr(p.W), ptr(p.bias), ptr(p.scale_vec), ptr(Y), ptr(out))
            assert rc == fgr.FGR_OK
            Yf = None if Y is None else (Y if p.dtype == gi.DTYPE_F32 else gi.bf16_bits_to_f32(Y).reshape(Y.shape)).astype(np.float64)
            compare(p, Yf, None if out is None else out.astype(np.float64), tcgen05=p.dtype == gi.DTYPE_BF16)
        fgr.fgr_destroy(h)


def test_host_buffer_entry_point_in_chunks(cuda_device):
    """fgr_run_host splits large problems into four chunks (blocks of rows, or of batches) whose copies and
    kernels overlap on three streams; the chunks must tile the problem exactly.  Shapes: ragged row blocks
    (1100 rows -> 512 + 512 + 76), batches that do not divide by four (6 -> 2 + 2 + 2), per-batch bias,
    softmax (P and no `out`), LSE (one float per row: the chunks' slices of `out` stay 8-byte aligned)."""
    cases = [
        gi.make_config("c2", M=1100, N=520, K=136),
        gi.make_config("c3", M=1030, N=264, K=72, scale=3.0),
        gi.make_config("c5", batch=6, M=130, N=264, K=72, bias_per_batch=1),
        gi.make_config("c4", batch=5, M=64, N=520, K=136, write_y=1),
        gi.make_config("c1", M=1024, N=136, K=64, write_y=1),
    ]
    for p in cases:
        desc = fgr.make_desc(p.batch, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, scale=p.scale,
                             write_y=p.write_y, bias_per_batch=p.bias_per_batch)
        h = fgr.fgr_create(desc)
        rows = p.batch * p.M
        need_y = bool(p.write_y) or p.reduce == gi.RED_SOFTMAX
        ydt = np.float32 if p.dtype == gi.DTYPE_F32 else np.uint16
        for _ in range(2):
            Y = np.zeros((rows, p.N), ydt) if need_y else None
            out = np.full((rows, max(p.out_width, 1)), -7.0, np.float32) if p.out_width else None
            ptr = lambda a: None if a is None else a.ctypes.data
            assert fgr.fgr_run_host(h, ptr(p.X), ptr(p.W), ptr(p.bias), ptr(p.scale_vec), ptr(Y), ptr(out)) == fgr.FGR_OK
            Yf = None if Y is None else (Y if p.dtype == gi.DTYPE_F32 else gi.bf16_bits_to_f32(Y).reshape(Y.shape)).astype(np.float64)
            compare(p, Yf, None if out is None else out.astype(np.float64), tcgen05=p.dtype == gi.DTYPE_BF16)
            assert out is None or not np.any(out == -7.0)
        fgr.fgr_destroy(h)


def test_softmax_back_to_back_runs_share_a_workspace(cuda_device):
    """The softmax normalise kernel runs beside the main kernel and follows per-row-block completion counters in
    the workspace, which the last normalise CTA zeroes.  Sixty runs in a row on one stream and one workspace,
    alternating two problems (so the next run's main kernel is resident while this run's normalise kernel is
    still working): every run must reproduce, bit for bit, what the same problem gives when run alone, and
    that must match the oracle."""
    probs = [gi.make_config("c3", M=1100, N=2056, K=264, scale=2.0, seed=s) for s in (81, 82)]
    desc = fgr.make_desc(1, 1100, 2056, 264, probs[0].dtype, probs[0].act, probs[0].scale_kind, probs[0].reduce, scale=2.0)
    h = fgr.fgr_create(desc)
    assert fgr.fgr_get_plan(h).path == fgr.FGR_PATH_UMMA_TILED
    ws = torch.empty(fgr.fgr_workspace_bytes(h), dtype=torch.uint8, device="cuda")
    dev = [to_device(p) for p in probs]
    stream = torch.cuda.current_stream().cuda_stream
    alone = []
    for (X, W, b, s_) in dev:
        P = torch.empty((1100, 2056), dtype=torch.bfloat16, device="cuda")
        fgr.fgr_run(h, X, W, b, s_, P, None, ws, ws.numel(), stream)
        assert fgr.fgr_get_status(h) == fgr.FGR_OK
        alone.append(P.clone())
    outs = [torch.empty((1100, 2056), dtype=torch.bfloat16, device="cuda") for _ in range(60)]
    for i, P in enumerate(outs):
        X, W, b, s_ = dev[i % 2]
        fgr.fgr_run(h, X, W, b, s_, P, None, ws, ws.numel(), stream)
    assert fgr.fgr_get_status(h) == fgr.FGR_OK
    for i, P in enumerate(outs):
        assert torch.equal(P.view(torch.int16), alone[i % 2].view(torch.int16)), "run %d differs" % i
    for p, P in zip(probs, alone):
        compare(p, P.float().cpu().numpy().astype(np.float64), None)
    fgr.fgr_destroy(h)


def test_null_and_misaligned_pointers_are_rejected(cuda_device):
    p = gi.make_config("c2", M=130, N=264, K=72)
    X, W, b, s = to_device(p)
    h = fgr.fgr_create(fgr.make_desc(1, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, write_y=1))
    ws = torch.empty(fgr.fgr_workspace_bytes(h) + 256, dtype=torch.uint8, device="cuda")
    Y = torch.empty((p.M, p.N), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((p.M, 2), dtype=torch.float32, device="cuda")
    n = fgr.fgr_workspace_bytes(h)
    run = lambda *a: fgr.fgr_run(h, *a, check=False)
    assert run(None, W, b, s, Y, out, ws, n) == fgr.FGR_ERR_INVALID_ARG
    assert run(X, W, b, None, Y, out, ws, n) == fgr.FGR_ERR_INVALID_ARG          # per-column scale needs its vector
    assert run(X, W, b, s, None, out, ws, n) == fgr.FGR_ERR_INVALID_ARG          # write_y needs Y
    assert run(X.data_ptr() + 2, W, b, s, Y, out, ws, n) == fgr.FGR_ERR_INVALID_ARG
    assert run(X, W, b, s, Y, out, None, n) == fgr.FGR_ERR_WORKSPACE
    assert run(X, W, b, s, Y, out, ws, n - 8) == fgr.FGR_ERR_WORKSPACE
    assert run(X, W, b, s, Y, out, ws.data_ptr() + 64, n) == fgr.FGR_ERR_WORKSPACE
    assert run(X, W, b, s, Y, out, ws, n) == fgr.FGR_OK and fgr.fgr_get_status(h) == fgr.FGR_OK
    fgr.fgr_destroy(h)


@pytest.mark.parametrize("path", [fgr.FGR_PATH_UMMA_TILED, fgr.FGR_PATH_UMMA_STREAM_W, fgr.FGR_PATH_SIMT])
@pytest.mark.parametrize("red", [gi.RED_LSE, gi.RED_SOFTMAX, gi.RED_MAXSUM])
def test_non_finite_inputs_stay_in_their_rows(cuda_device, path, red):
    """NaN and infinities in X are outside the contract, but they must neither stall a kernel nor leak
    into other rows: the run completes with a clean device status, the affected rows come out
    non-finite, every other row still matches the oracle."""
    p = _base(128, 520, 136, red, act=gi.ACT_GELU_TANH, seed=91)
    X = gi.bf16_bits_to_f32(p.X).reshape(p.X.shape).copy()
    X[0, 3, 17] = np.nan
    X[0, 70, 5] = np.inf
    X[0, 71, :] = -np.inf
    p.X = gi.f32_to_bf16_bits(X).reshape(X.shape)
    Y, out, plan = run_gpu(p, force_path=path)           # run_gpu asserts the device status word
    bad = [3, 70, 71]
    good = np.array([r for r in range(p.M) if r not in bad])
    compare(p, Y, out, rows=good, tcgen05=path != fgr.FGR_PATH_SIMT)
    assert not np.isfinite(Y[3]).all()
    if out is not None:
        assert not np.isfinite(out[3]).all()
