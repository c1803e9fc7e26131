"""1-D convolution as an implicit GEMM (conv_taps > 1): the rows of the implicit matrix are overlapping
windows of the channels-last input, addressed through the row stride; nothing is unfolded.  Host
validation on CPU; GPU parity of every path against the oracle's window-matrix definition."""
import numpy as np
import pytest

import fgr_inputs as gi
import paper_2511_06345_b200 as fgr

REDS = [gi.RED_LSE, gi.RED_SOFTMAX, gi.RED_MAXSUM, gi.RED_MAX_SUMEXP]


def test_conv_descriptor_validation():
    d = fgr.make_desc(2, 100, 64, 96, fgr.FGR_BF16, 0, 0, 0, conv_taps=3)       # C = 32
    assert fgr.fgr_plan(d).path in (fgr.FGR_PATH_UMMA_TILED, fgr.FGR_PATH_UMMA_STREAM_W)
    # X is read once: (M + R - 1) * C elements per batch
    assert fgr.fgr_plan(d).min_bytes == 2 * ((102 * 32 + 64 * 96) * 2) + 64 * 4 + 2 * 100 * 4
    with pytest.raises(fgr.FgrError):
        fgr.fgr_plan(fgr.make_desc(1, 100, 64, 100, fgr.FGR_BF16, 0, 0, 0, conv_taps=3))    # K % R != 0
    with pytest.raises(fgr.FgrError):
        fgr.fgr_plan(fgr.make_desc(1, 100, 64, 36, fgr.FGR_BF16, 0, 0, 0, conv_taps=3))     # C = 12 not a multiple of 8
    fgr.fgr_plan(fgr.make_desc(1, 100, 64, 36, fgr.FGR_F32, 0, 0, 0, conv_taps=3))          # fp32: multiples of 4
    with pytest.raises(fgr.FgrError):
        fgr.fgr_plan(fgr.make_desc(1, 100, 64, 96, fgr.FGR_BF16, 0, 0, 0, conv_taps=3, ldx=24))   # ldx < C
    with pytest.raises(fgr.FgrError):
        fgr.fgr_plan(fgr.make_desc(1, 100, 64, 96, fgr.FGR_BF16, 0, 0, 0, conv_taps=3, ldx=40))   # padded channels: windows not contiguous
    fgr.fgr_plan(fgr.make_desc(2, 100, 64, 96, fgr.FGR_BF16, 0, 0, 0, conv_taps=3, ldx=32, bsx=4096))  # gaps between signals are fine
    with pytest.raises(fgr.FgrError):
        fgr.fgr_plan(fgr.make_desc(1, 100, 64, 96, fgr.FGR_BF16, 0, 0, 0, conv_taps=-1))


def _problem(dtype, B, M, N, C, R, act, sk, red, seed, write_y=1, w_shared=0):
    K = R * C
    return gi.make_problem("conv", B, M, N, K, dtype, act, sk, red, scale=0.7, write_y=write_y, x_std=1.0,
                           w_std=2.0 / np.sqrt(K), bias_range=(-0.5, 0.5), scale_range=(-1.5, 1.5), seed=seed, conv_taps=R,
                           w_shared=w_shared)


CASES = [
    # dtype, B, M (= output length), N, C, taps, force_path, tile_n, pair
    (gi.DTYPE_BF16, 1, 300, 264, 64, 3, fgr.FGR_PATH_UMMA_TILED, 0, 0),
    (gi.DTYPE_BF16, 2, 257, 520, 72, 2, fgr.FGR_PATH_UMMA_TILED, 0, 1),     # C not a multiple of the 64-wide k-block
    (gi.DTYPE_BF16, 3, 130, 136, 8, 5, fgr.FGR_PATH_UMMA_TILED, 64, 2),     # a k-block spans several taps
    (gi.DTYPE_BF16, 1, 128, 2048, 32, 4, fgr.FGR_PATH_UMMA_STREAM_W, 0, 0),
    (gi.DTYPE_BF16, 2, 3, 520, 40, 3, fgr.FGR_PATH_SIMT_GEMV, 0, 0),
    (gi.DTYPE_BF16, 2, 70, 136, 24, 3, fgr.FGR_PATH_SIMT, 0, 0),
    (gi.DTYPE_F32, 2, 70, 132, 12, 3, fgr.FGR_PATH_SIMT, 0, 0),
    (gi.DTYPE_F32, 2, 300, 260, 36, 4, fgr.FGR_PATH_UMMA_TF32X3, 0, 0),
]


@pytest.mark.gpu
@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("red", REDS)
def test_conv1d_matches_oracle(cuda_device, case, red):
    from parity import compare, run_gpu
    dtype, B, M, N, C, R, path, tn, pair = case
    if path == fgr.FGR_PATH_SIMT_GEMV and red == gi.RED_SOFTMAX:
        pytest.skip("the skinny CUDA-core path has no softmax")
    for i, act in enumerate([gi.ACT_NONE, gi.ACT_GELU_TANH]):
        p = _problem(dtype, B, M, N, C, R, act, (i + 1) % 3, red, seed=70 + i, w_shared=i)   # per-signal and shared filters
        assert p.X.shape == (B, M + R - 1, C) and p.W.shape[0] == (1 if i else B)
        Y, out, plan = run_gpu(p, force_path=path, force_tile_n=tn, force_cta_pair=pair)
        assert plan["path"] == path
        kw = {}
        if path == fgr.FGR_PATH_UMMA_TF32X3:
            from test_tf32x3 import _slack
            import copy, oracle
            q = copy.copy(p)
            q.X, q.conv_taps = oracle.conv1d_windows(p.X, R), 0
            q.W = np.broadcast_to(p.W, (B,) + p.W.shape[1:])
            ys, os_, yr = _slack(q)
            kw = dict(y_slack=ys, out_slack=os_, y_rel_slack=yr)
        compare(p, Y, out, tcgen05=path not in (fgr.FGR_PATH_SIMT,) and dtype == gi.DTYPE_BF16, **kw)


@pytest.mark.gpu
def test_conv1d_shift_filter_is_exact(cuda_device):
    """A filter that is 1 at one (tap, channel) copies the shifted input: the addressing of every tap
    and channel block, checked exactly."""
    from parity import run_gpu
    B, M, N, C, R = 2, 200, 64, 72, 3
    p = _problem(gi.DTYPE_BF16, B, M, N, C, R, gi.ACT_NONE, gi.SCALE_NONE, gi.RED_MAXSUM, seed=5)
    p.bias = None
    W = np.zeros((B, N, R * C), np.float32)
    picks = [(n % R, (7 * n) % C) for n in range(N)]
    for n, (r, c) in enumerate(picks):
        W[:, n, r * C + c] = 1.0
    p.W = gi.f32_to_bf16_bits(W)
    Y, out, plan = run_gpu(p, force_path=fgr.FGR_PATH_UMMA_TILED)
    x = gi.bf16_bits_to_f32(p.X).astype(np.float64)
    for n, (r, c) in enumerate(picks):
        assert np.array_equal(Y.reshape(B, M, N)[:, :, n], x[:, r:r + M, c])


@pytest.mark.gpu
def test_conv1d_host_buffers(cuda_device):
    """fgr_run_host with the overlapping-row layout: the staging copy takes the signal once."""
    import torch
    from parity import compare
    p = _problem(gi.DTYPE_BF16, 2, 150, 136, 16, 4, gi.ACT_RELU, gi.SCALE_NONE, gi.RED_MAXSUM, seed=8)
    desc = fgr.make_desc(p.batch, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, write_y=1, conv_taps=4)
    h = fgr.fgr_create(desc)
    X = torch.from_numpy(p.X.copy()); W = torch.from_numpy(p.W.copy()); b = torch.from_numpy(p.bias.copy())
    Y = torch.empty((p.batch, p.M, p.N), dtype=torch.int16); out = torch.empty((p.batch * p.M, 2), dtype=torch.float32)
    assert fgr.fgr_run_host(h, X, W, b, None, Y, out) == fgr.FGR_OK
    fgr.fgr_destroy(h)
    Yf = gi.bf16_bits_to_f32(Y.numpy().view(np.uint16)).astype(np.float64).reshape(p.batch * p.M, p.N)
    compare(p, Yf, out.numpy().astype(np.float64))


@pytest.mark.gpu
@pytest.mark.parametrize("case", [(gi.DTYPE_BF16, fgr.FGR_PATH_UMMA_TILED, 2), (gi.DTYPE_BF16, fgr.FGR_PATH_UMMA_STREAM_W, 3),
                                  (gi.DTYPE_BF16, fgr.FGR_PATH_SIMT, 2), (gi.DTYPE_F32, fgr.FGR_PATH_UMMA_TF32X3, 2),
                                  (gi.DTYPE_BF16, fgr.FGR_PATH_UMMA_TILED, 5)])
def test_conv1d_strided(cuda_device, case):
    """Stride s: the row stride of the implicit matrix is s * C (for s > R samples are skipped altogether)."""
    from parity import compare, run_gpu
    dtype, path, stride = case
    B, M, N, C, R = 2, 130, 264, 24, 3
    p = gi.make_problem("conv", B, M, N, R * C, dtype, gi.ACT_GELU_TANH, gi.SCALE_NONE, gi.RED_LSE, write_y=1, x_std=1.0,
                        w_std=2.0 / np.sqrt(R * C), seed=21, conv_taps=R, conv_stride=stride, w_shared=1)
    assert p.X.shape == (B, (M - 1) * stride + R, C)
    Y, out, plan = run_gpu(p, force_path=path)
    assert plan["path"] == path
    kw = {}
    if path == fgr.FGR_PATH_UMMA_TF32X3:
        from test_tf32x3 import _slack
        import copy, oracle
        q = copy.copy(p)
        q.X, q.conv_taps, q.W = oracle.conv1d_windows(p.X, R, stride), 0, np.broadcast_to(p.W, (B,) + p.W.shape[1:])
        ys, os_, yr = _slack(q)
        kw = dict(y_slack=ys, out_slack=os_, y_rel_slack=yr)
    compare(p, Y, out, tcgen05=dtype == gi.DTYPE_BF16 and path != fgr.FGR_PATH_SIMT, **kw)
