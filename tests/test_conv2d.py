"""2-D convolution as an implicit GEMM (conv_rows > 1): host-side plan / validation checks (no GPU) and GPU
parity against the oracle's window-matrix definition, every valid output element, on the tensor-core paths
(CTA pairs, single CTAs, weight streaming) and the CUDA-core path (fp32 and bf16).

The library keeps the image's row pitch in its output (GEMM row m = p * conv_width + q); rows with q >= Q are
not outputs of the convolution and are skipped here, the others map to the oracle's row p * Q + q."""
import numpy as np
import pytest

import fgr_inputs as gi
import paper_2511_06345_b200 as fgr
from parity import compare, run_gpu


def _desc(B, M, N, K, **kw):
    return fgr.make_desc(B, M, N, K, fgr.FGR_BF16, 0, 0, fgr.FGR_RED_MAXSUM, **kw)


def test_descriptor_validation_and_plan():
    ok = _desc(2, 3 * 20 + 18, 64, 3 * 3 * 16, conv_rows=3, conv_taps=3, conv_width=20, w_shared=1)
    p = fgr.fgr_plan(ok, 148)
    assert p.path in (fgr.FGR_PATH_UMMA_TILED, fgr.FGR_PATH_UMMA_STREAM_W)
    # the image is read once: (M - 1 + (R - 1) * width) * C + S * C elements per batch element, W once
    x_elems = (3 * 20 + 18 - 1 + 2 * 20) * 16 + 3 * 16
    assert p.min_bytes == 2 * x_elems * 2 + 64 * 144 * 2 + 64 * 4 + 2 * 78 * 2 * 4
    for bad in (dict(conv_rows=3, conv_taps=3, conv_width=2, w_shared=1),          # the filter is wider than the image
                dict(conv_rows=3, conv_taps=3, conv_width=20, w_shared=0),         # batched filters
                dict(conv_rows=3, conv_taps=3, conv_width=20, w_shared=1, ldx=32), # stride
                dict(conv_rows=5, conv_taps=3, conv_width=20, w_shared=1)):        # K not a multiple of R * S
        with pytest.raises(fgr.FgrError):
            fgr.fgr_plan(_desc(2, 78, 64, 144, **bad), 148)
    with pytest.raises(fgr.FgrError):      # no 2-D convolution on the GEMV path
        fgr.fgr_plan(_desc(1, 2, 64, 144, conv_rows=3, conv_taps=3, conv_width=20, force_path=fgr.FGR_PATH_SIMT_GEMV), 148)
    f32 = fgr.make_desc(1, 4096, 512, 3 * 3 * 64, fgr.FGR_F32, 0, 0, 0, conv_rows=3, conv_taps=3, conv_width=70)
    assert fgr.fgr_plan(f32, 148).path == fgr.FGR_PATH_SIMT      # fp32: CUDA cores (the operand split has no 2-D form)


def _problem(dtype, B, P, Wd, C, N, R, S, act, sk, red, seed, write_y=1):
    Q = Wd - S + 1
    return gi.make_problem("conv2d", B, (P - 1) * Wd + Q, N, R * S * C, dtype, act, sk, red, scale=0.7, write_y=write_y,
                           x_std=1.0, w_std=2.0 / np.sqrt(R * S * C), bias_range=(-0.5, 0.5), scale_range=(-1.5, 1.5),
                           seed=seed, conv_rows=R, conv_taps=S, conv_width=Wd, w_shared=1)


def _check(p, Y, out, tcgen05):
    """Compares the valid rows (q < Q) with the oracle, whose rows are [batch, P, Q] flattened."""
    import copy
    import oracle
    S, Wd = max(p.conv_taps, 1), p.conv_width
    Q = Wd - S + 1
    P = (p.M - Q) // Wd + 1
    b, pp, q = np.meshgrid(np.arange(p.batch), np.arange(P), np.arange(Q), indexing="ij")
    gpu_rows = (b * p.M + pp * Wd + q).ravel()
    ref = copy.copy(p)                       # the same operator on the explicit window matrix
    ref.X = oracle.conv2d_windows(p.X, p.conv_rows, S)
    ref.conv_rows = ref.conv_taps = ref.conv_width = 0
    ref.M, ref.w_shared = P * Q, 1
    compare(ref, None if Y is None else Y[gpu_rows], None if out is None else out[gpu_rows], tcgen05=tcgen05)
    if Y is not None:
        assert np.isfinite(Y).all()          # the skipped rows hold finite values too


SHAPES = [
    # B, P, width, C, N, R, S, path, tile_n, pair
    (1, 9, 20, 16, 72, 3, 3, fgr.FGR_PATH_UMMA_TILED, 0, 0),      # S C = 48: one zero-filled k-block per filter row
    (2, 30, 17, 64, 264, 3, 3, fgr.FGR_PATH_UMMA_TILED, 64, 2),   # S C = 192 = 3 k-blocks, CTA pairs, ragged M and N
    (2, 30, 17, 64, 264, 3, 3, fgr.FGR_PATH_UMMA_TILED, 128, 1),
    (1, 12, 33, 40, 136, 2, 5, fgr.FGR_PATH_UMMA_TILED, 0, 0),    # S C = 200: 3 k-blocks + a ragged 8-element one
    (3, 6, 24, 32, 520, 5, 1, fgr.FGR_PATH_UMMA_TILED, 0, 0),     # a 5 x 1 filter (S = 1)
    (1, 4, 30, 64, 2048, 3, 3, fgr.FGR_PATH_UMMA_STREAM_W, 0, 0), # few output rows: the weight-streaming shape
    (2, 9, 20, 16, 72, 3, 3, fgr.FGR_PATH_SIMT, 0, 0),
]


@pytest.mark.gpu
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("red", [gi.RED_LSE, gi.RED_SOFTMAX, gi.RED_MAXSUM, gi.RED_MEANVAR])
def test_conv2d_parity_bf16(cuda_device, shape, red):
    B, P, Wd, C, N, R, S, path, tn, pair = shape
    for i, act in enumerate([gi.ACT_NONE, gi.ACT_RELU, gi.ACT_GELU_TANH]):
        p = _problem(gi.DTYPE_BF16, B, P, Wd, C, N, R, S, act, (i + red) % 3, red, seed=400 + i)
        Y, out, plan = run_gpu(p, force_path=path, force_tile_n=tn, force_cta_pair=pair)
        assert plan["path"] == path
        _check(p, Y, out, tcgen05=path != fgr.FGR_PATH_SIMT)


@pytest.mark.gpu
def test_conv2d_parity_fp32(cuda_device):
    for red in (gi.RED_LSE, gi.RED_SOFTMAX):
        p = _problem(gi.DTYPE_F32, 2, 7, 19, 12, 68, 3, 2, gi.ACT_GELU_TANH, gi.SCALE_PER_COLUMN, red, seed=410)
        Y, out, plan = run_gpu(p)
        assert plan["path"] == fgr.FGR_PATH_SIMT
        _check(p, Y, out, tcgen05=False)


@pytest.mark.gpu
def test_conv2d_through_host_buffers(cuda_device):
    p = _problem(gi.DTYPE_BF16, 2, 10, 18, 32, 136, 3, 3, gi.ACT_RELU, gi.SCALE_NONE, gi.RED_MAXSUM, seed=420)
    desc = fgr.make_desc(p.batch, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, write_y=1, conv_rows=3, conv_taps=3,
                         conv_width=18, w_shared=1)
    h = fgr.fgr_create(desc)
    Y = np.zeros((p.batch * p.M, p.N), np.uint16)
    out = np.zeros((p.batch * p.M, 2), np.float32)
    ptr = lambda a: None if a is None else a.ctypes.data
    assert fgr.fgr_run_host(h, ptr(p.X), ptr(p.W), ptr(p.bias), None, ptr(Y), ptr(out)) == fgr.FGR_OK
    fgr.fgr_destroy(h)
    _check(p, gi.bf16_bits_to_f32(Y).reshape(Y.shape).astype(np.float64), out.astype(np.float64), tcgen05=True)
