"""GPU parity of the stand-alone row reduction (fgr_reduce_rows) against the CPU oracle, through the
C ABI: every kind, both dtypes, short rows (a warp per row), long rows (a CTA per row), ragged
widths, strided rows, large magnitudes."""
import numpy as np
import pytest
import torch

import fgr_inputs as gi
import oracle
import paper_2511_06345_b200 as fgr

pytestmark = pytest.mark.gpu

KINDS = [fgr.FGR_RED_LSE, fgr.FGR_RED_SOFTMAX, fgr.FGR_RED_MAXSUM, fgr.FGR_RED_MAX_SUMEXP, fgr.FGR_REDUCE_MAX, fgr.FGR_REDUCE_SUM]


def _matrix(M, N, dtype, seed, std=2.0, lda=None):
    lda = lda or N
    a = gi.normal(seed, 9, M * lda, std).reshape(M, lda)
    if dtype == gi.DTYPE_BF16:
        a = gi.f32_to_bf16_bits(a).reshape(M, lda)
    return a


def _run(a_host, N, dtype, kind, ldp=None):
    M, lda = a_host.shape
    t = torch.from_numpy(a_host)
    if dtype == gi.DTYPE_BF16:
        t = t.view(torch.int16).view(torch.bfloat16)
    A = t.cuda()
    tdt = torch.bfloat16 if dtype == gi.DTYPE_BF16 else torch.float32
    ldp = ldp or N
    P = torch.full((M, ldp), 7.0, dtype=tdt, device="cuda") if kind == fgr.FGR_RED_SOFTMAX else None
    w = {fgr.FGR_RED_MAXSUM: 2, fgr.FGR_RED_MAX_SUMEXP: 2}.get(kind, 1)
    out = None if kind == fgr.FGR_RED_SOFTMAX else torch.full((M, w), -7.0, dtype=torch.float32, device="cuda")
    fgr.fgr_reduce_rows(M, N, dtype, kind, A, P, out, lda=lda, ldp=ldp, stream=torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return (None if P is None else P.float().cpu().numpy().astype(np.float64),
            None if out is None else out.cpu().numpy().astype(np.float64))


def _check(a_host, N, dtype, kind, ldp=None):
    P, out = _run(a_host, N, dtype, kind, ldp)
    Pr, outr = oracle.reduce_rows(a_host[:, :N], dtype=dtype, kind=kind)
    Af = (gi.bf16_bits_to_f32(a_host).reshape(a_host.shape) if dtype == gi.DTYPE_BF16 else a_host)[:, :N].astype(np.float64)
    if kind == fgr.FGR_RED_SOFTMAX:
        got = P[:, :N]
        # fp32 output: fast exp2 (2^-22) and one rounding; bf16 output: one rounding to 8 significant bits
        bound = (1e-5 if dtype == gi.DTYPE_F32 else 4.5e-3) * np.abs(Pr) + 1e-9
        assert (np.abs(got - Pr) <= bound).all(), float((np.abs(got - Pr) / bound).max())
        assert np.abs(got.sum(1) - 1).max() <= (1e-5 if dtype == gi.DTYPE_F32 else 1e-2)
        if ldp and ldp > N:
            assert (P[:, N:] == 7.0).all()                    # the padding of P is untouched
        return
    outr = outr.reshape(out.shape)
    err = np.abs(out - outr)
    official = 1e-4 if dtype == gi.DTYPE_F32 else 2e-2
    assert (err / (1 + np.abs(outr))).max() <= official
    # inputs are exact in both dtypes, accumulation is fp32: 1e-5 (1 + |ref|) plus cancellation in sums
    bound = 1e-5 * (1 + np.abs(outr)) + 1e-6 * np.abs(Af).sum(1, keepdims=True) * (kind in (fgr.FGR_RED_MAXSUM, fgr.FGR_REDUCE_SUM))
    assert (err <= bound).all(), float((err / bound).max())
    if kind in (fgr.FGR_RED_MAXSUM, fgr.FGR_RED_MAX_SUMEXP, fgr.FGR_REDUCE_MAX):
        np.testing.assert_array_equal(out[:, 0], Af.max(1))   # a maximum is exact


@pytest.mark.parametrize("dtype", [gi.DTYPE_F32, gi.DTYPE_BF16])
@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("shape", [(1, 8), (5, 24), (70, 1000), (33, 2048), (9, 2056), (300, 8200), (3, 70000)])
def test_reduce_rows_parity(cuda_device, dtype, kind, shape):
    M, N = shape
    N = (N + 7) // 8 * 8
    _check(_matrix(M, N, dtype, seed=90 + M), N, dtype, kind)


@pytest.mark.parametrize("kind", [fgr.FGR_RED_LSE, fgr.FGR_RED_SOFTMAX, fgr.FGR_RED_MAXSUM])
def test_reduce_rows_strided_and_large_magnitudes(cuda_device, kind):
    for dtype in (gi.DTYPE_F32, gi.DTYPE_BF16):
        a = _matrix(40, 1000, dtype, seed=97, std=30.0, lda=1024)        # logits of about +-100
        _check(a, 1000, dtype, kind, ldp=1008)


def test_reduce_rows_deterministic_and_argument_checks(cuda_device):
    a = _matrix(64, 4096, gi.DTYPE_BF16, seed=98)
    r = [_run(a, 4096, gi.DTYPE_BF16, fgr.FGR_RED_LSE)[1] for _ in range(3)]
    assert np.array_equal(r[0], r[1]) and np.array_equal(r[0], r[2])
    x = torch.zeros(64, dtype=torch.float32, device="cuda")
    f = lambda *args, **kw: fgr.fgr_reduce_rows(*args, check=False, **kw)
    assert f(4, 12, fgr.FGR_BF16, fgr.FGR_RED_LSE, x, None, x) == fgr.FGR_ERR_UNSUPPORTED      # N % 8
    assert f(4, 16, fgr.FGR_BF16, fgr.FGR_RED_LSE, x, None, None) == fgr.FGR_ERR_INVALID_ARG    # out missing
    assert f(4, 16, fgr.FGR_BF16, fgr.FGR_RED_SOFTMAX, x, None, x) == fgr.FGR_ERR_INVALID_ARG   # P missing
    assert f(4, 16, fgr.FGR_BF16, 7, x, None, x) == fgr.FGR_ERR_INVALID_ARG
    assert f(4, 16, fgr.FGR_BF16, fgr.FGR_RED_LSE, x, None, x, lda=8) == fgr.FGR_ERR_INVALID_ARG
    assert f(4, 16, fgr.FGR_BF16, fgr.FGR_RED_LSE, x.data_ptr() + 4, None, x) == fgr.FGR_ERR_INVALID_ARG


@pytest.mark.parametrize("dtype", [gi.DTYPE_F32, gi.DTYPE_BF16])
@pytest.mark.parametrize("kind", KINDS)
@pytest.mark.parametrize("shape", [(1, 1048576), (16, 262144), (5, 100008), (2, 33000), (40, 65536 + 8),
                                   (20, 400000), (7, 600008), (100, 131072), (200, 70000), (300, 66000)])
def test_reduce_rows_few_long_rows_cluster(cuda_device, dtype, kind, shape):
    """Few, long rows: a cluster of 1 to 16 CTAs of 1024 threads shares a row (16, 13, 12, 8, 6, 4, 3, 2 and 1
    with these shapes; the last one takes this kernel for softmax only) and the per-CTA states are combined through distributed shared memory (ragged
    segments included)."""
    M, N = shape
    _check(_matrix(M, N, dtype, seed=60 + M, std=3.0), N, dtype, kind)


def test_reduce_rows_cluster_deterministic_and_dominant_segment(cuda_device):
    a = _matrix(4, 524288, gi.DTYPE_BF16, seed=77)
    r = [_run(a, 524288, gi.DTYPE_BF16, fgr.FGR_RED_LSE)[1] for _ in range(3)]
    assert np.array_equal(r[0], r[1]) and np.array_equal(r[0], r[2])
    # the row maximum, by a wide margin, in the last CTA's segment only: the other states rescale to zero
    f = gi.normal(78, 9, 4 * 524288, 1.0).reshape(4, 524288)
    f[:, -5] = 300.0
    for dtype in (gi.DTYPE_F32, gi.DTYPE_BF16):
        a = f if dtype == gi.DTYPE_F32 else gi.f32_to_bf16_bits(f).reshape(f.shape)
        _check(a, 524288, dtype, fgr.FGR_RED_LSE)
        _check(a, 524288, dtype, fgr.FGR_RED_SOFTMAX)
