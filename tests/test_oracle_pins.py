"""Pins for the CPU oracle: closed forms, invariants, brute force, hand-computed values and
library routines.  None of these re-uses the oracle's own loop, so a dropped term, a wrong
sign or index, or a transposed operand in the oracle fails at least one of them."""
from decimal import Decimal, getcontext
from fractions import Fraction
import math
import os

import numpy as np
import pytest
import torch

import fgr_inputs as gi
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed, tid=7, std=1.0):
    return gi.normal(seed, tid, int(np.prod(shape)), std).reshape(shape)


def _run(X, W, b, s, **kw):
    kw.setdefault("dtype", oracle.F32)
    kw.setdefault("act", oracle.ACT_NONE)
    kw.setdefault("scale_kind", oracle.SCALE_NONE)
    kw.setdefault("reduce", oracle.RED_LSE)
    return oracle.run(X, W, b, s, **kw)


# ---------------------------------------------------------------- hand-computed fixture
def _golden(name):
    for line in open(os.path.join(GOLDEN, "hand_2x2.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        if k == name:
            return np.array([float(x) for x in v])
    raise KeyError(name)


@pytest.mark.parametrize("reduce,key", [(oracle.RED_MAXSUM, "maxsum"), (oracle.RED_LSE, "lse"),
                                        (oracle.RED_MAX_SUMEXP, "max_sumexp"), (oracle.RED_SOFTMAX, "softmax")])
def test_hand_example(reduce, key):
    X = np.array([[1, 0], [1, 1]], dtype=np.float32)
    W = np.array([[1, 2], [3, 4]], dtype=np.float32)
    b = np.array([0, -1], dtype=np.float32)
    s = np.array([2, 0.5], dtype=np.float32)
    Y, out, _ = _run(X, W, b, s, act=oracle.ACT_RELU, scale_kind=oracle.SCALE_PER_COLUMN, reduce=reduce)
    if reduce == oracle.RED_SOFTMAX:
        np.testing.assert_allclose(Y.ravel(), _golden("softmax"), rtol=0, atol=1e-15)
    else:
        np.testing.assert_array_equal(Y.ravel(), _golden("y"))
        np.testing.assert_allclose(out.ravel(), _golden(key), rtol=0, atol=1e-14)


# ---------------------------------------------------------------- GEMM closed forms
@pytest.mark.parametrize("act", [oracle.ACT_NONE, oracle.ACT_RELU])
def test_identity_weights(act):
    """W = I  =>  y = act(X + b) * s exactly."""
    n = 24
    X = _rand((5, n), 1)
    b = gi.uniform(1, 3, n, -0.5, 0.5)
    s = gi.uniform(1, 4, n, -1.5, 1.5)
    Y, _, _ = _run(X, np.eye(n, dtype=np.float32), b, s, act=act, scale_kind=oracle.SCALE_PER_COLUMN,
                   reduce=oracle.RED_MAXSUM)
    u = X.astype(np.float64) + b.astype(np.float64)
    if act == oracle.ACT_RELU:
        u = np.maximum(u, 0)
    np.testing.assert_array_equal(Y, u * s.astype(np.float64))


def test_zero_weights_lse_is_log_n():
    """W = 0, b = 0  =>  every y is 0, LSE = ln N, softmax = 1/N, (max, sum) = (0, 0)."""
    M, N, K = 3, 40, 8
    X, W = _rand((M, K), 2), np.zeros((N, K), np.float32)
    _, out, _ = _run(X, W, None, None, act=oracle.ACT_GELU_TANH)
    np.testing.assert_allclose(out[:, 0], math.log(N), rtol=0, atol=1e-15)
    P, _, _ = _run(X, W, None, None, reduce=oracle.RED_SOFTMAX)
    np.testing.assert_allclose(P, 1.0 / N, rtol=1e-15)
    _, ms, _ = _run(X, W, None, None, reduce=oracle.RED_MAXSUM)
    np.testing.assert_array_equal(ms, 0.0)


def test_zero_weights_bias_only():
    """W = 0  =>  y[m, n] = relu(b[n]) * s for every row."""
    N = 16
    b = gi.uniform(3, 3, N, -1, 1)
    Y, out, _ = _run(_rand((4, 8), 3), np.zeros((N, 8), np.float32), b, None, act=oracle.ACT_RELU,
                     scale_kind=oracle.SCALE_SCALAR, scale=-2.0, reduce=oracle.RED_MAXSUM)
    ref = np.maximum(b.astype(np.float64), 0) * -2.0
    np.testing.assert_array_equal(Y, np.tile(ref, (4, 1)))
    np.testing.assert_array_equal(out[:, 0], ref.max())      # the max is taken after scaling
    np.testing.assert_allclose(out[:, 1], ref.sum(), rtol=1e-15)


def test_one_hot_rows_select_weight_columns():
    """X[m, :] = e_j  =>  z[m, n] = W[n, j]; a transposed operand or swapped index fails this."""
    M, N, K = 6, 10, 7
    W = _rand((N, K), 4)
    js = [0, 3, 6, 1, 5, 2]
    X = np.zeros((M, K), np.float32)
    X[np.arange(M), js] = 1
    Y, _, _ = _run(X, W, None, None, reduce=oracle.RED_MAXSUM)
    np.testing.assert_array_equal(Y, W[:, js].T.astype(np.float64))


@pytest.mark.parametrize("dtype", [oracle.F32, oracle.BF16])
def test_integer_inputs_are_exact(dtype):
    """Small integers: every product and partial sum is an integer, so the result is exact."""
    rng = np.random.default_rng(5)
    B, M, N, K = 2, 9, 11, 33
    Xi, Wi = rng.integers(-8, 9, (B, M, K)), rng.integers(-8, 9, (B, N, K))
    bi = rng.integers(-4, 5, (B, N))
    X, W = Xi.astype(np.float32), Wi.astype(np.float32)
    if dtype == oracle.BF16:
        X, W = gi.f32_to_bf16_bits(X).reshape(X.shape), gi.f32_to_bf16_bits(W).reshape(W.shape)
    Y, out, _ = _run(X, W, bi.astype(np.float32), None, dtype=dtype, reduce=oracle.RED_MAXSUM, bias_per_batch=1)
    Z = np.einsum("bmk,bnk->bmn", Xi, Wi) + bi[:, None, :]
    np.testing.assert_array_equal(Y.reshape(B, M, N), Z.astype(np.float64))
    np.testing.assert_array_equal(out.reshape(B, M, 2)[..., 0], Z.max(-1))
    np.testing.assert_array_equal(out.reshape(B, M, 2)[..., 1], Z.sum(-1))


def test_brute_force_4x4x4_rational():
    """4x4x4 in exact rational arithmetic (ReLU, per-column scale, max+sum), then float LSE."""
    X, W = _rand((4, 4), 6), _rand((4, 4), 6, tid=8)
    b, s = gi.uniform(6, 3, 4, -1, 1), gi.uniform(6, 4, 4, 0.5, 1.5)
    fx = [[Fraction(float(v)) for v in r] for r in X]
    fw = [[Fraction(float(v)) for v in r] for r in W]
    fy = [[max(sum(fx[m][k] * fw[n][k] for k in range(4)) + Fraction(float(b[n])), 0) * Fraction(float(s[n]))
           for n in range(4)] for m in range(4)]
    Y, ms, _ = _run(X, W, b, s, act=oracle.ACT_RELU, scale_kind=oracle.SCALE_PER_COLUMN, reduce=oracle.RED_MAXSUM)
    for m in range(4):
        for n in range(4):
            assert abs(Y[m, n] - float(fy[m][n])) <= 4 * np.spacing(abs(float(fy[m][n])) + 1e-300)
        assert ms[m, 0] == Y[m].max()
        assert abs(ms[m, 1] - float(sum(fy[m]))) < 1e-15
    _, lse, _ = _run(X, W, b, s, act=oracle.ACT_RELU, scale_kind=oracle.SCALE_PER_COLUMN, reduce=oracle.RED_LSE)
    for m in range(4):
        direct = math.log(math.fsum(math.exp(float(v)) for v in fy[m]))   # no max subtraction needed here
        assert abs(lse[m, 0] - direct) < 1e-14


# ---------------------------------------------------------------- GELU (tanh form)
def test_gelu_symmetry_limits_monotone():
    assert oracle.gelu_tanh(0.0) == 0.0
    for x in [1e-3, 0.1, 0.5, 1.0, 2.5, 7.0]:
        assert abs(oracle.gelu_tanh(x) - oracle.gelu_tanh(-x) - x) < 1e-15 * max(1, x)   # tanh is odd
    assert oracle.gelu_tanh(8.0) == pytest.approx(8.0, abs=1e-12)
    assert abs(oracle.gelu_tanh(-8.0)) < 1e-12
    xs = np.linspace(0, 6, 200)
    g = np.array([oracle.gelu_tanh(x) for x in xs])
    assert np.all(np.diff(g) > 0)


def test_gelu_against_decimal_arithmetic():
    """The same function evaluated with 40-digit decimal exponentials (pins the two constants)."""
    getcontext().prec = 40
    pi = Decimal("3.14159265358979323846264338327950288420")
    c = (Decimal(2) / pi).sqrt()
    for x in ["-3.25", "-1", "-0.3", "0.2", "1", "1.7", "4.5"]:
        u = Decimal(x)
        t = c * (u + Decimal("0.044715") * u ** 3)
        e2 = (2 * t).exp()
        ref = Decimal("0.5") * u * (1 + (e2 - 1) / (e2 + 1))
        assert abs(oracle.gelu_tanh(float(x)) - float(ref)) < 2e-16 * max(1.0, abs(float(ref)))


def test_gelu_against_library():
    xs = torch.linspace(-6, 6, 97, dtype=torch.float64)
    ref = torch.nn.functional.gelu(xs, approximate="tanh").numpy()
    got = np.array([oracle.act(oracle.ACT_GELU_TANH, float(x)) for x in xs])
    np.testing.assert_allclose(got, ref, rtol=0, atol=2e-15)
    assert oracle.act(oracle.ACT_RELU, -2.0) == 0.0 and oracle.act(oracle.ACT_RELU, 2.0) == 2.0
    assert oracle.act(oracle.ACT_NONE, -2.0) == -2.0


# ---------------------------------------------------------------- the whole chain vs library routines
def _torch_chain(X, W, b, s_vec, act, scale_kind, scale, reduce, bias_per_batch):
    X, W = torch.as_tensor(X, dtype=torch.float64), torch.as_tensor(W, dtype=torch.float64)
    z = torch.matmul(X, W.transpose(-1, -2))
    if b is not None:
        bb = torch.as_tensor(b, dtype=torch.float64)
        z = z + (bb.reshape(X.shape[0], 1, -1) if bias_per_batch else bb)
    if act == oracle.ACT_RELU:
        z = torch.relu(z)
    elif act == oracle.ACT_GELU_TANH:
        z = torch.nn.functional.gelu(z, approximate="tanh")
    if scale_kind == oracle.SCALE_SCALAR:
        z = z * scale
    elif scale_kind == oracle.SCALE_PER_COLUMN:
        z = z * torch.as_tensor(s_vec, dtype=torch.float64)
    y = z.reshape(-1, z.shape[-1])
    if reduce == oracle.RED_LSE:
        return y, torch.logsumexp(y, 1, keepdim=True)
    if reduce == oracle.RED_SOFTMAX:
        return torch.softmax(y, 1), None
    mx = y.amax(1, keepdim=True)
    if reduce == oracle.RED_MAXSUM:
        return y, torch.cat([mx, y.sum(1, keepdim=True)], 1)
    return y, torch.cat([mx, torch.exp(y - mx).sum(1, keepdim=True)], 1)


@pytest.mark.parametrize("dtype", [oracle.F32, oracle.BF16])
@pytest.mark.parametrize("act", [0, 1, 2])
@pytest.mark.parametrize("scale_kind", [0, 1, 2])
@pytest.mark.parametrize("reduce", [0, 1, 2, 3])
def test_against_fp64_library_chain(dtype, act, scale_kind, reduce):
    B, M, N, K = 2, 7, 19, 13
    seed = 100 + 16 * act + 4 * scale_kind + reduce
    Xf, Wf = _rand((B, M, K), seed, std=1.5), _rand((B, N, K), seed, tid=8, std=1.5)
    if dtype == oracle.BF16:
        X, W = gi.f32_to_bf16_bits(Xf).reshape(Xf.shape), gi.f32_to_bf16_bits(Wf).reshape(Wf.shape)
        Xf, Wf = gi.bf16_bits_to_f32(X).reshape(Xf.shape), gi.bf16_bits_to_f32(W).reshape(Wf.shape)
    else:
        X, W = Xf, Wf
    b = gi.uniform(seed, 3, B * N, -1, 1)
    s = gi.uniform(seed, 4, N, -1.5, 1.5)
    Y, out, _ = oracle.run(X, W, b, s, dtype=dtype, act=act, scale_kind=scale_kind, reduce=reduce, scale=0.37,
                           bias_per_batch=1)
    ry, rout = _torch_chain(Xf, Wf, b, s, act, scale_kind, 0.37, reduce, 1)
    np.testing.assert_allclose(Y, ry.numpy(), rtol=1e-12, atol=1e-13)
    if rout is not None:
        np.testing.assert_allclose(out, rout.numpy(), rtol=1e-12, atol=1e-13)


def test_row_subset_and_batch_indexing():
    p = gi.make_problem("t", 3, 5, 8, 16, gi.DTYPE_BF16, gi.ACT_GELU_TANH, gi.SCALE_SCALAR, gi.RED_LSE, scale=0.5, seed=9)
    Yall, oall, _ = oracle.run_problem(p)
    rows = np.array([14, 0, 7, 7, 3])
    Y, o, _ = oracle.run_problem(p, rows=rows, nthreads=2)
    np.testing.assert_array_equal(Y, Yall[rows])
    np.testing.assert_array_equal(o, oall[rows])
    Y1, o1, t1 = oracle.run_problem(p, nthreads=1)
    assert t1 == 1
    np.testing.assert_array_equal(Y1, Yall)      # independent of the thread count
    with pytest.raises(ValueError):
        oracle.run_problem(p, rows=[15])


# ---------------------------------------------------------------- reductions: invariants
def test_lse_bounds_shift_and_ties_between_kinds():
    M, N, K = 9, 50, 12
    X, W, b = _rand((M, K), 11, std=2.0), _rand((N, K), 11, tid=8, std=2.0), gi.uniform(11, 3, N, -1, 1)
    Y, lse, _ = _run(X, W, b, None, reduce=oracle.RED_LSE)
    mx = Y.max(1)
    assert np.all(lse[:, 0] >= mx) and np.all(lse[:, 0] <= mx + math.log(N) + 1e-12)
    _, lse_shift, _ = _run(X, W, b + np.float32(2.0), None, reduce=oracle.RED_LSE)   # b + 2 is exact in fp32 here? compare loosely
    np.testing.assert_allclose(lse_shift[:, 0], lse[:, 0] + 2.0, rtol=0, atol=5e-7)
    _, mse, _ = _run(X, W, b, None, reduce=oracle.RED_MAX_SUMEXP)
    np.testing.assert_array_equal(mse[:, 0], mx)
    assert np.all(mse[:, 1] >= 1.0) and np.all(mse[:, 1] <= N)
    np.testing.assert_allclose(mse[:, 0] + np.log(mse[:, 1]), lse[:, 0], rtol=0, atol=1e-14)
    P, _, _ = _run(X, W, b, None, reduce=oracle.RED_SOFTMAX)
    np.testing.assert_allclose(P.sum(1), 1.0, rtol=0, atol=1e-12)
    assert P.min() >= 0 and P.max() <= 1
    np.testing.assert_allclose(P, np.exp(Y - lse), rtol=1e-12)
    assert np.array_equal(np.argsort(P, 1, kind="stable"), np.argsort(Y, 1, kind="stable"))


def test_lse_all_equal_row_and_large_logits():
    """Equal logits: LSE = y + ln N.  Logits of +-800 (exp overflows in fp64 without the max shift)."""
    N, K = 32, 4
    X = np.ones((1, K), np.float32)
    W = np.full((N, K), 0.25, np.float32)          # z = 1 for every n
    _, lse, _ = _run(X, W, None, None, scale_kind=oracle.SCALE_SCALAR, scale=800.0)
    assert lse[0, 0] == pytest.approx(800.0 + math.log(N), abs=1e-12)
    _, lse, _ = _run(X, W, None, None, scale_kind=oracle.SCALE_SCALAR, scale=-800.0)
    assert lse[0, 0] == pytest.approx(-800.0 + math.log(N), abs=1e-12)
    W[5] = 0.5                                      # one dominant column: z = 2 -> 1600 vs 800
    P, _, _ = _run(X, W, None, None, scale_kind=oracle.SCALE_SCALAR, scale=800.0, reduce=oracle.RED_SOFTMAX)
    assert P[0, 5] == 1.0 and P[0].sum() == 1.0


def test_maxsum_row_sum_is_a_gemv():
    """act = NONE, s = 1:  sum_n y[m, n] = X[m, :] . (sum_n W[n, :]) + sum(b)."""
    M, N, K = 8, 30, 20
    X, W, b = _rand((M, K), 13), _rand((N, K), 13, tid=8), gi.uniform(13, 3, N, -1, 1)
    _, ms, _ = _run(X, W, b, None, reduce=oracle.RED_MAXSUM)
    ref = X.astype(np.float64) @ W.astype(np.float64).sum(0) + b.astype(np.float64).sum()
    np.testing.assert_allclose(ms[:, 1], ref, rtol=0, atol=1e-13)
    _, ms_relu, _ = _run(X, W, b, None, act=oracle.ACT_RELU, reduce=oracle.RED_MAXSUM)
    assert np.all(ms_relu >= 0)


def test_negative_scale_flips_the_max():
    M, N, K = 4, 12, 6
    X, W = _rand((M, K), 14), _rand((N, K), 14, tid=8)
    Y, ms, _ = _run(X, W, None, None, reduce=oracle.RED_MAXSUM)
    _, msn, _ = _run(X, W, None, None, scale_kind=oracle.SCALE_SCALAR, scale=-1.0, reduce=oracle.RED_MAXSUM)
    np.testing.assert_array_equal(msn[:, 0], -Y.min(1))
    np.testing.assert_allclose(msn[:, 1], -ms[:, 1], rtol=1e-15)


def test_bad_arguments_are_rejected():
    X, W = _rand((2, 4), 15), _rand((3, 4), 15, tid=8)
    with pytest.raises(ValueError):
        _run(X, W, None, None, scale_kind=oracle.SCALE_PER_COLUMN)      # needs a vector
    with pytest.raises(TypeError):
        _run(X.astype(np.float64), W, None, None)
    with pytest.raises(ValueError):
        _run(X, _rand((3, 5), 15), None, None)


# ---------------------------------------------------------------- stand-alone reduction over rows
def test_reduce_rows_hand_example():
    """The y matrix of the hand-computed fixture, reduced directly."""
    A = _golden("y").reshape(2, 2).astype(np.float32)
    np.testing.assert_allclose(oracle.reduce_rows(A, dtype=oracle.F32, kind=oracle.RED_LSE)[1], _golden("lse"), atol=1e-14)
    np.testing.assert_allclose(oracle.reduce_rows(A, dtype=oracle.F32, kind=oracle.RED_SOFTMAX)[0].ravel(), _golden("softmax"), atol=1e-15)
    np.testing.assert_array_equal(oracle.reduce_rows(A, dtype=oracle.F32, kind=oracle.RED_MAXSUM)[1].ravel(), _golden("maxsum"))
    np.testing.assert_allclose(oracle.reduce_rows(A, dtype=oracle.F32, kind=oracle.RED_MAX_SUMEXP)[1].ravel(), _golden("max_sumexp"), atol=1e-14)
    np.testing.assert_array_equal(oracle.reduce_rows(A, dtype=oracle.F32, kind=oracle.RED_MAX)[1], [2, 6])
    np.testing.assert_array_equal(oracle.reduce_rows(A, dtype=oracle.F32, kind=oracle.RED_SUM)[1], [3, 9])


@pytest.mark.parametrize("dtype", [oracle.F32, oracle.BF16])
def test_reduce_rows_against_library_and_strides(dtype):
    M, N, lda = 13, 77, 96
    buf = _rand((M, lda), 31, std=3.0)
    if dtype == oracle.BF16:
        bits = gi.f32_to_bf16_bits(buf).reshape(M, lda)
        A, Af = bits[:, :N], torch.from_numpy(gi.bf16_bits_to_f32(bits).reshape(M, lda)[:, :N].copy()).double()
    else:
        A, Af = buf[:, :N], torch.from_numpy(buf[:, :N].copy()).double()
    assert A.strides[0] == lda * A.itemsize                       # a strided view: the padding must be skipped
    get = lambda k: oracle.reduce_rows(A, dtype=dtype, kind=k)
    np.testing.assert_allclose(get(oracle.RED_LSE)[1], torch.logsumexp(Af, 1).numpy(), rtol=1e-13)
    np.testing.assert_allclose(get(oracle.RED_SOFTMAX)[0], torch.softmax(Af, 1).numpy(), rtol=1e-12)
    np.testing.assert_array_equal(get(oracle.RED_MAX)[1], Af.amax(1).numpy())
    np.testing.assert_allclose(get(oracle.RED_SUM)[1], Af.sum(1).numpy(), rtol=0, atol=1e-12)
    ms = get(oracle.RED_MAXSUM)[1]
    np.testing.assert_array_equal(ms[:, 0], Af.amax(1).numpy())
    np.testing.assert_allclose(ms[:, 1], Af.sum(1).numpy(), rtol=0, atol=1e-12)
    mse = get(oracle.RED_MAX_SUMEXP)[1]
    np.testing.assert_allclose(mse[:, 0] + np.log(mse[:, 1]), get(oracle.RED_LSE)[1], atol=1e-13)


def test_reduce_rows_equals_fused_operator_with_identity_weights():
    """Reducing A directly = the fused operator with W = I, no bias, no activation, no scale."""
    n = 40
    A = _rand((9, n), 32, std=2.0)
    for kind in (oracle.RED_LSE, oracle.RED_MAXSUM, oracle.RED_MAX_SUMEXP, oracle.RED_SOFTMAX):
        Y, out, _ = _run(A, np.eye(n, dtype=np.float32), None, None, reduce=kind)
        P, o = oracle.reduce_rows(A, dtype=oracle.F32, kind=kind)
        if kind == oracle.RED_SOFTMAX:
            np.testing.assert_array_equal(P, Y)
        else:
            np.testing.assert_array_equal(o.reshape(out.shape), out)


def test_reduce_rows_large_magnitudes_and_bad_arguments():
    A = np.full((2, 16), 900.0, np.float32)           # exp(900) overflows fp64 without the max shift
    A[1] = -900.0
    lse = oracle.reduce_rows(A, dtype=oracle.F32, kind=oracle.RED_LSE)[1]
    np.testing.assert_allclose(lse, [900 + math.log(16), -900 + math.log(16)], rtol=0, atol=1e-12)
    with pytest.raises(TypeError):
        oracle.reduce_rows(A.astype(np.float64), dtype=oracle.F32, kind=0)
    with pytest.raises(KeyError):
        oracle.reduce_rows(A, dtype=oracle.F32, kind=7)


# ---------------------------------------------------------------- further activations
def test_sigmoid_tanh_silu_closed_forms_and_library():
    sg = lambda x: oracle.act(oracle.ACT_SIGMOID, x)
    th = lambda x: oracle.act(oracle.ACT_TANH, x)
    si = lambda x: oracle.act(oracle.ACT_SILU, x)
    assert sg(0.0) == 0.5 and th(0.0) == 0.0 and si(0.0) == 0.0
    assert sg(1.0) == pytest.approx(0.7310585786300049, abs=1e-16)      # 1 / (1 + e^-1), tabulated
    assert th(1.0) == pytest.approx(0.7615941559557649, abs=1e-16)      # tanh 1, tabulated
    for x in [0.01, 0.3, 1.0, 2.5, 9.0]:
        assert sg(x) + sg(-x) == pytest.approx(1.0, abs=1e-15)           # logistic symmetry
        assert th(x) == -th(-x)                                          # odd
        assert th(x) == pytest.approx(2 * sg(2 * x) - 1, abs=1e-15)      # tanh x = 2 sigmoid(2x) - 1
        assert si(x) == pytest.approx(x * sg(x), rel=1e-15)              # SiLU = x sigmoid(x)
        assert si(x) - si(-x) == pytest.approx(x, rel=1e-14)
    assert sg(40.0) == pytest.approx(1.0, abs=1e-15) and sg(-745.0) >= 0.0 and th(20.0) == 1.0
    xs = torch.linspace(-8, 8, 65, dtype=torch.float64)
    for kind, fn in [(oracle.ACT_SIGMOID, torch.sigmoid), (oracle.ACT_TANH, torch.tanh), (oracle.ACT_SILU, torch.nn.functional.silu)]:
        got = np.array([oracle.act(kind, float(x)) for x in xs])
        np.testing.assert_allclose(got, fn(xs).numpy(), rtol=0, atol=2e-15)


@pytest.mark.parametrize("act,fn", [(oracle.ACT_SIGMOID, torch.sigmoid), (oracle.ACT_TANH, torch.tanh),
                                    (oracle.ACT_SILU, torch.nn.functional.silu)])
def test_further_activations_in_the_chain(act, fn):
    X, W, b = _rand((6, 10), 41, std=1.5), _rand((14, 10), 41, tid=8, std=1.5), gi.uniform(41, 3, 14, -1, 1)
    Y, out, _ = _run(X, W, b, None, act=act, scale_kind=oracle.SCALE_SCALAR, scale=-0.5, reduce=oracle.RED_LSE)
    y = fn(torch.from_numpy(X).double() @ torch.from_numpy(W).double().T + torch.from_numpy(b).double()) * -0.5
    np.testing.assert_allclose(Y, y.numpy(), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(out[:, 0], torch.logsumexp(y, 1).numpy(), rtol=1e-13)


# ---------------------------------------------------------------- 1-D convolution as window matrix
def test_conv1d_windows_hand_example():
    # x [L=4, C=2] = rows (1,2) (3,4) (5,6) (7,8); taps = 2 -> windows (1,2,3,4) (3,4,5,6) (5,6,7,8)
    x = np.arange(1, 9, dtype=np.float32).reshape(1, 4, 2)
    A = oracle.conv1d_windows(x, 2)
    assert A.shape == (1, 3, 4)
    np.testing.assert_array_equal(A[0], [[1, 2, 3, 4], [3, 4, 5, 6], [5, 6, 7, 8]])
    # one filter w[r, c] = ((1, 0), (0, -1)): z[l] = x[l, 0] - x[l + 1, 1] = 1 - 4, 3 - 6, 5 - 8
    w = np.array([[[1, 0], [0, -1]]], dtype=np.float32).reshape(1, 1, 4)
    Y, out, _ = _run(A, w, None, None, reduce=oracle.RED_MAXSUM)
    np.testing.assert_array_equal(Y.ravel(), [-3, -3, -3])
    np.testing.assert_array_equal(oracle.conv1d_windows(x, 1), x)          # one tap: the plain linear layer
    np.testing.assert_array_equal(oracle.conv1d_windows(x, 4)[0], x.reshape(1, 8))
    with pytest.raises(ValueError):
        oracle.conv1d_windows(x, 5)


def test_conv1d_matches_library_fp64_and_shift_kernel():
    B, L, C, N, R = 2, 19, 6, 5, 4
    x = _rand((B, L, C), 51)
    w = _rand((N, R, C), 52, tid=8)
    b = gi.uniform(53, 3, N, -1, 1)
    A = oracle.conv1d_windows(x, R)
    Y, out, _ = oracle.run(A, np.broadcast_to(w.reshape(1, N, R * C), (B, N, R * C)).copy(), b, None, dtype=oracle.F32,
                           act=oracle.ACT_RELU, scale_kind=oracle.SCALE_NONE, reduce=oracle.RED_LSE)
    # library routine: torch's conv1d takes [B, C, L] and weights [N, C, R]
    ref = torch.nn.functional.conv1d(torch.from_numpy(x).double().permute(0, 2, 1), torch.from_numpy(w).double().permute(0, 2, 1),
                                     torch.from_numpy(b).double()).relu().permute(0, 2, 1).reshape(B * (L - R + 1), N)
    np.testing.assert_allclose(Y, ref.numpy(), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(out[:, 0], torch.logsumexp(ref, 1).numpy(), rtol=1e-13)
    # a filter that is 1 at (tap r0, channel c0) and 0 elsewhere copies the shifted input: z[b, l] = x[b, l + r0, c0]
    r0, c0 = 2, 3
    d = np.zeros((1, 1, R * C), np.float32)
    d[0, 0, r0 * C + c0] = 1.0
    Yd, _, _ = oracle.run(A[:1], d, None, None, dtype=oracle.F32, act=oracle.ACT_NONE, scale_kind=oracle.SCALE_NONE, reduce=oracle.RED_MAXSUM)
    np.testing.assert_array_equal(Yd.ravel(), x[0, r0:r0 + L - R + 1, c0].astype(np.float64))


# ---------------------------------------------------------------- 2-D convolution as window matrix
def test_conv2d_windows_hand_example():
    # one channel, a 3 x 3 image 1..9, a 2 x 2 filter: four windows, each (top-left, top-right, bottom-left, bottom-right)
    x = np.arange(1, 10, dtype=np.float32).reshape(1, 3, 3, 1)
    A = oracle.conv2d_windows(x, 2, 2)
    assert A.shape == (1, 4, 4)
    np.testing.assert_array_equal(A[0], [[1, 2, 4, 5], [2, 3, 5, 6], [4, 5, 7, 8], [5, 6, 8, 9]])
    # the filter ((1, 0), (0, -1)) gives top-left minus bottom-right: 1-5, 2-6, 4-8, 5-9
    w = np.array([1, 0, 0, -1], dtype=np.float32).reshape(1, 1, 4)
    Y, _, _ = _run(A, w, None, None, reduce=oracle.RED_MAXSUM)
    np.testing.assert_array_equal(Y.ravel(), [-4, -4, -4, -4])
    # two channels interleave per pixel: window (p, q) = pixels (p,q) (p,q+1) (p+1,q) (p+1,q+1), channels inside
    x2 = np.stack([x[..., 0], 10 * x[..., 0]], -1)
    np.testing.assert_array_equal(oracle.conv2d_windows(x2, 2, 2)[0, 3], [5, 50, 6, 60, 8, 80, 9, 90])
    # a 1 x 1 filter is the plain linear layer on the pixels; a filter of the image's size gives one window
    np.testing.assert_array_equal(oracle.conv2d_windows(x2, 1, 1)[0], x2.reshape(9, 2))
    np.testing.assert_array_equal(oracle.conv2d_windows(x2, 3, 3)[0], x2.reshape(1, 18))
    with pytest.raises(ValueError):
        oracle.conv2d_windows(x, 4, 1)


def test_conv2d_reduces_to_conv1d_and_matches_library_fp64():
    B, H, Wd, C, N, R, S = 2, 7, 9, 4, 5, 3, 2
    x = _rand((B, H, Wd, C), 61)
    w = _rand((N, R, S, C), 62, tid=8)
    b = gi.uniform(63, 3, N, -1, 1)
    A = oracle.conv2d_windows(x, R, S)
    P, Q = H - R + 1, Wd - S + 1
    assert A.shape == (B, P * Q, R * S * C)
    # one filter row (R = 1): every image row is a 1-D convolution of its own
    A1 = oracle.conv2d_windows(x, 1, S)
    for h in range(H):
        np.testing.assert_array_equal(A1[:, h * Q:(h + 1) * Q], oracle.conv1d_windows(x[:, h], S))
    Y, out, _ = oracle.run(A, np.broadcast_to(w.reshape(1, N, R * S * C), (B, N, R * S * C)).copy(), b, None, dtype=oracle.F32,
                           act=oracle.ACT_RELU, scale_kind=oracle.SCALE_NONE, reduce=oracle.RED_LSE)
    # library routine: torch's conv2d takes [B, C, H, W] and weights [N, C, R, S]
    ref = torch.nn.functional.conv2d(torch.from_numpy(x).double().permute(0, 3, 1, 2), torch.from_numpy(w).double().permute(0, 3, 1, 2),
                                     torch.from_numpy(b).double()).relu().permute(0, 2, 3, 1).reshape(B * P * Q, N)
    np.testing.assert_allclose(Y, ref.numpy(), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(out[:, 0], torch.logsumexp(ref, 1).numpy(), rtol=1e-13)
    # a filter that is 1 at (r0, s0, c0) and 0 elsewhere copies the shifted image: z[b, p, q] = x[b, p + r0, q + s0, c0]
    r0, s0, c0 = 2, 1, 3
    d = np.zeros((1, 1, R * S * C), np.float32)
    d[0, 0, (r0 * S + s0) * C + c0] = 1.0
    Yd, _, _ = oracle.run(A[:1], d, None, None, dtype=oracle.F32, act=oracle.ACT_NONE, scale_kind=oracle.SCALE_NONE, reduce=oracle.RED_MAXSUM)
    np.testing.assert_array_equal(Yd.reshape(P, Q), x[0, r0:r0 + P, s0:s0 + Q, c0].astype(np.float64))


# ---------------------------------------------------------------- mean / variance over N
def test_meanvar_closed_forms():
    N = 12
    # W = I, b = 0: y = X.  Row 0 constant (variance 0), row 1 the sequence 0 .. N-1: mean (N-1)/2, variance (N^2-1)/12
    X = np.stack([np.full(N, 3.25, np.float32), np.arange(N, dtype=np.float32)])
    _, out, _ = _run(X, np.eye(N, dtype=np.float32), None, None, reduce=oracle.RED_MEANVAR)
    np.testing.assert_allclose(out, [[3.25, 0.0], [(N - 1) / 2, (N * N - 1) / 12]], rtol=0, atol=1e-15)
    out2 = oracle.reduce_rows(X, dtype=oracle.F32, kind=oracle.RED_MEANVAR)[1]
    np.testing.assert_array_equal(out2, out)
    # two values a, b: mean (a+b)/2, variance ((a-b)/2)^2 -- a large common offset must not spoil it
    A = np.array([[1.0e6 + 1.0, 1.0e6 + 3.0]], np.float32)
    np.testing.assert_allclose(oracle.reduce_rows(A, dtype=oracle.F32, kind=oracle.RED_MEANVAR)[1], [[1.0e6 + 2.0, 1.0]], rtol=0, atol=0)


def test_meanvar_matches_library_and_invariants():
    X, W, b = _rand((7, 20), 61, std=2.0), _rand((33, 20), 61, tid=8), gi.uniform(61, 3, 33, -1, 1)
    Y, out, _ = _run(X, W, b, None, act=oracle.ACT_GELU_TANH, reduce=oracle.RED_MEANVAR)
    y = torch.nn.functional.gelu(torch.from_numpy(X).double() @ torch.from_numpy(W).double().T + torch.from_numpy(b).double(),
                                 approximate="tanh")
    np.testing.assert_allclose(Y, y.numpy(), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(out[:, 0], y.mean(1).numpy(), rtol=1e-13)
    np.testing.assert_allclose(out[:, 1], y.var(1, unbiased=False).numpy(), rtol=1e-12)
    # tie to the (max, sum) kind: mean = sum / N
    _, ms, _ = _run(X, W, b, None, act=oracle.ACT_GELU_TANH, reduce=oracle.RED_MAXSUM)
    np.testing.assert_allclose(out[:, 0], ms[:, 1] / 33, rtol=1e-14)
    # no activation: shifting every bias by c shifts the mean by c and leaves the variance; scaling by a scales it by a^2
    _, o0, _ = _run(X, W, b, None, reduce=oracle.RED_MEANVAR)
    _, o1, _ = _run(X, W, (b + 2.5).astype(np.float32), None, reduce=oracle.RED_MEANVAR)
    np.testing.assert_allclose(o1[:, 0] - o0[:, 0], 2.5, atol=1e-6)
    np.testing.assert_allclose(o1[:, 1], o0[:, 1], rtol=1e-6)
    _, o2, _ = _run(X, W, b, None, scale_kind=oracle.SCALE_SCALAR, scale=-3.0, reduce=oracle.RED_MEANVAR)
    np.testing.assert_allclose(o2[:, 0], -3.0 * o0[:, 0], rtol=1e-13)
    np.testing.assert_allclose(o2[:, 1], 9.0 * o0[:, 1], rtol=1e-13)
    assert (out[:, 1] >= 0).all()


def test_meanvar_merge_of_slices_is_exact_identity():
    """The pairwise update used to merge per-tile (mean, M2) pairs:  delta = mean_b - mean_a,
    mean = mean_a + delta n_b / n,  M2 = M2_a + M2_b + delta^2 n_a n_b / n  reproduces the whole-row
    statistics from any split of the row (checked in fp64 on the oracle's own output)."""
    A = _rand((5, 200), 62, std=3.0) + 7.0
    whole = oracle.reduce_rows(A.astype(np.float32), dtype=oracle.F32, kind=oracle.RED_MEANVAR)[1]
    for cuts in ([64, 128, 192], [8], [100], [16, 24, 184]):
        edges = [0] + cuts + [200]
        n = 0.0
        mean = np.zeros(5)
        M2 = np.zeros(5)
        for a, b in zip(edges, edges[1:]):
            part = oracle.reduce_rows(np.ascontiguousarray(A[:, a:b].astype(np.float32)), dtype=oracle.F32, kind=oracle.RED_MEANVAR)[1]
            nb = float(b - a)
            delta = part[:, 0] - mean
            tot = n + nb
            mean = mean + delta * nb / tot
            M2 = M2 + part[:, 1] * nb + delta * delta * n * nb / tot
            n = tot
        np.testing.assert_allclose(mean, whole[:, 0], rtol=1e-13)
        np.testing.assert_allclose(M2 / n, whole[:, 1], rtol=1e-12)


# ---------------------------------------------------------------- residual (skip connection)
def test_residual_closed_forms_and_library():
    X, W, b = _rand((6, 10), 71), _rand((14, 10), 71, tid=8), gi.uniform(71, 3, 14, -1, 1)
    R = _rand((6, 14), 72, tid=5, std=3.0)
    # W = 0: y = act(b) * s + R exactly
    Y, out, _ = oracle.run(X, np.zeros_like(W), b, None, dtype=oracle.F32, act=oracle.ACT_RELU, scale_kind=oracle.SCALE_SCALAR,
                           scale=2.0, reduce=oracle.RED_MAXSUM, residual=R)
    want = np.maximum(b.astype(np.float64), 0) * 2.0 + R.astype(np.float64)
    np.testing.assert_allclose(Y, want, rtol=0, atol=1e-15)
    np.testing.assert_allclose(out, np.stack([want.max(1), want.sum(1)], 1), rtol=1e-15)
    # the residual is added AFTER activation and scale (not inside the activation): library chain in fp64
    Y, out, _ = oracle.run(X, W, b, None, dtype=oracle.F32, act=oracle.ACT_GELU_TANH, scale_kind=oracle.SCALE_SCALAR, scale=-0.5,
                           reduce=oracle.RED_LSE, residual=R)
    y = torch.nn.functional.gelu(torch.from_numpy(X).double() @ torch.from_numpy(W).double().T + torch.from_numpy(b).double(),
                                 approximate="tanh") * -0.5 + torch.from_numpy(R).double()
    np.testing.assert_allclose(Y, y.numpy(), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(out[:, 0], torch.logsumexp(y, 1).numpy(), rtol=1e-13)
    # a zero residual changes nothing; rows can be sampled; bf16 residual bits are widened exactly
    Y0, out0, _ = oracle.run(X, W, b, None, dtype=oracle.F32, act=oracle.ACT_NONE, scale_kind=oracle.SCALE_NONE, reduce=oracle.RED_SOFTMAX)
    Y1, _, _ = oracle.run(X, W, b, None, dtype=oracle.F32, act=oracle.ACT_NONE, scale_kind=oracle.SCALE_NONE, reduce=oracle.RED_SOFTMAX,
                          residual=np.zeros_like(R))
    np.testing.assert_array_equal(Y0, Y1)
    Ys, _, _ = oracle.run(X, W, b, None, dtype=oracle.F32, act=oracle.ACT_NONE, scale_kind=oracle.SCALE_NONE, reduce=oracle.RED_MAXSUM,
                          residual=R, rows=[4, 1])
    Yf, _, _ = oracle.run(X, W, b, None, dtype=oracle.F32, act=oracle.ACT_NONE, scale_kind=oracle.SCALE_NONE, reduce=oracle.RED_MAXSUM, residual=R)
    np.testing.assert_array_equal(Ys, Yf[[4, 1]])
    Xb, Wb, Rb = gi.f32_to_bf16_bits(X), gi.f32_to_bf16_bits(W), gi.f32_to_bf16_bits(R)
    Yb, _, _ = oracle.run(Xb, np.zeros_like(Wb), None, None, dtype=oracle.BF16, act=oracle.ACT_NONE, scale_kind=oracle.SCALE_NONE,
                          reduce=oracle.RED_MAXSUM, residual=Rb)
    np.testing.assert_array_equal(Yb, gi.bf16_bits_to_f32(Rb).reshape(6, 14).astype(np.float64))


def test_conv1d_stride_matches_library_fp64():
    B, L, C, N, R, S = 2, 23, 4, 3, 3, 2
    x = _rand((B, L, C), 54)
    w = _rand((N, R, C), 55, tid=8)
    A = oracle.conv1d_windows(x, R, stride=S)
    assert A.shape == (B, (L - R) // S + 1, R * C)
    np.testing.assert_array_equal(A[1, 4], x[1, 8:11].reshape(-1))            # window l = 4 starts at sample l * S = 8
    Y, _, _ = oracle.run(A, np.broadcast_to(w.reshape(1, N, R * C), (B, N, R * C)).copy(), None, None, dtype=oracle.F32,
                         act=oracle.ACT_NONE, scale_kind=oracle.SCALE_NONE, reduce=oracle.RED_MAXSUM)
    ref = torch.nn.functional.conv1d(torch.from_numpy(x).double().permute(0, 2, 1), torch.from_numpy(w).double().permute(0, 2, 1),
                                     stride=S).permute(0, 2, 1).reshape(-1, N)
    np.testing.assert_allclose(Y, ref.numpy(), rtol=1e-13, atol=1e-15)
