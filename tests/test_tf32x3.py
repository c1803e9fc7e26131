"""The fp32 tensor-core path (three tf32 products on split operands): plan selection on the host and
GPU parity against the fp64 oracle at the fp32 path's tolerances, every element of Y / P and of the
reduction, through the C ABI."""
import numpy as np
import pytest

import fgr_inputs as gi
import paper_2511_06345_b200 as fgr

ACTS = [gi.ACT_NONE, gi.ACT_RELU, gi.ACT_GELU_TANH, gi.ACT_SIGMOID, gi.ACT_TANH, gi.ACT_SILU]
REDS = [gi.RED_LSE, gi.RED_SOFTMAX, gi.RED_MAXSUM, gi.RED_MAX_SUMEXP]


def _plan(B, M, N, K, dtype=fgr.FGR_F32, **kw):
    return fgr.fgr_plan(fgr.make_desc(B, M, N, K, dtype, 0, 0, 0, **kw))


def test_plan_selects_tf32x3_for_large_fp32_only():
    assert _plan(1, 256, 256, 256).path == fgr.FGR_PATH_SIMT                 # the small named workload stays on FMA
    big = _plan(1, 4096, 4096, 4096)
    assert big.path == fgr.FGR_PATH_UMMA_TF32X3 and (big.tile_m, big.tile_n, big.cta_pair, big.ksub) == (256, 256, 2, 2)
    assert big.launches == 4 and big.stages >= 3
    # workspace: status + partial pairs + the hi/lo planes of X and W (2 * 4 bytes per element each)
    planes = 2 * 4096 * 2 * 4096 * 4
    assert planes <= big.workspace_bytes <= planes + 4096 * big.parts_per_row * 8 + 1024
    assert _plan(1, 64, 16384, 8192).path == fgr.FGR_PATH_SIMT               # skinny: the split would triple the traffic
    assert _plan(1, 4096, 4096, 4096, dtype=fgr.FGR_BF16).path == fgr.FGR_PATH_UMMA_TILED
    with pytest.raises(fgr.FgrError):
        _plan(1, 256, 256, 256, dtype=fgr.FGR_BF16, force_path=fgr.FGR_PATH_UMMA_TF32X3)
    p = _plan(1, 100, 72, 20, force_path=fgr.FGR_PATH_UMMA_TF32X3)           # K = 20 is padded to one 32-wide block
    assert p.path == fgr.FGR_PATH_UMMA_TF32X3 and p.cta_pair == 1
    assert fgr.fgr_path_name(fgr.FGR_PATH_UMMA_TF32X3) == "umma_tf32x3"


def _problem(B, M, N, K, act, sk, red, seed, write_y=1, std=1.0, bias_per_batch=0, scale=0.7):
    return gi.make_problem("t", B, M, N, K, gi.DTYPE_F32, act, sk, red, scale=scale, write_y=write_y, x_std=std,
                           w_std=std / np.sqrt(K) * 2.0, bias_range=(-0.5, 0.5), scale_range=(-1.5, 1.5),
                           bias_per_batch=bias_per_batch, seed=seed)


def _slack(p, rows=None):
    """Extra absolute allowance of the tensor-core fp32 path.  tcgen05 truncates (rounds toward zero) its
    fp32 accumulator once per instruction; a chunk of 128 K elements is 48 instructions (3 products x 16),
    so a pre-activation sum z carries up to 48 ulp = 5.7e-6 of the largest partial sum on its way, plus
    3 x 2^-22 per product from the tf32 split.  Partial sums are a random walk of the products: their
    size is taken as 4 sqrt(sum_k x^2 w^2), and the allowance on z as 2.5e-6 of that.  Activations
    have slope <= 1.13; the per-column or scalar scale multiplies the error."""
    X2 = p.X.astype(np.float64).reshape(p.batch, p.M, p.K) ** 2
    W2 = p.W.astype(np.float64).reshape(p.batch, p.N, p.K) ** 2
    if rows is None:
        walk = np.sqrt(np.matmul(X2, W2.transpose(0, 2, 1))).reshape(p.batch * p.M, p.N)
    else:
        walk = np.sqrt(np.stack([X2[r // p.M, r % p.M] @ W2[r // p.M].T for r in rows]))
    s = np.abs(p.scale_vec.astype(np.float64))[None, :] if p.scale_kind == gi.SCALE_PER_COLUMN else (
        abs(p.scale) if p.scale_kind == gi.SCALE_SCALAR else 1.0)
    ez = 2.5e-6 * 4.0 * walk * 1.13 * s                       # allowance on y, per element
    mx = ez.max(1)
    if p.reduce == gi.RED_SOFTMAX:
        return None, None, 2.0 * mx[:, None]                  # an error e of the logits is a relative error <= 2 e of P
    mx = ez.max(1)
    if p.reduce == gi.RED_LSE:
        return ez, mx[:, None], None
    if p.reduce == gi.RED_MAXSUM:
        return ez, np.stack([mx, ez.sum(1)], 1), None
    return ez, np.stack([mx, 2.0 * mx * p.N], 1), None        # sum-exp <= N; relative error of each term <= 2 ez


SHAPES = [
    # B, M, N, K, force_tile_n, force_cta_pair
    (1, 1, 4, 4, 0, 0),
    (1, 128, 256, 64, 0, 0),
    (1, 100, 260, 36, 0, 0),       # N tail of 4 columns, K tail of 4
    (1, 300, 524, 200, 0, 0),      # 3 row blocks (CTA pairs), 3 column tiles, ragged everywhere
    (1, 257, 1000, 132, 240, 1),
    (1, 129, 120, 512, 64, 2),
    (3, 130, 268, 72, 0, 0),       # batched, ragged
    (1, 512, 2048, 160, 0, 0),     # more tiles than SMs: persistent loop, both accumulator buffers, ring wrap-around
]


@pytest.mark.gpu
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("red", REDS)
def test_tf32x3_matches_oracle(cuda_device, shape, red):
    from parity import compare, run_gpu
    B, M, N, K, tn, pair = shape
    for i, act in enumerate(ACTS):
        p = _problem(B, M, N, K, act, i % 3, red, seed=40 + i, bias_per_batch=i % 2)
        Y, out, plan = run_gpu(p, force_path=fgr.FGR_PATH_UMMA_TF32X3, force_tile_n=tn, force_cta_pair=pair)
        assert plan["path"] == fgr.FGR_PATH_UMMA_TF32X3
        ys, os_, yr = _slack(p)
        compare(p, Y, out, tcgen05=False, y_slack=ys, out_slack=os_, y_rel_slack=yr)


@pytest.mark.gpu
def test_tf32x3_exact_on_integers(cuda_device):
    """Integer-valued inputs up to 2^11 need the lo plane (tf32 keeps 11 significant bits); their
    products and sums are exact in fp32, so the result must equal the oracle's exactly."""
    from parity import run_gpu
    import oracle
    rng = np.random.default_rng(5)
    p = _problem(1, 200, 264, 96, gi.ACT_NONE, gi.SCALE_NONE, gi.RED_MAXSUM, seed=1)
    p.X = rng.integers(-3000, 3001, size=p.X.shape).astype(np.float32)       # beyond 11 bits: hi + lo both non-zero
    p.W = rng.integers(-3, 4, size=p.W.shape).astype(np.float32)
    p.bias = rng.integers(-8, 9, size=p.N).astype(np.float32)
    Y, out, plan = run_gpu(p, force_path=fgr.FGR_PATH_UMMA_TF32X3)
    Yr, outr, _ = oracle.run_problem(p)
    assert np.array_equal(Y, Yr) and np.array_equal(out, outr)


@pytest.mark.gpu
def test_tf32x3_needs_all_three_products(cuda_device):
    """With W exactly representable in tf32 its lo plane is zero, and X's lo plane carries 1e-3-level
    detail: the result is right only if X_lo W_hi is accumulated.  The transposed case checks X_hi W_lo."""
    from parity import compare, run_gpu
    for which in ("X", "W"):
        p = _problem(1, 130, 264, 64, gi.ACT_NONE, gi.SCALE_NONE, gi.RED_MAXSUM, seed=3)
        coarse = p.W if which == "X" else p.X
        coarse[...] = (coarse.view(np.uint32) & np.uint32(0xFFFFE000)).view(np.float32)   # 10 mantissa bits
        Y, out, _ = run_gpu(p, force_path=fgr.FGR_PATH_UMMA_TF32X3)
        ys, os_, yr = _slack(p)
        compare(p, Y, out, tcgen05=False, y_slack=ys, out_slack=os_, y_rel_slack=yr)


@pytest.mark.gpu
def test_tf32x3_large_auto_sampled_rows(cuda_device):
    """A problem large enough for the automatic selection; sampled rows against the oracle."""
    from parity import compare, run_gpu
    p = gi.make_problem("t", 1, 1024, 2048, 1024, gi.DTYPE_F32, gi.ACT_GELU_TANH, gi.SCALE_PER_COLUMN, gi.RED_LSE,
                        write_y=1, seed=8)
    Y, out, plan = run_gpu(p)
    assert plan["path"] == fgr.FGR_PATH_UMMA_TF32X3 and plan["cta_pair"] == 2
    rows = np.array([0, 1, 127, 128, 255, 256, 511, 700, 1023])
    ys, os_, yr = _slack(p, rows)
    compare(p, Y, out, rows=rows, tcgen05=False, y_slack=ys, out_slack=os_, y_rel_slack=yr)
    p2 = gi.make_problem("t", 1, 1024, 2048, 1024, gi.DTYPE_F32, gi.ACT_NONE, gi.SCALE_SCALAR, gi.RED_SOFTMAX, scale=40.0, seed=9)
    Y, out, plan = run_gpu(p2)
    assert plan["path"] == fgr.FGR_PATH_UMMA_TF32X3
    ys, os_, yr = _slack(p2, rows)
    compare(p2, Y, out, rows=rows, tcgen05=False, y_slack=ys, out_slack=os_, y_rel_slack=yr)
