"""(mean, population variance) over N: plan rules on CPU; GPU parity of the fused operator on every
path and of the stand-alone row reduction against the oracle, through the C ABI."""
import numpy as np
import pytest

import fgr_inputs as gi
import paper_2511_06345_b200 as fgr


def test_plan_rules_for_meanvar():
    mk = lambda M, **kw: fgr.fgr_plan(fgr.make_desc(1, M, 2048, 512, fgr.FGR_BF16, 0, 0, fgr.FGR_RED_MEANVAR, **kw))
    assert mk(2).path == fgr.FGR_PATH_SIMT_GEMV and mk(8).path == fgr.FGR_PATH_UMMA_STREAM_W
    assert mk(512).path == fgr.FGR_PATH_UMMA_TILED
    with pytest.raises(fgr.FgrError):
        fgr.fgr_plan(fgr.make_desc(1, 8, 64, 64, fgr.FGR_BF16, 0, 0, 5))     # 4 and 5 belong to fgr_reduce_rows only


def _problem(dtype, B, M, N, K, act, sk, seed, write_y=1, bias_range=(-0.5, 0.5)):
    return gi.make_problem("t", B, M, N, K, dtype, act, sk, gi.RED_MEANVAR, scale=0.7, write_y=write_y, x_std=1.0,
                           w_std=2.0 / np.sqrt(K), bias_range=bias_range, scale_range=(-1.5, 1.5), seed=seed)


CASES = [
    # dtype, B, M, N, K, force_path, tile_n, pair
    (gi.DTYPE_F32, 2, 70, 132, 36, fgr.FGR_PATH_SIMT, 0, 0),
    (gi.DTYPE_BF16, 1, 70, 136, 72, fgr.FGR_PATH_SIMT, 0, 0),
    (gi.DTYPE_BF16, 1, 300, 520, 200, fgr.FGR_PATH_UMMA_TILED, 0, 0),
    (gi.DTYPE_BF16, 2, 257, 1000, 136, fgr.FGR_PATH_UMMA_TILED, 240, 1),
    (gi.DTYPE_BF16, 1, 129, 120, 512, fgr.FGR_PATH_UMMA_TILED, 64, 2),
    (gi.DTYPE_BF16, 1, 128, 2048, 320, fgr.FGR_PATH_UMMA_STREAM_W, 0, 0),
    (gi.DTYPE_BF16, 1, 3, 2056, 128, fgr.FGR_PATH_AUTO, 0, 0),             # the skinny CUDA-core path
    (gi.DTYPE_BF16, 2, 11, 520, 72, fgr.FGR_PATH_SIMT_GEMV, 0, 0),
    (gi.DTYPE_BF16, 1, 1, 8, 8, fgr.FGR_PATH_SIMT_GEMV, 0, 0),
    (gi.DTYPE_F32, 1, 300, 524, 200, fgr.FGR_PATH_UMMA_TF32X3, 0, 0),
    (gi.DTYPE_F32, 2, 129, 260, 36, fgr.FGR_PATH_UMMA_TF32X3, 64, 1),
]


@pytest.mark.gpu
@pytest.mark.parametrize("case", CASES)
def test_meanvar_matches_oracle(cuda_device, case):
    from parity import compare, run_gpu
    dtype, B, M, N, K, path, tn, pair = case
    for i, act in enumerate([gi.ACT_NONE, gi.ACT_RELU, gi.ACT_GELU_TANH]):
        for wy in (0, 1):
            p = _problem(dtype, B, M, N, K, act, i % 3, seed=90 + i, write_y=wy)
            Y, out, plan = run_gpu(p, force_path=path, force_tile_n=tn, force_cta_pair=pair)
            assert path == fgr.FGR_PATH_AUTO or plan["path"] == path
            kw = {}
            if plan["path"] == fgr.FGR_PATH_UMMA_TF32X3:
                from test_tf32x3 import _slack
                ys, _, _ = _slack(p)
                # mean: the mean error of y; variance: 2 sigma times it (sigma <= 3 here)
                kw = dict(y_slack=ys, out_slack=np.stack([ys.mean(1), 6.0 * ys.max(1)], 1))
            compare(p, Y, out, tcgen05=dtype == gi.DTYPE_BF16 and plan["path"] != fgr.FGR_PATH_SIMT, **kw)
            assert (out[:, 1] >= 0).all()


@pytest.mark.gpu
def test_meanvar_large_offset(cuda_device):
    """Every y near 300 with unit-scale spread: E[y^2] - E[y]^2 in fp32 would lose the variance
    (9e4 * 2^-24 = 5e-3 per term); the two-pass / pairwise form keeps it."""
    from parity import run_gpu
    import oracle
    for dtype, path in [(gi.DTYPE_F32, fgr.FGR_PATH_SIMT), (gi.DTYPE_BF16, fgr.FGR_PATH_UMMA_TILED), (gi.DTYPE_F32, fgr.FGR_PATH_UMMA_TF32X3)]:
        p = _problem(dtype, 1, 200, 520, 64, gi.ACT_NONE, gi.SCALE_NONE, seed=4, write_y=0, bias_range=(299.5, 300.5))
        _, out, _ = run_gpu(p, force_path=path)
        _, ref, _ = oracle.run_problem(p, want_y=False)
        assert np.abs(out[:, 0] - ref[:, 0]).max() <= 1e-4 * 300
        assert (np.abs(out[:, 1] - ref[:, 1]) <= 2e-3 * ref[:, 1]).all()


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [gi.DTYPE_F32, gi.DTYPE_BF16])
@pytest.mark.parametrize("shape", [(1, 8), (5, 24), (300, 1000), (64, 2048), (9, 8200), (3, 40000),
                                   # from here on: clusters of 1 to 16 CTAs of 1024 threads per row
                                   (1, 1048576), (16, 262144), (5, 100008), (2, 33000), (20, 400000), (7, 600008),
                                   (100, 131072), (200, 70000)])
def test_reduce_rows_meanvar(cuda_device, dtype, shape):
    import torch
    import oracle
    M, N = shape
    a = gi.normal(7, 9, M * N, 2.0).reshape(M, N) + 50.0
    if dtype == gi.DTYPE_BF16:
        bits = gi.f32_to_bf16_bits(a)
        A = torch.from_numpy(bits).view(torch.int16).view(torch.bfloat16).cuda()
        ref = oracle.reduce_rows(bits, dtype=oracle.BF16, kind=oracle.RED_MEANVAR)[1]
    else:
        A = torch.from_numpy(a).cuda()
        ref = oracle.reduce_rows(a, dtype=oracle.F32, kind=oracle.RED_MEANVAR)[1]
    out = torch.full((M, 2), -1.0, device="cuda")
    for _ in range(2):
        fgr.fgr_reduce_rows(M, N, dtype, fgr.FGR_RED_MEANVAR, A, None, out)
    got = out.cpu().numpy().astype(np.float64)
    assert np.abs(got[:, 0] - ref[:, 0]).max() <= 1e-5 * 52
    assert (np.abs(got[:, 1] - ref[:, 1]) <= 1e-4 * ref[:, 1] + 1e-6).all()
