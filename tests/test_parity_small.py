"""GPU parity, small shapes: every element of Y / P and of the reduction against the CPU oracle,
through the C ABI.  Shapes span several tiles and ragged tails in M, N and K."""
import numpy as np
import pytest
import torch

import fgr_inputs as gi
import paper_2511_06345_b200 as fgr
from parity import compare, run_gpu, to_device

pytestmark = pytest.mark.gpu

ACTS = [gi.ACT_NONE, gi.ACT_RELU, gi.ACT_GELU_TANH, gi.ACT_SIGMOID, gi.ACT_TANH, gi.ACT_SILU]
REDS = [gi.RED_LSE, gi.RED_SOFTMAX, gi.RED_MAXSUM, gi.RED_MAX_SUMEXP]


def _problem(dtype, B, M, N, K, act, sk, red, seed, write_y=1, std=1.0, bias_per_batch=0, scale=0.7):
    return gi.make_problem("t", B, M, N, K, dtype, act, sk, red, scale=scale, write_y=write_y, x_std=std,
                           w_std=std / np.sqrt(K) * 2.0, bias_range=(-0.5, 0.5), scale_range=(-1.5, 1.5),
                           bias_per_batch=bias_per_batch, seed=seed)


SIMT_SHAPES = [(1, 1, 4, 4), (1, 7, 12, 20), (1, 64, 64, 16), (1, 65, 68, 36), (1, 130, 200, 100), (3, 33, 72, 40)]


@pytest.mark.parametrize("shape", SIMT_SHAPES)
@pytest.mark.parametrize("red", REDS)
def test_simt_fp32(cuda_device, shape, red):
    B, M, N, K = shape
    for i, act in enumerate(ACTS):
        p = _problem(gi.DTYPE_F32, B, M, N, K, act, i % 3, red, seed=10 + i, bias_per_batch=i % 2)
        Y, out, plan = run_gpu(p)
        assert plan["path"] == fgr.FGR_PATH_SIMT
        compare(p, Y, out, tcgen05=False)


def test_simt_c1_config(cuda_device):
    p = gi.make_config("c1")
    Y, out, plan = run_gpu(p)
    assert plan["path"] == fgr.FGR_PATH_SIMT and Y is None
    w = compare(p, Y, out, tcgen05=False)
    assert w["out"] < 1e-6
    p = gi.make_config("c1", write_y=1)
    Y, out, _ = run_gpu(p)
    compare(p, Y, out, tcgen05=False)


@pytest.mark.parametrize("red", REDS)
def test_simt_bf16_forced(cuda_device, red):
    p = _problem(gi.DTYPE_BF16, 2, 70, 136, 72, gi.ACT_GELU_TANH, gi.SCALE_PER_COLUMN, red, seed=21)
    Y, out, plan = run_gpu(p, force_path=fgr.FGR_PATH_SIMT)
    assert plan["path"] == fgr.FGR_PATH_SIMT
    compare(p, Y, out, tcgen05=False)


UMMA_SHAPES = [
    # B, M, N, K, force_tile_n
    (1, 128, 256, 64, 0),
    (1, 1, 8, 8, 0),
    (1, 100, 264, 72, 0),      # N tail of 8 columns, K tail of 8
    (1, 300, 520, 200, 0),     # 3 row blocks, 3 column tiles, ragged everywhere
    (1, 257, 1000, 136, 240),
    (1, 129, 120, 512, 64),
    (3, 130, 264, 72, 0),      # batched, ragged
    (2, 256, 512, 1024, 128),
    (1, 140, 2048, 320, 112),  # the weight-streaming tile shape
    (1, 512, 2048, 256, 0),    # more tiles than SMs: persistent loop, both accumulator buffers, ring wrap-around
]


@pytest.mark.parametrize("shape", UMMA_SHAPES)
@pytest.mark.parametrize("red", REDS)
def test_umma_tiled(cuda_device, shape, red):
    B, M, N, K, tn = shape
    for i, act in enumerate(ACTS):
        p = _problem(gi.DTYPE_BF16, B, M, N, K, act, (i + red) % 3, red, seed=30 + i, bias_per_batch=i % 2)
        Y, out, plan = run_gpu(p, force_path=fgr.FGR_PATH_UMMA_TILED, force_tile_n=tn, force_cta_pair=1)
        assert plan["path"] == fgr.FGR_PATH_UMMA_TILED and plan["cta_pair"] == 1
        compare(p, Y, out)


PAIR_SHAPES = [
    # B, M, N, K, force_tile_n: clusters of two CTAs on 256-row tiles (tcgen05 cta_group::2)
    (1, 256, 256, 64, 0),
    (1, 129, 264, 72, 0),      # the second CTA of the pair owns a single real row
    (1, 300, 520, 200, 64),
    (2, 515, 1000, 136, 96),
    (1, 1024, 4096, 320, 0),   # more tiles than clusters: persistent loop, both accumulator buffers, ring wrap-around
]


@pytest.mark.parametrize("shape", PAIR_SHAPES)
@pytest.mark.parametrize("red", REDS)
def test_umma_cta_pairs(cuda_device, shape, red):
    B, M, N, K, tn = shape
    for i, act in enumerate(ACTS):
        p = _problem(gi.DTYPE_BF16, B, M, N, K, act, (i + red + 1) % 3, red, seed=50 + i, bias_per_batch=(i + 1) % 2)
        Y, out, plan = run_gpu(p, force_path=fgr.FGR_PATH_UMMA_TILED, force_tile_n=tn, force_cta_pair=2)
        assert plan["cta_pair"] == 2 and plan["tile_m"] == 256 and plan["grid"] % 2 == 0
        compare(p, Y, out)


def test_cta_pair_and_single_agree_bitwise(cuda_device):
    """Same tile width, same accumulation order per element: a pair must reproduce single CTAs exactly."""
    p = _problem(gi.DTYPE_BF16, 1, 700, 1544, 264, gi.ACT_GELU_TANH, gi.SCALE_PER_COLUMN, gi.RED_LSE, seed=55)
    t = to_device(p)
    Y1, o1, p1 = run_gpu(p, tensors=t, force_path=fgr.FGR_PATH_UMMA_TILED, force_cta_pair=1)
    Y2, o2, p2 = run_gpu(p, tensors=t, force_path=fgr.FGR_PATH_UMMA_TILED, force_cta_pair=2)
    assert p1["cta_pair"] == 1 and p2["cta_pair"] == 2
    assert np.array_equal(Y1, Y2) and np.array_equal(o1, o2)


GEMV_SHAPES = [(1, 1, 8, 8), (1, 3, 1000, 264), (1, 8, 2056, 1096), (1, 16, 520, 8200), (3, 5, 264, 72), (1, 2, 4096, 640)]


@pytest.mark.parametrize("shape", GEMV_SHAPES)
@pytest.mark.parametrize("red", [gi.RED_LSE, gi.RED_MAXSUM, gi.RED_MAX_SUMEXP])
def test_skinny_gemv_path(cuda_device, shape, red):
    B, M, N, K = shape
    for i, act in enumerate(ACTS):
        p = _problem(gi.DTYPE_BF16, B, M, N, K, act, (i + red) % 3, red, seed=60 + i, bias_per_batch=i % 2, write_y=i % 2)
        Y, out, plan = run_gpu(p, force_path=fgr.FGR_PATH_SIMT_GEMV)
        assert plan["path"] == fgr.FGR_PATH_SIMT_GEMV and plan["parts_per_row"] == plan["grid"] // B
        compare(p, Y, out, tcgen05=False)


def test_skinny_selection(cuda_device):
    """M <= 4 goes to the GEMV path by itself; softmax and larger M stay on the tensor-core paths."""
    assert fgr.fgr_plan(fgr.make_desc(1, 8, 2048, 512, fgr.FGR_BF16, 0, 0, 0)).path == fgr.FGR_PATH_UMMA_STREAM_W
    p = _problem(gi.DTYPE_BF16, 1, 4, 2048, 512, gi.ACT_GELU_TANH, gi.SCALE_NONE, gi.RED_LSE, seed=63)
    Y, out, plan = run_gpu(p)
    assert plan["path"] == fgr.FGR_PATH_SIMT_GEMV
    compare(p, Y, out, tcgen05=False)
    ref = out
    Y, out, plan = run_gpu(p, force_path=fgr.FGR_PATH_UMMA_STREAM_W)      # the same problem on tensor cores
    compare(p, Y, out)
    np.testing.assert_allclose(out, ref, rtol=0, atol=2e-4 * (1 + np.abs(ref).max()))
    p.reduce = gi.RED_SOFTMAX
    Y, out, plan = run_gpu(p)
    assert plan["path"] in (fgr.FGR_PATH_UMMA_STREAM_W, fgr.FGR_PATH_UMMA_TILED)
    compare(p, Y, out)
    with pytest.raises(fgr.FgrError) as e:
        fgr.fgr_plan(fgr.make_desc(1, 4, 2048, 512, fgr.FGR_BF16, 0, 0, fgr.FGR_RED_SOFTMAX, force_path=fgr.FGR_PATH_SIMT_GEMV))
    assert e.value.status == fgr.FGR_ERR_UNSUPPORTED
    with pytest.raises(fgr.FgrError):
        fgr.fgr_plan(fgr.make_desc(1, 17, 2048, 512, fgr.FGR_BF16, 0, 0, 0, force_path=fgr.FGR_PATH_SIMT_GEMV))


def test_k_sub_blocks_per_stage_agree_bitwise(cuda_device):
    """1, 2 or 4 K sub-blocks per ring stage change how operands are fetched, not what is summed."""
    for B, M, N, K, tn, pair, path in [(1, 128, 2048, 1096, 112, 1, fgr.FGR_PATH_UMMA_STREAM_W),
                                       (2, 300, 520, 200, 64, 2, fgr.FGR_PATH_UMMA_TILED),
                                       (1, 257, 520, 72, 0, 0, fgr.FGR_PATH_UMMA_TILED)]:
        p = _problem(gi.DTYPE_BF16, B, M, N, K, gi.ACT_GELU_TANH, gi.SCALE_PER_COLUMN, gi.RED_LSE, seed=57)
        t = to_device(p)
        ref = None
        for ks in (1, 2, 4):
            Y, out, plan = run_gpu(p, tensors=t, force_path=path, force_tile_n=tn, force_cta_pair=pair, force_ksub=ks)
            if ref is None:
                compare(p, Y, out)
                ref = (Y, out)
            assert np.array_equal(Y, ref[0]) and np.array_equal(out, ref[1]), (B, M, N, K, ks, plan)


@pytest.mark.parametrize("red", [gi.RED_LSE, gi.RED_MAXSUM])
def test_umma_no_y(cuda_device, red):
    p = _problem(gi.DTYPE_BF16, 1, 200, 776, 128, gi.ACT_RELU, gi.SCALE_NONE, red, seed=40, write_y=0)
    Y, out, _ = run_gpu(p)
    assert Y is None
    compare(p, Y, out)


def test_stream_w_selected_for_skinny(cuda_device):
    p = gi.make_problem("skinny", 1, 128, 4096, 1024, gi.DTYPE_BF16, gi.ACT_GELU_TANH, gi.SCALE_NONE, gi.RED_LSE,
                        x_std=1.0, seed=41)
    Y, out, plan = run_gpu(p)
    assert plan["path"] == fgr.FGR_PATH_UMMA_STREAM_W and plan["tile_n"] < 256
    compare(p, Y, out)
    p.write_y = 1
    Y, out, _ = run_gpu(p)
    compare(p, Y, out)


def test_paths_and_tile_widths_agree(cuda_device):
    """The split-N merge must not depend on how N was split."""
    p = _problem(gi.DTYPE_BF16, 1, 150, 1032, 136, gi.ACT_NONE, gi.SCALE_SCALAR, gi.RED_LSE, seed=42, scale=3.0)
    ref = None
    for path, tn in [(fgr.FGR_PATH_SIMT, 0), (fgr.FGR_PATH_UMMA_TILED, 16), (fgr.FGR_PATH_UMMA_TILED, 96),
                     (fgr.FGR_PATH_UMMA_TILED, 256), (fgr.FGR_PATH_UMMA_STREAM_W, 0)]:
        Y, out, _ = run_gpu(p, force_path=path, force_tile_n=tn)
        compare(p, Y, out)
        if ref is None:
            ref = out
        np.testing.assert_allclose(out, ref, rtol=0, atol=2e-4 * (1 + np.abs(ref).max()))


def test_strided_operands(cuda_device):
    """ldx > K, ldw > K, ldy > N and padded batch strides; the padding must stay untouched."""
    B, M, N, K = 2, 130, 264, 72
    p = _problem(gi.DTYPE_BF16, B, M, N, K, gi.ACT_RELU, gi.SCALE_PER_COLUMN, gi.RED_MAXSUM, seed=43)
    X, W, b, s = to_device(p)
    ldx, ldw, ldy = K + 8, K + 16, N + 24
    Xp = torch.full((B, M + 3, ldx), 7.0, dtype=torch.bfloat16, device="cuda")
    Wp = torch.full((B, N + 5, ldw), -7.0, dtype=torch.bfloat16, device="cuda")
    Yp = torch.full((B, M + 2, ldy), 123.0, dtype=torch.bfloat16, device="cuda")
    Xp[:, :M, :K], Wp[:, :N, :K] = X, W
    desc = fgr.make_desc(B, M, N, K, p.dtype, p.act, p.scale_kind, p.reduce, write_y=1, ldx=ldx, ldw=ldw, ldy=ldy,
                         bsx=(M + 3) * ldx, bsw=(N + 5) * ldw, bsy=(M + 2) * ldy)
    for path in (fgr.FGR_PATH_UMMA_TILED, fgr.FGR_PATH_SIMT):
        desc.force_path = path
        h = fgr.fgr_create(desc)
        ws = torch.empty(fgr.fgr_workspace_bytes(h), dtype=torch.uint8, device="cuda")
        out = torch.empty((B * M, 2), dtype=torch.float32, device="cuda")
        Yp.fill_(123.0)
        fgr.fgr_run(h, Xp, Wp, b, s, Yp, out, ws, ws.numel(), torch.cuda.current_stream().cuda_stream)
        assert fgr.fgr_get_status(h) == fgr.FGR_OK
        fgr.fgr_destroy(h)
        Yh = Yp[:, :M, :N].float().cpu().numpy().astype(np.float64).reshape(B * M, N)
        compare(p, Yh, out.cpu().numpy().astype(np.float64), tcgen05=path != fgr.FGR_PATH_SIMT)
        assert (Yp[:, M:, :] == 123.0).all() and (Yp[:, :, N:] == 123.0).all()


def test_bitwise_deterministic(cuda_device):
    p = _problem(gi.DTYPE_BF16, 1, 300, 1544, 264, gi.ACT_GELU_TANH, gi.SCALE_PER_COLUMN, gi.RED_LSE, seed=44)
    t = to_device(p)
    runs = [run_gpu(p, tensors=t) for _ in range(3)]
    for Y, out, _ in runs[1:]:
        assert np.array_equal(Y, runs[0][0]) and np.array_equal(out, runs[0][1])
    p.reduce = gi.RED_SOFTMAX
    runs = [run_gpu(p, tensors=t) for _ in range(3)]
    for Y, out, _ in runs[1:]:
        assert np.array_equal(Y, runs[0][0])


def test_integer_inputs_exact(cuda_device):
    """Small integers: products and partial sums are exact in fp32, so the GPU must equal the oracle."""
    rng = np.random.default_rng(45)
    B, M, N, K = 1, 200, 520, 136
    for dtype, path in [(gi.DTYPE_BF16, fgr.FGR_PATH_UMMA_TILED), (gi.DTYPE_F32, fgr.FGR_PATH_SIMT)]:
        p = gi.make_problem("int", B, M, N, K, dtype, gi.ACT_NONE, gi.SCALE_NONE, gi.RED_MAXSUM, write_y=1,
                            bias_range=None, materialize=False)
        Xi, Wi = rng.integers(-8, 9, (B, M, K)).astype(np.float32), rng.integers(-8, 9, (B, N, K)).astype(np.float32)
        p.X = Xi if dtype == gi.DTYPE_F32 else gi.f32_to_bf16_bits(Xi).reshape(Xi.shape)
        p.W = Wi if dtype == gi.DTYPE_F32 else gi.f32_to_bf16_bits(Wi).reshape(Wi.shape)
        p.write_y = 0                       # z reaches ~ +-3000: not exact in bf16, so compare the fp32 reduction
        Y, out, _ = run_gpu(p, force_path=path)
        import oracle
        _, ref, _ = oracle.run_problem(p, want_y=False)
        np.testing.assert_array_equal(out, ref)


def test_identity_weights(cuda_device):
    """W = I: Y = relu(X + b) * s, exact up to the single rounding of Y."""
    n = 264
    p = gi.make_problem("eye", 1, 140, n, n, gi.DTYPE_BF16, gi.ACT_RELU, gi.SCALE_PER_COLUMN, gi.RED_MAXSUM,
                        write_y=1, x_std=1.0, seed=46)
    p.W = gi.f32_to_bf16_bits(np.eye(n, dtype=np.float32)).reshape(1, n, n)
    Y, out, _ = run_gpu(p)
    X = gi.bf16_bits_to_f32(p.X).reshape(140, n)
    ref = np.maximum(X + p.bias, 0).astype(np.float32) * p.scale_vec
    got = torch.from_numpy(ref).to(torch.bfloat16).float().numpy()
    np.testing.assert_array_equal(Y.astype(np.float32), got)
    compare(p, Y, out)


def test_shared_weights_plain_gemm(cuda_device):
    """w_shared = 1 without a convolution: one [N, K] weight matrix for a batch of inputs, on every path."""
    for dtype, path in [(gi.DTYPE_BF16, fgr.FGR_PATH_UMMA_TILED), (gi.DTYPE_BF16, fgr.FGR_PATH_UMMA_STREAM_W),
                        (gi.DTYPE_BF16, fgr.FGR_PATH_SIMT), (gi.DTYPE_F32, fgr.FGR_PATH_SIMT), (gi.DTYPE_F32, fgr.FGR_PATH_UMMA_TF32X3)]:
        p = gi.make_problem("t", 3, 130, 264, 72, dtype, gi.ACT_RELU, gi.SCALE_NONE, gi.RED_MAX_SUMEXP, write_y=1, x_std=1.0,
                            w_std=0.2, seed=31, w_shared=1)
        assert p.W.shape == (1, 264, 72)
        Y, out, plan = run_gpu(p, force_path=path)
        assert plan["path"] == path
        compare(p, Y, out, tcgen05=dtype == gi.DTYPE_BF16 and path != fgr.FGR_PATH_SIMT)
    p = gi.make_problem("t", 3, 4, 264, 72, gi.DTYPE_BF16, gi.ACT_RELU, gi.SCALE_NONE, gi.RED_LSE, write_y=1, w_std=0.2, seed=32, w_shared=1)
    Y, out, plan = run_gpu(p)
    assert plan["path"] == fgr.FGR_PATH_SIMT_GEMV
    compare(p, Y, out)


def test_run_inside_a_cuda_graph(cuda_device):
    """fgr_run only enqueues kernels (with programmatic dependent launch between them), so after one
    ordinary call (which clears the workspace's status word and encodes the tensor maps) it can be
    captured into a CUDA graph; replays give bit-identical results."""
    p = gi.make_problem("t", 2, 300, 520, 200, gi.DTYPE_BF16, gi.ACT_GELU_TANH, gi.SCALE_NONE, gi.RED_LSE, write_y=1, seed=77)
    X, W, b, s = to_device(p)
    op = fgr.FusedGemmReduce(p.batch, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, write_y=1, device=0)
    Y = torch.empty((p.batch, p.M, p.N), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((p.batch * p.M,), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        op(X, W, b, s, Y=Y, out=out)
        stream.synchronize()
        Y0, out0 = Y.clone(), out.clone()
        Y.zero_(); out.zero_()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(3):
                op(X, W, b, s, Y=Y, out=out)
        g.replay()
        stream.synchronize()
    assert op.status() == fgr.FGR_OK
    assert torch.equal(Y, Y0) and torch.equal(out, out0)
    compare(p, Y.float().cpu().numpy().astype(np.float64).reshape(p.batch * p.M, p.N), out.cpu().numpy().astype(np.float64).reshape(-1, 1))
    op.close()
