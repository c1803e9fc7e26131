"""Host-side checks that need no GPU: the library loads, exports what include/fgr.h declares,
validates descriptors, and selects paths / tiles / workspace sizes as documented."""
import ctypes
import os
import re

import pytest

import paper_2511_06345_b200 as fgr
from paper_2511_06345_b200 import build as fgr_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    fgr_build.build()


def _declared():
    names = []
    for f in os.listdir(os.path.join(ROOT, "include")):
        if f.endswith(".h"):
            names += re.findall(r"FGR_API\s+[\w\s\*]+?\b(fgr_\w+)\s*\(", open(os.path.join(ROOT, "include", f)).read())
    return names


def test_library_exports_every_declared_symbol():
    names = _declared()
    assert len(names) >= 12 and set(names) == set(fgr.EXPORTS)
    L = ctypes.CDLL(fgr.binding.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n


def test_struct_layout_matches_header():
    assert ctypes.sizeof(fgr.fgr_desc) == 136      # the value sizeof(fgr_desc) has in C (gcc, x86-64)
    assert ctypes.sizeof(fgr.fgr_plan_info) == 72
    assert fgr.fgr_status_string(0) == "ok" and "wait" in fgr.fgr_status_string(fgr.FGR_ERR_DEVICE_TIMEOUT)
    assert fgr.fgr_path_name(fgr.FGR_PATH_UMMA_STREAM_W) == "umma_stream_w"


def _plan(*a, **k):
    return fgr.fgr_plan(fgr.make_desc(*a, **k), 148)


def test_path_selection_for_the_five_workloads():
    c1 = _plan(1, 256, 256, 256, fgr.FGR_F32, fgr.FGR_ACT_GELU_TANH, 0, fgr.FGR_RED_LSE)
    assert c1.path == fgr.FGR_PATH_SIMT and c1.parts_per_row == 4 and c1.num_tiles == 16
    c2 = _plan(1, 4096, 4096, 4096, fgr.FGR_BF16, fgr.FGR_ACT_RELU, 2, fgr.FGR_RED_MAXSUM, write_y=1)
    assert c2.path == fgr.FGR_PATH_UMMA_TILED and (c2.tile_m, c2.tile_n) == (256, 256) and c2.cta_pair == 2
    assert c2.num_tiles == 256 and c2.grid == 148 and c2.parts_per_row == 32 and c2.stages == 3 and c2.ksub == 2
    assert c2.workspace_bytes == 256 + 4096 * 32 * 8 and c2.flop == 2.0 * 4096 ** 3
    assert c2.min_bytes == 3 * 4096 * 4096 * 2 + 2 * 4096 * 4 + 4096 * 2 * 4
    c3 = _plan(1, 8192, 8192, 2048, fgr.FGR_BF16, 0, 1, fgr.FGR_RED_SOFTMAX, scale=2048 ** -0.5)
    assert c3.path == fgr.FGR_PATH_UMMA_TILED and c3.parts_per_row == 64
    c4 = _plan(1, 128, 16384, 8192, fgr.FGR_BF16, 2, 0, fgr.FGR_RED_LSE)
    assert c4.path == fgr.FGR_PATH_UMMA_STREAM_W and c4.cta_pair == 1
    assert 120 <= c4.num_tiles <= 148 and c4.grid == c4.num_tiles   # one wave over (nearly) the whole machine
    assert c4.stages >= 3 and c4.ksub == 2 and c4.smem_bytes <= 232448
    c5 = _plan(32, 1024, 1024, 512, fgr.FGR_BF16, 1, 0, fgr.FGR_RED_MAXSUM)
    assert c5.path == fgr.FGR_PATH_UMMA_TILED and c5.num_tiles == 512 and c5.cta_pair == 2
    g = _plan(1, 2, 16384, 8192, fgr.FGR_BF16, 2, 0, fgr.FGR_RED_LSE)          # a few GEMVs: the CUDA-core streaming path
    assert g.path == fgr.FGR_PATH_SIMT_GEMV and g.grid == g.parts_per_row <= 148 and g.tile_n * g.grid >= 16384
    assert _plan(1, 2, 16384, 8192, fgr.FGR_BF16, 0, 0, fgr.FGR_RED_SOFTMAX).path == fgr.FGR_PATH_UMMA_STREAM_W
    assert _plan(1, 8, 16384, 8192, fgr.FGR_BF16, 2, 0, fgr.FGR_RED_LSE).path == fgr.FGR_PATH_UMMA_STREAM_W
    small_sm = fgr.fgr_plan(fgr.make_desc(1, 128, 16384, 8192, fgr.FGR_BF16, 2, 0, 0), 64)
    assert small_sm.grid <= 64


def test_forced_tiles_and_paths():
    p = _plan(1, 300, 520, 200, fgr.FGR_BF16, 0, 0, 0, force_path=fgr.FGR_PATH_UMMA_TILED, force_tile_n=112)
    assert p.tile_n == 112 and p.parts_per_row == 2 * 5 and p.num_tiles == 3 * 5
    p = _plan(1, 300, 520, 200, fgr.FGR_BF16, 0, 0, 0, force_path=fgr.FGR_PATH_UMMA_TILED, force_cta_pair=1)
    # 9 tiles of 256 columns would leave most SMs idle: the tiles are narrowed until one wave fills more of them
    assert p.cta_pair == 1 and p.tile_m == 128 and p.tile_n == 32 and p.num_tiles == 3 * 17
    p = _plan(1, 300, 520, 200, fgr.FGR_BF16, 0, 0, 0, force_path=fgr.FGR_PATH_UMMA_TILED, force_cta_pair=1, force_tile_n=256)
    assert p.num_tiles == 3 * 3 and p.stages == 4
    mid = _plan(1, 256, 8192, 4096, fgr.FGR_BF16, 0, 0, 0)
    assert mid.path == fgr.FGR_PATH_UMMA_TILED and (mid.tile_n, mid.cta_pair, mid.num_tiles) == (128, 2, 64)
    p = _plan(1, 300, 520, 200, fgr.FGR_BF16, 0, 0, 0, force_path=fgr.FGR_PATH_UMMA_TILED, force_cta_pair=2, force_tile_n=64)
    assert p.cta_pair == 2 and p.tile_m == 256 and p.num_tiles == 2 * 9 and p.grid == 36
    with pytest.raises(fgr.FgrError):
        _plan(1, 300, 520, 200, fgr.FGR_BF16, 0, 0, 0, force_cta_pair=2, force_tile_n=112)   # halves must be whole 16-row groups
    assert _plan(1, 100, 520, 200, fgr.FGR_BF16, 0, 0, 0, force_path=fgr.FGR_PATH_UMMA_TILED).cta_pair == 1   # one row block
    p = _plan(1, 300, 520, 200, fgr.FGR_BF16, 0, 0, 0, force_path=fgr.FGR_PATH_SIMT)
    assert p.path == fgr.FGR_PATH_SIMT and p.tile_n == 64 and p.parts_per_row == 9
    with pytest.raises(fgr.FgrError) as e:
        _plan(1, 64, 64, 64, fgr.FGR_F32, 0, 0, 0, force_path=fgr.FGR_PATH_UMMA_TILED)
    assert e.value.status == fgr.FGR_ERR_UNSUPPORTED


@pytest.mark.parametrize("kw,status", [
    (dict(N=12), fgr.FGR_ERR_UNSUPPORTED),            # bf16 needs N % 8 == 0
    (dict(K=20), fgr.FGR_ERR_UNSUPPORTED),
    (dict(M=0), fgr.FGR_ERR_INVALID_ARG),
    (dict(act=6), fgr.FGR_ERR_INVALID_ARG),
    (dict(reduce=4), fgr.FGR_ERR_INVALID_ARG),
    (dict(dtype=2), fgr.FGR_ERR_INVALID_ARG),
    (dict(ldx=8), fgr.FGR_ERR_INVALID_ARG),           # smaller than K
    (dict(ldy=68), fgr.FGR_ERR_UNSUPPORTED),          # not 16-byte aligned rows
    (dict(force_tile_n=24), fgr.FGR_ERR_INVALID_ARG),
    (dict(force_cta_pair=3), fgr.FGR_ERR_INVALID_ARG),
    (dict(force_ksub=5), fgr.FGR_ERR_INVALID_ARG),
    (dict(scale_kind=1, scale=float("inf")), fgr.FGR_ERR_INVALID_ARG),
    (dict(batch=2, bsx=16), fgr.FGR_ERR_INVALID_ARG),  # batches would overlap
])
def test_bad_descriptors(kw, status):
    base = dict(batch=1, M=32, N=64, K=16, dtype=fgr.FGR_BF16, act=0, scale_kind=0, reduce=0)
    base.update(kw)
    with pytest.raises(fgr.FgrError) as e:
        fgr.fgr_plan(fgr.make_desc(**base))
    assert e.value.status == status


def test_wrong_struct_size_and_nulls():
    d = fgr.make_desc(1, 32, 64, 16, fgr.FGR_BF16, 0, 0, 0)
    d.struct_bytes = 8
    with pytest.raises(fgr.FgrError):
        fgr.fgr_plan(d)
    L = fgr.lib()
    assert L.fgr_plan(None, 0, None) == fgr.FGR_ERR_INVALID_ARG
    assert L.fgr_destroy(None) == fgr.FGR_OK
    assert L.fgr_workspace_bytes(None) == 0
    assert L.fgr_get_status(None) == fgr.FGR_ERR_INVALID_ARG
    assert L.fgr_run(None, None, None, None, None, None, None, None, 0, None) == fgr.FGR_ERR_INVALID_ARG


def test_create_without_a_device_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(fgr.FgrError) as e:
        fgr.fgr_create(fgr.make_desc(1, 32, 64, 16, fgr.FGR_BF16, 0, 0, 0))
    assert e.value.status == fgr.FGR_ERR_CUDA
    with pytest.raises(RuntimeError):
        fgr.FusedGemmReduce(1, 32, 64, 16, fgr.FGR_BF16, 0, 0, 0)
