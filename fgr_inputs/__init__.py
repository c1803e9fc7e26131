"""Seeded synthetic inputs for the fused GEMM + epilogue + row-reduce operator.

This module only draws numbers and rounds them to the storage type.  It holds
none of the operator's arithmetic (no GEMM, activation, scaling or reduction)
and is the one module that both the CPU oracle's tests and the CUDA path's
tests/bench may import.

Generator (counter based, independent of numpy's/torch's RNG versions and of
thread count): for element ``i`` of tensor ``tensor_id`` under ``seed``

    base = mix64(seed * GOLDEN + tensor_id)
    z1   = mix64(base + (2 i + 1) * GOLDEN),   z2 = mix64(base + (2 i + 2) * GOLDEN)
    u1   = ((z1 >> 11) + 1) * 2^-53   in (0, 1]
    u2   =  (z2 >> 11)      * 2^-53   in [0, 1)
    normal  = sqrt(-2 ln u1) * cos(2 pi u2)        (Box-Muller, fp64)
    uniform = lo + (hi - lo) * u2

``mix64`` is the splitmix64 finaliser.  Values are then scaled and rounded
(round-to-nearest-even) to fp32 or bf16.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from concurrent.futures import ThreadPoolExecutor
import math
import os

import numpy as np

GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 20

TENSOR_X, TENSOR_W, TENSOR_BIAS, TENSOR_SCALE, TENSOR_RESIDUAL = 1, 2, 3, 4, 5

# enum values of the operator descriptor (documented in include/fgr.h)
DTYPE_F32, DTYPE_BF16 = 0, 1
ACT_NONE, ACT_RELU, ACT_GELU_TANH, ACT_SIGMOID, ACT_TANH, ACT_SILU = 0, 1, 2, 3, 4, 5
SCALE_NONE, SCALE_SCALAR, SCALE_PER_COLUMN = 0, 1, 2
RED_LSE, RED_SOFTMAX, RED_MAXSUM, RED_MAX_SUMEXP = 0, 1, 2, 3
RED_MEANVAR = 6


def _mix64(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _base(seed: int, tensor_id: int) -> np.uint64:
    with np.errstate(over="ignore"):
        return _mix64(np.asarray(np.uint64(seed) * GOLDEN + np.uint64(tensor_id)))[()]


def _uniform_pair(seed: int, tensor_id: int, start: int, count: int):
    with np.errstate(over="ignore"):
        i = np.arange(start, start + count, dtype=np.uint64)
        base = _base(seed, tensor_id)
        z1 = _mix64(base + (np.uint64(2) * i + np.uint64(1)) * GOLDEN)
        z2 = _mix64(base + (np.uint64(2) * i + np.uint64(2)) * GOLDEN)
    u1 = ((z1 >> np.uint64(11)).astype(np.float64) + 1.0) * (2.0 ** -53)
    u2 = (z2 >> np.uint64(11)).astype(np.float64) * (2.0 ** -53)
    return u1, u2


def _fill(out: np.ndarray, fn) -> np.ndarray:
    """Fills ``out`` chunk by chunk (chunks are independent: element i depends on i only)."""
    starts = range(0, out.size, _CHUNK)
    workers = min(len(starts), os.cpu_count() or 1, 16)
    if workers <= 1:
        for s in starts:
            fn(s, min(_CHUNK, out.size - s))
    else:
        with ThreadPoolExecutor(workers) as ex:
            list(ex.map(lambda s: fn(s, min(_CHUNK, out.size - s)), starts))
    return out


def normal(seed: int, tensor_id: int, count: int, std: float = 1.0) -> np.ndarray:
    """``count`` draws of N(0, std^2) as fp32 (drawn in fp64, rounded once)."""
    out = np.empty(count, dtype=np.float32)

    def fn(s, c):
        u1, u2 = _uniform_pair(seed, tensor_id, s, c)
        out[s:s + c] = (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2) * std).astype(np.float32)
    return _fill(out, fn)


def uniform(seed: int, tensor_id: int, count: int, lo: float, hi: float) -> np.ndarray:
    """``count`` draws of U(lo, hi) as fp32."""
    out = np.empty(count, dtype=np.float32)

    def fn(s, c):
        _, u2 = _uniform_pair(seed, tensor_id, s, c)
        out[s:s + c] = (lo + (hi - lo) * u2).astype(np.float32)
    return _fill(out, fn)


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round finite fp32 values to bf16 (nearest even); returns the uint16 bit patterns."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Problem:
    """One operator instance: shapes, kinds and the host copies of its inputs.

    ``X`` and ``W`` are fp32 arrays for ``dtype == DTYPE_F32`` and uint16 bf16 bit
    patterns for ``DTYPE_BF16``; ``bias`` and ``scale_vec`` are fp32 (or ``None``).
    Shapes: X [batch, M, K], W [batch, N, K] (K contiguous), bias [N] (or [batch, N]),
    scale_vec [N].
    """
    name: str
    batch: int
    M: int
    N: int
    K: int
    dtype: int
    act: int
    scale_kind: int
    reduce: int
    scale: float = 1.0
    write_y: int = 0
    bias_per_batch: int = 0
    w_shared: int = 0      # 1: W is [1, N, K], one matrix for every batch element
    conv_taps: int = 0     # R > 1: 1-D convolution; X is then [batch, (M - 1) * stride + R, K / R] (channels last)
    conv_stride: int = 1
    conv_rows: int = 0     # R > 1: 2-D convolution; X is then the image [batch, H, conv_width, K / (R * S)], S = max(conv_taps, 1),
    conv_width: int = 0    # and M = (P - 1) * conv_width + Q output rows at the image's row pitch (P = H - R + 1, Q = conv_width - S + 1)
    X: np.ndarray | None = None
    W: np.ndarray | None = None
    bias: np.ndarray | None = None
    scale_vec: np.ndarray | None = None
    residual: np.ndarray | None = None    # [batch, M, N] in the dtype of X, added after activation and scale
    recipe: dict = field(default_factory=dict)

    @property
    def flop(self) -> float:
        return 2.0 * self.batch * self.M * self.N * self.K

    @property
    def out_width(self) -> int:
        return {RED_LSE: 1, RED_SOFTMAX: 0, RED_MAXSUM: 2, RED_MAX_SUMEXP: 2, RED_MEANVAR: 2}[self.reduce]

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == DTYPE_F32 else 2

    def min_bytes(self) -> int:
        """Algorithmic minimum traffic: every operand read once, every output written once."""
        e = self.elem_bytes
        taps = max(self.conv_taps, 1)
        x_elems = (self.M - 1) * min(self.conv_stride * (self.K // taps), self.K) + self.K if taps > 1 else self.M * self.K
        if self.conv_rows > 1:     # the pixels the M windows cover
            c = self.K // (self.conv_rows * taps)
            x_elems = (self.M - 1 + (self.conv_rows - 1) * self.conv_width) * c + taps * c
        b = (self.batch * x_elems + (1 if self.w_shared else self.batch) * self.N * self.K) * e
        if self.bias is not None:
            b += self.bias.size * 4
        if self.scale_vec is not None:
            b += self.scale_vec.size * 4
        if self.residual is not None:
            b += self.batch * self.M * self.N * e
        if self.reduce == RED_SOFTMAX or self.write_y:
            b += self.batch * self.M * self.N * e
        b += self.batch * self.M * self.out_width * 4
        return b


def _store(a: np.ndarray, dtype: int) -> np.ndarray:
    return a if dtype == DTYPE_F32 else f32_to_bf16_bits(a)


def make_problem(name, batch, M, N, K, dtype, act, scale_kind, reduce, *, scale=1.0, write_y=0,
                 x_std=None, w_std=None, bias_range=(-0.1, 0.1), scale_range=(0.5, 1.5),
                 bias_per_batch=0, seed=0, materialize=True, conv_taps=0, w_shared=0, residual_std=None, conv_stride=1,
                 conv_rows=0, conv_width=0) -> Problem:
    """Draws a problem with the value distributions of the named workloads.

    x_std / w_std default to 1/sqrt(K); bias ~ U(bias_range) (None -> no bias);
    per-column scale ~ U(scale_range).
    """
    x_std = 1.0 / math.sqrt(K) if x_std is None else x_std
    w_std = 1.0 / math.sqrt(K) if w_std is None else w_std
    p = Problem(name, batch, M, N, K, dtype, act, scale_kind, reduce, scale=float(scale),
                write_y=write_y, bias_per_batch=bias_per_batch, conv_taps=conv_taps, w_shared=w_shared, conv_stride=conv_stride,
                conv_rows=conv_rows, conv_width=conv_width,
                recipe=dict(seed=seed, x_std=x_std, w_std=w_std, bias_range=bias_range,
                            scale_range=scale_range if scale_kind == SCALE_PER_COLUMN else None))
    if not materialize:
        if bias_range is not None:
            p.bias = np.empty((batch if bias_per_batch else 1) * N, dtype=np.float32)
        if scale_kind == SCALE_PER_COLUMN:
            p.scale_vec = np.empty(N, dtype=np.float32)
        return p
    if conv_rows > 1:      # the image itself: M = (P - 1) * conv_width + Q output rows need H = P + conv_rows - 1 image rows
        S = max(conv_taps, 1)
        Q = conv_width - S + 1
        if (M - Q) % conv_width != 0 or M < Q:
            raise ValueError("M must be (P - 1) * conv_width + Q for a whole number P of output rows")
        H, C = (M - Q) // conv_width + conv_rows, K // (conv_rows * S)
        p.X = _store(normal(seed, TENSOR_X, batch * H * conv_width * C, x_std), dtype).reshape(batch, H, conv_width, C)
    elif conv_taps > 1:    # the input signal itself; the operator reads overlapping windows of it
        L, C = (M - 1) * conv_stride + conv_taps, K // conv_taps
        p.X = _store(normal(seed, TENSOR_X, batch * L * C, x_std), dtype).reshape(batch, L, C)
    else:
        p.X = _store(normal(seed, TENSOR_X, batch * M * K, x_std), dtype).reshape(batch, M, K)
    wb = 1 if w_shared else batch
    p.W = _store(normal(seed, TENSOR_W, wb * N * K, w_std), dtype).reshape(wb, N, K)
    if bias_range is not None:
        nb = (batch if bias_per_batch else 1) * N
        p.bias = uniform(seed, TENSOR_BIAS, nb, *bias_range)
    if scale_kind == SCALE_PER_COLUMN:
        p.scale_vec = uniform(seed, TENSOR_SCALE, N, *scale_range)
    if residual_std is not None:
        p.residual = _store(normal(seed, TENSOR_RESIDUAL, batch * M * N, residual_std), dtype).reshape(batch, M, N)
    return p


# The five named workloads (seed 0).  c1 is the small case a CPU finishes in well
# under a second; c2 is the one the headline metric is quoted on.
CONFIGS = {
    "c1": dict(batch=1, M=256, N=256, K=256, dtype=DTYPE_F32, act=ACT_GELU_TANH,
               scale_kind=SCALE_NONE, reduce=RED_LSE),
    "c2": dict(batch=1, M=4096, N=4096, K=4096, dtype=DTYPE_BF16, act=ACT_RELU,
               scale_kind=SCALE_PER_COLUMN, reduce=RED_MAXSUM, write_y=1),
    "c3": dict(batch=1, M=8192, N=8192, K=2048, dtype=DTYPE_BF16, act=ACT_NONE,
               scale_kind=SCALE_SCALAR, scale=1.0 / math.sqrt(2048.0), reduce=RED_SOFTMAX,
               bias_range=None),
    "c4": dict(batch=1, M=128, N=16384, K=8192, dtype=DTYPE_BF16, act=ACT_GELU_TANH,
               scale_kind=SCALE_NONE, reduce=RED_LSE, x_std=1.0),
    "c5": dict(batch=32, M=1024, N=1024, K=512, dtype=DTYPE_BF16, act=ACT_RELU,
               scale_kind=SCALE_NONE, reduce=RED_MAXSUM),
}


def make_config(name: str, seed: int = 0, materialize: bool = True, **overrides) -> Problem:
    kw = dict(CONFIGS[name])
    kw.update(overrides)
    return make_problem(name, seed=seed, materialize=materialize, **kw)
