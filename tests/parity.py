"""Helpers of the GPU parity tests: run a problem through the C ABI on the device, run the same
bits through the CPU oracle, compare element by element.

Tolerances.  The stated bars are  max |err| <= 1e-4 (1 + |ref|)  for fp32 and  <= 2e-2 (1 + |ref|)
for bf16 inputs with fp32 accumulation.  They are loose for small outputs, so every comparison is
also held to tighter bounds derived from the arithmetic:

  Y / P stored as bf16 : bf16 keeps 8 significant bits, so one rounding is at most 2^-8 = 3.9e-3
                         relative; softmax rounds twice (the stored exponential and the rescaled value)
                         -> 7.8e-3; fast exp2/division add < 1e-5.  Bound: |err| <= 4.5e-3 |ref| + atol
                         (softmax: 9e-3 |ref| + 1e-7), atol = 2e-5 (1 + max|ref|) for the fp32
                         accumulation error of z where z + b nearly cancels.
  Y / P stored as fp32 : |err| <= 1e-5 |ref| + 1e-6 (1 + max|ref|).
  reductions (fp32)    : |err| <= tol (1 + |ref|) + 1e-6 * sum_n |y|  with tol = 2e-4 on the tcgen05
                         paths (fast exp2, bf16 inputs) and 1e-5 on the fp32 path; the second term
                         covers cancellation in sum_n y.
"""
from __future__ import annotations

import numpy as np
import torch

import fgr_inputs as gi
import oracle
import paper_2511_06345_b200 as fgr


def to_device(p: gi.Problem, device="cuda:0"):
    """Uploads the problem's host arrays; bf16 bit patterns are reinterpreted, not converted."""
    def up(a, bits16):
        if a is None:
            return None
        t = torch.from_numpy(np.ascontiguousarray(a))
        if bits16:
            t = t.view(torch.int16).view(torch.bfloat16)
        return t.to(device)
    b16 = p.dtype == gi.DTYPE_BF16
    return up(p.X, b16), up(p.W, b16), up(p.bias, False), up(p.scale_vec, False)


def run_gpu(p: gi.Problem, force_path=0, force_tile_n=0, device=0, tensors=None, repeat=1, force_cta_pair=0, force_ksub=0):
    """Runs the operator through fgr_create / fgr_run; returns (Y float64 [rows, N] or None,
    out float64 [rows, w] or None, plan dict)."""
    op = fgr.FusedGemmReduce(p.batch, p.M, p.N, p.K, p.dtype, p.act, p.scale_kind, p.reduce, scale=p.scale,
                             write_y=p.write_y, bias_per_batch=p.bias_per_batch, device=device,
                             force_path=force_path, force_tile_n=force_tile_n, force_cta_pair=force_cta_pair, force_ksub=force_ksub,
                             conv_taps=p.conv_taps, w_shared=p.w_shared, conv_rows=p.conv_rows, conv_width=p.conv_width,
                             ldx=(p.conv_stride * (p.K // p.conv_taps) if p.conv_taps > 1 and p.conv_stride > 1 else 0))
    X, W, b, s = tensors if tensors is not None else to_device(p, "cuda:%d" % device)
    R = None
    if getattr(p, "residual", None) is not None:
        t = torch.from_numpy(np.ascontiguousarray(p.residual))
        R = (t.view(torch.int16).view(torch.bfloat16) if p.dtype == gi.DTYPE_BF16 else t).to("cuda:%d" % device)
    for _ in range(repeat):
        Y, out = op(X, W, b, s, residual=R)
    st = op.status()
    assert st == fgr.FGR_OK, fgr.fgr_status_string(st)
    plan = op.plan.as_dict()
    op.close()
    Yh = None if Y is None else Y.float().cpu().numpy().astype(np.float64).reshape(p.batch * p.M, p.N)
    oh = None if out is None else out.cpu().numpy().astype(np.float64).reshape(p.batch * p.M, -1)
    return Yh, oh, plan


def compare(p: gi.Problem, Y, out, rows=None, tcgen05=True, softmax_rel=9e-3, y_slack=None, out_slack=None, y_rel_slack=None):
    """Asserts GPU results (all rows, or the listed global rows) against the oracle.  Returns the
    achieved maxima of |err| / (1 + |ref|) for Y and out.  ``softmax_rel``: relative bound on a bf16 P
    (4.5e-3 per rounding: two on the single-GPU path, three when a shard combine rescales once more).
    ``y_slack`` [rows, N] / ``out_slack`` [rows, w]: extra absolute allowance on the tight bounds that a
    path derives from its own arithmetic, ``y_rel_slack`` [rows, 1] the same relative to |ref| (the stated
    tolerance is never widened)."""
    Yr, outr, _ = oracle.run_problem(p, rows=rows, want_y=True)
    if rows is not None:
        Y = None if Y is None else Y[rows]
        out = None if out is None else out[rows]
    official = 1e-4 if p.dtype == gi.DTYPE_F32 else 2e-2
    worst = {}
    if Y is not None:
        err = np.abs(Y - Yr)
        worst["Y"] = float((err / (1 + np.abs(Yr))).max())
        assert worst["Y"] <= official, "Y/P beyond the stated tolerance: %g" % worst["Y"]
        big = np.abs(Yr).max()
        if p.dtype == gi.DTYPE_F32:
            bound = 1e-5 * np.abs(Yr) + 1e-6 * (1 + big)
        elif p.reduce == gi.RED_SOFTMAX:
            bound = softmax_rel * np.abs(Yr) + 1e-7
        else:
            bound = 4.5e-3 * np.abs(Yr) + 2e-5 * (1 + big)
        if y_slack is not None:
            bound = bound + y_slack
        if y_rel_slack is not None:      # [rows, 1]: extra relative allowance (softmax: an error of the logits)
            bound = bound + y_rel_slack * np.abs(Yr)
        bad = err > bound
        assert not bad.any(), "Y/P: %d elements beyond the tight bound, worst ratio %g at %s" % (
            bad.sum(), (err / bound).max(), np.unravel_index(np.argmax(err / bound), err.shape))
        if p.reduce == gi.RED_SOFTMAX:
            assert np.abs(Y.sum(1) - 1).max() <= (1e-2 if p.dtype == gi.DTYPE_BF16 else 1e-5)
            assert Y.min() >= 0 and Y.max() <= 1 + 1e-6
    if out is not None:
        err = np.abs(out - outr)
        worst["out"] = float((err / (1 + np.abs(outr))).max())
        assert worst["out"] <= official, "reduction beyond the stated tolerance: %g" % worst["out"]
        tol = 2e-4 if (tcgen05 and p.dtype == gi.DTYPE_BF16) else 1e-5
        cancel = 1e-6 * np.abs(Yr).sum(1, keepdims=True) if p.reduce == gi.RED_MAXSUM else 0.0
        bound = tol * (1 + np.abs(outr)) + cancel
        if out_slack is not None:
            bound = bound + out_slack
        bad = err > bound
        assert not bad.any(), "reduction: %d values beyond the tight bound, worst ratio %g" % (
            bad.sum(), (err / bound).max())
    return worst
