"""Convenience wrapper over the C ABI for torch users: allocates outputs and workspace with torch
and passes raw pointers and the current stream to ``fgr_run``.  No arithmetic happens here."""
from __future__ import annotations

import torch

from . import binding as B


class FusedGemmReduce:
    """One operator instance (a handle of the C library) bound to a CUDA device.

    ``__call__(X, W, bias=None, scale_vec=None)`` returns ``(Y_or_None, out_or_None)``:
    Y / P is bf16 or fp32 [batch, M, N]; out is fp32 [batch*M] (LSE) or [batch*M, 2].
    X [batch, M, K] and W [batch, N, K] are packed CUDA tensors (bf16 or fp32 as configured).
    With ``conv_taps = R > 1`` (1-D convolution as an implicit GEMM) X is the channels-last input
    [batch, M + R - 1, K / R] (stride s: ``ldx = s * K / R``, signal length (M - 1) s + R) and W the filters [batch, N, K]; ``w_shared=1``: W is one [N, K] matrix
    for all batch elements.  ``conv_rows = R > 1``: 2-D convolution, X the channels-last image
    [batch, H, conv_width, K / (R * conv_taps)], output rows at the image's row pitch (see ``include/fgr.h``).
    """

    def __init__(self, batch, M, N, K, dtype, act, scale_kind, reduce, *, scale=1.0, write_y=0, bias_per_batch=0,
                 device=0, force_path=B.FGR_PATH_AUTO, force_tile_n=0, force_cta_pair=0, force_ksub=0, conv_taps=0, w_shared=0, ldx=0, conv_rows=0,
                 conv_width=0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this operator has no CPU path")
        self.desc = B.make_desc(batch, M, N, K, dtype, act, scale_kind, reduce, scale=scale, write_y=write_y,
                                bias_per_batch=bias_per_batch, device=device, force_path=force_path,
                                force_tile_n=force_tile_n, force_cta_pair=force_cta_pair, force_ksub=force_ksub,
                                conv_taps=conv_taps, w_shared=w_shared, ldx=ldx, conv_rows=conv_rows, conv_width=conv_width)
        self.handle = B.fgr_create(self.desc)
        self.plan = B.fgr_get_plan(self.handle)
        self.device = torch.device("cuda", device)
        self.workspace_bytes = B.fgr_workspace_bytes(self.handle)
        self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=self.device)
        self.tdtype = torch.float32 if dtype == B.FGR_F32 else torch.bfloat16
        rows = batch * M
        self.need_y = bool(write_y) or reduce == B.FGR_RED_SOFTMAX
        self.out_shape = None if reduce == B.FGR_RED_SOFTMAX else ((rows,) if reduce == B.FGR_RED_LSE else (rows, 2))

    @property
    def path(self) -> str:
        return B.fgr_path_name(self.plan.path)

    def __call__(self, X, W, bias=None, scale_vec=None, Y=None, out=None, residual=None):
        d = self.desc
        B.fgr_set_residual(self.handle, residual)     # [batch, M, N] in the operator's dtype, packed; None = none
        self._residual = residual                     # keeps the tensor alive while the handle points at it
        if Y is None and self.need_y:
            Y = torch.empty((d.batch, d.M, d.N), dtype=self.tdtype, device=self.device)
        if out is None and self.out_shape is not None:
            out = torch.empty(self.out_shape, dtype=torch.float32, device=self.device)
        stream = torch.cuda.current_stream(self.device).cuda_stream
        B.fgr_run(self.handle, X, W, bias, scale_vec, Y if self.need_y else None, out, self.workspace,
                  self.workspace_bytes, stream)
        return (Y if self.need_y else None), out

    def status(self) -> int:
        return B.fgr_get_status(self.handle)

    def close(self):
        if self.handle is not None:
            B.fgr_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
