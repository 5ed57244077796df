"""`torch.autograd.Function` wrappers over the C ABI: the drop-in form of the operators
(Section 2 of the paper exposes each operator through `torch.autograd.Function`).

    residuals = fused_residual(op, fields, sources, spacing, coeffs, bc)      # tuple of tensors
    loss      = fused_residual_loss(op, fields, sources, spacing, coeffs, bc) # 0-dim fp64 tensor

`fused_residual` runs `fpde_fwd` (no loss) in the forward pass and `fpde_bwd` on the upstream
sensitivities autograd hands back.  `fused_residual_loss` also fuses the mean-square loss: the
forward pass is `fpde_fwd` with the loss, the backward pass is `fpde_bwd` on the residual
arrays with scale 2/N_r, times the incoming scalar gradient; in fp32, when a gradient is wanted,
the forward pass is `fpde_fwd_bwd` (loss and dL/dfield from one call, one kernel where the
operator has a single-pass kernel) and the backward pass only applies the incoming scalar.  Everything runs in the library's
kernels on the current CUDA stream; torch allocates the outputs and nothing else.  fp64 tensors go
through the double-precision verification kernels (`fpde_fwd_f64` / `fpde_bwd_f64`), which makes
`torch.autograd.gradcheck` usable on the operators.
"""
from __future__ import annotations

from typing import Sequence

import torch

from . import binding as B


def _check(fields, sources):
    """All tensors contiguous CUDA tensors of one dtype: fp32 (the fast kernels) or fp64 (the
    verification path).  Returns the dtype."""
    dt = fields[0].dtype
    if dt not in (torch.float32, torch.float64):
        raise ValueError("fields must be fp32 or fp64 CUDA tensors")
    for t in list(fields) + list(sources):
        if not (t.is_cuda and t.dtype == dt and t.is_contiguous()):
            raise ValueError("fields and sources must be contiguous CUDA tensors of one dtype")
    return dt


def _fwd(dt, op, fields, sources, res, loss, shape, spacing, coeffs, bc):
    dev = fields[0].device
    if dt == torch.float64:
        ws = torch.empty(B.workspace_bytes_f64(op, shape), dtype=torch.uint8, device=dev) if loss is not None else None
        B.fpde_fwd_f64(op, fields, sources, res, loss, shape, spacing, coeffs, bc, ws)
    else:
        ws = torch.empty(B.workspace_bytes(op, shape), dtype=torch.uint8, device=dev) if loss is not None else None
        B.fpde_fwd(op, fields, sources, res, loss, shape, spacing, coeffs, bc, ws)


def _bwd(dt, op, fields, gres, gscale, out, shape, spacing, coeffs, bc):
    if dt == torch.float64:
        B.fpde_bwd_f64(op, fields, gres, gscale, out, shape, spacing, coeffs, bc)
    else:
        B.fpde_bwd(op, fields, gres, gscale, out, shape, spacing, coeffs, bc)


class _FusedResidual(torch.autograd.Function):
    @staticmethod
    def forward(ctx, op, sources, spacing, coeffs, bc, *fields):
        dt = _check(fields, sources)
        shape = tuple(fields[0].shape)
        ne = B.op_info(op).nresiduals
        res = [torch.empty(shape, dtype=dt, device=fields[0].device) for _ in range(ne)]
        _fwd(dt, op, fields, sources, res, None, shape, spacing, coeffs, bc)
        ctx.op, ctx.shape, ctx.spacing, ctx.coeffs, ctx.bc, ctx.dt = op, shape, spacing, coeffs, bc, dt
        ctx.save_for_backward(*fields)
        return tuple(res)

    @staticmethod
    def backward(ctx, *gres):
        fields = ctx.saved_tensors
        g = [x.contiguous() if x is not None else torch.zeros(ctx.shape, dtype=ctx.dt, device=fields[0].device)
             for x in gres]
        out = [torch.empty(ctx.shape, dtype=ctx.dt, device=fields[0].device) for _ in fields]
        _bwd(ctx.dt, ctx.op, fields, g, None, out, ctx.shape, ctx.spacing, ctx.coeffs, ctx.bc)
        return (None, None, None, None, None) + tuple(out)


class _FusedResidualLoss(torch.autograd.Function):
    @staticmethod
    def forward(ctx, op, sources, spacing, coeffs, bc, *fields):
        dt = _check(fields, sources)
        shape = tuple(fields[0].shape)
        dev = fields[0].device
        ne = B.op_info(op).nresiduals
        loss = torch.empty(ne + 1, dtype=torch.float64, device=dev)
        ctx.op, ctx.shape, ctx.spacing, ctx.coeffs, ctx.bc, ctx.ne, ctx.dt = op, shape, spacing, coeffs, bc, ne, dt
        ctx.single_pass = dt == torch.float32 and any(ctx.needs_input_grad[5:])
        if ctx.single_pass:
            # one call: the loss and dL/dfield together (one kernel where the operator has a
            # single-pass kernel; forward + adjoint with scratch residual arrays elsewhere);
            # nothing but the gradients is kept for backward
            grads = [torch.empty(shape, dtype=torch.float32, device=dev) for _ in fields]
            ws = torch.empty(B.fwd_bwd_workspace_bytes(op, shape), dtype=torch.uint8, device=dev)
            res = None if B.has_single_pass(op) else [torch.empty(shape, dtype=torch.float32, device=dev) for _ in range(ne)]
            B.fpde_fwd_bwd(op, fields, sources, res, grads, loss, shape, spacing, coeffs, bc, ws)
            ctx.save_for_backward(*grads)
            return loss[ne]
        res = [torch.empty(shape, dtype=dt, device=dev) for _ in range(ne)]
        _fwd(dt, op, fields, sources, res, loss, shape, spacing, coeffs, bc)
        ctx.save_for_backward(*fields, *res)
        return loss[ne]

    @staticmethod
    def backward(ctx, gloss):
        saved = ctx.saved_tensors
        gl = gloss.to(ctx.dt)
        if ctx.single_pass:
            return (None, None, None, None, None) + tuple(g * gl for g in saved)
        nf = len(saved) - ctx.ne
        fields, res = saved[:nf], saved[nf:]
        out = [torch.empty(ctx.shape, dtype=ctx.dt, device=fields[0].device) for _ in fields]
        scale = 2.0 / B.row_count(ctx.op, ctx.shape)
        _bwd(ctx.dt, ctx.op, fields, res, [scale] * ctx.ne, out, ctx.shape, ctx.spacing, ctx.coeffs, ctx.bc)
        return (None, None, None, None, None) + tuple(o * gl for o in out)


def fused_residual(op, fields: Sequence[torch.Tensor], sources: Sequence[torch.Tensor], spacing, coeffs, bc):
    """All residual fields of operator `op` as differentiable tensors (zero at nodes without a row)."""
    return _FusedResidual.apply(op, tuple(sources), tuple(spacing), tuple(coeffs), tuple(bc), *fields)


def fused_residual_loss(op, fields: Sequence[torch.Tensor], sources: Sequence[torch.Tensor], spacing, coeffs, bc):
    """Sum over residual fields of the mean-square residual (fp64, 0-dim), differentiable w.r.t. the fields."""
    return _FusedResidualLoss.apply(op, tuple(sources), tuple(spacing), tuple(coeffs), tuple(bc), *fields)
