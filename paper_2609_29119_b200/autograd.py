"""Differentiable wrappers: torch.autograd.Function objects whose forward and backward are the library's own calls.

Under the real inner product <u, v> = Re(u^H v) (Sec. 3.2) the backward of the analysis T is the real adjoint
T^dagger (cqt_analyse_adjoint) applied to the coefficient cotangent, and the backward of the synthesis S is
S^dagger (cqt_synthesise_adjoint) applied to the signal cotangent.  That is PyTorch's convention for complex
tensors (the gradient of a real loss with respect to c is dL/dRe c + i dL/dIm c).  No transform activation is
saved: both backward passes need the cotangent only.  Argument marshalling only; all arithmetic runs in the kernels.
"""
import torch


class _Analyse(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x, plan, valid_len):
        ctx.plan, ctx.valid_len, ctx.width = plan, valid_len, x.shape[1]
        return plan.analyse(x.contiguous(), valid_len=valid_len)

    @staticmethod
    def backward(ctx, c_bar):
        g = ctx.plan.analyse_adjoint(c_bar.contiguous(), valid_len=ctx.valid_len)
        if g.shape[1] != ctx.width:                       # columns beyond valid_len were never read: zero gradient
            g = torch.nn.functional.pad(g, (0, ctx.width - g.shape[1]))
        return g, None, None


class _Synthesise(torch.autograd.Function):
    @staticmethod
    def forward(ctx, c, plan, valid_len):
        ctx.plan, ctx.valid_len = plan, valid_len
        return plan.synthesise(c.contiguous(), valid_len=valid_len)

    @staticmethod
    def backward(ctx, x_bar):
        return ctx.plan.synthesise_adjoint(x_bar.contiguous(), valid_len=ctx.valid_len), None, None


def analyse(plan, x, valid_len=None):
    """c = T x with gradient support; x [batch, >= valid_len] float32 on the plan's device."""
    return _Analyse.apply(x, plan, x.shape[1] if valid_len is None else valid_len)


def synthesise(plan, c, valid_len=None):
    """x = S c with gradient support; c [batch, coeff_count] complex64 on the plan's device."""
    return _Synthesise.apply(c, plan, plan.N if valid_len is None else valid_len)
