"""Helpers for the GPU parity tests: move seeded inputs to the device and call
the library through its binding.  Nothing here computes any part of the method."""
import numpy as np
import torch

from paper_2603_22370_b200 import faar

DEV = "cuda:0"


def dev_bf16(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(DEV).to(torch.bfloat16).contiguous()


def dev_f32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(DEV).contiguous()


def dev_u8(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint8)).to(DEV).contiguous()


def host(t):
    if t.dtype == torch.bfloat16:
        t = t.to(torch.float32)
    return t.detach().cpu().numpy()


class GpuLayer:
    """Device state of one layer problem: buffers allocated with torch, every
    operation performed by libfaar."""

    def __init__(self, ctx, W, X, w_dtype=faar.BF16, yref_dtype=faar.BF16, yref_transposed=0):
        self.ctx = ctx
        O, K = W.shape
        T = X.shape[0]
        self.O, self.K, self.T = O, K, T
        self.ldt = (T + 7) // 8 * 8
        self.yt = yref_transposed
        self.shape = faar.make_shape(O, K, T, ldxt=self.ldt, w_dtype=w_dtype, yref_dtype=yref_dtype,
                                     yref_transposed=yref_transposed)
        self.ws = ctx.workspace(self.shape)
        self.W = dev_bf16(W) if w_dtype == faar.BF16 else dev_f32(W)
        self.X = dev_bf16(X)
        self.Xt = torch.zeros((K, self.ldt), dtype=torch.bfloat16, device=DEV)
        faar.transpose_bf16(ctx, T, K, self.X, K, self.Xt, self.ldt)
        self.scales = torch.empty((O, K // 16), dtype=torch.uint8, device=DEV)
        self.code = torch.empty((O, K // 2), dtype=torch.uint8, device=DEV)
        self.s_global = torch.empty(1, dtype=torch.float32, device=DEV)
        self.V = torch.empty((O, K), dtype=torch.float32, device=DEV)
        self.m = torch.zeros((O, K), dtype=torch.float32, device=DEV)
        self.u = torch.zeros((O, K), dtype=torch.float32, device=DEV)
        self.dYt = torch.zeros((O, self.ldt), dtype=torch.bfloat16, device=DEV)
        self.loss = torch.zeros(2, dtype=torch.float32, device=DEV)
        self.Yref = None

    def init(self, s_global_in=0.0):
        faar.softquant_init(self.ctx, self.shape, self.W, s_global_in, self.scales, self.s_global, self.code,
                            self.V, self.ws)

    def set_yref(self, Yref):
        y = dev_bf16(Yref) if self.shape.yref_dtype == faar.BF16 else dev_f32(Yref)
        if self.yt:                                   # stored [O, ldy], rows padded to a multiple of 16
            buf = torch.zeros((self.O, self.shape.ldy), dtype=y.dtype, device=DEV)
            buf[:, :self.T] = y.t()
            y = buf
        self.Yref = y

    def set_state(self, V=None, m=None, u=None):
        if V is not None:
            self.V.copy_(dev_f32(V))
        if m is not None:
            self.m.copy_(dev_f32(m))
        if u is not None:
            self.u.copy_(dev_f32(u))

    def fwd(self, hp, want_yq=False):
        Yq = None
        if want_yq:
            Yq = torch.zeros((self.O, self.shape.ldy) if self.yt else (self.T, self.O), dtype=torch.bfloat16, device=DEV)
        faar.layer_fwd(self.ctx, self.shape, hp, self.X, self.Yref, self.V, self.code, self.scales, self.s_global,
                       self.dYt, self.loss[0:1], Yq, self.ws)
        return Yq[:, :self.T].t() if (want_yq and self.yt) else Yq

    def bwd(self, hp, want_dv=True):
        dV = torch.empty((self.O, self.K), dtype=torch.float32, device=DEV) if want_dv else None
        adam = hp.opt == 1
        faar.layer_bwd(self.ctx, self.shape, hp, self.dYt, self.Xt, self.V, self.code, self.scales, self.s_global,
                       self.m if adam else None, self.u if adam else None, dV, self.ws)
        return dV

    def step(self, hp):
        adam = hp.opt == 1
        faar.layer_step(self.ctx, self.shape, hp, self.X, self.Xt, self.Yref, self.V, self.code, self.scales,
                        self.s_global, self.m if adam else None, self.u if adam else None, self.loss, self.ws)

    def check(self):
        torch.cuda.synchronize()
        faar.check_status(self.ctx, self.ws)


def rel_l2(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def max_rel_to_peak(a, b):
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return float(np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-300))


# ---- BF16 operand ties ---------------------------------------------------------------------
# The forward GEMM multiplies W_soft rounded to BF16.  The library rounds the operand from an FP32
# evaluation whose relative error is below 3e-6 (the separate FP32 parity view is tested to 1e-6);
# where the exact value lies within that error of a BF16 rounding boundary, either neighbour is a
# correct rounding.  The helpers below
# find those elements from the ORACLE's W_soft and give the exact first-order effect of moving
# one of them by one BF16 step, so that a comparison can allow for it and nothing else.

W_SOFT_FP32_TOL = 3e-6


def bf16_tie_elements(W_soft, tol=W_SOFT_FP32_TOL):
    """(mask of elements within tol*|w| of a BF16 rounding boundary, BF16 spacing at each element)."""
    w = np.abs(np.asarray(W_soft, np.float64))
    with np.errstate(divide="ignore"):
        step = np.where(w > 0, np.exp2(np.floor(np.log2(np.where(w > 0, w, 1.0))) - 7), 0.0)
    frac = np.where(step > 0, w / np.where(step > 0, step, 1.0), 0.0) % 1.0
    tie = (step > 0) & (np.abs(frac - 0.5) * step <= tol * w)
    return tie, step


def dy_column_allowance(X, tie, step, mse_scale):
    """Per output feature o: norm of the largest change of dY[:, o] that re-rounding the tie
    elements of row o can cause (dY = 2c (X W_soft^T - Y_ref))."""
    Xd = np.asarray(X, np.float64)
    xn = np.linalg.norm(Xd, axis=0)                                   # ||X[:, k]||
    return 2.0 * mse_scale * (np.where(tie, step, 0.0) * xn[None, :]).sum(axis=1)


def dv_row_allowance(X, tie, step, chain, mse_scale):
    """Per weight row o: norm of the largest change of dV[o, :] from re-rounding its tie elements:
    delta dV[o, :] = 2c * step * (X[:, k]^T X) * chain[o, :]."""
    Xd = np.asarray(X, np.float64)
    out = np.zeros(tie.shape[0])
    for o, k in zip(*np.nonzero(tie)):
        out[o] += np.linalg.norm(2.0 * mse_scale * step[o, k] * (Xd[:, k] @ Xd) * chain[o])
    return out
