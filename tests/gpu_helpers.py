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

    def __init__(self, ctx, W, X, w_dtype=faar.BF16, yref_dtype=faar.BF16):
        self.ctx = ctx
        O, K = W.shape
        T = X.shape[0]
        self.O, self.K, self.T = O, K, T
        self.ldt = (T + 7) // 8 * 8
        self.shape = faar.make_shape(O, K, T, ldxt=self.ldt, w_dtype=w_dtype, yref_dtype=yref_dtype)
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
        self.Yref = dev_bf16(Yref) if self.shape.yref_dtype == faar.BF16 else dev_f32(Yref)

    def set_state(self, V=None, m=None, u=None):
        if V is not None:
            self.V.copy_(dev_f32(V))
        if m is not None:
            self.m.copy_(dev_f32(m))
        if u is not None:
            self.u.copy_(dev_f32(u))

    def fwd(self, hp, want_yq=False):
        Yq = torch.empty((self.T, self.O), dtype=torch.bfloat16, device=DEV) if want_yq else None
        faar.layer_fwd(self.ctx, self.shape, hp, self.X, self.Yref, self.V, self.code, self.scales, self.s_global,
                       self.dYt, self.loss[0:1], Yq, self.ws)
        return Yq

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
