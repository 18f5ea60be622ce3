"""Stage-2 driver: full-model alignment (Eq. 6, Procedure steps 15-24) of a Llama-style decoder model whose
linears all carry their own rounding tensor V.  Host loop and buffer management only: every arithmetic step --
embedding, norms, rotary embedding, attention, the gated MLP, every matrix product, the loss with its gradients,
the chain rule into V, the optimiser update -- is a call into the CUDA library through `faar`.

One step (`Stage2Model.step`):
  frozen model forward (BF16 weights)                      -> Z_fp, H_fp            Procedure 16
  quantised model forward (Eq. 2 soft weights of every V)  -> Z_q, H_q, activations Procedure 17
  faar_align_loss                                          -> L_KL, L_MSE, dZ_q, dH_q   Procedure 18-20, Eq. 6
  backward through the quantised model; per linear: input gradient dX = dY W_soft (faar_layer_dx_operand on the
  forward pass's soft weights, i.e. at the pre-update V), then dW GEMM + chain rule + Round Loss gradient + optimiser update + clip (faar_layer_bwd)
                                                                                     Procedure 21-23
Embedding, norms and LM head are frozen and stay in BF16 / FP32; the seven linears of every block are quantised.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from . import faar

LINEARS = ("q_proj", "k_proj", "v_proj", "o_proj", "gate_proj", "up_proj", "down_proj")
GROUPS = {"qkv": ("q_proj", "k_proj", "v_proj"), "gate_up": ("gate_proj", "up_proj")}      # linears with a common input


@dataclass
class ModelConfig:
    vocab: int
    hidden: int
    n_layers: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    eps: float = 1e-5
    theta: float = 10000.0

    def linear_shapes(self) -> dict:
        d, q, kv, f = self.hidden, self.n_heads * self.head_dim, self.n_kv_heads * self.head_dim, self.ffn
        return {"q_proj": (q, d), "k_proj": (kv, d), "v_proj": (kv, d), "o_proj": (d, q),
                "gate_proj": (f, d), "up_proj": (f, d), "down_proj": (d, f)}


class QuantLinear:
    """Device state of one quantised linear: frozen W, its NVFP4 bracket (scales, code, tensor scale), the
    rounding tensor V with its Adam moments, and a BF16 buffer for the soft weights of the current step."""

    def __init__(self, ctx: faar.Context, W: torch.Tensor, ws: torch.Tensor, opt: int = 1, Wsoft: torch.Tensor | None = None):
        O, K = W.shape
        dev = W.device
        self.W, self.O, self.K = W, O, K
        self.scales = torch.empty((O, K // 16), dtype=torch.uint8, device=dev)
        self.code = torch.empty((O, K // 2), dtype=torch.uint8, device=dev)
        self.s_global = torch.empty(1, dtype=torch.float32, device=dev)
        self.V = torch.empty((O, K), dtype=torch.float32, device=dev)
        self.m = torch.zeros((O, K), dtype=torch.float32, device=dev) if opt == 1 else None
        self.u = torch.zeros((O, K), dtype=torch.float32, device=dev) if opt == 1 else None
        self.Wsoft = Wsoft if Wsoft is not None else torch.empty((O, K), dtype=torch.bfloat16, device=dev)
        faar.softquant_init(ctx, faar.make_shape(O, K, 8), W, 0.0, self.scales, self.s_global, self.code, self.V, ws)


class Stage2Model:
    """A decoder model on one GPU.  params: "embed" [vocab, hidden] bf16, "lm_head" [vocab, hidden] bf16,
    "final_norm", "attn_norm.l", "mlp_norm.l" [hidden] float32; weights[l][name]: [O, K] bf16 (frozen)."""

    def __init__(self, ctx: faar.Context, cfg: ModelConfig, params: dict, weights: list, batch: int, seq: int, opt: int = 1):
        self.ctx, self.cfg, self.params, self.opt = ctx, cfg, params, opt
        self.batch, self.seq, self.T = batch, seq, batch * seq
        assert cfg.vocab % 16 == 0 and cfg.hidden % 16 == 0 and cfg.ffn % 16 == 0 and cfg.head_dim in (64, 128)
        dev = params["embed"].device
        self.dev = dev
        T, c = self.T, cfg
        shapes = c.linear_shapes()
        # q / k / v read the same input, and so do gate / up: each group is one matrix product over the stacked
        # weights (forward) and one input-gradient product over the stacked output gradients (backward)
        self.group_rows = {g: [shapes[n][0] for n in names] for g, names in GROUPS.items()}
        ws_shapes = list(shapes.values()) + [(sum(self.group_rows[g]), shapes[names[0]][1]) for g, names in GROUPS.items()]
        self.ws = torch.empty(max(faar.workspace_size(faar.make_shape(o, k, T)) for o, k in ws_shapes), dtype=torch.uint8,
                              device=dev)
        faar.workspace_init(ctx, self.ws)
        self.lin, self.w_group, self.wsoft_group = [], [], []
        for l in range(c.n_layers):
            lins, wg, wsg = {}, {}, {}
            for g, names in GROUPS.items():
                wg[g] = torch.cat([weights[l][n] for n in names], dim=0).contiguous()
                wsg[g] = torch.empty_like(wg[g])
                r0 = 0
                for n in names:
                    r1 = r0 + shapes[n][0]
                    lins[n] = QuantLinear(ctx, wg[g][r0:r1], self.ws, opt, Wsoft=wsg[g][r0:r1])
                    r0 = r1
            for n in LINEARS:
                if n not in lins:
                    lins[n] = QuantLinear(ctx, weights[l][n], self.ws, opt)
            self.lin.append(lins)
            self.w_group.append(wg)
            self.wsoft_group.append(wsg)
        self.pos = torch.arange(seq, dtype=torch.int32, device=dev).repeat(batch)
        self.lm_head_t = torch.empty((c.hidden, (c.vocab + 7) // 8 * 8), dtype=torch.bfloat16, device=dev)
        faar.transpose_bf16(ctx, c.vocab, c.hidden, params["lm_head"], c.hidden, self.lm_head_t, self.lm_head_t.shape[1])
        self.aws = torch.empty(faar.align_loss_workspace_size(T, c.vocab), dtype=torch.uint8, device=dev)
        faar.workspace_init(ctx, self.aws)
        self.loss = torch.zeros(2, dtype=torch.float32, device=dev)
        self.ldt = (T + 7) // 8 * 8
        self.dsum = torch.empty((batch, c.n_heads, seq), dtype=torch.float32, device=dev)
        self.step_count = 0

    # ---- helpers ------------------------------------------------------------------------------------
    def _new(self, cols, dtype=torch.bfloat16):
        return torch.empty((self.T, cols), dtype=dtype, device=self.dev)

    def _matmul(self, X, W):
        """Y[T, O] = X[T, K] W[O, K]^T on the tensor cores (the frozen-target GEMM)."""
        O, K = W.shape
        Y = self._new(O)
        faar.layer_ref(self.ctx, faar.make_shape(O, K, self.T), X, W, Y, self.ws)
        return Y

    def _linear_group(self, l, group, X, quantised, beta):
        """The linears of one group on their common input: one product with the stacked weights.  Returns the
        [T, sum of widths] result; each linear's output is a column range of it."""
        if not quantised:
            return self._matmul(X, self.w_group[l][group])
        for n in GROUPS[group]:
            lin = self.lin[l][n]
            faar.softquant_eval(self.ctx, faar.make_shape(lin.O, lin.K, self.T), lin.V, lin.code, lin.scales, lin.s_global,
                                beta, None, None, lin.Wsoft)
        return self._matmul(X, self.wsoft_group[l][group])

    def _linear(self, l, name, X, quantised, beta):
        lin = self.lin[l][name]
        if not quantised:
            return self._matmul(X, lin.W)
        faar.softquant_eval(self.ctx, faar.make_shape(lin.O, lin.K, self.T), lin.V, lin.code, lin.scales, lin.s_global, beta,
                            None, None, lin.Wsoft)
        return self._matmul(X, lin.Wsoft)

    # ---- forward -------------------------------------------------------------------------------------
    def forward(self, tokens: torch.Tensor, quantised: bool, beta: float = 4.0, keep: bool = False):
        """tokens: [batch*seq] int32 on the device.  Returns (Z [T, vocab], H [T, hidden], cache or None)."""
        c, ctx, T = self.cfg, self.ctx, self.T
        d, qd, kvd, f = c.hidden, c.n_heads * c.head_dim, c.n_kv_heads * c.head_dim, c.ffn
        x = self._new(d)
        faar.embedding(ctx, T, d, c.vocab, self.params["embed"], d, tokens, x, d)
        cache = []
        hn, rstd1 = self._new(d), torch.empty(T, dtype=torch.float32, device=self.dev)
        faar.rmsnorm(ctx, T, d, x, d, self.params["attn_norm.0"], c.eps, hn, d, rstd1)
        for l in range(c.n_layers):
            s = {"x_in": x, "rstd1": rstd1}
            qkv = self._linear_group(l, "qkv", hn, quantised, beta)
            ldp = qkv.shape[1]
            q, k, v = qkv[:, :qd], qkv[:, qd:qd + kvd], qkv[:, qd + kvd:]
            faar.rope(ctx, T, c.n_heads, c.head_dim, q, ldp, self.pos, c.theta, 0, q, ldp)
            faar.rope(ctx, T, c.n_kv_heads, c.head_dim, k, ldp, self.pos, c.theta, 0, k, ldp)
            a = self._new(qd)
            lse = torch.empty((self.batch, c.n_heads, self.seq), dtype=torch.float32, device=self.dev)
            faar.attention_fwd(ctx, self.batch, self.seq, c.n_heads, c.n_kv_heads, c.head_dim, q, ldp, k, v, ldp, a, qd, lse)
            o = self._linear(l, "o_proj", a, quantised, beta)
            # residual connection and the MLP's norm in one pass
            x_mid, mn, s["rstd2"] = self._new(d), self._new(d), torch.empty(T, dtype=torch.float32, device=self.dev)
            faar.add_rmsnorm(ctx, T, d, x, d, o, d, x_mid, d, self.params[f"mlp_norm.{l}"], c.eps, mn, d, s["rstd2"])
            gu = self._linear_group(l, "gate_up", mn, quantised, beta)
            g, u = gu[:, :f], gu[:, f:]
            act = self._new(f)
            faar.silu_mul(ctx, T, f, g, 2 * f, u, 2 * f, act, f)
            dn = self._linear(l, "down_proj", act, quantised, beta)
            if keep:
                s.update(hn=hn, q=q, k=k, v=v, a=a, lse=lse, x_mid=x_mid, mn=mn, g=g, u=u, act=act)
                cache.append(s)
            # residual connection and the next block's attention norm (after the last block: the final norm)
            g_next = self.params[f"attn_norm.{l + 1}"] if l + 1 < c.n_layers else self.params["final_norm"]
            x, hn, rstd1 = self._new(d), self._new(d), torch.empty(T, dtype=torch.float32, device=self.dev)
            faar.add_rmsnorm(ctx, T, d, x_mid, d, dn, d, x, d, g_next, c.eps, hn, d, rstd1)
        H, rstd_f = hn, rstd1
        Z = self._matmul(H, self.params["lm_head"])
        return Z, H, ((cache, x, rstd_f) if keep else None)

    # ---- backward ------------------------------------------------------------------------------------
    def _update(self, l, name, dY, ldy, X, hp, want_dv):
        """dW GEMM of one quantised linear with the chain rule into V, the Round Loss gradient, the optimiser update
        and the clip.  dY [T, O] (row stride ldy) and X [T, K] as the backward pass holds them: no transposed
        copies.  Returns dV or None."""
        lin = self.lin[l][name]
        shape = faar.make_shape(lin.O, lin.K, self.T, ldxt=self.ldt, ldy=ldy)
        dV = torch.empty((lin.O, lin.K), dtype=torch.float32, device=self.dev) if want_dv else None
        faar.layer_bwd_rowmajor(self.ctx, shape, hp, dY, X, lin.V, lin.code, lin.scales, lin.s_global, lin.m, lin.u, dV, self.ws)
        return dV

    def _linear_bwd(self, l, name, dY, X, hp, want_dv):
        """One quantised linear: dX = dY W_soft at the pre-update V, then its update.  Returns (dX, dV or None)."""
        lin = self.lin[l][name]
        dX = self._new(lin.K)
        # lin.Wsoft still holds this step's soft weights: V changes only in the update below
        faar.layer_dx_operand(self.ctx, faar.make_shape(lin.O, lin.K, self.T), dY, lin.Wsoft, dX, self.ws)
        return dX, self._update(l, name, dY, lin.O, X, hp, want_dv)

    def _group_bwd(self, l, group, dY, X, hp, want_dv, grads):
        """The linears of one group: the gradient towards their common input is one product of the stacked output
        gradients dY [T, sum of widths] with the stacked soft weights (the sum over the linears is the contraction),
        then each linear's update from its column range of dY."""
        K = self.lin[l][GROUPS[group][0]].K
        dX = self._new(K)
        faar.layer_dx_operand(self.ctx, faar.make_shape(dY.shape[1], K, self.T), dY, self.wsoft_group[l][group], dX, self.ws)
        c0 = 0
        for n in GROUPS[group]:
            O = self.lin[l][n].O
            grads[(l, n)] = self._update(l, n, dY[:, c0:c0 + O], dY.shape[1], X, hp, want_dv)
            c0 += O
        return dX

    def backward(self, dZ, dH, saved, hp, want_dv=False):
        """From the loss gradients at the logits and at the last hidden state back to every V (updated in place).
        Follows the quantised forward pass of the same step: every linear's Wsoft buffer is read as that pass left it.
        Returns {(l, name): dV} if want_dv."""
        c, ctx, T = self.cfg, self.ctx, self.T
        d, qd, kvd, f = c.hidden, c.n_heads * c.head_dim, c.n_kv_heads * c.head_dim, c.ffn
        cache, x_last, rstd_f = saved
        grads = {}
        # LM head (frozen): dH += dZ W_lm, then the final norm
        dHz = self._new(d)
        faar.layer_ref(ctx, faar.make_shape(d, self.lm_head_t.shape[1], T, ldw=self.lm_head_t.shape[1], ldx=dZ.shape[1]), dZ,
                       self.lm_head_t, dHz, self.ws)
        dx = self._new(d)
        faar.rmsnorm_bwd_sum(ctx, T, d, dHz, dH, None, d, x_last, d, self.params["final_norm"], rstd_f, None, d, dx, d)
        for l in reversed(range(c.n_layers)):
            s = cache[l]
            # MLP branch: x = x_mid + act W_down^T
            dact, grads[(l, "down_proj")] = self._linear_bwd(l, "down_proj", dx, s["act"], hp, want_dv)
            dgu = self._new(2 * f)
            faar.silu_mul_bwd(ctx, T, f, dact, f, s["g"], 2 * f, s["u"], 2 * f, dgu[:, :f], 2 * f, dgu[:, f:], 2 * f)
            dmn = self._group_bwd(l, "gate_up", dgu, s["mn"], hp, want_dv, grads)
            faar.rmsnorm_bwd(ctx, T, d, dmn, d, s["x_mid"], d, self.params[f"mlp_norm.{l}"], s["rstd2"], dx, d, dx, d)
            # attention branch: x_mid = x_in + a W_o^T
            da, grads[(l, "o_proj")] = self._linear_bwd(l, "o_proj", dx, s["a"], hp, want_dv)
            dqkv = self._new(qd + 2 * kvd)
            ldp = qd + 2 * kvd
            dq, dk, dv = dqkv[:, :qd], dqkv[:, qd:qd + kvd], dqkv[:, qd + kvd:]
            faar.attention_bwd(ctx, self.batch, self.seq, c.n_heads, c.n_kv_heads, c.head_dim, s["q"], ldp, s["k"], s["v"], ldp,
                               s["a"], da, qd, s["lse"], self.dsum, dq, dk, dv)
            faar.rope(ctx, T, c.n_heads, c.head_dim, dq, ldp, self.pos, c.theta, 1, dq, ldp)
            faar.rope(ctx, T, c.n_kv_heads, c.head_dim, dk, ldp, self.pos, c.theta, 1, dk, ldp)
            dhn = self._group_bwd(l, "qkv", dqkv, s["hn"], hp, want_dv, grads)
            faar.rmsnorm_bwd(ctx, T, d, dhn, d, s["x_in"], d, self.params[f"attn_norm.{l}"], s["rstd1"], dx, d, dx, d)
        return grads if want_dv else None

    # ---- one step of Eq. 6 -----------------------------------------------------------------------------
    def step(self, tokens: torch.Tensor, beta: float, tau: float = 1.0, lambda_kl: float = 1.0, lambda_round: float = 1.0,
             lr: float = 5e-4, want_dv: bool = False, fp_outputs=None):
        """One alignment step on a batch of token ids ([batch*seq] int32, device).  Losses {L_KL, L_MSE} are left in
        self.loss (device).  fp_outputs = (Z_fp, H_fp) reuses a frozen-model forward of the same batch.  want_dv: also
        return the quantised model's outputs, the loss gradients and every linear's dV (for inspection)."""
        self.step_count += 1
        Z_fp, H_fp = fp_outputs if fp_outputs is not None else self.forward(tokens, quantised=False)[:2]
        Z_q, H_q, saved = self.forward(tokens, quantised=True, beta=beta, keep=True)
        c, T = self.cfg, self.T
        dZ, dH = torch.empty_like(Z_q), torch.empty_like(H_q)
        faar.align_loss(self.ctx, T, c.vocab, c.hidden, Z_fp, Z_q, Z_q.shape[1], H_fp, H_q, c.hidden, tau, lambda_kl, dZ, dH,
                        self.loss, self.aws)
        hp = faar.make_hparams(beta=beta, lambda_round=lambda_round, opt=self.opt, lr=lr, step=self.step_count)
        grads = self.backward(dZ, dH, saved, hp, want_dv)
        return {"Z_q": Z_q, "H_q": H_q, "dZ": dZ, "dH": dH, "dV": grads} if want_dv else None

    def round_loss_sum(self) -> float:
        """Sum over all linears of the Round Loss (Eq. 6's third term without lambda); reads back one float each."""
        out = torch.zeros(1, dtype=torch.float32, device=self.dev)
        total = 0.0
        for layer in self.lin:
            for lin in layer.values():
                faar.round_loss(self.ctx, lin.V, lin.O * lin.K, out, self.ws)
                total += float(out.item())
        return total

    def harden(self) -> list:
        """Eq. 7 for every linear: packed NVFP4 codes (the scales and tensor scale are the set-up's)."""
        res = []
        for layer in self.lin:
            d = {}
            for n, lin in layer.items():
                packed = torch.empty((lin.O, lin.K // 2), dtype=torch.uint8, device=self.dev)
                faar.harden_pack(self.ctx, faar.make_shape(lin.O, lin.K, 8), lin.V, lin.code, lin.scales, lin.s_global, packed,
                                 None, None, None)
                d[n] = packed
            res.append(d)
        faar.check_status(self.ctx, self.ws)
        return res
