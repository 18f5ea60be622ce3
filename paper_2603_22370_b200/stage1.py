"""Stage-1 driver: layer-wise rounding optimisation of one linear, or of the linears of a block, with
libfaar.  Host loop and buffer management only -- every arithmetic step (set-up, soft weights, both
GEMMs, update, hardening, packing) is a call into the CUDA library through `faar`.

    res = optimise_layer(ctx, W, X, steps=200)          # W [O,K], X [T,K]: torch tensors on the GPU
    res["packed"], res["scales"], res["s_global"]        # deployable NVFP4 weights
"""
from __future__ import annotations

import torch

from . import faar, shard


def beta_schedule(t: int, steps: int, beta0: float = 4.0, beta1: float = 32.0) -> float:
    """Temperature of the rounding function at step t: geometric from beta0 to beta1 (the method asks
    for a small value that grows; the values are this harness's)."""
    return beta0 if steps <= 1 else beta0 * (beta1 / beta0) ** (t / (steps - 1))


def optimise_layer(ctx: faar.Context, W: torch.Tensor, X: torch.Tensor, steps: int = 200, lr: float = 1e-2,
                   lambda_round: float = 1.0, mse_scale: float = 1.0, opt: int = 1, beta0: float = 4.0,
                   beta1: float = 32.0, quantise_activations: bool = False, loss_every: int = 0,
                   rows: tuple[int, int] | None = None, s_global_in: float = 0.0) -> dict:
    """Runs the whole path for one linear layer: soft-quantisation set-up, the frozen target, `steps`
    optimisation steps, hardening and packing.  W [O,K] and X [T,K] are BF16 CUDA tensors (row-major).
    With quantise_activations the GEMMs consume NVFP4-quantised activations (the target still comes from
    the unquantised X).  Returns the packed weights, their scales, the final V and the losses read back
    every `loss_every` steps (0 = only at the end).
    rows = (b, e) restricts the problem to output rows [b, e) of W (a row shard: Eq. 5 separates over
    output features); the Round Loss weight lambda / N keeps the whole layer's N, and s_global_in must
    then be the whole tensor's scale (optimise_layer_row_sharded finds it)."""
    assert W.is_cuda and X.is_cuda and W.dtype == torch.bfloat16 and X.dtype == torch.bfloat16
    dev = W.device
    if rows is not None:
        lambda_round = lambda_round * (rows[1] - rows[0]) / W.shape[0]
        W = W[rows[0]:rows[1]].contiguous()
    O, K = W.shape
    T = X.shape[0]
    ldt = (T + 7) // 8 * 8
    shape = faar.make_shape(O, K, T, ldxt=ldt, yref_transposed=1)   # the target lives one row per output feature
    ws = torch.empty(faar.workspace_size(shape), dtype=torch.uint8, device=dev)
    faar.workspace_init(ctx, ws)
    scales = torch.empty((O, K // 16), dtype=torch.uint8, device=dev)
    code = torch.empty((O, K // 2), dtype=torch.uint8, device=dev)
    s_global = torch.empty(1, dtype=torch.float32, device=dev)
    V = torch.empty((O, K), dtype=torch.float32, device=dev)
    m = torch.zeros((O, K), dtype=torch.float32, device=dev) if opt == 1 else None
    u = torch.zeros((O, K), dtype=torch.float32, device=dev) if opt == 1 else None
    Yref = torch.zeros((O, shape.ldy), dtype=torch.bfloat16, device=dev)
    loss = torch.zeros(2, dtype=torch.float32, device=dev)

    faar.softquant_init(ctx, shape, W, s_global_in, scales, s_global, code, V, ws)
    faar.layer_ref(ctx, shape, X, W, Yref, ws)
    act_scale = 0.0
    Xg = X
    if quantise_activations:
        Xg = torch.empty_like(X)
        sx = torch.empty(1, dtype=torch.float32, device=dev)
        faar.act_fakequant(ctx, T, K, X, K, 0.0, Xg, K, sx, None, None, ws)
        act_scale = float(sx.item())                     # one read-back at set-up
    Xt = torch.zeros((K, ldt), dtype=torch.bfloat16, device=dev)
    faar.transpose_bf16(ctx, T, K, Xg, K, Xt, ldt)

    history = []
    for t in range(steps):
        # the backward pass of step t builds step t+1's soft weights (same values, one kernel fewer per step)
        hp = faar.make_hparams(beta=beta_schedule(t, steps, beta0, beta1), lambda_round=lambda_round,
                               mse_scale=mse_scale, opt=opt, lr=lr, step=t + 1, act_scale=act_scale,
                               wsoft_ready=int(t > 0),
                               beta_next=beta_schedule(t + 1, steps, beta0, beta1) if t + 1 < steps else 0.0)
        faar.layer_step(ctx, shape, hp, Xg, Xt, Yref, V, code, scales, s_global, m, u, loss, ws)
        if loss_every and (t + 1) % loss_every == 0:
            history.append((t + 1, *loss.tolist()))
    packed = torch.empty((O, K // 2), dtype=torch.uint8, device=dev)
    faar.harden_pack(ctx, shape, V, code, scales, s_global, packed, None, None, None)
    faar.check_status(ctx, ws)
    history.append((steps, *loss.tolist()))
    return {"packed": packed, "scales": scales, "s_global": s_global, "code": code, "V": V, "history": history,
            "act_scale": act_scale}


class StreamedLayer:
    """One linear whose calibration set is larger than a step's batch: `Xall` [n_mb * mb, K] stays in HBM
    and every step takes the next minibatch of `mb` rows, round-robin (rows [(t * mb) mod Ttot, +mb) at step
    t).  Set-up, all through the library: soft-quantisation of W; per minibatch the frozen target
    Y_ref = X W^T stored one row per output feature, and X^T, the K-major operand of the dW GEMM.  After
    that a step only moves pointers.  With quantise_activations the GEMM operands are the NVFP4-quantised
    minibatches under ONE tensor scale (found on the whole set); the targets come from the unquantised X."""

    def __init__(self, ctx: faar.Context, W: torch.Tensor, Xall: torch.Tensor, mb: int = 4096, opt: int = 1,
                 quantise_activations: bool = False):
        assert W.is_cuda and Xall.is_cuda and W.dtype == torch.bfloat16 and Xall.dtype == torch.bfloat16
        assert mb % 16 == 0 and Xall.shape[0] >= mb and Xall.is_contiguous() and W.is_contiguous()
        self.ctx, self.W, self.mb, self.opt = ctx, W, mb, opt
        dev = W.device
        O, K = W.shape
        self.O, self.K = O, K
        self.n_mb = Xall.shape[0] // mb
        self.shape = faar.make_shape(O, K, mb, ldxt=mb, yref_transposed=1)
        self.ws = torch.empty(faar.workspace_size(self.shape), dtype=torch.uint8, device=dev)
        faar.workspace_init(ctx, self.ws)
        self.scales = torch.empty((O, K // 16), dtype=torch.uint8, device=dev)
        self.code = torch.empty((O, K // 2), dtype=torch.uint8, device=dev)
        self.s_global = torch.empty(1, dtype=torch.float32, device=dev)
        self.V = torch.empty((O, K), dtype=torch.float32, device=dev)
        self.m = torch.zeros((O, K), dtype=torch.float32, device=dev) if opt == 1 else None
        self.u = torch.zeros((O, K), dtype=torch.float32, device=dev) if opt == 1 else None
        self.loss = torch.zeros(2, dtype=torch.float32, device=dev)
        self.Yref = torch.empty((self.n_mb, O, mb), dtype=torch.bfloat16, device=dev)
        self.Xt = torch.empty((self.n_mb, K, mb), dtype=torch.bfloat16, device=dev)
        self.X = Xall[:self.n_mb * mb].view(self.n_mb, mb, K)
        self.act_scale = 0.0
        self.setup(quantise_activations)

    def setup(self, quantise_activations: bool = False):
        ctx, s = self.ctx, self.shape
        faar.softquant_init(ctx, s, self.W, 0.0, self.scales, self.s_global, self.code, self.V, self.ws)
        for j in range(self.n_mb):
            faar.layer_ref(ctx, s, self.X[j], self.W, self.Yref[j], self.ws)
        Xg = self.X
        if quantise_activations:
            # one tensor scale for the whole calibration set: first the set's scale, then every minibatch with it
            n, K = self.n_mb * self.mb, self.K
            sx = torch.empty(1, dtype=torch.float32, device=self.W.device)
            Xg = torch.empty_like(self.X)
            faar.act_fakequant(ctx, n, K, self.X, K, 0.0, Xg, K, sx, None, None, self.ws)
            self.act_scale = float(sx.item())
            self.X = Xg
        for j in range(self.n_mb):
            faar.transpose_bf16(ctx, self.mb, self.K, Xg[j], self.K, self.Xt[j], self.mb)
        if self.m is not None:
            self.m.zero_()
            self.u.zero_()

    def step(self, t: int, steps: int, lr: float = 1e-2, lambda_round: float = 1.0, mse_scale: float = 1.0,
             beta0: float = 4.0, beta1: float = 32.0, chain: bool = True):
        j = t % self.n_mb
        kw = {}
        if chain:          # the backward pass of step t builds step t+1's soft weights (they depend on V only)
            kw = dict(wsoft_ready=int(t > 0), beta_next=beta_schedule(t + 1, steps, beta0, beta1) if t + 1 < steps else 0.0)
        hp = faar.make_hparams(beta=beta_schedule(t, steps, beta0, beta1), lambda_round=lambda_round,
                               mse_scale=mse_scale, opt=self.opt, lr=lr, step=t + 1, act_scale=self.act_scale, **kw)
        faar.layer_step(self.ctx, self.shape, hp, self.X[j], self.Xt[j], self.Yref[j], self.V, self.code, self.scales,
                        self.s_global, self.m, self.u, self.loss, self.ws)

    def finish(self) -> dict:
        packed = torch.empty((self.O, self.K // 2), dtype=torch.uint8, device=self.W.device)
        faar.harden_pack(self.ctx, self.shape, self.V, self.code, self.scales, self.s_global, packed, None, None, None)
        faar.check_status(self.ctx, self.ws)
        return {"packed": packed, "scales": self.scales, "s_global": self.s_global, "code": self.code, "V": self.V,
                "losses": self.loss.tolist(), "act_scale": self.act_scale}


def optimise_layer_streamed(ctx: faar.Context, W: torch.Tensor, Xall: torch.Tensor, steps: int, mb: int = 4096,
                            opt: int = 1, quantise_activations: bool = False, **step_kw) -> dict:
    """Stage 1 for one linear over a calibration set of several minibatches (see StreamedLayer)."""
    lay = StreamedLayer(ctx, W, Xall, mb, opt, quantise_activations)
    for t in range(steps):
        lay.step(t, steps, **step_kw)
    return lay.finish()


#: the order in which the linears of a decoder block are optimised, and where each takes its input from
BLOCK_LINEARS = ("q_proj", "k_proj", "v_proj", "o_proj", "gate_proj", "up_proj", "down_proj")


def mlp_activation(ctx: faar.Context, W_gate: torch.Tensor, W_up: torch.Tensor, H: torch.Tensor, mb: int = 4096) -> torch.Tensor:
    """The frozen model's input of down_proj, silu(H W_gate^T) * (H W_up^T), for every calibration row: two
    tensor-core GEMMs and the gated product per minibatch, all by the library; nothing leaves the device."""
    n, hid = H.shape
    F = W_gate.shape[0]
    A = torch.empty((n, F), dtype=torch.bfloat16, device=H.device)
    G = torch.empty((mb, F), dtype=torch.bfloat16, device=H.device)
    ws = torch.empty(faar.workspace_size(faar.make_shape(F, hid, mb)), dtype=torch.uint8, device=H.device)
    faar.workspace_init(ctx, ws)
    for b in range(0, n, mb):
        rows = min(mb, n - b)
        s = faar.make_shape(F, hid, rows)
        faar.layer_ref(ctx, s, H[b:b + rows], W_gate, G[:rows], ws)
        faar.layer_ref(ctx, s, H[b:b + rows], W_up, A[b:b + rows], ws)
        faar.silu_mul(ctx, rows, F, G, F, A[b:b + rows], F, A[b:b + rows], F)
    faar.check_status(ctx, ws)
    return A


def optimise_decoder_block(ctx: faar.Context, weights: dict, H: torch.Tensor, H_o: torch.Tensor, steps: int,
                           mb: int = 4096, rank: int = 0, world: int = 1, **kw) -> dict:
    """Stage 1 for the seven linears of one decoder block against the frozen block.  `weights` maps the names
    in BLOCK_LINEARS to BF16 matrices [O, K]; H [Ttot, hidden] are the block's normalised input hidden states
    (input of q, k, v, gate and up); H_o [Ttot, hidden] is the input of o_proj (the attention output of the
    frozen model, supplied by the caller); down_proj's input is formed here from H and the frozen gate / up
    weights.  Every linear is an independent problem: with several processes the linears are dealt
    round-robin and nothing is exchanged."""
    out = {}
    mine = shard.layers_for_rank(len(BLOCK_LINEARS), rank, world)
    for i in mine:
        name = BLOCK_LINEARS[i]
        if name == "down_proj":
            X = mlp_activation(ctx, weights["gate_proj"], weights["up_proj"], H, mb)
        else:
            X = H_o if name == "o_proj" else H
        out[name] = optimise_layer_streamed(ctx, weights[name], X, steps, mb, **kw)
        del X
    return out


def optimise_model(ctx: faar.Context, blocks, steps: int, mb: int = 4096, rank: int = 0, world: int = 1, **kw):
    """Stage 1 over a whole model, block by block (Procedure steps 1-14, "for each layer").  `blocks` yields
    (weights, H, H_o) per decoder block -- the frozen model's hidden states at that block's input and at its
    o_proj, produced by the caller (a generator keeps only one block's calibration set in HBM at a time).
    Returns one result dict per block."""
    return [optimise_decoder_block(ctx, w, H, H_o, steps, mb, rank, world, **kw) for (w, H, H_o) in blocks]


def optimise_block(ctx: faar.Context, linears: list, steps: int, rank: int = 0, world: int = 1, **kw) -> dict:
    """Optimises the linears of a decoder block, `linears` = [(name, W, X), ...].  Layer problems are
    independent, so with several processes each rank takes its share (round-robin) and no data moves
    between ranks; the caller gathers the returned dicts if it needs them in one place."""
    out = {}
    for i in shard.layers_for_rank(len(linears), rank, world):
        name, W, X = linears[i]
        out[name] = optimise_layer(ctx, W, X, steps=steps, **kw)
    return out


def optimise_layer_row_sharded(ctx: faar.Context, W: torch.Tensor, X: torch.Tensor, rank: int, world: int,
                               **kw) -> dict:
    """One layer split by output rows over `world` processes (X replicated, W whole or at least this
    rank's rows valid).  Set-up: each rank derives the tensor scale of its rows, the ranks take the largest
    (one scalar MAX all-reduce); then every step is local.  Returns this rank's rows of the result, the row
    range, and the whole layer's final losses."""
    b, e = shard.rows_for_rank(W.shape[0], rank, world)
    O, K = e - b, W.shape[1]
    dev = W.device
    if O == 0:                     # more ranks than rows: this rank only takes part in the two collectives
        shard.global_tensor_scale(torch.zeros(1, dtype=torch.float32, device=dev))
        return {"rows": (b, e), "layer_losses": shard.combine_losses(torch.zeros(2, device=dev), 0, W.shape[0]).tolist()}
    Wl = W[b:e].contiguous()
    shape = faar.make_shape(O, K, 8)
    ws = torch.empty(faar.workspace_size(shape), dtype=torch.uint8, device=dev)
    faar.workspace_init(ctx, ws)
    s_local = torch.empty(1, dtype=torch.float32, device=dev)
    faar.softquant_init(ctx, shape, Wl, 0.0, torch.empty((O, K // 16), dtype=torch.uint8, device=dev), s_local,
                        torch.empty((O, K // 2), dtype=torch.uint8, device=dev),
                        torch.empty((O, K), dtype=torch.float32, device=dev), ws)
    s_all = float(shard.global_tensor_scale(s_local).item())
    res = optimise_layer(ctx, W, X, rows=(b, e), s_global_in=s_all, **kw)
    res["rows"] = (b, e)
    last = torch.tensor(res["history"][-1][1:], dtype=torch.float32, device=dev)
    res["layer_losses"] = shard.combine_losses(last, e - b, W.shape[0]).tolist()
    return res
