"""CPU oracle for full-model alignment (Stage 2: Eq. 6, Procedure steps 15-24) on a small Llama-style model.

TEST INFRASTRUCTURE ONLY, like faar_oracle.py: plain numpy, float64, one operation at a time in the order a
decoder block applies them; it imports nothing from the product path and shares no code with the CUDA sources.

The model family is the one the paper quantises (Llama 3 / Qwen 3 decoder blocks): token embedding; per block
RMSNorm -> q, k, v projections -> rotary position embedding on q and k -> causal attention with grouped
key/value heads -> output projection -> residual; RMSNorm -> gate, up projections -> silu(gate) * up -> down
projection -> residual; final RMSNorm; LM head.  The paper takes these as given and defines only what is
trained: every linear of every block carries its own rounding tensor V (Eq. 2 / Eq. 3), and one loss (Eq. 6)

    L = lambda_KL * KL(softmax(Z_fp / tau) || softmax(Z_q / tau)) + ||H_fp - H_q||_F^2 + lambda_round * sum_l L_round(V_l)

is minimised over all of them together.  Readings where the paper is silent: H is the hidden state the LM head
reads (after the final norm); the KL term is summed over the vocabulary and averaged over the tokens; embedding,
norms and LM head stay in full precision (the 7 linears per block are the quantised ones); activations are not
quantised in this oracle.

Every function has its backward next to it; the pins (tests/test_stage2_oracle_pins.py) check each backward
against central finite differences and the whole model against an independently written PyTorch double-precision
graph differentiated by autograd, and the pieces against library routines and closed forms.
"""
from __future__ import annotations

import numpy as np

from . import faar_oracle as fo

LINEARS = ("q_proj", "k_proj", "v_proj", "o_proj", "gate_proj", "up_proj", "down_proj")


# --------------------------------------------------------------------------
# pieces of a decoder block, each with its backward
# --------------------------------------------------------------------------

def rmsnorm(x, g, eps=1e-5):
    """y = x / sqrt(mean(x^2) + eps) * g over the last axis.  Returns (y, rstd)."""
    x = np.asarray(x, np.float64)
    rstd = 1.0 / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    return x * rstd * np.asarray(g, np.float64), rstd[..., 0]


def rmsnorm_bwd(dy, x, g, rstd):
    """Gradient of rmsnorm with respect to x (the norm weights are frozen).
    With xh = x * rstd and w = g * dy:  dx = rstd * (w - xh * mean(w * xh))."""
    x = np.asarray(x, np.float64)
    r = np.asarray(rstd, np.float64)[..., None]
    xh = x * r
    w = np.asarray(dy, np.float64) * np.asarray(g, np.float64)
    return r * (w - xh * np.mean(w * xh, axis=-1, keepdims=True))


def rope_angles(positions, head_dim, theta=10000.0):
    """Angle of pair i (i < head_dim / 2) at position p: p * theta^(-2 i / head_dim).  [T, head_dim / 2]."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    return np.asarray(positions, np.float64)[:, None] * theta ** (-2.0 * i / head_dim)[None, :]


def rope(x, positions, n_heads, head_dim, theta=10000.0, inverse=False):
    """Rotary position embedding in the half-split convention of the Llama / Qwen reference code: inside every
    head, element i pairs with element i + head_dim / 2 and the pair is rotated by the angle above.
    x: [T, n_heads * head_dim].  inverse=True rotates by the negative angle, which is also the backward pass
    (the map is orthogonal)."""
    x = np.asarray(x, np.float64)
    T = x.shape[0]
    a = rope_angles(positions, head_dim, theta)
    c, s = np.cos(a)[:, None, :], np.sin(a)[:, None, :]
    if inverse:
        s = -s
    xv = x.reshape(T, n_heads, head_dim)
    h = head_dim // 2
    x1, x2 = xv[..., :h], xv[..., h:]
    out = np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)
    return out.reshape(T, n_heads * head_dim)


def attention(q, k, v, batch, seq, n_heads, n_kv_heads, head_dim):
    """Causal softmax attention with grouped key/value heads: query head h reads key/value head
    h // (n_heads / n_kv_heads); token t of a sequence sees tokens <= t of the same sequence; scores scaled by
    1 / sqrt(head_dim).  q: [batch*seq, n_heads*head_dim], k, v: [batch*seq, n_kv_heads*head_dim].
    Returns (out [batch*seq, n_heads*head_dim], probabilities [batch, n_heads, seq, seq])."""
    q = np.asarray(q, np.float64).reshape(batch, seq, n_heads, head_dim)
    k = np.asarray(k, np.float64).reshape(batch, seq, n_kv_heads, head_dim)
    v = np.asarray(v, np.float64).reshape(batch, seq, n_kv_heads, head_dim)
    rep = n_heads // n_kv_heads
    out = np.zeros((batch, seq, n_heads, head_dim))
    P = np.zeros((batch, n_heads, seq, seq))
    mask = np.tril(np.ones((seq, seq), bool))
    for b in range(batch):
        for h in range(n_heads):
            kv = h // rep
            s = q[b, :, h, :] @ k[b, :, kv, :].T / np.sqrt(head_dim)
            s = np.where(mask, s, -np.inf)
            s = s - s.max(axis=1, keepdims=True)
            p = np.exp(s)
            p /= p.sum(axis=1, keepdims=True)
            P[b, h] = p
            out[b, :, h, :] = p @ v[b, :, kv, :]
    return out.reshape(batch * seq, n_heads * head_dim), P


def attention_bwd(dout, q, k, v, P, batch, seq, n_heads, n_kv_heads, head_dim):
    """Gradients of attention() with respect to q, k, v.  Per head: dV += P^T dO; dP = dO V^T;
    dS = P * (dP - rowsum(dP * P)); dQ = dS K / sqrt(d); dK += dS^T Q / sqrt(d) (key/value heads collect the
    contributions of the query heads that share them)."""
    q = np.asarray(q, np.float64).reshape(batch, seq, n_heads, head_dim)
    k = np.asarray(k, np.float64).reshape(batch, seq, n_kv_heads, head_dim)
    v = np.asarray(v, np.float64).reshape(batch, seq, n_kv_heads, head_dim)
    do = np.asarray(dout, np.float64).reshape(batch, seq, n_heads, head_dim)
    rep = n_heads // n_kv_heads
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    sc = 1.0 / np.sqrt(head_dim)
    for b in range(batch):
        for h in range(n_heads):
            kv = h // rep
            p = P[b, h]
            dv[b, :, kv, :] += p.T @ do[b, :, h, :]
            dp = do[b, :, h, :] @ v[b, :, kv, :].T
            ds = p * (dp - np.sum(dp * p, axis=1, keepdims=True))
            dq[b, :, h, :] = ds @ k[b, :, kv, :] * sc
            dk[b, :, kv, :] += ds.T @ q[b, :, h, :] * sc
    n = batch * seq
    return dq.reshape(n, -1), dk.reshape(n, -1), dv.reshape(n, -1)


def silu_mul_bwd(dout, gate, up):
    """Gradients of silu(g) * u: with s = sigmoid(g), d/dg = u * s * (1 + g * (1 - s)), d/du = g * s."""
    g = np.asarray(gate, np.float64)
    u = np.asarray(up, np.float64)
    d = np.asarray(dout, np.float64)
    with np.errstate(over="ignore"):
        s = 1.0 / (1.0 + np.exp(-g))
    return d * u * s * (1.0 + g * (1.0 - s)), d * g * s


def embedding(table, tokens):
    """Row gather: out[t] = table[tokens[t]]."""
    return np.asarray(table, np.float64)[np.asarray(tokens).reshape(-1)]


# --------------------------------------------------------------------------
# the model
# --------------------------------------------------------------------------

class ModelCfg:
    def __init__(self, vocab, hidden, n_layers, n_heads, n_kv_heads, head_dim, ffn, eps=1e-5, theta=10000.0):
        self.vocab, self.hidden, self.n_layers = vocab, hidden, n_layers
        self.n_heads, self.n_kv_heads, self.head_dim, self.ffn = n_heads, n_kv_heads, head_dim, ffn
        self.eps, self.theta = eps, theta

    def linear_shapes(self):
        """(O, K) of the seven linears of one block."""
        d, q, kv, f = self.hidden, self.n_heads * self.head_dim, self.n_kv_heads * self.head_dim, self.ffn
        return {"q_proj": (q, d), "k_proj": (kv, d), "v_proj": (kv, d), "o_proj": (d, q),
                "gate_proj": (f, d), "up_proj": (f, d), "down_proj": (d, f)}


def forward(cfg, params, weights, tokens, keep=False):
    """Forward pass.  params: dict with "embed" [vocab, hidden], "final_norm" [hidden], "lm_head" [vocab, hidden]
    and per layer l "attn_norm.l", "mlp_norm.l" [hidden]; weights: weights[l][name] = [O, K] matrix of each
    linear (the frozen ones, or Eq. 2's soft weights).  tokens: [batch, seq] ints.
    Returns (logits [batch*seq, vocab], H [batch*seq, hidden] read by the LM head, cache for backward)."""
    batch, seq = tokens.shape
    pos = np.tile(np.arange(seq), batch)
    x = embedding(params["embed"], tokens)
    cache = []
    for l in range(cfg.n_layers):
        W = weights[l]
        c = {"x_in": x}
        hn, c["rstd1"] = rmsnorm(x, params[f"attn_norm.{l}"], cfg.eps)
        c["hn"] = hn
        q0, k0, v = hn @ W["q_proj"].T, hn @ W["k_proj"].T, hn @ W["v_proj"].T
        q = rope(q0, pos, cfg.n_heads, cfg.head_dim, cfg.theta)
        k = rope(k0, pos, cfg.n_kv_heads, cfg.head_dim, cfg.theta)
        a, P = attention(q, k, v, batch, seq, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim)
        c.update(q=q, k=k, v=v, P=P, a=a)
        x = x + a @ W["o_proj"].T
        c["x_mid"] = x
        mn, c["rstd2"] = rmsnorm(x, params[f"mlp_norm.{l}"], cfg.eps)
        c["mn"] = mn
        g, u = mn @ W["gate_proj"].T, mn @ W["up_proj"].T
        act = fo.silu_mul(g, u)
        c.update(g=g, u=u, act=act)
        x = x + act @ W["down_proj"].T
        cache.append(c)
    H, rstd_f = rmsnorm(x, params["final_norm"], cfg.eps)
    Z = H @ np.asarray(params["lm_head"], np.float64).T
    return Z, H, (cache, x, rstd_f, pos, batch, seq) if keep else None


def backward(cfg, params, weights, dZ, dH, saved):
    """Backward pass from dL/dZ and dL/dH to dL/dW of every linear (the gradient that Eq. 2 / Eq. 3 then carry
    on to V).  Returns grads[l][name] = [O, K]."""
    cache, x_last, rstd_f, pos, batch, seq = saved
    dHt = np.asarray(dH, np.float64) + np.asarray(dZ, np.float64) @ np.asarray(params["lm_head"], np.float64)
    dx = rmsnorm_bwd(dHt, x_last, params["final_norm"], rstd_f)
    grads = [dict() for _ in range(cfg.n_layers)]
    for l in reversed(range(cfg.n_layers)):
        W, c, G = weights[l], cache[l], grads[l]
        # MLP: x = x_mid + act W_down^T
        G["down_proj"] = dx.T @ c["act"]
        dact = dx @ W["down_proj"]
        dg, du = silu_mul_bwd(dact, c["g"], c["u"])
        G["gate_proj"], G["up_proj"] = dg.T @ c["mn"], du.T @ c["mn"]
        dmn = dg @ W["gate_proj"] + du @ W["up_proj"]
        dx = dx + rmsnorm_bwd(dmn, c["x_mid"], params[f"mlp_norm.{l}"], c["rstd2"])
        # attention: x_mid = x_in + a W_o^T
        G["o_proj"] = dx.T @ c["a"]
        da = dx @ W["o_proj"]
        dq, dk, dv = attention_bwd(da, c["q"], c["k"], c["v"], c["P"], batch, seq, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim)
        dq0 = rope(dq, pos, cfg.n_heads, cfg.head_dim, cfg.theta, inverse=True)
        dk0 = rope(dk, pos, cfg.n_kv_heads, cfg.head_dim, cfg.theta, inverse=True)
        G["q_proj"], G["k_proj"], G["v_proj"] = dq0.T @ c["hn"], dk0.T @ c["hn"], dv.T @ c["hn"]
        dhn = dq0 @ W["q_proj"] + dk0 @ W["k_proj"] + dv @ W["v_proj"]
        dx = dx + rmsnorm_bwd(dhn, c["x_in"], params[f"attn_norm.{l}"], c["rstd1"])
    return grads


# --------------------------------------------------------------------------
# Eq. 6 over the rounding tensors of all linears
# --------------------------------------------------------------------------

def quantised_weights(state, beta):
    """Eq. 2 for every linear: state[l][name] = (V, code, scales, s_global) -> W_soft [O, K]."""
    return [{n: fo.soft_weights(*state[l][n], beta)[0] for n in LINEARS} for l in range(len(state))]


def stage2_loss_and_grads(cfg, params, W_fp, state, tokens, beta, tau=1.0, lambda_kl=1.0, lambda_round=1.0):
    """Eq. 6 and its gradient with respect to every V (Procedure steps 16-22): run the frozen model and the
    soft-quantised model on the same tokens; data terms and their gradients from align_loss; back-propagate
    through the quantised model to dL/dW_soft; Eq. 2 / Eq. 3 chain factor; plus the Round Loss term of every
    linear, lambda_round * (1 / N_l) * (4 - 8 v).
    Returns (L_total, (L_KL, L_MSE, L_round_sum), dV[l][name])."""
    Z_fp, H_fp, _ = forward(cfg, params, W_fp, tokens)
    Wq = quantised_weights(state, beta)
    Z_q, H_q, saved = forward(cfg, params, Wq, tokens, keep=True)
    l_kl, l_mse, dZ, dH = fo.align_loss(Z_fp, Z_q, H_fp, H_q, tau, lambda_kl)
    G = backward(cfg, params, Wq, dZ, dH, saved)
    l_round, dV = 0.0, [dict() for _ in range(cfg.n_layers)]
    for l in range(cfg.n_layers):
        for n in LINEARS:
            V, code, scales, sg = state[l][n]
            Vd = np.asarray(V, np.float64)
            l_round += fo.round_loss(Vd)
            dV[l][n] = G[l][n] * fo.chain_factor(Vd, code, scales, sg, beta) + (lambda_round / Vd.size) * (4.0 - 8.0 * Vd)
    total = lambda_kl * l_kl + l_mse + lambda_round * l_round
    return total, (l_kl, l_mse, l_round), dV
