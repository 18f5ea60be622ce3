"""Pins of the Stage-2 oracle (oracle/stage2_oracle.py): every piece of a decoder block against a library
routine or a closed form, every backward against central finite differences, and the whole of Eq. 6 with its
gradient towards the rounding tensors against (a) finite differences and (b) an independently written PyTorch
float64 graph differentiated by autograd."""
import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from oracle import stage2_oracle as so
from paper_2603_22370_b200 import inputs


def fd(f, x, idx, eps=1e-6):
    xp, xm = x.copy(), x.copy()
    xp[idx] += eps
    xm[idx] -= eps
    return (f(xp) - f(xm)) / (2 * eps)


def test_rmsnorm_matches_torch_and_its_backward_matches_finite_differences():
    rng = np.random.default_rng(0)
    x, g = rng.standard_normal((5, 24)), rng.uniform(0.5, 1.5, 24)
    y, rstd = so.rmsnorm(x, g, 1e-5)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (24,), torch.from_numpy(g), 1e-5).numpy()
    assert np.allclose(y, ref, rtol=1e-13, atol=1e-14)
    assert np.allclose(so.rmsnorm(3.0 * np.ones((1, 8)), np.ones(8), 0.0)[0], 1.0)      # constant row -> ones
    w = rng.standard_normal(y.shape)                                        # L = sum(w * y)
    dx = so.rmsnorm_bwd(w, x, g, rstd)
    for idx in [(0, 0), (2, 7), (4, 23)]:
        num = fd(lambda xx: float(np.sum(w * so.rmsnorm(xx, g, 1e-5)[0])), x, idx)
        assert abs(num - dx[idx]) <= 1e-7 * max(1.0, abs(num))


def test_rope_is_a_rotation_with_the_relative_position_property():
    rng = np.random.default_rng(1)
    n_heads, dh, T = 3, 8, 7
    pos = np.array([0, 1, 2, 5, 9, 3, 3])
    x = rng.standard_normal((T, n_heads * dh))
    y = so.rope(x, pos, n_heads, dh)
    assert np.array_equal(y[0], x[0])                                       # position 0: identity
    assert np.allclose(np.linalg.norm(y.reshape(T, n_heads, dh), axis=2), np.linalg.norm(x.reshape(T, n_heads, dh), axis=2))
    assert np.allclose(so.rope(y, pos, n_heads, dh, inverse=True), x, atol=1e-13)
    # <rope(q, m), rope(k, n)> depends on m - n only
    q, k = rng.standard_normal((1, dh)), rng.standard_normal((1, dh))

    def dot(m, n):
        return float((so.rope(q, [m], 1, dh) @ so.rope(k, [n], 1, dh).T)[0, 0])

    assert abs(dot(5, 2) - dot(13, 10)) < 1e-12 and abs(dot(5, 2) - dot(5, 3)) > 1e-6
    # the half-split pairing, written independently with torch: x * cos + rotate_half(x) * sin
    inv = 10000.0 ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
    ang = torch.from_numpy(pos.astype(np.float64))[:, None] * inv[None, :]
    cos, sin = torch.cat([ang.cos(), ang.cos()], -1)[:, None, :], torch.cat([ang.sin(), ang.sin()], -1)[:, None, :]
    xt = torch.from_numpy(x).reshape(T, n_heads, dh)
    rot = torch.cat([-xt[..., dh // 2:], xt[..., :dh // 2]], -1)
    assert np.allclose(y, (xt * cos + rot * sin).reshape(T, -1).numpy(), atol=1e-13)


def test_attention_matches_the_library_routine_and_its_backward_matches_autograd():
    rng = np.random.default_rng(2)
    B, S, H, HKV, D = 2, 6, 4, 2, 8
    q, k, v = rng.standard_normal((B * S, H * D)), rng.standard_normal((B * S, HKV * D)), rng.standard_normal((B * S, HKV * D))
    out, P = so.attention(q, k, v, B, S, H, HKV, D)
    assert np.allclose(P.sum(-1), 1.0) and np.all(np.triu(P[0, 0], 1) == 0)  # causal rows of probabilities
    tq = torch.from_numpy(q).reshape(B, S, H, D).transpose(1, 2).requires_grad_(True)
    tk = torch.from_numpy(k).reshape(B, S, HKV, D).transpose(1, 2).requires_grad_(True)
    tv = torch.from_numpy(v).reshape(B, S, HKV, D).transpose(1, 2).requires_grad_(True)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk.repeat_interleave(H // HKV, 1),
                                                           tv.repeat_interleave(H // HKV, 1), is_causal=True)
    assert np.allclose(out, ref.transpose(1, 2).reshape(B * S, H * D).detach().numpy(), atol=1e-12)
    w = rng.standard_normal(out.shape)
    (ref.transpose(1, 2).reshape(B * S, H * D) * torch.from_numpy(w)).sum().backward()
    dq, dk, dv = so.attention_bwd(w, q, k, v, P, B, S, H, HKV, D)
    for mine, t, n in ((dq, tq, H), (dk, tk, HKV), (dv, tv, HKV)):
        assert np.allclose(mine, t.grad.transpose(1, 2).reshape(B * S, n * D).numpy(), atol=1e-12)
    # the first token attends to itself only
    assert np.allclose(out.reshape(B, S, H, D)[:, 0, 0], v.reshape(B, S, HKV, D)[:, 0, 0])


def test_silu_mul_backward_matches_finite_differences():
    rng = np.random.default_rng(3)
    g, u, w = rng.standard_normal((4, 9)) * 3, rng.standard_normal((4, 9)), rng.standard_normal((4, 9))
    dg, du = so.silu_mul_bwd(w, g, u)
    for idx in [(0, 0), (3, 8), (1, 4)]:
        assert abs(fd(lambda gg: float(np.sum(w * fo.silu_mul(gg, u))), g, idx) - dg[idx]) < 1e-8
        assert abs(fd(lambda uu: float(np.sum(w * fo.silu_mul(g, uu))), u, idx) - du[idx]) < 1e-8
    assert so.silu_mul_bwd(np.ones(1), np.zeros(1), np.array([2.0]))[0][0] == 1.0      # silu'(0) = 1/2, times u = 2


def test_embedding_is_a_row_gather():
    tab = np.arange(12.0).reshape(4, 3)
    assert np.array_equal(so.embedding(tab, np.array([[3, 0], [1, 3]])), tab[[3, 0, 1, 3]])


# ---- the whole model ------------------------------------------------------------------------------

def tiny_model(seed=0):
    cfg = so.ModelCfg(vocab=37, hidden=32, n_layers=2, n_heads=4, n_kv_heads=2, head_dim=8, ffn=48)
    rng = np.random.default_rng(seed)
    params = {"embed": rng.standard_normal((cfg.vocab, cfg.hidden)), "final_norm": rng.uniform(0.8, 1.2, cfg.hidden),
              "lm_head": 0.3 * rng.standard_normal((cfg.vocab, cfg.hidden))}
    W_fp, state = [], []
    for l in range(cfg.n_layers):
        params[f"attn_norm.{l}"] = rng.uniform(0.8, 1.2, cfg.hidden)
        params[f"mlp_norm.{l}"] = rng.uniform(0.8, 1.2, cfg.hidden)
        Wl, Sl = {}, {}
        for name, (O, K) in cfg.linear_shapes().items():
            W = inputs.to_bf16_f32(inputs.weights(rng, O, K, sigma=0.25))
            scales, sg, code, V0 = fo.softquant_init(W)
            V = np.clip(V0.astype(np.float64) + 0.1 * rng.standard_normal(V0.shape), 0.02, 0.98)
            Wl[name], Sl[name] = W.astype(np.float64), (V, code, scales, sg)
        W_fp.append(Wl)
        state.append(Sl)
    tokens = rng.integers(0, cfg.vocab, (2, 5))
    return cfg, params, W_fp, state, tokens


def test_stage2_gradient_matches_finite_differences_of_eq6():
    cfg, params, W_fp, state, tokens = tiny_model(0)
    kw = dict(beta=6.0, tau=1.5, lambda_kl=0.7, lambda_round=0.9)
    total, (l_kl, l_mse, l_round), dV = so.stage2_loss_and_grads(cfg, params, W_fp, state, tokens, **kw)
    assert l_kl > 0 and l_mse > 0 and abs(total - (0.7 * l_kl + l_mse + 0.9 * l_round)) < 1e-12
    rng = np.random.default_rng(5)
    for l in range(cfg.n_layers):
        for name in so.LINEARS:
            V = state[l][name][0]
            for _ in range(2):
                idx = tuple(rng.integers(0, s) for s in V.shape)

                def loss_at(Vx, l=l, name=name):
                    st = [dict(s) for s in state]
                    st[l][name] = (Vx,) + state[l][name][1:]
                    return so.stage2_loss_and_grads(cfg, params, W_fp, st, tokens, **kw)[0]

                num = fd(loss_at, V, idx, eps=1e-6)
                assert abs(num - dV[l][name][idx]) <= 2e-6 * max(abs(num), np.abs(dV[l][name]).max() * 1e-2), (l, name, idx)


def test_stage2_gradient_matches_an_autograd_graph_written_with_torch_ops():
    """The same model written a second time, with PyTorch float64 ops (library norm, attention and softmax
    routines), Eq. 2 / Eq. 3 as tensor expressions of V, and the loss of Eq. 6; autograd supplies dL/dV."""
    cfg, params, W_fp, state, tokens = tiny_model(1)
    beta, tau, lam_kl, lam_r = 5.0, 2.0, 1.3, 0.4
    total, parts, dV = so.stage2_loss_and_grads(cfg, params, W_fp, state, tokens, beta, tau, lam_kl, lam_r)
    T = lambda a: torch.from_numpy(np.asarray(a, np.float64))
    B, S = tokens.shape
    pos = torch.arange(S, dtype=torch.float64).repeat(B)
    inv = cfg.theta ** (-torch.arange(0, cfg.head_dim, 2, dtype=torch.float64) / cfg.head_dim)
    ang = pos[:, None] * inv[None, :]
    cos, sin = torch.cat([ang.cos()] * 2, -1)[:, None, :], torch.cat([ang.sin()] * 2, -1)[:, None, :]

    def rope_t(x, n):
        xv = x.reshape(B * S, n, cfg.head_dim)
        rot = torch.cat([-xv[..., cfg.head_dim // 2:], xv[..., :cfg.head_dim // 2]], -1)
        return (xv * cos + rot * sin).reshape(B * S, -1)

    def run(weights):
        x = T(params["embed"])[torch.from_numpy(tokens.reshape(-1))]
        for l in range(cfg.n_layers):
            W = weights[l]
            hn = torch.nn.functional.rms_norm(x, (cfg.hidden,), T(params[f"attn_norm.{l}"]), cfg.eps)
            q, k, v = rope_t(hn @ W["q_proj"].T, cfg.n_heads), rope_t(hn @ W["k_proj"].T, cfg.n_kv_heads), hn @ W["v_proj"].T
            sh = lambda t, n: t.reshape(B, S, n, cfg.head_dim).transpose(1, 2)
            rep = cfg.n_heads // cfg.n_kv_heads
            a = torch.nn.functional.scaled_dot_product_attention(sh(q, cfg.n_heads), sh(k, cfg.n_kv_heads).repeat_interleave(rep, 1),
                                                                 sh(v, cfg.n_kv_heads).repeat_interleave(rep, 1), is_causal=True)
            x = x + a.transpose(1, 2).reshape(B * S, -1) @ W["o_proj"].T
            mn = torch.nn.functional.rms_norm(x, (cfg.hidden,), T(params[f"mlp_norm.{l}"]), cfg.eps)
            x = x + (torch.nn.functional.silu(mn @ W["gate_proj"].T) * (mn @ W["up_proj"].T)) @ W["down_proj"].T
        H = torch.nn.functional.rms_norm(x, (cfg.hidden,), T(params["final_norm"]), cfg.eps)
        return H @ T(params["lm_head"]).T, H

    Vt = [{n: T(state[l][n][0]).clone().requires_grad_(True) for n in so.LINEARS} for l in range(cfg.n_layers)]
    Wq = []
    for l in range(cfg.n_layers):
        d = {}
        for n in so.LINEARS:
            _, code, scales, sg = state[l][n]
            kk, neg = fo.unpack_code(code)
            s = T(np.repeat(fo.effective_scale(scales, sg), 16, axis=1))
            lo, hi = T(fo.NODES[kk]), T(fo.NODES[kk + 1])
            h = torch.sigmoid(beta * (Vt[l][n] - 0.5))
            d[n] = T(np.where(neg, -1.0, 1.0)) * (lo + h * (hi - lo)) * s
        Wq.append(d)
    with torch.no_grad():
        Z_fp, H_fp = run([{n: T(W_fp[l][n]) for n in so.LINEARS} for l in range(cfg.n_layers)])
    Z_q, H_q = run(Wq)
    kl = torch.nn.functional.kl_div(torch.log_softmax(Z_q / tau, -1), torch.softmax(Z_fp / tau, -1), reduction="sum") / (B * S)
    mse = ((H_fp - H_q) ** 2).sum()
    rl = sum(((1 - (2 * Vt[l][n] - 1) ** 2).sum() / Vt[l][n].numel()) for l in range(cfg.n_layers) for n in so.LINEARS)
    loss = lam_kl * kl + mse + lam_r * rl
    loss.backward()
    assert abs(float(loss.detach()) - total) <= 1e-10 * abs(total)
    assert abs(float(kl.detach()) - parts[0]) <= 1e-10 * parts[0] and abs(float(mse.detach()) - parts[1]) <= 1e-10 * parts[1]
    for l in range(cfg.n_layers):
        for n in so.LINEARS:
            g = Vt[l][n].grad.numpy()
            assert np.allclose(dV[l][n], g, rtol=1e-8, atol=1e-10 * np.abs(g).max()), (l, n)
