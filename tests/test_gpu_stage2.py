"""One full-model alignment step (Eq. 6) on the GPU against the Stage-2 oracle, on a small two-block model with
grouped key/value heads: the frozen and the quantised forward passes, the two data terms of the loss, the gradient
towards every one of the 14 rounding tensors, and the state after the update.  Activations are stored in BF16
between the library's calls (the oracle keeps float64), so tensors are compared norm-wise."""
import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from oracle import stage2_oracle as so
from paper_2603_22370_b200 import faar, inputs, stage2
from tests.gpu_helpers import DEV, dev_bf16, dev_f32, host, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2603_22370_b200 import build
    build.build()
    c = faar.Context(0)
    yield c
    torch.cuda.synchronize()
    c.close()


def small_model(seed=0):
    cfg = dict(vocab=512, hidden=128, n_layers=2, n_heads=2, n_kv_heads=1, head_dim=64, ffn=256)
    rng = np.random.default_rng(seed)
    bf = inputs.to_bf16_f32
    params = {"embed": bf(rng.standard_normal((cfg["vocab"], cfg["hidden"]))),
              "final_norm": bf(rng.uniform(0.8, 1.2, cfg["hidden"])),
              "lm_head": bf(0.2 * rng.standard_normal((cfg["vocab"], cfg["hidden"])))}
    ocfg = so.ModelCfg(**cfg)
    W_fp, state = [], []
    for l in range(cfg["n_layers"]):
        params[f"attn_norm.{l}"] = bf(rng.uniform(0.8, 1.2, cfg["hidden"]))
        params[f"mlp_norm.{l}"] = bf(rng.uniform(0.8, 1.2, cfg["hidden"]))
        Wl, Sl = {}, {}
        for name, (O, K) in ocfg.linear_shapes().items():
            W = bf(inputs.weights(rng, O, K, sigma=1.0 / np.sqrt(K)))
            scales, sg, code, V0 = fo.softquant_init(W)
            V = np.clip(V0 + 0.1 * rng.standard_normal(V0.shape), 0.02, 0.98).astype(np.float32)
            Wl[name], Sl[name] = W, (V, code, scales, sg)
        W_fp.append(Wl)
        state.append(Sl)
    tokens = rng.integers(0, cfg["vocab"], (2, 96))
    return cfg, ocfg, params, W_fp, state, tokens


def test_stage2_step_matches_the_oracle(ctx):
    cfg, ocfg, params, W_fp, state, tokens = small_model(0)
    B, S = tokens.shape
    dparams = {k: (dev_bf16(v) if k in ("embed", "lm_head") else dev_f32(v)) for k, v in params.items()}
    dweights = [{n: dev_bf16(W_fp[l][n]) for n in so.LINEARS} for l in range(cfg["n_layers"])]
    model = stage2.Stage2Model(ctx, stage2.ModelConfig(**cfg), dparams, dweights, B, S)
    for l in range(cfg["n_layers"]):
        for n in so.LINEARS:
            lin = model.lin[l][n]
            V, code, scales, sg = state[l][n]
            assert np.array_equal(host(lin.code), code) and np.array_equal(host(lin.scales), scales)   # same bracket
            lin.V.copy_(dev_f32(V))
    tok = torch.from_numpy(tokens.reshape(-1).astype(np.int32)).to(DEV)
    beta, tau, lam_kl, lam_r, lr = 6.0, 1.5, 0.7, 0.9, 5e-4
    # ---- forward passes
    Zf, Hf, _ = model.forward(tok, quantised=False)
    Zf_o, Hf_o, _ = so.forward(ocfg, params, W_fp, tokens)
    assert rel_l2(host(Zf), Zf_o) <= 1.5e-2 and rel_l2(host(Hf), Hf_o) <= 1.5e-2
    # ---- the step, with the gradients returned
    res = model.step(tok, beta, tau, lam_kl, lam_r, lr, want_dv=True, fp_outputs=(Zf, Hf))
    Zq, Hq, grads = res["Z_q"], res["H_q"], res["dV"]
    faar.check_status(ctx, model.ws)
    total_o, (l_kl_o, l_mse_o, l_round_o), dV_o = so.stage2_loss_and_grads(ocfg, params, W_fp, state, tokens, beta, tau,
                                                                           lam_kl, lam_r)
    Wq_o = so.quantised_weights(state, beta)
    Zq_o, Hq_o, saved = so.forward(ocfg, params, Wq_o, tokens, keep=True)
    assert rel_l2(host(Zq), Zq_o) <= 1.5e-2 and rel_l2(host(Hq), Hq_o) <= 1.5e-2
    loss = host(model.loss)
    print("L_KL gpu / oracle:", loss[0], l_kl_o, " L_MSE:", loss[1], l_mse_o)
    # The data terms are differences of two nearly equal forward passes: the BF16 storage of Z and H (2^-9 of each
    # pass) is a much larger share of their difference, in the loss values and in the loss gradients alike.
    assert abs(loss[0] - l_kl_o) <= 0.15 * l_kl_o and abs(loss[1] - l_mse_o) <= 0.15 * l_mse_o
    l_round_g = model.round_loss_sum()          # after the update: V has moved by at most lr
    assert abs(l_round_g - l_round_o) <= 4 * lr * 14 + 1e-3 * l_round_o
    # (a) the backward pass on its own: the oracle back-propagates the GPU's own loss gradients
    G = so.backward(ocfg, params, Wq_o, host(res["dZ"]).astype(np.float64), host(res["dH"]).astype(np.float64), saved)
    # (b) the whole step against the oracle's own gradients (looser: the seed noise explained above)
    worst_a, worst_b = 0.0, 0.0
    for l in range(cfg["n_layers"]):
        for n in so.LINEARS:
            V, code, scales, sg = state[l][n]
            Vd = V.astype(np.float64)
            ref_a = G[l][n] * fo.chain_factor(Vd, code, scales, sg, beta) + (lam_r / Vd.size) * (4.0 - 8.0 * Vd)
            g = host(grads[(l, n)]).astype(np.float64)
            ea, eb = rel_l2(g, ref_a), rel_l2(g, dV_o[l][n])
            worst_a, worst_b = max(worst_a, ea), max(worst_b, eb)
            assert ea <= 4e-2, (l, n, ea)
            assert eb <= 0.25, (l, n, eb)
            big = np.abs(dV_o[l][n]) > 0.3 * np.abs(dV_o[l][n]).max()
            assert np.mean(np.sign(g[big]) == np.sign(dV_o[l][n][big])) >= 0.97, (l, n)
    print("worst relative dV error over the 14 linears: backward alone %.3g, whole step %.3g" % (worst_a, worst_b))
    # ---- state after the update: Adam's first step is lr * sign-like; V stays in [0, 1]
    for l in range(cfg["n_layers"]):
        for n in so.LINEARS:
            V0 = state[l][n][0]
            Vn = host(model.lin[l][n].V)
            assert Vn.min() >= 0.0 and Vn.max() <= 1.0
            assert np.max(np.abs(Vn - V0)) <= lr * 1.001 + 1e-7
            moved = np.abs(dV_o[l][n]) > 0.3 * np.abs(dV_o[l][n]).max()
            assert np.mean(np.sign(V0 - Vn)[moved] == np.sign(dV_o[l][n])[moved]) >= 0.97


def test_stage2_steps_reduce_the_alignment_loss(ctx):
    cfg, ocfg, params, W_fp, state, tokens = small_model(1)
    B, S = tokens.shape
    dparams = {k: (dev_bf16(v) if k in ("embed", "lm_head") else dev_f32(v)) for k, v in params.items()}
    dweights = [{n: dev_bf16(W_fp[l][n]) for n in so.LINEARS} for l in range(cfg["n_layers"])]
    model = stage2.Stage2Model(ctx, stage2.ModelConfig(**cfg), dparams, dweights, B, S)
    tok = torch.from_numpy(tokens.reshape(-1).astype(np.int32)).to(DEV)
    fp = model.forward(tok, quantised=False)[:2]
    hist = []
    for t in range(30):
        model.step(tok, beta=4.0 + t * 0.5, lr=5e-3, lambda_round=0.1, fp_outputs=fp)
        hist.append(host(model.loss).copy())
    faar.check_status(ctx, model.ws)
    hist = np.array(hist)
    print("L_KL, L_MSE first -> last:", hist[0], hist[-1])
    assert hist[-1, 1] < 0.8 * hist[0, 1] and hist[-1, 0] < hist[0, 0]
    packed = model.harden()
    for l in range(cfg["n_layers"]):
        for n in so.LINEARS:
            lin = model.lin[l][n]
            p_o, _, _ = fo.harden_pack(host(lin.V), host(lin.code), host(lin.scales), host(lin.s_global)[0])
            assert np.array_equal(host(packed[l][n]), p_o)
