"""Pins for the CPU oracle: each test checks it against something the paper or
the mathematics fixes, never against itself."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from paper_2603_22370_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_pairs(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line.split())
    return out


def small_layer(seed=0, O=8, K=64, T=48):
    W, X = inputs.config1(seed, O, K, T)
    return W, X


# ---- I1: node table ("NVFP4 Overview") -----------------------------------

def test_nodes_match_paper():
    gold = np.array([float(r[0]) for r in _read_pairs("e2m1_nodes.txt")])
    assert np.array_equal(fo.NODES, gold)


def test_nodes_are_e2m1_bit_patterns():
    # E2M1: 2 exponent bits (bias 1), 1 mantissa bit, subnormal at e = 0.
    for c in range(8):
        e, m = c >> 1, c & 1
        val = m * 0.5 if e == 0 else (1 + m / 2) * 2.0 ** (e - 1)
        assert fo.NODES[c] == val


# ---- I2: E4M3 -------------------------------------------------------------

def test_e4m3_decode_golden():
    for hx, val in _read_pairs("e4m3_values.txt"):
        got = fo.e4m3_decode(int(hx, 16))
        assert got == float(val) and np.signbit(got) == (int(hx, 16) >= 0x80)
    assert np.isnan(fo.e4m3_decode(0x7F)) and np.isnan(fo.e4m3_decode(0xFF))


def test_e4m3_decode_matches_torch_float8():
    b = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    ref = b.view(torch.float8_e4m3fn).to(torch.float32).numpy()
    got = fo.e4m3_decode(np.arange(256))
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    ok = ~np.isnan(ref)
    assert np.array_equal(ref[ok].astype(np.float64), got[ok])


def test_e4m3_encode_roundtrip_monotone_midpoints():
    vals = fo.e4m3_decode(np.arange(0x7F))
    assert np.all(np.diff(vals) > 0)
    assert np.array_equal(fo.e4m3_encode(vals), np.arange(0x7F, dtype=np.uint8))
    mid = (vals[:-1] + vals[1:]) / 2
    enc = fo.e4m3_encode(mid)
    assert np.all(enc % 2 == 0)                              # ties to even mantissa
    assert np.all((enc == np.arange(0x7E)) | (enc == np.arange(1, 0x7F)))
    eps = np.minimum(1e-7, np.diff(vals) / 8)
    assert np.array_equal(fo.e4m3_encode(mid - eps), np.arange(0x7E, dtype=np.uint8))
    assert np.array_equal(fo.e4m3_encode(mid + eps), np.arange(1, 0x7F, dtype=np.uint8))
    # saturating, never NaN
    assert fo.e4m3_encode(np.array([448.0, 449.0, 464.0, 1e9, np.inf])).tolist() == [0x7E] * 5


def test_e4m3_encode_matches_torch_cast_in_range():
    rng = np.random.default_rng(1)
    q = np.concatenate([rng.uniform(0, 448, 20000), rng.uniform(0, 0.05, 20000),
                        np.exp(rng.uniform(np.log(1e-4), np.log(448), 20000))]).astype(np.float32)
    ref = torch.from_numpy(q).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(fo.e4m3_encode(q), ref)


def test_bf16_round_matches_torch_and_is_single_rounding():
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(50000) * np.exp(rng.uniform(-20, 20, 50000))).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(fo.bf16_round(x.astype(np.float64)).astype(np.float32), ref)
    # 1 + 2^-8 + 2^-30 lies above the midpoint of [1, 1+2^-7]: one rounding goes up,
    # rounding through binary32 first would land on the tie and go down to even.
    assert fo.bf16_round(1 + 2.0 ** -8 + 2.0 ** -30) == 1 + 2.0 ** -7
    assert fo.bf16_round(1 + 2.0 ** -8) == 1.0 and fo.bf16_round(1 + 3 * 2.0 ** -8) == 1 + 2.0 ** -6
    assert fo.bf16_round(0.0) == 0.0 and fo.bf16_round(-2.0 ** -133) == -2.0 ** -133


# ---- I3 / I4: scales and bracket -----------------------------------------

@pytest.mark.parametrize("seed", [0, 1, 2])
def test_scale_bound_and_bracket_invariants(seed):
    W, _ = inputs.config1(seed, 64, 256, 8)
    scales, sg = fo.compute_scales(W)
    assert sg == np.float32(np.abs(W).max()) / np.float32(2688.0)
    s = fo.effective_scale(scales, sg).astype(np.float64)
    amax_g = np.abs(W).reshape(64, 16, 16).max(axis=2).astype(np.float64)
    normal = scales >= 0x08
    # E4M3 RNE has relative error <= 2^-4 on normal numbers
    assert np.all(6 * s[normal] >= amax_g[normal] * (1 - 2.0 ** -4) * (1 - 1e-6))
    assert np.all(6 * s[normal] <= amax_g[normal] * (1 + 2.0 ** -4) * (1 + 1e-6))
    assert scales.max() <= 0x7E
    # the tensor-wide maximum maps to the top of the E4M3 range
    assert scales.max() == 0x7E
    k, neg, v = fo.bracket(W, scales, sg)
    sfull = np.repeat(s, 16, axis=1)
    wt = np.abs(W.astype(np.float64)) / sfull
    assert wt.max() <= 6 * (1 + 2.0 ** -4) * (1 + 1e-6)
    wtc = np.minimum(wt, 6.0)
    lo, hi = fo.NODES[k], fo.NODES[k + 1]
    assert np.all(lo <= wtc * (1 + 1e-6)) and np.all(wtc <= hi * (1 + 1e-6))
    assert set(np.unique(hi - lo)) <= {0.5, 1.0, 2.0}
    assert v.dtype == np.float32 and v.min() >= 0 and v.max() <= 1
    # Eq. 4 inverted: sign * (lo + v (hi - lo)) * s reproduces w unless clamped
    rec = np.where(neg, -1.0, 1.0) * (lo + v.astype(np.float64) * (hi - lo)) * sfull
    un = wt <= 6.0
    assert np.allclose(rec[un], W[un], rtol=3e-7, atol=1e-12)
    assert np.array_equal(neg, W < 0)


def test_bracket_exact_nodes_ties_clamp_zero_block_and_sign_of_zero():
    # one row, four blocks; s_global chosen so that every block scale is exactly 1.0 * s_global
    sgl = np.float32(2.0 ** -10)
    blk = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5, -6], dtype=np.float32)
    W = np.zeros((1, 64), dtype=np.float32)
    W[0, 0:16] = blk * sgl
    W[0, 16:32] = -blk * sgl
    W[0, 32:48] = 0.0                                   # all-zero block
    W[0, 48:64] = np.float32(6.0) * sgl
    W[0, 48] = -0.0
    scales, sg = fo.compute_scales(W, s_global_in=float(sgl))
    assert scales.tolist() == [[0x38, 0x38, 0x00, 0x38]]
    k, neg, v = fo.bracket(W, scales, sg)
    # a value on a node takes it as `lo` (v = 0); 6 is the closed end (k = 6, v = 1)
    assert k[0, :16].tolist() == [0, 1, 2, 3, 4, 5, 6, 6, 0, 1, 2, 3, 4, 5, 6, 6]
    assert v[0, :16].tolist() == [0, 0, 0, 0, 0, 0, 0, 1, .5, .5, .5, .5, .5, .5, .5, 1]
    assert neg[0, :16].tolist() == [False] * 15 + [True]
    assert neg[0, 16:32].tolist() == [False] + [True] * 14 + [False]      # -0.0 counts as +
    assert np.all(k[0, 32:48] == 0) and np.all(v[0, 32:48] == 0) and not neg[0, 32:48].any()
    assert not neg[0, 48]
    # ties harden upward (Eq. 7 uses >=)
    packed, vh, Wf = fo.harden_pack(v, fo.pack_code(k, neg), scales, sg)
    assert vh[0, 8:15].all()
    # w~ slightly above 6 after the block scale rounds down: clamp to the top node
    W2 = np.full((1, 16), 1.0, dtype=np.float32)
    W2[0, 0] = 1.06                                     # amax/6/s_global = 1.06 -> E4M3 1.0
    sc2, sg2 = fo.compute_scales(W2, s_global_in=1.0 / 6.0)
    k2, _, v2 = fo.bracket(W2, sc2, sg2)
    assert sc2[0, 0] == 0x38 and k2[0, 0] == 6 and v2[0, 0] == 1.0
    # all-zero tensor
    sc0, sg0 = fo.compute_scales(np.zeros((2, 16), np.float32))
    assert sg0 == 1.0 and not sc0.any()


# ---- I5: limits of Eq. 3 ---------------------------------------------------

def test_h_limits_and_floor_ceil():
    for beta in (0.5, 4.0, 32.0, 1e4):
        assert fo.h_beta(0.5, beta) == 0.5
    W, _ = small_layer()
    scales, sg, code, V = fo.softquant_init(W)
    k, neg = fo.unpack_code(code)
    s = np.repeat(fo.effective_scale(scales, sg), 16, axis=1).astype(np.float64)
    sgn = np.where(neg, -1.0, 1.0)
    Wlo, _ = fo.soft_weights(np.zeros_like(V), code, scales, sg, 80.0)
    Whi, _ = fo.soft_weights(np.ones_like(V), code, scales, sg, 80.0)
    assert np.allclose(Wlo, sgn * fo.NODES[k] * s, rtol=0, atol=1e-17)
    assert np.allclose(Whi, sgn * fo.NODES[k + 1] * s, rtol=1e-15, atol=1e-17)
    # beta -> infinity is a step function; no NaN on overflow
    h = fo.h_beta(np.array([0.0, 0.49, 0.51, 1.0]), 1e6)
    assert h.tolist() == [0.0, 0.0, 1.0, 1.0]
    # monotone in v, symmetric about 0.5
    v = np.linspace(0, 1, 101)
    hh = fo.h_beta(v, 7.0)
    assert np.all(np.diff(hh) > 0) and np.allclose(hh + hh[::-1], 1.0)


# ---- I6 / I7: hardening, packing -------------------------------------------

@pytest.mark.parametrize("seed", [0, 3])
def test_harden_vinit_is_rtn_and_pack_roundtrip(seed):
    W, _ = inputs.config1(seed, 32, 128, 8)
    scales, sg, code, V = fo.softquant_init(W)
    k, neg = fo.unpack_code(code)
    packed, vh, Wf = fo.harden_pack(V, code, scales, sg)
    mag_rtn = fo.rtn_nearest(W, scales, sg)
    nib = np.empty(W.shape, np.uint8)
    nib[:, 0::2], nib[:, 1::2] = packed & 0xF, packed >> 4
    assert np.array_equal(nib & 7, mag_rtn)
    assert np.array_equal(nib >> 3, (W < 0).astype(np.uint8))
    assert np.array_equal(fo.dequant_packed(packed, scales, sg).view(np.uint32), Wf.view(np.uint32))
    # RTN error is within half the local interval
    s = np.repeat(fo.effective_scale(scales, sg), 16, axis=1).astype(np.float64)
    wt = np.minimum(np.abs(W) / s, 6.0)
    assert np.all(np.abs(np.abs(Wf) / s - wt) <= (fo.NODES[k + 1] - fo.NODES[k]) / 2 + 1e-6)
    p0, _, _ = fo.harden_pack(np.zeros_like(V), code, scales, sg)
    p1, _, _ = fo.harden_pack(np.ones_like(V), code, scales, sg)
    assert np.array_equal(p0, code)
    assert np.array_equal(p1, code + 0x11)
    d = fo.pack_decisions(vh)
    assert d.shape == (32, 16) and ((d[0, 0] >> 3) & 1) == int(vh[0, 3])


def test_pack_decisions_every_bit_against_a_per_element_loop():
    """Element 8j+i of a row sits in bit i of byte j.  Checked on patterns whose neighbouring decisions
    differ (a single set element per byte position, an alternating row, a random matrix), element by
    element, so that a reversed bit order or a shifted byte index fails."""
    rng = np.random.default_rng(7)
    O, K = 5, 48
    pats = [rng.integers(0, 2, (O, K)).astype(bool), (np.arange(O * K).reshape(O, K) % 2 == 0),
            (np.arange(O * K).reshape(O, K) % 3 == 0)]
    for e in range(16):                                    # one decision alone, at every position of two bytes
        one = np.zeros((O, K), bool)
        one[e % O, e] = True
        pats.append(one)
    for vh in pats:
        d = fo.pack_decisions(vh)
        assert d.dtype == np.uint8 and d.shape == (O, K // 8)
        for o in range(O):
            for e in range(K):
                assert (int(d[o, e // 8]) >> (e % 8)) & 1 == int(vh[o, e]), (o, e)
    lone = np.zeros((1, 16), bool)
    lone[0, 1] = True                                      # element 1 -> bit 1 of byte 0: value 2, not 64
    assert fo.pack_decisions(lone).tolist() == [[2, 0]]
    lone[:] = False
    lone[0, 15] = True                                     # element 15 -> bit 7 of byte 1
    assert fo.pack_decisions(lone).tolist() == [[0, 128]]


# ---- I8: finite differences of Eq. 5 ---------------------------------------

@pytest.mark.parametrize("opt_beta,lam,c", [(4.0, 1.0, 1.0), (11.0, 0.3, 0.01), (32.0, 5.0, 1.0)])
def test_dv_matches_finite_differences(opt_beta, lam, c):
    W, X = small_layer(5, 6, 32, 40)
    scales, sg, code, V0 = fo.softquant_init(W)
    Yref = fo.layer_ref(X, W)
    rng = np.random.default_rng(0)
    V = rng.uniform(0.05, 0.95, V0.shape)

    def loss(Vx):
        l, _, _ = fo.layer_fwd(X, Yref, Vx, code, scales, sg, opt_beta, c, mode="smooth")
        return l + lam * fo.round_loss(Vx)

    _, dY, _ = fo.layer_fwd(X, Yref, V, code, scales, sg, opt_beta, c, mode="smooth")
    dV, _ = fo.layer_grad(dY, X, V, code, scales, sg, opt_beta, lam)
    idx = rng.choice(V.size, 64, replace=False)
    eps = 1e-6
    for i in idx:
        o, kk = divmod(int(i), V.shape[1])
        Vp, Vm = V.copy(), V.copy()
        Vp[o, kk] += eps
        Vm[o, kk] -= eps
        fd = (loss(Vp) - loss(Vm)) / (2 * eps)
        assert abs(fd - dV[o, kk]) <= 1e-6 * max(abs(dV[o, kk]), np.abs(dV).max() * 1e-3), (o, kk, fd, dV[o, kk])


# ---- I9: Round Loss closed forms -------------------------------------------

def test_round_loss_closed_forms():
    rng = np.random.default_rng(0)
    assert fo.round_loss(rng.integers(0, 2, (7, 32)).astype(float)) == 0.0
    assert fo.round_loss(np.full((3, 16), 0.5)) == 1.0
    n = 100001
    grid = np.linspace(0, 1, n).reshape(1, n)
    # (1/N) sum 4v(1-v) on a fine uniform grid tends to the integral of 4v(1-v) over [0,1] = 2/3
    assert abs(fo.round_loss(grid) - 2 / 3) < 1e-4
    assert abs(fo.round_loss(np.array([[0.25, 0.75]])) - 0.75) < 1e-15
    # its gradient is (4 - 8v)/N: isolate it with a zero data term
    V = rng.uniform(0, 1, (4, 16))
    code = np.zeros((4, 8), np.uint8)
    scales = np.zeros((4, 1), np.uint8)                   # s = 0 -> no data gradient
    dV, _ = fo.layer_grad(np.zeros((5, 4)), np.zeros((5, 16)), V, code, scales, 1.0, 4.0, 2.5)
    assert np.allclose(dV, 2.5 / 64 * (4 - 8 * V), rtol=1e-15)


# ---- I10: optimiser closed forms -------------------------------------------

def test_adam_first_step_and_clip():
    g = np.array([3.0, -0.2, 1e-3, -7.0, 0.0])
    V = np.array([0.5, 0.5, 0.5, 0.995, 0.3])
    Vn, m, u = fo.adam_update(V, g, np.zeros(5), np.zeros(5), 1e-2, 0.9, 0.999, 1e-8, 1)
    expect = np.clip(V - 1e-2 * g / (np.abs(g) + 1e-8), 0, 1)
    assert np.allclose(Vn, expect, rtol=1e-12)
    assert Vn[3] == 1.0 and Vn[4] == 0.3
    assert np.allclose(m, 0.1 * g) and np.allclose(u, 0.001 * g * g)
    # constant gradient: every bias-corrected step moves by lr
    Vc, m, u = np.array([0.9]), np.zeros(1), np.zeros(1)
    for t in range(1, 6):
        Vc, m, u = fo.adam_update(Vc, np.array([2.0]), m, u, 1e-2, 0.9, 0.999, 0.0, t)
    assert np.allclose(Vc, 0.85)
    assert fo.sgd_update(np.array([0.1, 0.9]), np.array([50.0, -50.0]), 0.01).tolist() == [0.0, 1.0]


def test_sgd_step_is_v_minus_lr_times_g_then_clip():
    """Plain gradient descent on values the clip does not touch: the step is exactly lr * g, downhill;
    halving lr halves it; a quadratic's minimiser is reached in one step of lr = 1 / curvature."""
    V = np.array([[0.25, 0.5, 0.75, 0.4]])
    g = np.array([[2.0, -3.0, 0.5, 0.0]])
    out = fo.sgd_update(V, g, 0.0625)                      # power-of-two lr: the products are exact
    assert out.tolist() == [[0.125, 0.6875, 0.71875, 0.4]]
    assert np.array_equal(V - fo.sgd_update(V, g, 0.03125), 0.5 * (V - out))
    # f(v) = 2 (v - 0.3)^2 has f' = 4 (v - 0.3): lr = 1/4 lands on the minimiser from anywhere inside [0, 1]
    v0 = np.array([0.9, 0.1, 0.3])
    assert np.allclose(fo.sgd_update(v0, 4.0 * (v0 - 0.3), 0.25), 0.3, rtol=0, atol=1e-16)
    # clip at both ends, and only there
    assert fo.sgd_update(np.array([0.02, 0.98, 0.5]), np.array([1.0, -1.0, 1.0]), 0.05).tolist() == [0.0, 1.0, 0.45]


# ---- I11: exhaustive search on a tiny layer (Eq. 1) -------------------------

@pytest.mark.parametrize("seed", [0, 1, 2])
def test_brute_force_4x16(seed):
    W, X = inputs.config1(seed, 4, 16, 64)
    scales, sg, code, V0 = fo.softquant_init(W)
    Yref = fo.layer_ref(X, W)
    k, neg = fo.unpack_code(code)
    s = np.repeat(fo.effective_scale(scales, sg), 16, axis=1).astype(np.float64)
    sgn = np.where(neg, -1.0, 1.0)
    bits = ((np.arange(1 << 16)[:, None] >> np.arange(16)[None, :]) & 1).astype(np.float64)   # [65536,16]
    Xd = X.astype(np.float64)

    def hard_loss(vh):
        Wq = sgn * (fo.NODES[k] + vh * (fo.NODES[k + 1] - fo.NODES[k])) * s
        return np.sum((Xd @ Wq.T - Yref) ** 2, axis=0)                                       # per output row

    # the loss separates over output rows, so 4 * 2^16 evaluations cover all 2^64 assignments
    l_opt = np.empty(4)
    for o in range(4):
        cand = sgn[o] * (fo.NODES[k[o]] + bits * (fo.NODES[k[o] + 1] - fo.NODES[k[o]])) * s[o]   # [65536,16]
        l_opt[o] = np.min(np.sum((Xd @ cand.T - Yref[:, o:o + 1]) ** 2, axis=0))
    l_rtn = hard_loss(fo.harden(V0).astype(np.float64))
    res = fo.run_layer(X, Yref, W, steps=150, lr=1e-2, mode="smooth")
    l_faar = hard_loss(fo.harden(res["V"]).astype(np.float64))
    assert np.all(l_opt <= l_rtn * (1 + 1e-12))
    assert np.all(l_faar >= l_opt * (1 - 1e-12))
    # hardening the soft solution matches evaluating Eq. 2 with a step function
    _, _, Wf = fo.harden_pack(res["V"], code, scales, sg)
    assert np.allclose(np.sum((Xd @ Wf.astype(np.float64).T - Yref) ** 2, axis=0), l_faar, rtol=1e-5)
    # the optimiser does reduce the soft objective it is given
    first, last = sum(res["hist"][0][:1]) + res["hist"][0][1], res["hist"][-1][0] + res["hist"][-1][1]
    assert last < first


# ---- I12: textbook GEMM special case ---------------------------------------

def test_forward_reduces_to_naive_matmul_on_hard_weights():
    W, X = small_layer(7, 5, 32, 9)
    scales, sg, code, V0 = fo.softquant_init(W)
    rng = np.random.default_rng(0)
    Vh = rng.integers(0, 2, V0.shape).astype(np.float64)
    _, _, Wf = fo.harden_pack(Vh, code, scales, sg)
    Yq_naive = np.zeros((9, 5))
    for t, o, kk in itertools.product(range(9), range(5), range(32)):
        Yq_naive[t, o] += float(X[t, kk]) * float(Wf[o, kk])
    loss, dY, Yq = fo.layer_fwd(X, np.zeros((9, 5)), Vh, code, scales, sg, 200.0, 1.0, mode="smooth")
    assert np.allclose(Yq, Yq_naive, rtol=1e-6, atol=1e-9)
    assert np.isclose(loss, np.sum(Yq_naive ** 2), rtol=1e-6)
    assert np.allclose(dY, 2 * Yq_naive, rtol=1e-6, atol=1e-9)
    # gradient GEMM against a naive loop
    _, G = fo.layer_grad(dY, X, Vh, code, scales, sg, 4.0, 0.0)
    Gn = np.zeros((5, 32))
    for t, o, kk in itertools.product(range(9), range(5), range(32)):
        Gn[o, kk] += dY[t, o] * float(X[t, kk])
    assert np.allclose(G, Gn, rtol=1e-12, atol=1e-12)


# ---- I13: zero-residual fixed point ----------------------------------------

def test_zero_residual_leaves_only_round_term():
    W, X = small_layer(9, 6, 32, 20)
    scales, sg, code, V0 = fo.softquant_init(W)
    rng = np.random.default_rng(0)
    V = rng.uniform(0.02, 0.98, V0.shape)
    Wsoft, _ = fo.soft_weights(V, code, scales, sg, 6.0)
    Yref = X.astype(np.float64) @ Wsoft.T
    hp = fo.HParams(beta=6.0, lambda_round=2.0, opt=0, lr=0.5)
    Vn, _, _, l_mse, l_round, dV = fo.layer_step(X, Yref, V, code, scales, sg, None, None, hp, mode="smooth")
    assert l_mse < 1e-20
    assert np.allclose(dV, 2.0 / V.size * (4 - 8 * V), rtol=1e-9, atol=1e-15)
    # the round term pushes each v toward the nearer of {0, 1}
    away = V != 0.5
    assert np.all(np.abs(Vn[away] - 0.5) > np.abs(V[away] - 0.5))


# ---- rounding points of mode "bf16" ----------------------------------------

def test_bf16_mode_rounds_only_at_the_stated_points():
    W, X = inputs.config2(0, 16, 64, 32)
    scales, sg, code, V = fo.softquant_init(W)
    Yref = inputs.to_bf16_f32(fo.layer_ref(X, W))
    l_b, dY_b, Yq_b = fo.layer_fwd(X, Yref, V, code, scales, sg, 4.0, 1.0, mode="bf16")
    Ws, _ = fo.soft_weights(V, code, scales, sg, 4.0)
    Wb = torch.from_numpy(Ws.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    # (binary32 then BF16 may differ from one rounding only on exact ties; none occur here)
    assert np.array_equal(Wb, fo.bf16_round(Ws))
    assert np.array_equal(Yq_b, X.astype(np.float64) @ Wb.T)
    assert np.array_equal(dY_b, fo.bf16_round(2 * (Yq_b - Yref)))
    Vn, m, u, *_ = fo.layer_step(X, Yref, V, code, scales, sg, np.zeros_like(V), np.zeros_like(V), fo.HParams(), "bf16")
    assert Vn.dtype == np.float32 and m.dtype == np.float32 and u.dtype == np.float32


# ---------------------------------------------------------------------------------------------
# activation fake-quantisation (the X_q of Eq. 5)
# ---------------------------------------------------------------------------------------------

def test_act_fake_quant_is_nearest_node_and_fits_bf16():
    import torch
    rng = np.random.default_rng(5)
    X = (rng.standard_t(4, size=(24, 64)) * np.where(rng.random(64) < 0.1, 20.0, 1.0)).astype(np.float32)
    X[0, :16] = 0.0                                   # an all-zero block
    X[1, 0] = -0.0
    units, sg, packed, scales = fo.act_fake_quant(X)
    # every value is sign * node * block scale, and those products need at most 7 significant bits
    assert np.array_equal(torch.from_numpy(units.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy(), units)
    # independent nearest-node search (ties to the larger node) gives the same magnitude codes
    codes = fo.rtn_nearest(X, scales, sg)
    k_mag, neg = fo.unpack_code(packed)
    assert np.array_equal(k_mag, codes)
    assert np.array_equal(neg, np.signbit(X) & (X != 0))
    # dequantised NVFP4 == units * s_global (up to the one binary32 rounding of the product)
    deq = fo.dequant_packed(packed, scales, sg).astype(np.float64)
    assert np.all(np.abs(deq - units * float(sg)) <= 2.0 ** -23 * np.abs(deq))
    # quantisation error of an in-range value is at most half the local node spacing (times the scale)
    s = np.repeat(fo.effective_scale(scales, sg), 16, axis=1).astype(np.float64)
    ok = s > 0
    err = np.abs(np.abs(X.astype(np.float64)) - np.abs(units) * float(sg))[ok] / s[ok]
    assert err.max() <= 1.0 + 1e-6                   # widest interval [4, 6]: half of 2


def test_act_fake_quant_exact_on_representable_inputs():
    # inputs that are already node * 2^e with block maximum 6 * 2^e survive unchanged
    nodes = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6, -0.5, -1, -1.5, -2, -3, -4, -6, 6], dtype=np.float32)
    X = np.stack([nodes * 2.0 ** e for e in (-3, 0, 2)]).astype(np.float32)
    units, sg, _, scales = fo.act_fake_quant(X, s_global_in=2.0 ** -3)
    assert np.array_equal((units * float(sg)).astype(np.float32), X)


def test_swizzled_scale_layout_is_a_padded_permutation():
    rng = np.random.default_rng(0)
    for rows, cols in [(128, 4), (130, 5), (300, 65), (1, 1)]:
        sc = rng.integers(1, 0x7F, size=(rows, cols)).astype(np.uint8)
        sw = fo.swizzle_scales(sc)
        rt, ct = -(-rows // 128), -(-cols // 4)
        assert sw.size == rt * ct * 512
        # the same bytes, every one exactly once, the rest padding
        assert np.array_equal(np.sort(sw[sw != 0]), np.sort(sc.ravel()))
        # reshape route: [row tile][col tile][r % 32][r // 32][c] is the padded matrix re-indexed
        padded = np.zeros((rt * 128, ct * 4), np.uint8)
        padded[:rows, :cols] = sc
        view = sw.reshape(rt, ct, 32, 4, 4)                     # tile, r % 32, r // 32, c
        back = view.transpose(0, 3, 2, 1, 4).reshape(rt * 128, ct * 4)   # rows = (rt, r // 32, r % 32)
        assert np.array_equal(back, padded)
    # the first 16 bytes of a tile: rows 0, 32, 64, 96 of its four columns
    sc = np.arange(128 * 4, dtype=np.uint8).reshape(128, 4)
    assert list(fo.swizzle_scales(sc)[:16]) == [sc[r, c] for r in (0, 32, 64, 96) for c in range(4)]


def test_layer_dx_matches_finite_differences_of_the_mse_term():
    rng = np.random.default_rng(11)
    W = (0.02 * rng.standard_normal((6, 32))).astype(np.float32)
    X = rng.standard_normal((5, 32))
    scales, sg, code, V = fo.softquant_init(W)
    V = rng.uniform(0, 1, V.shape)
    Yref = fo.layer_ref(X, W)
    beta, c = 6.0, 0.7
    _, dY, _ = fo.layer_fwd(X, Yref, V, code, scales, sg, beta, c, "smooth")
    dX = fo.layer_dx(dY, V, code, scales, sg, beta, "smooth")
    eps = 1e-6
    for (t, k) in [(0, 0), (4, 31), (2, 17), (3, 5)]:
        Xp, Xm = X.copy(), X.copy()
        Xp[t, k] += eps
        Xm[t, k] -= eps
        lp, _, _ = fo.layer_fwd(Xp, Yref, V, code, scales, sg, beta, c, "smooth")
        lm, _, _ = fo.layer_fwd(Xm, Yref, V, code, scales, sg, beta, c, "smooth")
        fd = (lp - lm) / (2 * eps)
        assert abs(fd - dX[t, k]) <= 1e-6 * max(abs(dX[t, k]), 1e-6) + 1e-9
    # transposed operand or a missing factor would show here: dX has X's shape and scales with dY
    assert dX.shape == X.shape
    assert np.allclose(fo.layer_dx(2 * dY, V, code, scales, sg, beta, "smooth"), 2 * dX)


# ---- full-model alignment loss (Eq. 6, Procedure steps 18-20) ---------------------------------

def test_align_loss_closed_forms():
    rng = np.random.default_rng(0)
    T, V, D = 5, 37, 8
    Zf, Zq = rng.standard_normal((T, V)) * 3, rng.standard_normal((T, V)) * 3
    Hf, Hq = rng.standard_normal((T, D)), rng.standard_normal((T, D))
    # identical models: no divergence, no gradient
    kl, mse, dZ, dH = fo.align_loss(Zf, Zf, Hf, Hf)
    assert kl == 0.0 and mse == 0.0 and not dZ.any() and not dH.any()
    # Gibbs: KL > 0 for different distributions; each token's gradient sums to zero over the vocabulary
    kl, mse, dZ, dH = fo.align_loss(Zf, Zq, Hf, Hq, tau=1.7, lambda_kl=0.3)
    assert kl > 0 and np.all(np.abs(dZ.sum(axis=1)) < 1e-15)
    assert abs(mse - np.sum((Hf - Hq) ** 2)) < 1e-12 and np.allclose(dH, 2 * (Hq - Hf), rtol=0, atol=1e-15)
    # softmax ignores a per-token shift of the logits
    kl2, _, dZ2, _ = fo.align_loss(Zf + rng.standard_normal((T, 1)) * 50, Zq - 7.0, Hf, Hq, tau=1.7, lambda_kl=0.3)
    assert abs(kl2 - kl) < 1e-12 and np.max(np.abs(dZ2 - dZ)) < 1e-15
    # the temperature divides the logits: (tau Z, tau) is (Z, 1) up to the 1/tau of the gradient
    kl3, _, dZ3, _ = fo.align_loss(1.7 * Zf, 1.7 * Zq, Hf, Hq, tau=1.7, lambda_kl=0.3)
    kl4, _, dZ4, _ = fo.align_loss(Zf, Zq, Hf, Hq, tau=1.0, lambda_kl=0.3)
    assert abs(kl3 - kl4) < 1e-12 and np.max(np.abs(dZ3 * 1.7 - dZ4)) < 1e-15
    # two classes: KL of two Bernoulli distributions with p = sigmoid(a / tau), q = sigmoid(b / tau)
    a, b, tau = 1.3, -0.4, 0.8
    p, q = 1 / (1 + np.exp(-a / tau)), 1 / (1 + np.exp(-b / tau))
    kl5, _, dZ5, _ = fo.align_loss(np.array([[a, 0.0]]), np.array([[b, 0.0]]), Hf[:1], Hf[:1], tau=tau)
    assert abs(kl5 - (p * np.log(p / q) + (1 - p) * np.log((1 - p) / (1 - q)))) < 1e-14
    assert abs(dZ5[0, 0] - (q - p) / tau) < 1e-15
    # uniform quantised model: KL = log V - entropy(P_fp), averaged over the tokens
    pf = np.exp(Zf - Zf.max(1, keepdims=True)); pf /= pf.sum(1, keepdims=True)
    ent = -(pf * np.log(pf)).sum(1)
    kl6, *_ = fo.align_loss(Zf, np.zeros_like(Zf), Hf, Hf)
    assert abs(kl6 - np.mean(np.log(V) - ent)) < 1e-12
    # logits far apart do not overflow
    kl7, _, dZ7, _ = fo.align_loss(np.array([[800.0, 0.0, -800.0]]), np.array([[0.0, 0.0, 0.0]]), Hf[:1], Hf[:1])
    assert np.isfinite(kl7) and abs(kl7 - np.log(3)) < 1e-12 and np.all(np.isfinite(dZ7))


def test_align_loss_gradients_match_finite_differences():
    rng = np.random.default_rng(1)
    T, V, D = 4, 23, 6
    Zf, Zq = rng.standard_normal((T, V)) * 2, rng.standard_normal((T, V)) * 2
    Hf, Hq = rng.standard_normal((T, D)), rng.standard_normal((T, D))
    tau, lam = 1.3, 0.7
    _, _, dZ, dH = fo.align_loss(Zf, Zq, Hf, Hq, tau, lam)
    eps = 1e-6
    for _ in range(40):
        t, v = rng.integers(T), rng.integers(V)
        Zp, Zm = Zq.copy(), Zq.copy()
        Zp[t, v] += eps; Zm[t, v] -= eps
        fd = lam * (fo.align_loss(Zf, Zp, Hf, Hq, tau, lam)[0] - fo.align_loss(Zf, Zm, Hf, Hq, tau, lam)[0]) / (2 * eps)
        assert abs(fd - dZ[t, v]) <= 1e-8 + 1e-6 * abs(dZ[t, v])
    for _ in range(10):
        t, d = rng.integers(T), rng.integers(D)
        Hp, Hm = Hq.copy(), Hq.copy()
        Hp[t, d] += eps; Hm[t, d] -= eps
        fd = (fo.align_loss(Zf, Zq, Hf, Hp, tau, lam)[1] - fo.align_loss(Zf, Zq, Hf, Hm, tau, lam)[1]) / (2 * eps)
        assert abs(fd - dH[t, d]) <= 1e-7


def test_silu_mul_closed_forms_and_library_routine():
    x = np.array([-30.0, -2.0, -0.5, 0.0, 0.5, 2.0, 30.0, 800.0, -800.0])
    one = np.ones_like(x)
    y = fo.silu_mul(x, one)
    assert y[3] == 0.0 and abs(y[6] - 30.0) < 1e-11 and y[7] == 800.0 and y[8] == 0.0
    assert np.allclose(y[:7] - fo.silu_mul(-x[:7], one[:7]), x[:7], rtol=0, atol=1e-14)      # silu(x) - silu(-x) = x
    assert abs(fo.silu_mul(np.array([1.0]), np.array([1.0]))[0] - 1.0 / (1.0 + np.exp(-1.0))) < 1e-16
    rng = np.random.default_rng(3)
    g, u = rng.standard_normal((17, 33)) * 4, rng.standard_normal((17, 33))
    ref = torch.nn.functional.silu(torch.from_numpy(g)) * torch.from_numpy(u)
    assert np.allclose(fo.silu_mul(g, u), ref.numpy(), rtol=1e-14, atol=1e-300)
    # the second argument multiplies, the first is gated (not the other way round)
    assert fo.silu_mul(np.array([0.0]), np.array([5.0]))[0] == 0.0 and fo.silu_mul(np.array([5.0]), np.array([0.0]))[0] == 0.0
    assert abs(fo.silu_mul(np.array([2.0]), np.array([3.0]))[0] - 3.0 * 2.0 / (1.0 + np.exp(-2.0))) < 1e-15


def test_nvfp4_matmul_against_a_hand_decoded_triple_loop():
    """Decode by hand from the format definitions (nibble order, E2M1 magnitudes, E4M3 bytes through torch's
    float8 type) and multiply with plain loops; also the defining special case: all block scales 1.0 (byte 0x38),
    tensor scales 1 -> an integer-valued product of node values."""
    rng = np.random.default_rng(11)
    M, N, K = 3, 2, 32
    nodes = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    e4m3 = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float64).tolist()   # the library's decode
    Ap, Bp = rng.integers(0, 256, (M, K // 2), dtype=np.uint8), rng.integers(0, 256, (N, K // 2), dtype=np.uint8)
    As, Bs = rng.integers(0x20, 0x50, (M, K // 16), dtype=np.uint8), rng.integers(0x20, 0x50, (N, K // 16), dtype=np.uint8)
    sa, sb = np.float32(0.75), np.float32(1.25)

    def elem(P, S, sg, r, k):
        nib = (int(P[r, k // 2]) >> (4 * (k % 2))) & 0xF
        mag = nodes[nib & 7] * e4m3[int(S[r, k // 16])] * float(sg)
        return -mag if nib & 8 else mag

    ref = np.zeros((M, N))
    for i in range(M):
        for j in range(N):
            for k in range(K):
                ref[i, j] += elem(Ap, As, sa, i, k) * elem(Bp, Bs, sb, j, k)
    got = fo.nvfp4_matmul(Ap, As, sa, Bp, Bs, sb)
    assert np.allclose(got, ref, rtol=1e-6, atol=1e-9)
    ones = np.full((M, K // 16), 0x38, np.uint8)
    got1 = fo.nvfp4_matmul(Ap, ones, 1.0, Bp, np.full((N, K // 16), 0x38, np.uint8), 1.0)
    assert np.array_equal(got1 * 4, np.round(got1 * 4))           # products of half-integers
    # transposed operands give the transposed product (A rows index the output's rows)
    assert np.allclose(fo.nvfp4_matmul(Bp, Bs, sb, Ap, As, sa), got.T, rtol=1e-12)
