"""CPU oracle for one FAAR layer-wise rounding-optimisation step (NVFP4).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may import it; the product path never does, and it
imports nothing from the product path.  It shares no code, table or constant
generator with the CUDA sources.

Everything is numpy.  Floating point is float64 except where a precision is
part of the method's contract:

* the scale / bracket / V_init path ("NVFP4 Overview", Procedure steps 2-4,
  Eq. 4) is evaluated in IEEE binary32, one correctly rounded operation at a
  time in a fixed order, because its outputs are bytes (E4M3 scales, E2M1
  codes) that must agree bit for bit with any other implementation;
* in mode "bf16" the tensors that a mixed-precision implementation stores in
  BF16 / FP32 are rounded at exactly those points (W_soft -> BF16, dY -> BF16,
  V / Adam moments -> FP32); dot products and loss sums stay float64.
  Mode "smooth" rounds nothing and is what the finite-difference and
  brute-force pins use.

Parity pins (tests/test_oracle_pins.py): node table, E4M3 format, bracket
invariants, beta-limits of Eq. 3, RTN == harden(V_init), pack/dequant
round trip, finite differences of Eq. 5, Round Loss closed forms, Adam
first-step closed form, exhaustive row-separable search on a 4x16 layer,
textbook GEMM special case, zero-residual fixed point; for the alignment loss
(Eq. 6): identical models, shift and temperature invariances, the two-class
closed form, the uniform-model closed form, finite differences of both
gradients.

Parity unpinned (free parameters the paper names but gives no value for; both
sides simply receive them as arguments): the beta schedule, lambda_round, the
optimiser and its hyper-parameters, the calibration batch, tau and lambda_KL
of Eq. 6 and its reduction over tokens (a mean here).
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------
# Formats ("NVFP4 Overview")
# --------------------------------------------------------------------------

#: Non-negative E2M1 nodes; index = 3-bit magnitude code.  ("NVFP4 Overview":
#: the node set N = {0, 0.5, 1, 1.5, 2, 3, 4, 6} with both signs.)
NODES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0], dtype=np.float64)

BLOCK = 16  # elements per scale block, along the contraction dimension K

E2M1_MAX = 6.0
E4M3_MAX = 448.0


def e4m3_decode(byte):
    """Value of an FP8 E4M3 byte (1 sign, 4 exponent bits with bias 7, 3
    mantissa bits, subnormals, no infinities, S.1111.111 = NaN)."""
    b = np.asarray(byte, dtype=np.int64)
    sign = np.where((b >> 7) & 1, -1.0, 1.0)
    e = (b >> 3) & 0xF
    m = b & 0x7
    sub = (m / 8.0) * 2.0 ** -6
    nor = (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64))
    val = np.where(e == 0, sub, nor)
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return sign * val


# all finite non-negative E4M3 values in increasing order: bytes 0x00 .. 0x7E
_E4M3_POS = e4m3_decode(np.arange(0x7F))


def e4m3_encode(q):
    """Round a non-negative real to the nearest finite E4M3 value, ties to the
    even mantissa, saturating at 448 (never NaN).  Written as the definition:
    search the table of the 127 finite values."""
    q = np.asarray(q, dtype=np.float64)
    assert np.all(q >= 0) and not np.any(np.isnan(q))
    qc = np.minimum(q, E4M3_MAX)
    hi = np.searchsorted(_E4M3_POS, qc, side="left")       # first value >= q
    hi = np.clip(hi, 0, 0x7E)
    lo = np.maximum(hi - 1, 0)
    d_lo = qc - _E4M3_POS[lo]
    d_hi = _E4M3_POS[hi] - qc
    # the differences above are exact in float64 (binary32 inputs, 4-bit grid)
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    return np.where(pick_hi, hi, lo).astype(np.uint8)


def bf16_round(x):
    """Round float64 to the nearest BF16 value (8 significant bits, binary32
    exponent range), ties to even, in one rounding.  Returned as float64."""
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                       # x = m * 2**e, 0.5 <= |m| < 1
    e = np.maximum(e, -125)                  # BF16 subnormals: fixed quantum 2**-133
    q = np.ldexp(np.rint(np.ldexp(x, 8 - e)), e - 8)
    assert np.all(np.abs(q) < 3.39e38)
    return q


def f32(x):
    return np.asarray(x, dtype=np.float32)


# --------------------------------------------------------------------------
# Part 1: two-level scales, bracket, V_init (Procedure steps 2-5, Eq. 4)
# --------------------------------------------------------------------------

def compute_scales(W, s_global_in=0.0):
    """Per-tensor FP32 scale and per-block E4M3 scales ("NVFP4 Overview").

    The paper names the two levels but not the rule; reading used: the amax
    rule.  s_global = amax(|W|) / (6 * 448); block scale = E4M3(amax_block /
    (6 * s_global)).  A caller-supplied s_global_in > 0 replaces the first.
    All arithmetic binary32, in this order.  Returns (scales u8 [O, K/16],
    s_global float32 scalar)."""
    W = f32(W)
    O, K = W.shape
    assert K % BLOCK == 0
    absW = np.abs(W)
    if s_global_in > 0:
        s_global = np.float32(s_global_in)
    else:
        amax_t = absW.max() if absW.size else np.float32(0)
        s_global = np.float32(amax_t) / np.float32(2688.0)
        if amax_t == 0:
            s_global = np.float32(1.0)
    d = np.float32(s_global * np.float32(6.0))
    amax_g = absW.reshape(O, K // BLOCK, BLOCK).max(axis=2)
    q = (amax_g / d).astype(np.float32)
    return e4m3_encode(q), np.float32(s_global)


def effective_scale(scales, s_global):
    """s = s_g * s_global as a binary32 product, one value per block."""
    sg = e4m3_decode(scales).astype(np.float32)
    return (sg * np.float32(s_global)).astype(np.float32)


def bracket(W, scales, s_global, smooth=False):
    """Procedure steps 2-4 / Eq. 4: normalised magnitude, FindInterval, V_init.

    Readings where the paper is silent: intervals are half-open [lo, hi) with
    the last one closed, so a value on a node takes that node as lo; w~ above
    6 (possible after the block scale is rounded down) is clamped to 6; a block
    whose scale is 0 has w~ = 0; the sign is the sign bit of w (w = +0 counts
    as positive).  Returns (k int [O,K] in 0..6, neg bool [O,K], v_init)."""
    W32 = f32(W)
    O, K = W32.shape
    s = np.repeat(effective_scale(scales, s_global), BLOCK, axis=1)     # [O,K] f32
    neg = np.signbit(W32) & (W32 != 0)
    if smooth:
        absW = np.abs(W32).astype(np.float64)
        sd = s.astype(np.float64)
    else:
        absW = np.abs(W32)
        sd = s
    with np.errstate(divide="ignore", invalid="ignore"):
        wt = np.where(sd > 0, absW / np.where(sd > 0, sd, 1), 0)
    wt = np.minimum(wt, wt.dtype.type(E2M1_MAX))
    k = np.zeros((O, K), dtype=np.int64)
    for j in range(1, 7):                       # largest j <= 6 with NODES[j] <= w~
        k = np.where(wt >= NODES[j], j, k)
    lo = NODES[k].astype(wt.dtype)
    inv_width = (1.0 / (NODES[k + 1] - NODES[k])).astype(wt.dtype)     # 2, 1 or 0.5
    v = (wt - lo) * inv_width
    return k, neg, v


def pack_code(k, neg):
    """Lower-node nibble (bit 3 = sign, bits 2:0 = k), two per byte, element
    2j in the low nibble."""
    nib = (k.astype(np.uint8) | (neg.astype(np.uint8) << 3))
    return (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8)


def unpack_code(code):
    O, Kh = code.shape
    nib = np.empty((O, Kh * 2), dtype=np.uint8)
    nib[:, 0::2] = code & 0xF
    nib[:, 1::2] = code >> 4
    return (nib & 7).astype(np.int64), (nib >> 3).astype(bool)


def softquant_init(W, s_global_in=0.0):
    """Whole of part 1 in the binary32 contract.  Returns
    (scales u8 [O,K/16], s_global f32, code u8 [O,K/2], V_init f32 [O,K])."""
    scales, s_global = compute_scales(W, s_global_in)
    k, neg, v = bracket(W, scales, s_global)
    return scales, s_global, pack_code(k, neg), v.astype(np.float32)


# --------------------------------------------------------------------------
# Part 2: soft weights (Eq. 2, Eq. 3; Procedure steps 6-7)
# --------------------------------------------------------------------------

def h_beta(V, beta):
    """Eq. 3: h = sigma(beta * (v - 0.5))."""
    V = np.asarray(V, dtype=np.float64)
    with np.errstate(over="ignore"):
        return 1.0 / (1.0 + np.exp(-float(beta) * (V - 0.5)))


def soft_weights(V, code, scales, s_global, beta):
    """Eq. 2: W_soft = sign * (lo + h * (hi - lo)) * s_g * s_global.
    Returns (W_soft, h), float64."""
    k, neg = unpack_code(code)
    s = np.repeat(effective_scale(scales, s_global), BLOCK, axis=1).astype(np.float64)
    h = h_beta(V, beta)
    lo, hi = NODES[k], NODES[k + 1]
    sgn = np.where(neg, -1.0, 1.0)
    return sgn * (lo + h * (hi - lo)) * s, h


# --------------------------------------------------------------------------
# Parts 3-4: forward, losses, gradient, update (Eq. 5; Procedure steps 8-13)
# --------------------------------------------------------------------------

def layer_ref(X, W):
    """Procedure step 8: frozen output Y_fp = X W^T (float64)."""
    return np.asarray(X, np.float64) @ np.asarray(W, np.float64).T


def round_loss(V):
    """Eq. 5, second term without lambda: (1/N) sum(1 - (2v - 1)^2)."""
    V = np.asarray(V, dtype=np.float64)
    return float(np.sum(1.0 - (2.0 * V - 1.0) ** 2) / V.size)


def layer_fwd(X, Y_ref, V, code, scales, s_global, beta, mse_scale=1.0, mode="bf16"):
    """Procedure steps 6-10.  Y_q = X W_soft^T, r = Y_q - Y_ref,
    L_MSE = c * sum r^2 (the paper's c is 1: a squared Frobenius norm),
    dY = dL_MSE/dY_q = 2 c r.  Returns (L_MSE, dY [T,O], Y_q [T,O])."""
    W_soft, _ = soft_weights(V, code, scales, s_global, beta)
    if mode == "bf16":
        W_soft = bf16_round(W_soft)
    Yq = np.asarray(X, np.float64) @ W_soft.T
    r = Yq - np.asarray(Y_ref, np.float64)
    loss = float(mse_scale) * float(np.sum(r * r))
    dY = 2.0 * float(mse_scale) * r
    if mode == "bf16":
        dY = bf16_round(dY)
    return loss, dY, Yq


def chain_factor(V, code, scales, s_global, beta):
    """dW_soft/dv through Eq. 2 and Eq. 3: sign * s * (hi - lo) * beta * h * (1 - h)
    (lo, hi, s and the sign are constants; only V is learnable)."""
    V = np.asarray(V, dtype=np.float64)
    k, neg = unpack_code(code)
    s = np.repeat(effective_scale(scales, s_global), BLOCK, axis=1).astype(np.float64)
    h = h_beta(V, beta)
    width = NODES[k + 1] - NODES[k]
    sgn = np.where(neg, -1.0, 1.0)
    return sgn * s * width * float(beta) * h * (1.0 - h)


def layer_grad(dY, X, V, code, scales, s_global, beta, lambda_round):
    """Gradient of Eq. 5 with respect to V (the paper states the loss; this is
    its derivative).  G = dY^T X is dL_MSE/dW_soft; the chain rule through
    Eq. 2 and Eq. 3 multiplies by chain_factor; the Round Loss adds
    (lambda / N) * (4 - 8 v).  Returns (dV, G)."""
    V = np.asarray(V, dtype=np.float64)
    G = np.asarray(dY, np.float64).T @ np.asarray(X, np.float64)
    dV = G * chain_factor(V, code, scales, s_global, beta)
    dV = dV + (float(lambda_round) / V.size) * (4.0 - 8.0 * V)
    return dV, G


def layer_dx(dY, V, code, scales, s_global, beta, mode="bf16"):
    """Gradient with respect to the layer's input: dX = dY W_soft (the derivative of Y_q = X W_soft^T;
    what full-model alignment, Procedure steps 16-23, must pass on to the layer below).  In mode "bf16"
    W_soft is the BF16 operand of the forward GEMM.  Returns dX [T,K], float64."""
    W_soft, _ = soft_weights(V, code, scales, s_global, beta)
    if mode == "bf16":
        W_soft = bf16_round(W_soft)
    return np.asarray(dY, np.float64) @ W_soft


def adam_update(V, g, m, u, lr, beta1, beta2, eps, step):
    """Adam with bias correction (step is 1-based), then the clip to [0, 1]
    that Stage 1 prescribes after each gradient update.  float64 in/out."""
    m = beta1 * m + (1.0 - beta1) * g
    u = beta2 * u + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** step)
    uhat = u / (1.0 - beta2 ** step)
    V = V - lr * mhat / (np.sqrt(uhat) + eps)
    return np.clip(V, 0.0, 1.0), m, u


def sgd_update(V, g, lr):
    """Plain gradient descent followed by the clip to [0, 1]."""
    return np.clip(V - lr * g, 0.0, 1.0)


class HParams:
    """Hyper-parameters of one step.  opt: 0 = SGD, 1 = Adam."""

    def __init__(self, beta=4.0, lambda_round=1.0, mse_scale=1.0, opt=1, lr=1e-2,
                 beta1=0.9, beta2=0.999, eps=1e-8, step=1):
        self.beta, self.lambda_round, self.mse_scale = beta, lambda_round, mse_scale
        self.opt, self.lr, self.beta1, self.beta2, self.eps, self.step = opt, lr, beta1, beta2, eps, step


def layer_step(X, Y_ref, V, code, scales, s_global, m, u, hp, mode="bf16"):
    """One pass of Procedure steps 6-13: losses and gradient at the current V,
    then the update and the clip.  Returns (V', m', u', L_MSE, L_round, dV).
    In mode "bf16" V, m, u are stored as binary32 between steps."""
    Vd = np.asarray(V, np.float64)
    l_mse, dY, _ = layer_fwd(X, Y_ref, Vd, code, scales, s_global, hp.beta, hp.mse_scale, mode)
    l_round = round_loss(Vd)
    dV, _ = layer_grad(dY, X, Vd, code, scales, s_global, hp.beta, hp.lambda_round)
    if hp.opt == 1:
        Vn, mn, un = adam_update(Vd, dV, np.asarray(m, np.float64), np.asarray(u, np.float64),
                                 hp.lr, hp.beta1, hp.beta2, hp.eps, hp.step)
    else:
        Vn, mn, un = sgd_update(Vd, dV, hp.lr), m, u
    if mode == "bf16":
        Vn, mn, un = f32(Vn), f32(mn), f32(un)
    return Vn, mn, un, l_mse, l_round, dV


def beta_schedule(t, steps, beta0=4.0, beta1=32.0):
    """Geometric annealing from beta0 to beta1 (the paper says beta starts
    small and is increased; it gives no values -- these are this harness's)."""
    if steps <= 1:
        return float(beta0)
    return float(beta0 * (beta1 / beta0) ** (t / (steps - 1)))


def run_layer(X, Y_ref, W, steps, lr=1e-2, lambda_round=1.0, mse_scale=1.0, opt=1, mode="bf16",
              beta0=4.0, beta1=32.0):
    """Procedure steps 1-13 for one layer: init, then `steps` updates.
    Returns dict with final V, the init outputs and the loss history."""
    scales, s_global, code, V = softquant_init(W)
    if mode == "smooth":
        k, neg, V = bracket(W, scales, s_global, smooth=True)
    m = np.zeros_like(V)
    u = np.zeros_like(V)
    hist = []
    for t in range(steps):
        hp = HParams(beta=beta_schedule(t, steps, beta0, beta1), lambda_round=lambda_round,
                     mse_scale=mse_scale, opt=opt, lr=lr, step=t + 1)
        V, m, u, l_mse, l_round, _ = layer_step(X, Y_ref, V, code, scales, s_global, m, u, hp, mode)
        hist.append((l_mse, l_round))
    return dict(V=V, m=m, u=u, scales=scales, s_global=s_global, code=code, hist=hist)


# --------------------------------------------------------------------------
# Part 5: hardening and packing (Eq. 7; Procedure steps 25-26)
# --------------------------------------------------------------------------

def harden(V):
    """Eq. 7: v_hat = 1 if v >= 0.5 else 0."""
    return (np.asarray(V) >= 0.5)


def harden_pack(V, code, scales, s_global):
    """Eq. 7 then Eq. 2 with h replaced by v_hat.  The hardened magnitude code
    is k + v_hat (the E2M1 bit pattern of the chosen node); nibble = sign<<3 |
    code; element 2j in the low nibble of byte j.  Returns (packed u8 [O,K/2],
    decisions bool [O,K], W_final float32 [O,K] = sign * node * s computed as a
    binary32 product)."""
    k, neg = unpack_code(code)
    vh = harden(V)
    mag = k + vh.astype(np.int64)
    nib = (mag.astype(np.uint8) | (neg.astype(np.uint8) << 3))
    packed = (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8)
    s = np.repeat(effective_scale(scales, s_global), BLOCK, axis=1)
    W_final = (NODES[mag].astype(np.float32) * s).astype(np.float32)
    W_final = np.where(neg, -W_final, W_final)
    return packed, vh, W_final


def pack_decisions(vh):
    """Bitmask of decisions, element 8j+i in bit i of byte j."""
    O, K = vh.shape
    return np.packbits(vh.astype(np.uint8).reshape(O, K // 8, 8), axis=2, bitorder="little").reshape(O, K // 8)


def dequant_packed(packed, scales, s_global):
    """Decode deployable NVFP4 (nibbles + E4M3 block scales + FP32 tensor
    scale) back to binary32 weights."""
    O, Kh = packed.shape
    nib = np.empty((O, Kh * 2), dtype=np.uint8)
    nib[:, 0::2] = packed & 0xF
    nib[:, 1::2] = packed >> 4
    s = np.repeat(effective_scale(scales, s_global), BLOCK, axis=1)
    val = (NODES[nib & 7].astype(np.float32) * s).astype(np.float32)
    return np.where((nib >> 3).astype(bool), -val, val)


def nvfp4_matmul(A_packed, A_scales, A_s_global, B_packed, B_scales, B_s_global):
    """What deployable NVFP4 operands mean as a product ("Hardening and Inference": the hardened weights run
    on NVFP4 hardware as they are): C = dequant(A) dequant(B)^T with every element decoded as
    sign * node * block scale * tensor scale, contraction in float64.  A: [M, K/2] codes + [M, K/16] scales,
    B: [N, K/2] + [N, K/16]; returns [M, N]."""
    A = dequant_packed(A_packed, A_scales, A_s_global).astype(np.float64)
    B = dequant_packed(B_packed, B_scales, B_s_global).astype(np.float64)
    return A @ B.T


def act_fake_quant(X, s_global_in=0.0):
    """Quantised activations X_q of the Stage-1 objective (Eq. 5 uses X_q W_q).  The paper gives no
    rule for them; reading used: the same NVFP4 format as the weights (blocks of 16 along the
    contraction dimension, E4M3 block scales under an FP32 tensor scale, amax rule) with
    round-to-nearest, a tie going to the larger magnitude -- i.e. Eq. 7 applied to the initial
    position v_init.  Returns (Xq_units float64 [T,K] = sign * node * s_g, exactly representable in
    BF16; s_global float32; packed u8 [T,K/2]; scales u8 [T,K/16]); X_q = Xq_units * s_global."""
    scales, s_global, code, v = softquant_init(X, s_global_in)
    packed, _, _ = harden_pack(v, code, scales, s_global)
    k_mag, neg = unpack_code(packed)
    sg = np.repeat(e4m3_decode(scales), BLOCK, axis=1)
    units = np.where(neg, -1.0, 1.0) * NODES[k_mag] * sg
    return units, s_global, packed, scales


def swizzle_scales(scales):
    """Block scales [rows, cols] (cols = K/16) in the tiled order that block-scaled tensor-core GEMMs
    read: the matrix is padded with zeros to multiples of 128 rows and 4 columns and cut into
    128 x 4 tiles stored one after another (tiles of a row band first); inside a tile the byte of
    (r, c) sits at (r % 32) * 16 + (r // 32) * 4 + c.  ("Directly deployable" output; the paper gives no
    layout -- this is the hardware's.)  Written as the definition: one element at a time."""
    rows, cols = scales.shape
    rt, ct = (rows + 127) // 128, (cols + 3) // 4
    out = np.zeros(rt * ct * 512, dtype=np.uint8)
    for r in range(rows):
        for c in range(cols):
            tile = (r // 128) * ct + (c // 4)
            rr, cc = r % 128, c % 4
            out[tile * 512 + (rr % 32) * 16 + (rr // 32) * 4 + cc] = scales[r, c]
    return out


def silu_mul(gate, up):
    """The MLP's gated product of a Llama / Qwen decoder block: silu(g) * u with silu(x) = x / (1 + e^-x)
    (the frozen model's input of down_proj, which Stage 1 optimises "for each layer").  float64."""
    g = np.asarray(gate, dtype=np.float64)
    with np.errstate(over="ignore"):
        return g / (1.0 + np.exp(-g)) * np.asarray(up, dtype=np.float64)


def rtn_nearest(W, scales, s_global):
    """Round-to-nearest onto the node set, written independently of the
    bracket: argmin over all 8 nodes of |w~ - node|, a tie going to the larger
    node (the convention Eq. 7's `>=` implies).  Returns magnitude codes."""
    W32 = f32(W)
    s = np.repeat(effective_scale(scales, s_global), BLOCK, axis=1)
    with np.errstate(divide="ignore", invalid="ignore"):
        wt = np.where(s > 0, np.abs(W32) / np.where(s > 0, s, 1), 0).astype(np.float32)
    wt = np.minimum(wt, np.float32(6.0)).astype(np.float64)
    dist = np.abs(wt[..., None] - NODES[None, None, :])
    best = dist.min(axis=2, keepdims=True)
    cand = np.where(dist == best, np.arange(8)[None, None, :], -1)
    return cand.max(axis=2)


# --------------------------------------------------------------------------
# Full-model alignment loss (Eq. 6, Procedure steps 18-20)
# --------------------------------------------------------------------------

def align_loss(Z_fp, Z_q, H_fp, H_q, tau=1.0, lambda_kl=1.0):
    """The two data terms of Eq. 6 and their gradients towards the quantised model's outputs.

    P_fp = softmax(Z_fp / tau), P_q = softmax(Z_q / tau) over the vocabulary (Procedure step 18);
    L_KL = KL(P_fp || P_q) (step 19), summed over the vocabulary and averaged over the T tokens (the
    paper gives no reduction over tokens; a mean keeps lambda_KL independent of the batch size);
    L_MSE = ||H_fp - H_q||_F^2 (step 20), a sum.
    Returns (L_KL, L_MSE, dZ_q, dH_q) with dZ_q = d(lambda_kl L_KL)/dZ_q = lambda_kl (P_q - P_fp) / (tau T)
    and dH_q = dL_MSE/dH_q = 2 (H_q - H_fp).  float64 throughout; log-softmax by the max-shifted form."""
    Zf = np.asarray(Z_fp, dtype=np.float64) / tau
    Zq = np.asarray(Z_q, dtype=np.float64) / tau
    T = Zf.shape[0]

    def log_softmax(Z):
        Zs = Z - Z.max(axis=1, keepdims=True)
        return Zs - np.log(np.exp(Zs).sum(axis=1, keepdims=True))

    lf, lq = log_softmax(Zf), log_softmax(Zq)
    pf, pq = np.exp(lf), np.exp(lq)
    l_kl = float((pf * (lf - lq)).sum() / T)
    dZ = lambda_kl * (pq - pf) / (tau * T)
    D = np.asarray(H_q, dtype=np.float64) - np.asarray(H_fp, dtype=np.float64)
    return l_kl, float((D * D).sum()), dZ, 2.0 * D
