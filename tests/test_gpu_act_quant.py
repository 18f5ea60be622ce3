"""GPU parity of the quantised-activation path: faar_act_fakequant against the oracle's X_q (bit for
bit: the BF16 unit values, the FP32 tensor scale, the packed E2M1 codes and the E4M3 block scales),
and one layer step in which the GEMMs consume X_q (units in BF16, the tensor scale applied in the
epilogues) against the oracle's step on the same X_q in float64."""
import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from paper_2603_22370_b200 import faar, inputs
from tests.gpu_helpers import DEV, GpuLayer, dev_bf16, host, max_rel_to_peak, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2603_22370_b200 import build
    build.build()
    c = faar.Context(0)
    yield c
    torch.cuda.synchronize()
    c.close()


def _quantise(ctx, X, s_global_in=0.0, ldx=None):
    T, K = X.shape
    ws = ctx.workspace(faar.make_shape(16, 16, 8))
    ldx = ldx or K
    Xd = torch.full((T, ldx), 3.0, dtype=torch.bfloat16, device=DEV)
    Xd[:, :K] = dev_bf16(X)
    Xq = torch.zeros((T, K), dtype=torch.bfloat16, device=DEV)
    sx = torch.zeros(1, dtype=torch.float32, device=DEV)
    packed = torch.zeros((T, K // 2), dtype=torch.uint8, device=DEV)
    scales = torch.zeros((T, K // 16), dtype=torch.uint8, device=DEV)
    faar.act_fakequant(ctx, T, K, Xd, ldx, s_global_in, Xq, K, sx, packed, scales, ws)
    torch.cuda.synchronize()
    faar.check_status(ctx, ws)
    return Xq, sx, packed, scales


@pytest.mark.parametrize("T,K,ldx,sg_in", [(77, 48, None, 0.0), (600, 1040, 1048, 0.0), (33, 256, None, 2.0 ** -7)])
def test_act_fakequant_bit_exact(ctx, T, K, ldx, sg_in):
    _, X = inputs.config2(3, 8, K, T)
    X[0, :16] = 0.0
    X[1, 16] = -0.0
    # a block whose scale is a power of two when the tensor scale is 2^-7 (block amax 6 * 8 * 2^-7), holding
    # every midpoint between two nodes: exact ties, which go to the larger node
    X[2, :16] = np.array([6, 5, 3.5, 2.5, 1.75, 1.25, 0.75, 0.25, -5, -3.5, -2.5, -1.75, -1.25, -0.75, -0.25, 0.125]) * 0.0625
    Xq, sx, packed, scales = _quantise(ctx, X, sg_in, ldx)
    units, sg, packed_o, scales_o = fo.act_fake_quant(X, sg_in)
    assert host(sx)[0] == sg
    assert np.array_equal(host(scales), scales_o)
    assert np.array_equal(host(packed), packed_o)
    assert np.array_equal(host(Xq).astype(np.float64), units)
    if sg_in > 0:       # the ties went up: 5 -> 6, 3.5 -> 4, ..., 0.25 -> 0.5 in units of the block scale 8
        assert np.array_equal(units[2, :16], 8.0 * np.array([6, 6, 4, 3, 2, 1.5, 1, 0.5, -6, -4, -3, -2, -1.5, -1, -0.5, 0]))
    # outputs are optional
    ws = ctx.workspace(faar.make_shape(16, 16, 8))
    Xq2 = torch.zeros_like(Xq)
    faar.act_fakequant(ctx, T, K, dev_bf16(X), K, sg_in, Xq2, K, sx, None, None, ws)
    torch.cuda.synchronize()
    assert torch.equal(Xq, Xq2)


@pytest.mark.parametrize("O,K,T", [(300, 1040, 600), (128, 256, 1024)])
def test_layer_step_on_quantised_activations(ctx, O, K, T):
    W, X = inputs.config2(9, O, K, T)
    Yref = inputs.to_bf16_f32(fo.layer_ref(X, W))          # the frozen target uses the unquantised X
    Xq, sx, _, _ = _quantise(ctx, X)
    units, sg, _, _ = fo.act_fake_quant(X)
    Xq_o = units * float(sg)                                # the oracle's X_q, float64
    lay = GpuLayer(ctx, W, host(Xq))                        # X = unit values, X^T built from them
    lay.init()
    lay.set_yref(Yref)
    scales, s_w, code, V0 = fo.softquant_init(W)
    kw = dict(beta=5.0, lambda_round=1.0, mse_scale=1.0, opt=1, lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, step=1)
    for k in ("lr", "beta1", "beta2", "eps"):
        kw[k] = float(np.float32(kw[k]))
    hp = faar.make_hparams(act_scale=float(sg), **kw)
    hpo = fo.HParams(**kw)
    Yq = lay.fwd(hp, want_yq=True)
    dV = lay.bwd(hp, want_dv=True)
    lay.check()
    zeros = np.zeros_like(V0)
    Vo, mo, _, l_mse, _, dV_o = fo.layer_step(Xq_o, Yref, V0, code, scales, s_w, zeros, zeros, hpo, "bf16")
    _, _, Yq_o = fo.layer_fwd(Xq_o, Yref, V0, code, scales, s_w, hpo.beta, 1.0, "bf16")
    assert abs(host(lay.loss)[0] - l_mse) <= 2e-3 * l_mse
    assert rel_l2(host(Yq), Yq_o) <= 2e-3 and max_rel_to_peak(host(Yq), Yq_o) <= 4e-3
    assert rel_l2(host(dV), dV_o) <= 2e-3 and max_rel_to_peak(host(dV), dV_o) <= 2e-3
    assert rel_l2(host(lay.V), Vo) <= 2e-3 and max_rel_to_peak(host(lay.m), mo) <= 2e-3
    # quantising the activations changes the problem: the same step on the raw X gives another loss
    l_raw, _, _ = fo.layer_fwd(X, Yref, V0, code, scales, s_w, hpo.beta, 1.0, "bf16")
    assert abs(l_raw - l_mse) > 1e-2 * l_mse
    # the fused step entry point takes the same hyper-parameter
    lay.set_state(V=V0, m=zeros, u=zeros)
    lay.step(hp)
    lay.check()
    assert abs(host(lay.loss)[0] - l_mse) <= 2e-3 * l_mse
    assert rel_l2(host(lay.V), Vo) <= 2e-3
    # two more steps, alone and chained (the backward pass writes the next operand): the same bits
    ends = []
    for chained in (False, True):
        lay.set_state(V=V0, m=zeros, u=zeros)
        for t in range(3):
            extra = dict(wsoft_ready=int(t > 0), beta_next=5.0 + t + 1 if t < 2 else 0.0) if chained else {}
            lay.step(faar.make_hparams(act_scale=float(sg), **{**kw, "beta": 5.0 + t, "step": t + 1}, **extra))
        lay.check()
        ends.append((host(lay.V).copy(), host(lay.loss).copy()))
    assert np.array_equal(ends[0][0], ends[1][0]) and np.array_equal(ends[0][1], ends[1][1])
