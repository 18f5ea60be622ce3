"""GPU parity at the size the benchmark times: the down_proj-shaped layer (W 2048 x 8192,
X 4096 x 8192, BF16), in the launch configuration bench.py uses (same entry points, same
tile shapes, persistent CTA pairs over all SMs).  numpy finishes one full oracle step of this
layer in a few seconds, so every output is compared, not a sample.  Tolerances as in
test_gpu_parity.py: bytes and V_init bit-exact; loss 2e-3 relative; dV and updated V 2e-3 in
the 2-norm and relative to the peak."""
import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from paper_2603_22370_b200 import faar, inputs
from tests.gpu_helpers import DEV, GpuLayer, dev_f32, host, max_rel_to_peak, rel_l2

pytestmark = pytest.mark.gpu

O, K, T = 2048, 8192, 4096


@pytest.fixture(scope="module")
def ctx():
    from paper_2603_22370_b200 import build
    build.build()
    c = faar.Context(0)
    yield c
    torch.cuda.synchronize()
    c.close()


@pytest.fixture(scope="module")
def problem():
    W, X = inputs.config2(0, O, K, T)
    return W, X


def test_init_step_and_pack_at_full_size(ctx, problem):
    W, X = problem
    lay = GpuLayer(ctx, W, X)

    # ---- part 1: set-up, bit-exact over all 16.7 M weights
    lay.init()
    lay.check()
    scales, sg, code, V0 = fo.softquant_init(W)
    assert host(lay.s_global)[0] == sg
    assert np.array_equal(host(lay.scales), scales)
    assert np.array_equal(host(lay.code), code)
    assert np.array_equal(host(lay.V).view(np.uint32), V0.view(np.uint32))

    # ---- frozen target on the tensor cores vs float64
    Yref_g = torch.empty((T, O), dtype=torch.bfloat16, device=DEV)
    faar.layer_ref(ctx, lay.shape, lay.X, lay.W, Yref_g, lay.ws)
    lay.check()
    Yref_o = fo.layer_ref(X, W)
    d = np.abs(host(Yref_g) - Yref_o)
    assert np.all(d <= 2.0 ** -8 * np.abs(Yref_o) + 1e-5 * np.abs(Yref_o).max())
    Yref = inputs.to_bf16_f32(Yref_o)                 # both sides continue from the oracle's target
    lay.set_yref(Yref)
    del Yref_g, d, Yref_o

    # ---- parts 2-4: one step from V_init, forward and backward called separately to see dV
    kw = dict(beta=4.0, lambda_round=1.0, mse_scale=1.0, opt=1, lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, step=1)
    for k in ("lr", "beta1", "beta2", "eps"):
        kw[k] = float(np.float32(kw[k]))
    hp, hpo = faar.make_hparams(**kw), fo.HParams(**kw)
    lay.fwd(hp)
    l_round = torch.zeros(1, device=DEV)
    faar.round_loss(ctx, lay.V, O * K, l_round, lay.ws)
    dV_g = lay.bwd(hp, want_dv=True)
    lay.check()
    zeros = np.zeros_like(V0)
    Vo, mo, uo, l_mse_o, l_round_o, dV_o = fo.layer_step(X, Yref, V0, code, scales, sg, zeros, zeros, hpo, "bf16")
    assert abs(host(lay.loss)[0] - l_mse_o) <= 2e-3 * l_mse_o
    assert abs(host(l_round)[0] - l_round_o) <= 1e-5 * l_round_o
    dV_g = host(dV_g)
    assert rel_l2(dV_g, dV_o) <= 2e-3 and max_rel_to_peak(dV_g, dV_o) <= 2e-3
    Vg = host(lay.V)
    assert Vg.min() >= 0.0 and Vg.max() <= 1.0
    # the first Adam step moves every v by lr * g / (|g| + eps): where the gradient's sign is
    # certain both sides agree to rounding; compare in the norms the target statement uses
    assert rel_l2(Vg, Vo) <= 2e-3 and max_rel_to_peak(host(lay.m), mo) <= 2e-3
    sure = np.abs(dV_o) > 1e-3 * np.abs(dV_o).max()
    assert np.all(np.abs(Vg - Vo)[sure] <= 1e-6)

    # ---- the fused step entry point from the same state gives the same update
    lay.set_state(V=V0, m=zeros, u=zeros)
    lay.step(hp)
    lay.check()
    assert np.array_equal(host(lay.V), Vg)
    loss = host(lay.loss)
    assert abs(loss[0] - l_mse_o) <= 2e-3 * l_mse_o and abs(loss[1] - l_round_o) <= 1e-5 * l_round_o

    # ---- part 5: harden + pack of the GPU's V, bit-exact
    packed = torch.empty((O, K // 2), dtype=torch.uint8, device=DEV)
    scales_out = torch.empty((O, K // 16), dtype=torch.uint8, device=DEV)
    dec = torch.empty((O, K // 8), dtype=torch.uint8, device=DEV)
    Wf = torch.empty((O, K), dtype=torch.float32, device=DEV)
    faar.harden_pack(ctx, lay.shape, lay.V, lay.code, lay.scales, lay.s_global, packed, scales_out, dec, Wf, faar.F32)
    lay.check()
    p_o, vh_o, Wf_o = fo.harden_pack(Vg, code, scales, sg)
    assert np.array_equal(host(packed), p_o)
    assert np.array_equal(host(scales_out), scales)
    assert np.array_equal(host(dec), fo.pack_decisions(vh_o))
    assert np.array_equal(host(Wf).view(np.uint32), Wf_o.view(np.uint32))
    assert np.array_equal(fo.dequant_packed(p_o, scales, sg).view(np.uint32), Wf_o.view(np.uint32))
