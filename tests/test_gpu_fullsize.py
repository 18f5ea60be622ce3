"""GPU parity at the size the benchmark times: the down_proj-shaped layer (W 2048 x 8192,
X 4096 x 8192, BF16).  The first test calls forward and backward separately to see dV; the second runs
the launch configuration bench.py and the Stage-1 driver use (target stored one row per output feature,
fused step call, chained soft weights) and checks both of its steps against the oracle.  numpy finishes one full oracle step of this
layer in a few seconds, so every output is compared, not a sample.  Tolerances as in
test_gpu_parity.py: bytes and V_init bit-exact; loss 2e-3 relative; dV and updated V 2e-3 in
the 2-norm and relative to the peak."""
import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from paper_2603_22370_b200 import faar, inputs
from tests.gpu_helpers import DEV, GpuLayer, bf16_tie_elements, dev_f32, host, max_rel_to_peak, rel_l2

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


def assert_dv_elementwise(X, dY_used, V, code, scales, sg, hpo, dV_g):
    """Every entry of dV, element by element, given the very dY^T the backward kernel read (the GPU's own,
    BF16): the float64 gradient from those inputs differs from the kernel's only by the FP32 accumulation
    of the T-term dot product (bounded against the sum of the magnitudes of its terms, which is about
    sqrt(K) times a typical entry) and by the FP32 evaluation of the chain factor.  A wrong value in a
    single weight fails here; how far the GPU's dY itself is from the oracle's is checked by the caller."""
    Xd = X.astype(np.float64)
    dV_ref, _ = fo.layer_grad(dY_used, Xd, V, code, scales, sg, hpo.beta, hpo.lambda_round)
    S = (np.abs(dY_used).astype(np.float32).T @ np.abs(X).astype(np.float32)).astype(np.float64)   # a bound: float32 will do
    chain = np.abs(fo.chain_factor(V, code, scales, sg, hpo.beta))
    err = np.abs(dV_g - dV_ref)
    bad = err > 2e-5 * np.abs(dV_ref) + 1e-5 * chain * S
    assert not bad.any(), (int(bad.sum()), float(err[bad].max()))
    typical = np.median(np.abs(dV_ref))
    assert np.median(1e-5 * chain * S) <= 5e-3 * typical          # the bound is tight against a typical entry
    return dV_ref


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
    dY_g = host(lay.dYt)[:, :T].T.astype(np.float64)          # what the backward kernel reads
    l_round = torch.zeros(1, device=DEV)
    faar.round_loss(ctx, lay.V, O * K, l_round, lay.ws)
    dV_g = lay.bwd(hp, want_dv=True)
    lay.check()
    zeros = np.zeros_like(V0)
    Vo, mo, uo, l_mse_o, l_round_o, dV_o = fo.layer_step(X, Yref, V0, code, scales, sg, zeros, zeros, hpo, "bf16")
    assert abs(host(lay.loss)[0] - l_mse_o) <= 2e-3 * l_mse_o
    assert abs(host(l_round)[0] - l_round_o) <= 1e-5 * l_round_o
    # dY against the oracle's, per output feature: 2e-3 of the column plus the effect of BF16-boundary weights
    _, dY_o, _ = fo.layer_fwd(X, Yref, V0, code, scales, sg, hpo.beta, hpo.mse_scale, "bf16")
    Wo, _ = fo.soft_weights(V0, code, scales, sg, hpo.beta)
    tie, bstep = bf16_tie_elements(Wo)
    from tests.gpu_helpers import dy_column_allowance
    col_err = np.linalg.norm(dY_g - dY_o, axis=0)
    assert np.all(col_err <= 2e-3 * np.linalg.norm(dY_o, axis=0) + dy_column_allowance(X, tie, bstep, hpo.mse_scale))
    print("dY entries that differ from the oracle's BF16 value: %.3f %%" % (100.0 * np.mean(dY_g != dY_o)))
    del dY_o, Wo
    dV_g = host(dV_g)
    assert rel_l2(dV_g, dV_o) <= 2e-3 and max_rel_to_peak(dV_g, dV_o) <= 2e-3
    assert_dv_elementwise(X, dY_g, V0, code, scales, sg, hpo, dV_g)
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


def test_benchmarked_launch_configuration_against_the_oracle(ctx, problem):
    """What bench.py and the Stage-1 driver launch: Y_ref stored [O, T] (one row per output feature), the
    fused step call, and chained soft weights (step 1's backward pass writes step 2's BF16 operand, step 2
    skips the soft-weights kernel).  Both steps are compared with the oracle: step 1 from V_init, step 2 from
    the state the GPU itself reached after step 1 (so that the operand it chained is the one under test)."""
    W, X = problem
    lay = GpuLayer(ctx, W, X, yref_transposed=1)
    lay.init()
    scales, sg, code, V0 = fo.softquant_init(W)
    assert np.array_equal(host(lay.code), code) and np.array_equal(host(lay.V), V0)
    Yref = inputs.to_bf16_f32(fo.layer_ref(X, W))
    lay.set_yref(Yref)
    betas = [float(np.float32(4.0)), float(np.float32(5.5))]
    common = dict(lambda_round=1.0, mse_scale=1.0, opt=1, lr=float(np.float32(1e-2)), beta1=float(np.float32(0.9)),
                  beta2=float(np.float32(0.999)), eps=float(np.float32(1e-8)))
    state = (V0, np.zeros_like(V0), np.zeros_like(V0))
    for t in range(2):
        hp = faar.make_hparams(beta=betas[t], step=t + 1, wsoft_ready=int(t > 0),
                               beta_next=betas[t + 1] if t + 1 < len(betas) else 0.0, **common)
        hpo = fo.HParams(beta=betas[t], step=t + 1, **common)
        lay.step(hp)
        lay.check()
        Vo, mo, uo, l_mse_o, l_round_o, dV_o = fo.layer_step(X, Yref, state[0], code, scales, sg, state[1], state[2],
                                                             hpo, "bf16")
        loss = host(lay.loss)
        assert abs(loss[0] - l_mse_o) <= 2e-3 * l_mse_o and abs(loss[1] - l_round_o) <= 1e-5 * l_round_o, t
        Vg, mg, ug = host(lay.V), host(lay.m), host(lay.u)
        assert Vg.min() >= 0.0 and Vg.max() <= 1.0
        assert rel_l2(Vg, Vo) <= 2e-3 and rel_l2(mg, mo) <= 2e-3 and max_rel_to_peak(mg, mo) <= 2e-3, t
        # m' = beta1 m + (1 - beta1) dV: the gradient the fused step used, recovered element by element
        dV_g = (mg.astype(np.float64) - hpo.beta1 * state[1].astype(np.float64)) / (1.0 - hpo.beta1)
        sure = np.abs(dV_o) > 1e-3 * np.abs(dV_o).max()
        if t == 0:
            assert np.all(np.abs(Vg - Vo)[sure] <= 1e-6)
            assert rel_l2(dV_g, dV_o) <= 2e-3 and max_rel_to_peak(dV_g, dV_o) <= 2e-3
        else:
            assert rel_l2(ug, uo) <= 4e-3
        state = (Vg, mg, ug)
