"""GPU parity on the linears of a Llama-3.2-1B-shaped and a Qwen3-1.7B-shaped decoder block
(Stage-1 layer-wise workloads): every distinct (O, K) of the two blocks, one 4096-token minibatch of
the synthetic hidden-state distribution, one full step on the GPU.  The loss separates over output
rows, so the oracle runs the same step on a sample of rows (an exact sub-problem) and the sampled rows
of every per-weight output are compared; the scalar loss is compared where the whole layer is small
enough for the oracle."""
import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from paper_2603_22370_b200 import faar, inputs
from tests.gpu_helpers import DEV, GpuLayer, host, max_rel_to_peak, rel_l2

pytestmark = pytest.mark.gpu

T = 4096
SHAPES = sorted({(o, k) for _, o, k in inputs.LLAMA32_1B_BLOCK + inputs.QWEN3_1P7B_BLOCK})


@pytest.fixture(scope="module")
def ctx():
    from paper_2603_22370_b200 import build
    build.build()
    c = faar.Context(0)
    yield c
    torch.cuda.synchronize()
    c.close()


@pytest.mark.parametrize("O,K", SHAPES)
def test_one_step_on_block_linear(ctx, O, K):
    W, X = inputs.block_linear(11, SHAPES.index((O, K)), O, K, T)
    lay = GpuLayer(ctx, W, X)
    lay.init()
    Yref_g = torch.empty((T, O), dtype=torch.bfloat16, device=DEV)
    faar.layer_ref(ctx, lay.shape, lay.X, lay.W, Yref_g, lay.ws)
    lay.check()

    rng = np.random.default_rng(O * 31 + K)
    rows = np.unique(np.concatenate([[0, O - 1, 127, 128, min(O - 1, 255), min(O - 1, 256)],
                                     rng.choice(O, size=90, replace=False)]))
    Wr = W[rows]
    # the tensor scale needs the whole tensor; the rest of the set-up is per row
    _, sg = fo.compute_scales(W)
    scales, sg2, code, V0 = fo.softquant_init(Wr, float(sg))
    assert host(lay.s_global)[0] == sg == sg2
    assert np.array_equal(host(lay.scales)[rows], scales)
    assert np.array_equal(host(lay.code)[rows], code)
    assert np.array_equal(host(lay.V)[rows].view(np.uint32), V0.view(np.uint32))

    Yref_r = fo.layer_ref(X, Wr)
    d = np.abs(host(Yref_g)[:, rows] - Yref_r)
    assert np.all(d <= 2.0 ** -8 * np.abs(Yref_r) + 1e-5 * np.abs(Yref_r).max())
    Yref_full = host(Yref_g)                          # both sides continue from the GPU's BF16 target
    lay.Yref = Yref_g

    kw = dict(beta=6.0, lambda_round=1.0, mse_scale=1.0, opt=1, lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8, step=1)
    for k in ("lr", "beta1", "beta2", "eps"):
        kw[k] = float(np.float32(kw[k]))
    hp, hpo = faar.make_hparams(**kw), fo.HParams(**kw)
    lay.fwd(hp)
    dV_g = lay.bwd(hp, want_dv=True)
    lay.check()

    # oracle on the sampled rows; lambda/N uses the whole layer's N, so pass lambda scaled to the sample
    hpo.lambda_round = kw["lambda_round"] * len(rows) / O
    zeros = np.zeros_like(V0)
    Vo, mo, uo, l_mse_rows, _, dV_o = fo.layer_step(X, Yref_full[:, rows], V0, code, scales, sg, zeros, zeros, hpo, "bf16")
    dV_gr = host(dV_g)[rows]
    assert rel_l2(dV_gr, dV_o) <= 2e-3 and max_rel_to_peak(dV_gr, dV_o) <= 2e-3
    Vg = host(lay.V)
    assert Vg.min() >= 0.0 and Vg.max() <= 1.0
    assert rel_l2(Vg[rows], Vo) <= 2e-3
    assert max_rel_to_peak(host(lay.m)[rows], mo) <= 2e-3
    sure = np.abs(dV_o) > 1e-3 * np.abs(dV_o).max()
    assert np.all(np.abs(Vg[rows] - Vo)[sure] <= 1e-6)

    if O * K <= 2048 * 2048:
        scales_f, _, code_f, V0_f = fo.softquant_init(W)
        l_full, _, _ = fo.layer_fwd(X, Yref_full, V0_f, code_f, scales_f, sg, hpo.beta, 1.0, "bf16")
        assert abs(host(lay.loss)[0] - l_full) <= 2e-3 * l_full
    else:
        assert host(lay.loss)[0] >= l_mse_rows * (1 - 2e-3)      # the sampled rows' share is a lower bound

    packed = torch.empty((O, K // 2), dtype=torch.uint8, device=DEV)
    faar.harden_pack(ctx, lay.shape, lay.V, lay.code, lay.scales, lay.s_global, packed, None, None, None)
    lay.check()
    p_o, _, _ = fo.harden_pack(Vg[rows], code, scales, sg)
    assert np.array_equal(host(packed)[rows], p_o)
