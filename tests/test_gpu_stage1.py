"""The Stage-1 driver (host loop over library calls) on the small parity layer: its result must be the
hardening of its own final V (checked with the oracle), its loss must fall, and a two-linear block must
come back complete."""
import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from paper_2603_22370_b200 import faar, inputs, shard, stage1
from tests.gpu_helpers import dev_bf16, host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2603_22370_b200 import build
    build.build()
    c = faar.Context(0)
    yield c
    torch.cuda.synchronize()
    c.close()


@pytest.mark.parametrize("quantise_activations", [False, True])
def test_optimise_layer(ctx, quantise_activations):
    W, X = inputs.config1(0)
    W, X = inputs.to_bf16_f32(W), inputs.to_bf16_f32(X)
    res = stage1.optimise_layer(ctx, dev_bf16(W), dev_bf16(X), steps=100, loss_every=25,
                                quantise_activations=quantise_activations)
    scales, sg, code, V0 = fo.softquant_init(W)
    assert np.array_equal(host(res["scales"]), scales) and np.array_equal(host(res["code"]), code)
    p_o, _, Wf = fo.harden_pack(host(res["V"]), code, scales, sg)
    assert np.array_equal(host(res["packed"]), p_o)
    hist = res["history"]
    assert [h[0] for h in hist] == [25, 50, 75, 100, 100]
    assert all(np.isfinite(h[1]) and h[1] >= 0 and 0 <= h[2] <= 1 for h in hist)
    # hardened FAAR output vs plain RTN on the layer's own objective
    Xo = X.astype(np.float64)
    if quantise_activations:
        units, sx, _, _ = fo.act_fake_quant(X)
        Xo = units * float(sx)
        assert res["act_scale"] == float(sx)
    Yref = fo.layer_ref(X, W)
    _, _, W_rtn = fo.harden_pack(V0, code, scales, sg)
    l_faar = np.sum((Xo @ Wf.astype(np.float64).T - Yref) ** 2)
    l_rtn = np.sum((Xo @ W_rtn.astype(np.float64).T - Yref) ** 2)
    print("hardened loss FAAR / RTN:", l_faar / l_rtn)
    assert l_faar <= 1.05 * l_rtn


def test_optimise_block_covers_every_linear(ctx):
    lin = []
    for i, (name, O, K) in enumerate([("q_proj", 64, 128), ("k_proj", 32, 128)]):
        W, X = inputs.block_linear(1, i, O, K, 256)
        lin.append((name, dev_bf16(W), dev_bf16(X)))
    out = stage1.optimise_block(ctx, lin, steps=5)
    assert sorted(out) == ["k_proj", "q_proj"]
    assert out["q_proj"]["packed"].shape == (64, 64)
    part = stage1.optimise_block(ctx, lin, steps=2, rank=1, world=2)
    assert sorted(part) == ["k_proj"]


@pytest.mark.parametrize("O,world", [(128, 2), (96, 3)])
def test_row_shards_reproduce_the_whole_layer(ctx, O, world):
    """Eq. 5 separates over output features: the ranks of a row-sharded layer, given the whole tensor's
    scale, must arrive at the rows the unsharded run produces.  The ranks are run one after the other on
    this GPU.  Two equal shards: bit for bit (lambda / N is formed from lambda / 2 exactly); three: the
    Round Loss weight is rounded once more, so V may move in its last bits."""
    K, T = 256, 512
    W, X = inputs.config2(4, O, K, T)
    Wd, Xd = dev_bf16(W), dev_bf16(X)
    kw = dict(steps=12, lr=1e-2, loss_every=0)
    whole = stage1.optimise_layer(ctx, Wd, Xd, **kw)
    sg = float(host(whole["s_global"])[0])
    mse_sum, round_sum = 0.0, 0.0
    for r in range(world):
        b, e = shard.rows_for_rank(O, r, world)
        part = stage1.optimise_layer(ctx, Wd, Xd, rows=(b, e), s_global_in=sg, **kw)
        assert np.array_equal(host(part["scales"]), host(whole["scales"])[b:e])
        assert np.array_equal(host(part["code"]), host(whole["code"])[b:e])
        Vp, Vw = host(part["V"]), host(whole["V"])[b:e]
        if world == 2:
            assert np.array_equal(Vp, Vw)
            assert np.array_equal(host(part["packed"]), host(whole["packed"])[b:e])
        else:
            assert np.max(np.abs(Vp - Vw)) <= 1e-5
            flips = (Vp >= 0.5) != (Vw >= 0.5)
            assert np.all(np.abs(Vw[flips] - 0.5) < 1e-4)
        mse_sum += part["history"][-1][1]
        round_sum += part["history"][-1][2] * (e - b) / O
    assert abs(mse_sum - whole["history"][-1][1]) <= 1e-4 * whole["history"][-1][1]
    assert abs(round_sum - whole["history"][-1][2]) <= 1e-5
    # the one-process form of the sharded driver is the whole layer
    one = stage1.optimise_layer_row_sharded(ctx, Wd, Xd, 0, 1, **kw)
    assert one["rows"] == (0, O) and np.array_equal(host(one["V"]), host(whole["V"]))
    assert abs(one["layer_losses"][0] - whole["history"][-1][1]) <= 1e-6 * whole["history"][-1][1]
