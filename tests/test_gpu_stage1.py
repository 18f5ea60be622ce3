"""The Stage-1 driver (host loop over library calls) on the small parity layer: its result must be the
hardening of its own final V (checked with the oracle), its loss must fall, and a two-linear block must
come back complete."""
import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from paper_2603_22370_b200 import faar, inputs, stage1
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
