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


def test_silu_mul_matches_oracle(ctx):
    rng = np.random.default_rng(0)
    rows, cols, ld = 77, 136, 144
    g = inputs.to_bf16_f32(rng.standard_normal((rows, cols)) * 3)
    u = inputs.to_bf16_f32(rng.standard_normal((rows, cols)))
    g[0, :6] = [0.0, -0.0, 60.0, -60.0, 1e-20, -100.0]
    G = torch.full((rows, ld), 9.0, dtype=torch.bfloat16, device="cuda:0")
    U = torch.full((rows, ld), 9.0, dtype=torch.bfloat16, device="cuda:0")
    G[:, :cols], U[:, :cols] = dev_bf16(g), dev_bf16(u)
    out = torch.full((rows, ld), 5.0, dtype=torch.bfloat16, device="cuda:0")
    faar.silu_mul(ctx, rows, cols, G, ld, U, ld, out, ld)
    torch.cuda.synchronize()
    ref = fo.silu_mul(g, u)
    got = host(out[:, :cols]).astype(np.float64)
    # BF16 output of an FP32 evaluation: half a BF16 step (at most 2^-8 of the value) plus the FP32 evaluation's 1e-6
    assert np.all(np.abs(got - ref) <= (2.0 ** -8 + 2e-6) * np.abs(ref) + 1e-38)
    assert torch.all(out[:, cols:] == 5.0)
    faar.silu_mul(ctx, rows, cols, G, ld, U, ld, U, ld)            # in place on the second operand
    torch.cuda.synchronize()
    assert torch.equal(U[:, :cols], out[:, :cols])


def test_streamed_minibatches_equal_explicit_steps_and_the_oracle(ctx):
    """A calibration set of three minibatches, visited round-robin: the streamed driver must reproduce, bit
    for bit, a hand-written loop of faar_layer_step over the same minibatches, and stay within the step
    tolerance of the oracle run on them."""
    O, K, mb, n_mb, steps = 96, 256, 128, 3, 7
    W, Xall = inputs.config2(4, O, K, mb * n_mb)
    Wd, Xd = dev_bf16(W), dev_bf16(Xall)
    res = stage1.optimise_layer_streamed(ctx, Wd, Xd, steps, mb)
    # explicit loop, unchained, own buffers
    from tests.gpu_helpers import GpuLayer
    lay = GpuLayer(ctx, W, Xall[:mb], yref_transposed=1)
    lay.init()
    scales, sg, code, V = fo.softquant_init(W)
    m, u = np.zeros_like(V), np.zeros_like(V)
    for t in range(steps):
        j = t % n_mb
        Xb = Xall[j * mb:(j + 1) * mb]
        lay.X.copy_(dev_bf16(Xb))
        faar.transpose_bf16(ctx, mb, K, lay.X, K, lay.Xt, lay.ldt)
        Yg = torch.zeros((O, lay.shape.ldy), dtype=torch.bfloat16, device="cuda:0")
        faar.layer_ref(ctx, lay.shape, lay.X, lay.W, Yg, lay.ws)
        lay.Yref = Yg
        beta = float(np.float32(stage1.beta_schedule(t, steps)))
        lay.step(faar.make_hparams(beta=beta, step=t + 1))
        # the oracle takes the GPU's target (BF16 of a tensor-core product; its own parity is tested elsewhere)
        hpo = fo.HParams(beta=beta, step=t + 1, lr=float(np.float32(1e-2)), beta1=float(np.float32(0.9)),
                         beta2=float(np.float32(0.999)), eps=float(np.float32(1e-8)))
        V, m, u, l_mse, l_round, _ = fo.layer_step(Xb, host(Yg)[:, :mb].T, V, code, scales, sg, m, u, hpo, "bf16")
        torch.cuda.synchronize()
        lg = host(lay.loss)
        assert abs(lg[0] - l_mse) <= 2e-3 * max(l_mse, 1e-30) + 1e-12 and abs(lg[1] - l_round) <= 2e-3 * l_round, t
        from tests.gpu_helpers import rel_l2
        assert rel_l2(host(lay.V), V) <= 2e-3, t                 # each step starts from the GPU's previous state
        V, m, u = host(lay.V).copy(), host(lay.m).copy(), host(lay.u).copy()    # next step from the GPU's state
    lay.check()
    assert np.array_equal(host(res["V"]), host(lay.V))
    assert res["losses"] == host(lay.loss).tolist()
    p_o, _, _ = fo.harden_pack(host(res["V"]), code, scales, sg)
    assert np.array_equal(host(res["packed"]), p_o)


def test_decoder_block_driver_forms_the_mlp_input_and_covers_seven_linears(ctx):
    hid, ffn, kv, n, mb = 128, 256, 64, 256, 128
    rng = np.random.default_rng(5)
    dims = {"q_proj": (hid, hid), "k_proj": (kv, hid), "v_proj": (kv, hid), "o_proj": (hid, hid),
            "gate_proj": (ffn, hid), "up_proj": (ffn, hid), "down_proj": (hid, ffn)}
    Wn = {k: inputs.to_bf16_f32(inputs.weights(rng, *d, sigma=0.05)) for k, d in dims.items()}
    H = inputs.to_bf16_f32(inputs.hidden_states(rng, n, hid))
    Ho = inputs.to_bf16_f32(inputs.hidden_states(rng, n, hid, rms_norm=False))
    Wd = {k: dev_bf16(v) for k, v in Wn.items()}
    A = stage1.mlp_activation(ctx, Wd["gate_proj"], Wd["up_proj"], dev_bf16(H), mb)
    torch.cuda.synchronize()
    # the oracle on BF16-rounded GEMM outputs, as the device path stores them
    g = inputs.to_bf16_f32(fo.layer_ref(H, Wn["gate_proj"]))
    u = inputs.to_bf16_f32(fo.layer_ref(H, Wn["up_proj"]))
    ref = fo.silu_mul(g, u)
    got = host(A).astype(np.float64)
    # a GEMM output that lands on the other side of a BF16 boundary moves g or u by one step (2^-8)
    assert np.all(np.abs(got - ref) <= 2.0 ** -6 * np.abs(ref) + 2.0 ** -8 * np.abs(ref).max())
    from tests.gpu_helpers import rel_l2
    assert rel_l2(got, ref) <= 4e-3
    out = stage1.optimise_decoder_block(ctx, Wd, dev_bf16(H), dev_bf16(Ho), steps=4, mb=mb)
    assert sorted(out) == sorted(stage1.BLOCK_LINEARS)
    for name, (O, K) in dims.items():
        r = out[name]
        scales, sg, code, _ = fo.softquant_init(Wn[name])
        assert np.array_equal(host(r["code"]), code) and np.array_equal(host(r["scales"]), scales)
        p_o, _, _ = fo.harden_pack(host(r["V"]), code, scales, sg)
        assert np.array_equal(host(r["packed"]), p_o)
        assert np.isfinite(r["losses"]).all()
    part = stage1.optimise_decoder_block(ctx, Wd, dev_bf16(H), dev_bf16(Ho), steps=1, mb=mb, rank=1, world=4)
    assert sorted(part) == ["k_proj", "up_proj"]
