"""GPU parity of the attention kernels (forward, backward) against the Stage-2 oracle on the same BF16 inputs:
ragged sequence lengths (not a multiple of the 64-token tile), several sequences, grouped key/value heads, both
head sizes.  The kernels round the probabilities (and dS) to BF16 before the second matrix product, as every
tensor-core attention does, and store BF16 results: outputs are compared norm-wise and against the peak."""
import numpy as np
import pytest
import torch

from oracle import stage2_oracle as so
from paper_2603_22370_b200 import faar, inputs
from tests.gpu_helpers import DEV, dev_bf16, host, max_rel_to_peak, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2603_22370_b200 import build
    build.build()
    c = faar.Context(0)
    yield c
    torch.cuda.synchronize()
    c.close()


def padded(a, ld, fill=9.0):
    t = torch.full((a.shape[0], ld), fill, dtype=torch.bfloat16, device=DEV)
    t[:, :a.shape[1]] = dev_bf16(a)
    return t


@pytest.mark.parametrize("fragments", [0, 1, 2])
@pytest.mark.parametrize("B,S,H,HKV,D", [(2, 100, 4, 2, 64), (1, 64, 2, 2, 64), (3, 7, 2, 1, 64), (1, 200, 4, 1, 128),
                                         (2, 129, 8, 2, 64), (1, 321, 4, 4, 64)])
def test_attention_forward_and_backward_match_the_oracle(ctx, B, S, H, HKV, D, fragments):
    """fragments = 0: the default kernels (head_dim 64: forward and backward on tcgen05); 2: head_dim 64 with scores
    in registers (mma.sync) forward and backward; 1: head_dim 64 through the shared-memory fragment kernels that
    head_dim 128 always uses."""
    if fragments and D != 64:
        pytest.skip("head_dim 128 has one kind of kernel")
    faar.tune_attention(ctx, fragments)
    try:
        _attention_case(ctx, B, S, H, HKV, D)
    finally:
        faar.tune_attention(ctx, 0)


@pytest.mark.parametrize("q_scale", [3.0, 8.0])
def test_attention_with_peaked_scores(ctx, q_scale):
    """Scores whose row maxima keep growing along the key sweep by amounts on both sides of the forward kernel's
    slack (it moves a row's reference only past 2^8): the result must not depend on when the reference moves."""
    _attention_case(ctx, 2, 321, 4, 2, 64, q_scale=q_scale)


def _attention_case(ctx, B, S, H, HKV, D, q_scale=1.0):
    rng = np.random.default_rng(S + D)
    T = B * S
    q = inputs.to_bf16_f32(rng.standard_normal((T, H * D)) * q_scale)
    k = inputs.to_bf16_f32(rng.standard_normal((T, HKV * D)))
    v = inputs.to_bf16_f32(rng.standard_normal((T, HKV * D)))
    do = inputs.to_bf16_f32(rng.standard_normal((T, H * D)))
    ldq, ldk = H * D + 8, HKV * D + 16
    Q, K, V, DO = padded(q, ldq), padded(k, ldk), padded(v, ldk), padded(do, ldq)
    O = torch.full((T, ldq), 5.0, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros((B, H, S), dtype=torch.float32, device=DEV)
    faar.attention_fwd(ctx, B, S, H, HKV, D, Q, ldq, K, V, ldk, O, ldq, lse)
    torch.cuda.synchronize()
    faar.attention_status(ctx)
    out_o, P = so.attention(q, k, v, B, S, H, HKV, D)
    got = host(O[:, :H * D]).astype(np.float64)
    assert rel_l2(got, out_o) <= 6e-3 and max_rel_to_peak(got, out_o) <= 1e-2
    assert torch.all(O[:, H * D:] == 5.0)
    # lse (log2 domain) against the definition: log2 sum_u exp(score_u)
    qh = q.reshape(B, S, H, D).astype(np.float64)
    kh = k.reshape(B, S, HKV, D).astype(np.float64)
    for (b, h, t) in [(0, 0, 0), (B - 1, H - 1, S - 1), (0, H - 1, S // 2)]:
        sc = qh[b, t, h] @ kh[b, :t + 1, h // (H // HKV)].T / np.sqrt(D)
        ref = np.log2(np.sum(np.exp(sc - sc.max()))) + sc.max() * np.log2(np.e)
        assert abs(float(lse[b, h, t]) - ref) <= 1e-3 * max(1.0, abs(ref))
    # first token of every sequence attends to itself only
    for b in range(B):
        assert np.allclose(got.reshape(B, S, H, D)[b, 0], v.reshape(B, S, HKV, D)[b, 0].repeat(H // HKV, axis=0), atol=1e-2)

    # backward from the GPU's own out / lse
    dsum = torch.zeros((B, H, S), dtype=torch.float32, device=DEV)
    DQ = torch.full((T, ldq), 5.0, dtype=torch.bfloat16, device=DEV)
    DK = torch.full((T, ldk), 5.0, dtype=torch.bfloat16, device=DEV)
    DV = torch.full((T, ldk), 5.0, dtype=torch.bfloat16, device=DEV)
    faar.attention_bwd(ctx, B, S, H, HKV, D, Q, ldq, K, V, ldk, O, DO, ldq, lse, dsum, DQ, DK, DV)
    torch.cuda.synchronize()
    faar.attention_status(ctx)
    dq_o, dk_o, dv_o = so.attention_bwd(do, q, k, v, P, B, S, H, HKV, D)
    for name, g_t, ref, n in (("dq", DQ, dq_o, H * D), ("dk", DK, dk_o, HKV * D), ("dv", DV, dv_o, HKV * D)):
        g = host(g_t[:, :n]).astype(np.float64)
        assert rel_l2(g, ref) <= 1e-2 and max_rel_to_peak(g, ref) <= 2e-2, (name, rel_l2(g, ref), max_rel_to_peak(g, ref))
        assert torch.all(g_t[:, n:] == 5.0), name
    # reproducible: a second backward call gives the same bits
    DQ2, DK2, DV2 = torch.empty_like(DQ), torch.empty_like(DK), torch.empty_like(DV)
    faar.attention_bwd(ctx, B, S, H, HKV, D, Q, ldq, K, V, ldk, O, DO, ldq, lse, dsum, DQ2, DK2, DV2)
    torch.cuda.synchronize()
    assert torch.equal(DQ2[:, :H * D], DQ[:, :H * D]) and torch.equal(DK2[:, :HKV * D], DK[:, :HKV * D])


@pytest.mark.parametrize("fragments", [0, 2])
def test_attention_at_the_alignment_benchmark_size_on_sampled_head_groups(ctx, fragments):
    """4 sequences of 2048 tokens, 32 query / 8 key-value heads of 64 (the launch the full-model benchmark makes:
    dense rows, 16 query tiles per head, CTAs ordered by work over the whole launch).  Attention separates over
    (sequence, key/value head), so the oracle runs on three such groups, each with its 4 query heads, and every
    output of those groups is compared."""
    B, S, H, HKV, D = 4, 2048, 32, 8, 64
    G = H // HKV
    rng = np.random.default_rng(2048)
    T = B * S
    q = inputs.to_bf16_f32(rng.standard_normal((T, H * D)))
    k = inputs.to_bf16_f32(rng.standard_normal((T, HKV * D)))
    v = inputs.to_bf16_f32(rng.standard_normal((T, HKV * D)))
    do = inputs.to_bf16_f32(rng.standard_normal((T, H * D)))
    Q, K, V, DO = dev_bf16(q), dev_bf16(k), dev_bf16(v), dev_bf16(do)
    O = torch.empty_like(Q)
    lse = torch.zeros((B, H, S), dtype=torch.float32, device=DEV)
    dsum = torch.zeros_like(lse)
    DQ, DK, DV = torch.empty_like(Q), torch.empty_like(K), torch.empty_like(V)
    faar.tune_attention(ctx, fragments)
    try:
        faar.attention_fwd(ctx, B, S, H, HKV, D, Q, H * D, K, V, HKV * D, O, H * D, lse)
        faar.attention_bwd(ctx, B, S, H, HKV, D, Q, H * D, K, V, HKV * D, O, DO, H * D, lse, dsum, DQ, DK, DV)
        torch.cuda.synchronize()
        faar.attention_status(ctx)
    finally:
        faar.tune_attention(ctx, 0)
    got_o, got_dq = host(O).astype(np.float64), host(DQ).astype(np.float64)
    got_dk, got_dv = host(DK).astype(np.float64), host(DV).astype(np.float64)
    for (b, g) in [(0, 0), (3, 7), (1, 3)]:
        rows = slice(b * S, (b + 1) * S)
        qc, kc = slice(g * G * D, (g + 1) * G * D), slice(g * D, (g + 1) * D)
        out_o, P = so.attention(q[rows, qc], k[rows, kc], v[rows, kc], 1, S, G, 1, D)
        dq_o, dk_o, dv_o = so.attention_bwd(do[rows, qc], q[rows, qc], k[rows, kc], v[rows, kc], P, 1, S, G, 1, D)
        a = got_o[rows, qc]
        assert rel_l2(a, out_o) <= 6e-3 and max_rel_to_peak(a, out_o) <= 1e-2, (b, g)
        for name, a, ref in (("dq", got_dq[rows, qc], dq_o), ("dk", got_dk[rows, kc], dk_o), ("dv", got_dv[rows, kc], dv_o)):
            assert rel_l2(a, ref) <= 1e-2 and max_rel_to_peak(a, ref) <= 2e-2, (name, b, g, rel_l2(a, ref), max_rel_to_peak(a, ref))
        # lse (log2 domain) of the group's last query head at the last position
        h = (g + 1) * G - 1
        sc = q[rows, qc][S - 1, (G - 1) * D:].astype(np.float64) @ k[rows, kc].astype(np.float64).T / np.sqrt(D)
        ref = np.log2(np.sum(np.exp(sc - sc.max()))) + sc.max() * np.log2(np.e)
        assert abs(float(lse[b, h, S - 1]) - ref) <= 1e-3 * max(1.0, abs(ref))


def test_attention_argument_checks(ctx):
    x = torch.zeros((64, 128), dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(128, dtype=torch.float32, device=DEV)
    for kw, status in [(dict(D=32), faar.ERR_SHAPE), (dict(H=3, HKV=2), faar.ERR_SHAPE), (dict(ldq=64), faar.ERR_SHAPE),
                       (dict(ldq=132), faar.ERR_ALIGN)]:
        a = dict(B=1, S=64, H=2, HKV=1, D=64, ldq=128)
        a.update(kw)
        with pytest.raises(faar.FaarError) as e:
            faar.attention_fwd(ctx, a["B"], a["S"], a["H"], a["HKV"], a["D"], x, a["ldq"], x, x, 128, x, 128, lse)
        assert e.value.status == status
