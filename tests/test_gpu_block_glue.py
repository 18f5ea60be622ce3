"""GPU parity of the element-wise pieces of a decoder block (RMSNorm forward / backward, rotary position
embedding, the gated product's backward, embedding gather) against the Stage-2 oracle on the same BF16 inputs.
Outputs are BF16 roundings of FP32 evaluations: an element may differ from the float64 value by half a BF16
step (at most 2^-8 of its magnitude) plus the FP32 evaluation's own error."""
import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from oracle import stage2_oracle as so
from paper_2603_22370_b200 import faar, inputs
from tests.gpu_helpers import DEV, dev_bf16, dev_f32, host

pytestmark = pytest.mark.gpu
BF16_HALF_STEP = 2.0 ** -8


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


def close_bf16(got, ref, extra_abs=0.0):
    return np.all(np.abs(got - ref) <= (BF16_HALF_STEP + 1e-5) * np.abs(ref) + extra_abs + 1e-30)


@pytest.mark.parametrize("rows,cols,ld", [(77, 136, 144), (5, 2048, 2048), (300, 8, 8), (9, 2056, 2064), (3, 4096, 4096)])
def test_rmsnorm_forward_and_backward(ctx, rows, cols, ld):
    rng = np.random.default_rng(rows)
    x = inputs.to_bf16_f32(rng.standard_normal((rows, cols)) * 2)
    x[0, :] *= 32.0                                                    # a row with a large norm (still BF16 values)
    g = inputs.to_bf16_f32(rng.uniform(0.5, 1.5, cols)).astype(np.float32)
    dy = inputs.to_bf16_f32(rng.standard_normal((rows, cols)))
    res = inputs.to_bf16_f32(rng.standard_normal((rows, cols)))
    eps = float(np.float32(1e-5))
    X, DY, R = padded(x, ld), padded(dy, ld), padded(res, ld)
    Y = torch.full((rows, ld), 5.0, dtype=torch.bfloat16, device=DEV)
    rstd = torch.zeros(rows, dtype=torch.float32, device=DEV)
    faar.rmsnorm(ctx, rows, cols, X, ld, dev_f32(g), eps, Y, ld, rstd)
    torch.cuda.synchronize()
    y_o, rstd_o = so.rmsnorm(x, g, eps)
    assert np.allclose(host(rstd), rstd_o, rtol=2e-6)
    assert close_bf16(host(Y[:, :cols]).astype(np.float64), y_o)
    assert torch.all(Y[:, cols:] == 5.0)
    # backward, alone and added to a residual gradient; the oracle takes the GPU's FP32 rstd
    for add in (None, R):
        DX = torch.full((rows, ld), 5.0, dtype=torch.bfloat16, device=DEV)
        faar.rmsnorm_bwd(ctx, rows, cols, DY, ld, X, ld, dev_f32(g), rstd, add, ld, DX, ld)
        torch.cuda.synchronize()
        r64 = host(rstd).astype(np.float64)[:, None]
        ref = so.rmsnorm_bwd(dy, x, g, r64[:, 0]) + (res if add is not None else 0.0)
        # dx = rstd * (w - xh * mean(w * xh)) is a difference of two terms (plus the residual): the FP32 error is
        # bounded against their sizes, the BF16 rounding against the result
        w, xh = dy * g, x * r64
        terms = r64 * (np.abs(w) + np.abs(xh) * np.abs(np.mean(w * xh, axis=1, keepdims=True))) + (np.abs(res) if add is not None else 0.0)
        got = host(DX[:, :cols]).astype(np.float64)
        assert np.all(np.abs(got - ref) <= BF16_HALF_STEP * np.abs(ref) + 1e-5 * terms + 1e-30)
        assert torch.all(DX[:, cols:] == 5.0)
    # in place on the residual gradient
    faar.rmsnorm_bwd(ctx, rows, cols, DY, ld, X, ld, dev_f32(g), rstd, R, ld, R, ld)
    torch.cuda.synchronize()
    assert torch.equal(R[:, :cols], DX[:, :cols])


@pytest.mark.parametrize("rows,cols,ld", [(77, 136, 144), (40, 2048, 2048), (9, 2056, 2064), (3, 4096, 4096)])
def test_residual_add_fused_with_the_norm_and_gradient_sums_inside_its_backward(ctx, rows, cols, ld):
    """Rows of up to 2048 elements stay in registers, longer ones are read twice: both forms, ragged widths."""
    rng = np.random.default_rng(cols + rows)
    a = inputs.to_bf16_f32(rng.standard_normal((rows, cols)) * 2)
    b = inputs.to_bf16_f32(rng.standard_normal((rows, cols)))
    g = inputs.to_bf16_f32(rng.uniform(0.5, 1.5, cols)).astype(np.float32)
    eps = float(np.float32(1e-5))
    A, B, G = padded(a, ld), padded(b, ld), dev_f32(g)
    # forward: the same bits as faar_add followed by faar_rmsnorm
    S1 = torch.full((rows, ld), 5.0, dtype=torch.bfloat16, device=DEV)
    Y1 = torch.full((rows, ld), 5.0, dtype=torch.bfloat16, device=DEV)
    r1 = torch.zeros(rows, dtype=torch.float32, device=DEV)
    faar.add(ctx, rows, cols, A, ld, B, ld, S1, ld)
    faar.rmsnorm(ctx, rows, cols, S1, ld, G, eps, Y1, ld, r1)
    S2, Y2, r2 = torch.full_like(S1, 5.0), torch.full_like(Y1, 5.0), torch.zeros_like(r1)
    faar.add_rmsnorm(ctx, rows, cols, A, ld, B, ld, S2, ld, G, eps, Y2, ld, r2)
    torch.cuda.synchronize()
    assert torch.equal(S2, S1) and torch.equal(Y2, Y1) and torch.equal(r2, r1)
    # ... and against the oracle: the sum is one BF16 rounding of a + b, the norm is taken of the rounded sum
    s_o = a.astype(np.float64) + b.astype(np.float64)
    assert close_bf16(host(S2[:, :cols]).astype(np.float64), s_o, extra_abs=1e-37)
    y_o, rstd_o = so.rmsnorm(host(S2[:, :cols]).astype(np.float64), g, eps)
    assert np.allclose(host(r2), rstd_o, rtol=2e-6) and close_bf16(host(Y2[:, :cols]).astype(np.float64), y_o)
    A2 = A.clone()
    faar.add_rmsnorm(ctx, rows, cols, A2, ld, B, ld, A2, ld, G, eps, Y2, ld, None)     # sum in place, no rstd wanted
    torch.cuda.synchronize()
    assert torch.equal(A2[:, :cols], S1[:, :cols]) and torch.equal(Y2, Y1)

    # backward with one, two and three gradients meeting at the norm's output
    x = host(S1[:, :cols]).astype(np.float64)
    dys = [inputs.to_bf16_f32(rng.standard_normal((rows, cols))) for _ in range(3)]
    res = inputs.to_bf16_f32(rng.standard_normal((rows, cols)))
    D = [padded(t, ld) for t in dys]
    R = padded(res, ld)
    r64 = host(r1).astype(np.float64)[:, None]
    for n in (1, 2, 3):
        for add in (None, R):
            DX = torch.full((rows, ld), 5.0, dtype=torch.bfloat16, device=DEV)
            faar.rmsnorm_bwd_sum(ctx, rows, cols, D[0], D[1] if n > 1 else None, D[2] if n > 2 else None, ld, S1, ld, G, r1,
                                 add, ld, DX, ld)
            torch.cuda.synchronize()
            dy = sum(t.astype(np.float64) for t in dys[:n])
            ref = so.rmsnorm_bwd(dy, x, g, r64[:, 0]) + (res if add is not None else 0.0)
            w, xh = dy * g, x * r64
            terms = r64 * (np.abs(w) + np.abs(xh) * np.abs(np.mean(w * xh, axis=1, keepdims=True))) + (np.abs(res) if add is not None else 0.0)
            got = host(DX[:, :cols]).astype(np.float64)
            assert np.all(np.abs(got - ref) <= BF16_HALF_STEP * np.abs(ref) + 1e-5 * terms + 1e-30), (n, add is not None)
            assert torch.all(DX[:, cols:] == 5.0)
            if n == 1:
                DX1 = torch.full_like(DX, 5.0)
                faar.rmsnorm_bwd(ctx, rows, cols, D[0], ld, S1, ld, G, r1, add, ld, DX1, ld)
                torch.cuda.synchronize()
                assert torch.equal(DX1, DX)
    with pytest.raises(faar.FaarError) as e:
        faar.rmsnorm_bwd_sum(ctx, rows, cols, D[0], None, D[2], ld, S1, ld, G, r1, None, ld, DX, ld)
    assert e.value.status == faar.ERR_INVALID_ARG


@pytest.mark.parametrize("n_heads,head_dim", [(3, 16), (8, 64), (2, 128), (12, 64), (4, 128)])
def test_rope_forward_inverse_and_in_place(ctx, n_heads, head_dim):
    rng = np.random.default_rng(head_dim)
    T = 50
    pos = rng.integers(0, 2048, T).astype(np.int32)
    pos[:3] = [0, 1, 2047]
    x = inputs.to_bf16_f32(rng.standard_normal((T, n_heads * head_dim)))
    cols = n_heads * head_dim
    ld = cols + 8
    X = padded(x, ld)
    P = torch.from_numpy(pos).to(DEV)
    theta = 10000.0
    for inverse in (0, 1):
        Y = torch.full((T, ld), 5.0, dtype=torch.bfloat16, device=DEV)
        faar.rope(ctx, T, n_heads, head_dim, X, ld, P, theta, inverse, Y, ld)
        torch.cuda.synchronize()
        ref = so.rope(x, pos, n_heads, head_dim, theta, inverse=bool(inverse))
        # FP32 angles: position * frequency carries an absolute error of about 2^-24 * 2048 radians
        pair_mag = np.abs(x).reshape(T, n_heads, 2, head_dim // 2).max(axis=2).repeat(2, axis=1).reshape(T, cols)
        assert np.all(np.abs(host(Y[:, :cols]).astype(np.float64) - ref) <= BF16_HALF_STEP * np.abs(ref) + 3e-4 * 2 * pair_mag + 1e-30)
        assert torch.all(Y[:, cols:] == 5.0)
        assert torch.equal(Y[0, :cols], X[0, :cols])                   # position 0: identity
    faar.rope(ctx, T, n_heads, head_dim, X, ld, P, theta, 1, X, ld)    # in place
    torch.cuda.synchronize()
    assert torch.equal(X[:, :cols], Y[:, :cols])


def test_silu_mul_backward(ctx):
    rng = np.random.default_rng(4)
    rows, cols, ld = 77, 136, 144
    g = inputs.to_bf16_f32(rng.standard_normal((rows, cols)) * 3)
    u = inputs.to_bf16_f32(rng.standard_normal((rows, cols)))
    d = inputs.to_bf16_f32(rng.standard_normal((rows, cols)))
    g[0, :4] = [0.0, 40.0, -40.0, -100.0]
    G, U, D = padded(g, ld), padded(u, ld), padded(d, ld)
    DG = torch.full((rows, ld), 5.0, dtype=torch.bfloat16, device=DEV)
    DU = torch.full((rows, ld), 5.0, dtype=torch.bfloat16, device=DEV)
    faar.silu_mul_bwd(ctx, rows, cols, D, ld, G, ld, U, ld, DG, ld, DU, ld)
    torch.cuda.synchronize()
    dg_o, du_o = so.silu_mul_bwd(d, g, u)
    assert close_bf16(host(DG[:, :cols]).astype(np.float64), dg_o, extra_abs=1e-37)
    assert close_bf16(host(DU[:, :cols]).astype(np.float64), du_o, extra_abs=1e-37)
    assert torch.all(DG[:, cols:] == 5.0) and torch.all(DU[:, cols:] == 5.0)
    faar.silu_mul_bwd(ctx, rows, cols, D, ld, G, ld, U, ld, G, ld, U, ld)        # in place on gate / up
    torch.cuda.synchronize()
    assert torch.equal(G[:, :cols], DG[:, :cols]) and torch.equal(U[:, :cols], DU[:, :cols])


def test_embedding_gather(ctx):
    rng = np.random.default_rng(5)
    vocab, hidden, T = 1000, 264, 333
    tab = inputs.to_bf16_f32(rng.standard_normal((vocab, hidden)))
    tok = rng.integers(0, vocab, T).astype(np.int32)
    tok[:4] = [0, vocab - 1, -1, vocab]                                # the last two are out of range
    out = torch.full((T, hidden + 8), 5.0, dtype=torch.bfloat16, device=DEV)
    faar.embedding(ctx, T, hidden, vocab, dev_bf16(tab), hidden, torch.from_numpy(tok).to(DEV), out, hidden + 8)
    torch.cuda.synchronize()
    ref = so.embedding(tab, np.clip(tok, 0, vocab - 1))
    ref[2:4] = 0.0
    assert np.array_equal(host(out[:, :hidden]).astype(np.float64), ref)
    assert torch.all(out[:, hidden:] == 5.0)


def test_glue_argument_checks(ctx):
    x = torch.zeros((8, 16), dtype=torch.bfloat16, device=DEV)
    g = torch.ones(16, dtype=torch.float32, device=DEV)
    pos = torch.zeros(8, dtype=torch.int32, device=DEV)
    for call, status in [
        (lambda: faar.rmsnorm(ctx, 8, 12, x, 16, g, 1e-5, x, 16), faar.ERR_SHAPE),
        (lambda: faar.rmsnorm(ctx, 8, 16, x, 8, g, 1e-5, x, 16), faar.ERR_SHAPE),
        (lambda: faar.rmsnorm(ctx, 8, 16, x, 16, g, -1.0, x, 16), faar.ERR_INVALID_ARG),
        (lambda: faar.rope(ctx, 8, 2, 8, x, 16, pos, 10000.0, 0, x, 16), faar.ERR_SHAPE),
        (lambda: faar.rope(ctx, 8, 1, 16, x, 16, pos, 0.5, 0, x, 16), faar.ERR_INVALID_ARG),
        (lambda: faar.embedding(ctx, 8, 16, 0, x, 16, pos, x, 16), faar.ERR_SHAPE),
        (lambda: faar.silu_mul_bwd(ctx, 8, 16, x, 16, x, 16, x, 16, x.view(-1)[1:], 16, x, 16), faar.ERR_ALIGN),
    ]:
        with pytest.raises(faar.FaarError) as e:
            call()
        assert e.value.status == status
