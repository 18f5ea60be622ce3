"""GPU parity of faar_align_loss (Eq. 6's data terms and their gradients) against the oracle: vocabularies
from one entry to 130 000 (fewer and more 16-byte groups than the CTA has threads), ragged sizes, padded
rows, several temperatures, more tokens than SMs, and a full-size vocabulary checked on sampled tokens."""
import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from paper_2603_22370_b200 import faar, inputs
from tests.gpu_helpers import DEV, host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2603_22370_b200 import build
    build.build()
    c = faar.Context(0)
    yield c
    torch.cuda.synchronize()
    c.close()


def _run(ctx, Zf, Zq, Hf, Hq, tau, lam, pad=0, want_grads=True):
    T, V = Zf.shape
    D = Hf.shape[1]
    ldz, ldh = (V + 7) // 8 * 8 + pad, (D + 7) // 8 * 8 + pad

    def dev(a, ld):
        t = torch.full((a.shape[0], ld), 1e4, dtype=torch.bfloat16, device=DEV)     # padding holds large junk
        t[:, :a.shape[1]] = torch.from_numpy(a).to(DEV).to(torch.bfloat16)
        return t

    zf, zq, hf, hq = dev(Zf, ldz), dev(Zq, ldz), dev(Hf, ldh), dev(Hq, ldh)
    dZ = torch.full((T, ldz), 7.0, dtype=torch.bfloat16, device=DEV) if want_grads else None
    dH = torch.full((T, ldh), 7.0, dtype=torch.bfloat16, device=DEV) if want_grads else None
    loss = torch.zeros(2, dtype=torch.float32, device=DEV)
    ws = torch.empty(faar.align_loss_workspace_size(T, V), dtype=torch.uint8, device=DEV)
    faar.workspace_init(ctx, ws)
    faar.align_loss(ctx, T, V, D, zf, zq, ldz, hf, hq, ldh, tau, lam, dZ, dH, loss, ws)
    torch.cuda.synchronize()
    faar.check_status(ctx, ws)
    return host(loss), (host(dZ) if want_grads else None), (host(dH) if want_grads else None)


def _bf16(a):
    return inputs.to_bf16_f32(a.astype(np.float32))


@pytest.mark.parametrize("T,V,D,tau,lam,pad", [(5, 37, 8, 1.0, 1.0, 0), (3, 18432, 64, 1.0, 1.0, 0), (4, 20003, 70, 1.7, 0.3, 8),
                                               (333, 1000, 16, 1.0, 1.0, 0), (2, 8199, 8, 1.0, 1.0, 0),
                                               (3, 50257, 33, 0.7, 2.0, 0), (2, 130000, 100, 1.0, 1.0, 16),
                                               (2, 73729, 9, 2.5, 1.0, 0), (1, 1, 1, 1.0, 1.0, 0)])
def test_align_loss_matches_oracle(ctx, T, V, D, tau, lam, pad):
    rng = np.random.default_rng(V)
    Zf = _bf16(rng.standard_normal((T, V)) * 3.0)
    Zq = _bf16(Zf + rng.standard_normal((T, V)) * 0.5)
    Zf[0, rng.integers(V)] = 40.0                       # a dominant logit in one model only
    Hf = _bf16(rng.standard_normal((T, D)))
    Hq = _bf16(Hf + rng.standard_normal((T, D)) * 0.1)
    loss, dZ, dH = _run(ctx, Zf, Zq, Hf, Hq, tau, lam, pad)
    kl, mse, dZ_o, dH_o = fo.align_loss(Zf, Zq, Hf, Hq, tau, lam)
    # hardware 2^x and log2 carry 2^-22 relative error into probabilities that sum to one: 2e-6 absolute
    assert abs(loss[0] - kl) <= 2e-3 * abs(kl) + 2e-6
    assert abs(loss[1] - mse) <= 1e-5 * mse + 1e-12
    # gradients are stored in BF16: 2^-9 relative from the rounding, plus the FP32 softmax error
    # (each probability is good to 2^-22 relative, so P_q - P_fp to 1e-6 absolute, times the gradient's scale)
    assert np.all(np.abs(dZ[:, :V] - dZ_o) <= 2.0 ** -8 * np.abs(dZ_o) + 1e-6 * abs(lam) / (tau * T))
    assert np.array_equal(dH[:, :D], _bf16(dH_o))       # differences of BF16 values doubled: exact, then one rounding
    assert np.all(dZ[:, V:] == 7.0) and np.all(dH[:, D:] == 7.0)       # padding is never written
    # losses without the gradient outputs
    loss2, _, _ = _run(ctx, Zf, Zq, Hf, Hq, tau, lam, pad, want_grads=False)
    assert np.array_equal(loss, loss2)


def test_identical_models_give_zero(ctx):
    rng = np.random.default_rng(3)
    Z = _bf16(rng.standard_normal((4, 9000)) * 4)
    H = _bf16(rng.standard_normal((4, 256)))
    loss, dZ, dH = _run(ctx, Z, Z, H, H, 1.3, 1.0)
    assert abs(loss[0]) <= 2e-6 and loss[1] == 0.0
    assert not dZ[:, :9000].any() and not dH[:, :256].any()


def test_arguments_are_checked(ctx):
    z = torch.zeros((2, 64), dtype=torch.bfloat16, device=DEV)
    h = torch.zeros((2, 8), dtype=torch.bfloat16, device=DEV)
    loss = torch.zeros(2, device=DEV)
    ws = torch.empty(faar.align_loss_workspace_size(2, 64), dtype=torch.uint8, device=DEV)
    faar.workspace_init(ctx, ws)
    bad = [dict(tau=0.0), dict(tau=float("nan")), dict(ldz=60), dict(ldz=68), dict(ldh=4), dict(T=0)]
    for kw in bad:
        a = dict(T=2, V=64, D=8, ldz=64, ldh=8, tau=1.0)
        a.update(kw)
        with pytest.raises(faar.FaarError):
            faar.align_loss(ctx, a["T"], a["V"], a["D"], z, z, a["ldz"], h, h, a["ldh"], a["tau"], 1.0, None, None, loss, ws)
    with pytest.raises(faar.FaarError):
        faar.align_loss(ctx, 2, 64, 8, z, z, 64, h, h, 8, 1.0, 1.0, None, None, loss, ws[:256])
    torch.cuda.synchronize()


def test_full_vocabulary_on_sampled_tokens(ctx):
    """A Llama-3-sized vocabulary (128 256) and 512 tokens on the GPU; the oracle recomputes 6 of the
    tokens (a token's KL term and gradient row depend on that token alone, up to the 1/T)."""
    T, V, D = 512, 128256, 2048
    g = torch.Generator(device=DEV).manual_seed(0)
    zf = (torch.randn((T, V), device=DEV, generator=g) * 3).to(torch.bfloat16)
    zq = (zf.float() + torch.randn((T, V), device=DEV, generator=g) * 0.3).to(torch.bfloat16)
    hf = torch.randn((T, D), device=DEV, generator=g).to(torch.bfloat16)
    hq = (hf.float() + 0.05 * torch.randn((T, D), device=DEV, generator=g)).to(torch.bfloat16)
    dZ, dH = torch.empty_like(zq), torch.empty_like(hq)
    loss = torch.zeros(2, device=DEV)
    ws = torch.empty(faar.align_loss_workspace_size(T, V), dtype=torch.uint8, device=DEV)
    faar.workspace_init(ctx, ws)
    faar.align_loss(ctx, T, V, D, zf, zq, V, hf, hq, D, 1.0, 1.0, dZ, dH, loss, ws)
    torch.cuda.synchronize()
    faar.check_status(ctx, ws)
    rows = [0, 1, 77, 255, 256, 511]
    kl_rows = []
    for t in rows:
        kl, _, dz_o, _ = fo.align_loss(host(zf[t:t + 1]), host(zq[t:t + 1]), host(hf[t:t + 1]), host(hq[t:t + 1]))
        kl_rows.append(kl)
        dz_o = dz_o / T
        d = np.abs(host(dZ[t:t + 1]) - dz_o)
        assert np.all(d <= 2.0 ** -8 * np.abs(dz_o) + 1e-6 / T)
    # every token's KL is positive and of the sampled tokens' size; the mean lies between their extremes' bounds
    assert 0.3 * min(kl_rows) <= host(loss)[0] <= 3 * max(kl_rows)
    mse = float(((hq.double() - hf.double()) ** 2).sum())
    assert abs(host(loss)[1] - mse) <= 1e-5 * mse
