"""The deployable output: block scales in the tiled order of block-scaled tensor-core GEMMs (bit-exact
against the oracle's definition), and -- where this PyTorch exposes the hardware's NVFP4 GEMM -- the
packed E2M1 codes and tiled E4M3 scales of weights and activations fed to that GEMM as they are,
against the float64 product of the dequantised values.  The library GEMM is a checker here, not part
of the product path."""
import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from paper_2603_22370_b200 import faar, inputs
from tests.gpu_helpers import DEV, GpuLayer, dev_bf16, dev_u8, host, max_rel_to_peak, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2603_22370_b200 import build
    build.build()
    c = faar.Context(0)
    yield c
    torch.cuda.synchronize()
    c.close()


def _tiled(ctx, scales_dev, rows, cols):
    n = -(-rows // 128) * -(-cols // 4) * 512
    out = torch.full((n,), 0xAB, dtype=torch.uint8, device=DEV)
    faar.swizzle_scales(ctx, rows, cols, scales_dev, out)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("rows,cols", [(128, 4), (130, 5), (300, 65), (1, 1), (2048, 512)])
def test_swizzle_scales_bit_exact(ctx, rows, cols):
    sc = np.random.default_rng(rows).integers(0, 0x7F, size=(rows, cols)).astype(np.uint8)
    out = _tiled(ctx, dev_u8(sc), rows, cols)
    assert np.array_equal(host(out), fo.swizzle_scales(sc))


def test_packed_output_runs_on_the_nvfp4_tensor_core_gemm(ctx):
    if not hasattr(torch, "float4_e2m1fn_x2"):
        pytest.skip("this PyTorch has no packed FP4 dtype")
    O, K, T = 256, 512, 384
    W, X = inputs.config2(4, O, K, T)
    lay = GpuLayer(ctx, W, X)
    lay.init()
    lay.V.copy_(torch.rand_like(lay.V))                      # arbitrary rounding decisions
    packed_w = torch.empty((O, K // 2), dtype=torch.uint8, device=DEV)
    faar.harden_pack(ctx, lay.shape, lay.V, lay.code, lay.scales, lay.s_global, packed_w, None, None, None)
    ws = lay.ws
    Xq = torch.empty((T, K), dtype=torch.bfloat16, device=DEV)
    sx = torch.empty(1, dtype=torch.float32, device=DEV)
    packed_x = torch.empty((T, K // 2), dtype=torch.uint8, device=DEV)
    scales_x = torch.empty((T, K // 16), dtype=torch.uint8, device=DEV)
    faar.act_fakequant(ctx, T, K, lay.X, K, 0.0, Xq, K, sx, packed_x, scales_x, ws)
    tiled_w = _tiled(ctx, lay.scales, O, K // 16)
    tiled_x = _tiled(ctx, scales_x, T, K // 16)
    lay.check()
    # float64 product of the dequantised operands (tensor scales applied at the end)
    _, _, Wf = fo.harden_pack(host(lay.V), host(lay.code), host(lay.scales), host(lay.s_global)[0])
    units_x = host(Xq).astype(np.float64)
    sg_w = float(host(lay.s_global)[0])
    Y_o = (units_x * float(host(sx)[0])) @ Wf.astype(np.float64).T
    try:
        a = packed_x.view(torch.float4_e2m1fn_x2)
        b = packed_w.view(torch.float4_e2m1fn_x2).t()
        y = torch._scaled_mm(a, b, tiled_x.view(torch.float8_e4m3fn), tiled_w.view(torch.float8_e4m3fn),
                             out_dtype=torch.bfloat16)
        torch.cuda.synchronize()
    except Exception as exc:                                 # the checker is unavailable, not the product
        pytest.skip(f"NVFP4 scaled_mm not available in this PyTorch build: {type(exc).__name__}: {exc}")
    Y_g = host(y).astype(np.float64) * float(host(sx)[0]) * sg_w
    assert rel_l2(Y_g, Y_o) <= 4e-3 and max_rel_to_peak(Y_g, Y_o) <= 8e-3     # BF16 output of the library GEMM


def _deployable_operands(ctx, O, K, T, seed):
    """Hardened weights and quantised activations of a layer, as the library's own calls produce them."""
    W, X = inputs.config2(seed, O, K, T)
    lay = GpuLayer(ctx, W, X)
    lay.init()
    g = torch.Generator(device=DEV).manual_seed(seed)
    lay.V.copy_(torch.rand(lay.V.shape, device=DEV, generator=g))     # arbitrary rounding decisions
    packed_w = torch.empty((O, K // 2), dtype=torch.uint8, device=DEV)
    scales_w = torch.empty((O, K // 16), dtype=torch.uint8, device=DEV)
    faar.harden_pack(ctx, lay.shape, lay.V, lay.code, lay.scales, lay.s_global, packed_w, scales_w, None, None)
    Xq = torch.empty((T, K), dtype=torch.bfloat16, device=DEV)
    sx = torch.empty(1, dtype=torch.float32, device=DEV)
    packed_x = torch.empty((T, K // 2), dtype=torch.uint8, device=DEV)
    scales_x = torch.empty((T, K // 16), dtype=torch.uint8, device=DEV)
    faar.act_fakequant(ctx, T, K, lay.X, K, 0.0, Xq, K, sx, packed_x, scales_x, lay.ws)
    tiled_w = _tiled(ctx, scales_w, O, K // 16)
    tiled_x = _tiled(ctx, scales_x, T, K // 16)
    lay.check()
    return lay, (packed_x, scales_x, tiled_x, sx), (packed_w, scales_w, tiled_w, lay.s_global)


def _check_nvfp4_gemm(ctx, O, K, T, seed, sample=None):
    lay, (px, sx_lin, sx_tiled, sx), (pw, sw_lin, sw_tiled, sw) = _deployable_operands(ctx, O, K, T, seed)
    ldc = O + 8
    Y = torch.full((T, ldc), 7.0, dtype=torch.bfloat16, device=DEV)
    faar.nvfp4_gemm(ctx, T, O, K, px, sx_tiled, sx, pw, sw_tiled, sw, Y, ldc, lay.ws)
    lay.check()
    assert torch.all(Y[:, O:] == 7.0)                               # the padding of the output rows is untouched
    rows = np.arange(T) if sample is None else np.random.default_rng(seed).choice(T, sample, replace=False)
    pxh, sxh = host(px)[rows], host(sx_lin)[rows]
    A = fo.dequant_packed(pxh, sxh, host(sx)[0]).astype(np.float64)
    B = fo.dequant_packed(host(pw), host(sw_lin), host(sw)[0]).astype(np.float64)
    ref = fo.nvfp4_matmul(pxh, sxh, host(sx)[0], host(pw), host(sw_lin), host(sw)[0])
    got = host(Y[:, :O])[rows].astype(np.float64)
    # BF16 result (2^-9 relative, taken as 2^-8) of an FP32 accumulation whose error is bounded against the
    # sum of the magnitudes of the products
    bound = 2.0 ** -8 * np.abs(ref) + 1e-5 * (np.abs(A) @ np.abs(B).T)
    assert np.all(np.abs(got - ref) <= bound), float(np.max(np.abs(got - ref) / bound))
    assert rel_l2(got, ref) <= 3e-3
    return lay, Y


@pytest.mark.parametrize("O,K,T", [(256, 512, 384), (128, 64, 128), (200, 96, 77), (130, 1056, 300), (1, 32, 1)])
def test_own_nvfp4_gemm_on_the_deployable_operands(ctx, O, K, T):
    """The library's block-scaled FP4 GEMM, fed the packed codes, tiled E4M3 scales and tensor scales that its own
    hardening and activation-quantisation calls produce, against the float64 product of the decoded operands:
    one tile; one MMA; ragged rows, columns and a contraction that ends inside a 256-element stage; several
    tiles per CTA's pipeline; the smallest problem."""
    _check_nvfp4_gemm(ctx, O, K, T, seed=O + K)


def test_own_nvfp4_gemm_at_the_down_proj_size(ctx):
    """2048 x 8192 weights, 4096 tokens: every output column of 64 sampled tokens against the oracle."""
    _check_nvfp4_gemm(ctx, 2048, 8192, 4096, seed=1, sample=64)


def test_own_nvfp4_gemm_agrees_with_the_layer_path(ctx):
    """X_q W_final^T computed two ways by this library: the FP4 GEMM on the packed operands, and the BF16
    tensor-core GEMM (frozen-target call) on the same values written out in BF16 (activations: units times
    the tensor scale applied afterwards; weights: W_final)."""
    O, K, T = 256, 512, 384
    lay, Y4 = _check_nvfp4_gemm(ctx, O, K, T, seed=9)
    Wf = torch.empty((O, K), dtype=torch.bfloat16, device=DEV)
    packed = torch.empty((O, K // 2), dtype=torch.uint8, device=DEV)
    faar.harden_pack(ctx, lay.shape, lay.V, lay.code, lay.scales, lay.s_global, packed, None, None, Wf, faar.BF16)
    Xq = torch.empty((T, K), dtype=torch.bfloat16, device=DEV)
    sx = torch.empty(1, dtype=torch.float32, device=DEV)
    faar.act_fakequant(ctx, T, K, lay.X, K, 0.0, Xq, K, sx, None, None, lay.ws)
    Yb = torch.empty((T, O), dtype=torch.float32, device=DEV)
    shape = faar.make_shape(O, K, T, yref_dtype=faar.F32)
    faar.layer_ref(ctx, shape, Xq, Wf, Yb, lay.ws)
    lay.check()
    a, b = host(Y4[:, :O]).astype(np.float64), host(Yb).astype(np.float64) * float(host(sx)[0])
    # W_final in BF16 carries one more rounding (s_g * s_global rounded to 8 bits) than the FP4 path
    assert rel_l2(a, b) <= 6e-3


def test_nvfp4_gemm_argument_checks(ctx):
    lay, (px, _, sxt, sx), (pw, _, swt, sw) = _deployable_operands(ctx, 128, 64, 128, 3)
    Y = torch.empty((128, 128), dtype=torch.bfloat16, device=DEV)
    import ctypes as C
    lib = faar.lib()

    def call(M=128, N=128, K=64, A=px, ldc=128, ws=lay.ws, ws_bytes=None):
        return lib.faar_nvfp4_gemm(ctx._h, M, N, K, A.data_ptr(), sxt.data_ptr(), sx.data_ptr(), pw.data_ptr(), swt.data_ptr(),
                                   sw.data_ptr(), Y.data_ptr(), ldc, ws.data_ptr(), ws.numel() if ws_bytes is None else ws_bytes)

    assert call() == faar.OK
    assert call(K=48) == faar.ERR_SHAPE and call(M=0) == faar.ERR_SHAPE and call(ldc=64) == faar.ERR_SHAPE
    assert call(A=px.view(-1)[1:]) == faar.ERR_ALIGN
    assert call(ws_bytes=16) == faar.ERR_WORKSPACE
    lay.check()
