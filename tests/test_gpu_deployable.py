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
