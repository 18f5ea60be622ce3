"""The bounds-checking build of the library (libfaar_debug.so, -DFAAR_DEBUG): every store of the tensor-core
kernels' epilogues is checked against the extent of the tensor it writes, and an index outside it would be
skipped and recorded in the workspace status word.  A child process binds that build (FAAR_LIB) and runs the
forward / backward / step / frozen-target / input-gradient calls on ragged and tile-aligned shapes: the status must
stay 0 and the results must equal, bit for bit, those of the normal build."""
import os
import subprocess
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r'''
import sys, numpy as np, torch
sys.path.insert(0, sys.argv[1])
from paper_2603_22370_b200 import faar, inputs
from tests.gpu_helpers import GpuLayer, host, DEV, dev_bf16
ctx = faar.Context(0)
out = {}
for (O, K, T) in [(300, 1040, 603), (512, 256, 512), (129, 48, 9), (1500, 272, 3300)]:
    W, X = inputs.config2(3, O, K, T)
    for yt in (0, 1):
        lay = GpuLayer(ctx, W, X, yref_transposed=yt)
        lay.init()
        Y = torch.zeros((O, lay.shape.ldy) if yt else (T, O), dtype=torch.bfloat16, device=DEV)
        faar.layer_ref(ctx, lay.shape, lay.X, lay.W, Y, lay.ws)
        lay.Yref = Y
        for t in range(3):
            hp = faar.make_hparams(beta=4.0 + t, step=t + 1, wsoft_ready=int(t > 0), beta_next=5.0 + t if t < 2 else 0.0)
            lay.step(hp)
        Yq = lay.fwd(faar.make_hparams(beta=7.0), want_yq=True)
        dV = lay.bwd(faar.make_hparams(beta=7.0, step=4), want_dv=True)
        lay.check()                                   # raises if a checked store was out of range
        out[f"{O}x{K}x{T}.{yt}"] = np.concatenate([host(lay.V).ravel(), host(dV).ravel(), host(Yq).ravel(), host(lay.loss)])
    dY = dev_bf16(np.random.default_rng(0).standard_normal((T, (O + 7) // 8 * 8)))
    plain = faar.make_shape(O, K, T, ldy=(O + 7) // 8 * 8)
    WsT = torch.empty((K, (O + 7) // 8 * 8), dtype=torch.bfloat16, device=DEV)
    dX = torch.empty((T, K), dtype=torch.bfloat16, device=DEV)
    faar.layer_dx(ctx, plain, 6.0, dY, lay.V, lay.code, lay.scales, lay.s_global, WsT, dX, lay.ws)
    lay.check()
    out[f"{O}x{K}x{T}.dx"] = host(dX).ravel()
np.savez(sys.argv[2], **out)
print("child ok", faar.LIB_PATH)
'''


def run_child(tmp_path, lib, name):
    env = dict(os.environ)
    if lib:
        env["FAAR_LIB"] = lib
    else:
        env.pop("FAAR_LIB", None)
    path = str(tmp_path / name)
    res = subprocess.run([sys.executable, "-c", CHILD, ROOT, path], env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    return res.stdout, np.load(path)


def test_debug_build_reports_no_out_of_range_store_and_matches_the_normal_build(tmp_path):
    from paper_2603_22370_b200 import build
    build.build()
    dbg_lib = build.build(debug=True)
    o_dbg, dbg = run_child(tmp_path, dbg_lib, "dbg.npz")
    assert "libfaar_debug.so" in o_dbg
    o_ref, ref = run_child(tmp_path, None, "ref.npz")
    assert "libfaar.so" in o_ref
    assert sorted(dbg.files) == sorted(ref.files) and len(ref.files) == 12
    for k in ref.files:
        assert np.array_equal(dbg[k], ref[k]), k
