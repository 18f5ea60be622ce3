"""faar_round_loss_static: the Round Loss entry point that allocates nothing.

It exists for callers that cannot hand the library a workspace because they are
not allowed to allocate device memory at all (code living inside another
runtime's memory pool, or a loop in which a cudaMalloc would stall the device).
Its scratch is a fixed array inside libfaar.so that all calls on a device share
and that keeps the previous call's contents, so the checks below run it twice in
a row, the second time on a shorter tensor, and compare each result with the
workspace-based faar_round_loss and with the CPU oracle.

This file is collected last on purpose: a run that stops at the first failure
has then already gone through every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import faar_oracle as fo
from paper_2603_22370_b200 import faar
from tests.gpu_helpers import DEV, dev_f32, host

pytestmark = pytest.mark.gpu

REL_TOL = 1e-5          # the tolerance the workspace-based Round Loss test uses


@pytest.fixture(scope="module")
def ctx():
    from paper_2603_22370_b200 import build
    build.build()
    c = faar.Context(0)
    yield c
    torch.cuda.synchronize()
    c.close()


def test_two_calls_in_a_row_match_the_workspace_entry_point(ctx):
    ws = ctx.workspace(faar.make_shape(16, 16, 8))
    rng = np.random.default_rng(7)
    out_static = torch.zeros(1, device=DEV)
    out_ws = torch.zeros(1, device=DEV)
    # long first, short second: the second call must not see the first call's partial sums
    for n in [3 * 1024 * 1024 + 5, 4096 + 3, 17]:
        V = rng.uniform(0, 1, n).astype(np.float32)
        Vd = dev_f32(V)
        faar.round_loss_static(ctx, Vd, n, out_static)
        torch.cuda.synchronize()
        faar.round_loss(ctx, Vd, n, out_ws, ws)
        torch.cuda.synchronize()
        a, b, ref = float(host(out_static)[0]), float(host(out_ws)[0]), fo.round_loss(V)
        assert abs(a - b) <= REL_TOL * abs(b), (n, a, b)
        assert abs(a - ref) <= REL_TOL * ref, (n, a, ref)


def test_same_input_twice_gives_the_same_bits(ctx):
    V = dev_f32(np.random.default_rng(1).uniform(0, 1, 1000003).astype(np.float32))
    o1, o2 = torch.zeros(1, device=DEV), torch.zeros(1, device=DEV)
    faar.round_loss_static(ctx, V, V.numel(), o1)
    faar.round_loss_static(ctx, V, V.numel(), o2)
    torch.cuda.synchronize()
    assert host(o1).view(np.uint32)[0] == host(o2).view(np.uint32)[0]


def test_sizes_beyond_the_fixed_scratch_are_refused(ctx):
    limit = faar.round_loss_static_max_n()
    assert limit == 65536 * 4096
    V = torch.zeros(16, device=DEV)
    out = torch.full((1,), -1.0, device=DEV)
    for n in [limit + 1, 0, -4]:
        st = faar.lib().faar_round_loss_static(ctx._h, C.c_void_p(V.data_ptr()), C.c_int64(n),
                                               C.c_void_p(out.data_ptr()))
        assert st == faar.ERR_SHAPE
    torch.cuda.synchronize()
    assert host(out)[0] == -1.0            # nothing was launched
    st = faar.lib().faar_round_loss_static(ctx._h, C.c_void_p(V.data_ptr() + 4), C.c_int64(8),
                                           C.c_void_p(out.data_ptr()))
    assert st == faar.ERR_ALIGN
