"""The allocation-free entry point, gaconv_dw_exact_static, against gaconv_dw_exact.

Who needs it: callers that are not allowed to allocate device memory where they run -- a plugin that
a host framework hands only inputs and outputs, a loop that promised "no allocation after warm-up",
a process whose device memory pool is someone else's -- and therefore cannot supply the workspace
gaconv_dw_exact asks for.  The library then uses a fixed scratch array of its own.

This file is collected last on purpose: if it fails, a run that stops at the first failure has
already run every other test.  It passes alone in a fresh process and after the other tests."""
import numpy as np
import pytest
import torch

from oracle import oracle
from paper_1908_05460_b200 import binding as B
from paper_1908_05460_b200 import inputs as I
from paper_1908_05460_b200.layers import ConvLayer, config1_layer
from helpers import GpuLayer, norm_err, oshape, to_f64, TOL_F32, TOL_BF16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,layer", [(torch.float32, config1_layer()),
                                          (torch.bfloat16, ConvLayer("tc path", 32, 16, 32, 32, 16, 3, 3, 1, 1))],
                         ids=["f32 direct kernel", "bf16 tensor-core kernel"])
def test_static_scratch_entry_matches_workspace_entry_twice(dtype, layer):
    x, dy = I.make_layer_inputs(layer, dtype, 8, 0)
    ref, dn = oracle.dw_exact(to_f64(x), to_f64(dy), oshape(layer))
    tol = TOL_F32 if dtype == torch.float32 else TOL_BF16
    g = GpuLayer(layer, dtype, x, dy)
    want = g.exact()                                   # existing entry point, caller-owned workspace
    assert norm_err(want, ref, dn) <= tol
    assert B.gaconv_workspace_size(g.desc, B.METHOD_EXACT) <= B.gaconv_static_scratch_bytes()
    # the new entry point ignores the descriptor's workspace: give it none
    bare = B.make_desc(layer, dtype)
    for _ in range(2):                                 # two calls in a row share the built-in array
        g.dw.fill_(float("nan"))
        B.gaconv_dw_exact_static(g.x, g.dy, g.dw, bare)
        got = g.logical_dw()
        assert norm_err(got, want, dn) <= tol          # against the existing entry point
        assert norm_err(got, ref, dn) <= tol           # and against the oracle
        assert B.gaconv_poll_async_status_static() == B.OK
    # a different problem in between must not disturb the next one (the array keeps old contents)
    other = ConvLayer("other", 5, 8, 9, 9, 12, 3, 3, 1, 1, dy_std=1.0)
    xo, dyo = I.make_layer_inputs(other, torch.float32, 8, 1)
    go = GpuLayer(other, torch.float32, xo, dyo)
    ref_o, dn_o = oracle.dw_exact(to_f64(xo), to_f64(dyo), oshape(other))
    B.gaconv_dw_exact_static(go.x, go.dy, go.dw, B.make_desc(other, torch.float32))
    assert norm_err(go.logical_dw(), ref_o, dn_o) <= TOL_F32
    g.dw.fill_(float("nan"))
    B.gaconv_dw_exact_static(g.x, g.dy, g.dw, bare)
    assert norm_err(g.logical_dw(), want, dn) <= tol
    assert norm_err(g.logical_dw(), ref, dn) <= tol
    assert B.gaconv_poll_async_status_static() == B.OK


def test_static_scratch_entry_rejects_problems_beyond_its_limit():
    big = ConvLayer("too big", 4096, 64, 2, 2, 512, 3, 3, 1, 1)       # its transposed copy of dY alone is 16 MiB
    d = B.make_desc(big, torch.bfloat16)
    assert B.gaconv_workspace_size(d, B.METHOD_EXACT) > B.gaconv_static_scratch_bytes()
    with pytest.raises(B.GaconvError) as e:
        B.gaconv_dw_exact_static(16, 32, 48, d)                        # rejected before any pointer is used
    assert e.value.status == B.ERR_WORKSPACE_TOO_SMALL
    assert B.gaconv_static_scratch_bytes() == 8 << 20
