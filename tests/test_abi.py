"""CPU-only checks of the boundary: the library loads, exports what the header declares, validates
arguments without touching a GPU, and its schedule driver agrees with the schedule oracle."""
import ctypes
import os
import re

import pytest
import torch

from oracle import schedule_oracle as so
from paper_1908_05460_b200 import binding as B
from paper_1908_05460_b200 import build as build_mod
from paper_1908_05460_b200.layers import ConvLayer, config1_layer, resnet20_layers, vgg19_layers, cnn2_layers

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build_mod.build()
    B.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "gaconv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gaconv_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    lib = ctypes.CDLL(B.LIB_PATH)
    names = declared_symbols()
    assert len(names) >= 12
    for name in names:
        assert hasattr(lib, name), name
    assert set(B.EXPORTS) == set(names)


def test_status_strings():
    assert B.status_string(B.OK) == "ok"
    assert len({B.status_string(i) for i in range(8)}) == 8


def test_workspace_size_and_descriptor_validation():
    d = B.make_desc(config1_layer(), torch.float32)
    for m in (B.METHOD_EXACT, B.METHOD_ZERO, B.METHOD_RANDOM, B.METHOD_TOP1):
        assert B.gaconv_workspace_size(d, m) >= 256
    bad = B.make_desc(config1_layer(), torch.float32); bad.struct_size = 4
    with pytest.raises(B.GaconvError) as e:
        B.gaconv_workspace_size(bad, B.METHOD_EXACT)
    assert e.value.status == B.ERR_BAD_DESC
    for field, value in (("n", 0), ("c", -1), ("stride_h", 0), ("pad_w", -1), ("in_dtype", 7), ("x_layout", 9),
                         ("dw_layout", 5), ("dy_layout", 3), ("r", 99)):
        bad = B.make_desc(config1_layer(), torch.float32); setattr(bad, field, value)
        with pytest.raises(B.GaconvError) as e:
            B.gaconv_workspace_size(bad, B.METHOD_TOP1)
        assert e.value.status == B.ERR_BAD_DESC, field
    with pytest.raises(B.GaconvError) as e:
        B.gaconv_workspace_size(d, 17)
    assert e.value.status == B.ERR_BAD_DESC


def test_pointer_validation_enqueues_nothing():
    lib = B.load()
    d = B.make_desc(config1_layer(), torch.float32)
    ref = ctypes.byref(d)
    assert lib.gaconv_dw_exact(None, None, None, ref, None) == B.ERR_NULL_POINTER
    assert lib.gaconv_dw_exact(16, 32, 48, None, None) == B.ERR_NULL_POINTER
    assert lib.gaconv_dw_exact(16, 32, 52, ref, None) == B.ERR_MISALIGNED
    assert lib.gaconv_dw_exact(16, 32, 48, ref, None) == B.ERR_NULL_POINTER          # no workspace attached
    d.workspace, d.workspace_bytes = 4096, 8
    assert lib.gaconv_dw_exact(16, 32, 48, ref, None) == B.ERR_WORKSPACE_TOO_SMALL
    assert lib.gaconv_dw_approx(B.METHOD_TOP1, 16, 32, 48, ref, 0, None) == B.ERR_WORKSPACE_TOO_SMALL
    assert lib.gaconv_dw_approx(B.METHOD_TOP1, None, 32, 48, ref, 0, None) == B.ERR_NULL_POINTER
    assert lib.gaconv_dw_approx(5, 16, 32, 48, ref, 0, None) == B.ERR_BAD_DESC
    assert lib.gaconv_dw_approx(B.METHOD_ZERO, None, None, None, ref, 0, None) == B.ERR_NULL_POINTER
    assert lib.gaconv_approx_select(16, None, 48, None, ref, None) == B.ERR_NULL_POINTER
    assert lib.gaconv_approx_select(16, 36, 48, None, ref, None) == B.ERR_MISALIGNED
    assert lib.gaconv_workspace_init(None, 1 << 20, None) == B.ERR_NULL_POINTER
    assert lib.gaconv_workspace_init(4096, 8, None) == B.ERR_WORKSPACE_TOO_SMALL
    assert lib.gaconv_poll_async_status(None, None) == B.ERR_NULL_POINTER


def test_layer_sets_match_the_networks():
    rn, vg, cn = resnet20_layers(), vgg19_layers(), cnn2_layers()
    assert (len(rn), len(vg), len(cn)) == (19, 16, 2)
    assert [(l.c, l.k, l.h, l.stride) for l in rn[:2]] == [(3, 16, 32, 1), (16, 16, 32, 1)]
    assert (rn[7].p, rn[13].p, rn[-1].p) == (16, 8, 8)
    assert [l.h for l in vg] == [32, 32, 16, 16, 8, 8, 8, 8, 4, 4, 4, 4, 2, 2, 2, 2]
    assert all(l.p == l.h for l in vg) and cn[0].p == 32 and cn[1].p == 16
    assert ConvLayer("t", 1, 1, 7, 7, 1, 3, 3, 2, 1).p == 4


@pytest.mark.parametrize("kind", range(5))
def test_schedule_driver_matches_schedule_oracle(kind):
    for L in (2, 5, 16, 19):
        for frac, seed in ((0.0, 1), (0.25, 2), (0.5, 3), (0.75, 4), (1.0, 5)):
            s = B.Schedule(L, kind, B.METHOD_TOP1, frac, seed)
            for step in range(8):
                got = [s.method(l, step) for l in range(L)]
                want = [B.METHOD_TOP1 if so.approximated(kind, L, l, step, frac, seed) else B.METHOD_EXACT
                        for l in range(L)]
                assert got == want, (kind, L, frac, step)
            assert s.method(L, 0) == -2 and s.method(-1, 0) == -2 and s.method(0, -1) == -2
            s.close()


def test_schedule_create_rejects_bad_arguments():
    for args in ((0, 0, B.METHOD_TOP1, 0.0, 0), (4, 9, B.METHOD_TOP1, 0.0, 0), (4, 0, 7, 0.0, 0),
                 (4, 4, B.METHOD_ZERO, 1.5, 0), (4, 0, B.METHOD_EXACT, 0.0, 0)):
        with pytest.raises(B.GaconvError):
            B.Schedule(*args)
    with pytest.raises(B.GaconvError):
        B.Schedule(4, 4, B.METHOD_ZERO, float("nan"), 0)
