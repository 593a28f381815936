"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments on
the host (no kernel is launched here, so this runs without a GPU)."""
import ctypes
import os
import re

import pytest

from paper_2102_04782_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return api.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "dai8.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dai8_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    syms = declared_symbols()
    assert len(syms) >= 12
    for name in syms:
        assert hasattr(lib, name), name
    assert sorted(api.EXPORTS) == syms


def test_status_strings_and_defaults(lib):
    assert api.status_string(api.OK) == "ok"
    assert len({api.status_string(i) for i in range(7)}) == 7
    p = api.mcs_defaults()
    assert (round(p.lam, 6), p.k, round(p.A, 6), p.std_unbiased, p.center_mean) == (0.3, 1.0, 0.8, 0, 1)
    assert [api.padded_channels(c) for c in (1, 3, 16, 17, 64, 2048)] == [16, 16, 16, 32, 64, 2048]


def test_workspace_sizes(lib):
    assert api.quantize_grad_workspace_bytes(64) > 64 * 20
    assert api.quantize_grad_workspace_bytes(0) == 0
    g = api.ConvGeom(8, 64, 64, 14, 14, 3, 3, 1, 1, 1, 1)
    assert (g.P, g.Q) == (14, 14)
    assert api.conv_workspace_bytes(api.OP_BWD_DATA, g) >= 64 * 64 * 9
    assert api.conv_workspace_bytes(api.OP_BWD_FILTER, g) >= 64 * 64 * 9 * 4
    bad = api.ConvGeom(8, 64, 64, 2, 2, 7, 7, 1, 1, 0, 0)  # filter larger than the padded input
    assert api.conv_workspace_bytes(api.OP_FWD, bad) == 0


def test_invalid_arguments_are_rejected_on_the_host(lib):
    null = None
    fake = ctypes.c_void_p(0x1000)      # never dereferenced: validation fails first
    odd = ctypes.c_void_p(0x1004)
    st = lib.dai8_quantize_tensor(null, api.F32, api.NHWC, 1, 1, 1, 1, 0, fake, 0, 0, fake, None, 0, None)
    assert st == api.ERR_INVALID_ARG
    st = lib.dai8_quantize_tensor(fake, api.F32, api.NHWC, 0, 1, 1, 1, 0, fake, 0, 0, fake, None, 0, None)
    assert st == api.ERR_INVALID_ARG
    st = lib.dai8_quantize_tensor(odd, api.F32, api.NHWC, 1, 1, 1, 1, 0, fake, 0, 0, fake, None, 0, None)
    assert st == api.ERR_INVALID_ARG
    st = lib.dai8_quantize_tensor(fake, 7, api.NHWC, 1, 1, 1, 1, 0, fake, 0, 0, fake, None, 0, None)
    assert st == api.ERR_INVALID_ARG
    st = lib.dai8_quantize_tensor(fake, api.F32, api.NHWC, 1, 1, 1, 1, 0, fake, 0, 0, fake, fake, 8, None)
    assert st == api.ERR_WORKSPACE
    assert api.quantize_tensor_workspace_bytes() >= 16
    st = lib.dai8_quantize_grad(fake, api.F32, api.NHWC, 2, 64, 4, 4, None, fake, 0, fake, None, None,
                                fake, None, 0, None, fake, 16, None)
    assert st == api.ERR_WORKSPACE
    g = api.ConvGeom(1, 16, 16, 4, 4, 3, 3, 1, 1, 1, 1)
    st = lib.dai8_conv_bwd_filter(fake, fake, fake, fake, ctypes.byref(g), fake, api.F32, fake, 8, None)
    assert st == api.ERR_WORKSPACE
    st = lib.dai8_conv_fwd(fake, fake, None, fake, ctypes.byref(g), fake, api.F32, api.NHWC, None, 0, None)
    assert st == api.ERR_INVALID_ARG
    g0 = api.ConvGeom(1, 16, 16, 4, 4, 3, 3, 0, 1, 1, 1)
    st = lib.dai8_conv_fwd(fake, fake, fake, fake, ctypes.byref(g0), fake, api.F32, api.NHWC, None, 0, None)
    assert st == api.ERR_INVALID_ARG
    with pytest.raises(api.Dai8Error):
        api._check(api.ERR_UNSUPPORTED, "x")
