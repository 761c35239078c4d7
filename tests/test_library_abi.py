"""The C-ABI library loads without a GPU and exports every symbol include/team.h declares."""
import ctypes
import os
import re

import pytest

from paper_2602_08404_b200 import binding as B
from paper_2602_08404_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def library():
    build_mod.build()
    return B.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "team.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(team_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(library):
    names = _declared_functions()
    assert {"team_create", "team_route", "team_select_experts", "team_moe_forward"} <= set(names)
    for n in names:
        assert hasattr(library, n), n
    assert sorted(B.EXPORTS) == names


def test_strerror_and_version(library):
    assert library.team_version() >= 1
    assert library.team_strerror(0) == b"ok"
    for code in (-1, -2, -3, -4, -5):
        assert library.team_strerror(code) not in (b"ok", b"unknown error")


def test_argument_checks_need_no_device(library):
    ctx = ctypes.c_void_p()
    assert library.team_create(None, ctypes.byref(ctx)) == B.TEAM_ERR_ARG
    bad = B.make_config(2048, 128, 200, 768)                  # top_k > n_experts
    assert library.team_create(ctypes.byref(bad), ctypes.byref(ctx)) == B.TEAM_ERR_SHAPE
    bad = B.make_config(2000, 128, 8, 768)                    # hidden not a multiple of 128 for bf16
    assert library.team_create(ctypes.byref(bad), ctypes.byref(ctx)) == B.TEAM_ERR_SHAPE
    bad = B.make_config(2048, 128, 8, 768, max_rows=1 << 20)
    assert library.team_create(ctypes.byref(bad), ctypes.byref(ctx)) == B.TEAM_ERR_SHAPE
    assert library.team_destroy(None) == B.TEAM_ERR_ARG
    assert library.team_moe_forward(None, None, None, None, None, None) == B.TEAM_ERR_ARG
    # weight packing: arguments are validated before anything touches the device
    p, q = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x2000)
    assert library.team_pack_w_down(None, q, 1, 128, 64, B.TEAM_DTYPE_BF16, None) == B.TEAM_ERR_ARG
    assert library.team_pack_w_down(p, p, 1, 128, 64, B.TEAM_DTYPE_BF16, None) == B.TEAM_ERR_ARG          # in place
    assert library.team_pack_w_down(ctypes.c_void_p(0x1008), q, 1, 128, 64, B.TEAM_DTYPE_BF16, None) == B.TEAM_ERR_ARG
    assert library.team_pack_w_down(p, q, 1, 128, 72, B.TEAM_DTYPE_BF16, None) == B.TEAM_ERR_SHAPE       # 72 % 16
    assert library.team_pack_w_down(p, q, 1, 128, 64, 7, None) == B.TEAM_ERR_SHAPE                       # dtype


def test_no_cpu_fallback(library):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    ok = B.make_config(2048, 128, 8, 768)
    ctx = ctypes.c_void_p()
    assert library.team_create(ctypes.byref(ok), ctypes.byref(ctx)) == B.TEAM_ERR_CUDA
    with pytest.raises(B.TeamError):
        B.team_create(ok)
