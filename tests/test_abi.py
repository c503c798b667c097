"""The C-ABI library: it loads, exports every symbol the header declares, and its host-side
argument checks return the documented codes without touching a GPU."""

import ctypes
import os
import re

import pytest

import paper_2502_20704_b200 as fsd
from paper_2502_20704_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(fsd_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(fsd.library_path())
    names = _declared_symbols()
    assert {"fsd_verify_chain", "fsd_verify_tree", "fsd_workspace_bytes", "fsd_status_string"} <= names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared but not exported"


def test_default_opts_and_workspace_size():
    o = fsd.fsd_default_opts()
    assert o.struct_size == ctypes.sizeof(fsd.FsdOpts)
    assert (o.divergence, o.mode, o.compare, o.sample, o.logit_dtype, o.threshold) == (0, 0, 0, 0, 1, 0.0)
    assert fsd.fsd_workspace_bytes(64, 8, 152064, o) >= 2 * 64 * 8 * 4
    assert fsd.fsd_workspace_bytes(64, 8, 152064, o) % 256 == 0
    with pytest.raises(fsd.FsdError):
        fsd.fsd_workspace_bytes(0, 8, 100, o)


def _chain(o, **kw):
    a = dict(t=4096, d=4096, tok=None, ua=None, us=4096, B=2, g=3, V=64, acc=4096, nt=4096, D=4096, st=4096,
             ws=4096, wsb=1 << 20)
    a.update(kw)
    return fsd.fsd_verify_chain(a["t"], a["d"], a["tok"], a["ua"], a["us"], a["B"], a["g"], a["V"], o,
                                a["acc"], a["nt"], a["D"], a["st"], a["ws"], a["wsb"], None)


def test_chain_argument_checks_launch_nothing():
    # every call below must be refused on the host (no device is present in this test)
    o = fsd.make_opts(T=0.2)
    assert _chain(o, t=None) == binding.FSD_ERR_NULL
    assert _chain(o, us=None) == binding.FSD_ERR_NULL
    assert _chain(o, ws=None) == binding.FSD_ERR_NULL
    assert _chain(None) == binding.FSD_ERR_NULL
    assert _chain(o, B=0) == binding.FSD_ERR_SHAPE
    assert _chain(o, g=0) == binding.FSD_ERR_SHAPE
    assert _chain(o, V=0) == binding.FSD_ERR_SHAPE
    assert _chain(o, B=1 << 20, g=1 << 12) == binding.FSD_ERR_SHAPE
    assert _chain(o, t=4097) == binding.FSD_ERR_ALIGN
    assert _chain(o, D=4098) == binding.FSD_ERR_ALIGN
    assert _chain(o, ws=4096 + 128) == binding.FSD_ERR_ALIGN
    assert _chain(o, wsb=16) == binding.FSD_ERR_WORKSPACE
    sd = fsd.make_opts(mode="sd")
    assert _chain(sd) == binding.FSD_ERR_NULL            # SD needs draft tokens and uniforms
    assert _chain(sd, tok=4096) == binding.FSD_ERR_NULL
    for field, bad in (("divergence", 3), ("mode", -1), ("compare", 2), ("sample", 9), ("logit_dtype", 2)):
        o2 = fsd.make_opts()
        setattr(o2, field, bad)
        assert _chain(o2) == binding.FSD_ERR_ENUM
    o3 = fsd.make_opts()
    o3.struct_size = 8
    assert _chain(o3) == binding.FSD_ERR_ENUM
    o4 = fsd.make_opts(T=float("nan"))
    assert _chain(o4) == binding.FSD_ERR_ENUM


def test_tree_argument_checks_launch_nothing():
    o = fsd.make_opts(T=0.2)

    def tree(opts=o, par=4096, N=5, depth=3, path=4096):
        return fsd.fsd_verify_tree(4096, 4096, par, 4096, 2, N, 64, depth, opts, 4096, path, 4096, 4096, 4096,
                                   4096, 1 << 20, None)

    assert tree(par=None) == binding.FSD_ERR_NULL
    assert tree(path=None) == binding.FSD_ERR_NULL
    assert tree(depth=0) == binding.FSD_ERR_SHAPE
    assert tree(N=5000) == binding.FSD_ERR_SHAPE
    assert tree(opts=fsd.make_opts(mode="sd")) == binding.FSD_ERR_UNSUPPORTED
    assert tree(opts=fsd.make_opts(mode="rfsd")) == binding.FSD_ERR_UNSUPPORTED


def test_status_strings():
    assert fsd.fsd_status_string(0) == "FSD_OK"
    for code in range(-7, 0):
        assert fsd.fsd_status_string(code).startswith("FSD_ERR_")
    assert "unknown" in fsd.fsd_status_string(-99)
    assert fsd.fsd_version() >= 100


def test_tuning_entry_points_check_their_arguments_on_the_host():
    # bad arguments are refused before anything is launched (no GPU needed)
    assert fsd.fsd_threshold_sweep(None, 1, 1, None, 1, 0, None, None) == -1           # FSD_ERR_NULL
    assert fsd.fsd_threshold_sweep(16, 0, 1, 16, 1, 0, 16, 16) == -2                   # FSD_ERR_SHAPE
    assert fsd.fsd_threshold_sweep(16, 1, 1, 16, 1, 5, 16, 16) == -4                   # FSD_ERR_ENUM
    assert fsd.fsd_calibrate_threshold(16, 1, 1, -1.0, 0, 16, 16) == -2
    assert fsd.fsd_calibrate_threshold(16, 1, 1, float("nan"), 0, 16, 16) == -2
    assert fsd.fsd_calibrate_threshold(None, 1, 1, 1.0, 0, 16, 16) == -1
    assert fsd.fsd_accept_labels(16, 1, 0, 0.1, 1, 16) == -2
    assert fsd.fsd_accept_labels(16, 1, 1, 0.1, 2, 16) == -4


def test_release_build_reports_no_debug_checks_and_a_word_inside_the_workspace():
    import paper_2502_20704_b200 as fsd
    on, off = fsd.fsd_debug_checks(4, 8)
    assert on is False
    assert 0 < off < fsd.fsd_workspace_bytes(4, 8, 32000, fsd.make_opts(T=0.1))
