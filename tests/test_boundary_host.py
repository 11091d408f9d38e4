"""Host-side checks of the C boundary that need no GPU: the library loads, exports every symbol
the header declares, and rejects bad descriptors before launching anything."""
import ctypes as C
import os
import re

import pytest

from paper_2510_02345_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_functions():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(cmoe_[a-z_0-9]+)\s*\(", text))
    return names


def test_exports_match_header(lib):
    names = declared_functions()
    assert {"cmoe_create", "cmoe_route", "cmoe_forward", "cmoe_destroy"} <= names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/ but not exported"
    assert names == set(binding.EXPORTS)


def desc(**kw):
    d = binding.cmoe_desc()
    base = dict(d=128, d_ff=512, E=8, G=2, r=4, k=2, quant_group=32, T_max=256)
    base.update(kw)
    for k, v in base.items():
        setattr(d, k, v)
    return d


def test_workspace_query_and_validation(lib):
    n = binding.cmoe_workspace_bytes(desc())
    assert n > 0 and n % 256 == 0
    assert binding.cmoe_workspace_bytes(desc(T_max=512)) > n
    bad = [dict(E=9), dict(k=5), dict(k=0), dict(d=100), dict(d_ff=100), dict(r=5), dict(r=64),
           dict(quant_group=64), dict(T_max=0), dict(G=128, E=128), dict(E=80, G=2, k=2), dict(k=9, E=32, G=2)]
    for kw in bad:
        out = C.c_size_t()
        rc = lib.cmoe_workspace_bytes(C.byref(desc(**kw)), C.byref(out))
        assert rc in (-1, -2), (kw, rc)
    assert lib.cmoe_workspace_bytes(None, C.byref(C.c_size_t())) == -1
    assert lib.cmoe_workspace_bytes(C.byref(desc()), None) == -1


def test_create_rejects_bad_arguments_before_any_launch(lib):
    h = C.c_void_p()
    d = desc()                                   # all pointers NULL
    assert lib.cmoe_create(C.byref(d), C.byref(h)) == -1 and not h.value
    assert lib.cmoe_create(C.byref(d), None) == -1
    fake = 0x10000                                # never dereferenced on the host
    for n in ("C", "R", "B1", "B2", "U1q", "V1q", "U2q", "V2q", "U1s", "V1s", "U2s", "V2s"):
        setattr(d, n, fake)
    d.workspace, d.workspace_bytes = fake, 16     # far too small
    assert lib.cmoe_create(C.byref(d), C.byref(h)) == -3
    d.workspace = fake + 8                        # misaligned arena
    d.workspace_bytes = 1 << 40
    assert lib.cmoe_create(C.byref(d), C.byref(h)) == -1
    d.workspace, d.C = fake, fake + 4             # misaligned weight pointer
    assert lib.cmoe_create(C.byref(d), C.byref(h)) == -1


def test_null_handles(lib):
    assert lib.cmoe_forward(None, None, 0, None, None) == -1
    assert lib.cmoe_route(None, None, 0, None, None, None, None) == -1
    assert lib.cmoe_destroy(None) == -1
    assert lib.cmoe_status(None, None) == -1
    assert binding.strerror(0) == "ok" and "workspace" in binding.strerror(-3)
