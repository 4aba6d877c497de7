"""C-ABI checks that need no GPU: the library builds, loads, exports every symbol the header
declares, and rejects host-detectable argument errors before launching anything."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_24698_b200.build import build_library
    return C.CDLL(build_library())


def declared_functions():
    src = open(os.path.join(ROOT, "include", "tsv.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"^\s*(?:const\s+)?(?:int|size_t|uint64_t|char\s*\*)\s*\*?\s*([a-z_][a-z0-9_]*)\s*\(", src, flags=re.M)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"branch_state_build", "tree_verify_attn", "accept_and_refresh", "tsv_workspace_bytes", "tsv_version",
            "tsv_error_string"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def _shape(**kw):
    from paper_2609_24698_b200.binding import CShape
    base = dict(dtype=1, B=2, D=8, H=64, d=512, m_csa=4, topk=512, HI=4, di=128, m_hca=128, window=128, sm_scale=0.0,
                max_L=4096, flags=0, reserved=0)
    base.update(kw)
    return CShape(**base)


def test_workspace_bytes_and_shape_validation(lib):
    from paper_2609_24698_b200.binding import CShape
    lib.tsv_workspace_bytes.restype = C.c_size_t
    lib.tsv_workspace_bytes.argtypes = [C.POINTER(CShape)]
    s = _shape()
    n = lib.tsv_workspace_bytes(C.byref(s))
    assert n > 2 * 8 * 512 * 4 and n % 256 == 0
    assert lib.tsv_workspace_bytes(C.byref(_shape(max_L=8192))) > n            # ranking scores need room
    for bad in (dict(D=33), dict(d=12), dict(window=4), dict(dtype=5), dict(di=4), dict(HI=17), dict(max_L=2), dict(B=0)):
        assert lib.tsv_workspace_bytes(C.byref(_shape(**bad))) == 0
    assert lib.tsv_workspace_bytes(None) == 0


def test_host_errors_return_before_any_launch(lib):
    from paper_2609_24698_b200 import binding as tsv
    fake = 0x10000                                           # never dereferenced: validation fails first
    cache = tsv.CCache(*[fake] * len(tsv.CACHE_TENSORS), 1 << 20, 1 << 20)
    nodes = tsv.CNodes(*[fake] * len(tsv.CNodes._fields_))
    scr = tsv.CScratch(*[fake] * len(tsv.CScratch._fields_))
    s = _shape()
    f = tsv._lib.branch_state_build
    assert f(None, C.byref(cache), C.byref(nodes), C.byref(scr), fake, None) == tsv.ERR_NULL
    assert f(C.byref(s), None, C.byref(nodes), C.byref(scr), fake, None) == tsv.ERR_NULL
    assert f(C.byref(s), C.byref(cache), C.byref(nodes), C.byref(scr), None, None) == tsv.ERR_NULL
    assert f(C.byref(_shape(D=40)), C.byref(cache), C.byref(nodes), C.byref(scr), fake, None) == tsv.ERR_SHAPE
    c2 = tsv.CCache(*[fake] * len(tsv.CACHE_TENSORS), 1 << 20, 1 << 20); c2.csa_kv = fake + 8
    assert f(C.byref(s), C.byref(c2), C.byref(nodes), C.byref(scr), fake, None) == tsv.ERR_ALIGN
    n2 = tsv.CNodes(*[fake] * len(tsv.CNodes._fields_)); n2.parent = None
    assert f(C.byref(s), C.byref(cache), C.byref(n2), C.byref(scr), fake, None) == tsv.ERR_NULL
    g = tsv._lib.tree_verify_attn
    assert g(C.byref(s), C.byref(cache), C.byref(nodes), C.byref(scr), fake, None, None, 0, fake, None) == tsv.ERR_WORKSPACE
    assert g(C.byref(s), C.byref(cache), C.byref(nodes), C.byref(scr), fake, None, fake, 16, fake, None) == tsv.ERR_WORKSPACE
    assert g(C.byref(s), C.byref(cache), C.byref(nodes), C.byref(scr), fake, None, fake + 64, 1 << 40, fake, None) == tsv.ERR_WORKSPACE
    assert g(C.byref(s), C.byref(cache), C.byref(nodes), C.byref(scr), None, None, fake, 1 << 40, fake, None) == tsv.ERR_NULL
    n3 = tsv.CNodes(*[fake] * len(tsv.CNodes._fields_)); n3.q = None
    assert g(C.byref(s), C.byref(cache), C.byref(n3), C.byref(scr), fake, None, fake, 1 << 40, fake, None) == tsv.ERR_NULL
    h = tsv._lib.accept_and_refresh
    assert h(C.byref(s), 0, None, None, None, fake, fake, fake, fake, fake, fake, None) == tsv.ERR_NULL
    pc = (C.POINTER(tsv.CCache) * 1)(C.pointer(cache)); pn = (C.POINTER(tsv.CNodes) * 1)(C.pointer(nodes)); ps = (C.POINTER(tsv.CScratch) * 1)(C.pointer(scr))
    assert h(C.byref(s), 0, pc, pn, ps, fake, fake, fake, fake, fake, fake, None) == tsv.ERR_SHAPE
    assert h(C.byref(s), 1, pc, pn, ps, fake, fake, None, fake, fake, fake, None) == tsv.ERR_NULL
    assert tsv._lib.tsv_error_string(tsv.ERR_ALIGN).decode().startswith("a vector pointer")
    assert tsv.version() >= 1000
