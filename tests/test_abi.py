"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every declared symbol, and rejects bad
arguments on the host before anything is enqueued."""
import ctypes
import os
import re

import pytest

from paper_2509_18467_b200 import api, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build()
    return api.lib()


def test_exports_every_declared_symbol(L):
    hdr = open(os.path.join(ROOT, "include", "lawcat.h")).read()
    declared = set(re.findall(r"\b(lawcat_[a-z_]+)\s*\(", hdr))
    assert declared == set(api.EXPORTS), declared ^ set(api.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_params_struct_matches_header():
    hdr = open(os.path.join(ROOT, "include", "lawcat.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} lawcat_params;", hdr, re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = []
    for decl in body.split(";"):
        decl = decl.strip()
        if decl:
            names += [n.strip() for n in decl.split(None, 1)[1].split(",")]
    assert names == [f[0] for f in api.Params._fields_]
    assert ctypes.sizeof(api.Params) == 4 * len(names)


def test_version_and_status_strings(L):
    assert L.lawcat_version() >= 100
    seen = {api.status_string(i) for i in range(7)}
    assert len(seen) == 7 and "unknown status" not in seen
    assert api.status_string(99) == "unknown status"


def test_workspace_bytes(L):
    p = api.params(2, 100, 8, 2, 64, 32)
    assert api.workspace_bytes(p, api.OP_CONV_FWD) == 0
    # decode: the token's features and decays (3 d_k floats) and one denominator per (sequence, head)
    assert api.workspace_bytes(p, api.OP_DECODE_STEP) >= 4 * 2 * 8 * (3 * 64 + 1)
    assert api.workspace_bytes(p, api.OP_GLA_BWD) >= 4 * 2 * 100 * 8 * 32
    assert api.workspace_bytes(p, api.OP_CONV_BWD) >= 4 * 2 * 100 * (8 + 2) * 64
    assert api.workspace_bytes(p, api.OP_LAYER_FWD) > 0
    bad = api.params(2, 100, 8, 3, 64, 32)
    assert api.workspace_bytes(bad, api.OP_GLA_BWD) == 0


@pytest.mark.parametrize("kw,status", [
    (dict(H_kv=3), 1), (dict(d_k=48), 2), (dict(d_v=256), 2), (dict(conv_k=9), 2), (dict(gate_dim=7), 2),
    (dict(gate_tau=0.0), 1), (dict(eps=-1.0), 1), (dict(dtype=5), 1), (dict(phi=9), 1), (dict(normalize=2), 1),
    (dict(T=-1), 1)])
def test_bad_parameters_rejected_on_host(L, kw, status):
    base = dict(B=1, T=8, H=4, H_kv=2, d_k=64, d_v=64)
    base.update(kw)
    p = api.params(**base)
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: validation fails first
    st = L.lawcat_gla_fwd(ctypes.byref(p), fake, fake, fake, fake, None, None, fake, None, None, None, None, 0, None,
                          None)
    assert st == status


def test_null_and_misaligned_pointers_rejected_on_host(L):
    p = api.params(1, 8, 4, 2, 64, 64)
    ok, odd = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1004)
    args = [ok, ok, ok, ok, None, None, ok, None, None, None]
    assert L.lawcat_gla_fwd(ctypes.byref(p), *[None if i == 2 else a for i, a in enumerate(args)], None, 0, None,
                            None) == 1
    assert L.lawcat_gla_fwd(ctypes.byref(p), *[odd if i == 0 else a for i, a in enumerate(args)], None, 0, None,
                            None) == 1
    # workspace too small is reported before any launch
    a13 = [ok] * 4 + [None, None] + [ok] * 7
    assert L.lawcat_gla_bwd(ctypes.byref(p), *a13, None, 0, None, None) == 4
    # decode needs its caches, and its workspace
    a12 = [ok] * 9 + [None, None, ok]
    assert L.lawcat_decode_step(ctypes.byref(p), *a12, None, 0, None, None) == 1
    assert L.lawcat_decode_step(ctypes.byref(p), *([ok] * 12), None, 0, None, None) == 4


def test_missing_library_is_a_hard_error(monkeypatch):
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "LIB_PATH", "/nonexistent/liblawcat.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        api.lib()
