"""Host-side checks that need no GPU: the library builds/loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2603_30033_b200 import binding as Bd
from paper_2603_30033_b200 import build as Bu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    Bu.build()
    return Bd.load_library()


def test_exports_match_header(lib):
    text = open(os.path.join(ROOT, "include", "tucker_attn.h")).read()
    declared = re.findall(r"TA_API[^;(]*?\b(tucker_\w+)\s*\(", text)
    assert sorted(declared) == sorted(Bd.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert Bd.status_string(0) == "ok"
    for code in (-1, -2, -3, -4, -5):
        assert Bd.status_string(code) not in ("ok", "unknown status")
    assert Bd.status_string(-99) == "unknown status"


def _desc(**kw):
    base = dict(B=2, N=64, d_model=128, n_H=4, r=(2, 16, 16), t=(2, 16, 16), causal=True, rope=False,
                dtype=Bd.TA_DTYPE_F32)
    base.update(kw)
    return Bd.make_desc(**base)


def test_desc_layout_matches_header():
    # 17 four-byte fields
    assert ctypes.sizeof(Bd.TuckerAttnDesc) == 17 * 4


def test_workspace_queries(lib):
    assert Bd.fwd_workspace_bytes(_desc()) > 0
    assert Bd.decode_workspace_bytes(_desc(), 128) > 0
    assert Bd.fwd_workspace_bytes(_desc(n_H=3)) == 0            # d_model % n_H != 0
    assert Bd.fwd_workspace_bytes(_desc(rope=True, r=(2, 16, 15))) == 0   # odd r3 with RoPE
    assert Bd.fwd_workspace_bytes(_desc(N=0)) == 0
    assert Bd.decode_workspace_bytes(_desc(), 0) == 0
    # grows with the problem
    assert Bd.fwd_workspace_bytes(_desc(N=128)) > Bd.fwd_workspace_bytes(_desc(N=64))


def test_bad_arguments_rejected_on_host(lib):
    d = _desc()
    fake = ctypes.c_void_p(4096)          # never dereferenced: validation fails first
    args = [fake] * 9
    # null X
    rc = lib.tucker_attn_fwd(ctypes.byref(d), None, *args[1:], fake, None, None, 0, fake, 1 << 30, None)
    assert rc == -1
    # only one cache pointer
    rc = lib.tucker_attn_fwd(ctypes.byref(d), *args, fake, fake, None, 64, fake, 1 << 30, None)
    assert rc == -1
    # misaligned pointer
    rc = lib.tucker_attn_fwd(ctypes.byref(d), ctypes.c_void_p(4100), *args[1:], fake, None, None, 0, fake, 1 << 30, None)
    assert rc == -1
    # workspace too small
    rc = lib.tucker_attn_fwd(ctypes.byref(d), *args, fake, None, None, 0, fake, 16, None)
    assert rc == -3
    # invalid descriptor
    bad = _desc(r=(2, 0, 16))
    rc = lib.tucker_attn_fwd(ctypes.byref(bad), *args, fake, None, None, 0, fake, 1 << 30, None)
    assert rc == -1
    # decode: null cache_len, bad Lmax
    rc = lib.tucker_attn_decode(ctypes.byref(d), *args, fake, fake, 128, None, 1, fake, fake, 1 << 30, None)
    assert rc == -1
    rc = lib.tucker_attn_decode(ctypes.byref(d), *args, fake, fake, 0, fake, 1, fake, fake, 1 << 30, None)
    assert rc == -1
    rc = lib.tucker_attn_decode(ctypes.byref(d), *args, fake, fake, 128, fake, 1, fake, fake, 8, None)
    assert rc == -3


def test_missing_library_raises(monkeypatch):
    monkeypatch.setattr(Bd, "_lib", None)
    monkeypatch.setattr(Bd, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(RuntimeError):
        Bd.load_library()


def test_binding_rejects_cpu_tensors(lib):
    import torch
    X = torch.zeros(1, 4, 8)
    w = [torch.zeros(2, 4, 4), torch.zeros(2, 2), torch.zeros(8, 4), torch.zeros(8, 4)] * 2
    with pytest.raises(ValueError):
        Bd.tucker_attn_fwd(X, *w, n_H=2, causal=True, rope=False)
