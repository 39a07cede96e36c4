"""Host-only checks of the C ABI: the library loads, exports what the header declares, and rejects bad
arguments before touching the device.  No compute call is made here."""
import ctypes as C
import os
import re

import pytest

from paper_2601_17818_b200 import binding as vb
from paper_2601_17818_b200.build import build_library

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build_library()
    return vb.lib()


def test_header_symbols_are_exported(L):
    text = open(os.path.join(ROOT, "include", "vitcop.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = sorted(set(re.findall(r"\b(vitcop_[a-z_]+)\s*\(", text)))
    assert len(declared) >= 10
    for name in declared:
        assert hasattr(L, name), name
    assert sorted(vb.EXPORTS) == declared


def test_status_strings(L):
    seen = set()
    for s in range(7):
        msg = L.vitcop_status_string(s).decode()
        assert msg and msg != "unknown status"
        seen.add(msg)
    assert len(seen) == 7
    assert L.vitcop_status_string(99).decode() == "unknown status"


def test_workspace_sizes():
    assert vb.vitcop_workspace_bytes(vb.OP_KNORM, B=4, Nv=100) == 0
    assert vb.vitcop_workspace_bytes(vb.OP_COMPACT, B=4, Nv=100) == 0
    assert vb.vitcop_workspace_bytes(vb.OP_SELECT, B=4, Nv=100) >= 4
    s1 = vb.vitcop_workspace_bytes(vb.OP_PRUNE_STEP, B=16, Nv=576)
    assert s1 >= 16 * 576 * 8 + 16 * 4
    f1 = vb.vitcop_workspace_bytes(vb.OP_FILTER, B=2, Nv=1000, D=128)
    f2 = vb.vitcop_workspace_bytes(vb.OP_FILTER, B=4, Nv=1000, D=128)
    assert f2 > f1 > 2 * 1000 * 20
    with pytest.raises(vb.VitcopError) as e:
        vb.vitcop_workspace_bytes(77)
    assert e.value.status == vb.ERR_INVALID_ARG
    with pytest.raises(vb.VitcopError):
        vb.vitcop_workspace_bytes(vb.OP_SELECT, B=-1)


def test_argument_validation_happens_on_the_host(L):
    """Every call below must return before any CUDA work (there may be no device at all)."""
    fake = C.c_void_p(0x1000)                       # 16-byte aligned, never dereferenced by the checks
    odd = C.c_void_p(0x1008)
    ws = C.c_void_p(0x10000)
    null = None
    # knorm
    assert L.vitcop_knorm_score(null, 1, 1, 8, 8, 64, 64, 8, 0, null, 4, fake, 4, null) == vb.ERR_INVALID_ARG
    assert L.vitcop_knorm_score(fake, 1, 1, 8, 8, 64, 64, 8, 6, null, 4, fake, 4, null) == vb.ERR_INVALID_ARG  # span > N
    assert L.vitcop_knorm_score(fake, 1, 1, 8, 8, 64, 64, 8, 0, null, 5, fake, 4, null) == vb.ERR_INVALID_ARG  # len > cap
    assert L.vitcop_knorm_score(fake, -1, 1, 8, 8, 64, 64, 8, 0, null, 4, fake, 4, null) == vb.ERR_INVALID_ARG
    assert L.vitcop_knorm_score(fake, 1, 1, 8, 12, 96, 96, 12, 0, null, 4, fake, 4, null) == vb.ERR_UNSUPPORTED  # d % 8
    assert L.vitcop_knorm_score(odd, 1, 1, 8, 8, 64, 64, 8, 0, null, 4, fake, 4, null) == vb.ERR_UNSUPPORTED   # alignment
    # select
    p = vb.SelectParams(0, 0, 3)
    assert L.vitcop_select(null, null, 1, null, 4, 4, C.byref(p), fake, 4, fake, null, ws, 256, null) == vb.ERR_INVALID_ARG
    assert L.vitcop_select(fake, null, 1, null, 4, 4, C.byref(p), fake, 2, fake, null, ws, 256, null) == vb.ERR_INVALID_ARG  # keep_stride < budget
    assert L.vitcop_select(fake, null, 1, null, 4, 4, C.byref(p), fake, 4, fake, null, null, 0, null) == vb.ERR_WORKSPACE
    assert L.vitcop_select(fake, null, 1, null, 4, 4, C.byref(p), fake, 4, fake, null, ws, 8, null) == vb.ERR_WORKSPACE
    q = vb.SelectParams(1, 0, 3)
    assert L.vitcop_select(fake, null, 1, null, 4, 4, C.byref(q), fake, 4, fake, null, ws, 256, null) == vb.ERR_INVALID_ARG  # quota needs labels
    neg = vb.SelectParams(0, 0, -1)
    assert L.vitcop_select(fake, null, 1, null, 4, 4, C.byref(neg), fake, 4, fake, null, ws, 256, null) == vb.ERR_INVALID_ARG
    big = vb.SelectParams(0, 0, 3)
    assert L.vitcop_select(fake, null, 1, null, 4, 20000, C.byref(big), fake, 4, fake, null, ws, 256, null) == vb.ERR_UNSUPPORTED
    # compact: missing output for a given input, aliasing, bad span
    a, b = C.c_void_p(0x100000), C.c_void_p(0x900000)
    assert L.vitcop_compact_kv(a, null, null, 1, 1, 8, 8, 8, null, 0, null, 4, fake, 4, fake, null, null, null, 8, null, fake, null) == vb.ERR_INVALID_ARG
    assert L.vitcop_compact_kv(a, null, null, 1, 1, 8, 8, 8, null, 0, null, 4, fake, 4, fake, a, null, null, 8, null, fake, null) == vb.ERR_INVALID_ARG
    assert L.vitcop_compact_kv(a, null, null, 1, 1, 8, 8, 8, null, 6, null, 4, fake, 4, fake, b, null, null, 8, null, fake, null) == vb.ERR_INVALID_ARG
    assert L.vitcop_compact_kv(a, null, null, 1, 1, 8, 8, 12, null, 0, null, 4, fake, 4, fake, b, null, null, 8, null, fake, null) == vb.ERR_UNSUPPORTED
    # filter
    fp = vb.FilterParams(0, 0.5, 0.6, 0.05, 0)
    assert L.vitcop_redundancy_filter(null, null, 1, 8, 64, C.byref(fp), fake, fake, null, null, null, ws, 1 << 20, null) == vb.ERR_INVALID_ARG
    assert L.vitcop_redundancy_filter(fake, null, 1, 8, 72, C.byref(fp), fake, fake, null, null, null, ws, 1 << 20, null) == vb.ERR_UNSUPPORTED
    assert L.vitcop_redundancy_filter(fake, null, 1, 8, 64, C.byref(fp), fake, fake, null, null, null, ws, 16, null) == vb.ERR_WORKSPACE
    bad = vb.FilterParams(0, 0.0, 0.6, 0.05, 0)
    assert L.vitcop_redundancy_filter(fake, null, 1, 8, 64, C.byref(bad), fake, fake, null, null, null, ws, 1 << 20, null) == vb.ERR_INVALID_ARG
    bad = vb.FilterParams(3, 0.5, 0.6, 0.05, 0)
    assert L.vitcop_redundancy_filter(fake, null, 1, 8, 64, C.byref(bad), fake, fake, null, null, null, ws, 1 << 20, null) == vb.ERR_INVALID_ARG
    assert L.vitcop_similarity_rows(fake, 1, 8, 64, 0, 4, 2, fake, ws, 1 << 20, null) == vb.ERR_INVALID_ARG
    # prune step
    assert L.vitcop_prune_step(null, null, null, 1, 1, 8, 8, 8, null, 0, null, 4, 4, null, 2, null, null, null, 8, null, fake, null, null, null, ws, 1 << 20, null) == vb.ERR_INVALID_ARG
    assert L.vitcop_prune_step(null, a, null, 1, 1, 8, 8, 8, null, 0, null, 4, 4, null, 2, null, b, null, 8, null, fake, null, null, null, null, 0, null) == vb.ERR_WORKSPACE


def test_argument_validation_of_the_wider_entry_points(L):
    fake, odd, ws, null = C.c_void_p(0x1000), C.c_void_p(0x1008), C.c_void_p(0x10000), None
    a, b = C.c_void_p(0x100000), C.c_void_p(0x900000)
    fp = vb.FilterParams(0, 0.5, 0.6, 0.05, 0)
    # merge: required pointers, Dh % 8, workspace
    assert L.vitcop_merge_clusters(null, 1, 8, 8, 0, null, 4, 4, fake, fake, null, null, fake, fake, fake, 4, ws, 1 << 20, null) == vb.ERR_INVALID_ARG
    assert L.vitcop_merge_clusters(a, 1, 8, 12, 0, null, 4, 4, fake, fake, null, null, fake, fake, fake, 4, ws, 1 << 20, null) == vb.ERR_UNSUPPORTED
    assert L.vitcop_merge_clusters(a, 1, 8, 8, 6, null, 4, 4, fake, fake, null, null, fake, fake, fake, 4, ws, 1 << 20, null) == vb.ERR_INVALID_ARG   # span > N
    assert L.vitcop_merge_clusters(a, 1, 8, 8, 0, null, 4, 4, fake, fake, null, null, fake, fake, fake, 4, ws, 8, null) == vb.ERR_WORKSPACE
    # saliency
    assert L.vitcop_cls_saliency(null, fake, 1, 1, 4, 8, 0.5, fake, null, ws, 1 << 20, null) == vb.ERR_INVALID_ARG
    assert L.vitcop_cls_saliency(fake, fake, 1, 1, 4, 12, 0.5, fake, null, ws, 1 << 20, null) == vb.ERR_UNSUPPORTED
    assert L.vitcop_cls_saliency(fake, odd, 1, 1, 4, 8, 0.5, fake, null, ws, 1 << 20, null) == vb.ERR_UNSUPPORTED
    assert L.vitcop_cls_saliency(fake, fake, 1, 1, 4, 8, 0.5, fake, null, ws, 16, null) == vb.ERR_WORKSPACE
    # one-call Stage II: needs labels out, a valid metric / cutoff, D % 64, a workspace
    args = lambda feat=fake, D=64, f=fp, lab=fake, wsb=1 << 24, B=1: (feat, null, D, C.byref(f), null, a, null, B, 1, 8, 8, 8, 0, 4, 2, null, b, null, 8, null, fake, lab, fake, null, null, null, null, null, null, ws, wsb, null)
    assert L.vitcop_collaborative_step(*args(lab=null)) == vb.ERR_INVALID_ARG
    assert L.vitcop_collaborative_step(*args(f=vb.FilterParams(0, 0.0, 0.6, 0.05, 0))) == vb.ERR_INVALID_ARG
    assert L.vitcop_collaborative_step(*args(D=72)) == vb.ERR_UNSUPPORTED
    assert L.vitcop_collaborative_step(*args(wsb=64)) == vb.ERR_WORKSPACE
    assert L.vitcop_collaborative_step(*args(B=65536, wsb=1 << 40)) == vb.ERR_UNSUPPORTED      # as its sibling calls
    # K projection: weights required, cos and sin together, rotation only for head sizes whose halves are chunk-aligned
    kp = lambda hid=fake, W=fake, Dh=64, d=64, cos=null, sin=null, npos=0, wsb=1 << 24: (hid, W, 1, 8, Dh, 2, d, cos, sin, null, npos, b, 0, 4, fake, ws, wsb, null)
    assert L.vitcop_kproj_knorm(*kp(W=null)) == vb.ERR_INVALID_ARG
    assert L.vitcop_kproj_knorm(*kp(cos=fake)) == vb.ERR_INVALID_ARG
    assert L.vitcop_kproj_knorm(*kp(Dh=72)) == vb.ERR_UNSUPPORTED
    assert L.vitcop_kproj_knorm(*kp(d=32, cos=fake, sin=fake, npos=8)) == vb.ERR_UNSUPPORTED
    assert L.vitcop_kproj_knorm(*kp(wsb=64)) == vb.ERR_WORKSPACE
    assert vb.vitcop_workspace_bytes(vb.OP_KPROJ, B=2, H=4, N=100, d=128) >= 2 * 2 * 100 * 4
    assert vb.vitcop_workspace_bytes(vb.OP_COLLAB_STEP, B=2, Nv=100, D=64) > vb.vitcop_workspace_bytes(vb.OP_FILTER, B=2, Nv=100, D=64)
    assert vb.vitcop_workspace_bytes(vb.OP_MERGE, B=2, Nv=100, N=10) >= 256 + 2 * 100 * 2
    assert vb.vitcop_workspace_bytes(vb.OP_SALIENCY, B=2, H=4, N=33) >= 2 * 4 * 33 * 4


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    monkeypatch.setattr(vb, "_lib", None)
    monkeypatch.setattr(vb, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        vb.lib()
