"""Host-side checks that need no GPU: the library loads, exports every declared symbol, reports
workspace sizes, and rejects bad arguments before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_2609_32420_b200 import build as cbuild
from paper_2609_32420_b200 import carnator as cn

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    cbuild.build_library()


def _shape(**kw):
    base = dict(B=1, H=2, N=1000, D=128, n_text=0, T=10, Hg=10, Wg=10, block_q=128, block_k=128)
    base.update(kw)
    return cn.make_shape(**base)


def test_exports_match_header():
    text = open(os.path.join(ROOT, "include", "carnator.h")).read()
    declared = set(re.findall(r"\b(carnator_[a-z_0-9]+)\s*\(", text))
    assert declared == set(cn.EXPORTS)
    L = cn.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert cn.version() >= 1
    assert cn.status_string(cn.OK) == "ok"


def test_workspace_sizes():
    s = _shape()
    nqb = nkb = 8
    rows = 1 * 2 * nqb
    al = lambda x: (x + 255) // 256 * 256
    assert cn.attn_workspace_bytes(s) == 256 + 2 * al(rows * 4) + al(rows * nkb * 4)
    p = cn.BuildParams(0, 0.25, 0.9, -1, 0, 1)
    assert cn.build_workspace_bytes(s, p) == 256 + al(1 * 2 * 4) + 2 * al(rows * 128 * 4) + al(rows * nkb * 4) + 2 * al(3 * rows * 128 * 2)
    assert cn.attn_host_arena_bytes(s) > 4 * 2 * 1000 * 128 * 2


@pytest.mark.parametrize("kw,expect", [
    (dict(N=999), cn.ERR_INVALID_ARG),                 # n_text + T*Hg*Wg != N
    (dict(D=96), cn.ERR_UNSUPPORTED),
    (dict(block_q=32), cn.ERR_UNSUPPORTED),
    (dict(B=0), cn.ERR_INVALID_ARG),
])
def test_bad_shapes_are_rejected_without_a_launch(kw, expect):
    s = _shape(**kw)
    before = cn.kernel_launches()
    st = cn.lib().carnator_sparse_attn(1 << 20, 1 << 20, 1 << 20, 1 << 20, None, ctypes.byref(s), 1 << 20, 1 << 20,
                                       1 << 20, 1 << 30, None)
    assert st == expect
    assert cn.attn_workspace_bytes(s) == 0
    assert cn.kernel_launches() == before


def test_bad_pointers_strides_and_workspace():
    s = _shape()
    L = cn.lib()
    ok_ptr = 1 << 20
    big = 1 << 30
    call = lambda **k: L.carnator_sparse_attn(k.get("Q", ok_ptr), ok_ptr, ok_ptr, k.get("mask", ok_ptr), None,
                                              ctypes.byref(k.get("s", s)), ok_ptr, ok_ptr, k.get("ws", ok_ptr),
                                              k.get("ws_bytes", big), None)
    assert call(Q=None) == cn.ERR_INVALID_ARG
    assert call(Q=ok_ptr + 2) == cn.ERR_INVALID_ARG           # not 16-byte aligned
    assert call(mask=None) == cn.ERR_INVALID_ARG
    assert call(ws=None) == cn.ERR_WORKSPACE
    assert call(ws=ok_ptr + 64) == cn.ERR_WORKSPACE           # not 256-byte aligned
    assert call(ws_bytes=1024) == cn.ERR_WORKSPACE
    s2 = _shape()
    s2.q_stride[2] = 132                                       # not a multiple of 8 elements
    assert call(s=s2) == cn.ERR_INVALID_ARG
    s3 = _shape(block_q=64, block_k=64)
    s3.attn_impl = cn.IMPL_TCGEN05
    assert call(s=s3) == cn.ERR_UNSUPPORTED
    s4 = _shape()
    s4.attn_impl = 9
    assert call(s=s4) == cn.ERR_INVALID_ARG
    s5 = _shape()                                              # K shared over the two heads: not expressible as a tensor map
    s5.k_stride[1] = 0
    s5.attn_impl = cn.IMPL_TCGEN05
    assert call(s=s5) == cn.ERR_UNSUPPORTED


def test_bad_build_params():
    s = _shape()
    L = cn.lib()
    ok_ptr, big = 1 << 20, 1 << 30
    def call(p):
        return L.carnator_build_connectivity(ok_ptr, ok_ptr, ctypes.byref(s), ctypes.byref(p), ok_ptr, None, ok_ptr, big, None)
    assert call(cn.BuildParams(7, 0.25, 0.9, -1, 0, 1)) == cn.ERR_INVALID_ARG
    assert call(cn.BuildParams(0, 0.0, 0.9, -1, 0, 1)) == cn.ERR_INVALID_ARG
    assert call(cn.BuildParams(0, 1.5, 0.9, -1, 0, 1)) == cn.ERR_INVALID_ARG
    assert call(cn.BuildParams(1, 0.25, 0.0, -1, 0, 1)) == cn.ERR_INVALID_ARG
    assert call(cn.BuildParams(0, 0.25, 0.9, -2, 0, 1)) == cn.ERR_INVALID_ARG
    big_s = _shape(N=128 * 5000, T=1, Hg=1, Wg=128 * 5000)     # more key blocks than the selection kernel sorts
    assert L.carnator_build_connectivity(ok_ptr, ok_ptr, ctypes.byref(big_s), ctypes.byref(cn.BuildParams(0, 0.25, 0.9, -1, 0, 1)),
                                         ok_ptr, None, ok_ptr, 1 << 40, None) == cn.ERR_UNSUPPORTED


def test_compute_call_without_a_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    s = _shape()
    st = cn.lib().carnator_compact_mask(1 << 20, None, ctypes.byref(s), 1 << 20, 1 << 30, None)
    assert st in (cn.ERR_UNSUPPORTED, cn.ERR_CUDA)


def test_missing_library_raises(monkeypatch):
    monkeypatch.setattr(cn, "_lib", None)
    monkeypatch.setattr(cn, "LIB_PATH", "/nonexistent/libcarnator.so")
    with pytest.raises(RuntimeError):
        cn.lib()
