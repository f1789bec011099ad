"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

import __graft_entry__  # noqa: F401  (builds the library on first use)
from paper_2608_27514_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    __graft_entry__.build()
    return B.lib()


def test_exports_match_header(lib):
    hdr = open(os.path.join(ROOT, "include", "tsd.h")).read()
    declared = set(re.findall(r"\b(tsd_[a-z0-9_]+)\s*\(", hdr))
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_strerror_and_status(lib):
    assert B.strerror(0) == "ok"
    assert "argument" in B.strerror(B.TSD_ERR_INVALID_ARG)
    assert B.tsd_check_status(0) == B.TSD_OK
    assert B.tsd_check_status(0x1) == B.TSD_ERR_TIMEOUT
    assert B.tsd_check_status(0x2) == B.TSD_ERR_DEVICE_DATA


def test_layout_validation_and_sizes(lib):
    ok = B.make_layout(1, 8, 32, 736, 32, 32, 128, B.TSD_BF16)
    assert B.tsd_branch_mask_bytes(ok) > 0 and B.tsd_branch_mask_bytes(ok) % 16 == 0
    for bad in (B.make_layout(0, 8, 32, 736, 32, 32, 128, 1), B.make_layout(1, 0, 32, 736, 32, 32, 128, 1),
                B.make_layout(1, 8, 48, 736, 32, 32, 128, 1), B.make_layout(1, 8, 32, 736, 32, 5, 128, 1),
                B.make_layout(1, 8, 32, 736, 32, 32, 96, 1), B.make_layout(1, 8, 32, 736, 32, 32, 128, 7),
                B.make_layout(1, 300, 32, 736, 32, 32, 128, 1)):
        assert B.tsd_branch_mask_bytes(bad) == 0
        rc = lib.tsd_build_branch_mask(ctypes.byref(bad), None, None, ctypes.c_void_p(256), 1 << 20, None, None)
        assert rc in (B.TSD_ERR_INVALID_ARG, B.TSD_ERR_UNSUPPORTED)
    # good layout, bad buffers: NULL, misaligned, too small
    big = 1 << 20
    assert lib.tsd_build_branch_mask(ctypes.byref(ok), None, None, None, big, None, None) == B.TSD_ERR_INVALID_ARG
    assert lib.tsd_build_branch_mask(ctypes.byref(ok), None, None, ctypes.c_void_p(260), big, None, None) == B.TSD_ERR_INVALID_ARG
    assert lib.tsd_build_branch_mask(ctypes.byref(ok), None, None, ctypes.c_void_p(256), 16, None, None) == B.TSD_ERR_WORKSPACE


def test_topk_validation(lib):
    p = ctypes.c_void_p(4096)
    f = lib.tsd_confidence_topk

    def call(logits=p, dtype=1, rows=4, vocab=1024, stride=1024, k=3, ws=p, ws_bytes=1 << 20):
        return f(logits, dtype, rows, vocab, stride, k, p, p, p, None, ws, ws_bytes, None, None)
    assert call(k=0) == B.TSD_ERR_INVALID_ARG
    assert call(k=9) == B.TSD_ERR_INVALID_ARG
    assert call(vocab=2, stride=8, k=3) == B.TSD_ERR_INVALID_ARG
    assert call(dtype=5) == B.TSD_ERR_UNSUPPORTED
    assert call(logits=None) == B.TSD_ERR_INVALID_ARG
    assert call(logits=ctypes.c_void_p(4098)) == B.TSD_ERR_INVALID_ARG
    assert call(stride=1020) == B.TSD_ERR_INVALID_ARG          # shorter than the vocabulary
    assert call(vocab=1000, stride=1004) == B.TSD_ERR_INVALID_ARG  # row pitch not a 16-byte multiple
    need = B.tsd_confidence_topk_workspace_bytes(4, 126464, 3)   # few rows: rows are split into segments
    assert need > 0
    assert call(vocab=126464, stride=126464, ws_bytes=need - 1) == B.TSD_ERR_WORKSPACE
    assert call(vocab=126464, stride=126464, ws=None) == B.TSD_ERR_INVALID_ARG
    assert call(rows=0) == B.TSD_OK                             # empty input: nothing to do
    assert B.tsd_confidence_topk_workspace_bytes(16384, 126464, 3) == 0  # many rows: no split


def test_accept_validation(lib):
    p = ctypes.c_void_p(4096)
    f = lib.tsd_accept_trajectories

    def call(S=1, B_=4, R=32, parent=p, stride=3, tau=0.9, rule=0, search=0):
        return f(S, B_, R, parent, p, 99, p, p, stride, tau, rule, search, p, p, p, p, p, p, p, None, None)
    assert call(B_=0) == B.TSD_ERR_INVALID_ARG
    assert call(B_=257) == B.TSD_ERR_INVALID_ARG
    assert call(R=129) == B.TSD_ERR_INVALID_ARG
    assert call(stride=0) == B.TSD_ERR_INVALID_ARG
    assert call(rule=2) == B.TSD_ERR_INVALID_ARG
    assert call(search=-1) == B.TSD_ERR_INVALID_ARG
    assert call(tau=float("nan")) == B.TSD_ERR_INVALID_ARG
    assert call(parent=None) == B.TSD_ERR_INVALID_ARG
    assert call(S=0) == B.TSD_OK


def test_attention_validation(lib):
    ok = B.make_layout(1, 8, 32, 736, 32, 32, 128, B.TSD_BF16)
    p = ctypes.c_void_p(4096)
    f = lib.tsd_verify_attention
    good = dict(q=p, qs=(1048576, 4096, 128), kc=p, vc=p, cs=(3014656, 4096, 128), kd=p, vd=p,
                ds=(1048576, 4096, 128), out=p, os_=(1048576, 4096, 128), scale=0.088)

    def call(**kw):
        a = dict(good, **kw)
        return f(ctypes.byref(ok), a.get("mask", p), a["q"], *a["qs"], a["kc"], a["vc"], *a["cs"], a["kd"],
                 a["vd"], *a["ds"], a["out"], *a["os_"], None, a["scale"], None, 0, 0, None, None)
    assert call(mask=None) == B.TSD_ERR_INVALID_ARG
    assert call(q=None) == B.TSD_ERR_INVALID_ARG
    assert call(kc=None) == B.TSD_ERR_INVALID_ARG
    assert call(out=ctypes.c_void_p(4100)) == B.TSD_ERR_INVALID_ARG
    assert call(qs=(1048576, 4097, 128)) == B.TSD_ERR_INVALID_ARG
    assert call(ds=(1048576, 4096, 64)) == B.TSD_ERR_INVALID_ARG
    assert call(scale=float("nan")) == B.TSD_ERR_INVALID_ARG


def test_missing_library_is_loud(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/libtsd.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        B.lib()


def test_tree_validation(lib):
    p = ctypes.c_void_p(4096)
    f = lib.tsd_build_draft_tree

    def call(S=1, Bp=4, R=32, k=3, prev=p, flag=p, tok=p, W=2, D=2, B_=4, stride=None, base=0):
        return f(S, Bp, R, k, prev, p, flag, tok, 99, p, p, W, D, B_, B_ if stride is None else stride, base,
                 None, p, p, p, p, None, None)
    assert call(R=129) == B.TSD_ERR_INVALID_ARG
    assert call(k=9) == B.TSD_ERR_INVALID_ARG
    assert call(W=0) == B.TSD_ERR_INVALID_ARG
    assert call(W=33) == B.TSD_ERR_INVALID_ARG
    assert call(B_=257) == B.TSD_ERR_INVALID_ARG
    assert call(flag=None) == B.TSD_ERR_INVALID_ARG      # flag without tokens
    assert call(prev=None) == B.TSD_ERR_INVALID_ARG
    assert call(stride=3) == B.TSD_ERR_INVALID_ARG       # forest narrower than the tree
    assert call(base=-1) == B.TSD_ERR_INVALID_ARG
    assert call(S=0) == B.TSD_OK


def test_interblock_validation(lib):
    p = ctypes.c_void_p(4096)
    assert lib.tsd_build_interblock_vis(1, 8, 0, p, None) == B.TSD_ERR_INVALID_ARG    # no current tree
    assert lib.tsd_build_interblock_vis(1, 8, 9, p, None) == B.TSD_ERR_INVALID_ARG
    assert lib.tsd_build_interblock_vis(1, 257, 4, p, None) == B.TSD_ERR_INVALID_ARG
    assert lib.tsd_build_interblock_vis(1, 8, 4, None, None) == B.TSD_ERR_INVALID_ARG
    assert lib.tsd_build_interblock_vis(0, 8, 4, None, None) == B.TSD_OK
    trig = lib.tsd_interblock_trigger
    assert trig(1, 8, 32, p, p, None, 8, 99, 0.9, p, None, None, None) == B.TSD_ERR_INVALID_ARG  # root outside
    assert trig(1, 8, 32, p, p, None, 4, 99, float("nan"), p, None, None, None) == B.TSD_ERR_INVALID_ARG
    assert trig(1, 8, 32, None, p, None, 4, 99, 0.9, p, None, None, None) == B.TSD_ERR_INVALID_ARG
    assert trig(0, 8, 32, None, None, None, 4, 99, 0.9, None, None, None, None) == B.TSD_OK
    acc = lib.tsd_accept_joint_trees

    def call(B_=8, n_cur=4, R=32, rule=0):
        return acc(1, B_, n_cur, R, p, p, 99, p, p, 1, 0.9, rule, 0, *([p] * 7), None, None)
    assert call(n_cur=0) == B.TSD_ERR_INVALID_ARG
    assert call(n_cur=9) == B.TSD_ERR_INVALID_ARG
    assert call(R=129) == B.TSD_ERR_INVALID_ARG
    assert call(rule=2) == B.TSD_ERR_INVALID_ARG


def test_relaxed_accept_validation(lib):
    p = ctypes.c_void_p(4096)
    f = lib.tsd_accept_relaxed

    def call(rule=2, stride=3, m=2, logits=None, dtype=1, vocab=100, ld=100, lse=p, R=32, n_cur=4):
        return f(1, 4, n_cur, R, p, p, 99, p, p, stride, m, logits, dtype, vocab, ld, lse, 0.9, rule, 0,
                 *([p] * 7), None, None, None)
    assert call(m=4) == B.TSD_ERR_INVALID_ARG                 # more candidates than the list holds
    assert call(m=0) == B.TSD_ERR_INVALID_ARG
    assert call(rule=3) == B.TSD_ERR_INVALID_ARG              # the probability rule needs logits
    assert call(rule=4) == B.TSD_ERR_INVALID_ARG
    assert call(rule=3, logits=p, lse=None) == B.TSD_ERR_INVALID_ARG
    assert call(rule=3, logits=p, ld=99) == B.TSD_ERR_INVALID_ARG
    assert call(rule=3, logits=p, dtype=5) == B.TSD_ERR_UNSUPPORTED
    assert call(n_cur=5) == B.TSD_ERR_INVALID_ARG
    # the strict entry points do not take the relaxed rules
    assert lib.tsd_accept_trajectories(1, 4, 32, p, p, 99, p, p, 1, 0.9, 2, 0, *([p] * 7), None, None) \
        == B.TSD_ERR_INVALID_ARG
