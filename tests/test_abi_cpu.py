"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the header
declares, and rejects bad arguments with a status before touching the device."""
import ctypes as C
import os
import re

import pytest

from paper_2502_01703_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2502_01703_b200 import build
    build.build()
    return B.lib()


def test_exports_every_declared_symbol(L):
    text = ""
    inc = os.path.join(ROOT, "include")
    for name in sorted(os.listdir(inc)):
        if name.endswith(".h"):
            text += open(os.path.join(inc, name)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = sorted(set(re.findall(r"\b(qless_[a-z0-9_]+)\s*\(", text)))
    assert len(declared) >= 13
    for sym in declared:
        assert hasattr(L, sym), sym
    assert sorted(B.EXPORTS) == [s for s in declared if s in B.EXPORTS]
    for sym in B.EXPORTS:
        assert sym in declared


def test_workspace_queries_are_pure_host_functions(L):
    assert B.qless_project_quantize_workspace(0, 1024, 512, 8) >= 256
    a = B.qless_project_quantize_workspace(256, 1 << 23, 8192, 4)
    assert a >= 256 * (1 << 23) * 2 + 256 * 8192 * 4
    assert a % 256 == 0
    assert B.qless_score_workspace(270_000, 448, 4, 3, 8192, 8) >= 4 * 270_000 * 4
    assert B.qless_select_topk_workspace(1000) >= 3 * 2048 * 4
    assert B.qless_select_topk_workspace(1 << 22) < (1 << 17)          # multi-pass select: histograms and block offsets
    assert 6.15 * (1 << 28) <= B.qless_select_topk_workspace(1 << 28) < 6.25 * (1 << 28)   # per score: key and offset pairs 6 B, their dense heads 0.05 B, a bitmap 1/8 B


def _status(call):
    try:
        call()
    except B.QlessError as e:
        return e.status
    return 0


def test_bad_arguments_return_statuses_before_any_launch(L):
    null = None
    # bits
    st = L.qless_quantize(null, 4, 512, 1, 3, null, null, null, null)
    assert st == B.ERR_UNSUPPORTED and b"bits" in L.qless_last_error()
    # d not a multiple of 128 / too large
    assert L.qless_quantize(null, 4, 500, 1, 8, null, null, null, null) == B.ERR_UNSUPPORTED
    assert L.qless_quantize(null, 4, 16384, 1, 8, null, null, null, null) == B.ERR_UNSUPPORTED
    # required pointers
    assert L.qless_quantize(null, 4, 512, 1, 8, null, null, null, null) == B.ERR_INVALID_ARG
    # zero rows succeed without touching anything
    assert L.qless_quantize(null, 0, 512, 1, 8, null, null, null, null) == B.QLESS_OK
    # negative sizes
    assert L.qless_quantize(null, -1, 512, 1, 8, null, null, null, null) == B.ERR_INVALID_ARG
    # projection: P not multiple of 128, one moment missing
    st = L.qless_project_quantize(null, B.F32, 1, 1000, null, null, None, 1000, 512, 1, 8, null, null, null, null, null, 0, null)
    assert st == B.ERR_UNSUPPORTED
    st = L.qless_project_quantize(null, B.F32, 1, 1024, C.c_void_p(16), null, None, 1024, 512, 1, 8, null, null, null, null, null, 0, null)
    assert st == B.ERR_INVALID_ARG
    st = L.qless_project_quantize(null, 7, 1, 1024, null, null, None, 1024, 512, 1, 8, null, null, null, null, null, 0, null)
    assert st == B.ERR_INVALID_ARG
    # workspace missing / too small (pointers are never dereferenced: the call stops first)
    fake = C.c_void_p(4096)
    st = L.qless_project_quantize(fake, B.F32, 2, 1024, null, null, None, 1024, 512, 1, 8, fake, fake, null, null, null, 0, null)
    assert st == B.ERR_WORKSPACE
    st = L.qless_project_quantize(fake, B.F32, 2, 1024, null, null, None, 1024, 512, 1, 8, fake, fake, null, null, fake, 16, null)
    assert st == B.ERR_WORKSPACE and b"too small" in L.qless_last_error()
    # adam config out of range
    cfg = B.AdamCfg(1.5, 0.999, 1e-8, 0)
    st = L.qless_project_quantize(fake, B.F32, 2, 1024, fake, fake, C.byref(cfg), 1024, 512, 1, 8, fake, fake, null, null, fake, 1 << 30, null)
    assert st == B.ERR_INVALID_ARG
    # select: frac out of range, NaN
    k = C.c_int64(-1)
    assert L.qless_select_topk(null, 10, 1.5, null, C.byref(k), null, 0, null) == B.ERR_INVALID_ARG
    assert L.qless_select_topk(null, 10, float("nan"), null, C.byref(k), null, 0, null) == B.ERR_INVALID_ARG
    assert L.qless_select_topk(null, 10, 0.5, null, None, null, 0, null) == B.ERR_INVALID_ARG
    # k = 0 succeeds and reports it
    assert L.qless_select_topk(null, 10, 0.0, null, C.byref(k), null, 0, null) == B.QLESS_OK and k.value == 0
    assert L.qless_select_topk(null, 0, 0.5, null, C.byref(k), null, 0, null) == B.QLESS_OK and k.value == 0
    # score: task offsets
    eta = (C.c_float * 2)(1.0, 0.5)
    def score(off, V=8, T=2, Cn=2, bits=8, d=128):
        o = (C.c_int32 * (T + 1))(*off)
        return L.qless_score(fake, 4096, fake, 4096, fake, fake, null, null, eta, o, 4, V, Cn, T, d, bits, 0,
                             fake, null, null, 0, null)
    assert score([0, 4, 7]) == B.ERR_INVALID_ARG          # does not end at V
    assert score([0, 4, 4]) == B.ERR_INVALID_ARG          # empty task
    assert score([1, 4, 8]) == B.ERR_INVALID_ARG
    assert score([0, 4, 8], bits=5) == B.ERR_UNSUPPORTED
    assert score([0, 4, 8]) == B.ERR_WORKSPACE            # valid shapes, no workspace given
    assert score([0, 4, 8], V=8, d=130) == B.ERR_UNSUPPORTED
    # the widened entry points check their arguments in the same way
    assert L.qless_quantize_absmean(null, 4, 500, 1, 8, null, null, null, null) == B.ERR_UNSUPPORTED
    assert L.qless_quantize_absmean(null, 4, 512, 1, 3, null, null, null, null) == B.ERR_UNSUPPORTED
    assert L.qless_quantize_absmean(null, 4, 512, 1, 4, null, null, null, null) == B.ERR_INVALID_ARG
    assert L.qless_quantize_absmean(null, 0, 512, 1, 4, null, null, null, null) == B.QLESS_OK
    o3 = (C.c_int32 * 3)(0, 4, 8)
    def score16(V=8, T=2, d=128, off=o3, ws=null, wsb=0):
        return L.qless_score_16bit(fake, 4096, fake, 4096, null, null, eta, off, 4, V, 2, T, d, fake, null, ws, wsb, null)
    assert score16(d=130) == B.ERR_UNSUPPORTED
    assert score16(T=9, off=(C.c_int32 * 10)(*range(10))) == B.ERR_UNSUPPORTED
    assert score16(off=(C.c_int32 * 3)(0, 4, 7)) == B.ERR_INVALID_ARG
    assert score16() == B.ERR_WORKSPACE
    assert B.qless_score_16bit_workspace(1000, 64, 2, 3) >= 2 * 1000 * 4
    assert L.qless_inv_norms_16bit(fake, 16, 4, 1, 128, fake, null) == B.ERR_INVALID_ARG      # stride does not cover a checkpoint
    assert L.qless_inv_norms_16bit(null, 4096, 0, 1, 128, null, null) == B.QLESS_OK
    # test hooks that choose a kernel variant: only the documented values
    for hook, bad in ((L.qless_set_projection_path, 2), (L.qless_set_score_path, -1), (L.qless_set_select_path, 3)):
        assert hook(bad) == B.ERR_INVALID_ARG
        assert hook(0) == B.QLESS_OK
    # the matrix travels with the call: only the two documented kinds, reserved fields zero; checked before anything else
    def pq_ex(cfg, host=False):
        fn = L.qless_project_quantize_host_ex if host else L.qless_project_quantize_ex
        tail = (fake, fake, null, null, 0, null) if host else (fake, fake, null, null, null, 0, null)
        return fn(fake, B.F32, 2, 1024, null, null, None, 1024, 512, 1, C.byref(cfg) if cfg is not None else None, 8, *tail)
    zero3 = (C.c_int32 * 3)(0, 0, 0)
    for host in (False, True):
        assert pq_ex(B.ProjectionCfg(2, zero3), host) == B.ERR_INVALID_ARG and b"matrix" in L.qless_last_error()
        assert pq_ex(B.ProjectionCfg(-1, zero3), host) == B.ERR_INVALID_ARG
        assert pq_ex(B.ProjectionCfg(B.GAUSSIAN, (C.c_int32 * 3)(0, 1, 0)), host) == B.ERR_INVALID_ARG
        assert pq_ex(B.ProjectionCfg(B.GAUSSIAN, zero3), host) == B.ERR_WORKSPACE        # valid: stops at the missing workspace
        assert pq_ex(None, host) == B.ERR_WORKSPACE
    assert not hasattr(L, "qless_set_projection_matrix")     # no process-wide matrix state
    # the bounded-wait self-test takes a poll limit in a documented range
    assert L.qless_selftest_timeout(10, null) == B.ERR_INVALID_ARG and L.qless_selftest_timeout(1 << 20, null) == B.ERR_INVALID_ARG
    assert L.qless_gaussian_entries(1, 0, 2, 2, 8, fake, null) == B.ERR_INVALID_ARG          # j0 not a multiple of 4
    assert L.qless_gaussian_entries(1, -1, 2, 0, 8, fake, null) == B.ERR_INVALID_ARG
    assert L.qless_gaussian_entries(1, 0, 2, 1 << 39, 8, fake, null) == B.ERR_UNSUPPORTED
    assert L.qless_gaussian_entries(1, 0, 2, 0, 8, null, null) == B.ERR_INVALID_ARG           # no output buffer
    assert L.qless_gaussian_entries(1, 0, 0, 0, 8, null, null) == B.QLESS_OK                  # empty range
    # micro-benchmarks: unknown kind, missing outputs (checked before anything is launched)
    ms, ops = C.c_float(0), C.c_double(0)
    assert L.qless_microbench(0, 10, None, C.byref(ops), null, 0, null) == B.ERR_INVALID_ARG
    assert L.qless_microbench(0, 0, C.byref(ms), C.byref(ops), null, 0, null) == B.ERR_INVALID_ARG
    # selection without a workspace: sizes beyond the built-in scratch are refused
    assert L.qless_select_topk_static(null, (1 << 22) + 1, 0.5, null, C.byref(k), null) == B.ERR_UNSUPPORTED
    assert L.qless_select_topk_static(null, 10, 0.0, null, C.byref(k), null) == B.QLESS_OK and k.value == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="build the CUDA library"):
        B.lib()
