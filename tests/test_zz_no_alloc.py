"""The allocation-free top-k entry point against the workspace-taking one.

Some callers cannot hand the library a workspace: they run inside a process whose device memory is a
fixed arena owned by someone else, or on a path where an allocation would synchronise the device.
qless_select_topk_static keeps its scratch in a fixed array inside the library instead. This test calls
it through the C ABI twice in a row, at sizes whose kernels do use that array (the second call sees
whatever the first left in it), and requires the same indices, bit for bit, as qless_select_topk. The file name sorts last so a
run that stops at the first failure has already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2502_01703_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _scores(N, seed, ties):
    gen = torch.Generator(device=DEV)
    gen.manual_seed(seed)
    s = torch.randn(N, generator=gen, device=DEV)
    if ties:
        s = torch.round(s * 8) / 8
    return s


def test_static_select_matches_workspace_select_on_two_calls_in_a_row():
    # Both sizes lie above what the one-launch cluster kernel takes (360 448 scores), so both calls run the multi-pass
    # select, the path that keeps its histograms, selection state and per-block counts and offsets in the library's
    # fixed array. Large first, smaller second: the second call finds the first one's 2048 block entries and full
    # histograms in the array and must not be misled by them. The calls are enqueued back to back on one stream.
    cases = [(B.SELECT_STATIC_MAX_N, 0.05, 1, False), (400_000, 0.3, 2, True)]
    outs = []
    for N, frac, seed, ties in cases:
        s = _scores(N, seed, ties)
        idx = torch.full((N,), -1, dtype=torch.int64, device=DEV)   # caller-owned output
        got = B.qless_select_topk_static(s, frac, idx)
        outs.append((s, frac, got))
    torch.cuda.synchronize()
    for s, frac, got in outs:
        want = B.qless_select_topk(s, frac)
        assert got.numel() == want.numel() == int(frac * s.numel() + 1e-6)
        assert torch.equal(got, want)
    # and once more with the first input: same answer after the array has been reused by a smaller problem
    s, frac, first = outs[0]
    idx = torch.empty(s.numel(), dtype=torch.int64, device=DEV)
    assert torch.equal(B.qless_select_topk_static(s, frac, idx), first)


def test_static_select_allocates_nothing():
    # Neither the driver's view of free device memory nor torch's allocator moves across warmed-up calls, whichever
    # kernel path the size selects (the one-launch cluster kernel below 360 448 scores, the multi-pass select above).
    for N in (100_000, 1_000_000):
        s = _scores(N, 7, False)
        idx = torch.empty(N, dtype=torch.int64, device=DEV)
        B.qless_select_topk_static(s, 0.05, idx)                    # first call on the device: resolves the array's address
        torch.cuda.synchronize()
        count = lambda: torch.cuda.memory_stats()["allocation.all.allocated"]      # allocations torch has made so far
        free0, allocs0 = torch.cuda.mem_get_info()[0], count()
        for _ in range(3):
            got = B.qless_select_topk_static(s, 0.05, idx)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] >= free0                # a device allocation would have lowered it
        assert count() == allocs0                                   # and torch's allocator was not asked for anything
        assert torch.equal(got, B.qless_select_topk(s, 0.05))


def test_static_select_edge_cases_and_limit():
    L = B.lib()
    k = C.c_int64(-1)
    # beyond the fixed array: refused with a message naming the limit, before anything is launched
    st = L.qless_select_topk_static(None, B.SELECT_STATIC_MAX_N + 1, 0.5, None, C.byref(k), None)
    assert st == B.ERR_UNSUPPORTED and str(B.SELECT_STATIC_MAX_N).encode() in L.qless_last_error()
    assert L.qless_select_topk_static(None, 10, 1.5, None, C.byref(k), None) == B.ERR_INVALID_ARG
    assert L.qless_select_topk_static(None, 10, 0.0, None, C.byref(k), None) == B.QLESS_OK and k.value == 0
    # at the limit, with ties and special values
    N = B.SELECT_STATIC_MAX_N
    s = _scores(N, 3, True)
    s[5] = float("nan"); s[6] = float("inf"); s[7] = -0.0
    idx = torch.empty(N, dtype=torch.int64, device=DEV)
    got = B.qless_select_topk_static(s, 0.01, idx)
    assert torch.equal(got, B.qless_select_topk(s, 0.01))
    z = torch.full((4096,), 1.5, device=DEV)
    assert np.array_equal(B.qless_select_topk_static(z, 0.25, idx).cpu().numpy(), np.arange(1024))
