"""The C ABI without a GPU: the library loads, exports every symbol the header
declares, and rejects bad arguments on the host before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_2412_18052_b200 import binding
from paper_2412_18052_b200.build import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gaf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gaf_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert len(names) >= 10
    for name in names:
        assert hasattr(L, name), f"{name} declared in gaf.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_error_strings(L):
    seen = {L.gaf_error_string(c) for c in range(0, 9)}
    assert len(seen) == 9 and b"unknown error code" not in seen
    assert L.gaf_error_string(1234) == b"unknown error code"


def test_workspace_bytes(L):
    out = ctypes.c_size_t()
    assert L.gaf_workspace_bytes(4, 1000, 0, ctypes.byref(out)) == 0 and out.value >= 4096
    small = out.value
    assert L.gaf_workspace_bytes(64, 1000, 1, ctypes.byref(out)) == 0 and out.value > small
    assert out.value % 256 == 0
    for K, D, dt in ((0, 10, 0), (65, 10, 0), (4, -1, 0), (4, 10, 2)):
        assert L.gaf_workspace_bytes(K, D, dt, ctypes.byref(out)) == 1
    assert L.gaf_workspace_bytes(4, 10, 0, None) == 1
    assert L.gaf_host_staging_bytes(4, 1000, 0, ctypes.byref(out)) == 0
    assert out.value >= 4 * 4000 + 4000


# Fake, never dereferenced addresses: the checks below must return before any CUDA call.
A = 0x7000_0000_0000


def _filter(L, ptrs, K, D, dtype=0, tau=0.97, order=None, out=A + (1 << 30), mask=A + (2 << 30),
            count=A + (3 << 30), ws=A + (4 << 30), ws_bytes=1 << 22, sched=0):
    arr = (ctypes.c_void_p * max(1, len(ptrs)))(*ptrs) if ptrs is not None else None
    ordp = (ctypes.c_int32 * len(order))(*order) if order is not None else None
    return L.gaf_filter_accumulate(
        ctypes.cast(arr, ctypes.c_void_p) if arr is not None else None, K, D, dtype, tau,
        ctypes.cast(ordp, ctypes.c_void_p) if ordp is not None else None,
        out, mask, None, count, ws, ws_bytes, sched, None)


def test_filter_argument_errors(L):
    g = [A + i * (1 << 24) for i in range(4)]
    assert _filter(L, None, 4, 100) == 1
    assert _filter(L, g, 0, 100) == 1
    assert _filter(L, g, 65, 100) == 1
    assert _filter(L, g, 4, -1) == 1
    assert _filter(L, g, 4, 100, dtype=7) == 1
    assert _filter(L, g, 4, 100, sched=9) == 1
    assert _filter(L, g, 4, 100, tau=float("nan")) == 1
    assert _filter(L, [g[0], 0, g[2], g[3]], 4, 100) == 1
    assert _filter(L, g, 4, 100, out=0) == 1
    assert _filter(L, g, 4, 100, order=[0, 1, 1, 3]) == 1
    assert _filter(L, g, 4, 100, order=[0, 1, 2, 4]) == 1
    assert _filter(L, [g[0], g[1] + 4, g[2], g[3]], 4, 100) == 2          # misaligned gradient
    assert _filter(L, g, 4, 100, out=A + (1 << 30) + 8) == 2              # misaligned output
    assert _filter(L, g, 4, 100, out=g[2] + 64) == 3                      # output inside an input
    assert _filter(L, g, 4, 100, out=g[2] - 16 * 4) == 3                  # output tail overlaps input head
    assert _filter(L, g, 4, 100, ws=0) == 4
    assert _filter(L, g, 4, 100, ws=A + (4 << 30) + 16) == 4              # workspace not 256-aligned
    assert _filter(L, g, 4, 100, ws_bytes=100) == 4


def test_repeat_and_test_hook_argument_errors(L):
    g = [A + i * (1 << 24) for i in range(8)]
    arr = (ctypes.c_void_p * 8)(*g)
    p = ctypes.cast(arr, ctypes.c_void_p)
    out, mask, count, ws = A + (1 << 30), A + (2 << 30), A + (3 << 30), A + (4 << 30)

    def rep(repeats, n_sets, K, grads=p, workspace=ws):
        return L.gaf_filter_accumulate_repeat(repeats, n_sets, grads, K, 100, 0, 0.97, None, out, mask, None, count,
                                              workspace, 1 << 22, 0, None)
    assert rep(-1, 2, 4) == 1 and rep(3, 0, 4) == 1 and rep(3, 2, 0) == 1 and rep(3, 2, 4, grads=None) == 1
    assert rep(0, 2, 4) == 0                        # no repetition: nothing is launched, nothing is checked further
    assert rep(2, 2, 4, workspace=0) == 4           # the first repetition's own checks apply
    assert L.gaf_test_set_wait_fault(1000, 1) == 0 and L.gaf_test_set_wait_fault(0, 0) == 0


def test_cosdist_and_pairwise_argument_errors(L):
    ws, n = A + (4 << 30), 1 << 22
    assert L.gaf_cosdist(None, A, 10, 0, A + 4096, None, ws, n, None) == 1
    assert L.gaf_cosdist(A, A + 1024, -1, 0, A + 4096, None, ws, n, None) == 1
    assert L.gaf_cosdist(A, A + 1024, 10, 3, A + 4096, None, ws, n, None) == 1
    assert L.gaf_cosdist(A, A + 1024, 10, 0, None, None, ws, n, None) == 1
    assert L.gaf_cosdist(A + 2, A + 1024, 10, 1, A + 4096, None, ws, n, None) == 2
    assert L.gaf_cosdist(A, A + 1024, 10, 0, A + 4096, None, ws, 64, None) == 4
    arr = (ctypes.c_void_p * 2)(A, A + 4096)
    p = ctypes.cast(arr, ctypes.c_void_p)
    assert L.gaf_pairwise_cosdist(p, 2, 10, 0, None, None, ws, n, None) == 1
    assert L.gaf_pairwise_cosdist(p, 0, 10, 0, A + 8192, None, ws, n, None) == 1
    assert L.gaf_pairwise_cosdist(p, 2, 10, 0, A + 8192, None, ws, 4096, None) == 4
    assert L.gaf_read_status(None, None, None) == 1
    assert L.gaf_workspace_init(None, 0, None) == 4


def test_binding_fails_loudly_without_library(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", "/nonexistent/libgaf.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        binding.lib()
