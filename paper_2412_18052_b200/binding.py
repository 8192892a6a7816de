"""Thin ctypes binding of the C ABI in ``include/gaf.h``.

Argument marshalling only: every step of the path runs in the CUDA library.
PyTorch supplies device memory and the stream.  There is no fallback: if the
shared library has not been built, or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import torch

GAF_F32, GAF_BF16 = 0, 1
GAF_SCHED_AUTO, GAF_SCHED_STEPWISE, GAF_SCHED_GRAM, GAF_SCHED_GRAM_FUSED = 0, 1, 2, 3
GAF_STATUS_ZERO_NORM, GAF_STATUS_NONFINITE, GAF_STATUS_TIMEOUT, GAF_STATUS_ILL_CONDITIONED = 1, 2, 4, 8
GAF_MAX_K = 64

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libgaf.so")
_lib = None

EXPORTS = [
    "gaf_error_string", "gaf_workspace_bytes", "gaf_workspace_init", "gaf_cosdist",
    "gaf_filter_accumulate", "gaf_host_staging_bytes", "gaf_filter_accumulate_host",
    "gaf_pairwise_cosdist", "gaf_read_status", "gaf_last_launch_count", "gaf_cosdist_static",
    "gaf_filter_accumulate_any_seed", "gaf_stream_begin", "gaf_stream_push", "gaf_stream_end",
    "gaf_filter_accumulate_bucketed", "gaf_last_schedule", "gaf_last_gram_loader", "gaf_test_set_wait_fault",
    "gaf_filter_accumulate_repeat",
]


class GafError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib().gaf_error_string(code).decode()} (code {code})")


def lib() -> ctypes.CDLL:
    """The loaded CUDA library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2412_18052_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, i64, dbl, sz = (ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_double,
                                 ctypes.c_size_t)
        L.gaf_error_string.argtypes = [i32]
        L.gaf_error_string.restype = ctypes.c_char_p
        L.gaf_workspace_bytes.argtypes = [i32, i64, i32, ctypes.POINTER(sz)]
        L.gaf_workspace_init.argtypes = [vp, sz, vp]
        L.gaf_cosdist.argtypes = [vp, vp, i64, i32, vp, vp, vp, sz, vp]
        L.gaf_filter_accumulate.argtypes = [vp, i32, i64, i32, dbl, vp, vp, vp, vp, vp, vp, sz, i32, vp]
        L.gaf_filter_accumulate_repeat.argtypes = [i32, i32, vp, i32, i64, i32, dbl, vp, vp, vp, vp, vp, vp, sz,
                                                   i32, vp]
        L.gaf_host_staging_bytes.argtypes = [i32, i64, i32, ctypes.POINTER(sz)]
        L.gaf_filter_accumulate_host.argtypes = [vp, i32, i64, i32, dbl, vp, vp, vp, vp, vp, vp, sz,
                                                 vp, sz, i32, vp]
        L.gaf_pairwise_cosdist.argtypes = [vp, i32, i64, i32, vp, vp, vp, sz, vp]
        L.gaf_read_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
        L.gaf_last_launch_count.argtypes = []
        L.gaf_last_schedule.argtypes = []
        L.gaf_last_gram_loader.argtypes = []
        L.gaf_test_set_wait_fault.argtypes = [ctypes.c_uint, i32]
        L.gaf_cosdist_static.argtypes = [vp, vp, i64, i32, vp, vp, vp]
        L.gaf_filter_accumulate_any_seed.argtypes = [vp, i32, i64, i32, dbl, vp, vp, vp, vp, vp, vp, sz, vp]
        L.gaf_filter_accumulate_bucketed.argtypes = [vp, i32, i64, i32, dbl, vp, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.gaf_stream_begin.argtypes = [vp, i64, i32, vp, vp, sz, vp]
        L.gaf_stream_push.argtypes = [vp, i32, i64, i32, dbl, vp, vp, sz, vp]
        L.gaf_stream_end.argtypes = [i32, i64, vp, vp, vp, vp, vp, sz, vp]
        for name in EXPORTS:
            if name != "gaf_error_string":
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def _check(code: int, where: str) -> None:
    if code != 0:
        raise GafError(code, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return GAF_F32
    if t.dtype == torch.bfloat16:
        return GAF_BF16
    raise TypeError(f"gradients must be float32 or bfloat16, got {t.dtype}")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr_array(tensors: Sequence[torch.Tensor]):
    return (ctypes.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])


def _order_array(order: Optional[Sequence[int]]):
    if order is None:
        return None
    return (ctypes.c_int32 * len(order))(*[int(o) for o in order])


def gaf_workspace_bytes(K: int, D: int, dtype: int) -> int:
    out = ctypes.c_size_t()
    _check(lib().gaf_workspace_bytes(K, D, dtype, ctypes.byref(out)), "gaf_workspace_bytes")
    return out.value


def gaf_host_staging_bytes(K: int, D: int, dtype: int) -> int:
    out = ctypes.c_size_t()
    _check(lib().gaf_host_staging_bytes(K, D, dtype, ctypes.byref(out)), "gaf_host_staging_bytes")
    return out.value


def new_workspace(K: int, D: int, dtype: int, device=None) -> torch.Tensor:
    """Allocate (with torch) and initialise a workspace for calls up to this K."""
    nbytes = gaf_workspace_bytes(K, D, dtype)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device or "cuda")
    gaf_workspace_init(ws)
    return ws


def gaf_workspace_init(workspace: torch.Tensor) -> None:
    _check(lib().gaf_workspace_init(workspace.data_ptr(), workspace.numel(), _stream()),
           "gaf_workspace_init")


def gaf_cosdist(x: torch.Tensor, y: torch.Tensor, workspace: torch.Tensor,
                dist_out: Optional[torch.Tensor] = None,
                stats_out: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Eq. 4 between two device tensors.  Returns (dist[1] float32, stats[3] float64)."""
    assert x.numel() == y.numel() and x.dtype == y.dtype
    if dist_out is None:
        dist_out = torch.empty(1, dtype=torch.float32, device=x.device)
    if stats_out is None:
        stats_out = torch.empty(3, dtype=torch.float64, device=x.device)
    _check(lib().gaf_cosdist(x.data_ptr(), y.data_ptr(), x.numel(), _dtype_code(x),
                             dist_out.data_ptr(), stats_out.data_ptr(),
                             workspace.data_ptr(), workspace.numel(), _stream()), "gaf_cosdist")
    return dist_out, stats_out


def gaf_cosdist_static(x: torch.Tensor, y: torch.Tensor, dist_out: torch.Tensor,
                       stats_out: Optional[torch.Tensor] = None) -> None:
    """Eq. 4 between two device tensors without any workspace: for callers that
    may not allocate device memory (the scratch is a fixed array inside the
    library).  The outputs are the caller's tensors; nothing is allocated here
    either.  Calls must not overlap on the GPU; D is limited to 2**31."""
    assert x.numel() == y.numel() and x.dtype == y.dtype
    _check(lib().gaf_cosdist_static(x.data_ptr(), y.data_ptr(), x.numel(), _dtype_code(x),
                                    dist_out.data_ptr(),
                                    None if stats_out is None else stats_out.data_ptr(), _stream()),
           "gaf_cosdist_static")


def gaf_filter_accumulate(grads: Sequence[torch.Tensor], tau: float, workspace: torch.Tensor,
                          order: Optional[Sequence[int]] = None,
                          macro_out: Optional[torch.Tensor] = None,
                          mask_out: Optional[torch.Tensor] = None,
                          dist_out: Optional[torch.Tensor] = None,
                          count_out: Optional[torch.Tensor] = None,
                          schedule: int = GAF_SCHED_AUTO):
    """Algorithm 1 + Eq. 5 on device tensors.  Returns (macro, mask, dist, count) device tensors."""
    K, D = len(grads), grads[0].numel()
    dev = grads[0].device
    code = _dtype_code(grads[0])
    for g in grads:
        assert g.numel() == D and g.dtype == grads[0].dtype and g.is_contiguous()
    if macro_out is None:
        macro_out = torch.empty(D, dtype=torch.float32, device=dev)
    if mask_out is None:
        mask_out = torch.empty(K, dtype=torch.uint8, device=dev)
    if dist_out is None:
        dist_out = torch.empty(K, dtype=torch.float32, device=dev)
    if count_out is None:
        count_out = torch.empty(1, dtype=torch.int32, device=dev)
    ptrs = _ptr_array(grads)
    ordp = _order_array(order)
    _check(lib().gaf_filter_accumulate(ctypes.cast(ptrs, ctypes.c_void_p), K, D, code, float(tau),
                                       ordp and ctypes.cast(ordp, ctypes.c_void_p),
                                       macro_out.data_ptr(), mask_out.data_ptr(), dist_out.data_ptr(),
                                       count_out.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                       int(schedule), _stream()), "gaf_filter_accumulate")
    return macro_out, mask_out, dist_out, count_out


def gaf_filter_accumulate_repeat(repeats: int, sets: Sequence[Sequence[torch.Tensor]], tau: float,
                                 workspace: torch.Tensor, macro_out: torch.Tensor, mask_out: torch.Tensor,
                                 dist_out: torch.Tensor, count_out: torch.Tensor,
                                 order: Optional[Sequence[int]] = None, schedule: int = GAF_SCHED_AUTO) -> None:
    """``repeats`` calls of gaf_filter_accumulate issued by one C loop, call r on ``sets[r % len(sets)]``."""
    K, D = len(sets[0]), sets[0][0].numel()
    flat = [g for s in sets for g in s]
    assert all(len(s) == K for s in sets) and all(g.numel() == D and g.dtype == flat[0].dtype for g in flat)
    ptrs = _ptr_array(flat)
    ordp = _order_array(order)
    _check(lib().gaf_filter_accumulate_repeat(
        int(repeats), len(sets), ctypes.cast(ptrs, ctypes.c_void_p), K, D, _dtype_code(flat[0]), float(tau),
        ordp and ctypes.cast(ordp, ctypes.c_void_p), macro_out.data_ptr(), mask_out.data_ptr(),
        dist_out.data_ptr(), count_out.data_ptr(), workspace.data_ptr(), workspace.numel(), int(schedule),
        _stream()), "gaf_filter_accumulate_repeat")


def gaf_filter_accumulate_any_seed(grads: Sequence[torch.Tensor], tau: float, workspace: torch.Tensor,
                                   macro_out: Optional[torch.Tensor] = None):
    """Order-indifferent variant (end of Section 3.1): every gradient in turn is the seed, ring
    order, largest accepted count wins.  Returns (macro, mask, dist, count, seed) device tensors."""
    K, D = len(grads), grads[0].numel()
    dev = grads[0].device
    if macro_out is None:
        macro_out = torch.empty(D, dtype=torch.float32, device=dev)
    mask_out = torch.empty(K, dtype=torch.uint8, device=dev)
    dist_out = torch.empty(K, dtype=torch.float32, device=dev)
    count_out = torch.empty(1, dtype=torch.int32, device=dev)
    seed_out = torch.empty(1, dtype=torch.int32, device=dev)
    ptrs = _ptr_array(grads)
    _check(lib().gaf_filter_accumulate_any_seed(
        ctypes.cast(ptrs, ctypes.c_void_p), K, D, _dtype_code(grads[0]), float(tau),
        macro_out.data_ptr(), mask_out.data_ptr(), dist_out.data_ptr(), count_out.data_ptr(),
        seed_out.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream()),
        "gaf_filter_accumulate_any_seed")
    return macro_out, mask_out, dist_out, count_out, seed_out


def gaf_filter_accumulate_bucketed(grads: Sequence[torch.Tensor], tau: float, offsets: Sequence[int],
                                   workspace: torch.Tensor, order: Optional[Sequence[int]] = None,
                                   macro_out: Optional[torch.Tensor] = None):
    """Bucketed variant: Algorithm 1 + Eq. 5 independently on every bucket [offsets[b], offsets[b+1]).
    Returns (macro[D], mask[S,K], dist[S,K], count[S]) device tensors."""
    K, D = len(grads), grads[0].numel()
    S = len(offsets) - 1
    dev = grads[0].device
    if macro_out is None:
        macro_out = torch.empty(D, dtype=torch.float32, device=dev)
    mask_out = torch.empty(S, K, dtype=torch.uint8, device=dev)
    dist_out = torch.empty(S, K, dtype=torch.float32, device=dev)
    count_out = torch.empty(S, dtype=torch.int32, device=dev)
    ptrs = _ptr_array(grads)
    ordp = _order_array(order)
    offs = (ctypes.c_int64 * (S + 1))(*[int(o) for o in offsets])
    _check(lib().gaf_filter_accumulate_bucketed(
        ctypes.cast(ptrs, ctypes.c_void_p), K, D, _dtype_code(grads[0]), float(tau),
        ordp and ctypes.cast(ordp, ctypes.c_void_p), S, ctypes.cast(offs, ctypes.c_void_p),
        macro_out.data_ptr(), mask_out.data_ptr(), dist_out.data_ptr(), count_out.data_ptr(),
        workspace.data_ptr(), workspace.numel(), _stream()), "gaf_filter_accumulate_bucketed")
    return macro_out, mask_out, dist_out, count_out


def gaf_stream_begin(seed: torch.Tensor, acc: torch.Tensor, workspace: torch.Tensor) -> None:
    """Streaming form: g <- seed, c <- 1 (``acc`` is the caller's float32 running sum)."""
    _check(lib().gaf_stream_begin(seed.data_ptr(), seed.numel(), _dtype_code(seed), acc.data_ptr(),
                                  workspace.data_ptr(), workspace.numel(), _stream()), "gaf_stream_begin")


def gaf_stream_push(g: torch.Tensor, t: int, tau: float, acc: torch.Tensor, workspace: torch.Tensor) -> None:
    """Streaming form: test gradient number t (arrival order, from 1) and add it if accepted."""
    _check(lib().gaf_stream_push(g.data_ptr(), int(t), g.numel(), _dtype_code(g), float(tau), acc.data_ptr(),
                                 workspace.data_ptr(), workspace.numel(), _stream()), "gaf_stream_push")


def gaf_stream_end(K: int, acc: torch.Tensor, workspace: torch.Tensor):
    """Streaming form: acc <- g / c.  Returns (mask[K], dist[K], count) in arrival order."""
    dev = acc.device
    mask = torch.empty(K, dtype=torch.uint8, device=dev)
    dist = torch.empty(K, dtype=torch.float32, device=dev)
    count = torch.empty(1, dtype=torch.int32, device=dev)
    _check(lib().gaf_stream_end(int(K), acc.numel(), acc.data_ptr(), mask.data_ptr(), dist.data_ptr(),
                                count.data_ptr(), workspace.data_ptr(), workspace.numel(), _stream()),
           "gaf_stream_end")
    return mask, dist, count


def gaf_filter_accumulate_host(grads_host: Sequence[torch.Tensor], tau: float,
                               staging: torch.Tensor, workspace: torch.Tensor,
                               macro_out_host: torch.Tensor, mask_out_host: torch.Tensor,
                               dist_out_host: torch.Tensor, count_out_host: torch.Tensor,
                               order: Optional[Sequence[int]] = None,
                               schedule: int = GAF_SCHED_AUTO) -> None:
    """Same operation on HOST tensors (pinned for speed); synchronises the stream."""
    K, D = len(grads_host), grads_host[0].numel()
    code = _dtype_code(grads_host[0])
    ptrs = _ptr_array(grads_host)
    ordp = _order_array(order)
    _check(lib().gaf_filter_accumulate_host(
        ctypes.cast(ptrs, ctypes.c_void_p), K, D, code, float(tau),
        ordp and ctypes.cast(ordp, ctypes.c_void_p),
        macro_out_host.data_ptr(), mask_out_host.data_ptr(), dist_out_host.data_ptr(),
        count_out_host.data_ptr(), staging.data_ptr(), staging.numel(),
        workspace.data_ptr(), workspace.numel(), int(schedule), _stream()),
        "gaf_filter_accumulate_host")


def gaf_pairwise_cosdist(grads: Sequence[torch.Tensor], workspace: torch.Tensor,
                         dist_out: Optional[torch.Tensor] = None,
                         gram_out: Optional[torch.Tensor] = None):
    """K x K cosine-distance matrix (float32) and Gram matrix (float64) on the device."""
    K, D = len(grads), grads[0].numel()
    dev = grads[0].device
    if dist_out is None:
        dist_out = torch.empty(K, K, dtype=torch.float32, device=dev)
    if gram_out is None:
        gram_out = torch.empty(K, K, dtype=torch.float64, device=dev)
    ptrs = _ptr_array(grads)
    _check(lib().gaf_pairwise_cosdist(ctypes.cast(ptrs, ctypes.c_void_p), K, D, _dtype_code(grads[0]),
                                      dist_out.data_ptr(), gram_out.data_ptr(),
                                      workspace.data_ptr(), workspace.numel(), _stream()),
           "gaf_pairwise_cosdist")
    return dist_out, gram_out


def gaf_read_status(workspace: torch.Tensor) -> int:
    """Status bits of the latest call on this workspace (synchronises the stream)."""
    out = ctypes.c_int()
    _check(lib().gaf_read_status(workspace.data_ptr(), _stream(), ctypes.byref(out)), "gaf_read_status")
    return out.value


def gaf_last_launch_count() -> int:
    return lib().gaf_last_launch_count()


def gaf_last_schedule() -> int:
    """The GAF_SCHED_* value the latest gaf_filter_accumulate call of this thread ran with."""
    return lib().gaf_last_schedule()


def gaf_last_gram_loader() -> int:
    """How the tensor-memory Gram kernel of this thread's latest call fetched its tiles: 0 not used,
    1 16-byte copies, 2 tensor copies (gradients that are rows of one matrix)."""
    return lib().gaf_last_gram_loader()


def gaf_test_set_wait_fault(wait_limit: int, withhold: bool) -> None:
    """Test hook: poll limit of the kernels' bounded waits and whether the awaited signal is withheld,
    for the following launches of this thread.  ``(0, False)`` restores normal operation."""
    _check(lib().gaf_test_set_wait_fault(int(wait_limit), 1 if withhold else 0), "gaf_test_set_wait_fault")
