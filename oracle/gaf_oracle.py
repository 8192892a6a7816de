"""ctypes front end of the fp64 CPU oracle (``gaf_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  The product package never imports it, and it
imports nothing from the product package.

The arithmetic lives in the C file, one plain loop per step of Algorithm 1 /
Eq. 4 / Eq. 5 of the paper; this module only compiles it with gcc and marshals
numpy arrays.  Inputs are numpy arrays of dtype float32 (fp32 gradients) or
uint16 (bfloat16 bit patterns).

Parity unpinned (conventions of this implementation, the paper is silent): the
zero-norm rule, the treatment of NaN distances, and reading the update/skip
block of Algorithm 1 as sitting after the inner loop.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gaf_oracle.c")
_LIB = os.path.join(_HERE, "libgaf_oracle.so")
_SRC_MT = os.path.join(_HERE, "gaf_oracle_mt.c")
_LIB_MT = os.path.join(_HERE, "libgaf_oracle_mt.so")
_lib = None
_lib_mt = None
_lib_override = None   # set by tests that load a deliberately broken copy


def compile_c(src: str, lib: str) -> str:
    """gcc, no fast-math: every sum keeps the order it is written in."""
    tmp = lib + f".{os.getpid()}.tmp"
    subprocess.check_call(
        ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fno-fast-math", "-pthread",
         "-I", _HERE, "-o", tmp, src, "-lm"])
    os.replace(tmp, lib)
    return lib


def build(force: bool = False) -> str:
    """Compile the oracle if its shared object is missing or older than the source."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        compile_c(_SRC, _LIB)
    # the several-threads form of the filter (gaf_oracle_mt.c includes gaf_oracle.c)
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_MT))
    if force or (not os.path.exists(_LIB_MT)) or os.path.getmtime(_LIB_MT) < newest:
        compile_c(_SRC_MT, _LIB_MT)
    return _LIB


def use_library(path: Optional[str]) -> None:
    """Point the wrapper at another build of the oracle (``None`` = the real
    one).  Only the mutation tests use this, to check that the pins notice a
    planted mistake."""
    global _lib, _lib_override
    _lib_override = path
    _lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_lib_override or build())
        vp, i64, i32, dbl = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_double
        lib.gaf_oracle_cosdist.argtypes = [vp, vp, i64, i32, vp, vp]
        lib.gaf_oracle_filter_accumulate.argtypes = [vp, i32, i64, i32, dbl, vp, vp, vp, vp, vp, vp, vp]
        lib.gaf_oracle_filter_any_seed.argtypes = [vp, i32, i64, i32, dbl, vp, vp, vp, vp, vp, vp, vp]
        lib.gaf_oracle_filter_any_seed.restype = ctypes.c_int
        lib.gaf_oracle_filter_bucketed.argtypes = [vp, i32, i64, i32, dbl, vp, i32, vp, vp, vp, vp, vp]
        lib.gaf_oracle_filter_bucketed.restype = ctypes.c_int
        lib.gaf_oracle_pairwise.argtypes = [vp, i32, i64, i32, vp, vp]
        lib.gaf_oracle_plain_average.argtypes = [vp, i32, i64, i32, vp]
        for f in (lib.gaf_oracle_cosdist, lib.gaf_oracle_filter_accumulate,
                  lib.gaf_oracle_pairwise, lib.gaf_oracle_plain_average):
            f.restype = ctypes.c_int
        _lib = lib
    return _lib


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return 0
    if a.dtype == np.uint16:
        return 1
    raise TypeError(f"oracle takes float32 or uint16 (bf16 bits) arrays, got {a.dtype}")


def _prep(grads: Sequence[np.ndarray]):
    arrs = [np.ascontiguousarray(g).reshape(-1) for g in grads]
    code = _dtype_code(arrs[0])
    D = arrs[0].size
    for a in arrs:
        if a.size != D or _dtype_code(a) != code:
            raise ValueError("all micro-gradients must share length and dtype")
    ptrs = (ctypes.c_void_p * len(arrs))(*[a.ctypes.data for a in arrs])
    return arrs, ptrs, code, D


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns (uint16) to float64."""
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def cosdist(x: np.ndarray, y: np.ndarray):
    """Eq. 4.  Returns (distance, (x.y, |x|^2, |y|^2))."""
    (x, y), _, code, D = _prep([x, y])
    dist = ctypes.c_double()
    stats = (ctypes.c_double * 3)()
    _load().gaf_oracle_cosdist(x.ctypes.data, y.ctypes.data, D, code,
                               ctypes.addressof(dist), ctypes.addressof(stats))
    return dist.value, tuple(stats)


@dataclass
class FilterResult:
    out: np.ndarray      # float64 [D]: g / c
    mask: np.ndarray     # uint8 [K], original index
    dist: np.ndarray     # float64 [K], original index, 0 at the seed
    count: int           # c
    stats: np.ndarray    # float64 [K, 3]: {g_i.g, |g|^2, |g_i|^2} at the test of g_i


def filter_accumulate(grads: Sequence[np.ndarray], tau: float,
                      order: Optional[Sequence[int]] = None,
                      forced: Optional[Sequence[int]] = None) -> FilterResult:
    """Algorithm 1 (one macrobatch) followed by Eq. 5.

    ``forced[t]`` (t = step index 1..K-1; entry 0 ignored) overrides the
    decision of step t when it is 0 or 1; -1 leaves the test in charge.
    """
    arrs, ptrs, code, D = _prep(grads)
    K = len(arrs)
    order_arr = None
    if order is not None:
        order_arr = np.ascontiguousarray(order, dtype=np.int32)
        if sorted(order_arr.tolist()) != list(range(K)):
            raise ValueError("order must be a permutation of 0..K-1")
    forced_arr = None
    if forced is not None:
        forced_arr = np.ascontiguousarray(forced, dtype=np.int8)
        if forced_arr.size != K:
            raise ValueError("forced needs K entries")
    out = np.empty(D, dtype=np.float64)
    mask = np.zeros(K, dtype=np.uint8)
    dist = np.zeros(K, dtype=np.float64)
    stats = np.zeros((K, 3), dtype=np.float64)
    count = ctypes.c_int32()
    rc = _load().gaf_oracle_filter_accumulate(
        ctypes.cast(ptrs, ctypes.c_void_p), K, D, code, float(tau),
        None if order_arr is None else order_arr.ctypes.data,
        None if forced_arr is None else forced_arr.ctypes.data,
        out.ctypes.data, mask.ctypes.data, dist.ctypes.data,
        ctypes.addressof(count), stats.ctypes.data)
    if rc != 0:
        raise ValueError("oracle rejected its arguments")
    return FilterResult(out, mask, dist, int(count.value), stats)


def filter_accumulate_all_cores(grads: Sequence[np.ndarray], tau: float,
                                order: Optional[Sequence[int]] = None,
                                n_threads: Optional[int] = None) -> FilterResult:
    """The same Algorithm 1 + Eq. 5 with every pass over the D parameters split into
    ``n_threads`` consecutive chunks (default: the cores this process may run on), the sums
    of each test combined in chunk order.  For the all-cores CPU baseline of the benchmark."""
    global _lib_mt
    if _lib_mt is None:
        build()
        lib = ctypes.CDLL(_LIB_MT)
        vp, i64, i32, dbl = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_double
        lib.gaf_oracle_filter_accumulate_mt.argtypes = [vp, i32, i64, i32, dbl, vp, vp, vp, vp, vp, i32]
        lib.gaf_oracle_filter_accumulate_mt.restype = ctypes.c_int
        _lib_mt = lib
    if n_threads is None:
        n_threads = host_cores()
    arrs, ptrs, code, D = _prep(grads)
    K = len(arrs)
    order_arr = None if order is None else np.ascontiguousarray(order, dtype=np.int32)
    out = np.empty(D, dtype=np.float64)
    mask = np.zeros(K, dtype=np.uint8)
    dist = np.zeros(K, dtype=np.float64)
    count = ctypes.c_int32()
    rc = _lib_mt.gaf_oracle_filter_accumulate_mt(
        ctypes.cast(ptrs, ctypes.c_void_p), K, D, code, float(tau),
        None if order_arr is None else order_arr.ctypes.data,
        out.ctypes.data, mask.ctypes.data, dist.ctypes.data, ctypes.addressof(count), int(n_threads))
    if rc != 0:
        raise ValueError("oracle rejected its arguments or could not start its threads")
    return FilterResult(out, mask, dist, int(count.value), np.zeros((K, 3)))


def host_cores() -> int:
    """Cores this process may run on."""
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def filter_any_seed(grads: Sequence[np.ndarray], tau: float):
    """Order-indifferent variant (end of Section 3.1): Algorithm 1 from every seed in ring
    order, keep the largest accepted count (ties: smallest seed).
    Returns (FilterResult of the winner, seed, counts per seed)."""
    arrs, ptrs, code, D = _prep(grads)
    K = len(arrs)
    out = np.empty(D, dtype=np.float64)
    work = np.empty(D, dtype=np.float64)
    mask = np.zeros(K, dtype=np.uint8)
    dist = np.zeros(K, dtype=np.float64)
    counts = np.zeros(K, dtype=np.int32)
    count, seed = ctypes.c_int32(), ctypes.c_int32()
    rc = _load().gaf_oracle_filter_any_seed(
        ctypes.cast(ptrs, ctypes.c_void_p), K, D, code, float(tau), out.ctypes.data,
        mask.ctypes.data, dist.ctypes.data, ctypes.addressof(count), ctypes.addressof(seed),
        counts.ctypes.data, work.ctypes.data)
    if rc != 0:
        raise ValueError("oracle rejected its arguments")
    res = FilterResult(out, mask, dist, int(count.value), np.zeros((K, 3)))
    return res, int(seed.value), counts


def filter_bucketed(grads: Sequence[np.ndarray], tau: float, offsets: Sequence[int],
                    order: Optional[Sequence[int]] = None):
    """Bucketed variant: Algorithm 1 + Eq. 5 independently on every bucket
    [offsets[b], offsets[b+1]).  Returns (out[D], mask[S,K], dist[S,K], count[S])."""
    arrs, ptrs, code, D = _prep(grads)
    K = len(arrs)
    off = np.ascontiguousarray(offsets, dtype=np.int64)
    S = off.size - 1
    order_arr = None if order is None else np.ascontiguousarray(order, dtype=np.int32)
    out = np.empty(D, dtype=np.float64)
    mask = np.zeros((S, K), dtype=np.uint8)
    dist = np.zeros((S, K), dtype=np.float64)
    count = np.zeros(S, dtype=np.int32)
    rc = _load().gaf_oracle_filter_bucketed(
        ctypes.cast(ptrs, ctypes.c_void_p), K, D, code, float(tau),
        None if order_arr is None else order_arr.ctypes.data, S, off.ctypes.data,
        out.ctypes.data, mask.ctypes.data, dist.ctypes.data, count.ctypes.data)
    if rc != 0:
        raise ValueError("oracle rejected its arguments")
    return out, mask, dist, count


def pairwise_cosdist(grads: Sequence[np.ndarray]):
    """K x K Gram matrix and cosine-distance matrix (Eq. 4 for every pair)."""
    arrs, ptrs, code, D = _prep(grads)
    K = len(arrs)
    gram = np.zeros((K, K), dtype=np.float64)
    dist = np.zeros((K, K), dtype=np.float64)
    _load().gaf_oracle_pairwise(ctypes.cast(ptrs, ctypes.c_void_p), K, D, code,
                                gram.ctypes.data, dist.ctypes.data)
    return gram, dist


def plain_average(grads: Sequence[np.ndarray]) -> np.ndarray:
    """Eq. 2: (1/k) sum_i g_i."""
    arrs, ptrs, code, D = _prep(grads)
    out = np.empty(D, dtype=np.float64)
    _load().gaf_oracle_plain_average(ctypes.cast(ptrs, ctypes.c_void_p), len(arrs), D, code,
                                     out.ctypes.data)
    return out
