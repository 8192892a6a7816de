"""Parity harness: the CUDA library against the CPU oracle on the same bits.

Tolerances (the bar the method's target states):
  * cosine distances: 1e-5 absolute;
  * accept masks: bit-exact, except that a decision whose oracle distance lies
    within 1e-5 of tau may differ -- everything after such a flip legitimately
    changes, so the oracle is re-run with that one decision forced to the GPU's
    and the comparison continues against the replayed oracle;
  * macro-gradient: relative L2 error 1e-6 for fp32 inputs, 1e-3 for bf16.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np
import torch

import paper_2412_18052_b200 as gaf
from oracle import gaf_oracle as orc
from paper_2412_18052_b200.workloads import as_numpy_bits

DIST_ATOL = 1e-5
MACRO_RTOL = {torch.float32: 1e-6, torch.bfloat16: 1e-3}


def rel_l2(got: np.ndarray, want: np.ndarray) -> float:
    """|got - want|_2 / |want|_2, accumulated in float64 chunk by chunk."""
    num = den = 0.0
    step = 1 << 24
    for lo in range(0, want.size, step):
        w = want[lo:lo + step].astype(np.float64)
        g = got[lo:lo + step].astype(np.float64)
        num += float(np.dot(g - w, g - w))
        den += float(np.dot(w, w))
    if den == 0.0:
        return 0.0 if num == 0.0 else float("inf")
    return (num / den) ** 0.5


def oracle_with_replay(np_grads, tau, order, gpu_mask):
    """Oracle result, re-run with forced decisions where the GPU legitimately
    flipped a decision that sits within DIST_ATOL of tau.  Returns (result, replays)."""
    K = len(np_grads)
    steps = list(order) if order is not None else list(range(K))
    forced = [-1] * K
    replays = 0
    while True:
        r = orc.filter_accumulate(np_grads, tau, order=order, forced=forced if replays else None)
        bad = None
        for t in range(1, K):
            i = steps[t]
            if int(r.mask[i]) != int(gpu_mask[i]):
                bad = (t, i)
                break
        if bad is None:
            return r, replays
        t, i = bad
        assert abs(r.dist[i] - tau) < DIST_ATOL, (
            f"mask differs at step {t} (gradient {i}) with oracle distance {r.dist[i]!r} "
            f"not within {DIST_ATOL} of tau={tau}")
        forced[t] = int(gpu_mask[i])
        replays += 1
        assert replays <= K


def check_filter(grads: Sequence[torch.Tensor], tau: float, workspace: torch.Tensor,
                 order: Optional[Sequence[int]] = None, schedule: int = 0,
                 np_grads=None, expect_status: Optional[int] = 0, allow_ill_conditioned: bool = False):
    """Run gaf_filter_accumulate on the GPU and compare everything with the oracle.
    Returns a dict of the measured errors.  With `allow_ill_conditioned` a comparison that fails is
    forgiven when (and only when) the library itself raised GAF_STATUS_ILL_CONDITIONED for the call:
    the accepted gradients nearly cancelled and the library said that its tolerances do not hold."""
    try:
        return _check_filter(grads, tau, workspace, order, schedule, np_grads, expect_status)
    except AssertionError:
        if allow_ill_conditioned and (gaf.gaf_read_status(workspace) & gaf.GAF_STATUS_ILL_CONDITIONED):
            return {"ill_conditioned": True}
        raise


def _check_filter(grads, tau, workspace, order, schedule, np_grads, expect_status):
    K, D = len(grads), grads[0].numel()
    dev = grads[0].device
    # guard bands around every output catch out-of-bounds writes
    pad = 64
    macro_buf = torch.full((D + 2 * pad,), 777.0, dtype=torch.float32, device=dev)
    mask_buf = torch.full((K + 2 * pad,), 99, dtype=torch.uint8, device=dev)
    dist_buf = torch.full((K + 2 * pad,), 777.0, dtype=torch.float32, device=dev)
    count_buf = torch.full((1 + 2 * pad,), -5, dtype=torch.int32, device=dev)
    macro, mask, dist, count = gaf.gaf_filter_accumulate(
        grads, tau, workspace, order=order, schedule=schedule,
        macro_out=macro_buf[pad:pad + D], mask_out=mask_buf[pad:pad + K],
        dist_out=dist_buf[pad:pad + K], count_out=count_buf[pad:pad + 1])
    status = gaf.gaf_read_status(workspace)
    if expect_status is not None:
        assert status == expect_status, f"device status {status}, expected {expect_status}"
    for buf, fill, n in ((macro_buf, 777.0, D), (mask_buf, 99, K), (dist_buf, 777.0, K), (count_buf, -5, 1)):
        assert bool((buf[:pad] == fill).all()) and bool((buf[pad + n:] == fill).all()), "guard band overwritten"

    g_mask = mask.cpu().numpy()
    g_dist = dist.cpu().numpy().astype(np.float64)
    g_count = int(count.cpu().item())
    g_macro = macro.cpu().numpy()

    if np_grads is None:
        np_grads = [as_numpy_bits(g) for g in grads]
    r, replays = oracle_with_replay(np_grads, tau, order, g_mask)
    assert g_mask.tolist() == r.mask.tolist()
    assert g_count == r.count
    finite = np.isfinite(r.dist)
    dist_err = float(np.max(np.abs(g_dist[finite] - r.dist[finite]))) if finite.any() else 0.0
    assert dist_err <= DIST_ATOL, f"distance error {dist_err}"
    assert np.array_equal(np.isnan(g_dist), np.isnan(r.dist))
    err = rel_l2(g_macro, r.out)
    assert err <= MACRO_RTOL[grads[0].dtype], f"macro-gradient relative L2 error {err}"
    return {"dist_err": dist_err, "macro_rel_l2": err, "replays": replays, "count": g_count,
            "mask": g_mask.tolist(), "dist": g_dist.tolist()}


def check_cosdist(x: torch.Tensor, y: torch.Tensor, workspace: torch.Tensor):
    d, stats = gaf.gaf_cosdist(x, y, workspace)
    want, (p, nx, ny) = orc.cosdist(as_numpy_bits(x), as_numpy_bits(y))
    got = float(d.cpu().item())
    assert abs(got - want) <= DIST_ATOL, (got, want)
    st = stats.cpu().numpy()
    scale = (nx * ny) ** 0.5
    assert abs(st[0] - p) <= 1e-6 * scale + 1e-300
    assert abs(st[1] - nx) <= 1e-6 * nx + 1e-300 and abs(st[2] - ny) <= 1e-6 * ny + 1e-300
    return abs(got - want)


def check_pairwise(grads: Sequence[torch.Tensor], workspace: torch.Tensor):
    K = len(grads)
    dist, gram = gaf.gaf_pairwise_cosdist(grads, workspace)
    o_gram, o_dist = orc.pairwise_cosdist([as_numpy_bits(g) for g in grads])
    g_dist = dist.cpu().numpy().astype(np.float64)
    g_gram = gram.cpu().numpy()
    err = float(np.max(np.abs(g_dist - o_dist)))
    assert err <= DIST_ATOL, f"pairwise distance error {err}"
    assert np.array_equal(g_dist, g_dist.T), "distance matrix not symmetric"
    nrm = np.sqrt(np.abs(np.diag(o_gram)))
    scale = np.outer(nrm, nrm) + 1e-300
    assert float(np.max(np.abs(g_gram - o_gram) / scale)) <= 1e-5
    for i in range(K):
        assert g_dist[i, i] == (0.0 if o_gram[i, i] > 0 else 1.0)
    return err


def check_any_seed(grads: Sequence[torch.Tensor], tau: float, workspace: torch.Tensor,
                   allow_ill_conditioned: bool = False):
    """gaf_filter_accumulate_any_seed against the oracle: the winning seed, and for that
    seed everything check_filter checks (ring order starting at the seed).  `allow_ill_conditioned`
    as in check_filter."""
    K = len(grads)
    macro, mask, dist, count, seed = gaf.gaf_filter_accumulate_any_seed(grads, tau, workspace)
    status = gaf.gaf_read_status(workspace)
    try:
        return _check_any_seed(grads, tau, workspace, macro, mask, dist, count, seed)
    except AssertionError:
        if allow_ill_conditioned and (status & gaf.GAF_STATUS_ILL_CONDITIONED):
            return {"ill_conditioned": True}
        raise


def _check_any_seed(grads, tau, workspace, macro, mask, dist, count, seed):
    K = len(grads)
    np_grads = [as_numpy_bits(g) for g in grads]
    want, want_seed, counts = orc.filter_any_seed(np_grads, tau)
    g_seed = int(seed.cpu().item())
    g_mask = mask.cpu().numpy()
    order = [(g_seed + t) % K for t in range(K)]
    r, replays = oracle_with_replay(np_grads, tau, order, g_mask)
    if replays == 0:
        assert g_seed == want_seed, (g_seed, want_seed, counts.tolist())
    assert int(count.cpu().item()) == r.count and g_mask.tolist() == r.mask.tolist()
    assert r.count >= int(counts.max()) - replays
    g_dist = dist.cpu().numpy().astype(np.float64)
    assert float(np.max(np.abs(g_dist - r.dist))) <= DIST_ATOL
    assert rel_l2(macro.cpu().numpy(), r.out) <= MACRO_RTOL[grads[0].dtype]
    # bit-identical to the plain filter run in the winning order
    plain = gaf.gaf_filter_accumulate(grads, tau, workspace, order=order)
    assert torch.equal(plain[0], macro) and torch.equal(plain[1], mask)
    return {"seed": g_seed, "count": r.count, "counts": counts.tolist()}


def check_bucketed(grads: Sequence[torch.Tensor], tau: float, offsets, workspace: torch.Tensor,
                   order: Optional[Sequence[int]] = None):
    """gaf_filter_accumulate_bucketed against the oracle, bucket by bucket (with the
    near-tau replay rule applied per bucket)."""
    K, D = len(grads), grads[0].numel()
    S = len(offsets) - 1
    macro, mask, dist, count = gaf.gaf_filter_accumulate_bucketed(grads, tau, offsets, workspace, order=order)
    np_grads = [as_numpy_bits(g) for g in grads]
    g_macro = macro.cpu().numpy()
    g_mask, g_dist, g_count = mask.cpu().numpy(), dist.cpu().numpy().astype(np.float64), count.cpu().numpy()
    patterns = set()
    for b in range(S):
        lo, hi = offsets[b], offsets[b + 1]
        sub = [g[lo:hi] for g in np_grads]
        r, _ = oracle_with_replay(sub, tau, order, g_mask[b])
        assert g_mask[b].tolist() == r.mask.tolist() and int(g_count[b]) == r.count, (b, lo, hi)
        assert float(np.max(np.abs(g_dist[b] - r.dist))) <= DIST_ATOL, (b, g_dist[b], r.dist)
        if hi > lo:
            assert rel_l2(g_macro[lo:hi], r.out) <= MACRO_RTOL[grads[0].dtype], (b, lo, hi)
        patterns.add(tuple(g_mask[b].tolist()))
    return patterns
