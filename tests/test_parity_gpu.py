"""GPU parity tests proper: every entry point, through the C ABI, against the CPU
oracle on the same seeded inputs."""
import math

import numpy as np
import pytest
import torch

import paper_2412_18052_b200 as gaf
from paper_2412_18052_b200 import workloads
from parity import check_any_seed, check_bucketed, check_cosdist, check_filter, check_pairwise

pytestmark = pytest.mark.gpu

SCHEDULES = [gaf.GAF_SCHED_STEPWISE, gaf.GAF_SCHED_GRAM, gaf.GAF_SCHED_GRAM_FUSED]
SCHED_IDS = ["stepwise", "gram", "gram-one-launch"]
DTYPES = ["f32", "bf16"]


@pytest.fixture(scope="module")
def ws():
    return gaf.new_workspace(gaf.binding.GAF_MAX_K, 1 << 20, gaf.GAF_F32)


def _mix(K, D, dtype, seed, rho=None, sigma=1e-3, stacked=False):
    rng = np.random.RandomState(seed)
    if rho is None:
        rho = rng.uniform(-0.4, 0.9, size=K)
    return workloads.mixture(K, D, dtype, list(rho), seed, device="cuda", sigma=sigma, stacked=stacked)


def _scattered(grads):
    """The same gradients at unequal distances from one another: rows of a wider matrix, two of them swapped."""
    K, D = len(grads), grads[0].numel()
    matrix = torch.empty(K + 1, (D + 127) // 128 * 128 + 128, dtype=grads[0].dtype, device=grads[0].device)
    rows = list(range(K))
    rows[1], rows[K - 1] = K, 1
    out = [matrix[r, :D] for r in rows]
    for o, g in zip(out, grads):
        o.copy_(g)
    return out


# ------------------------------------------------------------------ Eq. 4 ----

@pytest.mark.parametrize("dtype", DTYPES)
def test_cosdist_every_small_length(ws, dtype):
    for D in list(range(0, 41)) + [63, 64, 65, 511, 4095, 4097]:
        w = _mix(2, D, dtype, seed=100 + D, rho=[0.6, 0.3])
        check_cosdist(w.grads[0], w.grads[1], ws)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("D", [1_000_003, 8 * 512 * 296 * 3 + 5])
def test_cosdist_several_waves_and_ragged_tail(ws, dtype, D):
    w = _mix(2, D, dtype, seed=7, rho=[0.2, -0.5])
    err = check_cosdist(w.grads[0], w.grads[1], ws)
    assert err < 1e-6


def test_cosdist_stated_values(ws):
    x = torch.randn(10_001, device="cuda")
    for y, want in ((x.clone(), 0.0), (-x, 2.0)):
        d, _ = gaf.gaf_cosdist(x, y, ws)
        assert abs(float(d.item()) - want) < 1e-6
    a = torch.zeros(10_001, device="cuda"); a[:5000] = 1.0
    b = torch.zeros(10_001, device="cuda"); b[5000:] = 2.0
    d, _ = gaf.gaf_cosdist(a, b, ws)
    assert float(d.item()) == 1.0
    # zero-norm convention: distance 1 and a status bit
    d, _ = gaf.gaf_cosdist(a, torch.zeros_like(a), ws)
    assert float(d.item()) == 1.0 and gaf.gaf_read_status(ws) == gaf.GAF_STATUS_ZERO_NORM


# ------------------------------------------------------------ Algorithm 1 ----

@pytest.mark.parametrize("schedule", SCHEDULES, ids=SCHED_IDS)
@pytest.mark.parametrize("dtype", DTYPES)
def test_filter_small_shapes_every_tail(ws, schedule, dtype):
    """K = 1, 2, 3, 5 and every D mod 8 (and D below one vector), several thresholds."""
    for K in (1, 2, 3, 5):
        for D in (0, 1, 3, 7, 8, 9, 15, 16, 17, 31, 33, 100, 257, 4096, 4099, 8200 + K):
            w = _mix(K, D, dtype, seed=K * 1000 + D)
            for tau in (0.5, 0.97, 1.2):
                status = None if D == 0 else 0
                check_filter(w.grads, tau, ws, schedule=schedule, expect_status=status)


@pytest.mark.parametrize("schedule", SCHEDULES, ids=SCHED_IDS)
@pytest.mark.parametrize("dtype", DTYPES)
def test_filter_several_tiles_ragged(ws, schedule, dtype):
    """Sizes that span several tiles per CTA, with a ragged tail, all accept patterns."""
    D = 148 * 4096 * 3 + 148 * 1000 + 5
    w = _mix(6, D, dtype, seed=42, rho=[0.8, 0.7, -0.6, 0.5, 0.0, 0.6])
    seen = set()
    for tau in (0.2, 0.6, 0.97, 1.5):
        r = check_filter(w.grads, tau, ws, schedule=schedule)
        seen.add(tuple(r["mask"]))
        assert r["dist_err"] < 1e-6
    assert len(seen) >= 3


@pytest.mark.parametrize("schedule", SCHEDULES, ids=SCHED_IDS)
def test_filter_order_and_special_thresholds(ws, schedule):
    w = _mix(5, 50_001, "f32", seed=3, rho=[0.9, 0.8, 0.0, 0.7, -0.5])
    for order in (None, [4, 3, 2, 1, 0], [2, 0, 1, 3, 4], [1, 4, 0, 2, 3]):
        check_filter(w.grads, 0.9, ws, order=order, schedule=schedule)
    # tau >= 2 admits everything: the plain mean of Eq. 2
    r = check_filter(w.grads, 2.0, ws, schedule=schedule)
    assert r["mask"] == [1] * 5 and r["count"] == 5
    macro, *_ = gaf.gaf_filter_accumulate(w.grads, 2.0, ws, schedule=schedule)
    mean = torch.stack([g.double() for g in w.grads]).mean(0)
    assert float((macro.double() - mean).norm() / mean.norm()) < 1e-6
    # a threshold nothing meets keeps only the seed, bit for bit
    for order in (None, [3, 1, 0, 2, 4]):
        r = check_filter(w.grads, -1.0, ws, order=order, schedule=schedule)
        s = 0 if order is None else order[0]
        assert r["count"] == 1 and r["mask"] == [1 if i == s else 0 for i in range(5)]
        macro, *_ = gaf.gaf_filter_accumulate(w.grads, -1.0, ws, order=order, schedule=schedule)
        assert torch.equal(macro, w.grads[s])


@pytest.mark.parametrize("schedule", SCHEDULES, ids=SCHED_IDS)
def test_filter_degenerate_inputs(ws, schedule):
    D = 20_011
    g = torch.randn(D, device="cuda") * 1e-3
    z = torch.zeros(D, device="cuda")
    # identical and opposite gradients
    r = check_filter([g, g.clone(), -g], 0.97, ws, schedule=schedule)
    assert r["mask"] == [1, 1, 0] and abs(r["dist"][1]) < 1e-6 and abs(r["dist"][2] - 2.0) < 1e-6
    # inclusive threshold: exactly orthogonal integer vectors, tau = 1
    a = torch.zeros(D, device="cuda"); a[: D // 2] = 3.0
    b = torch.zeros(D, device="cuda"); b[D // 2:] = -2.0
    r = check_filter([a, b], 1.0, ws, schedule=schedule)
    assert r["dist"][1] == 1.0 and r["mask"] == [1, 1]
    r = check_filter([a, b], math.nextafter(1.0, 0.0), ws, schedule=schedule)
    assert r["mask"] == [1, 0]
    # zero-norm convention (distance 1) raises a status bit, on either side of the pair
    r = check_filter([g, z, g.clone()], 0.97, ws, schedule=schedule,
                     expect_status=gaf.GAF_STATUS_ZERO_NORM)
    assert r["mask"] == [1, 0, 1] and r["dist"][1] == 1.0
    r = check_filter([z, g], 1.0, ws, schedule=schedule, expect_status=gaf.GAF_STATUS_ZERO_NORM)
    assert r["mask"] == [1, 1]
    # accepted gradients that cancel exactly leave a zero running sum (tau = 2 admits all)
    h = torch.randn(D, device="cuda") * 1e-3
    # (the library flags both facts: the zero norm at the next test, and the cancellation that caused it)
    r = check_filter([g, -g, h], 2.0, ws, schedule=schedule,
                     expect_status=gaf.GAF_STATUS_ZERO_NORM | gaf.GAF_STATUS_ILL_CONDITIONED)
    assert r["mask"] == [1, 1, 1] and r["dist"][2] == 1.0
    # a NaN makes the distance NaN, which is rejected
    bad = g.clone(); bad[17] = float("nan")
    r = check_filter([g, bad, g.clone()], 1.5, ws, schedule=schedule,
                     expect_status=gaf.GAF_STATUS_NONFINITE)
    assert r["mask"] == [1, 0, 1] and math.isnan(r["dist"][1])
    # wide dynamic range across the vector (a few large tensors dominate the sums)
    scale = torch.ones(D, device="cuda"); scale[:100] = 1e4; scale[100:5000] = 1e-4
    gs = [(torch.randn(D, device="cuda") + 0.5) * scale for _ in range(4)]
    check_filter(gs, 0.97, ws, schedule=schedule)


@pytest.mark.parametrize("schedule", SCHEDULES, ids=SCHED_IDS)
def test_filter_maximum_k(ws, schedule):
    K = gaf.binding.GAF_MAX_K
    w = _mix(K, 10_007, "bf16", seed=64)
    if schedule == gaf.GAF_SCHED_GRAM_FUSED:
        # the one-launch form handles up to 8 gradients and says so beyond
        with pytest.raises(gaf.GafError) as e:
            gaf.gaf_filter_accumulate(w.grads, 0.97, ws, schedule=schedule)
        assert e.value.code == 7
        w = _mix(8, 10_007, "bf16", seed=64)
        r = check_filter(w.grads, 0.97, ws, schedule=schedule)
        assert 1 < r["count"] < 8
        return
    r = check_filter(w.grads, 0.97, ws, schedule=schedule)
    assert 1 < r["count"] < K


@pytest.mark.parametrize("K", [9, 16, 24, 32, 33, 48, 64])
def test_filter_gram_first_on_tensor_cores(ws, K):
    """bf16 with 9..64 gradients: the Gram matrix comes from the tensor cores -- warp-level MMAs fed from
    the global loads up to 16 gradients (two blocks of 8 rows), the tcgen05 tile beyond."""
    w = _mix(K, 1_000_003 + 64 * K, "bf16", seed=200 + K)
    r = check_filter(w.grads, 0.97, ws, schedule=gaf.GAF_SCHED_GRAM)
    assert 1 < r["count"] < K


@pytest.mark.parametrize("schedule", SCHEDULES, ids=SCHED_IDS)
def test_filter_bitwise_reproducible_and_workspace_reusable(ws, schedule):
    """Fixed-order reductions: two runs agree bit for bit; the workspace needs no
    re-initialisation between calls."""
    w = _mix(4, 3_000_017, "f32", seed=9, rho=[0.8, 0.6, -0.2, 0.7])
    outs = []
    for _ in range(3):
        macro, mask, dist, count = gaf.gaf_filter_accumulate(w.grads, 0.8, ws, schedule=schedule)
        outs.append((macro.clone(), mask.clone(), dist.clone(), count.clone()))
    for o in outs[1:]:
        for x, y in zip(outs[0], o):
            assert torch.equal(x, y)


def test_schedules_agree(ws):
    w = _mix(5, 2_000_003, "bf16", seed=12)
    a = gaf.gaf_filter_accumulate(w.grads, 0.9, ws, schedule=gaf.GAF_SCHED_STEPWISE)
    a = [t.clone() for t in a]
    outs = {}
    for other in (gaf.GAF_SCHED_GRAM, gaf.GAF_SCHED_GRAM_FUSED, gaf.GAF_SCHED_AUTO):
        b = gaf.gaf_filter_accumulate(w.grads, 0.9, ws, schedule=other)
        assert torch.equal(a[1], b[1]) and torch.equal(a[3], b[3])
        assert float((a[2] - b[2]).abs().max()) < 1e-6
        assert torch.equal(a[0], b[0])       # element arithmetic is identical in every schedule
        outs[other] = [t.clone() for t in b]
    # the two forms of the Gram-first schedule take the same sums in the same order
    for x, y in zip(outs[gaf.GAF_SCHED_GRAM], outs[gaf.GAF_SCHED_GRAM_FUSED]):
        assert torch.equal(x, y)


def test_filter_host_entry_point(ws):
    w = _mix(4, 100_003, "f32", seed=5, rho=[0.8, 0.6, -0.2, 0.7])
    host = [g.cpu().pin_memory() for g in w.grads]
    K, D = 4, 100_003
    staging = torch.empty(gaf.gaf_host_staging_bytes(K, D, gaf.GAF_F32), dtype=torch.uint8, device="cuda")
    macro_h = torch.empty(D, dtype=torch.float32).pin_memory()
    mask_h = torch.empty(K, dtype=torch.uint8).pin_memory()
    dist_h = torch.empty(K, dtype=torch.float32).pin_memory()
    count_h = torch.empty(1, dtype=torch.int32).pin_memory()
    gaf.gaf_filter_accumulate_host(host, 0.8, staging, ws, macro_h, mask_h, dist_h, count_h)
    macro, mask, dist, count = gaf.gaf_filter_accumulate(w.grads, 0.8, ws)
    assert torch.equal(macro.cpu(), macro_h) and torch.equal(mask.cpu(), mask_h)
    assert torch.equal(dist.cpu(), dist_h) and int(count.item()) == int(count_h.item())


def test_repeat_entry_point(ws):
    """gaf_filter_accumulate_repeat is a host loop in C around gaf_filter_accumulate: after r calls over
    rotating input sets the outputs are those of the last set used, and the launches add up."""
    sets = [_mix(4, 200_003, "f32", seed=70 + i, rho=[0.8, 0.6, -0.2, 0.7] if i else [0.7, -0.3, 0.5, 0.1]).grads
            for i in range(3)]
    D = 200_003
    macro = torch.empty(D, device="cuda"); mask = torch.empty(4, dtype=torch.uint8, device="cuda")
    dist = torch.empty(4, device="cuda"); count = torch.empty(1, dtype=torch.int32, device="cuda")
    for repeats in (1, 3, 5):
        gaf.gaf_filter_accumulate_repeat(repeats, sets, 0.9, ws, macro, mask, dist, count)
        launches = gaf.gaf_last_launch_count()
        want = gaf.gaf_filter_accumulate(sets[(repeats - 1) % 3], 0.9, ws)
        assert launches == repeats * gaf.gaf_last_launch_count()
        assert torch.equal(macro, want[0]) and torch.equal(mask, want[1])
        assert torch.equal(dist, want[2]) and torch.equal(count, want[3])
    gaf.gaf_filter_accumulate_repeat(0, sets, 0.9, ws, macro, mask, dist, count)     # nothing to do is legal
    assert gaf.gaf_last_launch_count() == 0


def test_one_launch_calls_do_not_overlap_across_streams(ws):
    """A one-launch call needs the whole device.  While one is in flight on a stream, an explicit request on
    another stream is refused and the library's own choice takes two launches; ordered on one stream, or once
    the first stream is idle, the one-launch form runs again.  Results are correct throughout."""
    w = _mix(4, 30_000_011, "f32", seed=88, rho=[0.8, 0.6, -0.2, 0.7])       # a call of about 150 us
    small = _mix(4, 100_003, "f32", seed=89, rho=[0.8, 0.6, -0.2, 0.7])
    ws2 = gaf.new_workspace(4, 1 << 20, gaf.GAF_F32)
    want = [t.clone() for t in gaf.gaf_filter_accumulate(small.grads, 0.9, ws2, schedule=gaf.GAF_SCHED_GRAM)]
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    refused = fell_back = 0
    for _ in range(5):
        with torch.cuda.stream(s1):
            for _ in range(4):
                gaf.gaf_filter_accumulate(w.grads, 0.9, ws, schedule=gaf.GAF_SCHED_GRAM_FUSED)   # same stream: fine
        with torch.cuda.stream(s2):
            try:
                gaf.gaf_filter_accumulate(small.grads, 0.9, ws2, schedule=gaf.GAF_SCHED_GRAM_FUSED)
            except gaf.GafError as e:
                assert e.code == 7
                refused += 1
            got = gaf.gaf_filter_accumulate(small.grads, 0.9, ws2)            # AUTO: whatever may run now
            fell_back += gaf.gaf_last_schedule() == gaf.GAF_SCHED_GRAM
        torch.cuda.synchronize()
        for x, y in zip(got, want):
            assert torch.equal(x, y)
    assert refused >= 1 and fell_back >= 1          # (0.6 ms of work was pending on the first stream each time)
    with torch.cuda.stream(s2):
        gaf.gaf_filter_accumulate(small.grads, 0.9, ws2, schedule=gaf.GAF_SCHED_GRAM_FUSED)      # first stream idle: fine
    torch.cuda.synchronize()
    check_filter(w.grads, 0.9, ws, schedule=gaf.GAF_SCHED_GRAM_FUSED)


def test_calls_captured_into_a_graph(ws):
    """Calls made while the stream is being captured into a CUDA graph: the library's own choice takes the forms
    that need no co-resident grid (two launches), an explicit request for the one-launch form is refused, and
    replaying the graph on new inputs (same buffers) gives what the oracle gives."""
    from oracle import gaf_oracle as orc
    cases = [(4, 300_007, "f32"), (2, 100_003, "f32"), (8, 200_001, "bf16"), (32, 70_001, "bf16")]
    for K, D, dtype in cases:
        w = _mix(K, D, dtype, seed=40 + K)
        macro = torch.empty(D, dtype=torch.float32, device="cuda")
        mask = torch.empty(K, dtype=torch.uint8, device="cuda")
        dist = torch.empty(K, dtype=torch.float32, device="cuda")
        count = torch.empty(1, dtype=torch.int32, device="cuda")
        args = dict(macro_out=macro, mask_out=mask, dist_out=dist, count_out=count)
        gaf.gaf_filter_accumulate(w.grads, 0.97, ws, **args)            # plans and attributes outside the capture
        gaf.gaf_filter_accumulate(w.grads, 0.97, ws, schedule=gaf.GAF_SCHED_GRAM, **args)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            gaf.gaf_filter_accumulate(w.grads, 0.97, ws, **args)
            assert gaf.gaf_last_schedule() == gaf.GAF_SCHED_GRAM, (K, gaf.gaf_last_schedule())
            if K <= 8:
                with pytest.raises(gaf.GafError):
                    gaf.gaf_filter_accumulate(w.grads, 0.97, ws, schedule=gaf.GAF_SCHED_GRAM_FUSED, **args)
        other = _mix(K, D, dtype, seed=90 + K)
        for g, o in zip(w.grads, other.grads):
            g.copy_(o)
        macro.fill_(7.0)
        graph.replay()
        torch.cuda.synchronize()
        want = orc.filter_accumulate([workloads.as_numpy_bits(g) for g in w.grads], 0.97)
        assert mask.cpu().numpy().tolist() == want.mask.tolist() and int(count.item()) == want.count
        assert float(np.max(np.abs(dist.cpu().numpy() - want.dist))) < 1e-5
        got = macro.cpu().numpy().astype(np.float64)
        assert float(np.linalg.norm(got - want.out) / np.linalg.norm(want.out)) < (1e-6 if dtype == "f32" else 1e-3)
        # and outside a capture the one-launch form is back
        gaf.gaf_filter_accumulate(w.grads, 0.97, ws, **args)
        if K <= 8:
            assert gaf.gaf_last_schedule() == gaf.GAF_SCHED_GRAM_FUSED


def test_filter_random_cases(ws):
    """Seeded random shapes, thresholds, orders and schedules against the oracle."""
    rng = np.random.RandomState(2024)
    for case in range(48):
        K = int(rng.choice([1, 2, 3, 4, 5, 8, 9, 13, 16, 31, 32, 33, 40]))
        D = int(rng.choice([0, 1, 7, 63, 1000, 4099, 65_537, 300_001, 1_048_576 + 3]))
        if K > 16:
            D = min(D, 65_537)
        dtype = "bf16" if rng.rand() < 0.5 else "f32"
        tau = float(rng.choice([0.3, 0.8, 0.97, 1.0, 1.1, 1.6]))
        order = [int(x) for x in rng.permutation(K)] if rng.rand() < 0.5 else None
        schedule = int(rng.choice([gaf.GAF_SCHED_AUTO, gaf.GAF_SCHED_STEPWISE, gaf.GAF_SCHED_GRAM,
                                   gaf.GAF_SCHED_GRAM_FUSED]))
        if schedule == gaf.GAF_SCHED_GRAM_FUSED and K > 8:
            schedule = gaf.GAF_SCHED_GRAM
        w = _mix(K, D, dtype, seed=5000 + case, sigma=float(rng.choice([1e-3, 1.0, 30.0])))
        check_filter(w.grads, tau, ws, order=order, schedule=schedule, expect_status=None)


def test_random_cases_all_entry_points(ws):
    """A seeded sweep over every Gram path and schedule: 1..64 gradients, lengths from 0 to a few
    waves with ragged ends, both types, all schedules, filter / pairwise matrix / any-seed variant.
    Thresholds above 1 on a handful of elements make accepted gradients cancel almost exactly; there the
    tolerances need not hold, and the library must say so itself (GAF_STATUS_ILL_CONDITIONED)."""
    rng = np.random.RandomState(77)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for case in range(240):
        K = int(rng.choice([1, 2, 3, 4, 5, 6, 7, 8, 9, 12, 16, 17, 24, 31, 32, 33, 40, 41, 48, 57, 64]))
        if rng.rand() < 0.3:
            D = int(rng.randint(100_000, 1_500_000))
        else:
            D = int(rng.choice([0, 1, 2, 3, 5, 8, 17, 100, 511, 512, 513, 4096, 65_537]))
        if rng.rand() < 0.15:
            D = int(sms * 512 * rng.randint(1, 4) * (4 if rng.rand() < 0.5 else 8) + rng.randint(-9, 9))
        if K > 16:
            D = min(D, 300_000)
        dtype = "bf16" if rng.rand() < 0.5 else "f32"
        tau = float(rng.choice([0.3, 0.8, 0.97, 1.0, 1.05, 1.6, 2.0, -1.0]))
        order = [int(x) for x in rng.permutation(K)] if rng.rand() < 0.5 else None
        schedule = int(rng.choice([0, 1, 2] + ([3] if 2 <= K <= 8 else [])))
        rho = rng.uniform(-0.6, 0.95, size=K)
        w = workloads.mixture(K, D, dtype, list(rho), int(rng.randint(1 << 30)), device="cuda",
                              sigma=float(rng.choice([1e-3, 1.0, 30.0])))
        kind = rng.rand()
        if kind < 0.6:
            check_filter(w.grads, tau, ws, order=order, schedule=schedule, expect_status=None,
                         allow_ill_conditioned=True)
        elif kind < 0.85:
            check_pairwise(w.grads, ws)
        else:
            check_any_seed(w.grads, tau, ws, allow_ill_conditioned=True)


@pytest.mark.parametrize("dtype", DTYPES)
def test_gram_loop_ends_inside_a_warp_at_the_flush_period(ws, dtype):
    """Lengths for which some lanes of a warp run exactly 16 rounds of the Gram loop (one
    binary64 flush, a warp-wide shuffle) and their neighbours 15: the flush must still be
    reached by whole warps."""
    threads = 2 * torch.cuda.get_device_properties(0).multi_processor_count * 512
    per_vec = 4 if dtype == "f32" else 8
    for extra in (1000, 40):
        D = (threads * 15 + extra) * per_vec + 3
        w = _mix(3, D, dtype, seed=77, rho=[0.7, 0.5, -0.4])
        check_filter(w.grads, 0.9, ws, schedule=gaf.GAF_SCHED_GRAM)
        check_filter(w.grads, 0.9, ws, schedule=gaf.GAF_SCHED_GRAM_FUSED)
        check_pairwise(w.grads, ws)


def test_filter_partly_cancelling_gradients(ws):
    """Accepted gradients that nearly cancel: the norm of the running sum is a small
    difference of large Gram entries in the Gram-first schedule."""
    D = 200_003
    g = torch.randn(D, device="cuda") * 1e-3
    gs = [g, -0.99 * g + 1e-6 * torch.randn(D, device="cuda"), torch.randn(D, device="cuda") * 1e-3,
          0.5 * g + 1e-4 * torch.randn(D, device="cuda")]
    for schedule in SCHEDULES:
        # tau = 2 accepts -0.99 g after g: the sum shrinks to 1 % of its terms and the library says so
        check_filter(gs, 2.0, ws, schedule=schedule, expect_status=gaf.GAF_STATUS_ILL_CONDITIONED)
        check_filter(gs, 1.2, ws, schedule=schedule)


def test_ill_conditioned_bit(ws):
    """GAF_STATUS_ILL_CONDITIONED is raised exactly when an accept leaves a running sum with
    c * sum |g_i|^2 > 167 |g|^2, by every schedule and variant, and never with tau <= 1."""
    D = 50_000
    g = torch.randn(D, device="cuda")
    h = torch.randn(D, device="cuda")
    ILL = gaf.GAF_STATUS_ILL_CONDITIONED
    # g then -0.9 g: kappa = 2 * 1.81 / 0.01 = 362 (raised); g then -0.8 g: 2 * 1.64 / 0.04 = 82 (not raised)
    for factor, want in ((-0.9, ILL), (-0.8, 0)):
        gs = [g, factor * g, h]
        for schedule in SCHEDULES:
            gaf.gaf_filter_accumulate(gs, 2.0, ws, schedule=schedule)
            assert gaf.gaf_read_status(ws) == want, (factor, schedule)
            gaf.gaf_filter_accumulate(gs, 1.0, ws, schedule=schedule)        # the opposing gradient is rejected
            assert gaf.gaf_read_status(ws) == 0
        gaf.gaf_filter_accumulate_any_seed(gs, 2.0, ws)
        assert gaf.gaf_read_status(ws) == want
        gaf.gaf_filter_accumulate_bucketed(gs, 2.0, [0, 20_000, D], ws)
        assert gaf.gaf_read_status(ws) == want
        acc = torch.empty(D, device="cuda")
        gaf.gaf_stream_begin(gs[0], acc, ws)
        for t in (1, 2):
            gaf.gaf_stream_push(gs[t], t, 2.0, acc, ws)
        gaf.gaf_stream_end(3, acc, ws)
        assert gaf.gaf_read_status(ws) == want
    # bfloat16 with 8 and 16 gradients: the tensor-core and the tiled Gram paths walk in their own launch
    for K in (8, 16):
        gs = [g.bfloat16(), (-0.9 * g).bfloat16()] + [torch.randn(D, device="cuda").bfloat16() for _ in range(K - 2)]
        gaf.gaf_filter_accumulate(gs, 2.0, ws, schedule=gaf.GAF_SCHED_GRAM)
        assert gaf.gaf_read_status(ws) & ILL
        gaf.gaf_filter_accumulate(gs, 1.0, ws, schedule=gaf.GAF_SCHED_GRAM)
        assert gaf.gaf_read_status(ws) == 0
        gaf.gaf_filter_accumulate_any_seed(gs, 2.0, ws)
        assert gaf.gaf_read_status(ws) & ILL


def test_bounded_waits_run_out_and_the_workspace_recovers(ws):
    """The two kernels that wait on another part of their own launch give up after a bounded number
    of attempts: with the test hook the awaited signal is withheld and the limit is a thousand polls,
    so every wait runs out.  The call must end by itself with GAF_STATUS_TIMEOUT, and the next
    ordinary call on the same workspace must be correct."""
    cases = [
        # one-launch Gram-first schedule: the waiting CTAs are never shown the full arrival counter
        (_mix(4, 600_011, "f32", seed=11, rho=[0.8, 0.6, -0.2, 0.7]), gaf.GAF_SCHED_GRAM_FUSED),
        (_mix(8, 300_007, "bf16", seed=12), gaf.GAF_SCHED_GRAM_FUSED),
        # tcgen05 Gram pipeline (17..64 bfloat16 gradients): the first tile's barrier never completes --
        # with the 16-byte-copy loaders (gradients anywhere) ...
        (_scattered(_mix(17, 300_007, "bf16", seed=13).grads), gaf.GAF_SCHED_GRAM, 1),
        (_scattered(_mix(40, 100_003, "bf16", seed=14).grads), gaf.GAF_SCHED_GRAM, 1),
        # ... and with the tensor-copy loader (gradients that are rows of one matrix), ragged and whole last chunk
        (_mix(17, 300_007, "bf16", seed=13, stacked=True), gaf.GAF_SCHED_GRAM, 2),
        (_mix(40, 64 * 1500, "bf16", seed=14, stacked=True), gaf.GAF_SCHED_GRAM, 2),
    ]
    cases = [(c[0] if isinstance(c[0], list) else c[0].grads, c[1], c[2] if len(c) > 2 else 0) for c in cases]
    for grads, schedule, loader in cases:
        try:
            gaf.gaf_test_set_wait_fault(1000, True)
            gaf.gaf_filter_accumulate(grads, 0.97, ws, schedule=schedule)
            status = gaf.gaf_read_status(ws)
        finally:
            gaf.gaf_test_set_wait_fault(0, False)
        assert status & gaf.GAF_STATUS_TIMEOUT, (schedule, status)
        assert gaf.gaf_last_gram_loader() == loader
        check_filter(grads, 0.97, ws, schedule=schedule)
    # a short limit alone, with the signal given, must not time out
    try:
        gaf.gaf_test_set_wait_fault(1 << 20, False)
        check_filter(cases[0][0], 0.97, ws, schedule=gaf.GAF_SCHED_GRAM_FUSED)
        check_filter(cases[-1][0], 0.97, ws, schedule=gaf.GAF_SCHED_GRAM)
    finally:
        gaf.gaf_test_set_wait_fault(0, False)


# ------------------------------------------------------------ streaming form --

@pytest.mark.parametrize("dtype", DTYPES)
def test_streaming_form_matches_oracle_and_batch_call(ws, dtype):
    from oracle import gaf_oracle as orc
    for K, D, tau in ((1, 1001, 0.97), (2, 8, 0.97), (4, 300_007, 0.6), (7, 1_000_003, 0.97)):
        w = _mix(K, D, dtype, seed=700 + K)
        acc = torch.empty(D, dtype=torch.float32, device="cuda")
        gaf.gaf_stream_begin(w.grads[0], acc, ws)
        for t in range(1, K):
            gaf.gaf_stream_push(w.grads[t], t, tau, acc, ws)
        mask, dist, count = gaf.gaf_stream_end(K, acc, ws)
        assert gaf.gaf_read_status(ws) == 0
        want = orc.filter_accumulate([workloads.as_numpy_bits(g) for g in w.grads], tau)
        assert mask.cpu().numpy().tolist() == want.mask.tolist() and int(count.item()) == want.count
        assert float(np.max(np.abs(dist.cpu().numpy() - want.dist))) < 1e-5
        got = acc.cpu().numpy().astype(np.float64)
        assert float(np.linalg.norm(got - want.out) / np.linalg.norm(want.out)) < (1e-6 if dtype == "f32" else 1e-3)
        batch = gaf.gaf_filter_accumulate(w.grads, tau, ws, schedule=gaf.GAF_SCHED_STEPWISE)
        assert torch.equal(batch[0], acc) and torch.equal(batch[1], mask) and torch.equal(batch[2], dist)


# ---------------------------------------- order-indifferent variant (Section 3.1) --

@pytest.mark.parametrize("dtype", DTYPES)
def test_any_seed_variant(ws, dtype):
    # the paper's degenerate case: a first gradient orthogonal to all the others
    D = 70_001
    base = torch.randn(D, device="cuda") * 1e-3
    odd = torch.zeros(D, device="cuda"); odd[::2] = 1e-3
    odd = odd - (odd @ base) / (base @ base) * base                 # orthogonal to base
    gs = [odd] + [base + 0.3 * torch.randn(D, device="cuda") * 1e-3 for _ in range(3)]
    if dtype == "bf16":
        gs = [g.to(torch.bfloat16) for g in gs]
    macro, mask, dist, count, *_ = gaf.gaf_filter_accumulate(gs, 0.5, ws)
    assert int(count.item()) == 1                                    # plain Algorithm 1 wastes the macrobatch
    r = check_any_seed(gs, 0.5, ws)
    assert r["seed"] == 1 and r["count"] == 3
    # mixtures over every Gram path: K <= 8, tensor cores (bf16, K <= 32), tiled (the rest)
    for K, Dk in ((1, 1000), (2, 5003), (5, 300_007), (8, 1_000_001), (12, 400_003), (32, 200_001), (40, 50_001)):
        w = _mix(K, Dk, dtype, seed=900 + K)
        r = check_any_seed(w.grads, 0.97, ws)
        assert r["count"] == max(r["counts"])


# ------------------------------------------------------------ bucketed variant --

@pytest.mark.parametrize("dtype", DTYPES)
def test_bucketed_variant(ws, dtype):
    # one bucket = the plain filter
    w = _mix(4, 100_003, dtype, seed=31, rho=[0.8, 0.6, -0.2, 0.7])
    check_bucketed(w.grads, 0.8, [0, w.D], ws)
    plain = gaf.gaf_filter_accumulate(w.grads, 0.8, ws)
    buck = gaf.gaf_filter_accumulate_bucketed(w.grads, 0.8, [0, w.D], ws)
    assert torch.equal(plain[0], buck[0]) and torch.equal(plain[1], buck[1][0])
    # many buckets of very different sizes, empty ones, a ragged end, a non-identity order
    rng = np.random.RandomState(7)
    for K, D in ((1, 5000), (2, 64), (3, 300_011), (5, 2_000_005), (8, 777_777)):
        cuts = sorted(set(int(x) // 8 * 8 for x in rng.randint(0, D, size=24)) | {0})
        offsets = cuts + [cuts[-1], D] if cuts[-1] < D else cuts + [D]
        offsets = [0] + [o for o in offsets[1:]]
        if offsets[1] != 0:
            offsets.insert(1, 0)                                    # an empty first bucket
        w = _mix(K, D, dtype, seed=400 + K)
        for g in w.grads[1:2]:
            g[: D // 3] = -w.grads[0][: D // 3]                       # buckets must disagree with each other
        order = [int(x) for x in rng.permutation(K)]
        patterns = check_bucketed(w.grads, 0.9, offsets, ws, order=order)
        if K >= 3:
            assert len(patterns) >= 2


def test_bucketed_resnet18_layout(ws):
    """Configuration 2 cut at its 62 parameter tensors."""
    w = workloads.config(2, device="cuda")
    sizes = workloads.resnet18_tensor_sizes(100)
    offsets = [0] + list(np.cumsum(sizes))
    assert offsets[-1] == w.D and len(offsets) == 63
    check_bucketed(w.grads, 0.97, [int(o) for o in offsets], ws)


def test_bucketed_argument_errors(ws):
    w = _mix(3, 1000, "f32", seed=1)
    for bad in ([0, 500], [1, 1000], [0, 700, 600, 1000]):
        with pytest.raises(gaf.GafError) as e:
            gaf.gaf_filter_accumulate_bucketed(w.grads, 0.9, bad, ws)
        assert e.value.code == 1
    with pytest.raises(gaf.GafError) as e:
        gaf.gaf_filter_accumulate_bucketed(w.grads, 0.9, [0, 100, 1000], ws)      # 100 is not a multiple of 8
    assert e.value.code == 2
    with pytest.raises(gaf.GafError) as e:
        gaf.gaf_filter_accumulate_bucketed(_mix(9, 1000, "f32", seed=2).grads, 0.9, [0, 1000], ws)
    assert e.value.code == 7


# ------------------------------------------------- the named configurations --

@pytest.mark.parametrize("schedule", SCHEDULES, ids=SCHED_IDS)
def test_config1(ws, schedule):
    w = workloads.config(1, device="cuda")
    r = check_filter(w.grads, w.taus[0], ws, schedule=schedule)
    assert r["mask"] == [1, 1, 0, 0] and r["count"] == 2       # closed form of the mixture model


@pytest.mark.parametrize("schedule", SCHEDULES, ids=SCHED_IDS)
def test_config2_resnet18_layout(ws, schedule):
    w = workloads.config(2, device="cuda")
    np_grads = [workloads.as_numpy_bits(g) for g in w.grads]
    for tau in w.taus:
        check_filter(w.grads, tau, ws, schedule=schedule, np_grads=np_grads)


@pytest.mark.slow
def test_config4_gpt2_small_sized(ws):
    w = workloads.config(4, device="cuda")
    np_grads = [workloads.as_numpy_bits(g) for g in w.grads]
    for schedule in SCHEDULES:
        r = check_filter(w.grads, w.taus[0], ws, schedule=schedule, np_grads=np_grads)
        assert 1 <= r["count"] <= 8


@pytest.mark.slow
def test_config5_billion_bf16(ws):
    """Full size: 8 x 1e9 bf16 (16 GB of gradients), 64-bit offsets, both schedules."""
    free, _ = torch.cuda.mem_get_info()
    assert free > 24 << 30, "configuration 5 needs about 21 GB of device memory"
    w = workloads.config(5, device="cuda")
    np_grads = [workloads.as_numpy_bits(g) for g in w.grads]
    for schedule in SCHEDULES:
        check_filter(w.grads, w.taus[0], ws, schedule=schedule, np_grads=np_grads)


# ---------------------------------------------------------- pairwise matrix --

@pytest.mark.parametrize("dtype", DTYPES)
def test_pairwise_small(ws, dtype):
    for K in (1, 2, 3, 8, 9, 17, 32, 33):
        for D in (0, 1, 5, 64, 1001, 40_003):
            if K > 9 and D > 1001:
                continue
            w = _mix(K, D, dtype, seed=K * 77 + D)
            check_pairwise(w.grads, ws)
    w = _mix(12, 3_000_001, dtype, seed=1)
    check_pairwise(w.grads, ws)


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("K", [10, 16, 24, 32, 40, 48, 64])
def test_pairwise_general_kernel_shapes(ws, dtype, K):
    """More than 8 gradients: the general CUDA-core Gram kernel (binary32) in each of its shapes (warps
    sharing a tile pair, one warp per pair, tile pairs split over groups of CTAs) and the tensor-core
    kernels (bfloat16: warp-level MMAs up to 16 gradients, the tcgen05 tile in its 32- and 64-row forms):
    several panels or tiles per CTA, a ragged end."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    for D in (sms * 512 * 3 + 1234 + 3, 100_001):
        w = _mix(K, D, dtype, seed=300 + K)
        check_pairwise(w.grads, ws)


def test_auto_schedule_choice(ws):
    """What GAF_SCHED_AUTO resolves to (gaf_last_schedule), shape by shape."""
    cases = [(1, 1000, "f32", gaf.GAF_SCHED_STEPWISE), (4, 100_000, "f32", gaf.GAF_SCHED_GRAM_FUSED),
             (8, 100_000, "bf16", gaf.GAF_SCHED_GRAM_FUSED), (6, 50_000, "bf16", gaf.GAF_SCHED_GRAM_FUSED),
             (9, 50_000, "f32", gaf.GAF_SCHED_GRAM), (32, 20_000, "f32", gaf.GAF_SCHED_GRAM),
             (33, 20_000, "f32", gaf.GAF_SCHED_STEPWISE), (16, 50_000, "bf16", gaf.GAF_SCHED_GRAM),
             (33, 20_000, "bf16", gaf.GAF_SCHED_GRAM), (64, 20_000, "bf16", gaf.GAF_SCHED_GRAM)]
    for K, D, dtype, want in cases:
        w = _mix(K, D, dtype, seed=11)
        gaf.gaf_filter_accumulate(w.grads, 0.97, ws)
        assert gaf.gaf_last_schedule() == want, (K, D, dtype, gaf.gaf_last_schedule())
    # 8 binary32 gradients of more than 512 MB in all: Gram-first in two launches
    big = [torch.zeros(17_000_000, device="cuda") for _ in range(8)]
    for i, g in enumerate(big):
        g[i::8] = 1.0
    gaf.gaf_filter_accumulate(big, 0.97, ws)
    assert gaf.gaf_last_schedule() == gaf.GAF_SCHED_GRAM
    # 8 bfloat16 gradients of more than 1 GB in all: two launches as well (warp-level MMA Gram kernel, masked mean)
    big = [torch.zeros(70_000_000, device="cuda", dtype=torch.bfloat16) for _ in range(8)]
    for i, g in enumerate(big):
        g[i::8] = 1.0
    gaf.gaf_filter_accumulate(big, 0.97, ws)
    assert gaf.gaf_last_schedule() == gaf.GAF_SCHED_GRAM and gaf.gaf_last_launch_count() == 2


@pytest.mark.parametrize("dtype", DTYPES)
def test_two_gradients_mean_written_in_the_first_pass(ws, dtype):
    """Two gradients (the setting of the paper's Section 4): the one-launch kernel writes the mean of both while
    it forms the sums and rewrites the output with the first gradient alone when the second is rejected.  Both
    outcomes, both orders, ragged lengths, the order-indifferent variant, and bit-identity with the other schedules."""
    for D in (1, 7, 1001, 300_007, 5_000_003):
        for rho, tau in (([0.8, 0.7], 0.97), ([0.8, -0.5], 0.97), ([0.3, 0.2], 2.0), ([0.9, 0.9], 0.0)):
            w = _mix(2, D, dtype, seed=D % 89 + int(10 * tau), rho=rho)
            for order in (None, [1, 0]):
                r = check_filter(w.grads, tau, ws, order=order)
                assert gaf.gaf_last_schedule() == gaf.GAF_SCHED_GRAM_FUSED and gaf.gaf_last_launch_count() == 1
                got = gaf.gaf_filter_accumulate(w.grads, tau, ws, order=order)
                for schedule in (gaf.GAF_SCHED_GRAM, gaf.GAF_SCHED_STEPWISE):
                    other = gaf.gaf_filter_accumulate(w.grads, tau, ws, order=order, schedule=schedule)
                    if torch.equal(other[1], got[1]):                      # (masks may differ on a tie only)
                        assert torch.equal(other[0], got[0]), (D, rho, tau, order, schedule)
            check_any_seed(w.grads, tau, ws)
    # rejected and accepted counts really both occurred above; and at a length beyond the old one-launch limit
    big = _mix(2, 70_000_003, "f32", seed=5, rho=[0.6, 0.5])
    check_filter(big.grads, 0.97, ws)
    assert gaf.gaf_last_schedule() == gaf.GAF_SCHED_GRAM_FUSED
    check_filter(big.grads, 0.0, ws)


def test_wide_mma_gram_kernel_shapes_and_long_runs(ws):
    """9..16 bfloat16 gradients (and the first counts of the tcgen05 tile behind them): absent rows feed zeros;
    lengths below one tile, ragged ends, and a length from which the CTAs walk in runs of several trips."""
    for K in (9, 12, 15, 16, 17, 24, 25):
        for D in (37, 64 * 16 * 5 + 11, 300_001):
            check_pairwise(_mix(K, D, "bf16", seed=700 + K).grads, ws)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    D = 32 * 8 * 16 * 64 * 2 * sms + 64 * 16 * 3 + 5      # just over the threshold for long runs
    check_pairwise(_mix(12, D, "bf16", seed=777).grads, ws)


def test_mma_gram_kernel_long_runs(ws):
    """7 and 8 bfloat16 gradients take the warp-level tensor-core Gram kernel; from about 19 M elements on its
    CTAs walk the vectors in runs of several trips.  Both mappings, with ragged ends, against the oracle."""
    for K, D in ((8, 20_000_000 + 37), (7, 19_500_003), (8, 2_500_000 + 63), (7, 64 * 16 * 296 * 2 + 5)):
        w = _mix(K, D, "bf16", seed=600 + K)
        check_filter(w.grads, 0.97, ws, schedule=gaf.GAF_SCHED_GRAM)
        check_pairwise(w.grads, ws)


def test_gram_sums_of_few_fp32_gradients_are_exact_to_binary64_rounding(ws):
    """Up to 4 binary32 gradients the Gram kernels accumulate in binary64, where every product is exact:
    the Gram matrix agrees with the oracle's to binary64 rounding, not merely to binary32 precision."""
    from oracle import gaf_oracle as orc
    for K in (2, 3, 4):
        w = _mix(K, 1_000_003, "f32", seed=40 + K)
        _, gram = gaf.gaf_pairwise_cosdist(w.grads, ws)
        o_gram, _ = orc.pairwise_cosdist([workloads.as_numpy_bits(g) for g in w.grads])
        nrm = np.sqrt(np.diag(o_gram))
        assert float(np.max(np.abs(gram.cpu().numpy() - o_gram) / np.outer(nrm, nrm))) < 1e-12


def test_pairwise_zero_norm_row(ws):
    w = _mix(4, 5001, "f32", seed=2)
    w.grads[2].zero_()
    check_pairwise(w.grads, ws)
    dist, _ = gaf.gaf_pairwise_cosdist(w.grads, ws)
    assert bool((dist[2] == 1.0).all()) and bool((dist[:, 2] == 1.0).all())


@pytest.mark.parametrize("K", [17, 19, 25, 32, 33, 42, 52, 64])
def test_tensor_copy_loader_of_the_tcgen05_gram_kernel(ws, K):
    """bfloat16 gradients that are rows of one matrix are fetched by tensor copies (gradient-major tile rows, the
    epilogue picks the Gram entries out of all columns), any other placement by 16-byte copies (chunk-major rows):
    both against the oracle and against each other, for every kind of end of the vector -- shorter than a chunk
    (no tensor copies), one whole chunk, a ragged chunk in each position of its block, whole chunks that do not
    fill the last block or tile, several tiles."""
    sizes = (40, 64, 65, 64 + 63, 200, 64 * 7, 64 * 8 + 1, 3072 + 192, 3072 + 192 + 17, 70_001, 262_152, 1_000_003)
    for D in sizes:
        w = _mix(K, D, "bf16", seed=3 * K + D % 97, stacked=True)
        check_pairwise(w.grads, ws)
        assert gaf.gaf_last_gram_loader() == (2 if D >= 64 and K <= 42 else 1), D
        gram_rows = gaf.gaf_pairwise_cosdist(w.grads, ws)[1].clone()
        elsewhere = _scattered(w.grads)
        check_pairwise(elsewhere, ws)
        assert gaf.gaf_last_gram_loader() == 1
        gram_any = gaf.gaf_pairwise_cosdist(elsewhere, ws)[1]
        scale = gram_any.diagonal().sqrt()
        assert float(((gram_rows - gram_any).abs() / scale[:, None] / scale[None, :]).max()) < 2e-6
    # the filter on top of it, and a row distance that is not a multiple of 128 bytes (16-byte copies then)
    w = _mix(K, 300_007, "bf16", seed=5 * K, stacked=True)
    check_filter(w.grads, 0.97, ws, schedule=gaf.GAF_SCHED_GRAM)
    assert gaf.gaf_last_gram_loader() == (2 if K <= 42 else 1)
    tight = torch.stack([g[:300_000] for g in w.grads])                 # rows 600,000 bytes apart
    check_pairwise(list(tight.unbind(0)), ws)
    assert gaf.gaf_last_gram_loader() == 1


def test_config3_pairwise(ws):
    w = workloads.config(3, device="cuda")
    check_pairwise(w.grads, ws)
    stacked = workloads.config(3, device="cuda", stacked=True)
    check_pairwise(stacked.grads, ws)
    assert gaf.gaf_last_gram_loader() == 2
    dist, _ = gaf.gaf_pairwise_cosdist(w.grads, ws)
    rho = np.array(w.rho)
    want = 1.0 - np.sign(rho)[:, None] * np.sign(rho)[None, :] * np.sqrt(np.abs(np.outer(rho, rho)))
    np.fill_diagonal(want, 0.0)
    assert float(np.max(np.abs(dist.cpu().numpy() - want))) < 5e-3      # closed form of the mixture
