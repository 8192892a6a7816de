"""Pins for the CPU oracle: checks against what the paper and the mathematics fix.

Every function here asserts one fact that does not come from the oracle itself:
values the paper states, closed forms, invariants of Eq. 4, reductions to a
library routine (numpy / scipy), and brute-force enumeration from the
definition written with Python integers.  ``ALL_PINS`` is used twice: once
against the real oracle, and once against deliberately broken copies of it to
show that a plausible mistake makes at least one pin fail.
"""
from __future__ import annotations

import itertools
import math
import os

import numpy as np

from oracle import gaf_oracle as orc

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def f32(*v):
    return np.array(v, dtype=np.float32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bfloat16 bit patterns, integer arithmetic only."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


# ---------------------------------------------------------------- Eq. 4 ------

def pin_stated_values():
    """Introduction: identical -> 0, orthogonal -> 1, opposite -> 2."""
    want = {}
    with open(os.path.join(GOLDEN, "stated_values.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                want[k] = float(v)
    x = f32(3.0, -4.0, 12.0, 0.5)
    orth = f32(4.0, 3.0, 0.0, 0.0)
    for conv in (lambda a: a, to_bf16_bits):
        # sqrt(n)*sqrt(n) may differ from n in the last bit: allow two ulps
        assert abs(orc.cosdist(conv(x), conv(x))[0] - want["identical"]) < 5e-16
        assert orc.cosdist(conv(x), conv(orth))[0] == want["orthogonal"]
        assert abs(orc.cosdist(conv(x), conv(-x))[0] - want["opposite"]) < 5e-16
    # with an integer norm the stated values come out exactly
    y = f32(3.0, -4.0, 12.0)
    assert orc.cosdist(y, y)[0] == 0.0 and orc.cosdist(y, -y)[0] == 2.0


def pin_figure2_angles():
    """Figure 2: unit arrows at the printed angles; D_c = 1 - cos(angle difference)."""
    with open(os.path.join(GOLDEN, "fig2_angles.txt")) as fh:
        rows = [l.split() for l in fh if l.strip() and not l.startswith("#")]
    seen = []
    for _, cls, *angles in rows:
        angles = [float(a) for a in angles]
        for a, b in itertools.combinations(angles, 2):
            va = np.array([2 * math.cos(math.radians(a)), 2 * math.sin(math.radians(a))], dtype=np.float32)
            vb = np.array([2 * math.cos(math.radians(b)), 2 * math.sin(math.radians(b))], dtype=np.float32)
            d = orc.cosdist(va, vb)[0]
            closed = 1.0 - math.cos(math.radians(a - b))
            assert abs(d - closed) < 1e-6, (a, b, d, closed)
            assert (d < 1.0) if cls == "lt1" else (d >= 1.0)
            seen.append(round(closed, 4))
    assert sorted(seen) == sorted([0.1808, 0.7412, 0.2340, 1.7071, 1.5736, 1.1736])


def pin_invariants():
    """Symmetry, positive-scale invariance, D_c(-x, y) = 2 - D_c(x, y), range [0, 2]."""
    rng = np.random.RandomState(11)
    for n in (1, 2, 7, 64, 1001):
        x = rng.standard_normal(n).astype(np.float32)
        y = rng.standard_normal(n).astype(np.float32)
        d = orc.cosdist(x, y)[0]
        assert 0.0 <= d <= 2.0
        assert orc.cosdist(y, x)[0] == d
        # powers of two scale exactly in binary floating point
        assert abs(orc.cosdist(x * np.float32(4.0), y * np.float32(0.125))[0] - d) < 1e-15
        assert abs(orc.cosdist(-x, y)[0] - (2.0 - d)) < 1e-15
        assert abs(orc.cosdist(x * np.float32(3.7), y)[0] - d) < 1e-6
    # rounding in p / (sqrt sqrt) must not leave the stated range [0, 2]
    for _ in range(300):
        x = rng.standard_normal(rng.randint(1, 9)).astype(np.float32)
        assert orc.cosdist(x, x)[0] >= 0.0
        assert orc.cosdist(x, -x)[0] <= 2.0


def pin_matches_scipy_and_numpy():
    """Eq. 4 is scipy's cosine distance; the three sums are numpy dot products."""
    from scipy.spatial.distance import cosine
    rng = np.random.RandomState(5)
    for n in (3, 50, 4097):
        x = rng.standard_normal(n).astype(np.float32)
        y = (0.3 * x + rng.standard_normal(n)).astype(np.float32)
        d, (p, nx, ny) = orc.cosdist(x, y)
        x64, y64 = x.astype(np.float64), y.astype(np.float64)
        assert abs(d - cosine(x64, y64)) < 1e-12
        assert abs(p - x64 @ y64) <= 1e-12 * abs(x64 @ y64) + 1e-300
        assert abs(nx - x64 @ x64) <= 1e-12 * nx
        assert abs(ny - y64 @ y64) <= 1e-12 * ny
    # operands are not interchangeable in the stats: a transposed use shows here
    x = f32(1, 2, 3)
    y = f32(0, 0, 2)
    _, (p, nx, ny) = orc.cosdist(x, y)
    assert (p, nx, ny) == (6.0, 14.0, 4.0)


def pin_bf16_widening():
    """bfloat16 widens exactly: every finite bit pattern agrees with the integer rule
    value = (-1)^s * 2^(e-127) * (1 + m/128) (subnormals: 2^-126 * m/128)."""
    bits = np.arange(0, 1 << 16, dtype=np.uint32)
    exp = (bits >> 7) & 0xFF
    finite = exp != 0xFF
    bits = bits[finite].astype(np.uint16)
    s = np.where(bits >> 15, -1.0, 1.0)
    e = ((bits >> 7) & 0xFF).astype(np.int64)
    m = (bits & 0x7F).astype(np.float64)
    val = np.where(e == 0, s * np.ldexp(m / 128.0, -126), s * np.ldexp(1.0 + m / 128.0, e - 127))
    # |x|^2 of a one-element vector against a unit partner exposes the widened value
    ones = to_bf16_bits(np.ones(1, dtype=np.float32))
    for idx in list(range(0, bits.size, 257)) + [1, 127, 128, bits.size - 1]:
        b = bits[idx:idx + 1]
        _, (p, nx, _) = orc.cosdist(b, ones)
        assert p == val[idx] and nx == val[idx] * val[idx], (hex(int(b[0])), p, val[idx])


# ------------------------------------------------------------ Algorithm 1 ----

def _rand_grads(rng, K, D, dtype="f32", shared=0.5):
    s = rng.standard_normal(D)
    gs = [(shared * s + rng.standard_normal(D)).astype(np.float32) for _ in range(K)]
    return [to_bf16_bits(g) for g in gs] if dtype == "bf16" else gs


def _widen(g):
    return orc.bf16_bits_to_f64(g) if g.dtype == np.uint16 else g.astype(np.float64)


def pin_tau2_is_plain_mean():
    """A threshold of 2 admits everything: the result is the plain mean of Eq. 2
    (numpy's mean here), all mask bits set, c = K -- including an exactly
    opposite vector, whose distance must not exceed 2 through rounding."""
    rng = np.random.RandomState(3)
    for dtype in ("f32", "bf16"):
        for K, D in ((2, 5), (4, 33), (7, 1000)):
            gs = _rand_grads(rng, K, D, dtype)
            gs[-1] = (-np.asarray(gs[0], dtype=np.float32)) if dtype == "f32" else (gs[0] ^ np.uint16(0x8000))
            r = orc.filter_accumulate(gs, 2.0)
            mean = np.mean(np.stack([_widen(g) for g in gs]), axis=0)
            assert r.count == K and r.mask.tolist() == [1] * K
            assert np.allclose(r.out, mean, rtol=1e-13, atol=1e-300)
            assert np.allclose(orc.plain_average(gs), mean, rtol=1e-13, atol=1e-300)


def pin_reject_all_keeps_seed():
    """Nothing meets the threshold: c = 1, one-hot mask, g_GAF is the seed itself."""
    rng = np.random.RandomState(4)
    for dtype in ("f32", "bf16"):
        gs = _rand_grads(rng, 5, 77, dtype)
        for order in (None, [3, 0, 4, 1, 2]):
            r = orc.filter_accumulate(gs, -0.5, order=order)
            s = 0 if order is None else order[0]
            assert r.count == 1
            assert r.mask.tolist() == [1 if i == s else 0 for i in range(5)]
            assert np.array_equal(r.out, _widen(gs[s]))
            assert r.dist[s] == 0.0 and all(r.dist[i] > 0 for i in range(5) if i != s)


def pin_k2_operating_point():
    """k = 2 (the paper's experiments): (g0+g1)/2 iff D_c(g0,g1) <= tau, else g0."""
    from scipy.spatial.distance import cosine
    rng = np.random.RandomState(6)
    for trial in range(20):
        g0 = rng.standard_normal(40).astype(np.float32)
        g1 = (rng.uniform(-1, 1) * g0 + rng.standard_normal(40)).astype(np.float32)
        d = cosine(g0.astype(np.float64), g1.astype(np.float64))
        for tau in (0.5, 0.97, 1.0, 1.3):
            r = orc.filter_accumulate([g0, g1], tau)
            assert abs(r.dist[1] - d) < 1e-12
            if d <= tau:
                assert r.count == 2 and np.allclose(r.out, (g0.astype(np.float64) + g1) / 2, rtol=1e-15)
            else:
                assert r.count == 1 and np.array_equal(r.out, g0.astype(np.float64))


def pin_threshold_is_inclusive():
    """Acceptance is D_c <= tau: an exactly orthogonal integer vector has D_c = 1
    exactly and is accepted at tau = 1, rejected just below."""
    g0 = f32(1, 2, 0, 0)
    g1 = f32(-2, 1, 5, 0)
    r = orc.filter_accumulate([g0, g1], 1.0)
    assert r.dist[1] == 1.0 and r.mask.tolist() == [1, 1] and r.count == 2
    r = orc.filter_accumulate([g0, g1], math.nextafter(1.0, 0.0))
    assert r.mask.tolist() == [1, 0] and r.count == 1


def pin_order_dependence():
    """Section 3.1's degenerate case: a seed orthogonal to all others rejects
    everything; with an agreeing vector as the seed the others are accepted and
    only the orthogonal one is dropped."""
    e = f32(0, 0, 0, 1)
    a = f32(1, 0.1, 0, 0)
    b = f32(1, -0.1, 0.1, 0)
    c = f32(0.9, 0, -0.1, 0)
    r = orc.filter_accumulate([e, a, b, c], 0.5)
    assert r.mask.tolist() == [1, 0, 0, 0] and r.count == 1
    r = orc.filter_accumulate([e, a, b, c], 0.5, order=[1, 2, 3, 0])
    assert r.mask.tolist() == [0, 1, 1, 1] and r.count == 3
    assert np.allclose(r.out, (a.astype(np.float64) + b + c) / 3, rtol=1e-15)
    # mask, dist are indexed by the original position, not by step
    r2 = orc.filter_accumulate([a, e, b, c], 0.5)
    assert r2.mask.tolist() == [1, 0, 1, 1] and r2.dist[1] == 1.0


def pin_running_sum_not_pairwise():
    """The test is against the running SUM of accepted gradients, not against the
    seed alone and not against the last gradient."""
    g0 = f32(1, 0)
    g1 = f32(1, 1)          # 45 degrees from g0: accepted at tau = 0.5
    g2 = f32(0.2, 1)        # 78.7 degrees from g0 (D_c = 0.804: would be rejected),
                            # 52.1 degrees from g0+g1=(2,1) (D_c = 0.386: accepted)
    r = orc.filter_accumulate([g0, g1, g2], 0.5)
    assert r.mask.tolist() == [1, 1, 1]
    x = float(np.float32(0.2))
    want = 1.0 - (2 * x + 1) / (math.sqrt(5.0) * math.sqrt(x * x + 1))
    assert abs(r.dist[2] - want) < 1e-12
    assert np.allclose(r.stats[2], [2 * x + 1, 5.0, x * x + 1], rtol=1e-15)
    # a rejected gradient leaves the sum untouched and is never retried
    g1r = f32(-1, 0.1)
    r = orc.filter_accumulate([g0, g1r, g2], 0.5)
    assert r.mask.tolist() == [1, 0, 0] and np.array_equal(r.out, g0.astype(np.float64))


def _consistent_masks(vecs, tau, order):
    """All accept patterns consistent with Algorithm 1's rule, from the definition,
    with Python integers for the dot products."""
    K = len(vecs)
    found = []
    for bits in itertools.product((0, 1), repeat=K - 1):
        m = {order[0]: 1}
        ok = True
        for t in range(1, K):
            i = order[t]
            acc = [sum(vecs[order[u]][d] for u in range(t) if m[order[u]]) for d in range(len(vecs[0]))]
            p = sum(a * b for a, b in zip(acc, vecs[i]))
            na = sum(a * a for a in acc)
            ng = sum(b * b for b in vecs[i])
            dist = 1.0 - p / (math.sqrt(na) * math.sqrt(ng))
            want = 1 if dist <= tau else 0
            if bits[t - 1] != want:
                ok = False
                break
            m[i] = bits[t - 1]
        if ok:
            found.append([m[i] for i in range(K)])
    return found


def pin_brute_force_masks():
    """Tiny K and D, entries in {-1, 0, 1}: exactly one accept pattern satisfies the
    rule of Algorithm 1 evaluated from the definition; it is the oracle's, and the
    output is the mean of the accepted vectors."""
    rng = np.random.RandomState(8)
    cases = []
    for K, D in ((2, 2), (3, 2)):
        for flat in itertools.product((-1, 0, 1), repeat=K * D):
            cases.append([list(flat[i * D:(i + 1) * D]) for i in range(K)])
    for K, D in ((4, 2), (4, 3), (5, 3)):
        for _ in range(150):
            cases.append(rng.randint(-1, 2, size=(K, D)).tolist())
    n = 0
    for vecs in cases:
        if any(all(v == 0 for v in vec) for vec in vecs):
            continue            # zero-norm vectors fall under a convention, not under the paper
        K = len(vecs)
        for tau in (0.25, 0.5, 0.97, 1.0, 1.5):
            order = list(range(K)) if n % 3 else list(rng.permutation(K))
            masks = _consistent_masks(vecs, tau, order)
            assert len(masks) == 1
            r = orc.filter_accumulate([np.array(v, dtype=np.float32) for v in vecs], tau,
                                      order=[int(o) for o in order])
            assert r.mask.tolist() == masks[0], (vecs, tau, order)
            acc = np.sum([np.array(v, dtype=np.float64) for v, m in zip(vecs, masks[0]) if m], axis=0)
            assert r.count == sum(masks[0])
            assert np.allclose(r.out, acc / sum(masks[0]), rtol=1e-15, atol=0)
            n += 1
    assert n > 2000


def pin_bilinearity_ties_filter_to_pairwise():
    """<sum_A g_j, g_i> = sum_A G_ji and |sum_A g_j|^2 = sum_{j,l in A} G_jl: the
    filter's sums recomputed from the pairwise Gram matrix (numpy matmul as a
    second source for the Gram matrix itself)."""
    rng = np.random.RandomState(9)
    for dtype in ("f32", "bf16"):
        K, D = 6, 513
        sh = rng.standard_normal(D)
        gs = [(a * sh + rng.standard_normal(D)).astype(np.float32)
              for a in (0.8, -0.8, 0.8, 0.0, 0.8, 0.8)]
        if dtype == "bf16":
            gs = [to_bf16_bits(g) for g in gs]
        gram, dist = orc.pairwise_cosdist(gs)
        X = np.stack([_widen(g) for g in gs])
        G = X @ X.T
        assert np.allclose(gram, G, rtol=1e-12, atol=1e-12)
        nrm = np.sqrt(np.diag(G))
        want = 1.0 - G / np.outer(nrm, nrm)
        np.fill_diagonal(want, 0.0)
        assert np.allclose(dist, want, atol=1e-12)
        assert np.array_equal(dist, dist.T) and np.all(np.diag(dist) == 0.0)
        order = [2, 0, 5, 1, 4, 3]
        r = orc.filter_accumulate(gs, 0.9, order=order)
        assert 1 < r.count < K        # the case exercises both branches
        A = [order[0]]
        for t in range(1, K):
            i = order[t]
            p = sum(gram[j, i] for j in A)
            na = sum(gram[j, l] for j in A for l in A)
            assert np.allclose(r.stats[i], [p, na, gram[i, i]], rtol=1e-11)
            d = 1.0 - p / math.sqrt(na * gram[i, i])
            assert abs(r.dist[i] - d) < 1e-12
            if r.mask[i]:
                A.append(i)
        assert np.allclose(r.out, X[A].sum(axis=0) / len(A), rtol=1e-12, atol=1e-15)


def pin_forced_decisions():
    """Forcing a decision replaces the test at that step only."""
    rng = np.random.RandomState(10)
    gs = _rand_grads(rng, 4, 50, "f32", shared=0.0)
    free = orc.filter_accumulate(gs, 0.3)
    assert free.mask.tolist() == [1, 0, 0, 0]
    r = orc.filter_accumulate(gs, 0.3, forced=[-1, 1, -1, 1])
    assert r.mask.tolist() == [1, 1, 0, 1] and r.count == 3
    X = np.stack([g.astype(np.float64) for g in gs])
    assert np.allclose(r.out, (X[0] + X[1] + X[3]) / 3, rtol=1e-14)
    assert r.dist[1] == free.dist[1]          # the distance is still reported
    r = orc.filter_accumulate(gs, 2.0, forced=[-1, 0, 0, 0])
    assert r.mask.tolist() == [1, 0, 0, 0]


def pin_closed_form_mixture():
    """Shared-plus-private mixture (configuration 1 of the workloads): with
    alpha_i = sign(rho_i) sqrt|rho_i|, beta_i^2 = 1 - |rho_i| and accepted set A,
    E cos(g_i, sum_A g_j) = alpha_i S_a / sqrt(S_a^2 + S_b^2), S_a = sum_A alpha_j,
    S_b^2 = sum_A beta_j^2, scatter ~ 1/sqrt(D)."""
    from paper_2412_18052_b200 import workloads
    w = workloads.config(1)
    gs = [workloads.as_numpy_bits(g) for g in w.grads]
    r = orc.filter_accumulate(gs, w.taus[0])
    alpha = [math.copysign(math.sqrt(abs(x)), x) for x in w.rho]
    beta2 = [1 - abs(x) for x in w.rho]
    A = [0]
    for i in range(1, 4):
        sa = sum(alpha[j] for j in A)
        sb2 = sum(beta2[j] for j in A)
        want = 1.0 - alpha[i] * sa / math.sqrt(sa * sa + sb2)
        assert abs(r.dist[i] - want) < 5e-3, (i, r.dist[i], want)
        if r.mask[i]:
            A.append(i)
    assert r.mask.tolist() == [1, 1, 0, 0] and r.count == 2
    assert [round(float(x), 2) for x in r.dist] == [0.0, 0.33, 1.0, 1.5]


def pin_any_seed_variant():
    """Order-indifferent variant: it is Algorithm 1 run from every seed in ring order with
    the largest count kept (checked against the plain routine, seed by seed), and it rescues
    Section 3.1's degenerate example of a first gradient orthogonal to all others."""
    e = f32(0, 0, 0, 1)
    a = f32(1, 0.1, 0, 0)
    b = f32(1, -0.1, 0.1, 0)
    c = f32(0.9, 0, -0.1, 0)
    gs = [e, a, b, c]
    plain = orc.filter_accumulate(gs, 0.5)
    assert plain.count == 1                                  # the whole macrobatch would be wasted
    r, seed, counts = orc.filter_any_seed(gs, 0.5)
    assert seed == 1 and r.count == 3 and r.mask.tolist() == [0, 1, 1, 1]
    assert counts.tolist() == [1, 3, 3, 3]                   # ties go to the smallest seed
    assert np.allclose(r.out, (a.astype(np.float64) + b + c) / 3, rtol=1e-15)
    rng = np.random.RandomState(12)
    for K, D, tau in ((3, 7, 0.6), (5, 40, 0.8), (6, 129, 0.97)):
        gs = _rand_grads(rng, K, D, "f32", shared=0.4)
        gs[1] = (-gs[0]).astype(np.float32)
        r, seed, counts = orc.filter_any_seed(gs, tau)
        per_seed = [orc.filter_accumulate(gs, tau, order=[(s + t) % K for t in range(K)]) for s in range(K)]
        assert counts.tolist() == [p.count for p in per_seed]
        best = max(range(K), key=lambda s: (per_seed[s].count, -s))
        assert seed == best and r.count == per_seed[best].count
        assert r.mask.tolist() == per_seed[best].mask.tolist()
        assert np.array_equal(r.out, per_seed[best].out) and np.array_equal(r.dist, per_seed[best].dist)


def pin_bucketed_variant():
    """Bucketed variant: one bucket is plain GAF; several buckets are plain GAF on each slice;
    an empty bucket is legal; buckets decide independently."""
    rng = np.random.RandomState(13)
    K, D = 4, 60
    gs = _rand_grads(rng, K, D, "f32", shared=0.6)
    gs[2][:20] = -gs[0][:20]                       # disagrees in the first bucket only
    whole = orc.filter_accumulate(gs, 0.9)
    out, mask, dist, count = orc.filter_bucketed(gs, 0.9, [0, D])
    assert np.array_equal(out, whole.out) and mask[0].tolist() == whole.mask.tolist()
    assert count.tolist() == [whole.count] and np.array_equal(dist[0], whole.dist)
    offsets = [0, 20, 20, 47, D]
    out, mask, dist, count = orc.filter_bucketed(gs, 0.9, offsets, order=[1, 0, 3, 2])
    seen = set()
    for b in range(4):
        lo, hi = offsets[b], offsets[b + 1]
        r = orc.filter_accumulate([g[lo:hi] for g in gs], 0.9, order=[1, 0, 3, 2])
        assert np.array_equal(out[lo:hi], r.out) and mask[b].tolist() == r.mask.tolist()
        assert count[b] == r.count and np.array_equal(dist[b], r.dist)
        seen.add(tuple(mask[b].tolist()))
    assert mask[1].tolist() == [0, 1, 0, 0] and count[1] == 1   # empty bucket: zero norms, distance 1 > tau
    assert len(seen) >= 2                           # buckets really decide on their own


def pin_all_cores_form_equals_single_thread():
    """The several-threads form of the filter (the benchmark's all-cores CPU baseline) is the same
    computation: identical masks and counts, distances and outputs equal to 1e-12 (only the order
    in which the chunk sums are combined differs), for every thread count including more threads
    than elements, both element types, an explicit order, and the tau = 2 / reject-all pins."""
    rng = np.random.RandomState(31)
    for K, D, dtype in ((4, 10_007, np.float32), (5, 1_001, np.uint16), (3, 5, np.float32), (1, 40, np.float32)):
        if dtype == np.float32:
            grads = [rng.randn(D).astype(np.float32) + 0.6 * (i % 2) for i in range(K)]
        else:
            grads = [(rng.randn(D).astype(np.float32) + 0.5).view(np.uint32).__rshift__(16).astype(np.uint16)
                     for _ in range(K)]
        order = [int(x) for x in rng.permutation(K)]
        for tau in (0.9, 1.0, 2.0, -1.0):
            want = orc.filter_accumulate(grads, tau, order=order)
            for n_threads in (1, 2, 3, 7, 16):
                got = orc.filter_accumulate_all_cores(grads, tau, order=order, n_threads=n_threads)
                assert got.mask.tolist() == want.mask.tolist() and got.count == want.count
                assert np.max(np.abs(got.dist - want.dist)) <= 1e-12
                scale = np.max(np.abs(want.out)) + 1e-300
                assert np.max(np.abs(got.out - want.out)) <= 1e-12 * scale
    # tau = 2 is the plain mean of Eq. 2, also through this route
    grads = [rng.randn(999).astype(np.float32) for _ in range(4)]
    got = orc.filter_accumulate_all_cores(grads, 2.0, n_threads=4)
    assert np.allclose(got.out, np.mean(np.stack(grads).astype(np.float64), axis=0), rtol=0, atol=1e-15)


ALL_PINS = [
    pin_stated_values,
    pin_figure2_angles,
    pin_invariants,
    pin_matches_scipy_and_numpy,
    pin_bf16_widening,
    pin_tau2_is_plain_mean,
    pin_reject_all_keeps_seed,
    pin_k2_operating_point,
    pin_threshold_is_inclusive,
    pin_order_dependence,
    pin_running_sum_not_pairwise,
    pin_brute_force_masks,
    pin_bilinearity_ties_filter_to_pairwise,
    pin_forced_decisions,
    pin_closed_form_mixture,
    pin_any_seed_variant,
    pin_bucketed_variant,
    pin_all_cores_form_equals_single_thread,
]
