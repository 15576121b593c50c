"""The cache-pool planner (Section 3.4, Algorithms 2-4 and the iterative proportional fitting of
the appendix): the CPU oracle against brute force and worked examples, then the library against the
oracle.  Host only."""
import itertools

import numpy as np
import pytest

from oracle import planner as op
from paper_2601_21198_b200 import build


@pytest.fixture(scope="module")
def zb():
    build.build()
    from paper_2601_21198_b200 import binding
    return binding


def subsets_distribution(q):
    """P(exactly h selected) by enumerating all 2^n outcomes of the independent trials."""
    n = len(q)
    out = np.zeros(n + 1)
    for bits in itertools.product((0, 1), repeat=n):
        out[sum(bits)] += np.prod([qi if b else 1 - qi for qi, b in zip(q, bits)])
    return out


def rank_model(n, k, s=1.2):
    """Zipf-like inclusion probabilities by rank that sum to k and stay below one."""
    f = 1.0 / np.arange(1, n + 1) ** s
    f = f / f.sum() * k
    while f.max() >= 0.98:                      # flatten until feasible
        f = np.minimum(f, 0.9)
        f = f / f.sum() * k
    return f


# ------------------------------------------------------------------ oracle pins
def test_oracle_hit_distribution_is_the_poisson_binomial():
    rng = np.random.default_rng(0)
    for n in (1, 2, 5, 9):
        q = rng.uniform(0, 1, n)
        phi = np.array(op.hit_distribution(list(q)))
        assert np.allclose(phi, subsets_distribution(q), atol=1e-14)
        assert abs(phi.sum() - 1) < 1e-14 and abs((phi * np.arange(n + 1)).sum() - q.sum()) < 1e-13
    # equal probabilities: the binomial distribution
    from math import comb
    phi = op.hit_distribution([0.3] * 6)
    assert np.allclose(phi, [comb(6, h) * 0.3 ** h * 0.7 ** (6 - h) for h in range(7)])
    assert op.hit_distribution([]) == [1.0] and op.hit_distribution([1.0, 0.0]) == [0.0, 1.0, 0.0]


def test_oracle_makespan_worked_example():
    # k = 6 experts of n = 3 tensors, K = 4 shards; hits: 1 full, 2 compressed, 1 SM-only, 1 E-only, 1 miss.
    # SM-chunks to read: E-only hit + miss = 2 experts -> 6 chunks; E-chunks to read: SM-only hit + miss = 2
    # experts -> 24 chunks; E-chunks to decompress: all but the full one = 5 experts -> 60 chunks.
    c, v, u, L = 2.0, 0.5, 3.0, 4
    t_io = 6 * 3.0 + 24 * 0.5                    # 30
    t_dec = (24 * 0.5 + 60 * 2.0) / 4            # 33
    assert op.makespan(6, (1, 2, 1, 1), c, v, u, L, 4, 3) == max(t_io, t_dec) == 33.0
    assert op.makespan(6, (6, 0, 0, 0), c, v, u, L, 4, 3) == 0.0            # everything resident in full
    assert op.makespan(6, (0, 0, 0, 0), c, v, 30.0, L, 4, 3) == 18 * 30.0 + 72 * 0.5   # I/O bound when u is large


def test_oracle_selection_probs_reproduce_the_inclusion_probabilities():
    """Choosing k of n ranks with probability proportional to the product of w_i = q_i / (1 - q_i) -- the
    independent trials conditioned on exactly k successes -- must include rank i with probability f_i."""
    for n, k in ((5, 2), (8, 3), (9, 6)):
        f = rank_model(n, k)
        q = op.selection_probs(f, k)
        w = q / (1 - q)
        incl, total = np.zeros(n), 0.0
        for S in itertools.combinations(range(n), k):
            pr = np.prod(w[list(S)])
            total += pr
            incl[list(S)] += pr
        assert np.allclose(incl / total, f, atol=1e-9)
    # equal inclusion probabilities: equal selection probabilities
    q = op.selection_probs([0.25] * 8, 2)
    assert np.allclose(q, q[0])


def test_oracle_pattern_probabilities_are_a_distribution_and_match_enumeration():
    n, k = 9, 3
    q = op.selection_probs(rank_model(n, k), k)
    cap = [2, 1, 2, 1]
    pats = [h for h in itertools.product(*[range(c + 1) for c in cap]) if sum(h) <= k]
    assert abs(sum(op.pattern_probability(q, k, cap, h) for h in pats) - 1) < 1e-12
    # brute force: every k-subset with its conditional probability, binned by hit pattern
    iv = op.pool_intervals(cap, n)
    w = q / (1 - q)
    prob, total = {}, 0.0
    for S in itertools.combinations(range(n), k):
        pr = np.prod(w[list(S)])
        total += pr
        h = tuple(sum(1 for r in S if iv[p][0] <= r < iv[p][1]) for p in range(4))
        prob[h] = prob.get(h, 0.0) + pr
    for h in pats:
        assert abs(op.pattern_probability(q, k, cap, h) - prob.get(h, 0.0) / total) < 1e-12
    costs = dict(c=2.0, v=0.5, u=3.0, L=4, K=4, n=3)
    want = sum(pr / total * op.makespan(k, h, **costs) for h, pr in prob.items())
    assert abs(op.expected_makespan(q, k, cap, **costs) - want) < 1e-10


def test_oracle_plan_prefers_what_the_costs_say():
    n, k = 12, 3
    f = rank_model(n, k)
    size = [1.0, 0.68, 0.5, 0.18]
    base = dict(L=4, K=4, n=3, step=0.25)
    # free decompression and free E-chunk reads: only SM-chunk reads cost, and the SM pool holds the most experts per byte
    r, cap, cost = op.plan(f, k, {0, 1, 2, 3}, 3.0, size, c=0.0, v=0.0, u=1.0, **base)
    assert r == [0, 0, 1, 0] and cap == [0, 0, 6, 0]
    # only decompression costs: nothing but full tensors helps
    r, cap, _ = op.plan(f, k, {0, 1, 2, 3}, 3.0, size, c=1.0, v=0.0, u=0.0, **base)
    assert r == [1, 0, 0, 0] and cap == [3, 0, 0, 0]
    # a pool outside the candidate set stays empty
    r, cap, _ = op.plan(f, k, {0, 1}, 3.0, size, c=0.0, v=0.0, u=1.0, **base)
    assert r[2] == r[3] == 0 and cap[2] == cap[3] == 0 and r == [0, 1, 0, 0]
    # with memory for every expert in full the makespan is zero
    assert op.plan(f, k, {0}, 12.0, size, c=1.0, v=1.0, u=1.0, **base)[2] == 0.0


# ------------------------------------------------------------------ library against the oracle
def test_library_matches_the_oracle(zb):
    rng = np.random.default_rng(1)
    for n in (1, 7, 40):
        q = rng.uniform(0, 1, n)
        assert np.allclose(zb.zipmoe_plan_hit_distribution(q), op.hit_distribution(list(q)), atol=1e-14)
    costs = zb.PlanCosts(2.0, 0.5, 3.0, 4, 4, 3)
    for h in itertools.product(range(3), repeat=4):
        if sum(h) <= 6:
            assert zb.zipmoe_plan_makespan(6, h, costs) == op.makespan(6, h, 2.0, 0.5, 3.0, 4, 4, 3)
    for n, k in ((8, 3), (64, 6), (60, 4)):
        f = rank_model(n, k)
        q, iters = zb.zipmoe_plan_selection_probs(f, k)
        if n <= 8:
            assert np.allclose(q, op.selection_probs(f, k), atol=1e-9)
        # the fixed point itself: the inclusion probabilities of the fitted weights are f
        w = q / (1 - q)
        Rk = op.elementary_symmetric(w, k)
        ft = np.array([w[i] * op.elementary_symmetric(np.delete(w, i), k - 1) / Rk for i in range(n)])
        assert np.allclose(ft, f, atol=1e-10) and iters < 1000
        cap = [2, 1, 2, 1]
        got = zb.zipmoe_plan_expected_makespan(q, k, cap, costs)
        assert abs(got - op.expected_makespan(q, k, cap, 2.0, 0.5, 3.0, 4, 4, 3)) < 1e-9 * max(1.0, got)


def test_library_plan_matches_the_oracle(zb):
    n, k = 12, 3
    f = rank_model(n, k)
    size = [1.0, 0.68, 0.5, 0.18]
    for mask, pools in ((15, {0, 1, 2, 3}), (3, {0, 1}), (12, {2, 3}), (8, {3})):
        for c, v, u in ((0.0, 0.0, 1.0), (1.0, 0.0, 0.0), (0.4, 0.1, 1.0), (0.05, 0.3, 1.0)):
            want = op.plan(f, k, pools, 3.0, size, c=c, v=v, u=u, L=4, K=4, n=3, step=0.25)
            r, cap, cost = zb.zipmoe_plan_cache_pools(f, k, mask, 3.0, size, zb.PlanCosts(c, v, u, 4, 4, 3), 0.25)
            # the minimum is unique, the partition that reaches it need not be (ties): the library's partition
            # must be on the grid, inside the candidate set, and reach the minimum when the oracle evaluates it
            assert abs(cost - want[2]) < 1e-9
            assert abs(sum(r) - 1) < 1e-12 and all(abs(x * 4 - round(x * 4)) < 1e-12 for x in r)
            assert all(r[p] == 0 for p in range(4) if p not in pools)
            assert cap == op.capacities(list(r), 3.0, size, n)
            q = op.selection_probs(f, k)
            assert abs(op.expected_makespan(q, k, cap, c, v, u, 4, 4, 3) - want[2]) < 1e-9


def test_library_rejects_bad_arguments(zb):
    costs = zb.PlanCosts(1.0, 1.0, 1.0, 4, 4, 3)
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_plan_hit_distribution([0.5, 1.5])
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_plan_selection_probs([0.5, 0.6, 0.7], 2)          # sums to 1.8, not 2
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_plan_selection_probs([1.0, 0.5, 0.5], 2)          # an inclusion probability of one
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_plan_makespan(2, (1, 1, 1, 0), costs)             # more hits than experts
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_plan_expected_makespan([0.5] * 4, 2, (3, 2, 0, 0), costs)   # pools larger than the rank list
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_plan_cache_pools(rank_model(8, 2), 2, 15, 3.0, [1, 1, 1, 1], costs, 0.3)   # 1 / step not an integer
    with pytest.raises(zb.ZipMoEError):
        zb.zipmoe_plan_cache_pools(rank_model(8, 2), 2, 0, 3.0, [1, 1, 1, 1], costs, 0.25)   # no pool to use
