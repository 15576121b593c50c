"""CPU oracle for the cache-pool planner (plain Python / numpy, fp64).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests may import this module.  It shares
nothing with the library.  Every function restates one numbered algorithm or
equation of the paper in the paper's order and notation:

  hit_distribution      Algorithm 2 "Probabilistic Modeling of Cache Hits"
  makespan              Algorithm 3 "Makespan Estimation"
  pattern_probability   Section 3.4, the conditional probability of a cache hit pattern
  expected_makespan     Algorithm 4, the cost of one memory partition (its inner loops)
  plan                  Algorithm 4 "Hierarchical Cache Pool Planning" (the grid search)
  selection_probs       appendix on the maximum-entropy property: modified iterative
                        proportional fitting, weight update with elementary symmetric polynomials

Pools are indexed 0 = F, 1 = C, 2 = S, 3 = E, the cache hierarchy's order.
Readings where the paper is loose: Algorithm 4 reuses the letter u for the rank
offset of a pool (it is the SM-chunk delay elsewhere): here the offset is `at`.
The number of experts a pool holds is floor(ratio * budget / size of one expert in
that pool's state), cut so that the pools together hold at most |N| experts.
"""
import itertools

import numpy as np


def hit_distribution(q):
    """Algorithm 2: Phi_S(h) for h = 0..|S|, the ranks of S being selected independently with probabilities q."""
    S = len(q)
    phi = [0.0] * (S + 1)
    phi[0] = 1.0
    for r in range(1, S + 1):
        qr = q[r - 1]
        for h in range(S, 0, -1):
            phi[h] = phi[h] * (1 - qr) + phi[h - 1] * qr
        phi[0] = phi[0] * (1 - qr)
    return phi


def makespan(k, h, c, v, u, L, K, n):
    """Algorithm 3.  h = (h_F, h_C, h_S, h_E)."""
    hF, hC, hS, hE = h
    n_SM = n * (k - (hF + hC + hS))
    n_E = n * K * (k - (hF + hC + hE))
    T_io = n_SM * u + n_E * v
    n_D = n * K * (k - hF)
    T_decomp = (n_E * v + n_D * c) / L
    return max(T_io, T_decomp)


def pool_intervals(capacity, n_ranks):
    """Rank intervals of the pools F, C, S, E laid on the ranks one after the other, then the miss pool."""
    at, out = 0, []
    for S_p in capacity:
        out.append((at, at + S_p))
        at += S_p
    assert at <= n_ranks
    out.append((at, n_ranks))
    return out


def pattern_probability(q, k, capacity, h):
    """P(h | exactly k experts selected) = Phi_M(k_rem) / Phi_N(k) * prod_p Phi_p(h_p)  (Section 3.4)."""
    iv = pool_intervals(capacity, len(q))
    k_rem = k - sum(h)
    phi_M = hit_distribution(q[iv[4][0]:iv[4][1]])
    if k_rem < 0 or k_rem >= len(phi_M):
        return 0.0
    pr = phi_M[k_rem] / hit_distribution(q)[k]
    for p in range(4):
        pr *= hit_distribution(q[iv[p][0]:iv[p][1]])[h[p]]
    return pr


def expected_makespan(q, k, capacity, c, v, u, L, K, n):
    """Algorithm 4, cost of one partition: sum over hit patterns of delay times probability."""
    cost = 0.0
    for h in itertools.product(*[range(S_p + 1) for S_p in capacity]):
        if sum(h) > k:
            continue
        cost += makespan(k, h, c, v, u, L, K, n) * pattern_probability(q, k, capacity, h)
    return cost


def elementary_symmetric(w, n):
    """R(n, C) = sum over n-subsets of C of the product of their weights: the coefficient of x^n in
    prod_j (1 + w_j x)."""
    poly = np.array([1.0])
    for wj in w:
        poly = np.convolve(poly, [1.0, wj])
    return poly[n] if n < len(poly) else 0.0


def selection_probs(f, k, iters=2000):
    """Modified iterative proportional fitting: w(0) = f, w(t+1)_i = w(t)_i f_i / f(t)_i with
    f(t)_i = w_i R(k-1, N minus i) / R(k, N); q_i = w_i / (1 + w_i)."""
    f = np.asarray(f, dtype=np.float64)
    w = f.copy()
    for _ in range(iters):
        Rk = elementary_symmetric(w, k)
        ft = np.array([w[i] * elementary_symmetric(np.delete(w, i), k - 1) / Rk for i in range(len(w))])
        w = w * f / ft
    return w / (1 + w)


def capacities(ratios, budget, expert_size, n_ranks):
    cap, used = [], 0
    for g, size in zip(ratios, expert_size):
        S_p = int(np.floor(g * budget / size + 1e-9)) if g > 0 else 0
        S_p = min(S_p, n_ranks - used)
        cap.append(S_p)
        used += S_p
    return cap


def plan(f, k, pools, budget, expert_size, c, v, u, L, K, n, step):
    """Algorithm 4: every vector of memory ratios on the grid of width `step` that sums to one and is zero
    outside `pools`; returns (best ratios, their capacities, minimal expected makespan)."""
    q = selection_probs(f, k)
    G = int(round(1 / step))
    best = (None, None, float("inf"))
    for g in itertools.product(range(G + 1), repeat=4):          # F varies slowest
        if sum(g) != G or any(g[p] and p not in pools for p in range(4)):
            continue
        ratios = [x / G for x in g]
        cap = capacities(ratios, budget, expert_size, len(f))
        cost = expected_makespan(q, k, cap, c, v, u, L, K, n)
        if cost < best[2]:
            best = (ratios, cap, cost)
    return best
