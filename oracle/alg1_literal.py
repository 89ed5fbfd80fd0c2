"""Pure-Python restatements used to cross-check the C oracle on small inputs.

TEST INFRASTRUCTURE, not a product path.  Three independent pieces:

* ``alg1_token``   -- the routing rule of Algorithm 1 stated as set definitions over all n
  experts (pool membership, candidates as the pool members with fewer than c pool members
  ahead of them, the choice as the candidates with fewer than k smaller (load, rank) keys),
  evaluated by counting; nothing is sorted or trimmed step by step.
* ``brute_force_token`` -- the selection step by exhaustive search: among all k-subsets of
  the candidate set, the one whose sorted (load, score-rank) key vector is smallest.
* ``imbalance`` / ``max_violation`` -- the imbalance factor of Motivation and MV of
  Evaluation/Metrics.
"""
from __future__ import annotations

import itertools

import numpy as np


def score_order(s, x=None):
    """Indices by score descending; ties by logit descending (if given), then index."""
    n = len(s)
    if x is None:
        return sorted(range(n), key=lambda i: (-float(s[i]), i))
    return sorted(range(n), key=lambda i: (-float(s[i]), -float(x[i]), i))


def alg1_token(s, L, k, c, eps_high, t_fix, x=None):
    """The routing rule for one token (Algorithm 1 with TOP trimming is the source of the rule),
    written as definitions over all n experts rather than as a procedure.  s: fp32 scores,
    L: integer loads.

      peaked      the k best scores add up (fp32, best first) to at least eps_high
      in the pool an expert is one of the k best, or its score reaches t_fix times the best score
      candidate   a pool member with fewer than c pool members ranked ahead of it by score
      chosen      a candidate with fewer than k candidates whose (load, score rank) is smaller

    Returns (the chosen experts by ascending (load, score rank) -- for a peaked token the k
    best by score --, expanded flag, number of candidates).  All comparisons on scores are
    made in fp32, as the scores are given.
    """
    s = np.asarray(s, np.float32)
    n = len(s)
    rank = {i: r for r, i in enumerate(score_order(s, x))}
    best = [i for i in range(n) if rank[i] < k]
    best.sort(key=rank.get)
    mass = np.float32(s[best[0]])
    for i in best[1:]:
        mass = np.float32(mass + s[i])
    if mass >= np.float32(eps_high):
        return best, False, 0
    floor = np.float32(np.float32(t_fix) * s[best[0]])
    pool = [i for i in range(n) if rank[i] < k or s[i] >= floor]
    cand = [i for i in pool if sum(rank[j] < rank[i] for j in pool) < c]
    key = lambda i: (int(L[i]), rank[i])
    chosen = [i for i in cand if sum(key(j) < key(i) for j in cand) < k]
    return sorted(chosen, key=key), True, len(cand)


def alg1_sequence(S, loads, k, c, eps_high, t_fix, X=None):
    """Route the rows of S in order, adding one to the load of each chosen expert after
    every token.  Returns (ids [T][k], final loads, expanded flags)."""
    L = [int(v) for v in loads]
    ids, flags = [], []
    for t in range(len(S)):
        A, expanded, _ = alg1_token(S[t], L, k, c, eps_high, t_fix, None if X is None else X[t])
        for e in A:
            L[e] += 1
        ids.append(A)
        flags.append(expanded)
    return ids, L, flags


def brute_force_token(cand_in_rank_order, L, k):
    """Best k-subset of the candidates by exhaustive search.

    A candidate's key is (load, score rank).  A subset is scored by its keys sorted
    ascending; the lexicographically smallest vector wins.  Returned in key order.
    """
    keyed = [(int(L[e]), r, e) for r, e in enumerate(cand_in_rank_order)]
    best = None
    for sub in itertools.combinations(keyed, k):
        vec = sorted(sub)
        if best is None or vec < best:
            best = vec
    return [e for (_, _, e) in best]


def imbalance(counts) -> float:
    """I = max_e N_e / mean_e N_e  (Motivation, expert imbalance of one layer and batch)."""
    counts = np.asarray(counts, np.float64)
    mean = counts.mean()
    return float(counts.max() / mean) if mean > 0 else 1.0


def imbalance_stats(counts, expert_to_bin, n_bins, placement=None):
    """Imbalance figures of one call over several layers, in fp64 (Motivation: expert imbalance
    I_L = max_e N_e / mean_e N_e per layer, its token-weighted aggregate I_agg = sum_L w_L I_L
    with w_L = tokens of layer L / all tokens, and the same on device bins with
    N_g = sum_e A[g,e] N_e; A is the 0/1 matrix of expert_to_bin unless a general placement
    [n_bins, E] with unit column sums is given).  counts: [L, E].
    Returns dict(I [L], MV [L] = I - 1, I_bins [L], I_agg, I_agg_bins); a layer without
    assignments has I = 1."""
    counts = np.asarray(counts, np.float64)
    L, E = counts.shape
    bins = np.zeros((L, n_bins), np.float64)
    for e in range(E):
        if placement is None:
            bins[:, int(expert_to_bin[e])] += counts[:, e]
        else:
            for g in range(n_bins):
                bins[:, g] += float(placement[g][e]) * counts[:, e]
    tot = counts.sum(1)

    def ratio(a):
        mean = a.mean(1)
        return np.where(mean > 0, a.max(1) / np.where(mean > 0, mean, 1.0), 1.0)

    I, Ib = ratio(counts), ratio(bins)
    w = tot / tot.sum() if tot.sum() > 0 else np.full(L, 1.0 / L)
    return dict(I=I, MV=I - 1.0, I_bins=Ib, I_agg=float((w * I).sum()),
                I_agg_bins=float((w * Ib).sum()))


def max_violation(counts) -> float:
    """MV, read as how far the most loaded expert exceeds the average, relative to it:
    max/mean - 1 (zero for perfect balance, as the load-only baseline attains)."""
    return imbalance(counts) - 1.0
