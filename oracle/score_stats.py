"""Gate-score statistics of a batch of tokens (Layer Variability in Gate Score Distributions:
top-k mass M_k, Shannon entropy, routing regimes), written out plainly.

TEST INFRASTRUCTURE, not a product path.  Input: the fp32 scores of each token, as the oracle's
softmax gives them, and the logits they came from (for the ranking).  Everything the paper
defines is taken as defined:

* M_k of a token = sum of its k highest scores, ranked by (logit descending, index ascending)
  and added left to right in fp32, exactly as the routing rule forms it; the statistic is the
  mean over tokens.
* entropy of a token = -sum_i s_i ln s_i (nats), terms with s_i = 0 contributing 0, in fp64.
* regimes: the paper names single-head, plateau and smooth and gives no numeric criterion.
  The criterion here is a reading -- parity unpinned by the paper -- and counts the experts whose score is
  comparable to the best one, n_near = #{i : s_i >= fl32(near_ratio * s_max)}:
      n_near == 1                 single-head   (nothing else comes near the top expert)
      2 <= n_near <= plateau_max  plateau       (a few comparable experts at the top)
      n_near >  plateau_max       smooth        (many comparable experts)
  n_near is the size of the routing rule's candidate pool for t_fix = near_ratio.

Also returned: the histogram of M_k over 64 equal bins of [0, 1] (bin = min(63, floor(64 M_k))),
from which a dominance cutoff can be read off as a quantile, and the means of s_max and n_near.
"""
from __future__ import annotations

import math

import numpy as np

HIST_BINS = 64


def token_stats(x, s, k, near_ratio, plateau_max):
    """(M_k fp32, entropy fp64, n_near, regime 0/1/2, s_max fp32) of one token."""
    x = np.asarray(x, np.float32)
    s = np.asarray(s, np.float32)
    order = sorted(range(len(x)), key=lambda i: (-float(x[i]), i))
    Mk = np.float32(s[order[0]])
    for j in range(1, k):
        Mk = np.float32(Mk + s[order[j]])
    H = 0.0
    for v in s:
        if v > 0:
            H -= float(v) * math.log(float(v))
    smax = np.float32(s[order[0]])
    thr = np.float32(np.float32(near_ratio) * smax)
    n_near = int(sum(1 for v in s if v >= thr))
    regime = 0 if n_near == 1 else (1 if n_near <= plateau_max else 2)
    return Mk, H, n_near, regime, smax


def score_stats(x, s, k, near_ratio, plateau_max):
    """Statistics of T tokens.  x, s: [T, E] fp32 logits and scores.  Returns a dict:
    tokens, mass_sum (exact, as a Python float of the fp64 sum of fp32 values), mean_mass,
    entropy_sum, mean_entropy, regimes [3], near_sum, mean_near, smax_sum, mean_smax,
    mass_hist [64]."""
    T = len(x)
    mass = ent = smx = 0.0
    near = 0
    regimes = [0, 0, 0]
    hist = [0] * HIST_BINS
    for t in range(T):
        Mk, H, n_near, regime, smax = token_stats(x[t], s[t], k, near_ratio, plateau_max)
        mass += float(Mk)          # fp32 values >= 2^-9 summed in fp64: exact for T < 2^20
        ent += H
        smx += float(smax)
        near += n_near
        regimes[regime] += 1
        hist[min(HIST_BINS - 1, int(math.floor(float(Mk) * HIST_BINS)))] += 1
    d = max(T, 1)
    return dict(tokens=T, mass_sum=mass, mean_mass=mass / d, entropy_sum=ent,
                mean_entropy=ent / d, regimes=regimes, near_sum=near, mean_near=near / d,
                smax_sum=smx, mean_smax=smx / d, mass_hist=hist)
