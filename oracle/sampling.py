"""CPU ORACLE -- test infrastructure, not product code.

The vocabulary-wide part of speculative sampling, step by step, in numpy:
temperature softmax, inverse-CDF sampling, and the accept / reject / resample rule.

The paper names the method (Section "Speculative Sampling", Figure 2: the target model
passes or refuses each of the K draft tokens, and samples one token itself when a
rejection occurs) and quotes its guarantee (Section "Autoregressive vs Speculative
Sampling": the target distribution is recovered).  The rule that achieves the guarantee is
the modified rejection sampling of the scheme the paper cites:

    accept draft token x~_i  with probability  min(1, p_i(x~_i) / q_i(x~_i));
    at the first rejection draw from the residual  max(0, p_i - q_i) / sum(max(0, p_i - q_i));
    if all K are accepted draw a bonus token from p_{K+1}.

Readings where the paper is silent:
  * the acceptance test is evaluated division-free in fp32 as  u * q(x~) < p(x~)  (strict),
    so q(x~) = 0 accepts iff p(x~) > 0 and no NaN can arise;
  * an all-zero residual (p == q to rounding, yet a rejection happened) falls back to p;
  * inverse CDF: the smallest index i whose inclusive prefix sum c_i exceeds u * S, prefix sums
    in index order in float64; if rounding leaves none, the largest index with weight > 0;
  * temperature divides the logits of both models; T = 0 is greedy: the distribution is the
    one-hot at the argmax (lowest index on ties), which makes the same rule reduce to
    "accept iff x~ equals the target argmax".

Probabilities handed between steps are fp32 (the storage type of p and q rows); sums run in
float64.  Pins: tests/test_oracle_sampling.py (closed-form identity, brute-force grids,
special cases).
"""
from __future__ import annotations

import numpy as np


def argmax_lowest(row: np.ndarray) -> int:
    return int(np.argmax(row))  # numpy returns the first maximal index


def softmax_t(logits_row: np.ndarray, temperature: float) -> np.ndarray:
    """softmax(logits / T) as fp32; T == 0 gives the one-hot at the argmax."""
    row = np.asarray(logits_row)
    if temperature == 0.0:
        p = np.zeros(row.shape[0], np.float32)
        p[argmax_lowest(row)] = 1.0
        return p
    z = row.astype(np.float64) / float(temperature)
    z = z - z.max()
    e = np.exp(z)
    return (e / e.sum()).astype(np.float32)


def filter_top_k_top_p(p_row: np.ndarray, top_k: int = 0, top_p: float = 1.0) -> np.ndarray:
    """Restrict a distribution to its most probable tokens and renormalise (the paper's Section
    "Autoregressive vs Speculative Sampling" names sampling "from top-p" as the alternative to the argmax;
    it prints no formula, so this is the reading used for both models' distributions):

      1. top-k (top_k > 0): t_k = the top_k-th largest probability; keep every token with p >= t_k
         (tokens tied with the threshold are all kept, so the kept set can exceed top_k);
      2. top-p (0 < top_p < 1), applied to what step 1 kept: walk the kept tokens in order of decreasing
         probability, adding them up in float64; t_p = the probability at which the running sum first
         reaches top_p x (mass kept by step 1); keep every token with p >= t_p (ties again all kept);
      3. every other token gets probability 0 and the kept ones are divided by the kept mass (summed in
         float64 in index order, rounded to fp32; the division is fp32).

    top_k = 0 and top_p = 1 return the row unchanged."""
    p = np.asarray(p_row, np.float32)
    if top_k <= 0 and not (0.0 < top_p < 1.0):
        return p
    keep = np.ones(p.shape[0], bool)
    if top_k > 0 and top_k < p.shape[0]:
        t_k = np.sort(p)[::-1][top_k - 1]
        keep &= p >= t_k
    if 0.0 < top_p < 1.0:
        mass_k = float(p[keep].astype(np.float64).sum())
        vals = np.sort(p[keep])[::-1]
        c = np.cumsum(vals.astype(np.float64))
        i = int(np.searchsorted(c, float(np.float32(top_p)) * mass_k, side="left"))
        i = min(i, vals.shape[0] - 1)
        keep &= p >= vals[i]
    mass = np.float32(p[keep].astype(np.float64).sum())
    out = np.zeros_like(p)
    out[keep] = p[keep] / mass
    return out


def inv_cdf(weights: np.ndarray, u) -> int:
    """Smallest i with c_i > u * S (c inclusive float64 prefix sums, S = c[-1])."""
    w = np.asarray(weights)
    c = np.cumsum(w.astype(np.float64))
    t = float(np.float32(u)) * float(c[-1])
    i = int(np.searchsorted(c, t, side="right"))
    if i >= w.shape[0]:
        nz = np.nonzero(w > 0)[0]
        i = int(nz[-1]) if nz.size else w.shape[0] - 1
    return i


def accept_test(u, q_x, p_x) -> bool:
    """Accept with probability min(1, p/q):  u * q < p  in fp32."""
    return bool(np.float32(u) * np.float32(q_x) < np.float32(p_x))


def residual(p_row: np.ndarray, q_row: np.ndarray) -> np.ndarray:
    return np.maximum(np.float32(0.0), p_row.astype(np.float32) - q_row.astype(np.float32))


def accept_resample(p_rows, q_rows, draft_tokens, u_accept, u_resample):
    """One verification: p_rows [K+1,V], q_rows [K,V], draft_tokens [K], u_accept [K].

    Returns (a, y): the number of accepted draft tokens and the token emitted after them.
    """
    K = len(draft_tokens)
    a = 0
    for i in range(K):
        x = int(draft_tokens[i])
        if accept_test(u_accept[i], q_rows[i][x], p_rows[i][x]):
            a += 1
        else:
            break
    if a < K:
        r = residual(p_rows[a], q_rows[a])
        if float(r.astype(np.float64).sum()) <= 0.0:
            y = inv_cdf(p_rows[a], u_resample)
        else:
            y = inv_cdf(r, u_resample)
    else:
        y = inv_cdf(p_rows[K], u_resample)
    return a, y
