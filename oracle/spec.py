"""CPU ORACLE -- test infrastructure, not product code.

The two generation loops the paper compares (Section "Autoregressive vs Speculative
Sampling"; Appendix: "Autoregressive Decode" vs "Speculative Decode"), for one sequence,
on top of the cached decoder:

  * autoregressive: one target forward per token (Eq. 1), token drawn from softmax(logits/T);
  * speculative with two KV caches (Section "So, what's the problem?"): the draft model
    proposes K tokens with its own cache, the target scores the pending token and the K
    drafts in ONE pass against its cache (Figure 2), the accept/reject rule decides, and
    both caches are cut back to the accepted prefix so that nothing is recomputed.

Cache protocol (the paper poses it as questions; this is the reading used):
  committed tokens x[0..n).  The target cache holds rows 0..n-2 (it is behind by exactly the
  pending token x[n-1]).  The draft cache holds n-1 or n-2 rows.  One iteration:
    1. draft: feed x[n_d..n) (1 or 2 catch-up rows), draw x~_1 from q_1; then K-1 single-row
       steps feeding x~_{i-1}.  Draft cache length becomes n+K-1.
    2. verify: feed [x[n-1], x~_1..x~_K] (K+1 rows) to the target without committing.
    3. accept scan and resample / bonus  ->  a, y.
    4. emit x~_1..x~_a, y.  Target length += a+1.  Draft length = min(n+a, n+K-1).
  Every iteration consumes its own block of 2K+1 uniforms (K draft draws, K accept tests,
  1 resample), used or not.  Generation stops at >= N new tokens and is truncated to N.
"""
from __future__ import annotations

from typing import Callable, Dict, List

import numpy as np

from . import sampling
from .decoder import Model


def autoregressive_generate(target: Model, prompt, n_new: int, temperature: float,
                            uniforms: Callable[[int], np.ndarray], s_max: int, top_k: int = 0,
                            top_p: float = 1.0) -> Dict:
    prompt = [int(t) for t in prompt]
    cache = target.new_cache(s_max)
    if len(prompt) > 1:
        cache.feed(prompt[:-1], want_logits=False)
    pending = prompt[-1]
    out: List[int] = []
    for j in range(n_new):
        logits = cache.feed([pending])
        p = sampling.filter_top_k_top_p(sampling.softmax_t(logits[0], temperature), top_k, top_p)
        y = sampling.inv_cdf(p, uniforms(j)[0])
        out.append(y)
        pending = y
    return {"tokens": out}


def speculative_generate(target: Model, draft: Model, prompt, n_new: int, K: int,
                         temperature: float, uniforms: Callable[[int], np.ndarray],
                         s_max: int, keep_trace: bool = False, top_k: int = 0, top_p: float = 1.0,
                         k_of: Callable[[int, List[int]], int] = None) -> Dict:
    """top_k / top_p: both models' distributions are restricted (sampling.filter_top_k_top_p) before the
    draft draws and before the accept / resample rule, so the emitted tokens follow the restricted
    target distribution.
    k_of: optional schedule of the number of draft tokens: iteration `it` drafts k_of(it, accepted so far)
    tokens (1 <= k <= K).  The block of uniforms keeps the layout of K: draft draws u[0:k], accept tests
    u[K:K+k], the target's draw u[2K]."""
    x = [int(t) for t in prompt]
    tc, dc = target.new_cache(s_max), draft.new_cache(s_max)
    if len(x) > 1:
        tc.feed(x[:-1], want_logits=False)
        dc.feed(x[:-1], want_logits=False)
    n0 = len(x)
    trace, accepted, target_rows, catchups = [], [], 0, []
    it = 0
    while len(x) - n0 < n_new:
        n = len(x)
        u = np.asarray(uniforms(it), np.float32)
        assert u.shape[0] == 2 * K + 1
        Kmax = K
        if k_of is not None:
            K = int(k_of(it, accepted))
            assert 1 <= K <= Kmax
        u_d, u_a, u_r = u[:K], u[Kmax:Kmax + K], u[2 * Kmax]
        assert tc.len == n - 1 and dc.len in (n - 1, n - 2)
        # 1. draft K tokens
        catchups.append(n - dc.len)
        q_rows, drafts = [], []
        feed = x[dc.len:n]
        for i in range(K):
            logits = dc.feed(feed)
            q = sampling.filter_top_k_top_p(sampling.softmax_t(logits[-1], temperature), top_k, top_p)
            t = sampling.inv_cdf(q, u_d[i])
            q_rows.append(q)
            drafts.append(t)
            feed = [t]
        assert dc.len == n + K - 1
        # 2. verify: K+1 rows in one target pass, not committed yet
        logits = tc.feed([x[n - 1]] + drafts, advance=False)
        target_rows += K + 1
        p_rows = [sampling.filter_top_k_top_p(sampling.softmax_t(logits[i], temperature), top_k, top_p)
                  for i in range(K + 1)]
        # 3. accept / reject / resample
        a, y = sampling.accept_resample(p_rows, q_rows, drafts, u_a, u_r)
        # 4. emit and fix both caches
        x.extend(drafts[:a])
        x.append(y)
        tc.len += a + 1
        dc.rollback(min(n + a, n + K - 1))
        accepted.append(a)
        if keep_trace:
            trace.append(dict(n=n, drafts=list(drafts), a=a, y=y, u=u.copy(), k=K,
                              p=np.stack(p_rows), q=np.stack(q_rows), logits=logits.copy()))
        K = Kmax
        it += 1
    return {"tokens": x[n0:n0 + n_new], "all_tokens": x, "accepted": accepted, "iterations": it,
            "target_rows": target_rows, "catchups": catchups, "trace": trace,
            "target_cache": tc, "draft_cache": dc}
