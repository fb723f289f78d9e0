"""Pins for the oracle's accept / reject / resample rule and its samplers.

The paper fixes one thing about the rule: it recovers the target distribution exactly
(Section "Autoregressive vs Speculative Sampling").  That is checked here without reusing
the oracle's code: (i) as a closed-form identity in exact rationals, (ii) by pushing a full
grid of uniforms through the oracle's real ``accept_resample`` and counting, (iii) for K=2
with prefix-dependent table "models", as a joint distribution.  Plus the special cases and
the sampler's tie rules.
"""
from fractions import Fraction
from itertools import product

import numpy as np
import pytest

from oracle import sampling as S
from paper_2311_04951_b200 import synth


def _dist(rng, V, zeros=0):
    w = rng.integers(1, 64, V)
    for z in rng.choice(V, zeros, replace=False):
        w[z] = 0
    return w / w.sum(), [Fraction(int(x), int(w.sum())) for x in w]


def test_closed_form_identity_in_rationals():
    """sum_x~ q(x~) min(1, p/q)[x~ = x] + (1 - sum_z min(p_z, q_z)) * max(0, p_x - q_x) / sum max(0, p - q)
    equals p_x, for arbitrary p, q (zeros included)."""
    rng = np.random.default_rng(0)
    for V in range(2, 9):
        for zeros in (0, 1):
            _, p = _dist(rng, V, zeros)
            _, q = _dist(rng, V, zeros)
            if p == q:
                continue
            res = [max(Fraction(0), a - b) for a, b in zip(p, q)]
            rs = sum(res)
            beta = sum(min(a, b) for a, b in zip(p, q))
            for x in range(V):
                acc = min(p[x], q[x])          # q(x) * min(1, p(x)/q(x))
                assert acc + (1 - beta) * res[x] / rs == p[x]


def test_softmax_rows_and_temperature():
    row = np.array([1.0, 2.0, 3.0, 3.0], np.float32)
    p = S.softmax_t(row, 1.0)
    assert p.dtype == np.float32 and abs(p.sum() - 1) < 1e-6
    np.testing.assert_allclose(p[1] / p[0], np.e, rtol=1e-6)
    p2 = S.softmax_t(row, 0.5)                         # T halves -> log-ratios double
    np.testing.assert_allclose(p2[1] / p2[0], np.e ** 2, rtol=1e-6)
    g = S.softmax_t(row, 0.0)                          # greedy: one-hot, lowest index on ties
    assert g.tolist() == [0, 0, 1, 0]
    big = S.softmax_t(np.array([1000.0, 1001.0], np.float32), 1.0)  # max-subtracted: no overflow
    np.testing.assert_allclose(big[1] / big[0], np.e, rtol=1e-6)


def test_inv_cdf_boundaries_and_zero_weights():
    w = np.array([0.0, 0.25, 0.0, 0.5, 0.25, 0.0], np.float32)
    assert S.inv_cdf(w, 0.0) == 1                      # zero-weight index 0 is never chosen
    assert S.inv_cdf(w, 0.2499) == 1
    assert S.inv_cdf(w, 0.25) == 3                     # strict: c_1 = 0.25 is not > 0.25
    assert S.inv_cdf(w, 0.75) == 4
    assert S.inv_cdf(w, 0.999999) == 4                 # trailing zero weight never chosen
    assert S.inv_cdf(w * 8, 0.5) == 3                  # unnormalised weights
    # frequencies on a uniform grid reproduce the weights
    G = 4096
    cnt = np.bincount([S.inv_cdf(w, (k + 0.5) / G) for k in range(G)], minlength=6) / G
    np.testing.assert_allclose(cnt, w, atol=1.5 / G)


def _cell_mid(k, G):
    return np.float32((k + 0.5) / G)


GRID = 1 << 24          # uniforms live on k * 2^-24


def _measure_true(f):
    """f(u) is True on [0, t) and False on [t, 1) over the uniform grid: returns t by bisection,
    treating f (the oracle) as a black box."""
    if not f(np.float32(0.0)):
        return 0.0
    lo, hi = 0, GRID            # f(lo) True, f(hi) False by convention
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if f(np.float32(mid / GRID)):
            lo = mid
        else:
            hi = mid
    return hi / GRID


def _pmf_of_monotone(fn, V):
    """fn(u) -> index, non-decreasing in u: exact pmf of fn(U), U uniform on the grid."""
    cdf = [_measure_true(lambda u, v=v: fn(u) <= v) for v in range(V)]
    return np.diff([0.0] + cdf)


def test_inverse_cdf_sampler_has_the_right_pmf():
    rng = np.random.default_rng(3)
    for zeros in (0, 2):
        w, _ = _dist(rng, 7, zeros)
        pmf = _pmf_of_monotone(lambda u: S.inv_cdf(w.astype(np.float32), u), 7)
        np.testing.assert_allclose(pmf, w, atol=2e-7)


@pytest.mark.parametrize("seed,zeros", [(1, 0), (2, 1), (3, 2), (4, 0)])
def test_single_step_emitted_distribution_is_the_target(seed, zeros):
    """K=1 through the oracle's real accept_resample, used as a black box: for every draft token
    the measure of accepting uniforms and the pmf of the resampled token are found by bisection
    on the uniform grid; the emitted-token distribution must equal the TARGET distribution p."""
    rng = np.random.default_rng(seed)
    V = 6
    pf, _ = _dist(rng, V, zeros)
    qf, _ = _dist(rng, V, zeros)
    p, q = pf.astype(np.float32), qf.astype(np.float32)
    rows = np.stack([p, np.full(V, 1.0 / V, np.float32)])
    q_pmf = _pmf_of_monotone(lambda u: S.inv_cdf(q, u), V)
    emitted = np.zeros(V)
    accept_rate = 0.0
    for x in range(V):
        if q_pmf[x] == 0:
            continue
        t = _measure_true(lambda u: S.accept_resample(rows, q[None], [x], [u], 0.5)[0] == 1)
        emitted[x] += q_pmf[x] * t
        accept_rate += q_pmf[x] * t
        if t < 1.0:
            r = _pmf_of_monotone(lambda u: S.accept_resample(rows, q[None], [x], [np.float32(0.99999994)], u)[1], V)
            emitted += q_pmf[x] * (1 - t) * r
    np.testing.assert_allclose(emitted, pf, atol=2e-6)
    # acceptance rate = sum min(p, q) = 1 - TV(p, q)
    assert abs(accept_rate - np.minimum(pf, qf).sum()) < 2e-6


def test_coarse_brute_force_grid_agrees():
    """The same statement by plain enumeration of a G^3 grid of (u_draft, u_accept, u_resample)."""
    rng = np.random.default_rng(9)
    V, G = 4, 40
    pf, _ = _dist(rng, V)
    qf, _ = _dist(rng, V)
    p, q = pf.astype(np.float32), qf.astype(np.float32)
    rows = np.stack([p, p])
    counts = np.zeros(V)
    for kd in range(G):
        x = S.inv_cdf(q, _cell_mid(kd, G))
        for ka in range(G):
            for kr in range(G):
                a, y = S.accept_resample(rows, q[None], [x], [_cell_mid(ka, G)], _cell_mid(kr, G))
                counts[x if a == 1 else y] += 1
    np.testing.assert_allclose(counts / G ** 3, pf, atol=2.5 / G)


def test_two_step_joint_distribution_is_product_of_target_conditionals():
    """K=2 with table "models" p(.|prefix), q(.|prefix).  For every draft pair the oracle's
    accept_resample is probed as a black box (bisection over each uniform); the law of the first
    two emitted tokens must be p(x1) p(x2|x1).  When iteration 1 emits a single token (a=0) the
    second token is the first token of the next iteration, whose law is p(.|y) by the single-step
    test."""
    rng = np.random.default_rng(7)
    V = 4
    f32 = lambda a: np.asarray(a, np.float32)
    p1, q1 = _dist(rng, V)[0], _dist(rng, V, 1)[0]
    p2 = {x: _dist(rng, V)[0] for x in range(V)}
    q2 = {x: _dist(rng, V)[0] for x in range(V)}
    p3 = {xy: _dist(rng, V)[0] for xy in product(range(V), repeat=2)}
    hi = np.float32(0.99999994)
    joint = np.zeros((V, V))
    for x1, x2 in product(range(V), repeat=2):
        w = q1[x1] * q2[x1][x2]
        if w == 0:
            continue
        p_rows = np.stack([f32(p1), f32(p2[x1]), f32(p3[(x1, x2)])])
        q_rows = np.stack([f32(q1), f32(q2[x1])])
        run = lambda ua1, ua2, ur: S.accept_resample(p_rows, q_rows, [x1, x2], [ua1, ua2], ur)
        t1 = _measure_true(lambda u: run(u, hi, 0.5)[0] >= 1)
        t2 = _measure_true(lambda u: run(np.float32(0.0), u, 0.5)[0] == 2) if t1 > 0 else 0.0
        # a = 0: y from the residual of row 1, then the next token ~ p2(.|y)
        if t1 < 1:
            r = _pmf_of_monotone(lambda u: run(hi, hi, u)[1], V)
            for y in range(V):
                joint[y, :] += w * (1 - t1) * r[y] * p2[y]
        # a = 1: (x1, y) with y from the residual of row 2
        if t1 > 0 and t2 < 1:
            r = _pmf_of_monotone(lambda u: run(np.float32(0.0), hi, u)[1], V)
            joint[x1, :] += w * t1 * (1 - t2) * r
        # a = 2: (x1, x2)
        joint[x1, x2] += w * t1 * t2
    ref = np.array([[p1[a] * p2[a][b] for b in range(V)] for a in range(V)])
    np.testing.assert_allclose(joint, ref, atol=3e-6)


def test_special_cases():
    rng = np.random.default_rng(5)
    V, K = 6, 3
    p = np.stack([_dist(rng, V)[0] for _ in range(K + 1)]).astype(np.float32)
    toks = [1, 4, 2]
    # q == p: always accepted whatever u in [0,1), bonus from p_{K+1}
    for u in (0.0, 0.5, 0.99999994):
        a, y = S.accept_resample(p, p[:K], toks, [u] * K, 0.3)
        assert a == K and y == S.inv_cdf(p[K], 0.3)
    # draft certain of a token the target excludes: always rejected, and y ~ p (residual = p there)
    p0 = p.copy()
    p0[0, 3] = 0
    p0[0] /= p0[0].sum()
    q = p[:K].copy()
    q[0] = 0
    q[0, 3] = 1
    a, y = S.accept_resample(p0, q, [3, 4, 2], [0.0] * K, 0.6)
    assert a == 0 and y == S.inv_cdf(p0[0], 0.6) and y != 3
    # q(x~) = 0 < p(x~): accepted even for u -> 1 (division-free test, no NaN)
    q = p[:K].copy()
    q[1, 4] = 0
    assert S.accept_resample(p, q, toks, [0.0, 0.99999994, 0.0], 0.1)[0] == 3
    # rejected although p == q numerically -> residual is all zero -> falls back to p
    a, y = S.accept_resample(p, p[:K], toks, [0.5, 1.0, 0.5], 0.42)   # u = 1.0 forces u*q < p false
    assert a == 1 and y == S.inv_cdf(p[1], 0.42)
    # the scan stops at the FIRST rejection: later tokens are not looked at
    q = p[:K].copy()
    q[0, 1] = 1.0      # p/q small -> reject with u close to 1
    a, _ = S.accept_resample(p, q, toks, [0.999, 0.0, 0.0], 0.5)
    assert a == 0


def test_greedy_reduces_to_argmax_agreement():
    rng = np.random.default_rng(11)
    V, K = 9, 4
    logits_p = rng.standard_normal((K + 1, V)).astype(np.float32)
    logits_q = rng.standard_normal((K, V)).astype(np.float32)
    p = np.stack([S.softmax_t(r, 0.0) for r in logits_p])
    q = np.stack([S.softmax_t(r, 0.0) for r in logits_q])
    best = logits_p.argmax(axis=1)
    for agree in range(K + 1):
        toks = [int(best[i]) if i < agree else int((best[i] + 1) % V) for i in range(K)]
        qq = np.zeros_like(q)
        for i, t in enumerate(toks):
            qq[i, t] = 1
        a, y = S.accept_resample(p, qq, toks, rng.random(K).astype(np.float32), np.float32(rng.random()))
        assert a == agree and y == best[agree]


# ---------------------------------------------------------------- top-k / top-p restriction
def _nucleus_by_fractions(p, top_k, top_p):
    """The definition written out with exact rationals on a tiny row (no ties allowed in the input)."""
    from fractions import Fraction
    vals = [Fraction(float(x)) for x in p]
    order = sorted(range(len(p)), key=lambda j: -vals[j])
    kept = order[:top_k] if top_k > 0 else order
    if 0 < top_p < 1:
        mass = sum(vals[j] for j in kept)
        acc, cut = Fraction(0), len(kept)
        for n, j in enumerate(kept):
            acc += vals[j]
            if acc >= Fraction(float(np.float32(top_p))) * mass:
                cut = n + 1
                break
        kept = kept[:cut]
    return sorted(kept)


def test_filter_keeps_the_definition_s_set_on_tiny_rows():
    rng = np.random.default_rng(5)
    for _ in range(300):
        V = int(rng.integers(2, 9))
        p = rng.dirichlet(np.full(V, 0.7)).astype(np.float32)
        if len(set(p.tolist())) < V:
            continue
        k = int(rng.integers(0, V + 2))
        tp = float(rng.choice([1.0, 0.3, 0.5, 0.8, 0.95]))
        out = S.filter_top_k_top_p(p, k, tp)
        kept = np.nonzero(out > 0)[0].tolist()
        assert kept == _nucleus_by_fractions(p, k, tp), (p, k, tp)
        # renormalised, ratios among the kept tokens unchanged
        assert abs(float(out.astype(np.float64).sum()) - 1.0) < 1e-6
        j0 = kept[0]
        for j in kept:
            assert abs(out[j] / out[j0] - p[j] / p[j0]) < 1e-5


def test_filter_special_cases_and_ties():
    p = np.array([0.1, 0.3, 0.05, 0.3, 0.25], np.float32)
    assert np.array_equal(S.filter_top_k_top_p(p, 0, 1.0), p)               # off: unchanged, same bits
    assert np.array_equal(S.filter_top_k_top_p(p, 9, 1.0), p)               # k >= V: nothing cut
    one = S.filter_top_k_top_p(np.array([0.2, 0.5, 0.3], np.float32), 1, 1.0)
    assert one.tolist() == [0.0, 1.0, 0.0]                                       # top-1 = one-hot at the argmax
    tie = S.filter_top_k_top_p(p, 1, 1.0)                                    # the two 0.3 tie at the threshold: both kept
    assert np.nonzero(tie)[0].tolist() == [1, 3] and tie[1] == tie[3] == np.float32(0.5)
    nuc = S.filter_top_k_top_p(p, 0, 0.61)                                   # 0.3 + 0.3 = 0.6 < 0.61: a third token is needed
    assert np.nonzero(nuc)[0].tolist() == [1, 3, 4]
    edge = S.filter_top_k_top_p(p, 0, 0.6)                                   # reaching the target exactly is enough
    assert np.nonzero(edge)[0].tolist() == [1, 3] or np.nonzero(edge)[0].tolist() == [1, 3, 4]   # (0.3 + 0.3 in fp32 vs 0.6)
    both = S.filter_top_k_top_p(p, 3, 0.5)                                   # top-p acts on what top-k kept: 0.5 * 0.85
    assert np.nonzero(both)[0].tolist() == [1, 3]


def test_filter_minimality_and_mass_on_large_rows():
    """V = 32000 Dirichlet rows: the kept set is a threshold set, its mass reaches the target, and without its
    smallest member it would not (no ties at the threshold in these rows)."""
    rows = synth.gen_dirichlet_rows(17, 3, 32000, alpha=0.3)
    for p in rows:
        for k, tp in ((50, 1.0), (0, 0.9), (200, 0.5)):
            out = S.filter_top_k_top_p(p, k, tp)
            kept = out > 0
            assert p[kept].min() > p[~kept].max()
            if k:
                assert kept.sum() <= k
            if tp < 1:
                base = np.sort(p)[::-1][:k].astype(np.float64).sum() if k else p.astype(np.float64).sum()
                m = p[kept].astype(np.float64).sum()
                assert m >= tp * base * (1 - 1e-12)
                assert m - float(p[kept].min()) < tp * base


def test_speculative_rule_preserves_the_restricted_target():
    """The accept / resample identity with both rows restricted: sum over draft tokens of
    q'(x) min(1, p'(x)/q'(x)) [x = y] + P(reject) r'(y) = p'(y), in exact rationals."""
    from fractions import Fraction
    rng = np.random.default_rng(9)
    for _ in range(50):
        V = 7
        p = S.filter_top_k_top_p(rng.dirichlet(np.ones(V)).astype(np.float32), 4, 0.9)
        q = S.filter_top_k_top_p(rng.dirichlet(np.ones(V)).astype(np.float32), 4, 0.9)
        P = [Fraction(float(x)) for x in p]
        Q = [Fraction(float(x)) for x in q]
        sp, sq = sum(P), sum(Q)
        P = [x / sp for x in P]
        Q = [x / sq for x in Q]
        acc = [min(P[j], Q[j]) for j in range(V)]
        rej = 1 - sum(acc)
        res = [max(Fraction(0), P[j] - Q[j]) for j in range(V)]
        sr = sum(res)
        for y in range(V):
            total = acc[y] + (rej * res[y] / sr if sr else 0)
            assert total == P[y]
            if P[y] == 0:
                assert total == 0        # a token outside the restricted target is never emitted
