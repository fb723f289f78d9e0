"""Host logic of the adaptive choice of K (no GPU): the closed form for tokens per iteration and the policy."""
import itertools

import numpy as np

from paper_2311_04951_b200.engine import AdaptiveK, expected_tokens


def test_expected_tokens_is_the_mean_of_the_emission_count():
    """With independent acceptance alpha the iteration emits a + 1 tokens, a = accepted prefix length (at most
    k): the closed form equals the enumeration of all accept / refuse patterns."""
    for alpha in (0.0, 0.2, 0.5, 0.9):
        for k in (1, 2, 5):
            mean = 0.0
            for pat in itertools.product([0, 1], repeat=k):
                prob = np.prod([alpha if b else 1 - alpha for b in pat])
                a = next((i for i, b in enumerate(pat) if not b), k)
                mean += prob * (a + 1)
            assert abs(mean - expected_tokens(alpha, k)) < 1e-12
    assert expected_tokens(1.0, 4) == 5.0


def test_policy_picks_the_best_k_and_moves_with_the_acceptance_rate():
    pol = AdaptiveK(k_max=8, cost=0.1, forget=1.0, alpha0=0.5)
    best = max(range(1, 9), key=lambda k: expected_tokens(0.5, k) / (1 + 0.1 * k))
    assert pol.choose() == best
    for _ in range(50):                       # every draft accepted: the longest draft pays
        pol.update([pol.choose()], pol.choose())
    assert pol.alpha > 0.95 and pol.choose() == 8
    low = AdaptiveK(k_max=8, cost=0.1, forget=0.5)
    for _ in range(20):                       # every first draft refused
        low.update([0, 0], low.choose())
    assert low.alpha < 0.01 and low.choose() == 1
    assert AdaptiveK(k_max=8, cost=100.0).choose() == 1        # drafting as dear as verifying: shortest draft
    assert AdaptiveK(k_max=8, cost=0.0, alpha0=0.3).choose() == 8   # free drafts: longest draft


def test_policy_counts_the_tests_up_to_the_first_refusal():
    pol = AdaptiveK(k_max=4, cost=0.2, forget=1.0, alpha0=0.0)
    pol.acc, pol.tested = 0.0, 0.0
    pol.update([2, 4, 0], 4)                  # 3 tests (2 accepted), 4 tests (4 accepted), 1 test (0 accepted)
    assert pol.acc == 6 and pol.tested == 8 and abs(pol.alpha - 0.75) < 1e-12
