"""Test-time tree search (paper Section 4.2): the oracle against facts fixed outside it, then the library's host
code against the oracle, decision by decision and bit for bit."""

import math

import numpy as np
import pytest

from oracle import tree_search as ots

PAPER_TREES = [(3, 3, 2, 1), (3, 2, 2, 1, 1), (2, 2, 2, 1, 1, 1)]   # the candidate set of the paper's Table 5 / Table 6


# ------------------------------------------------------------------ pins of the oracle
def test_reward_is_the_negative_inverse_speedup_of_the_appendix():
    """Appendix A.4: T_total = T_target(gamma) + gamma T_draft; per accepted token T_avg = T_total / N_accept;
    speed-up = T_target / T_avg.  With T_target(gamma) = T_target and T_draft / T_target = lambda_gamma the reward of
    Eq. 2 is -1 / speed-up.  The expected value below is computed from that timing model, not from Eq. 2."""
    for T_target, lam, gamma, n_acc in [(30.0, 0.1, 5, 3), (12.5, 0.04, 4, 1), (7.0, 0.25, 6, 6)]:
        T_draft = lam * T_target
        T_total = T_target + gamma * T_draft
        speedup = T_target / (T_total / n_acc)
        assert math.isclose(ots.reward(lam, gamma, n_acc), -1.0 / speedup, rel_tol=1e-15)
    # worked by hand: lambda = 0.1, gamma = 5, 3 accepted tokens -> -(1/3 + 0.5/3) = -0.5
    assert ots.reward(0.1, 5, 3) == pytest.approx(-0.5, abs=1e-16)
    # more accepted tokens is better, a longer draft for the same acceptance is worse
    assert ots.reward(0.1, 5, 4) > ots.reward(0.1, 5, 3) > ots.reward(0.1, 6, 3)


def test_hand_worked_rounds():
    b = ots.Bandit(2, lambda_ucb=1.0, lambda_gamma=0.0)
    assert b.select() == 0; b.update(0, 4, 2)          # r = -0.5
    assert b.select() == 1; b.update(1, 4, 4)          # r = -0.25
    # round 3: arm 0: -0.5 + sqrt(2 ln 3 / 1) = 0.98230..., arm 1: -0.25 + 1.48230... -> arm 1
    bonus = math.sqrt(2 * math.log(3))
    assert bonus == pytest.approx(1.4823038073675112, abs=1e-15)
    assert b.select() == 1; b.update(1, 4, 1)          # r = -1 -> mean of arm 1 = -0.625
    # round 4: arm 0: -0.5 + sqrt(2 ln 4) = 1.16511, arm 1: -0.625 + sqrt(ln 4) = 0.55241 -> arm 0
    assert -0.5 + math.sqrt(2 * math.log(4)) > -0.625 + math.sqrt(2 * math.log(4) / 2)
    assert b.select() == 0
    assert b.r_sum == [-0.5, -1.25] and b.n == [1, 2] and b.rounds == 3


def test_limits_and_invariances():
    g = np.random.default_rng(0)
    # lambda_UCB = 0: after one pull each, always the arm with the best mean
    b = ots.Bandit(3, 0.0, 0.1)
    for k, acc in enumerate((2, 5, 3)):
        assert b.select() == k
        b.update(k, 5, acc)
    for _ in range(5):
        assert b.select() == 1
        b.update(1, 5, 5)
    # a huge exploration weight: the least-played arm is always next (round robin)
    b = ots.Bandit(3, 1e9, 0.1)
    picks = []
    for _ in range(9):
        k = b.select(); picks.append(k); b.update(k, 5, int(g.integers(1, 6)))
    assert picks == [0, 1, 2] * 3
    # adding the same constant to every arm's mean changes no decision
    r_sum, n = [-1.3, -0.7, -2.0], [3, 2, 4]
    shifted = [s + 10.0 * c for s, c in zip(r_sum, n)]
    for t in (10, 11, 50):
        assert ots.select(r_sum, n, t, 0.7) == ots.select(shifted, n, t, 0.7)


# ------------------------------------------------------------------ the library's host code against the oracle
@pytest.fixture(scope="module")
def md():
    from paper_2506_01206_b200.build import build_library
    build_library()
    import paper_2506_01206_b200 as m
    m.load_library()
    return m


@pytest.mark.parametrize("lam_ucb,lam_gamma,seed", [(1.0, 0.1, 0), (0.3, 0.04, 1), (0.0, 0.2, 2), (2.5, 0.0, 3)])
def test_library_follows_the_oracle_decision_by_decision(md, lam_ucb, lam_gamma, seed):
    g = np.random.default_rng(seed)
    K = len(PAPER_TREES)
    lib, ora = md.UcbBandit(K, lam_ucb, lam_gamma), ots.Bandit(K, lam_ucb, lam_gamma)
    accept_p = g.uniform(0.4, 0.9, K)     # a synthetic verifier: per-arm chance that each further level is accepted
    for _ in range(300):
        k = lib.mdraft_ucb_select()
        assert k == ora.select()
        gamma = len(PAPER_TREES[k])
        n_acc = 1
        while n_acc <= gamma and g.random() < accept_p[k]:
            n_acc += 1
        lib.mdraft_ucb_update(k, gamma, n_acc)
        ora.update(k, gamma, n_acc)
        assert lib.reward_sum == ora.r_sum and lib.count == ora.n and lib.round == ora.rounds   # bit for bit
        assert md.mdraft_ucb_reward(lam_gamma, gamma, n_acc) == ots.reward(lam_gamma, gamma, n_acc)


def test_library_rejects_bad_arguments(md):
    b = md.UcbBandit(2, 1.0, 0.1)
    for args in ((2, 4, 1), (-1, 4, 1), (0, 0, 1), (0, 4, 0)):
        with pytest.raises(md.MdraftError):
            b.mdraft_ucb_update(*args)
    assert b.round == 0 and b.count == [0, 0]
