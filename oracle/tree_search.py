"""Oracle for the test-time tree search (paper Section 4.2): the UCB rule of Eq. 1 and the reward of Eq. 2, written
out in plain Python floats (fp64), one line per term, in the paper's notation.

TEST INFRASTRUCTURE ONLY, like the rest of ``oracle/``: nothing in the product package imports it.

Readings where the paper is garbled or silent: r_hat_k is the running MEAN of arm k's rewards (the text says "mean"
but prints a bare sum); the reward is the NEGATIVE inverse speed-up, maximised (Eq. 2; Appendix A.4 writes the same
quantity with the opposite sign and says "minimize"); an arm that was never played is tried first, lowest index
first, which is what an unbounded exploration term means; ties go to the lowest index; t counts rounds from 1.

Pins (tests/test_tree_search.py): the reward against the speed-up formula of Appendix A.4 evaluated from its
timing model; hand-worked rounds; the limits lambda_UCB = 0 (greedy on the mean) and lambda_UCB -> large (round
robin); invariance of the choice under a common shift of all means.
"""

from __future__ import annotations

import math
from typing import List, Sequence


def reward(lambda_gamma: float, gamma: int, n_accept: int) -> float:
    """Eq. 2 for the arm that was selected (indicator I = 1)."""
    return -(1.0 / n_accept + lambda_gamma * gamma / n_accept)


def select(r_sum: Sequence[float], n: Sequence[int], t: int, lambda_ucb: float) -> int:
    """Eq. 1 at round t (1-based)."""
    K = len(n)
    for k in range(K):
        if n[k] == 0:
            return k
    best, best_score = 0, None
    for k in range(K):
        r_hat = r_sum[k] / n[k]
        score = r_hat + lambda_ucb * math.sqrt(2.0 * math.log(t) / n[k])
        if best_score is None or score > best_score:
            best, best_score = k, score
    return best


class Bandit:
    def __init__(self, K: int, lambda_ucb: float, lambda_gamma: float):
        self.r_sum: List[float] = [0.0] * K
        self.n: List[int] = [0] * K
        self.rounds = 0
        self.lambda_ucb, self.lambda_gamma = lambda_ucb, lambda_gamma

    def select(self) -> int:
        return select(self.r_sum, self.n, self.rounds + 1, self.lambda_ucb)

    def update(self, k: int, gamma: int, n_accept: int) -> None:
        self.r_sum[k] += reward(self.lambda_gamma, gamma, n_accept)
        self.n[k] += 1
        self.rounds += 1
