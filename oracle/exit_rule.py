"""CPU oracle of the adaptive-drafting exit rule (Section 3.3, Eq. (4)-(6)).

TEST INFRASTRUCTURE ONLY: imported by the tests; shares nothing with the CUDA
library.  Plain fp64 loops in the paper's order:

    P(y_i accepted | y_<i accepted) = sigmoid(f_phi(e_i))                  Eq. (4)
    P(some y_i, i <= k, rejected)   = 1 - prod_{i <= k} sigmoid(f_i)       Eq. (5)
    exit as soon as that probability exceeds gamma                         Eq. (6)

Readings where the paper is silent: the test is made after each proposed token,
in order, and is strict (>); the token whose test fires is still part of the
proposal (the drafter has produced it when its acceptance is predicted), so the
draft length is the first k with 1 - prod_{i<=k} sigma(f_i) > gamma, and K
(the number of head outputs given) when the test never fires.  A proposal of
zero tokens stays empty.

Pins (tests/test_oracle_exit_rule.py): constant head outputs give the geometric
closed form k = floor(log(1 - gamma) / log(sigma)) + 1; large positive outputs
never exit; the length is non-decreasing in gamma and in every head output; the product is compared against math.prod on small cases.
"""
from __future__ import annotations

import math

import numpy as np


def sigmoid(x: float) -> float:
    # the two branches avoid overflow of exp for large |x|
    if x >= 0.0:
        return 1.0 / (1.0 + math.exp(-x))
    e = math.exp(x)
    return e / (1.0 + e)


def exit_rule(head_logits, avail_len, gamma: float):
    """head_logits: [B, K] outputs f_phi(e_i) of the acceptance head; avail_len: [B]
    tokens available per sequence (<= K).  Returns (draft_len int32 [B],
    reject_prob float64 [B, K]: Eq. (5) after each token; entries at and beyond
    avail_len are 0)."""
    f = np.asarray(head_logits, dtype=np.float64)
    B, K = f.shape
    avail = np.asarray(avail_len, dtype=np.int64)
    draft_len = np.zeros(B, dtype=np.int32)
    reject = np.zeros((B, K), dtype=np.float64)
    for b in range(B):
        n = int(min(max(avail[b], 0), K))
        keep = 1.0                      # running product of Eq. (5)
        length = n
        fired = False
        for i in range(n):
            keep *= sigmoid(float(f[b, i]))
            reject[b, i] = 1.0 - keep
            if not fired and reject[b, i] > gamma:
                length = i + 1
                fired = True
        draft_len[b] = length
    return draft_len, reject
