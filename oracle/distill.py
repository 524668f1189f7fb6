"""CPU oracle of the hybrid cross-vocabulary distillation loss (Section 3.2, Eq. (3))
and of its gradient with respect to the drafter's logits.

TEST INFRASTRUCTURE ONLY; fp64 numpy, written from the formulas, shares nothing with
the CUDA library.

Per proposed draft position j of a sequence (drafter distribution q_j = softmax(z_j)):
  * j is a directly mapped token (its piece of the translated proposal has one
    sub-token, target position i):           L_j = KL(q'_j || p_i)
        = sum over draft ids d with a direct map of q_j(d) * (ln q_j(d) - ln p_i(map[d]))
    q' is q carried through the map (Eq. (1), not renormalised; terms with q = 0 are 0);
  * j is a sub-token of a cached n-gram:      L_j = -lambda_j * ln q_j(d_j)
    with lambda_j = lambda (hyper-parameter), or the verified target probability
    p_i(t_i) of the n-gram (the "dynamic weight" the section mentions);
  * j was not translated (at or after an unmapped stop, or beyond K_b): L_j = 0.
p_i = softmax(target logits row i / T).

Gradients with respect to z_j (q_j = softmax(z_j); if the drafter samples at a
temperature, z_j stands for its logits divided by it):
  KL term:   g(d) = [d mapped] * (ln q(d) - ln p(map[d]) + 1),  dL/dz(d) = q(d) * (g(d) - sum_e q(e) g(e))
  NLL term:  dL/dz(d) = lambda_j * (q(d) - [d == d_j])

Readings: the masks I_DM / I_N-gram follow the pieces of the translation (Eq. (1));
every sub-token of a merged run gets the NLL term, whether or not the target accepted
the n-gram (the loss is applied to the drafter's own proposals, "on-policy"); the mean
over positions / the batch is left to the caller.

Pins (tests/test_oracle_distill.py): torch's kl_div and autograd on an identity map;
central finite differences of the loss through softmax; KL >= 0 and = 0 iff q = p on a
full map; the NLL gradient sums to zero; the mapped-mass identity of the KL gradient.
"""
from __future__ import annotations

import numpy as np

LAMBDA_CONSTANT, LAMBDA_TARGET_PROB = 0, 1


def log_softmax_row(x: np.ndarray, T: float) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64) / T
    m = x.max()
    return x - m - np.log(np.exp(x - m).sum())


def position_kl(q: np.ndarray, log_p: np.ndarray, vocab_map: np.ndarray):
    """KL(q' || p) over the mapped ids and its gradient w.r.t. the drafter's logits."""
    q = np.asarray(q, dtype=np.float64)
    mapped = vocab_map >= 0
    g = np.zeros_like(q)
    pos = mapped & (q > 0)
    f = np.zeros_like(q)
    f[pos] = np.log(q[pos]) - log_p[vocab_map[pos]]
    loss = float((q * f).sum())
    g[pos] = f[pos] + 1.0
    # ids with q = 0 carry no mass and no gradient (q * anything = 0)
    grad = q * (g - float((q * g).sum()))
    return loss, grad


def position_nll(q: np.ndarray, d: int, lam: float):
    q = np.asarray(q, dtype=np.float64)
    loss = -lam * float(np.log(q[d])) if q[d] > 0 else float("inf")
    grad = lam * q.copy()
    grad[d] -= lam
    return loss, grad


def distill_sequence(q_rows, draft_ids, span_start, span_len, m, logits_rows, T, vocab_map, tgt_ids,
                     lam: float, lambda_mode: int = LAMBDA_CONSTANT):
    """One sequence: q_rows [K, V_q], logits_rows [K+1, V_p] (float64 values of the
    target logits), pieces from the translation.  Returns (loss [K], grad [K, V_q])."""
    K, V_q = q_rows.shape
    loss = np.zeros(K)
    grad = np.zeros((K, V_q))
    for i in range(int(m)):
        log_p = log_softmax_row(logits_rows[i], T)
        s0, L = int(span_start[i]), int(span_len[i])
        if L == 1:
            loss[s0], grad[s0] = position_kl(q_rows[s0], log_p, vocab_map)
        else:
            w = lam if lambda_mode == LAMBDA_CONSTANT else float(np.exp(log_p[int(tgt_ids[i])]))
            for j in range(s0, s0 + L):
                loss[j], grad[j] = position_nll(q_rows[j], int(draft_ids[j]), w)
    return loss, grad
