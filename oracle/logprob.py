"""Behaviour log-probability of a sampled token: log pi_theta_old(o_t | q, o_<t), the denominator of the token
importance ratio of Eq. 2.  TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

With sampling temperature T the behaviour policy is softmax(logits / T), so
    log pi(o_t) = logits[o_t] / T - log sum_v exp(logits[v] / T).
Pins: torch.log_softmax, normalisation, shift invariance, the uniform case -log V (tests/test_oracle_logprob.py).
"""
from __future__ import annotations

import numpy as np


def token_logprob(logits: np.ndarray, token: int, temperature: float = 1.0) -> float:
    x = np.asarray(logits, dtype=np.float64) / float(temperature)
    m = np.max(x)
    return float(x[int(token)] - m - np.log(np.sum(np.exp(x - m))))
