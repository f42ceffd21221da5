"""Pins for oracle/logprob.py (the behaviour log-probability that Eq. 2 divides by)."""
import math

import numpy as np
import pytest
import torch

from oracle.logprob import token_logprob


def test_matches_library_log_softmax():
    rng = np.random.default_rng(0)
    for T in (1.0, 0.7):
        x = rng.normal(size=1000) * 5
        ref = torch.log_softmax(torch.from_numpy(x) / T, dim=0).numpy()
        for tok in (0, 17, 999):
            assert token_logprob(x, tok, T) == pytest.approx(ref[tok], abs=1e-12)


def test_normalised_shift_invariant_and_uniform():
    rng = np.random.default_rng(1)
    x = rng.normal(size=64) * 3
    assert sum(math.exp(token_logprob(x, v)) for v in range(64)) == pytest.approx(1.0, abs=1e-12)
    assert token_logprob(x + 123.0, 5) == pytest.approx(token_logprob(x, 5), abs=1e-9)
    assert token_logprob(np.zeros(4096), 7) == pytest.approx(-math.log(4096), abs=1e-12)
    assert token_logprob(np.array([1e4, 0.0]), 0) == pytest.approx(0.0, abs=1e-12)      # no overflow
