"""Seeded sampling of the next token: an exact draw from softmax(logits / T) by Gumbel-max.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

Training rollouts use temperature 1.0 and top_p = 1.0 (Section 4.2, "Training
Details"), i.e. the full categorical distribution.  argmax_v(logit_v / T + g_v)
with independent standard Gumbel g_v is such a draw, and makes the draw a pure
function of (seed, prompt, rollout, step), so a rollout does not depend on which
other rollouts share its batch.
"""
from __future__ import annotations

import numpy as np

from . import philox


def sample(logits: np.ndarray, temperature: float, seed: int, prompt: int, rollout: int, step: int):
    """Returns (token, gap): the arg-max of the perturbed scores (lowest id on an exact tie)
    and the difference between the largest and second-largest perturbed score."""
    logits = np.asarray(logits, dtype=np.float64)
    g = philox.gumbel_noise(logits.shape[0], seed, prompt, rollout, step)
    score = logits / float(temperature) + g
    tok = int(np.argmax(score))                 # numpy returns the first maximum
    if score.shape[0] > 1:
        top2 = np.partition(score, -2)[-2:]
        gap = float(top2[1] - top2[0])
    else:
        gap = float("inf")
    return tok, gap
