"""Group statistics, pilot estimate, pilot filter / eviction / commit allocation, advantages.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

  group mean and standard deviation            Eq. 3 (population form: divide by G)
  advantage  A_i = (r_i - mu) / sigma          Section 3.1, text after Eq. 3
  pilot estimate  p_hat = (1/n_pilot) sum r_j  Section 3.3, "Pilot stage"
  filter  p_lower <= p_hat <= p_upper          Section 3.3 and Algorithm 1 (Filter)
  evict   p_hat >= p_solve                     Section 3.4 and Algorithm 1 (Evict solved prompts)
  commit  n_commit more rollouts for kept prompts, at most b_t prompts
                                               Section 3.3, "Commit stage"; Algorithm 1 (Commit)
  cost    b_g * n_pilot + b_t * n_commit       Section 4.3

Readings where the paper is silent:
  * sigma = 0 (all rewards of the group equal): the advantage is 0 -- the introduction
    says such prompts "produce zero advantage".  No epsilon is added otherwise.
  * p_hat is the IEEE double quotient m / n and the three comparisons are done in
    double, as a plain implementation of the formulas would do.
  * A prompt can both pass the filter and be evicted (when p_solve <= p_upper):
    Algorithm 1 applies the two rules independently, so eviction is a separate flag.
  * When more than b_t prompts pass the filter, the first b_t in batch order commit
    and the rest are handed to the replay buffer (status BUFFERED).  Algorithm 1 only
    says "sample prompt q from R"; any choice of b_t survivors is valid.
"""
from __future__ import annotations

import numpy as np

COMMIT, BUFFERED, DEFER_HARD, SKIP_EASY, LOW_VARIANCE = 0, 1, 2, 3, 4


def group_stats(rewards: np.ndarray, start: np.ndarray, count: np.ndarray):
    """Per group g = rewards[start[g] : start[g] + count[g]]: n, number of rewards equal to 1, mean,
    population variance."""
    P = len(start)
    n = np.zeros(P, dtype=np.int32)
    m = np.zeros(P, dtype=np.int32)
    mean = np.zeros(P, dtype=np.float64)
    var = np.zeros(P, dtype=np.float64)
    for g in range(P):
        r = np.asarray(rewards[start[g]:start[g] + count[g]], dtype=np.float64)
        n[g] = r.shape[0]
        m[g] = int(np.sum(r == 1.0))
        if n[g] > 0:
            mu = np.sum(r) / n[g]
            mean[g] = mu
            var[g] = np.sum((r - mu) ** 2) / n[g]
    return n, m, mean, var


def allocate(pilot_success, pilot_n, p_lower: float, p_upper: float, p_solve: float, n_commit: int, b_t: int):
    """Pilot filter, eviction and commit allocation for one sampling batch.

    Returns status [P], extra_rollouts [P], evict [P], n_selected, total_rollouts
    where total_rollouts = sum(pilot_n) + n_selected * n_commit.
    """
    P = len(pilot_success)
    status = np.zeros(P, dtype=np.int32)
    extra = np.zeros(P, dtype=np.int32)
    evict = np.zeros(P, dtype=np.int32)
    selected = 0
    for p in range(P):
        if pilot_n[p] <= 0:
            raise ValueError("every prompt of the sampling batch needs at least one pilot rollout")
        p_hat = float(pilot_success[p]) / float(pilot_n[p])
        evict[p] = 1 if p_hat >= p_solve else 0
        if p_lower <= p_hat <= p_upper:
            if selected < b_t:
                status[p] = COMMIT
                extra[p] = n_commit
                selected += 1
            else:
                status[p] = BUFFERED
        elif p_hat < p_lower:
            status[p] = DEFER_HARD
        else:
            status[p] = SKIP_EASY
    total = int(np.sum(np.asarray(pilot_n, dtype=np.int64))) + selected * int(n_commit)
    return status, extra, evict, selected, total


def grpo_advantage(rewards: np.ndarray, start: np.ndarray, count: np.ndarray, status=None) -> np.ndarray:
    """A_i = (r_i - mu) / sigma within each group rewards[start[g] : start[g] + count[g]]; 0 for a
    group whose rewards are all equal, for groups whose status is given and is not COMMIT, and for
    every element outside the groups."""
    rewards = np.asarray(rewards, dtype=np.float64)
    adv = np.zeros(rewards.shape[0], dtype=np.float64)
    for g in range(len(start)):
        if status is not None and status[g] != COMMIT:
            continue
        r = rewards[start[g]:start[g] + count[g]]
        if r.shape[0] == 0 or np.max(r) == np.min(r):
            continue
        mu = np.sum(r) / r.shape[0]
        sigma = np.sqrt(np.sum((r - mu) ** 2) / r.shape[0])
        adv[start[g]:start[g] + count[g]] = (r - mu) / sigma
    return adv


def sampling_cost(method: str, b_t: int, s: int, n_pilot: int, n_commit: int) -> int:
    """Rollouts generated per training step (Section 4.3): GRPO b_t n, DAPO b_g n, PC b_g n_pilot + b_t n_commit."""
    n = n_pilot + n_commit
    b_g = s * b_t
    if method == "grpo":
        return b_t * n
    if method == "dapo":
        return b_g * n
    if method == "pc":
        return b_g * n_pilot + b_t * n_commit
    raise ValueError(method)


def dapo_filter(rewards: np.ndarray, start: np.ndarray, count: np.ndarray) -> np.ndarray:
    """The baseline filter of Section 4.3 (DAPO): every prompt of the oversampled batch gets the full budget n and
    prompts whose rewards are all correct or all incorrect are dropped.  Returns keep[g] in {0, 1}."""
    keep = np.zeros(len(start), dtype=np.int32)
    for g in range(len(start)):
        r = np.asarray(rewards[start[g]:start[g] + count[g]], dtype=np.float64)
        keep[g] = 1 if r.shape[0] > 0 and np.max(r) != np.min(r) else 0
    return keep


def allocate_by_variance(pilot_var, pilot_n, var_min: float, n_commit: int, b_t: int):
    """The pilot filter for general scalar rewards.  Section 3.3 argues from reward variance (Var = p (1 - p) for binary
    rewards, p_hat being its proxy) and says the method applies to any scalar reward signal, without a formula for that
    case.  Reading: keep iff the population variance of the pilot rewards (Eq. 3) is at least var_min; the variance is
    taken in single precision, the precision in which the statistics are reported, and compared in double.  The first
    b_t kept prompts in batch order commit, later ones are BUFFERED, the others LOW_VARIANCE.
    Returns status, extra_rollouts, n_selected, total_rollouts."""
    P = len(pilot_var)
    status = np.zeros(P, dtype=np.int32)
    extra = np.zeros(P, dtype=np.int32)
    selected = 0
    for p in range(P):
        if pilot_n[p] > 0 and float(np.float32(pilot_var[p])) >= var_min:
            if selected < b_t:
                status[p], extra[p] = COMMIT, n_commit
                selected += 1
            else:
                status[p] = BUFFERED
        else:
            status[p] = LOW_VARIANCE
    total = int(np.sum(np.asarray(pilot_n, dtype=np.int64))) + selected * int(n_commit)
    return status, extra, selected, total
