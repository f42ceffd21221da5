"""One Pilot-Commit step over a sampling batch: pilot rollouts, allocation, commit rollouts,
union statistics and advantages (Section 3.3; Algorithm 1, the Pilot / Filter / Evict /
Commit / Train-on-union lines for a single step).

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

A rollout (p, i) is generated token by token: generated token 0 is sampled from the
logits at the prompt's last position, token s >= 1 from the logits after feeding
token s-1.  It ends when it has `cap[p, i]` tokens (the synthetic workloads have no
end-of-sequence token).  Its reward is 1 iff its last token id is below the prompt's
threshold (the stand-in for the paper's binary verifier R(q, o) in {0, 1}).
"""
from __future__ import annotations

from typing import Dict, List, Sequence

import numpy as np

from . import sampler, stats
from .decoder import Decoder


def generate_group(dec: Decoder, prompt_tokens, prompt_index: int, rollouts: Sequence[int], caps: Sequence[int],
                   seed: int, temperature: float, prefilled=None, shared_prefix: bool = False,
                   record_logits: bool = False):
    """Rollouts `rollouts` (indices within the group) of one prompt, decoded in lock step.

    Returns {rollout: tokens [cap]} (and, with record_logits, {rollout: [logits per generated token]}).
    `prefilled` = (prompt_kv, last_logits) reuses an earlier prefill of the same prompt:
    the prompt is evaluated once and shared by the pilot and the commit rollouts.
    """
    Lp = len(prompt_tokens)
    prompt_kv, last_logits = prefilled if prefilled is not None else dec.prefill(prompt_tokens)
    toks: Dict[int, List[int]] = {}
    logs: Dict[int, list] = {}
    suffix = {}
    cap = {i: int(c) for i, c in zip(rollouts, caps)}
    for i in rollouts:
        t, _ = sampler.sample(last_logits, temperature, seed, prompt_index, i, 0)
        toks[i] = [t]
        logs[i] = [np.array(last_logits)]
        suffix[i] = dec.empty_suffix()
    s = 0                                   # number of suffix tokens already cached
    while True:
        live = [i for i in rollouts if cap[i] > s + 1]
        if not live:
            break
        x = np.array([toks[i][s] for i in live])
        pos = np.full(len(live), Lp + s)
        kv_list = [suffix[i] for i in live]
        logits = dec.decode(x, pos, prompt_kv, kv_list, shared_prefix=shared_prefix)
        for r, i in enumerate(live):
            t, _ = sampler.sample(logits[r], temperature, seed, prompt_index, i, s + 1)
            toks[i].append(t)
            if record_logits:
                logs[i].append(np.array(logits[r]))
        s += 1
    out = {i: np.array(toks[i], dtype=np.int32) for i in rollouts}
    return (out, logs) if record_logits else out


def reward(tokens: np.ndarray, threshold: int) -> float:
    return 1.0 if int(tokens[-1]) < int(threshold) else 0.0


def pilot_commit_step(dec: Decoder, wl, batch, b_t=None, shared_prefix: bool = False):
    """Runs the whole step on the CPU.  Returns a dict of every output the GPU path also produces."""
    P, G, k = wl.n_prompts, wl.group_size, wl.n_pilot
    b_t = P if b_t is None else b_t
    tokens = [[None] * G for _ in range(P)]
    rewards = np.zeros((P, G), dtype=np.float64)
    generated = np.zeros((P, G), dtype=bool)
    prefilled = []
    for p in range(P):
        pt = batch.prompt_tokens[batch.prompt_offsets[p]:batch.prompt_offsets[p + 1]]
        pf = dec.prefill(pt)
        prefilled.append(pf)
        out = generate_group(dec, pt, p, list(range(k)), batch.caps[p, :k], wl.sample_seed, wl.temperature,
                             prefilled=pf, shared_prefix=shared_prefix)
        for i in range(k):
            tokens[p][i] = out[i]
            rewards[p, i] = reward(out[i], batch.reward_threshold[p])
            generated[p, i] = True
    start = np.arange(P) * G                 # rewards are laid out [P, G]; a group is its generated prefix
    pn, pm, pmean, pvar = stats.group_stats(rewards.reshape(-1), start, np.full(P, k))
    status, extra, evict, n_sel, total = stats.allocate(pm, pn, wl.p_lower, wl.p_upper, wl.p_solve, G - k, b_t)
    for p in range(P):
        if status[p] != stats.COMMIT or G == k:
            continue
        pt = batch.prompt_tokens[batch.prompt_offsets[p]:batch.prompt_offsets[p + 1]]
        out = generate_group(dec, pt, p, list(range(k, G)), batch.caps[p, k:], wl.sample_seed, wl.temperature,
                             prefilled=prefilled[p], shared_prefix=shared_prefix)
        for i in range(k, G):
            tokens[p][i] = out[i]
            rewards[p, i] = reward(out[i], batch.reward_threshold[p])
            generated[p, i] = True
    count = np.where(status == stats.COMMIT, G, k)
    un, um, umean, uvar = stats.group_stats(rewards.reshape(-1), start, count)
    adv = stats.grpo_advantage(rewards.reshape(-1), start, count, status).reshape(P, G)
    return dict(tokens=tokens, rewards=rewards, generated=generated,
                pilot_n=pn, pilot_success=pm, pilot_mean=pmean, pilot_var=pvar,
                status=status, extra=extra, evict=evict, n_selected=n_sel, total_rollouts=total,
                union_n=un, union_success=um, union_mean=umean, union_var=uvar, advantages=adv)
