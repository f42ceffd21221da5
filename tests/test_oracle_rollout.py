"""Pins for oracle/rollout.py: the single Pilot-Commit step (Algorithm 1, one iteration)."""
import dataclasses

import numpy as np
import pytest

from oracle import rollout, stats
from oracle.decoder import Decoder
from paper_2605_26606_b200 import workloads as wl


@pytest.fixture(scope="module")
def cfg0():
    w = wl.WORKLOADS["config0"]
    dec = Decoder(w.model, wl.gen_weights(w.model, seed=0, threads=2))
    batch = wl.gen_batch(w)
    return w, dec, batch, rollout.pilot_commit_step(dec, w, batch)


def test_config0_step_shapes_and_invariants(cfg0):
    w, dec, batch, out = cfg0
    P, G, k = w.n_prompts, w.group_size, w.n_pilot
    # forced prompts: tau = 0 -> never rewarded -> deferred; tau = 1 -> always rewarded -> skipped and evicted
    assert out["pilot_success"][0] == 0 and out["status"][0] == stats.DEFER_HARD and out["evict"][0] == 0
    assert out["pilot_success"][3] == k and out["status"][3] == stats.SKIP_EASY and out["evict"][3] == 1
    assert np.array_equal(out["pilot_var"], out["pilot_mean"] * (1 - out["pilot_mean"]))
    # budget conservation (Section 4.3 with b_g = P):  P k + |COMMIT| (G - k)
    ncommit = int(np.sum(out["status"] == stats.COMMIT))
    assert out["total_rollouts"] == P * k + ncommit * (G - k) == int(out["generated"].sum())
    for p in range(P):
        n_gen = G if out["status"][p] == stats.COMMIT else k
        assert out["generated"][p].sum() == n_gen and out["union_n"][p] == n_gen
        for i in range(n_gen):
            assert len(out["tokens"][p][i]) == batch.caps[p, i]
        a = out["advantages"][p]
        assert abs(a.sum()) < 1e-12
        if out["status"][p] != stats.COMMIT:
            assert np.all(a == 0)
        elif 0 < out["union_success"][p] < G:
            assert a @ a == pytest.approx(G)


def test_pilot_commit_rollouts_are_a_subset_of_full_group_rollouts(cfg0):
    """Keys are (seed, prompt, rollout, step): a rollout does not depend on the stage it ran in or on its batch mates."""
    w, dec, batch, out = cfg0
    p = int(np.flatnonzero(out["status"] == stats.COMMIT)[0]) if np.any(out["status"] == stats.COMMIT) else 1
    pt = batch.prompt_tokens[batch.prompt_offsets[p]:batch.prompt_offsets[p + 1]]
    full = rollout.generate_group(dec, pt, p, list(range(w.group_size)), batch.caps[p], w.sample_seed, w.temperature)
    for i in range(w.group_size):
        if out["tokens"][p][i] is not None:
            assert np.array_equal(out["tokens"][p][i], full[i])
    alone = rollout.generate_group(dec, pt, p, [5], batch.caps[p, 5:6], w.sample_seed, w.temperature, shared_prefix=True)
    assert np.array_equal(alone[5], full[5])


def test_ragged_caps_and_first_token_from_prompt_logits(cfg0):
    w, dec, batch, _ = cfg0
    pt = batch.prompt_tokens[batch.prompt_offsets[1]:batch.prompt_offsets[2]]
    out, logs = rollout.generate_group(dec, pt, 1, [0, 1, 2], [1, 3, 5], w.sample_seed, 1.0, record_logits=True)
    assert [len(out[i]) for i in range(3)] == [1, 3, 5]
    full = dec.forward_full(np.concatenate([pt, out[2][:-1]]))
    for s in range(5):
        assert np.max(np.abs(logs[2][s] - full[len(pt) - 1 + s])) < 1e-11


def test_group_success_rate_tracks_threshold():
    """With N(0, 0.02) weights the logits are nearly flat, so P(r = 1) is close to floor(tau V) / V."""
    w = dataclasses.replace(wl.WORKLOADS["config0"], n_prompts=1, group_size=200, n_pilot=200,
                            forced_explicit=((0, 0.3),), max_new=2, cap_lo=2, cap_hi=2)
    dec = Decoder(w.model, wl.gen_weights(w.model, seed=0, threads=2))
    out = rollout.pilot_commit_step(dec, w, wl.gen_batch(w))
    assert abs(out["pilot_mean"][0] - 0.3) < 0.1
