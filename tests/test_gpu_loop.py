"""Algorithm 1 as a running loop on the GPU: the host controller (replay buffer with delay d, eviction across epochs, second
sampling round) driving the rollout engine for several consecutive training steps, against the oracle's simulation of the
bookkeeping combined with the oracle's rollouts."""
import dataclasses

import numpy as np
import pytest

from oracle import controller as octl
from oracle import rollout as orollout
from oracle import stats as ostats
from oracle.decoder import Decoder
from paper_2605_26606_b200 import workloads as wl
from paper_2605_26606_b200.engine import RolloutEngine
from paper_2605_26606_b200.loop import RolloutLoop, SlotPool

from gpu_util import ensure_built


def test_slot_pool_first_fit_and_merge():
    p = SlotPool(100)
    a, b, c = p.alloc(30), p.alloc(30), p.alloc(40)
    assert (a, b, c) == (0, 30, 60)
    with pytest.raises(MemoryError):
        p.alloc(1)
    p.release(b, 30)
    p.release(a, 30)
    assert p.free == [(0, 60)]
    assert p.alloc(50) == 0 and p.alloc(10) == 50
    p.release(c, 40)
    assert p.alloc(40) == 60


def _oracle_loop(dec, w, data, ids, n_epochs, b_g, b_t, d, max_rounds):
    G, k = w.group_size, w.n_pilot
    pilots = {}

    def prompt_tokens(q):
        return data.prompt_tokens[data.prompt_offsets[q]:data.prompt_offsets[q + 1]]

    def pilot(q):
        if q not in pilots:
            toks = orollout.generate_group(dec, prompt_tokens(q), q, list(range(k)), data.caps[q, :k], w.sample_seed, w.temperature)
            rew = [orollout.reward(toks[i], data.reward_threshold[q]) for i in range(k)]
            pilots[q] = (toks, rew)
        return pilots[q]

    log = octl.simulate(list(ids), n_epochs, b_g, b_t, k, G - k, w.p_lower, w.p_upper, w.p_solve, d,
                        lambda q, t: sum(pilot(q)[1]) / k, max_rounds=max_rounds)
    commits = {}
    for e in log:
        for q, born in e["selected"]:
            toks = orollout.generate_group(dec, prompt_tokens(q), q, list(range(k, G)), data.caps[q, k:], w.sample_seed, w.temperature)
            rew = pilot(q)[1] + [orollout.reward(toks[i], data.reward_threshold[q]) for i in range(k, G)]
            adv = ostats.grpo_advantage(np.array(rew), np.array([0]), np.array([G]))
            commits[q] = (toks, rew, adv)
    return log, pilots, commits


@pytest.mark.gpu
@pytest.mark.parametrize("bind,max_rounds,b_t,data_seed", [(False, 1, 1, 17), (True, 1, 1, 17), (True, 2, 2, 5)],
                         ids=["two-passes", "bound", "bound-two-rounds"])
def test_training_loop_equals_the_oracle_step_by_step(cuda_device, bind, max_rounds, b_t, data_seed):
    ensure_built()
    n_prompts, b_g, d, n_epochs = 24, 6, 1, 2
    w = dataclasses.replace(wl.WORKLOADS["config0"], n_prompts=n_prompts, prompt_len_lo=4, prompt_len_hi=40, cap_lo=2, cap_hi=12, max_new=12,
                            data_seed=data_seed, forced_explicit=tuple((q, 0.5) for q in range(0, n_prompts, 2)) + ((1, 1.0), (3, 0.0)))
    weights = wl.gen_weights(w.model, seed=0, threads=2, gain_jitter=0.1)
    data = wl.gen_batch(w)
    dec = Decoder(w.model, weights)
    ids = list(range(n_prompts))
    log, pilots, commits = _oracle_loop(dec, w, data, ids, n_epochs, b_g, b_t, d, max_rounds)
    assert len(log) >= 4 and any(e["selected"] for e in log) and any(e["solved"] for e in log)
    if max_rounds == 2:
        assert any(e["rounds"] == 2 for e in log)
    else:
        assert any(e["stale"] for e in log) and any(e["buffered"] for e in log)
    eng = RolloutEngine(w.model, weights, max_rows=b_g * w.n_pilot + b_t * (w.group_size - w.n_pilot) + 8,
                        max_prefill_tokens=b_g * 40)
    loop = RolloutLoop(eng, w, data, b_g, b_t, d, max_rounds=max_rounds, bind=bind)
    recs = loop.run(ids, n_epochs)
    assert len(recs) == len(log)
    G, k = w.group_size, w.n_pilot
    seen_commits = set()
    for rec, e in zip(recs, log):
        p = rec.plan
        assert (p.step, p.rounds, p.committed, p.dropped_stale, p.buffered_after, p.rollouts_sampled) == \
            (e["step"], e["rounds"], e["selected"], e["stale"], e["buffered"], e["rollouts"])
        assert sorted(p.newly_evicted) == sorted(e["solved"])
        assert [q for b in rec.batches for q in b] == e["batch"]
        for q in e["batch"]:
            assert rec.pilot_success[q] == int(sum(pilots[q][1]))
        for (q, i), t in rec.tokens.items():
            want = pilots[q][0][i] if i < k else commits[q][0][i]
            assert np.array_equal(t, want), (p.step, q, i)
            assert rec.rewards[(q, i)] == (pilots[q][1][i] if i < k else commits[q][1][i])
        for q, _ in e["selected"]:
            assert all((q, i) in rec.tokens for i in range(G)), q          # the union group is complete
            assert np.max(np.abs(rec.advantages[q] - commits[q][2])) < 1e-5
            seen_commits.add(q)
    assert seen_commits == set(commits)
    # nothing stays resident once every survivor was committed or dropped, except what still waits in the buffer
    assert len(loop.row_of) == recs[-1].plan.buffered_after
