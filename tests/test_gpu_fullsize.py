"""The headline configuration (Qwen2.5-1.5B shape, 16 prompts x G = 128, k = 16, up to 2048 new tokens) in the launch
configuration bench.py times, checked on sampled outputs the oracle can recompute and on properties that hold at any size."""
import numpy as np
import pytest
import torch

from oracle import sampler as osampler
from oracle import stats as ostats
from oracle.decoder import Decoder
from paper_2605_26606_b200 import binding as B
from paper_2605_26606_b200 import workloads as wl
from paper_2605_26606_b200.engine import RolloutEngine

from gpu_util import ensure_built

pytestmark = pytest.mark.gpu


def test_headline_step_sampled_logits_tokens_and_invariants(cuda_device):
    ensure_built()
    w = wl.WORKLOADS["config2"]
    weights = wl.gen_weights(w.model, seed=0)
    batch = wl.gen_batch(w)
    P, G, k = w.n_prompts, w.group_size, w.n_pilot
    eng = RolloutEngine(w.model, weights, max_rows=max(P * k, P * (G - k)), max_prefill_tokens=int(batch.prompt_offsets[-1]))
    steps = [0, 37, 120]
    eng.record_pilot_logits = {s: None for s in steps}
    out = eng.pilot_commit_step(w, batch)
    rec = eng.record_pilot_logits
    last_logits = eng.last_logits.cpu().numpy()

    # ---- properties that hold at any size
    gen, status = out["generated"], out["status"]
    n_commit = int((status == ostats.COMMIT).sum())
    assert out["total_rollouts"] == P * k + n_commit * (G - k) == int(gen.sum())          # budget (Section 4.3)
    assert out["generated_tokens"] == int(batch.caps[gen].sum())
    for p in range(P):
        for i in range(G):
            if gen[p, i]:
                t = out["tokens"][p][i]
                assert len(t) == batch.caps[p, i] and t.min() >= 0 and t.max() < w.model.vocab
                assert out["rewards"][p, i] == (1.0 if t[-1] < batch.reward_threshold[p] else 0.0)
    start = np.arange(P) * G
    n, m, mean, var = ostats.group_stats(out["rewards"].reshape(-1), start, np.full(P, k))
    assert np.array_equal(m, out["pilot_success"]) and np.array_equal(n, out["pilot_n"])
    assert np.max(np.abs(out["pilot_var"] - mean * (1 - mean))) < 1e-6                       # Var = p (1 - p)
    st, extra, ev, nsel, total = ostats.allocate(m, n, w.p_lower, w.p_upper, w.p_solve, G - k, P)
    assert np.array_equal(st, status) and np.array_equal(ev, out["evict"]) and np.array_equal(extra, out["extra"])
    count = np.where(status == ostats.COMMIT, G, k)
    adv = ostats.grpo_advantage(out["rewards"].reshape(-1), start, count, status).reshape(P, G)
    assert np.max(np.abs(adv - out["advantages"])) < 1e-5
    assert np.all(np.abs(out["advantages"].sum(axis=1)) < 1e-4)
    forced = np.flatnonzero((batch.tau == 0.0) | (batch.tau == 1.0))
    assert len(forced) >= 4 and not np.any(status[forced] == ostats.COMMIT)                # collapsed groups never commit

    # ---- sampled outputs against the oracle: one rollout of the shortest prompt, teacher-forced by the GPU's own tokens
    p = int(np.argmin(batch.prompt_lens))
    i = 1
    toks = out["tokens"][p][i]
    Lp = int(batch.prompt_lens[p])
    pt = batch.prompt_tokens[batch.prompt_offsets[p]:batch.prompt_offsets[p + 1]]
    dec = Decoder(w.model, weights, cache_weights=False)
    upto = max(steps) + 1                                   # decode step s consumes generated token s
    full = dec.forward_full(np.concatenate([pt, toks[:upto]]))
    # generated token 0 comes from the prompt's last position; decode step s yields the logits of generated token s + 1
    checks = [(0, last_logits[p], full[Lp - 1])]
    for s in steps:
        logits, rp, rr = rec[s]
        row = int(np.flatnonzero((rp == p) & (rr == i))[0])
        checks.append((s + 1, logits[row].cpu().numpy(), full[Lp + s]))
    worst = 0.0
    for gen_idx, got, want in checks:
        worst = max(worst, float(np.max(np.abs(got - want))))
        tok_o, gap = osampler.sample(want, w.temperature, w.sample_seed, p, i, gen_idx)
        if gap > 1e-1:
            assert int(toks[gen_idx]) == tok_o, (gen_idx, gap)
    assert worst <= 5e-2, worst
