"""The 1.5B-shape configurations at full size, in the launch configuration bench.py times (captured decode steps, the
row counts of the pilot stage, of the commit stage and of all 2048 rollouts at once), checked on sampled outputs the
oracle can recompute one by one and on properties that hold at any size.

Sampled outputs: for a few rollouts the GPU's own tokens are fed to the oracle (a full causal recompute in float64) and
the logits the GPU produced at 8 consecutive decode steps of up to three depths (the deepest beyond 1,500 suffix slots)
must agree within 5e-2; the token the GPU drew must be the oracle's wherever the oracle's top-two gap exceeds 1e-1."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import sampler as osampler
from oracle import stats as ostats
from oracle.decoder import Decoder
from paper_2605_26606_b200 import workloads as wl
from paper_2605_26606_b200.engine import RolloutEngine

from gpu_util import ensure_built

pytestmark = pytest.mark.gpu

WINDOW = 8


@pytest.fixture(scope="module")
def shape_1p5b(cuda_device):
    ensure_built()
    model = wl.QWEN25_1P5B
    weights = wl.gen_weights(model, seed=0)
    return model, weights, Decoder(model, weights, cache_weights=True)          # float64 copies made once, on first use


def _free(eng):
    eng._arenas.clear()
    eng.prompt_kv = eng.suffix_kv = None
    del eng
    torch.cuda.empty_cache()


def check_step_invariants(out, w, batch, b_t=None):
    """Properties of a finished step that hold at any size, recomputed by the oracle's statistics on the GPU's own rewards."""
    P, G, k = w.n_prompts, w.group_size, w.n_pilot
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
    st, extra, ev, nsel, total = ostats.allocate(m, n, w.p_lower, w.p_upper, w.p_solve, G - k, P if b_t is None else b_t)
    assert np.array_equal(st, status) and np.array_equal(ev, out["evict"]) and np.array_equal(extra, out["extra"])
    count = np.where(status == ostats.COMMIT, G, k)
    adv = ostats.grpo_advantage(out["rewards"].reshape(-1), start, count, status).reshape(P, G)
    assert np.max(np.abs(adv - out["advantages"])) < 1e-5
    assert np.all(np.abs(out["advantages"].sum(axis=1)) < 1e-4)


def compare_rollout_windows(dec, w, batch, out, p, i, windows, records, last_logits=None):
    """Rollout (p, i): oracle logits (full recompute over prompt + the GPU's own tokens) against the GPU's recorded logits
    at the decode steps of `windows` (each a first step; WINDOW consecutive steps are compared).  records[s] =
    (logits rows, row prompts, row rollouts).  Returns (max |dlogit|, positions compared, positions outside the gap rule)."""
    toks = out["tokens"][p][i]
    Lp = int(batch.prompt_lens[p])
    pt = batch.prompt_tokens[batch.prompt_offsets[p]:batch.prompt_offsets[p + 1]]
    steps = [s for s0 in windows for s in range(s0, s0 + WINDOW) if s + 1 < len(toks) and s in records]
    assert steps, (p, i, len(toks), windows)
    upto = max(steps) + 1                                       # decode step s consumes generated token s
    positions = [Lp + s for s in steps] + ([Lp - 1] if last_logits is not None else [])
    want = dec.forward_full(np.concatenate([pt, toks[:upto]]), positions=positions)
    worst, n_cmp, n_exempt = 0.0, 0, 0
    checks = []
    for j, s in enumerate(steps):
        logits, rp, rr = records[s]
        row = np.flatnonzero((rp == p) & (rr == i))
        assert row.size == 1, (p, i, s)
        checks.append((s + 1, logits[int(row[0])].cpu().numpy(), want[j]))
    if last_logits is not None:
        checks.append((0, last_logits[p], want[len(steps)]))
    for gen_idx, got, ref in checks:
        worst = max(worst, float(np.max(np.abs(got - ref))))
        tok_o, gap = osampler.sample(ref, w.temperature, w.sample_seed, p, i, gen_idx)
        n_cmp += 1
        if gap > 1e-1:
            assert int(toks[gen_idx]) == tok_o, (p, i, gen_idx, gap)
        else:
            n_exempt += 1
    return worst, n_cmp, n_exempt


def test_headline_step_pilot_and_commit_stage_deep_windows_and_invariants(shape_1p5b):
    """config2 as benchmarked: 256 pilot rows, then 112 rows per committed prompt; logits at depths 30, 600 and 1,500."""
    model, weights, dec = shape_1p5b
    w = wl.WORKLOADS["config2"]
    batch = wl.gen_batch(w)
    P, G, k = w.n_prompts, w.group_size, w.n_pilot
    eng = RolloutEngine(w.model, weights, max_rows=max(P * k, P * (G - k)), max_prefill_tokens=int(batch.prompt_offsets[-1]))
    windows = [30, 600, 1500]
    steps = [s for s0 in windows for s in range(s0, s0 + WINDOW)]
    eng.record_pilot_logits = {s: None for s in steps}
    eng.record_commit_logits = {s: None for s in steps}
    # candidates: of every prompt the two longest pilot rollouts and the two longest commit rollouts (which prompts commit
    # is only known after the pilot stage)
    cand = {}
    for p in range(P):
        pil = sorted(range(k), key=lambda i: -int(batch.caps[p, i]))[:2]
        com = sorted(range(k, G), key=lambda i: -int(batch.caps[p, i]))[:2]
        cand[p] = (pil, com)
    eng.record_rows = {(p, i) for p in range(P) for i in cand[p][0] + cand[p][1]}
    out = eng.pilot_commit_step(w, batch)
    last_logits = eng.last_logits.cpu().numpy()
    check_step_invariants(out, w, batch)
    status = out["status"]
    forced = np.flatnonzero((batch.tau == 0.0) | (batch.tau == 1.0))
    assert len(forced) >= 4 and not np.any(status[forced] == ostats.COMMIT)                # collapsed groups never commit

    committed = [p for p in np.argsort(batch.prompt_lens) if status[p] == ostats.COMMIT]
    others = [p for p in np.argsort(batch.prompt_lens) if status[p] != ostats.COMMIT]
    # prompt A: the shortest committed prompt with a pilot and a commit rollout that both go beyond the deepest window
    committed = [p for p in committed if min(batch.caps[p, cand[p][0][0]], batch.caps[p, cand[p][1][0]]) > windows[2] + WINDOW]
    assert committed and others
    pa, pb = int(committed[0]), int(others[0])
    rec_p, rec_c = eng.record_pilot_logits, eng.record_commit_logits
    worst, n_cmp = 0.0, 0
    # prompt A (committed): one pilot and one commit rollout through all three depths, one more of each to depth 600
    plan = [(pa, cand[pa][0][0], windows, rec_p), (pa, cand[pa][1][0], windows, rec_c),
            (pa, cand[pa][0][1], windows[:2], rec_p), (pa, cand[pa][1][1], windows[:2], rec_c),
            # prompt B (pilot stage only): two pilot rollouts
            (pb, cand[pb][0][0], windows[:2], rec_p), (pb, cand[pb][0][1], windows[:1], rec_p)]
    deep = 0
    for p, i, wins, rec in plan:
        wv, n, _ = compare_rollout_windows(dec, w, batch, out, p, i, wins, rec, last_logits if rec is rec_p else None)
        worst, n_cmp = max(worst, wv), n_cmp + n
        deep += int(len(wins) == 3 and batch.caps[p, i] > windows[2] + WINDOW)
    assert deep == 2                       # a pilot-stage and a commit-stage rollout were compared beyond 1,500 suffix slots
    assert n_cmp >= 2 * 3 * WINDOW + 3 * WINDOW
    assert worst <= 5e-2, worst
    _free(eng)


def test_all_rollouts_at_once_2048_rows(shape_1p5b):
    """The 2048-concurrent launch configuration (wide tiles without K split, one-pass sampler) on a short-cap variant of config2."""
    model, weights, dec = shape_1p5b
    w = dataclasses.replace(wl.WORKLOADS["config2"], n_pilot=128, max_new=24, cap_lo=12, cap_hi=24)
    batch = wl.gen_batch(w)
    P, G = w.n_prompts, w.group_size
    eng = RolloutEngine(w.model, weights, max_rows=P * G, max_prefill_tokens=int(batch.prompt_offsets[-1]))
    eng.record_pilot_logits = {s: None for s in range(2, 2 + WINDOW)}
    order = np.argsort(batch.prompt_lens)
    pa, pb = int(order[0]), int(order[1])
    long_of = lambda p: sorted(range(G), key=lambda i: -int(batch.caps[p, i]))
    rows = [(pa, long_of(pa)[0]), (pa, long_of(pa)[1]), (pb, long_of(pb)[0]), (pb, long_of(pb)[1])]
    eng.record_rows = set(rows)
    out = eng.pilot_commit_step(w, batch)
    check_step_invariants(out, w, batch)
    last_logits = eng.last_logits.cpu().numpy()
    worst, n_cmp = 0.0, 0
    for p, i in rows:
        wv, n, _ = compare_rollout_windows(dec, w, batch, out, p, i, [2], eng.record_pilot_logits, last_logits)
        worst, n_cmp = max(worst, wv), n_cmp + n
    assert n_cmp == 4 * (WINDOW + 1) and worst <= 5e-2, (n_cmp, worst)
    _free(eng)


def test_headline_shape_with_bf16_operands(shape_1p5b):
    """The other operand mode at the 1.5B shape (bfloat16 GEMM operands, value + rounding remainder for QKV / output projection /
    LM head): pilot stage of a short-cap variant of config2, logits of two rollouts over one window against the oracle."""
    model, weights, dec = shape_1p5b
    w = dataclasses.replace(wl.WORKLOADS["config2"], max_new=24, cap_lo=12, cap_hi=24)
    batch = wl.gen_batch(w)
    P, G, k = w.n_prompts, w.group_size, w.n_pilot
    eng = RolloutEngine(w.model, weights, max_rows=max(P * k, P * (G - k)), max_prefill_tokens=int(batch.prompt_offsets[-1]), half_gemm=False)
    eng.record_pilot_logits = {s: None for s in range(2, 2 + WINDOW)}
    pa = int(np.argsort(batch.prompt_lens)[0])
    long_of = sorted(range(k), key=lambda i: -int(batch.caps[pa, i]))
    rows = [(pa, long_of[0]), (pa, long_of[1])]
    eng.record_rows = set(rows)
    out = eng.pilot_commit_step(w, batch)
    check_step_invariants(out, w, batch)
    last_logits = eng.last_logits.cpu().numpy()
    worst, n_cmp = 0.0, 0
    for p, i in rows:
        wv, n, _ = compare_rollout_windows(dec, w, batch, out, p, i, [2], eng.record_pilot_logits, last_logits)
        worst, n_cmp = max(worst, wv), n_cmp + n
    print("bf16 operands, 1.5B shape: max |dlogit|", worst)
    assert n_cmp == 2 * (WINDOW + 1) and worst <= 5e-2, (n_cmp, worst)
    _free(eng)


def test_config1_full_step(shape_1p5b):
    """Workload config1 in full (32 prompts of 256 tokens, G = 16, k = 4, up to 512 new tokens): 128 pilot rows, then 12 rows
    per committed prompt."""
    model, weights, dec = shape_1p5b
    w = wl.WORKLOADS["config1"]
    batch = wl.gen_batch(w)
    P, G, k = w.n_prompts, w.group_size, w.n_pilot
    eng = RolloutEngine(w.model, weights, max_rows=max(P * k, P * (G - k)), max_prefill_tokens=int(batch.prompt_offsets[-1]))
    windows = [100]
    steps = list(range(100, 100 + WINDOW))
    eng.record_pilot_logits = {s: None for s in steps}
    eng.record_commit_logits = {s: None for s in steps}
    cand = {p: (max(range(k), key=lambda i: int(batch.caps[p, i])), max(range(k, G), key=lambda i: int(batch.caps[p, i])))
            for p in range(P)}
    eng.record_rows = {(p, i) for p in range(P) for i in cand[p]}
    out = eng.pilot_commit_step(w, batch)
    check_step_invariants(out, w, batch)
    committed = np.flatnonzero(out["status"] == ostats.COMMIT)
    assert committed.size
    pa = int(committed[0])
    w1, n1, _ = compare_rollout_windows(dec, w, batch, out, pa, cand[pa][0], windows, eng.record_pilot_logits,
                                        eng.last_logits.cpu().numpy())
    w2, n2, _ = compare_rollout_windows(dec, w, batch, out, pa, cand[pa][1], windows, eng.record_commit_logits)
    assert n1 + n2 == 2 * WINDOW + 1 and max(w1, w2) <= 5e-2, (n1, n2, w1, w2)
    _free(eng)

