"""Helpers shared by the GPU parity tests (comparison of the CUDA path with the CPU oracle)."""
import numpy as np
import torch

from oracle import rollout as orollout
from oracle import sampler as osampler
from oracle.decoder import Decoder
from paper_2605_26606_b200 import binding as B
from paper_2605_26606_b200 import build
from paper_2605_26606_b200 import workloads as wl
from paper_2605_26606_b200.engine import RolloutEngine


def ensure_built():
    build.build()


def oracle_group_tokens(dec, w, batch, prompts, rollouts, record_logits=True):
    """Oracle tokens (and per-token logits) of the given rollouts: {(p, i): (tokens, [logits])}."""
    out = {}
    for p in sorted(set(int(x) for x in prompts)):
        idx = [int(i) for pp, i in zip(prompts, rollouts) if pp == p]
        pt = batch.prompt_tokens[batch.prompt_offsets[p]:batch.prompt_offsets[p + 1]]
        toks, logs = orollout.generate_group(dec, pt, p, idx, batch.caps[p, idx], w.sample_seed, w.temperature,
                                             record_logits=True)
        for i in idx:
            out[(p, i)] = (toks[i], logs[i])
    return out


def teacher_forced_compare(eng: RolloutEngine, w, batch, ref, prompts, rollouts, logit_tol, gap_tol):
    """Feeds the oracle's tokens through the CUDA path and compares, position by position, the logits and
    the token the CUDA sampler draws from the CUDA logits.  Returns (max |dlogit|, n compared, n gap-exempt)."""
    P, G = w.n_prompts, w.group_size
    eng.load_batch(w, batch)
    eng.prefill()
    tok_host = np.full((P, G, w.max_new), -1, dtype=np.int32)
    for (p, i), (t, _) in ref.items():
        tok_host[p, i, :len(t)] = t
    eng.tokens.copy_(torch.from_numpy(tok_host.reshape(-1)))
    n_steps = int(batch.caps[prompts, rollouts].max()) - 1
    rec = {s: None for s in range(n_steps)}
    eng.run_stage(np.asarray(prompts), np.asarray(rollouts), record_logits=rec, teacher_forced=True)
    eng.check_error_flag()
    last = eng.last_logits.cpu().numpy()
    worst, n_cmp, n_exempt = 0.0, 0, 0

    def check(gpu_logits, p, i, s):
        nonlocal worst, n_cmp, n_exempt
        want = ref[(p, i)][1][s]
        worst = max(worst, float(np.max(np.abs(gpu_logits - want))))
        # the CUDA sampler on the CUDA logits against the oracle's draw
        lg = torch.from_numpy(np.ascontiguousarray(gpu_logits[None])).cuda()
        ti = lambda v: torch.tensor([v], dtype=torch.int32, device="cuda")
        out = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.pc_sample(1, w.model.vocab, lg, None, w.temperature, w.sample_seed, ti(p), ti(i), ti(s), out)
        tok_o, gap_o = osampler.sample(want, w.temperature, w.sample_seed, p, i, s)
        assert tok_o == ref[(p, i)][0][s]
        n_cmp += 1
        if gap_o > gap_tol:
            assert int(out.item()) == tok_o, (p, i, s, gap_o)
        else:
            n_exempt += 1

    for p, i in zip(prompts, rollouts):
        check(last[p], int(p), int(i), 0)
    for s in range(n_steps):
        logits, rp, rr = rec[s]
        logits = logits.cpu().numpy()
        for r in range(len(rp)):
            check(logits[r], int(rp[r]), int(rr[r]), s + 1)
    assert worst <= logit_tol, worst
    return worst, n_cmp, n_exempt
