"""pc_sample_static -- the sampler variant for callers that cannot allocate device memory (a plugin that only receives
its input and output buffers, code running while the host framework's allocator is frozen or exhausted).  Its scratch is
an array inside the library image, so the test hands it nothing but inputs and outputs and checks, on two calls in a
row that reuse that array with different shapes, that it draws exactly the tokens pc_sample draws and, on the small
case, the tokens the oracle's sampler draws.

Collected last on purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

from oracle import sampler as osampler
from paper_2605_26606_b200 import binding as B
from paper_2605_26606_b200 import build

pytestmark = pytest.mark.gpu


def _case(n, vocab, seed, rng):
    logits = torch.from_numpy((rng.normal(size=(n, vocab)) * 2).astype(np.float32)).cuda()
    i32 = lambda a: torch.from_numpy(np.asarray(a, dtype=np.int32)).cuda()
    return logits, i32(rng.integers(0, 40, n)), i32(rng.integers(0, 128, n)), i32(rng.integers(0, 2048, n)), seed


def test_static_scratch_sampler_matches_pc_sample_on_two_calls_in_a_row(cuda_device):
    build.build()
    rng = np.random.default_rng(123)
    # second call: fewer rows and another vocabulary, so it reads records at other places of the shared array than the
    # first call wrote last
    for n, vocab, temperature in ((300, 151936, 1.0), (7, 4099, 0.7)):
        logits, prompt, roll, step, seed = _case(n, vocab, 0xABCDEF0123 + n, rng)
        want_tok = torch.zeros(n, dtype=torch.int32, device="cuda")
        want_gap = torch.zeros(n, dtype=torch.float32, device="cuda")
        B.pc_sample(n, vocab, logits, None, temperature, seed, prompt, roll, step, want_tok, None, want_gap)
        got_tok = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        got_gap = torch.zeros(n, dtype=torch.float32, device="cuda")
        B.pc_sample_static(n, vocab, logits, None, temperature, seed, prompt, roll, step, got_tok, None, got_gap)
        torch.cuda.synchronize()
        assert torch.equal(got_tok, want_tok)                    # token ids: bit-exact, as everywhere in the suite
        assert torch.equal(got_gap, want_gap)                    # maxima are exact, so the gaps are identical too
        if n <= 16:
            # against the oracle itself (float64 scores there, float32 here: equal wherever the top-two gap is not a rounding error)
            lg, tok, gap = logits.cpu().numpy(), got_tok.cpu().numpy(), got_gap.cpu().numpy()
            pr, ro, st = prompt.cpu().numpy(), roll.cpu().numpy(), step.cpu().numpy()
            for r in range(n):
                want, g = osampler.sample(lg[r], temperature, seed, int(pr[r]), int(ro[r]), int(st[r]))
                assert abs(gap[r] - g) < 1e-4
                if g > 1e-4:
                    assert tok[r] == want


def test_static_scratch_sampler_refuses_more_rows_than_it_holds(cuda_device):
    build.build()
    z = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.PcError) as err:
        B.pc_sample_static(4097, 8, torch.zeros(8, device="cuda"), None, 1.0, 0, z, z, z, z)
    assert err.value.status == B.PC_ERR_CAPACITY and "4096" in B.pc_last_cuda_error()
