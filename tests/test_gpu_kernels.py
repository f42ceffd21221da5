"""CUDA entry points against the CPU oracle, one operation at a time (through the C ABI)."""
import itertools

import numpy as np
import pytest
import torch

from oracle import philox as ophilox
from oracle import sampler as osampler
from oracle import stats as ostats
from paper_2605_26606_b200 import binding as B

from gpu_util import ensure_built

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built(cuda_device):
    ensure_built()


def _i32(a):
    return torch.from_numpy(np.asarray(a, dtype=np.int32)).cuda()


@pytest.mark.parametrize("vocab", [1, 3, 8, 1003, 2048, 151936])
@pytest.mark.parametrize("temperature", [1.0, 0.7])
def test_sample_matches_oracle(vocab, temperature):
    rng = np.random.default_rng(vocab)
    n = 24
    logits = (rng.normal(size=(n, vocab)) * 2).astype(np.float32)
    prompt, roll, step = rng.integers(0, 50, n), rng.integers(0, 128, n), rng.integers(0, 2048, n)
    seed = (77 << 32) | 12345
    out = torch.zeros(n, dtype=torch.int32, device="cuda")
    gap = torch.zeros(n, dtype=torch.float32, device="cuda")
    B.pc_sample(n, vocab, torch.from_numpy(logits).cuda(), None, temperature, seed, _i32(prompt), _i32(roll), _i32(step), out,
                None, gap)
    # the two-pass form (vocabulary of a row split over several blocks) must give the very same answer
    out2 = torch.zeros(n, dtype=torch.int32, device="cuda")
    gap2 = torch.zeros(n, dtype=torch.float32, device="cuda")
    scratch = torch.empty(n * 32 * 16, dtype=torch.uint8, device="cuda")
    B.pc_sample(n, vocab, torch.from_numpy(logits).cuda(), None, temperature, seed, _i32(prompt), _i32(roll), _i32(step), out2,
                None, gap2, scratch)
    assert torch.equal(out, out2) and torch.equal(gap, gap2)
    out, gap = out.cpu().numpy(), gap.cpu().numpy()
    for r in range(n):
        tok, g = osampler.sample(logits[r], temperature, seed, int(prompt[r]), int(roll[r]), int(step[r]))
        if g > 1e-4:
            assert out[r] == tok
        if np.isfinite(g):
            assert abs(gap[r] - g) < 1e-4
        else:
            assert np.isinf(gap[r])


def test_sample_row_mapping_and_scatter():
    rng = np.random.default_rng(0)
    V, P, G = 512, 3, 5
    logits = rng.normal(size=(P, V)).astype(np.float32)
    prompt, roll = np.repeat(np.arange(P), G), np.tile(np.arange(G), P)
    out = torch.full((P * G * 4,), -1, dtype=torch.int32, device="cuda")
    idx = torch.arange(P * G, dtype=torch.int64, device="cuda") * 4 + 1
    B.pc_sample(P * G, V, torch.from_numpy(logits).cuda(), _i32(prompt), 1.0, 9, _i32(prompt), _i32(roll),
                _i32(np.zeros(P * G)), out, idx)
    out = out.cpu().numpy().reshape(P * G, 4)
    assert np.all(out[:, [0, 2, 3]] == -1)
    for r in range(P * G):
        assert out[r, 1] == osampler.sample(logits[prompt[r]], 1.0, 9, int(prompt[r]), int(roll[r]), 0)[0]


def test_sample_exact_tie_takes_lowest_id():
    V = 64
    logits = np.zeros((1, V), dtype=np.float32)
    logits[0, [40, 9, 22]] = 1e30          # absorbs the noise: an exact three-way tie
    out = torch.zeros(1, dtype=torch.int32, device="cuda")
    gap = torch.zeros(1, dtype=torch.float32, device="cuda")
    B.pc_sample(1, V, torch.from_numpy(logits).cuda(), None, 1.0, 1, _i32([0]), _i32([0]), _i32([0]), out, None, gap)
    assert out.item() == 9 and gap.item() == 0.0


def test_reward_last_token():
    tokens = _i32([5, 9, 100, 3, 7, 0])
    last = torch.tensor([1, 2, 5, 3], dtype=torch.int64, device="cuda")
    thr = _i32([9, 101, 0, 4])
    r = torch.zeros(4, dtype=torch.float32, device="cuda")
    B.pc_reward_last_token(4, tokens, last, thr, r)
    assert r.cpu().tolist() == [0.0, 1.0, 0.0, 1.0]


def _stats_gpu(rewards, start, count):
    P = len(start)
    n, m = torch.zeros(P, dtype=torch.int32, device="cuda"), torch.zeros(P, dtype=torch.int32, device="cuda")
    mean, var = torch.zeros(P, device="cuda"), torch.zeros(P, device="cuda")
    B.pc_group_stats(P, torch.from_numpy(rewards.astype(np.float32)).cuda(), _i32(start), _i32(count), n, m, mean, var)
    return n.cpu().numpy(), m.cpu().numpy(), mean.cpu().numpy(), var.cpu().numpy()


def test_group_stats_and_advantage_match_oracle():
    rng = np.random.default_rng(3)
    P = 37
    count = rng.integers(0, 300, P); count[:4] = [0, 1, 128, 33]
    start = np.r_[0, np.cumsum(count + rng.integers(0, 5, P))[:-1]]
    total = int(start[-1] + count[-1] + 3)
    for binary in (True, False):
        r = (rng.random(total) < rng.random(total)).astype(np.float64) if binary else rng.normal(size=total)
        if binary:
            r[start[5]:start[5] + count[5]] = 1.0
            r[start[6]:start[6] + count[6]] = 0.0
        r32 = r.astype(np.float32).astype(np.float64)
        n, m, mean, var = _stats_gpu(r32, start, count)
        on, om, omean, ovar = ostats.group_stats(r32, start, count)
        assert np.array_equal(n, on) and np.array_equal(m, om)
        assert np.max(np.abs(mean - omean)) < 1e-6 and np.max(np.abs(var - ovar)) < 1e-6
        if binary:
            p = om / np.maximum(on, 1)
            assert np.max(np.abs(var - p * (1 - p))) < 1e-6
        status = rng.integers(0, 4, P)
        for st in (None, status):
            adv = torch.full((total,), 7.0, device="cuda")
            B.pc_grpo_advantage(P, torch.from_numpy(r32.astype(np.float32)).cuda(), _i32(start), _i32(count),
                                None if st is None else _i32(st), adv)
            adv = adv.cpu().numpy().astype(np.float64)
            want = ostats.grpo_advantage(r32, start, count, st)
            inside = np.zeros(total, dtype=bool)
            for g in range(P):
                inside[start[g]:start[g] + count[g]] = True
            assert np.max(np.abs(adv[inside] - want[inside])) < 1e-5
            assert np.all(adv[~inside] == 7.0)                  # nothing outside the groups is written
            for g in range(P):
                seg = adv[start[g]:start[g] + count[g]]
                assert abs(seg.sum()) < 1e-4 * max(1, count[g])


def _alloc_gpu(m, n, pl, pu, ps, nc, bt):
    P = len(m)
    st, ex, ev = (torch.zeros(P, dtype=torch.int32, device="cuda") for _ in range(3))
    nsel = torch.zeros(1, dtype=torch.int32, device="cuda")
    tot = torch.zeros(1, dtype=torch.int64, device="cuda")
    B.pc_allocate(P, _i32(m), _i32(n), B.AllocParams(pl, pu, ps, nc, bt), st, ex, ev, nsel, tot)
    return st.cpu().numpy(), ex.cpu().numpy(), ev.cpu().numpy(), int(nsel.item()), int(tot.item())


def test_allocate_matches_oracle_bit_exact():
    rng = np.random.default_rng(4)
    cases = []
    for pu, pl, ps in itertools.product([1.0, 0.875, 0.75, 0.625], [0.0, 0.125, 0.25, 0.375], [0.75, 0.875, 1.0]):
        k = int(rng.integers(1, 33)); P = int(rng.integers(1, 70))
        cases.append((rng.integers(0, k + 1, P), np.full(P, k), pl, pu, ps, int(rng.integers(0, 97)), int(rng.integers(0, P + 2))))
    # non-dyadic thresholds and mixed pilot counts, a batch larger than one block, the paper's b_g = 384 / b_t = 128
    n_big = rng.integers(1, 40, 3000)
    cases.append((rng.integers(0, 40, 3000) % (n_big + 1), n_big, 0.1, 0.7, 0.9, 48, 1000))
    cases.append((rng.integers(0, 17, 384), np.full(384, 16), 0.125, 0.75, 1.0, 48, 128))
    cases.append((np.array([3]), np.array([10]), 0.3, 0.3, 1.0, 5, 1))
    for m, n, pl, pu, ps, nc, bt in cases:
        got = _alloc_gpu(m, n, pl, pu, ps, nc, bt)
        want = ostats.allocate(m, n, pl, pu, ps, nc, bt)
        for a, b in zip(got[:3], want[:3]):
            assert np.array_equal(a, b)
        assert got[3] == want[3] and got[4] == want[4]
    st, ex, ev, nsel, tot = _alloc_gpu(np.full(384, 8), np.full(384, 16), 0.125, 0.75, 1.0, 48, 128)
    assert nsel == 128 and tot == 12288          # Table 2: PC generates 12,288 rollouts per step at n = 64


def test_philox_words_match_oracle_through_uniform_logits():
    """With flat logits the arg-max is the arg-max of the Gumbel noise: checks the device generator
    against the oracle's over many (prompt, rollout, step) keys and the whole vocabulary range."""
    V, n = 151936, 64
    rng = np.random.default_rng(6)
    prompt, roll, step = rng.integers(0, 2 ** 20, n), rng.integers(0, 2 ** 10, n), rng.integers(0, 2 ** 14, n)
    seed = 0xDEADBEEF12345678
    out = torch.zeros(n, dtype=torch.int32, device="cuda")
    B.pc_sample(n, V, torch.zeros((1, V), device="cuda"), _i32(np.zeros(n)), 1.0, seed, _i32(prompt), _i32(roll), _i32(step), out)
    out = out.cpu().numpy()
    for r in range(n):
        g = ophilox.gumbel_noise(V, seed, int(prompt[r]), int(roll[r]), int(step[r]))
        assert out[r] == int(np.argmax(g))


def test_token_logprob_matches_oracle():
    from oracle.logprob import token_logprob
    rng = np.random.default_rng(8)
    for vocab, T in ((7, 1.0), (4099, 0.7), (151936, 1.0)):
        n = 9
        logits = (rng.normal(size=(3, vocab)) * 4).astype(np.float32)
        row = rng.integers(0, 3, n)
        toks = rng.integers(0, vocab, n)
        tok_buf = torch.from_numpy(np.stack([np.full(n, -7), toks], axis=1).reshape(-1).astype(np.int32)).cuda()
        tok_idx = torch.arange(n, dtype=torch.int64, device="cuda") * 2 + 1
        out = torch.full((n * 3,), 9.0, device="cuda")
        out_idx = torch.arange(n, dtype=torch.int64, device="cuda") * 3 + 2
        B.pc_token_logprob(n, vocab, torch.from_numpy(logits).cuda(), _i32(row), T, tok_buf, tok_idx, out, out_idx)
        out = out.cpu().numpy().reshape(n, 3)
        assert np.all(out[:, :2] == 9.0)
        for r in range(n):
            assert abs(out[r, 2] - token_logprob(logits[row[r]], int(toks[r]), T)) < 1e-4


def test_dapo_and_grpo_modes_through_pc_allocate():
    """DAPO's zero-variance filter (Section 4.3) = pc_allocate on full groups with thresholds 1/n, (n-1)/n and no commit."""
    rng = np.random.default_rng(10)
    for n in (2, 16, 64, 128):
        P = 300
        m = rng.integers(0, n + 1, size=P); m[:3] = [0, n, 1]
        r = np.zeros((P, n))
        for p in range(P):
            r[p, rng.permutation(n)[:m[p]]] = 1.0
        start, count = np.arange(P) * n, np.full(P, n)
        cn, cm, _, var = _stats_gpu(r.reshape(-1), start, count)
        assert np.array_equal(cm, m)
        st, ex, ev, nsel, tot = _alloc_gpu(cm, cn, 1.0 / n, (n - 1.0) / n, 1.0, 0, P)
        keep = ostats.dapo_filter(r.reshape(-1), start, count)
        assert np.array_equal(st == B.PC_STATUS_COMMIT, keep == 1) and tot == P * n
        assert np.array_equal(var > 0, keep == 1)
        st, ex, ev, nsel, tot = _alloc_gpu(cm, cn, 0.0, 1.0, 2.0, 0, P)          # GRPO: nothing filtered
        assert np.all(st == B.PC_STATUS_COMMIT) and nsel == P


def test_bounded_wait_gives_up_and_the_context_stays_usable():
    """A wait on an mbarrier nobody arrives at (no copy in flight) runs out after its limit, leaves DEV_ERR_WAIT_TIMEOUT in
    the error flag and the kernel returns; the next launches work."""
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.pc_selftest_wait_timeout(1 << 10, flag)
    torch.cuda.synchronize()
    assert int(flag.item()) == 3
    # the device is still usable: an ordinary entry point gives the right answer afterwards
    tokens = _i32([5, 9, 100, 3, 7, 0])
    last = torch.tensor([1, 2, 5, 3], dtype=torch.int64, device="cuda")
    r = torch.zeros(4, dtype=torch.float32, device="cuda")
    B.pc_reward_last_token(4, tokens, last, _i32([9, 101, 0, 4]), r)
    assert r.cpu().tolist() == [0.0, 1.0, 0.0, 1.0]
    with pytest.raises(B.PcError):
        B.pc_selftest_wait_timeout(0, flag)


def test_reward_of_a_never_generated_cell_is_zero():
    tokens = _i32([-1, 4, -1])
    last = torch.tensor([0, 1, 2], dtype=torch.int64, device="cuda")
    r = torch.full((3,), 7.0, device="cuda")
    B.pc_reward_last_token(3, tokens, last, _i32([10, 10, 10]), r)
    assert r.cpu().tolist() == [0.0, 1.0, 0.0]


def test_variance_filter_for_scalar_rewards_matches_oracle():
    """pc_allocate_variance on the variances pc_group_stats returns: decisions identical to the oracle's, for continuous
    rewards and for binary ones (where it reproduces the success-rate band)."""
    rng = np.random.default_rng(11)
    P, k = 300, 16
    for binary in (False, True):
        r = (rng.random((P, k)) < rng.random((P, 1))).astype(np.float64) if binary else rng.normal(size=(P, k)) * rng.uniform(0, 2, size=(P, 1))
        start, count = np.arange(P) * k, np.full(P, k)
        n, m, mean, var = _stats_gpu(r.reshape(-1), start, count)
        var_min = 0.1875 if binary else 0.7
        status, extra = torch.zeros(P, dtype=torch.int32, device="cuda"), torch.zeros(P, dtype=torch.int32, device="cuda")
        nsel, total = torch.zeros(1, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.int64, device="cuda")
        B.pc_allocate_variance(P, torch.from_numpy(var).cuda(), _i32(n), var_min, 48, 100, status, extra, nsel, total)
        _, _, _, ovar = ostats.group_stats(r.astype(np.float32).astype(np.float64).reshape(-1), start, count)
        st, ex, sel, tot = ostats.allocate_by_variance(ovar, n, var_min, 48, 100)
        assert np.array_equal(status.cpu().numpy(), st) and np.array_equal(extra.cpu().numpy(), ex)
        assert int(nsel.item()) == sel and int(total.item()) == tot
        if binary:
            keep = (m / k >= 0.25) & (m / k <= 0.75)
            assert np.array_equal(st != ostats.LOW_VARIANCE, keep)
