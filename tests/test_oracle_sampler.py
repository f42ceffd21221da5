"""Pins for oracle/philox.py and oracle/sampler.py."""
import math
import os

import numpy as np
import pytest

from oracle import philox, sampler


_TRITON_SCRIPT = r"""
import json, sys
import numpy as np, torch, triton, triton.language as tl

@triton.jit
def kern(out, c0_ptr, c1, c2, c3, k0, k1, n: tl.constexpr):
    i = tl.arange(0, n)
    c0 = tl.load(c0_ptr + i).to(tl.uint32, bitcast=True)
    z = c0 * 0
    a, b, c, d = tl.philox_impl(c0, z + c1, z + c2, z + c3, z + k0, z + k1, 10)
    tl.store(out + i * 4 + 0, a.to(tl.int32, bitcast=True)); tl.store(out + i * 4 + 1, b.to(tl.int32, bitcast=True))
    tl.store(out + i * 4 + 2, c.to(tl.int32, bitcast=True)); tl.store(out + i * 4 + 3, d.to(tl.int32, bitcast=True))

cases = json.loads(sys.argv[1]); n = 256
c0 = (np.arange(n, dtype=np.uint64) * np.uint64(2654435761) + np.uint64(12345)) & np.uint64(0xFFFFFFFF)
c0[:4] = [0, 1, 0xFFFFFFFF, 0x80000000]
res = []
for (c1, c2, c3, k0, k1) in cases:
    out = torch.zeros(n * 4, dtype=torch.int32)
    kern[(1,)](out, torch.from_numpy(c0.astype(np.uint32).view(np.int32)), c1, c2, c3, k0, k1, n)
    res.append(out.numpy().view(np.uint32).tolist())
print(json.dumps(res))
"""


def test_philox_matches_independent_library_implementation():
    """Triton ships its own Philox4x32 (`philox_impl`); its CPU interpreter runs it without a GPU.
    It runs in a fresh process because the interpreter mode must be chosen before triton is imported."""
    import json
    import subprocess
    import sys
    cases = [(0, 0, 0, 0, 0), (7, 3, 1, 5, 9), (2047, 127, 15, 0x7FFFFFFF, 0x12345678)]
    env = dict(os.environ, TRITON_INTERPRET="1", CUDA_VISIBLE_DEVICES="")
    res = subprocess.run([sys.executable, "-c", _TRITON_SCRIPT, json.dumps(cases)], capture_output=True, text=True, env=env,
                         timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    theirs = json.loads(res.stdout.strip().splitlines()[-1])
    n = 256
    c0 = (np.arange(n, dtype=np.uint64) * np.uint64(2654435761) + np.uint64(12345)) & np.uint64(0xFFFFFFFF)
    c0[:4] = [0, 1, 0xFFFFFFFF, 0x80000000]
    for (c1, c2, c3, k0, k1), ref in zip(cases, theirs):
        mine = np.stack(philox.philox4x32_10(c0, c1, c2, c3, k0, k1), axis=1).reshape(-1)
        assert np.array_equal(mine, np.array(ref, dtype=np.uint32))


def test_counter_layout_and_word_selection():
    V = 1003
    w = philox.vocab_words(V, seed=(9 << 32) | 5, prompt=1, rollout=3, step=7)
    assert w.shape == (V,) and w.dtype == np.uint32
    for v in (0, 1, 2, 3, 4, 501, 1002):
        blk = philox.philox4x32_10(v >> 2, 7, 3, 1, 5, 9)
        assert w[v] == blk[v & 3][()]
    # every coordinate of the key matters
    base = philox.vocab_words(64, 11, 1, 2, 3)
    for args in ((12, 1, 2, 3), (11, 0, 2, 3), (11, 1, 0, 3), (11, 1, 2, 0), (11 + (1 << 32), 1, 2, 3)):
        assert not np.array_equal(base, philox.vocab_words(64, *args))


def test_uniform_is_open_interval_and_float32_exact():
    w = np.array([0, 1, 511, 512, 2 ** 32 - 1], dtype=np.uint32)
    u = philox.uniform_from_word(w)
    assert u[0] == 2.0 ** -24 and u[-1] == 1.0 - 2.0 ** -24 and u[0] == u[2] and u[3] == 1.5 * 2.0 ** -23
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)
    assert np.all(np.isfinite(philox.gumbel_from_word(w)))


def test_uniform_and_gumbel_moments():
    words = np.concatenate([philox.vocab_words(1 << 16, 77, p, 0, 0) for p in range(16)])
    u = philox.uniform_from_word(words)
    n = u.shape[0]
    hist, _ = np.histogram(u, bins=64, range=(0, 1))
    chi2 = np.sum((hist - n / 64) ** 2 / (n / 64))
    assert chi2 < 120                      # 63 dof: mean 63, sd 11
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 5e-3
    # each of the 32 bits of the raw word is balanced
    bits = (words[:, None] >> np.arange(32, dtype=np.uint32)[None]) & 1
    assert np.all(np.abs(bits.mean(0) - 0.5) < 5e-3)
    g = philox.gumbel_from_word(words)
    assert np.mean(g) == pytest.approx(0.5772156649, abs=6e-3)
    assert np.var(g) == pytest.approx(math.pi ** 2 / 6, rel=1e-2)


def test_gumbel_max_draws_follow_softmax():
    # temperature 1.0, top_p 1.0 (Section 4.2): token frequencies must equal softmax(logits)
    logits = np.array([0.3, -1.2, 2.0, 0.0, 1.1, -0.5, 0.7, -3.0])
    for T in (1.0, 0.7):
        p = np.exp(logits / T) / np.exp(logits / T).sum()
        N = 40000
        counts = np.zeros(8)
        for i in range(N):
            t, gap = sampler.sample(logits, T, seed=99, prompt=i % 50, rollout=i // 50, step=3)
            counts[t] += 1
            assert gap >= 0
        chi2 = np.sum((counts - N * p) ** 2 / (N * p))
        assert chi2 < 30                   # 7 dof


def test_sample_is_argmax_lowest_index_on_ties_and_gap():
    logits = np.zeros(16)
    g = philox.gumbel_noise(16, 1, 2, 3, 4)
    t, gap = sampler.sample(logits, 1.0, 1, 2, 3, 4)
    order = np.argsort(-g)
    assert t == order[0] and gap == pytest.approx(g[order[0]] - g[order[1]])
    big = np.zeros(16); big[[5, 9]] = 1e18    # the noise is absorbed: an exact tie between ids 5 and 9
    t, gap = sampler.sample(big, 1.0, 1, 2, 3, 4)
    assert t == 5 and gap == 0.0
