"""Counter-based random numbers for the sampler: Philox4x32-10, uniforms and Gumbel noise.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).

The paper samples rollouts at temperature 1.0 with top_p = 1.0 (Section 4.2,
"Training Details"): an exact draw from softmax(logits / T).  It says nothing about
the random number generator.  The reading taken here: Philox4x32 with 10 rounds as
published by Salmon, Moraes, Dror and Shaw ("Parallel random numbers: as easy as
1, 2, 3", SC'11) -- two 32x32->64 multiplies per round by the constants
0xD2511F53 and 0xCD9E8D57, a word permutation with key injection, and a Weyl key
schedule with increments 0x9E3779B9 and 0xBB67AE85.

Layout for the sampler (one 128-bit block serves four vocabulary ids):
    key     = (seed low 32 bits, seed high 32 bits)
    counter = (v >> 2, step, rollout, prompt)
    word    = output word (v & 3)
    u       = ((word >> 9) + 0.5) * 2^-23        in (0, 1), exact in float32
    g       = -ln(-ln u)                          standard Gumbel

Pins: the paper fixes nothing here, so the generator is pinned to an independent
library implementation of the same published algorithm (Triton's `philox_impl`
run by its CPU interpreter) plus distribution tests of u and g.
"""
from __future__ import annotations

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint64(0x9E3779B9)
_W1 = np.uint64(0xBB67AE85)
_MASK = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten Philox rounds on arrays of 32-bit words (held in uint64).  Returns four uint32 arrays."""
    c0, c1, c2, c3 = np.broadcast_arrays(*(np.asarray(c, dtype=np.uint64) & _MASK for c in (c0, c1, c2, c3)))
    k0 = np.uint64(int(k0) & 0xFFFFFFFF)
    k1 = np.uint64(int(k1) & 0xFFFFFFFF)
    for r in range(10):
        if r > 0:
            k0 = (k0 + _W0) & _MASK
            k1 = (k1 + _W1) & _MASK
        p0 = _M0 * c0          # < 2^64, no overflow
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _S32, p0 & _MASK
        hi1, lo1 = p1 >> _S32, p1 & _MASK
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return tuple(c.astype(np.uint32) for c in (c0, c1, c2, c3))


def vocab_words(vocab: int, seed: int, prompt: int, rollout: int, step: int) -> np.ndarray:
    """The 32-bit random word of every vocabulary id for one (prompt, rollout, step) draw."""
    n_blocks = (vocab + 3) // 4
    blk = np.arange(n_blocks, dtype=np.uint64)
    w = philox4x32_10(blk, step, rollout, prompt, seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    return np.stack(w, axis=1).reshape(-1)[:vocab]


def uniform_from_word(word: np.ndarray) -> np.ndarray:
    """u = ((word >> 9) + 1/2) / 2^23, strictly inside (0, 1)."""
    return ((np.asarray(word, dtype=np.uint32) >> np.uint32(9)).astype(np.float64) + 0.5) * (2.0 ** -23)


def gumbel_from_word(word: np.ndarray) -> np.ndarray:
    u = uniform_from_word(word)
    return -np.log(-np.log(u))


def gumbel_noise(vocab: int, seed: int, prompt: int, rollout: int, step: int) -> np.ndarray:
    return gumbel_from_word(vocab_words(vocab, seed, prompt, rollout, step))
