"""Pins for oracle/stats.py: closed forms, invariants the paper states, values it prints, brute force."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import stats

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _one_group(r):
    r = np.asarray(r, dtype=np.float64)
    return r, np.array([0]), np.array([len(r)])


@pytest.mark.parametrize("n", [1, 2, 4, 8, 16, 64, 128])
def test_binary_variance_is_p_one_minus_p(n):
    # Section 3.3: for binary rewards Var[r | q] = p (1 - p).
    for m in range(n + 1):
        r, s, c = _one_group([1.0] * m + [0.0] * (n - m))
        nn, mm, mean, var = stats.group_stats(r, s, c)
        p = Fraction(m, n)
        assert nn[0] == n and mm[0] == m
        assert mean[0] == pytest.approx(float(p), abs=1e-15)
        assert var[0] == pytest.approx(float(p * (1 - p)), abs=1e-15)


def test_group_stats_textbook_and_ragged():
    rng = np.random.default_rng(0)
    r = rng.normal(size=37)
    start = np.array([0, 5, 5, 20])
    count = np.array([5, 0, 15, 17])
    n, m, mean, var = stats.group_stats(r, start, count)
    for g in range(4):
        seg = r[start[g]:start[g] + count[g]]
        assert n[g] == len(seg)
        if len(seg):
            assert mean[g] == pytest.approx(np.mean(seg), abs=1e-14)
            assert var[g] == pytest.approx(np.var(seg), abs=1e-14)      # numpy's var is the population form (Eq. 3)
            assert var[g] != pytest.approx(np.var(seg, ddof=1), abs=1e-6)


@pytest.mark.parametrize("G", [2, 4, 8, 16, 64, 128])
def test_advantage_invariants_binary(G):
    for m in range(G + 1):
        r, s, c = _one_group([1.0] * m + [0.0] * (G - m))
        a = stats.grpo_advantage(r, s, c)
        if m in (0, G):
            assert np.all(a == 0.0)          # zero-variance group: zero advantage (Section 1)
            continue
        p = m / G
        assert abs(a.sum()) < 1e-10          # sum A_i = 0 (Proposition 3.1)
        assert a @ a == pytest.approx(G, rel=1e-12)
        assert a[0] == pytest.approx(math.sqrt((1 - p) / p), rel=1e-12)
        assert a[-1] == pytest.approx(-math.sqrt(p / (1 - p)), rel=1e-12)
        s_plus = a[r >= r.mean()].sum()
        assert s_plus <= G / 2 + 1e-9        # Lemma A.1
        if 2 * m == G:
            assert np.allclose(np.abs(a), 1.0) and s_plus == pytest.approx(G / 2)   # tight at p = 1/2


def test_advantage_mass_identity_and_bound_real_rewards():
    rng = np.random.default_rng(1)
    for G in (3, 7, 16):
        r, s, c = _one_group(rng.normal(size=G))
        a = stats.grpo_advantage(r, s, c)
        d = r - r.mean()
        sigma = math.sqrt(np.mean(d * d))
        s_plus = a[d >= 0].sum()
        assert s_plus == pytest.approx(np.abs(d).sum() / (2 * sigma), rel=1e-12)     # Appendix A.3 identity
        assert s_plus <= G / 2
        assert abs(a.sum()) < 1e-10
        assert np.allclose(a, (r - np.mean(r)) / np.std(r))


def test_advantage_respects_status_and_layout():
    r = np.array([1, 0, 9, 9, 0, 1, 1, 0, 5, 5], dtype=np.float64)
    start, count = np.array([0, 4, 8]), np.array([2, 4, 2])
    a = stats.grpo_advantage(r, start, count, status=np.array([stats.COMMIT, stats.SKIP_EASY, stats.COMMIT]))
    assert np.allclose(a[:2], [1, -1])
    assert np.all(a[2:] == 0)
    a = stats.grpo_advantage(r, start, count)
    assert np.allclose(a[4:8], [-1, 1, 1, -1]) and np.all(a[2:4] == 0) and np.all(a[8:] == 0)


def test_filter_edges_paper_defaults_k8():
    # Section 4.2: skipped if success rate > 0.75, deferred if < 0.125, evicted only when all pilot rollouts are correct.
    k = 8
    m = np.arange(k + 1)
    st, extra, ev, nsel, total = stats.allocate(m, np.full(k + 1, k), 0.125, 0.75, 1.0, n_commit=8, b_t=100)
    assert st[0] == stats.DEFER_HARD
    assert all(st[i] == stats.COMMIT for i in range(1, 7))
    assert st[7] == stats.SKIP_EASY and st[8] == stats.SKIP_EASY
    assert list(ev) == [0] * 8 + [1]
    assert list(extra) == [0] + [8] * 6 + [0, 0]
    assert nsel == 6 and total == 9 * k + 6 * 8


def test_filter_brute_force_against_exact_rationals():
    grids = dict(p_upper=[1.0, 0.875, 0.75, 0.625], p_lower=[0.0, 0.125, 0.25, 0.375], p_solve=[0.75, 0.875, 1.0])
    for pu, pl, ps in itertools.product(grids["p_upper"], grids["p_lower"], grids["p_solve"]):   # Section 6.2 grids
        for k in range(1, 17):
            m = np.arange(k + 1)
            st, extra, ev, nsel, total = stats.allocate(m, np.full(k + 1, k), pl, pu, ps, n_commit=3, b_t=10 ** 6)
            for mm in range(k + 1):
                ph = Fraction(mm, k)
                keep = Fraction(pl) <= ph <= Fraction(pu)
                assert (st[mm] == stats.COMMIT) == keep
                assert (st[mm] == stats.DEFER_HARD) == (ph < Fraction(pl))
                assert (st[mm] == stats.SKIP_EASY) == (ph > Fraction(pu))
                assert bool(ev[mm]) == (ph >= Fraction(ps))
            assert total == (k + 1) * k + nsel * 3


def test_commit_cap_and_buffering():
    m = np.array([1, 0, 2, 3, 4, 2, 1])
    n = np.full(7, 4)
    st, extra, ev, nsel, total = stats.allocate(m, n, 0.125, 0.75, 1.0, n_commit=12, b_t=3)
    assert list(st) == [stats.COMMIT, stats.DEFER_HARD, stats.COMMIT, stats.COMMIT, stats.SKIP_EASY,
                        stats.BUFFERED, stats.BUFFERED]
    assert nsel == 3 and extra.sum() == 36 and total == 28 + 36 and list(ev) == [0, 0, 0, 0, 1, 0, 0]
    st, extra, ev, nsel, total = stats.allocate(m, n, 0.125, 0.75, 1.0, n_commit=12, b_t=0)
    assert nsel == 0 and total == 28 and not np.any(st == stats.COMMIT)


def test_keep_and_evict_can_coincide():
    # with p_upper = 1 (Section 6.2 ablation) a fully solved prompt passes the filter and is evicted (Algorithm 1)
    st, extra, ev, nsel, total = stats.allocate(np.array([4]), np.array([4]), 0.125, 1.0, 1.0, 5, 1)
    assert st[0] == stats.COMMIT and ev[0] == 1 and extra[0] == 5


def test_printed_sampling_costs():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "sampling_cost.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 9
    for method, b_t, s, n_pilot, n_commit, sampled, trained in rows:
        b_t, s, n_pilot, n_commit = int(b_t), int(s), int(n_pilot), int(n_commit)
        assert stats.sampling_cost(method, b_t, s, n_pilot, n_commit) == int(sampled)
        assert b_t * (n_pilot + n_commit) == int(trained)
    # the allocation reproduces the PC figure when every commit slot is filled (b_g = 3 b_t survivors or more)
    b_g, b_t = 384, 128
    for n_pilot, n_commit, want in ((32, 96, 24576), (16, 48, 12288), (8, 8, 4096)):
        m = np.full(b_g, n_pilot // 2)
        *_, nsel, total = stats.allocate(m, np.full(b_g, n_pilot), 0.125, 0.75, 1.0, n_commit, b_t)
        assert nsel == b_t and total == want
    # Section 5.3: a PC step generates 1.5x GRPO's rollouts under ample budgets, 2x under limited, DAPO 3x
    assert stats.sampling_cost("pc", 128, 3, 16, 48) / stats.sampling_cost("grpo", 128, 3, 16, 48) == 1.5
    assert stats.sampling_cost("pc", 128, 3, 8, 8) / stats.sampling_cost("grpo", 128, 3, 8, 8) == 2.0
    assert stats.sampling_cost("dapo", 128, 3, 8, 8) / stats.sampling_cost("grpo", 128, 3, 8, 8) == 3.0


def test_statuses_partition_and_budget_conserved_random():
    rng = np.random.default_rng(5)
    for _ in range(50):
        P, k = int(rng.integers(1, 40)), int(rng.integers(1, 33))
        m = rng.integers(0, k + 1, size=P)
        b_t, nc = int(rng.integers(0, P + 2)), int(rng.integers(0, 100))
        st, extra, ev, nsel, total = stats.allocate(m, np.full(P, k), 0.125, 0.75, 1.0, nc, b_t)
        kept = np.sum((m / k >= 0.125) & (m / k <= 0.75))
        assert nsel == min(b_t, kept) == np.sum(st == stats.COMMIT)
        assert np.sum(st == stats.BUFFERED) == kept - nsel
        assert total == P * k + extra.sum() and extra.sum() == nsel * nc
        assert set(np.unique(st)) <= {0, 1, 2, 3}


def test_dapo_filter_is_the_pilot_filter_with_k_equal_n():
    """Section 4.3: DAPO gives every prompt n rollouts and drops all-correct / all-incorrect groups.  That is the pilot
    filter evaluated on the full group with thresholds 1/n and (n-1)/n and nothing left to commit."""
    rng = np.random.default_rng(9)
    for n in (2, 16, 64, 128):
        P = 40
        m = rng.integers(0, n + 1, size=P); m[:3] = [0, n, 1]
        r = np.zeros((P, n)); 
        for p in range(P):
            r[p, :m[p]] = 1.0
        keep = stats.dapo_filter(r.reshape(-1), np.arange(P) * n, np.full(P, n))
        assert list(keep[:3]) == [0, 0, 1]
        st, extra, ev, nsel, total = stats.allocate(m, np.full(P, n), 1.0 / n, (n - 1.0) / n, 1.0, n_commit=0, b_t=P)
        assert np.array_equal(keep == 1, st == stats.COMMIT)
        assert np.array_equal(st == stats.DEFER_HARD, m == 0) and np.array_equal(st == stats.SKIP_EASY, m == n)
        assert total == P * n == stats.sampling_cost("dapo", P, 1, n, 0)       # b_g n rollouts generated
    # GRPO: every prompt of the training batch gets n rollouts, none is filtered
    st, *_ , total = stats.allocate(np.array([0, 3, 8]), np.full(3, 8), 0.0, 1.0, 2.0, 0, 3)
    assert np.all(st == stats.COMMIT) and total == 24 == stats.sampling_cost("grpo", 3, 3, 8, 0)


def test_variance_filter_equals_the_success_rate_filter_for_binary_rewards_and_symmetric_thresholds():
    """Section 3.3: Var[r | q] = p (1 - p), so for binary rewards a variance threshold v is the success-rate band
    [p_lo, 1 - p_lo] with p_lo (1 - p_lo) = v.  Checked for every (m, k) with k a power of two (all values exact)."""
    from oracle import stats as S
    for k in (2, 4, 8, 16, 32):
        for p_lo in (0.125, 0.25, 0.375):
            m = np.arange(k + 1)
            n = np.full(k + 1, k)
            var = (m / k) * (1 - m / k)
            st_v, ex_v, sel_v, tot_v = S.allocate_by_variance(var, n, p_lo * (1 - p_lo), 5, k + 1)
            st_p, ex_p, ev_p, sel_p, tot_p = S.allocate(m, n, p_lo, 1 - p_lo, 2.0, 5, k + 1)
            assert np.array_equal(st_v == S.COMMIT, st_p == S.COMMIT), (k, p_lo)
            assert np.array_equal(ex_v, ex_p) and sel_v == sel_p and tot_v == tot_p
            assert np.all(st_v[st_p != S.COMMIT] == S.LOW_VARIANCE)
    # continuous rewards: the decision is the plain definition, a population variance (numpy) against the threshold
    rng = np.random.default_rng(4)
    r = rng.normal(size=(40, 8)) * rng.uniform(0, 2, size=(40, 1))
    var = r.var(axis=1)
    st, ex, sel, tot = S.allocate_by_variance(var, np.full(40, 8), 0.5, 3, 7)
    kept = np.flatnonzero(var.astype(np.float32) >= 0.5)
    assert np.array_equal(np.flatnonzero(st == S.COMMIT), kept[:7]) and np.array_equal(np.flatnonzero(st == S.BUFFERED), kept[7:])
    assert sel == min(7, len(kept)) and tot == 40 * 8 + sel * 3 and ex.sum() == sel * 3
