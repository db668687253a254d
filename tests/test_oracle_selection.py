"""Pins for the oracle's selection stage (Eq. 3-4 and the top-p rule of Section 4.2).

Each check holds the oracle against something that is not the oracle: a closed
form, a hand-expanded value from tests/golden, a library convolution, a
rank-counting definition of top-k, an exhaustive search over subsets for top-p.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import selection as sel

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            parts = line.split()
            out[parts[0]] = [float(x) for x in parts[1:]]
    return out


def test_density_closed_forms():
    g = _golden("density_closed_forms.txt")
    mask = np.zeros(401, dtype=np.uint8); mask[200] = 1
    assert abs(sel.density(mask, 10.0)[200] - g["interior"][0]) < 1e-9
    mask = np.zeros(400, dtype=np.uint8); mask[200:] = 1
    D = sel.density(mask, 10.0)
    assert abs(D[200] - g["edge"][0]) < 1e-9
    # deeper into a fully masked suffix the density can only fall
    assert np.all(np.diff(D[200:]) <= 0) and D[399] < 1e-12
    mask = np.array([0, 0, 1, 0], dtype=np.uint8)
    assert abs(sel.density(mask, 1.0)[2] - g["tiny"][0]) < 1e-12
    assert np.all(sel.density(mask, 1.0)[[0, 1, 3]] == 0)


def test_density_is_a_convolution_of_the_known_indicator():
    rng = np.random.default_rng(1)
    for L, sigma in [(37, 3.0), (300, 10.0), (129, 40.0)]:
        mask = (rng.random(L) < 0.4).astype(np.uint8)
        kern = np.exp(-np.arange(-(L - 1), L, dtype=np.float64) ** 2 / (2 * sigma * sigma))
        conv = np.convolve((mask == 0).astype(np.float64), kern)[L - 1: 2 * L - 1]
        D = sel.density(mask, sigma)
        np.testing.assert_allclose(D[mask == 1], conv[mask == 1], rtol=1e-12, atol=1e-12)


def test_fixed_point_density_stays_within_its_bound_of_eq3():
    rng = np.random.default_rng(2)
    for L in (64, 500, 1024):
        mask = (rng.random(L) < 0.3).astype(np.uint8)
        D = sel.density(mask, 10.0)
        Dq = np.array(sel.density_q30(mask, 10.0), dtype=np.float64) / sel.Q30
        assert np.max(np.abs(D - Dq)) <= L * 2.0 ** -31


def test_phi_table_shape_and_rounding_margin():
    tab = sel.phi_table_q30(10.0, 200)
    assert tab[0] == 1 << 30
    assert all(a >= b for a, b in zip(tab, tab[1:]))
    assert tab[65] > 0 and tab[66] == 0                      # window of +-65 at sigma = 10
    # no entry sits close enough to a rounding boundary for a last-bit difference in exp() to matter
    for r in range(66):
        x = math.exp(-(r * r) / 200.0) * (1 << 30)
        assert abs((x % 1.0) - 0.5) > 1e-6


def test_stage1_keys_one_fp32_multiply():
    mask = np.zeros(300, dtype=np.uint8); mask[150] = 1
    conf = np.full(300, 0.37, dtype=np.float32)
    key = sel.stage1_keys(mask, conf, 10.0)
    want = np.float32(24.066282746310002) * np.float32(0.37)
    assert abs(float(key[150]) - float(want)) <= 4e-6 and key.dtype == np.float32
    assert np.count_nonzero(key) == 1


def _rank_topk(mask, key, k):
    """top-k by counting, for each member, how many members beat it."""
    members = np.flatnonzero(mask)
    out = []
    for i in members:
        beat = sum(1 for j in members if key[j] > key[i] or (key[j] == key[i] and j < i))
        if beat < k:
            out.append(i)
    return np.array(out, dtype=np.int64)


@pytest.mark.parametrize("seed", range(12))
def test_stage1_topk_matches_rank_counting(seed):
    rng = np.random.default_rng(seed)
    L = int(rng.integers(1, 200))
    mask = (rng.random(L) < rng.random()).astype(np.uint8)
    levels = int(rng.integers(2, 50))
    key = (np.floor(rng.random(L) * levels) / levels).astype(np.float32)    # many ties
    nm = int(mask.sum())
    for k in {0, 1, max(nm - 1, 0), nm, nm + 1, int(rng.integers(0, L + 1))}:
        got = sel.stage1_select(mask, None, k, 10.0, key=key)
        np.testing.assert_array_equal(got, _rank_topk(mask, key, k))
        assert len(got) == min(k, nm)


def test_stage1_uses_density_times_confidence():
    # two masked positions with equal confidence: the one next to known tokens wins;
    # with a much higher confidence the far one wins.
    mask = np.zeros(200, dtype=np.uint8); mask[100:] = 1
    conf = np.full(200, 0.5, dtype=np.float32)
    assert sel.stage1_select(mask, conf, 1, 10.0).tolist() == [100]
    conf[130] = 0.5 * 1000.0
    assert sel.stage1_select(mask, conf, 1, 10.0).tolist() == [130]
    assert sel.stage1_select(mask, conf, 2, 10.0).tolist() == [100, 130]


def _exhaustive_top_p(c, cand, p):
    """Smallest subset of the candidates whose exact mass exceeds p * total (ties by position)."""
    idx = [int(j) for j in np.flatnonzero(cand)]
    tot = sum(Fraction(float(c[j])) for j in idx)
    pf = Fraction(float(np.float32(p)))
    if pf <= 0:
        return []
    for m in range(1, len(idx) + 1):
        best = None
        for sub in itertools.combinations(idx, m):
            mass = sum(Fraction(float(c[j])) for j in sub)
            if mass > pf * tot:
                # among equally small sets the rule keeps the heaviest, then the lowest positions
                keyv = (-mass, sub)
                if best is None or keyv < best[0]:
                    best = (keyv, sub)
        if best is not None:
            return sorted(best[1])
    return idx


@pytest.mark.parametrize("seed", range(10))
def test_stage2_top_p_matches_exhaustive_search(seed):
    rng = np.random.default_rng(100 + seed)
    L = int(rng.integers(1, 11))
    c = (rng.integers(0, 64, L) / 64.0).astype(np.float32)          # dyadic: fixed point is exact
    cand = rng.random(L) < 0.8
    for p in (0.0, 0.015625, 0.25, 0.5, 0.75, 0.9375, 1.0, 2.0):
        got = sel.stage2_select(c, cand, p).tolist()
        assert got == _exhaustive_top_p(c, cand, p), (c, cand, p)


@pytest.mark.parametrize("seed", range(8))
def test_stage2_prefix_invariants(seed):
    rng = np.random.default_rng(200 + seed)
    L = int(rng.integers(5, 400))
    c = rng.random(L).astype(np.float32) ** 4
    cand = rng.random(L) < 0.7
    q = {j: int(math.floor(float(c[j]) * 2 ** 32)) for j in np.flatnonzero(cand)}
    T = sum(q.values())
    for p in (1e-6, 0.1, 0.5, 0.9, 1 - 2.0 ** -24):
        U = sel.stage2_select(c, cand, p).tolist()
        assert all(cand[j] for j in U) and len(U) >= 1
        worst = min(U, key=lambda j: (float(c[j]), -j))
        outside = [j for j in q if j not in U]
        # a prefix of the sorted order: nothing outside beats the weakest member
        assert all((float(c[j]), -j) < (float(c[worst]), -worst) for j in outside)
        mass = sum(q[j] for j in U)
        pf = float(np.float32(p))
        assert float(mass) > pf * float(T)
        assert not (float(mass - q[worst]) > pf * float(T))             # minimal
    assert sel.stage2_select(c, cand, 1.0).tolist() == np.flatnonzero(cand).tolist()
    assert sel.stage2_select(c, cand, 0.0).size == 0
    assert sel.stage2_select(c, cand, -1.0).size == 0


def test_stage2_ties_prefer_lower_positions_and_bad_scores_count_as_zero():
    c = np.array([0.5, 0.5, 0.5, 0.5], dtype=np.float32)
    cand = np.ones(4, dtype=bool)
    assert sel.stage2_select(c, cand, 0.3).tolist() == [0, 1]
    c = np.array([np.nan, -1.0, 0.25, 0.75], dtype=np.float32)
    assert sel.stage2_select(c, cand, 0.5).tolist() == [3]
    assert sel.stage2_select(c, cand, 0.8).tolist() == [2, 3]
    c = np.array([np.inf, -np.inf, 0.25, 0.75], dtype=np.float32)
    assert sel.stage2_select(c, cand, 0.5).tolist() == [3]
    c = np.array([1e30, 262144.0, 1.0, 1.0], dtype=np.float32)          # capped: the two large ones tie
    assert sel.stage2_select(c, cand, 0.4).tolist() == [0]
    assert sel.stage2_select(c, cand, 0.6).tolist() == [0, 1]


def test_select_rows_union_and_candidate_modes():
    L = 64
    mask = np.zeros(L, dtype=np.uint8); mask[40:56] = 1
    rng = np.random.default_rng(5)
    conf = rng.random(L).astype(np.float32)
    c = rng.random(L).astype(np.float32)
    S, m_star, u = sel.select_rows(mask, conf, c, 4, 0.5, 10.0, forced=[3, 41])
    assert len(m_star) == 4 and all(mask[i] for i in m_star)
    assert all(not mask[j] for j in u)
    assert S.tolist() == sorted(set(m_star.tolist()) | set(u.tolist()) | {3, 41})
    S1, m1, u1 = sel.select_rows(mask, conf, c, 4, 0.5, 10.0, stage2_candidates=1)
    assert m1.tolist() == m_star.tolist() and not (set(u1.tolist()) & set(m1.tolist()))
    # select all / select none
    S, _, _ = sel.select_rows(mask, conf, c, L, 1.0, 10.0)
    assert S.tolist() == list(range(L))
    S, _, _ = sel.select_rows(mask, conf, c, 0, 0.0, 10.0)
    assert S.size == 0


def test_stage1_block_restriction():
    mask = np.zeros(128, dtype=np.uint8); mask[64:] = 1
    conf = np.linspace(0.1, 0.9, 128).astype(np.float32)          # later positions are more confident
    whole = sel.stage1_select(mask, conf, 4, 10.0)
    blocked = sel.stage1_select(mask, conf, 4, 10.0, block=(64, 96))
    assert all(64 <= i < 96 for i in blocked) and len(blocked) == 4
    assert blocked.tolist() == _rank_topk(np.where(np.arange(128) < 96, mask, 0), sel.stage1_keys(mask, conf, 10.0), 4).tolist()
    assert sel.stage1_select(mask, conf, 4, 10.0, block=(5, 5)).tolist() == whole.tolist()     # empty block = no restriction
    assert sel.stage1_select(mask, conf, 100, 10.0, block=(64, 70)).tolist() == list(range(64, 70))
    S, m_star, u = sel.select_rows(mask, conf, np.ones(128, np.float32), 4, 0.1, 10.0, block=(64, 96))
    assert m_star.tolist() == blocked.tolist() and all(j < 64 for j in u)
