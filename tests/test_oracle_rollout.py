"""Pins for the oracle's attention rollout (Eq. 6-9): hand-worked rationals, closed forms, invariants."""
import os

import numpy as np
import pytest

from oracle import rollout

GOLD = os.path.join(os.path.dirname(__file__), "golden", "rollout_2x2.txt")


def _golden():
    out = {}
    with open(GOLD) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            parts = line.split()
            out[parts[0]] = np.array([float(x) for x in parts[1:]])
    return out


def _stochastic(rng, n, L, peaked=False):
    a = rng.random((n, L)) ** (6 if peaked else 1)
    return a / a.sum(axis=1, keepdims=True)


@pytest.mark.parametrize("fn", [rollout.literal, rollout.chain])
def test_hand_worked_examples(fn):
    g = _golden()
    a1 = np.array([[0.5, 0.5], [1.0, 0.0]]); a2 = np.array([[0.0, 1.0], [0.25, 0.75]])
    np.testing.assert_allclose(fn([a1, a2], np.array([0, 1]), 2), g["c_two_layers"], atol=1e-15)
    np.testing.assert_allclose(fn([np.array([[0.25, 0.75]])], np.array([0]), 2), g["c_one_row"], atol=1e-15)


@pytest.mark.parametrize("seed", range(8))
def test_chain_equals_literal_and_mass_is_conserved(seed):
    rng = np.random.default_rng(seed)
    L = int(rng.integers(2, 120)); N = int(rng.integers(1, 6))
    n = int(rng.integers(0, L + 1))
    S = np.sort(rng.choice(L, n, replace=False))
    abar = [_stochastic(rng, n, L, peaked=bool(seed % 2)) for _ in range(N)]
    lit = rollout.literal(abar, S, L)
    ch = rollout.chain(abar, S, L)
    np.testing.assert_allclose(ch, lit, rtol=0, atol=1e-12)
    assert abs(lit.sum() - L) < 1e-9                       # every W is row-stochastic
    off = np.setdiff1d(np.arange(L), S)
    assert np.all(lit[off] >= 1 - 1e-12) and np.all(lit[S] >= 2.0 ** -N - 1e-12)


def test_single_layer_closed_form():
    rng = np.random.default_rng(11)
    L, n = 50, 17
    S = np.sort(rng.choice(L, n, replace=False))
    A = _stochastic(rng, n, L)
    want = np.ones(L); want[S] = 0.5
    want += 0.5 * A.sum(axis=0)
    np.testing.assert_allclose(rollout.literal([A], S, L), want, atol=1e-13)
    np.testing.assert_allclose(rollout.chain([A], S, L), want, atol=1e-13)


@pytest.mark.parametrize("n,L,N", [(5, 40, 1), (13, 64, 4), (64, 64, 3), (1, 9, 7)])
def test_uniform_attention_closed_form(n, L, N):
    S = np.arange(0, 2 * n, 2) if 2 * n <= L else np.arange(n)
    abar = [np.full((n, L), 1.0 / L) for _ in range(N)]
    rho = 0.5 + n / (2.0 * L)
    want = np.full(L, 1.0 + (n * (1 - rho ** N) / (L - n) if n < L else 0.0))
    want[S] = rho ** N
    for fn in (rollout.literal, rollout.chain):
        np.testing.assert_allclose(fn(abar, S, L), want, atol=1e-12)


def test_no_selected_rows_is_the_identity_rollout():
    np.testing.assert_array_equal(rollout.literal([np.zeros((0, 7))] * 3, np.zeros(0, int), 7), np.ones(7))
    np.testing.assert_array_equal(rollout.chain([np.zeros((0, 7))] * 3, np.zeros(0, int), 7), np.ones(7))
