"""Pins for the oracle's whole step: the two bracketing cases (all rows / no rows), the
single-layer exactness of a partial update, and which cache rows may change."""
import copy

import numpy as np
import pytest
import torch

from oracle import step as ostep
from paper_2509_23094_b200 import inputs
from test_oracle_model import torch_full_forward


def _setup(shape, L=40, prompt=24, n_masked=10, seed=0, batch=1):
    wl = inputs.Workload("t", shape, batch, L, prompt, n_masked, "random", 4, 0.5, seed=seed)
    w = inputs.make_weights(shape, seed=seed, gain_jitter=0.05, std=0.05)
    mask = inputs.make_mask(wl)
    tok = inputs.make_tokens(wl, mask)
    h0 = inputs.make_h0(w["embed"], tok)
    st = ostep.OracleState(shape.n_layers, batch, L, shape.n_kv_heads, shape.head_dim)
    return wl, w, ostep.weights_to_f64(w), mask.numpy(), h0, st


@pytest.mark.parametrize("shape", [inputs.TOY, inputs.TOY_GQA])
def test_select_all_equals_the_no_cache_forward(shape):
    wl, w, wf, mask, h0, st = _setup(shape, batch=2)
    r = ostep.oracle_step(st, wf, shape, h0.double().numpy(), mask, k=10 ** 6, p=1.0)
    for b in range(2):
        assert r.sel[b].tolist() == list(range(wl.seq_len))
        xt, Ks, Vs, As = torch_full_forward(w, shape, h0[b].double())
        np.testing.assert_allclose(r.hidden[b], xt.numpy(), rtol=1e-9, atol=1e-10)
        for l in range(shape.n_layers):
            np.testing.assert_allclose(st.Kc[l, b], Ks[l].numpy(), rtol=1e-9, atol=1e-11)
        assert r.lm_rows[b].tolist() == np.flatnonzero(mask[b]).tolist()
        assert abs(float(st.c[b].sum()) - wl.seq_len) < 1e-3
        # confidence only ever written for masked rows
        assert np.all(st.conf[b][mask[b] == 0] == 0) and np.all(st.conf[b][mask[b] == 1] > 0)


def test_select_none_changes_nothing():
    shape = inputs.TOY_GQA
    wl, w, wf, mask, h0, st = _setup(shape)
    h = h0.double().numpy()
    ostep.oracle_step(st, wf, shape, h, mask, k=10 ** 6, p=1.0)
    before = copy.deepcopy(st)
    r = ostep.oracle_step(st, wf, shape, h, mask, k=0, p=0.0)
    assert r.sel[0].size == 0
    for name in ("Kc", "Vc", "conf", "pred", "c"):
        assert np.array_equal(getattr(st, name), getattr(before, name)), name


def test_single_layer_partial_step_reproduces_the_prefill_rows():
    shape = inputs.TOY
    wl, w, wf, mask, h0, st = _setup(shape, L=64, prompt=32, n_masked=16)
    h = h0.double().numpy()
    full = ostep.oracle_step(st, wf, shape, h, mask, k=10 ** 6, p=1.0)
    K0, V0, conf0 = st.Kc.copy(), st.Vc.copy(), st.conf.copy()
    part = ostep.oracle_step(st, wf, shape, h, mask, k=4, p=0.5)
    S = part.sel[0]
    assert 0 < S.size < 64 and len(part.m_star[0]) == 4
    np.testing.assert_allclose(part.hidden[0], full.hidden[0][S], rtol=0, atol=1e-12)
    np.testing.assert_allclose(st.Kc, K0, rtol=0, atol=1e-13)
    np.testing.assert_allclose(st.Vc, V0, rtol=0, atol=1e-13)
    np.testing.assert_allclose(st.conf, conf0, rtol=0, atol=1e-7)


def test_partial_step_on_a_deep_model_touches_only_selected_cache_rows():
    shape = inputs.TOY_GQA
    wl, w, wf, mask, h0, st = _setup(shape, L=48, prompt=24, n_masked=12, seed=2)
    h = h0.double().numpy()
    ostep.oracle_step(st, wf, shape, h, mask, k=10 ** 6, p=1.0)
    # a decoded position changes its embedding: its neighbours' deeper K/V go stale
    h2 = h.copy(); h2[0, 30] = h[0, 5]; mask2 = mask.copy(); mask2[0, 30] = 0
    K0, V0 = st.Kc.copy(), st.Vc.copy()
    stale = copy.deepcopy(st)
    part = ostep.oracle_step(st, wf, shape, h2, mask2, k=3, p=0.3, forced=[[30]])
    S = part.sel[0]; rest = np.setdiff1d(np.arange(48), S)
    assert 30 in S and rest.size > 0
    assert np.array_equal(st.Kc[:, 0, rest], K0[:, 0, rest]) and np.array_equal(st.Vc[:, 0, rest], V0[:, 0, rest])
    # layer 1 K/V depend on the row's own input only: selected rows now hold the exact full-forward values
    full = ostep.OracleState(shape.n_layers, 1, 48, shape.n_kv_heads, shape.head_dim)
    ostep.oracle_step(full, wf, shape, h2, mask2, k=10 ** 6, p=1.0)
    np.testing.assert_allclose(st.Kc[0, 0, S], full.Kc[0, 0, S], rtol=0, atol=1e-12)
    # deeper layers are an approximation (stale keys of unselected rows), so they differ, but not wildly
    diff = np.abs(st.Kc[2, 0, S] - full.Kc[2, 0, S]).max()
    assert 1e-9 < diff < 0.5 * np.abs(full.Kc[2, 0, S]).max()
    # rollout through the step: literal dense product agrees with the chain
    st_lit = stale
    ostep.oracle_step(st_lit, wf, shape, h2, mask2, k=3, p=0.3, forced=[[30]], rollout_literal=True)
    np.testing.assert_allclose(st_lit.c, st.c, rtol=0, atol=1e-6)
    assert abs(float(st.c.sum()) - 48) < 1e-3


def test_repeated_select_all_steps_are_idempotent():
    shape = inputs.TOY_GQA
    wl, w, wf, mask, h0, st = _setup(shape)
    h = h0.double().numpy()
    a = ostep.oracle_step(st, wf, shape, h, mask, k=10 ** 6, p=1.0)
    c1 = st.c.copy()
    b = ostep.oracle_step(st, wf, shape, h, mask, k=10 ** 6, p=1.0)
    np.testing.assert_allclose(a.hidden[0], b.hidden[0], atol=1e-13)
    np.testing.assert_array_equal(c1, st.c)


def test_commit_rules():
    from oracle import decode
    mask = np.zeros(200, dtype=np.uint8); mask[100:] = 1
    conf = np.zeros(200, dtype=np.float32)
    conf[[100, 120, 150]] = [0.5, 0.9, 0.95]
    elig = [100, 120, 150, 160]
    assert decode.commit(mask, conf, elig, rule=0) == ([150], 150)                # highest confidence
    assert decode.commit(mask, conf, elig, rule=1) == ([100], 100)                # next to the known prefix wins
    assert decode.commit(mask, conf, elig, rule=2, threshold=0.8) == ([120, 150], 150)
    assert decode.commit(mask, conf, elig, rule=2, threshold=0.99) == ([150], 150)
    assert decode.commit(mask, conf, [5, 7], rule=0) == ([], -1)                   # known positions are not eligible
    conf[[120, 150]] = 0.9
    assert decode.commit(mask, conf, elig, rule=0) == ([120], 120)                # tie: lower position
