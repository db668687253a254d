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


def test_truncated_rollout_uses_the_first_layers_of_the_same_step():
    """The lightweight rollout variant of the paper's limitations section ("first five layers"): with
    rollout_layers = n the scores are Eq. 6-9 over layers 1..n of this step, not over the last n and not
    over all of them.  Pinned against the chain and the literal L x L product applied to the step's own
    head-averaged attention."""
    from oracle import rollout as orollout
    shape = inputs.TOY_GQA                                   # three layers
    assert shape.n_layers == 3
    wl, w, wf, mask, h0, st = _setup(shape, L=48, prompt=24, n_masked=12)
    h = h0.double().numpy()
    ostep.oracle_step(st, wf, shape, h, mask, k=10 ** 6, p=1.0)
    base = copy.deepcopy(st)
    L = wl.seq_len
    got = {}
    for depth in (0, 1, 2, 3, 7):
        s = copy.deepcopy(base)
        r = ostep.oracle_step(s, wf, shape, h, mask, k=4, p=0.4, rollout_layers=depth)
        S, abar = r.sel[0], r.abar[0]
        assert 0 < S.size < L and len(abar) == 3
        n = depth if 0 < depth < 3 else 3
        first = orollout.chain(abar[:n], S, L)
        np.testing.assert_allclose(s.c[0], first, rtol=1e-6, atol=1e-7)          # c is stored as fp32
        np.testing.assert_allclose(first, orollout.literal(abar[:n], S, L), rtol=1e-12, atol=1e-12)
        if n < 3:
            last = orollout.chain(abar[3 - n:], S, L)
            assert np.max(np.abs(s.c[0] - last)) > 1e-4                          # not the last n layers
            assert np.max(np.abs(s.c[0] - orollout.chain(abar, S, L))) > 1e-4    # and not all of them
        # the depth does not touch anything but c
        for name in ("Kc", "Vc", "conf", "pred"):
            assert np.array_equal(getattr(s, name), getattr(got.setdefault("ref", s), name)), name
        got[depth] = s.c[0].copy()
    np.testing.assert_array_equal(got[0], got[3])
    np.testing.assert_array_equal(got[7], got[3])
    assert abs(float(got[1].sum()) - L) < 1e-3 and abs(float(got[2].sum()) - L) < 1e-3


def _torch_subset_step(w, shape, h_rows, S, Ks, Vs):
    """An independently written torch fp64 version of Eq. 5 on a deep model: the layers run on the rows S
    only; every layer first overwrites rows S of its K/V cache (index assignment), then lets the S queries
    attend to all L cached keys through the library's scaled_dot_product_attention.  Ks / Vs: per layer
    [L][Hkv][Dh] tensors holding the (stale) cache, updated in place.  Returns (x_S, head-mean attention per layer)."""
    import math
    import torch.nn.functional as F
    Hq, Hkv, Dh = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    n = len(S)
    Si = torch.as_tensor(np.asarray(S), dtype=torch.long)

    def norm(x, g):
        return x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + shape.rms_eps) * g.double()

    inv = 1.0 / (shape.rope_base ** (torch.arange(0, Dh, 2, dtype=torch.float64) / Dh))
    fr = torch.outer(Si.double(), inv)                                     # angles at the rows' absolute positions
    cos, sin = torch.cat([fr, fr], -1).cos()[:, None], torch.cat([fr, fr], -1).sin()[:, None]      # [n][1][Dh]

    def rot(t):
        return t * cos + torch.cat([-t[..., Dh // 2:], t[..., : Dh // 2]], dim=-1) * sin

    x = h_rows.clone()
    As = []
    for l, lyr in enumerate(w["layers"]):
        a = norm(x, lyr["g_attn"])
        qkv = F.linear(a, lyr["wqkv"].double(), None if lyr["bqkv"] is None else lyr["bqkv"].double())
        q, k, v = qkv.split([Hq * Dh, Hkv * Dh, Hkv * Dh], dim=-1)
        q = rot(q.view(n, Hq, Dh)); k = rot(k.view(n, Hkv, Dh)); v = v.view(n, Hkv, Dh)
        Ks[l][Si] = k; Vs[l][Si] = v                                       # fresh rows in, everything else stale
        kr = Ks[l].transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)     # [Hq][L][Dh]
        vr = Vs[l].transpose(0, 1).repeat_interleave(Hq // Hkv, dim=0)
        qh = q.transpose(0, 1)                                             # [Hq][n][Dh]
        o = F.scaled_dot_product_attention(qh[None], kr[None], vr[None])[0]
        As.append(torch.softmax(qh @ kr.transpose(1, 2) / math.sqrt(Dh), dim=-1).mean(0))
        x = x + F.linear(o.transpose(0, 1).reshape(n, Hq * Dh), lyr["wo"].double())
        m = norm(x, lyr["g_ffn"])
        x = x + F.linear(F.silu(F.linear(m, lyr["w_gate"].double())) * F.linear(m, lyr["w_up"].double()), lyr["w_down"].double())
    return x, As


@pytest.mark.parametrize("shape", [inputs.TOY_GQA, inputs.TOY_HD128])
def test_strict_subset_step_on_a_deep_model_matches_an_independent_torch_version(shape):
    """The approximate step itself (a strict subset of rows, stale keys elsewhere, two or more layers) held
    against a second implementation that shares nothing with the oracle but the weights: hidden states, the
    rewritten cache rows, the head-averaged attention, the confidences and, through the chain, c."""
    from oracle import rollout as orollout
    assert shape.n_layers >= 2
    L = 48
    wl, w, wf, mask, h0, st = _setup(shape, L=L, prompt=24, n_masked=12, seed=5)
    h = h0.double().numpy()
    ostep.oracle_step(st, wf, shape, h, mask, k=10 ** 6, p=1.0)
    # two decoded positions change their embeddings, so the cache that the partial step meets is stale
    h2 = h.copy(); mask2 = mask.copy()
    dec = np.flatnonzero(mask[0])[[1, 4]]
    h2[0, dec[0]] = h[0, 3]; h2[0, dec[1]] = h[0, 7]; mask2[0, dec] = 0
    Ks = [torch.from_numpy(st.Kc[l, 0].copy()) for l in range(shape.n_layers)]
    Vs = [torch.from_numpy(st.Vc[l, 0].copy()) for l in range(shape.n_layers)]
    part = ostep.oracle_step(st, wf, shape, h2, mask2, k=3, p=0.35, forced=[list(dec)])
    S = part.sel[0]
    assert 3 < S.size < L and all(p in S for p in dec)
    xt, As = _torch_subset_step(w, shape, torch.from_numpy(h2[0][S]), S, Ks, Vs)
    np.testing.assert_allclose(part.hidden[0], xt.numpy(), rtol=1e-9, atol=1e-10)
    for l in range(shape.n_layers):
        np.testing.assert_allclose(st.Kc[l, 0], Ks[l].numpy(), rtol=1e-9, atol=1e-11)      # rows of S fresh, the rest untouched
        np.testing.assert_allclose(st.Vc[l, 0], Vs[l].numpy(), rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(part.abar[0][l], As[l].numpy(), rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(st.c[0], orollout.literal([a.numpy() for a in As], S, L), rtol=1e-6, atol=1e-6)
    # Eq. 1 on the selected rows that are still masked, from the torch hidden states and library softmax
    lm = part.lm_rows[0]
    assert lm.size and np.all(mask2[0][lm] == 1)
    loc = np.searchsorted(S, lm)
    xm = xt[loc]
    xm = xm * torch.rsqrt(xm.pow(2).mean(-1, keepdim=True) + shape.rms_eps) * w["g_final"].double()
    pr = torch.softmax(xm @ w["w_lm"].double().t(), dim=-1)
    np.testing.assert_allclose(st.conf[0, lm], pr.max(dim=-1).values.numpy(), rtol=1e-6)
    np.testing.assert_array_equal(st.pred[0, lm], pr.argmax(dim=-1).numpy())
