"""Pins for the oracle's transformer block and LM head.

The select-all case is an ordinary bidirectional pre-norm transformer forward,
so it is held against an independently written torch fp64 forward that uses
library routines (scaled_dot_product_attention, silu, softmax).  The remaining
checks are closed forms and invariances.
"""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import model, step as ostep
from paper_2509_23094_b200 import inputs


def torch_full_forward(w, shape, h0):
    """Textbook forward over every position of one sequence.  h0: [L][d] torch fp64.
    Returns (final residual stream, per-layer K, per-layer V, per-layer head-mean attention)."""
    L, d = h0.shape
    Hq, Hkv, Dh = shape.n_q_heads, shape.n_kv_heads, shape.head_dim

    def norm(x, g):
        return x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + shape.rms_eps) * g.double()

    inv = 1.0 / (shape.rope_base ** (torch.arange(0, Dh, 2, dtype=torch.float64) / Dh))
    fr = torch.outer(torch.arange(L, dtype=torch.float64), inv)
    emb = torch.cat([fr, fr], dim=-1)
    cos, sin = emb.cos()[None], emb.sin()[None]                    # [1][L][Dh]

    def rot_half(t):
        return torch.cat([-t[..., Dh // 2:], t[..., : Dh // 2]], dim=-1)

    x = h0.clone()
    Ks, Vs, As = [], [], []
    for lyr in w["layers"]:
        a = norm(x, lyr["g_attn"])
        qkv = F.linear(a, lyr["wqkv"].double(), None if lyr["bqkv"] is None else lyr["bqkv"].double())
        q, k, v = qkv.split([Hq * Dh, Hkv * Dh, Hkv * Dh], dim=-1)
        q = q.view(L, Hq, Dh).transpose(0, 1); k = k.view(L, Hkv, Dh).transpose(0, 1)
        v = v.view(L, Hkv, Dh).transpose(0, 1)
        q = q * cos + rot_half(q) * sin
        k = k * cos + rot_half(k) * sin
        Ks.append(k.transpose(0, 1).contiguous()); Vs.append(v.transpose(0, 1).contiguous())
        kr = k.repeat_interleave(Hq // Hkv, dim=0); vr = v.repeat_interleave(Hq // Hkv, dim=0)
        o = F.scaled_dot_product_attention(q[None], kr[None], vr[None])[0]          # no mask: bidirectional
        As.append(torch.softmax(q @ kr.transpose(1, 2) / math.sqrt(Dh), dim=-1).mean(0))
        x = x + F.linear(o.transpose(0, 1).reshape(L, Hq * Dh), lyr["wo"].double())
        m = norm(x, lyr["g_ffn"])
        x = x + F.linear(F.silu(F.linear(m, lyr["w_gate"].double())) * F.linear(m, lyr["w_up"].double()),
                         lyr["w_down"].double())
    return x, Ks, Vs, As


@pytest.mark.parametrize("shape", [inputs.TOY, inputs.TOY_GQA, inputs.TOY_HD128])
def test_select_all_is_the_textbook_forward(shape):
    L = 48
    w = inputs.make_weights(shape, seed=3, gain_jitter=0.1, std=0.05)
    g = torch.Generator().manual_seed(7)
    h0 = (torch.randn(L, shape.d_model, generator=g) * 0.5).to(torch.bfloat16)
    wf = ostep.weights_to_f64(w)
    x = h0.double().numpy()
    pos = np.arange(L)
    Kc = np.zeros((shape.n_layers, L, shape.n_kv_heads, shape.head_dim)); Vc = np.zeros_like(Kc)
    abars = []
    for l in range(shape.n_layers):
        x, ab = model.layer_on_rows(x, pos, Kc[l], Vc[l], wf["layers"][l], shape.n_q_heads,
                                    shape.n_kv_heads, shape.head_dim, shape.rope_base, shape.rms_eps)
        abars.append(ab)
        np.testing.assert_allclose(ab.sum(axis=1), 1.0, atol=1e-12)
    xt, Ks, Vs, As = torch_full_forward(w, shape, h0.double())
    np.testing.assert_allclose(x, xt.numpy(), rtol=1e-9, atol=1e-10)
    for l in range(shape.n_layers):
        np.testing.assert_allclose(Kc[l], Ks[l].numpy(), rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(Vc[l], Vs[l].numpy(), rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(abars[l], As[l].numpy(), rtol=1e-9, atol=1e-12)
    # LM head against library softmax
    conf, pred, logits = model.lm_head_conf(x, wf["g_final"], wf["w_lm"], shape.rms_eps)
    xn = xt * torch.rsqrt(xt.pow(2).mean(-1, keepdim=True) + shape.rms_eps) * w["g_final"].double()
    pt = torch.softmax(F.linear(xn, w["w_lm"].double()), dim=-1)
    np.testing.assert_allclose(conf, pt.max(dim=-1).values.numpy(), rtol=1e-9)
    np.testing.assert_array_equal(pred, pt.argmax(dim=-1).numpy())


def test_rope_properties():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((6, 3, 64)); y = rng.standard_normal((6, 3, 64))
    pos = np.array([0, 1, 5, 17, 100, 4095])
    r = model.rope(x, pos, 10000.0)
    np.testing.assert_allclose(r[0], x[0], atol=0)                                   # position 0: identity
    np.testing.assert_allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    # scores depend on the position difference only
    a = model.rope(x[:1], np.array([40]), 1e4)[0, 0] @ model.rope(y[:1], np.array([33]), 1e4)[0, 0]
    b = model.rope(x[:1], np.array([1007]), 1e4)[0, 0] @ model.rope(y[:1], np.array([1000]), 1e4)[0, 0]
    assert abs(a - b) < 1e-9
    # first pair rotates by exactly pos radians, pairing is (t, t + Dh/2)
    e = np.zeros((1, 1, 64)); e[0, 0, 0] = 1.0
    out = model.rope(e, np.array([2]), 1e4)[0, 0]
    assert abs(out[0] - math.cos(2.0)) < 1e-15 and abs(out[32] - math.sin(2.0)) < 1e-15
    assert np.count_nonzero(out) == 2


def test_rmsnorm_and_silu_closed_forms():
    x = np.full((2, 8), 3.0); g = np.arange(8, dtype=np.float64)
    np.testing.assert_allclose(model.rmsnorm(x, g, 1e-5), 3.0 / math.sqrt(9 + 1e-5) * g[None].repeat(2, 0))
    t = np.linspace(-6, 6, 25)
    np.testing.assert_allclose(model.silu(t) - model.silu(-t), t, atol=1e-12)
    np.testing.assert_allclose(model.silu(t), F.silu(torch.from_numpy(t)).numpy(), rtol=1e-12, atol=1e-15)


def test_zero_query_weights_give_uniform_attention_and_mean_of_values():
    shape = inputs.TOY
    w = inputs.make_weights(shape, seed=1)
    wf = ostep.weights_to_f64(w)["layers"][0]
    Hq, Dh, d = shape.n_q_heads, shape.head_dim, shape.d_model
    wf["wqkv"][: Hq * Dh] = 0.0                                                      # q = 0 -> all scores equal
    wf["w_down"][:] = 0.0
    L, n = 40, 9
    rng = np.random.default_rng(3)
    Kc = rng.standard_normal((L, shape.n_kv_heads, Dh)); Vc = rng.standard_normal((L, shape.n_kv_heads, Dh))
    x = rng.standard_normal((n, d)); pos = np.sort(rng.choice(L, n, replace=False))
    xo, ab = model.layer_on_rows(x, pos, Kc, Vc, wf, Hq, shape.n_kv_heads, Dh, 1e4, 1e-5)
    np.testing.assert_allclose(ab, 1.0 / L, atol=1e-14)
    o = np.broadcast_to(Vc.mean(axis=0).reshape(1, Hq * Dh), (n, Hq * Dh))           # MHA: kv head = q head
    np.testing.assert_allclose(xo, x + o @ wf["wo"].T, atol=1e-10)


def test_lm_head_zero_weights_and_identities():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((5, 32)); g = np.ones(32)
    conf, pred, logits = model.lm_head_conf(x, g, np.zeros((50, 32)), 1e-5)
    np.testing.assert_allclose(conf, 1.0 / 50, rtol=1e-14); assert pred.tolist() == [0] * 5
    W = rng.standard_normal((50, 32))
    conf, pred, logits = model.lm_head_conf(x, g, W, 1e-5)
    assert np.all(conf >= 1.0 / 50) and np.all(conf <= 1.0)
    # a one-hot-like head: logit of token 7 is t, the rest 0 -> conf = e^t / (e^t + V - 1)
    W = np.zeros((50, 32)); W[7, 0] = 1.0
    xx = np.zeros((1, 32)); xx[0, 0] = 2.0
    conf, pred, _ = model.lm_head_conf(xx, g, W, 0.0)
    t = 2.0 / math.sqrt(4.0 / 32)
    assert pred[0] == 7 and abs(conf[0] - math.exp(t) / (math.exp(t) + 49)) < 1e-12
