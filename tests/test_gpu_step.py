"""d2c_step against the oracle, end to end: prefill (all rows), partial steps, the degenerate steps."""
import numpy as np
import pytest
import torch

from paper_2509_23094_b200 import inputs
from gpu_util import ROW_TOL, Pair, check_lm_rows, check_rows, check_scores, row_rel_err

pytestmark = pytest.mark.gpu


def _compare_state(pair, res, sel, mask=None, gpu_logits=None):
    """Cache rows of the selected positions, confidences, predictions and rollout scores.  gpu_logits: the
    step's debug logits output (rows of all sequences that went through Eq. 1, in row order)."""
    wl, shape = pair.wl, pair.shape
    B, L = wl.batch, wl.seq_len
    mask = pair.mask if mask is None else mask
    kc = pair.ctx.view("kcache").float().cpu().numpy(); vc = pair.ctx.view("vcache").float().cpu().numpy()
    conf = pair.ctx.view("conf", B, L).cpu().numpy(); pred = pair.ctx.view("pred", B, L).cpu().numpy()
    c = pair.ctx.view("c", B, L).cpu().numpy()
    kv = shape.n_kv_heads * shape.head_dim
    lm_at = 0
    for b in range(B):
        S = sel[b]
        for l in range(shape.n_layers):
            check_rows("K", kc[l, b, S].reshape(len(S), kv), pair.ost.Kc[l, b, S].reshape(len(S), kv), (l, b))
            check_rows("V", vc[l, b, S].reshape(len(S), kv), pair.ost.Vc[l, b, S].reshape(len(S), kv), (l, b))
        lm = res.lm_rows[b]
        if len(lm):
            assert gpu_logits is not None, "a step with LM-head rows is compared with its logits output"
            check_lm_rows(gpu_logits[lm_at: lm_at + len(lm)], res.logits[b], pred[b, lm], conf[b, lm], pair.ost.conf[b, lm], b)
            lm_at += len(lm)
        if len(S):
            check_scores(c[b], pair.ost.c[b], b)


def _prefill(pair):
    g = pair.gpu_step(10 ** 6, 1.0, want_logits=True)
    for b in range(pair.wl.batch):
        assert g["sel"][b].tolist() == list(range(pair.wl.seq_len))
    res = pair.oracle_step(g["sel"])
    for b in range(pair.wl.batch):
        check_rows("hidden", g["hidden"][b], res.hidden[b], b)
    _compare_state(pair, res, g["sel"], gpu_logits=g["logits"])
    return g, res


WLS = {
    "toy": inputs.WORKLOADS["toy"],
    "gqa_bias_3layers": inputs.Workload("gqa", inputs.TOY_GQA, 2, 200, 120, 37, "random", 6, 0.7, seed=3),
    "hd128_ragged_vocab": inputs.Workload("hd128", inputs.TOY_HD128, 3, 130, 70, 33, "random", 5, 0.5, seed=4),
}


@pytest.mark.parametrize("name,flags", [(n, 0) for n in WLS] + [("gqa_bias_3layers", 16), ("hd128_ragged_vocab", 16)])
def test_prefill_then_partial_steps(name, flags):
    """flags = 16: the same steps with the layers' RMSNorms folded into the GEMM epilogues around them."""
    wl = WLS[name]
    pair = Pair(wl, flags=flags)
    _prefill(pair)
    kc0 = pair.ctx.view("kcache").clone(); vc0 = pair.ctx.view("vcache").clone()
    for step, (k, p) in enumerate([(wl.k, wl.p), (wl.k, 0.1), (3, 0.5)]):
        g = pair.gpu_step(k, p, want_logits=True)
        # bit-exact selection given the scores the GPU held before the step
        want_sel = pair.oracle_selection(g["conf_before"], g["c_before"], pair.mask, k, p)
        for b in range(wl.batch):
            np.testing.assert_array_equal(g["sel"][b], want_sel[b], err_msg=f"step {step} seq {b}")
            assert 0 < len(g["sel"][b]) < wl.seq_len
        res = pair.oracle_step(g["sel"])
        for b in range(wl.batch):
            check_rows("hidden", g["hidden"][b], res.hidden[b], (step, b))
        _compare_state(pair, res, g["sel"], gpu_logits=g["logits"])
        # reuse: cache rows of unselected positions are bit-identical
        kc1 = pair.ctx.view("kcache"); vc1 = pair.ctx.view("vcache")
        for b in range(wl.batch):
            rest = np.setdiff1d(np.arange(wl.seq_len), g["sel"][b])
            assert torch.equal(kc1[:, b, rest], kc0[:, b, rest]) and torch.equal(vc1[:, b, rest], vc0[:, b, rest])
        kc0, vc0 = kc1.clone(), vc1.clone()


def test_single_layer_partial_step_reproduces_prefill_rows():
    wl = WLS["toy"]
    pair = Pair(wl)
    g0, _ = _prefill(pair)
    kc0 = pair.ctx.view("kcache").clone()
    g = pair.gpu_step(wl.k, wl.p)
    S = g["sel"][0]
    assert len(S) < wl.seq_len
    # with one layer nothing in the cache is stale, so the partial step recomputes the same values
    assert row_rel_err(g["hidden"][0], g0["hidden"][0][S]) <= 1e-2
    assert torch.equal(pair.ctx.view("kcache"), kc0)


def test_select_none_changes_nothing():
    pair = Pair(WLS["gqa_bias_3layers"])
    _prefill(pair)
    names = ("kcache", "vcache")
    before = {n: pair.ctx.view(n).clone() for n in names}
    B, L = pair.wl.batch, pair.wl.seq_len
    sb = {n: pair.ctx.view(n, B, L).clone() for n in ("conf", "pred", "c")}
    g = pair.gpu_step(0, 0.0)
    assert g["row_off"].tolist() == [0] * (B + 1)
    for n in names:
        assert torch.equal(pair.ctx.view(n), before[n]), n
    for n in sb:
        assert torch.equal(pair.ctx.view(n, B, L), sb[n]), n


def test_forced_rows_decoded_token_and_mode1():
    wl = WLS["gqa_bias_3layers"]
    pair = Pair(wl, stage2_candidates=1)
    _prefill(pair)
    # commit one token per sequence by hand: its embedding changes and it is forced into the next step
    mask = pair.mask.clone(); h0 = pair.h0.clone(); forced = []
    for b in range(wl.batch):
        pos = int(np.flatnonzero(mask[b].numpy())[3])
        mask[b, pos] = 0; h0[b, pos] = pair.w_cpu["embed"][17 + b]; forced.append([pos])
    g = pair.gpu_step(4, 0.3, forced=forced, mask=mask, h0=h0, want_logits=True)
    want_sel = pair.oracle_selection(g["conf_before"], g["c_before"], mask, 4, 0.3, forced=forced)
    for b in range(wl.batch):
        np.testing.assert_array_equal(g["sel"][b], want_sel[b])
        assert forced[b][0] in g["sel"][b]
    res = pair.oracle_step(g["sel"], mask=mask, h0=h0)
    for b in range(wl.batch):
        check_rows("hidden", g["hidden"][b], res.hidden[b], b)
    _compare_state(pair, res, g["sel"], mask=mask, gpu_logits=g["logits"])


def test_step_is_deterministic():
    wl = WLS["hd128_ragged_vocab"]
    outs = []
    for _ in range(2):
        pair = Pair(wl)
        pair.gpu_step(10 ** 6, 1.0)
        g = pair.gpu_step(wl.k, wl.p)
        outs.append((g, pair.ctx.view("c", wl.batch, wl.seq_len).clone(), pair.ctx.view("kcache").clone()))
    for b in range(wl.batch):
        np.testing.assert_array_equal(outs[0][0]["sel"][b], outs[1][0]["sel"][b])
        np.testing.assert_array_equal(outs[0][0]["hidden"][b], outs[1][0]["hidden"][b])
    assert torch.equal(outs[0][1], outs[1][1]) and torch.equal(outs[0][2], outs[1][2])


def test_step_host_matches_device_step():
    wl = WLS["toy"]
    pair = Pair(wl)
    pair.gpu_step(10 ** 6, 1.0)
    B, L, d = wl.batch, wl.seq_len, wl.shape.d_model
    snap = {n: pair.ctx.view(n, B, L).clone() for n in ("conf", "c")}
    g = pair.gpu_step(wl.k, wl.p)
    conf_dev = pair.ctx.view("conf", B, L).cpu()
    for n, t in snap.items():
        pair.ctx.view(n, B, L).copy_(t)
    sel = torch.full((B * L,), -1, dtype=torch.int32).pin_memory(); ro = torch.zeros(B + 1, dtype=torch.int32).pin_memory()
    hid = torch.zeros(B * L, d, dtype=torch.bfloat16).pin_memory()
    conf = torch.zeros(B, L).pin_memory(); pred = torch.zeros(B, L, dtype=torch.int32).pin_memory()
    pair.ctx.step_host(pair.h0.pin_memory(), pair.mask.pin_memory(), wl.k, wl.p, sel_idx=sel, row_off=ro, hidden_out=hid,
                       conf=conf, pred=pred)
    n = int(ro[B])
    assert ro.numpy().tolist() == g["row_off"].tolist()
    np.testing.assert_array_equal(sel.numpy()[:n], np.concatenate(g["sel"]))
    np.testing.assert_array_equal(hid.float().numpy()[:n], np.concatenate(g["hidden"]))
    assert torch.equal(conf, conf_dev)


@pytest.mark.parametrize("rule", [0, 1, 2])
def test_decode_loop_commits_match_the_oracle_rule(rule):
    """commit + step for several iterations: every commit decision is checked against the oracle's
    scheduling function applied to the confidences the GPU holds, every step's selection against the
    oracle's selection, and the final hidden states against a teacher-forced oracle."""
    from oracle import decode
    wl = WLS["gqa_bias_3layers"]
    pair = Pair(wl)
    _prefill(pair)
    B, L = wl.batch, wl.seq_len
    mask = pair.mask.clone().cuda(); h0 = pair.h0.clone().cuda()
    tokens = pair.tokens.to(torch.int32).cuda().contiguous()
    committed = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    embed = pair.w_dev["embed"]
    fresh = [np.flatnonzero(pair.mask[b].numpy()) for b in range(B)]              # the prefill refreshed every masked row
    for it in range(5):
        conf = pair.ctx.view("conf", B, L).cpu().numpy(); pred = pair.ctx.view("pred", B, L).cpu().numpy()
        mask_before = mask.cpu().numpy()
        pair.ctx.commit(embed, h0, mask, tokens, committed, rule=rule, threshold=0.002)
        torch.cuda.synchronize()
        got_mask = mask.cpu().numpy(); forced = []
        for b in range(B):
            want, best = decode.commit(mask_before[b], conf[b], fresh[b], rule=rule, sigma=wl.sigma, threshold=0.002)
            assert int(committed[b]) == best
            assert np.flatnonzero(mask_before[b] != got_mask[b]).tolist() == want
            for pos in want:
                assert int(tokens[b, pos]) == int(pred[b, pos]) and torch.equal(h0[b, pos], embed[int(pred[b, pos])])
            forced.append(want[:1] if rule != 2 else want)
        f = torch.tensor([x for fb in forced for x in fb] or [0], dtype=torch.int32, device="cuda")
        fo = torch.tensor(np.cumsum([0] + [len(fb) for fb in forced]), dtype=torch.int32, device="cuda")
        conf_b = pair.ctx.view("conf", B, L).cpu().numpy().copy(); c_b = pair.ctx.view("c", B, L).cpu().numpy().copy()
        hid = torch.zeros(B * L, wl.shape.d_model, dtype=torch.bfloat16, device="cuda")
        pair.ctx.step(h0, mask, wl.k, 0.3, forced=f, forced_off=fo, hidden_out=hid)
        pair.ctx.sync_status()
        ro = pair.ctx.view("row_off", B, L).cpu().numpy(); sel = pair.ctx.view("sel_idx").cpu().numpy()
        S = [sel[ro[b]: ro[b + 1]].astype(np.int64) for b in range(B)]
        want_sel = pair.oracle_selection(conf_b, c_b, mask.cpu(), wl.k, 0.3, forced=forced)
        for b in range(B):
            np.testing.assert_array_equal(S[b], want_sel[b])
        res = pair.oracle_step(S, mask=mask.cpu(), h0=h0.cpu())
        for b in range(B):
            check_rows("hidden", hid[ro[b]: ro[b + 1]].float().cpu().numpy(), res.hidden[b], (it, b))
        fresh = [np.array([p for p in S[b] if got_mask[b, p]]) for b in range(B)]


def test_truncated_rollout_depth():
    """rollout_layers = 2 on a 3-layer model: the scores come from the first two layers' attention only."""
    wl = WLS["gqa_bias_3layers"]
    pair = Pair(wl, rollout_layers=2)
    _prefill(pair)
    g = pair.gpu_step(wl.k, wl.p, want_logits=True)
    res = pair.oracle_step(g["sel"])
    _compare_state(pair, res, g["sel"], gpu_logits=g["logits"])
    full = Pair(wl)                                                   # same inputs, full depth: the scores must differ
    _prefill(full)
    assert not torch.allclose(full.ctx.view("c", wl.batch, wl.seq_len), pair.ctx.view("c", wl.batch, wl.seq_len), atol=1e-4)


def test_kernel_variants_agree():
    """The mma.sync GEMM / attention kernels, the one-SM tcgen05 GEMM and the RMSNorms folded into the GEMM epilogues give the
    same step within tolerance."""
    wl = inputs.Workload("hd128_big", inputs.TOY_HD128, 2, 300, 150, 60, "random", 8, 0.6, seed=9)
    ref = None
    for flags in (0, 1 | 2, 4, 16):                                   # default; portable GEMM + attention; one-SM GEMM; RMSNorms folded into the GEMM epilogues
        pair = Pair(wl, flags=flags)
        pair.gpu_step(10 ** 6, 1.0)
        g = pair.gpu_step(wl.k, wl.p)
        if ref is None:
            ref = g
            continue
        for b in range(wl.batch):
            np.testing.assert_array_equal(g["sel"][b], ref["sel"][b])
            assert row_rel_err(g["hidden"][b], ref["hidden"][b].astype(np.float64)) <= ROW_TOL


def test_overlapped_and_serial_steps_are_identical():
    """The probabilities / rollout side stream changes when kernels run, not what they compute."""
    wl = inputs.Workload("hd128_overlap", inputs.TOY_HD128, 2, 300, 150, 60, "random", 8, 0.6, seed=11)
    got = []
    for flags in (0, 8):                                              # default (two streams); D2C_FLAG_SERIAL
        pair = Pair(wl, flags=flags)
        pair.gpu_step(10 ** 6, 1.0)
        steps = [pair.gpu_step(wl.k, wl.p) for _ in range(3)]         # each step selects from the previous step's rollout
        B, L = wl.batch, wl.seq_len
        got.append((steps, pair.ctx.view("c", B, L).clone(), pair.ctx.view("conf", B, L).clone(),
                    pair.ctx.view("kcache").clone()))
    (sa, ca, fa, ka), (sb, cb, fb, kb) = got
    for ga, gb in zip(sa, sb):
        for b in range(wl.batch):
            np.testing.assert_array_equal(ga["sel"][b], gb["sel"][b])
            np.testing.assert_array_equal(ga["hidden"][b], gb["hidden"][b])
    assert torch.equal(ca, cb) and torch.equal(fa, fb) and torch.equal(ka, kb)


@pytest.mark.parametrize("flags", [0, 8])
def test_step_replayed_from_a_cuda_graph(flags):
    """d2c_step captured into a CUDA graph (with and without the internal streams) replays to the same bits."""
    wl = inputs.Workload("hd128_graph", inputs.TOY_HD128, 2, 300, 150, 60, "random", 8, 0.6, seed=12)
    B, L, d = wl.batch, wl.seq_len, wl.shape.d_model
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        pair = Pair(wl, flags=flags)
        pair.gpu_step(10 ** 6, 1.0)
        snap = {n: pair.ctx.view(n, B, L).clone() for n in ("conf", "pred", "c")}
        kc = pair.ctx.view("kcache").clone(); vc = pair.ctx.view("vcache").clone()

        def restore():
            for n, t in snap.items():
                pair.ctx.view(n, B, L).copy_(t)
            pair.ctx.view("kcache").copy_(kc); pair.ctx.view("vcache").copy_(vc)

        h0, mask = pair.h0.cuda(), pair.mask.cuda()
        hid = torch.zeros(B * L, d, dtype=torch.bfloat16, device="cuda")
        restore()
        pair.ctx.step(h0, mask, wl.k, wl.p, hidden_out=hid)           # eager: also the first launch of every kernel
        pair.ctx.sync_status()
        want = (hid.clone(), pair.ctx.view("c", B, L).clone(), pair.ctx.view("conf", B, L).clone(),
                pair.ctx.view("kcache").clone())
        restore(); hid.zero_()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            pair.ctx.step(h0, mask, wl.k, wl.p, hidden_out=hid)
        for _ in range(2):
            restore(); hid.zero_()
            graph.replay()
            pair.ctx.sync_status()
            got = (hid, pair.ctx.view("c", B, L), pair.ctx.view("conf", B, L), pair.ctx.view("kcache"))
            assert all(torch.equal(a, b) for a, b in zip(got, want))


def test_semi_autoregressive_block_restricts_stage1():
    from oracle import selection as osel
    wl = inputs.Workload("semiar", inputs.TOY_HD128, 2, 192, 64, 128, "all", 6, 0.4, seed=5)
    pair = Pair(wl)
    _prefill(pair)
    B, L = wl.batch, wl.seq_len
    conf = pair.ctx.view("conf", B, L).cpu().numpy().copy(); c = pair.ctx.view("c", B, L).cpu().numpy().copy()
    hid = torch.zeros(B * L, wl.shape.d_model, dtype=torch.bfloat16, device="cuda")
    pair.ctx.step(pair.h0.cuda(), pair.mask.cuda(), wl.k, wl.p, hidden_out=hid, block=(96, 128))
    pair.ctx.sync_status()
    ro = pair.ctx.view("row_off", B, L).cpu().numpy(); sel = pair.ctx.view("sel_idx").cpu().numpy()
    key = pair.ctx.view("key", B, L).cpu().numpy()
    S = []
    for b in range(B):
        want, m_star, _ = osel.select_rows(pair.mask[b].numpy(), conf[b], c[b], wl.k, wl.p, wl.sigma, block=(96, 128))
        got = sel[ro[b]: ro[b + 1]]
        np.testing.assert_array_equal(got, want)
        # stage-1 keys: bit-exact inside the block (the density of Eq. 3 sees the whole sequence), 0 outside it
        want_key = osel.stage1_keys(pair.mask[b].numpy(), conf[b], wl.sigma)
        want_key[:96] = 0.0; want_key[128:] = 0.0
        np.testing.assert_array_equal(key[b].view(np.uint32), want_key.view(np.uint32))
        assert len(m_star) == wl.k and all(96 <= i < 128 for i in m_star)
        S.append(got.astype(np.int64))
    res = pair.oracle_step(S)
    for b in range(B):
        check_rows("hidden", hid[ro[b]: ro[b + 1]].float().cpu().numpy(), res.hidden[b], b)
