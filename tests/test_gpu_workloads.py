"""d2c_step at the full sizes of the benchmark workloads, in the launch configuration bench.py times.

The oracle cannot run a whole 32-layer step in test time, so each step is verified piecewise with
teacher forcing: the selection exhaustively (bit-exact, from the scores the GPU held), a seeded sample
of rows through a sample of layers (the oracle gets the GPU's layer input and the GPU's post-scatter
cache and recomputes K/V, the attention over all keys, the head-averaged probabilities and the layer
output for those rows), the LM head on (a sample of) the masked rows, the rollout chain of whole
sequences from the GPU's stored attention, and the bit-identity of every cache row outside the selected set.
"""
import numpy as np
import pytest
import torch

from oracle import model as omodel
from oracle import rollout as orollout
from oracle import selection as osel
from paper_2509_23094_b200 import binding, inputs
from gpu_util import ROW_TOL, check_lm_rows, check_rows, check_scores, row_rel_err

pytestmark = pytest.mark.gpu


def _f64(t):
    return None if t is None else t.detach().float().cpu().double().numpy()


class Runner:
    def __init__(self, wl):
        self.wl, self.shape = wl, wl.shape
        dev = "cuda"
        self.w = inputs.make_weights(wl.shape, seed=wl.seed, device=dev)
        self.cfg = binding.make_config(wl.shape, wl.batch, wl.seq_len, sigma=wl.sigma)
        self.ctx = binding.Context(self.cfg, self.w)
        self.mask = inputs.make_mask(wl)
        self.tokens = inputs.make_tokens(wl, self.mask)
        self.h0 = self.w["embed"][self.tokens.to(dev)].contiguous()
        B, L, d = wl.batch, wl.seq_len, wl.shape.d_model
        self.hid = torch.zeros(B * L, d, dtype=torch.bfloat16, device=dev)
        self.layer_in = torch.zeros(wl.shape.n_layers, B * L, d, dtype=torch.bfloat16, device=dev)
        # debug output of Eq. 1: fp32 logits of every row that went through the LM head, in row order
        self.logits = torch.zeros(int(self.mask.sum()), wl.shape.vocab, dtype=torch.float32, device=dev)

    def step(self, k, p, forced=None):
        wl = self.wl
        B, L = wl.batch, wl.seq_len
        conf = self.ctx.view("conf", B, L).cpu().numpy().copy()
        c = self.ctx.view("c", B, L).cpu().numpy().copy()
        f = fo = None
        if forced is not None:
            flat = [x for fb in forced for x in fb]
            f = torch.tensor(flat if flat else [0], dtype=torch.int32, device="cuda")
            fo = torch.tensor(np.cumsum([0] + [len(fb) for fb in forced]), dtype=torch.int32, device="cuda")
        self.ctx.step(self.h0, self.mask.cuda(), k, p, forced=f, forced_off=fo, hidden_out=self.hid, layer_in=self.layer_in,
                      logits=self.logits)
        self.ctx.sync_status()
        ro = self.ctx.view("row_off", B, L).cpu().numpy()
        sel = self.ctx.view("sel_idx").cpu().numpy()
        S = [sel[ro[b]: ro[b + 1]].astype(np.int64) for b in range(B)]
        # bit-exact selection from the scores the GPU held before the step
        for b in range(B):
            want, _, _ = osel.select_rows(self.mask[b].numpy(), conf[b], c[b], k, p, wl.sigma,
                                          forced=(forced[b] if forced is not None else ()))
            np.testing.assert_array_equal(S[b], want, err_msg=f"sequence {b}")
        return ro, S

    def check_layers(self, ro, S, layers, rows_per_seq=64, seqs=None, seed=0, local_rows=None):
        wl, shape = self.wl, self.shape
        B, L, d = wl.batch, wl.seq_len, shape.d_model
        rng = np.random.default_rng(seed)
        kc = self.ctx.view("kcache"); vc = self.ctx.view("vcache")
        worst = 0.0
        for l in layers:
            w = {k: _f64(v) for k, v in self.w["layers"][l].items()}
            x_next = self.layer_in[l + 1] if l + 1 < shape.n_layers else self.hid
            for b in (range(B) if seqs is None else seqs):
                nb = len(S[b])
                if nb == 0:
                    continue
                pick = np.sort(rng.choice(nb, min(rows_per_seq, nb), replace=False)) if local_rows is None else np.asarray(local_rows)
                rows = ro[b] + pick
                pos = S[b][pick]
                x_in = _f64(self.layer_in[l][rows])
                Kc = _f64(kc[l, b, :L]); Vc = _f64(vc[l, b, :L])
                Kg, Vg = Kc[pos].copy(), Vc[pos].copy()
                x_out, abar = omodel.layer_on_rows(x_in, pos, Kc, Vc, w, shape.n_q_heads, shape.n_kv_heads,
                                                   shape.head_dim, shape.rope_base, shape.rms_eps)
                kv = shape.n_kv_heads * shape.head_dim
                errs = [check_rows("K", Kg.reshape(-1, kv), Kc[pos].reshape(-1, kv), (l, b)),
                        check_rows("V", Vg.reshape(-1, kv), Vc[pos].reshape(-1, kv), (l, b)),
                        check_rows("hidden", _f64(x_next[rows]), x_out, (l, b)),
                        check_rows("abar", self.ctx.abar(l, ro[B], L)[rows].cpu().double().numpy(), abar, (l, b))]
                worst = max(worst, max(errs))
        return worst

    def check_lm_head(self, max_rows=96, seed=0):
        wl, shape = self.wl, self.shape
        B, L = wl.batch, wl.seq_len
        lm_off = self.ctx.view("lm_off", B, L).cpu().numpy()
        lm_rows = self.ctx.view("lm_rows").cpu().numpy()[: lm_off[B]]
        ro = self.ctx.view("row_off", B, L).cpu().numpy()
        sel = self.ctx.view("sel_idx").cpu().numpy()
        if len(lm_rows) == 0:
            return
        rng = np.random.default_rng(seed)
        pick = np.sort(rng.choice(len(lm_rows), min(max_rows, len(lm_rows)), replace=False))
        rows = lm_rows[pick]
        seq = np.searchsorted(ro, rows, side="right") - 1
        pos = sel[rows]
        conf_w, pred_w, logits = omodel.lm_head_conf(_f64(self.hid[rows]), _f64(self.w["g_final"]), _f64(self.w["w_lm"]),
                                                     shape.rms_eps)
        conf_g = self.ctx.view("conf", B, L).cpu().numpy()[seq, pos]
        pred_g = self.ctx.view("pred", B, L).cpu().numpy()[seq, pos]
        # row j of the logits output belongs to lm_rows[j]; at full vocabulary width the predicted token is held
        # to the exact arg-max of the kernel's own logits and to a near-maximum of the oracle's
        gpu_logits = self.logits[torch.from_numpy(pick).cuda()].cpu().numpy()
        check_lm_rows(gpu_logits, logits, pred_g, conf_g, conf_w, "full vocabulary")
        assert np.all(self.mask.numpy()[seq, pos] == 1)                  # Eq. 1 runs on masked rows only

    def check_rollout(self, ro, S, seqs):
        wl, shape = self.wl, self.shape
        B, L = wl.batch, wl.seq_len
        c = self.ctx.view("c", B, L).cpu().numpy()
        for b in seqs:
            if len(S[b]) == 0:
                continue
            abar = [self.ctx.abar(l, ro[B], L)[ro[b]: ro[b + 1]].cpu().double().numpy() for l in range(shape.n_layers)]
            want = orollout.chain(abar, S[b], L)
            check_scores(c[b], want, b)
            np.testing.assert_allclose(c[b], want, rtol=2e-3, atol=1e-4)
            assert abs(c[b].sum() - L) < 1e-3 * L


def _run(name, layers, prefill_layers, seqs):
    wl = inputs.WORKLOADS[name]
    r = Runner(wl)
    B, L = wl.batch, wl.seq_len
    ro, S = r.step(10 ** 6, 1.0)                                         # prefill: every row
    assert all(len(s) == L for s in S)
    r.check_layers(ro, S, prefill_layers, rows_per_seq=32, seqs=seqs[:1])
    r.check_lm_head(max_rows=48)
    kc0 = r.ctx.view("kcache").clone(); vc0 = r.ctx.view("vcache").clone()
    ro, S = r.step(wl.k, wl.p)
    assert all(0 < len(s) < L for s in S)
    worst = r.check_layers(ro, S, layers, seqs=seqs)
    r.check_lm_head()
    r.check_rollout(ro, S, seqs[:1])
    kc1 = r.ctx.view("kcache"); vc1 = r.ctx.view("vcache")
    for b in range(B):
        keep = torch.ones(L, dtype=torch.bool, device="cuda"); keep[torch.from_numpy(S[b]).cuda()] = False
        assert torch.equal(kc1[:, b, :L][:, keep], kc0[:, b, :L][:, keep]) and torch.equal(vc1[:, b, :L][:, keep], vc0[:, b, :L][:, keep])
    return r, ro, S, worst


def test_llada_single_layer_1024():
    r, ro, S, _ = _run("llada1l_1024", [0], [0], [0])
    assert 700 < len(S[0]) < 950                                         # flat scores: about 32 + 0.9 * 896 rows


def test_llada_single_layer_1024_few_rows():
    """The paper's default threshold p = 0.1: about a hundred selected rows, the weight-streaming regime.  The
    library switches kernels (one-SM GEMM with narrow tiles and split-K, probabilities pass on the side stream)
    on the row count of an earlier step, so the checked step is the second one with that count."""
    wl = inputs.WORKLOADS["llada1l_1024"]
    r = Runner(wl)
    B, L = wl.batch, wl.seq_len
    ro, S = r.step(10 ** 6, 1.0)
    snap = {n: r.ctx.view(n, B, L).clone() for n in ("conf", "pred", "c")}
    for _ in range(2):
        for n, t in snap.items():
            r.ctx.view(n, B, L).copy_(t)
        kc0 = r.ctx.view("kcache").clone(); vc0 = r.ctx.view("vcache").clone()
        ro, S = r.step(wl.k, 0.1)
        torch.cuda.synchronize()
    assert 64 < len(S[0]) <= 128                                         # flat scores: about 32 + 0.1 * 896 rows
    r.check_layers(ro, S, [0], seqs=[0])
    r.check_lm_head()
    r.check_rollout(ro, S, [0])
    kc1 = r.ctx.view("kcache"); vc1 = r.ctx.view("vcache")
    keep = torch.ones(L, dtype=torch.bool, device="cuda"); keep[torch.from_numpy(S[0]).cuda()] = False
    assert torch.equal(kc1[:, 0, :L][:, keep], kc0[:, 0, :L][:, keep]) and torch.equal(vc1[:, 0, :L][:, keep], vc0[:, 0, :L][:, keep])


@pytest.mark.parametrize("n_sel", [257, 323, 384, 385, 511, 600, 768, 835, 1023])
def test_llada_single_layer_row_counts_around_the_pair_tile(n_sel):
    """Selected-row counts with n mod 256 in {0, 1, 67, 88, 128, 129, 255} over two, three and four row tiles: the
    ragged last row tile of every projection (fused QKV + rotary + cache scatter, residual, SwiGLU), all of its rows
    checked, and the gate/up projection's stream-K shares for every number of row tiles (tiles split between
    clusters lie in every sampled row).  The rows are forced so
    that the count is exact; k = 0 and p = 0 select nothing else."""
    wl = inputs.WORKLOADS["llada1l_1024"]
    r = Runner(wl)
    B, L = wl.batch, wl.seq_len
    r.step(10 ** 6, 1.0)
    rng = np.random.default_rng(n_sel)
    forced = [sorted(rng.choice(L, n_sel, replace=False).tolist())]
    kc0 = r.ctx.view("kcache").clone(); vc0 = r.ctx.view("vcache").clone()
    ro, S = r.step(0, 0.0, forced=forced)
    assert len(S[0]) == n_sel
    # every row of the last, ragged tile and a sample of the others
    tail = np.arange((n_sel - 1) // 256 * 256, n_sel)
    r.check_layers(ro, S, [0], rows_per_seq=48, seqs=[0], seed=n_sel)
    r.check_layers(ro, S, [0], seqs=[0], local_rows=tail[:: max(1, len(tail) // 48)])
    r.check_lm_head()
    kc1 = r.ctx.view("kcache"); vc1 = r.ctx.view("vcache")
    keep = torch.ones(L, dtype=torch.bool, device="cuda"); keep[torch.from_numpy(S[0]).cuda()] = False
    assert torch.equal(kc1[:, 0, :L][:, keep], kc0[:, 0, :L][:, keep]) and torch.equal(vc1[:, 0, :L][:, keep], vc0[:, 0, :L][:, keep])


@pytest.mark.parametrize("n_sel", [1, 33, 64, 100, 128, 129, 200, 257, 384])
def test_llada_single_layer_few_forced_rows(n_sel):
    """At most 384 rows: from the second such step on the projections run on the one-SM kernel (one to three
    128-row tiles), every tile's K range split over several SMs whose parts each finish a share of the tile's
    columns; up to 128 rows the probabilities pass also moves beside the main stream."""
    wl = inputs.WORKLOADS["llada1l_1024"]
    r = Runner(wl)
    B, L = wl.batch, wl.seq_len
    r.step(10 ** 6, 1.0)
    rng = np.random.default_rng(1000 + n_sel)
    for rep in range(2):
        forced = [sorted(rng.choice(L, n_sel, replace=False).tolist())]
        kc0 = r.ctx.view("kcache").clone(); vc0 = r.ctx.view("vcache").clone()
        ro, S = r.step(0, 0.0, forced=forced)
        torch.cuda.synchronize()
        assert len(S[0]) == n_sel
        r.check_layers(ro, S, [0], rows_per_seq=64, seqs=[0], seed=n_sel + rep)
        r.check_lm_head()
        kc1 = r.ctx.view("kcache"); vc1 = r.ctx.view("vcache")
        keep = torch.ones(L, dtype=torch.bool, device="cuda"); keep[torch.from_numpy(S[0]).cuda()] = False
        assert torch.equal(kc1[:, 0, :L][:, keep], kc0[:, 0, :L][:, keep]) and torch.equal(vc1[:, 0, :L][:, keep], vc0[:, 0, :L][:, keep])


def test_llada_32_layers_768_with_a_committed_token():
    r, ro, S, _ = _run("llada_decode", [0, 1, 16, 31], [0, 31], [0])
    # decode-loop shape: commit the most confident masked row, force it into the next step
    wl = r.wl
    B, L = wl.batch, wl.seq_len
    committed = torch.full((B,), -2, dtype=torch.int32, device="cuda")
    tokens = r.tokens.to(torch.int32).cuda().contiguous()
    mask_dev = r.mask.cuda().contiguous()
    conf = r.ctx.view("conf", B, L).cpu().numpy(); pred = r.ctx.view("pred", B, L).cpu().numpy()
    fresh = [p for p in S[0] if r.mask[0, p]]
    want_pos = max(fresh, key=lambda p: (conf[0, p], -p))
    r.ctx.commit(r.w["embed"], r.h0, mask_dev, tokens, committed, rule=0)
    torch.cuda.synchronize()
    assert int(committed[0]) == want_pos and int(tokens[0, want_pos]) == int(pred[0, want_pos])
    assert int(mask_dev[0, want_pos]) == 0 and torch.equal(r.h0[0, want_pos], r.w["embed"][int(pred[0, want_pos])])
    r.mask = mask_dev.cpu()
    ro, S = r.step(wl.k, wl.p, forced=[[want_pos]])
    assert want_pos in S[0]
    r.check_layers(ro, S, [0, 31], rows_per_seq=32)


def test_dream_28_layers_batch4_1536():
    _run("dream_decode", [0, 1, 27], [0], [0, 3])


def test_llada_long_context_batch8_4096():
    r, ro, S, _ = _run("llada_long", [0, 31], [0], [0, 7])
    wl = r.wl
    # second threshold of the workload
    ro, S = r.step(wl.k, 0.95)
    r.check_layers(ro, S, [15], rows_per_seq=32, seqs=[5])
