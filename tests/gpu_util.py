"""Helpers shared by the GPU parity tests: context construction, oracle bridging, the float tolerance."""
from __future__ import annotations

import numpy as np
import torch

from oracle import selection as osel
from oracle import step as ostep
from paper_2509_23094_b200 import binding, inputs

# max |gpu - oracle| over a row, relative to the oracle row's L2 norm (bf16 storage, fp32 accumulation)
ROW_TOL = 2e-2

# Worst error seen per tensor in this process (printed in the terminal summary), and regression bounds:
# about four times the worst error the committed kernels showed on a B200 over the whole GPU suite.  A
# row-norm tolerance of 2e-2 at 4096 columns admits one element that is off by more than a row RMS; the
# regression bound is what catches a kernel that starts to drift or gets single elements wrong.
OBSERVED = {}
# (observed over the suite: K 2.2e-3, V 2.4e-3, hidden 2.0e-3, abar 3.2e-3, logits 8.6e-4, c 5.1e-4)
REGRESSION = {"K": 9e-3, "V": 1e-2, "hidden": 8e-3, "abar": 1.3e-2, "logits": 3.5e-3, "c": 2e-3}


def observe(name: str, err: float) -> float:
    OBSERVED[name] = max(OBSERVED.get(name, 0.0), float(err))
    return float(err)


def check_rows(name: str, got, want, what="") -> float:
    """Row-norm-relative error of one tensor kind: recorded, held to the stated tolerance and to its regression bound."""
    err = observe(name, row_rel_err(np.asarray(got), np.asarray(want)))
    assert err <= ROW_TOL, (name, what, err)
    assert err <= REGRESSION[name], (name, what, err, "regression bound")
    return err


def check_scores(got, want, what="") -> float:
    """Rollout scores c (Eq. 9): element-wise relative error."""
    got = np.asarray(got, dtype=np.float64); want = np.asarray(want, dtype=np.float64)
    err = observe("c", float(np.max(np.abs(got - want) / np.maximum(np.abs(want), 1e-4)))) if want.size else 0.0
    assert err <= 2e-2 and err <= REGRESSION["c"], ("c", what, err)
    return err


def check_lm_rows(gpu_logits, oracle_logits, pred, conf, oracle_conf, what="") -> float:
    """Eq. 1 on a set of rows.  The GPU's token must be the exact arg-max of the GPU's own logits (lowest id
    among equals); its logits must match the oracle's row within the tolerance; and in the oracle's logits
    the GPU's token may trail the oracle's best by no more than four times the observed logit error."""
    gpu_logits = np.asarray(gpu_logits, dtype=np.float64); oracle_logits = np.asarray(oracle_logits, dtype=np.float64)
    if oracle_logits.shape[0] == 0:
        return 0.0
    pred = np.asarray(pred, dtype=np.int64)
    np.testing.assert_array_equal(pred, np.argmax(gpu_logits, axis=1), err_msg=f"{what}: pred is not the arg-max of the kernel's own logits")
    err = check_rows("logits", gpu_logits, oracle_logits, what)
    abs_err = np.max(np.abs(gpu_logits - oracle_logits), axis=1)
    r = np.arange(len(pred))
    assert np.all(oracle_logits[r, pred] >= oracle_logits.max(axis=1) - 4.0 * abs_err), (what, "predicted token is not a near-maximum of the oracle's logits")
    np.testing.assert_allclose(conf, oracle_conf, rtol=0.1, atol=1e-7)
    return err


def row_rel_err(got: np.ndarray, want: np.ndarray) -> float:
    """max over rows of max|got-want| / ||want row||_2 (rows = all but the last axis flattened)."""
    got = np.asarray(got, dtype=np.float64).reshape(-1, got.shape[-1])
    want = np.asarray(want, dtype=np.float64).reshape(-1, want.shape[-1])
    if want.shape[0] == 0:
        return 0.0
    norm = np.linalg.norm(want, axis=1)
    err = np.max(np.abs(got - want), axis=1)
    return float(np.max(err / np.maximum(norm, 1e-30)))


def to_dev(w, device="cuda"):
    def mv(t):
        return None if t is None else t.to(device).contiguous()
    out = {"layers": [{k: mv(v) for k, v in lyr.items()} for lyr in w["layers"]],
           "g_final": mv(w["g_final"]), "w_lm": mv(w["w_lm"])}
    if "embed" in w:
        out["embed"] = mv(w["embed"])
    return out


class Pair:
    """A CUDA context and an oracle state fed the same weights and inputs."""

    def __init__(self, wl: inputs.Workload, gain_jitter=0.05, std=0.02, stage2_candidates=0, rollout_layers=0,
                 max_batch=None, max_seq=None, flags=0):
        self.wl, self.shape = wl, wl.shape
        self.w_cpu = inputs.make_weights(wl.shape, seed=wl.seed, gain_jitter=gain_jitter, std=std)
        self.w_dev = to_dev(self.w_cpu)
        self.wf = ostep.weights_to_f64(self.w_cpu)
        self.cfg = binding.make_config(wl.shape, max_batch or wl.batch, max_seq or wl.seq_len, sigma=wl.sigma,
                                       stage2_candidates=stage2_candidates, rollout_layers=rollout_layers, flags=flags)
        self.ctx = binding.Context(self.cfg, self.w_dev)
        self.ost = ostep.OracleState(wl.shape.n_layers, wl.batch, wl.seq_len, wl.shape.n_kv_heads, wl.shape.head_dim)
        self.mask = inputs.make_mask(wl)
        self.tokens = inputs.make_tokens(wl, self.mask)
        self.h0 = inputs.make_h0(self.w_cpu["embed"], self.tokens)
        self.stage2_candidates = stage2_candidates
        self.rollout_layers = rollout_layers

    def gpu_step(self, k, p, forced=None, want_logits=False, mask=None, h0=None):
        wl = self.wl
        B, L, d = wl.batch, wl.seq_len, wl.shape.d_model
        mask = self.mask if mask is None else mask
        h0 = self.h0 if h0 is None else h0
        hid = torch.zeros(B * L, d, dtype=torch.bfloat16, device="cuda")
        sel = torch.full((B * L,), -1, dtype=torch.int32, device="cuda")
        ro = torch.zeros(B + 1, dtype=torch.int32, device="cuda")
        f = fo = None
        if forced is not None:
            flat = [x for fb in forced for x in fb]
            offs = np.cumsum([0] + [len(fb) for fb in forced])
            f = torch.tensor(flat if flat else [0], dtype=torch.int32, device="cuda")
            fo = torch.tensor(offs, dtype=torch.int32, device="cuda")
        n_masked = int(mask.sum())
        logits = torch.zeros(max(n_masked, 1), wl.shape.vocab, dtype=torch.float32, device="cuda") if want_logits else None
        conf_before = self.ctx.view("conf", B, L).clone()
        c_before = self.ctx.view("c", B, L).clone()
        self.ctx.step(h0.cuda(), mask.cuda(), k, p, forced=f, forced_off=fo, hidden_out=hid, sel_idx=sel, row_off=ro,
                      logits=logits)
        self.ctx.sync_status()
        ro = ro.cpu().numpy()
        sel = sel.cpu().numpy()
        return dict(row_off=ro, sel=[sel[ro[b]: ro[b + 1]].astype(np.int64) for b in range(B)],
                    hidden=[hid[ro[b]: ro[b + 1]].float().cpu().numpy() for b in range(B)],
                    logits=None if logits is None else logits.cpu().numpy(),
                    conf_before=conf_before.cpu().numpy(), c_before=c_before.cpu().numpy())

    def oracle_selection(self, conf, c, mask, k, p, forced=None):
        """What the oracle selects from the given (GPU-side) scores: the bit-exact part of the parity."""
        out = []
        for b in range(self.wl.batch):
            S, _, _ = osel.select_rows(mask[b].numpy(), conf[b], c[b], k, p, self.wl.sigma,
                                       forced=(forced[b] if forced is not None else ()),
                                       stage2_candidates=self.stage2_candidates)
            out.append(S)
        return out

    def oracle_step(self, sel, mask=None, h0=None):
        mask = self.mask if mask is None else mask
        h0 = self.h0 if h0 is None else h0
        return ostep.oracle_step(self.ost, self.wf, self.shape, h0.double().numpy(), mask.numpy(), k=0, p=0.0,
                                 sigma=self.wl.sigma, sel_override=sel, rollout_layers=self.rollout_layers)
