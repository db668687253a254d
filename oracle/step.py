"""Oracle: one d2Cache decoding step, end to end.  Test infrastructure.

State carried between steps, per sequence: the KV cache of every layer, the
last confidence / prediction each position received (Eq. 1), and the rollout
influence scores c (Eq. 9) of the last forward pass.  A step is:

  1. selection from the *stored* scores (Eq. 3-4, top-p on c)            -> S
  2. the model on rows S only, attending to the whole cache (Eq. 5)       -> x_S, Abar^(l)
  3. confidence / prediction for the selected rows that are still masked  (Eq. 1)
  4. rollout of this step's attention (Eq. 6-9)                          -> c for the next step

Selecting every row (k >= #masked, p >= 1) is the ordinary full forward pass
and is how the state is first filled.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np

from . import model, rollout, selection


def weights_to_f64(w: Dict[str, object]) -> Dict[str, object]:
    """torch (bf16) weight dict -> the same dict as fp64 numpy arrays (exact widening, no arithmetic)."""
    def cv(t):
        return None if t is None else t.detach().cpu().double().numpy()
    out: Dict[str, object] = {"layers": [{k: cv(v) for k, v in lyr.items()} for lyr in w["layers"]],
                              "g_final": cv(w["g_final"]), "w_lm": cv(w["w_lm"])}
    return out


@dataclass
class OracleState:
    n_layers: int
    batch: int
    seq_len: int
    n_kv_heads: int
    head_dim: int
    Kc: np.ndarray = field(init=False)    # [N][B][L][Hkv][Dh]
    Vc: np.ndarray = field(init=False)
    conf: np.ndarray = field(init=False)  # [B][L] fp32
    pred: np.ndarray = field(init=False)  # [B][L] int32
    c: np.ndarray = field(init=False)     # [B][L] fp32

    def __post_init__(self):
        shp = (self.n_layers, self.batch, self.seq_len, self.n_kv_heads, self.head_dim)
        self.Kc = np.zeros(shp, dtype=np.float64)
        self.Vc = np.zeros(shp, dtype=np.float64)
        self.conf = np.zeros((self.batch, self.seq_len), dtype=np.float32)
        self.pred = np.zeros((self.batch, self.seq_len), dtype=np.int32)
        self.c = np.zeros((self.batch, self.seq_len), dtype=np.float32)


@dataclass
class StepResult:
    sel: List[np.ndarray]            # per sequence, ascending positions (Eq. 5's index set)
    m_star: List[np.ndarray]
    u: List[np.ndarray]
    hidden: List[np.ndarray]         # per sequence [n_b][d], residual stream after the last layer
    abar: List[List[np.ndarray]]     # per sequence, per layer [n_b][L]
    lm_rows: List[np.ndarray]        # per sequence: selected positions that are masked
    logits: List[np.ndarray]         # per sequence [len(lm_rows)][V]


def oracle_step(state: OracleState, w: Dict[str, object], shape, h0: np.ndarray, mask: np.ndarray,
                k: int, p: float, sigma: float = 10.0,
                forced: Optional[Sequence[Sequence[int]]] = None, stage2_candidates: int = 0,
                sel_override: Optional[Sequence[np.ndarray]] = None,
                rollout_literal: bool = False, rollout_layers: int = 0) -> StepResult:
    """One step.  h0: [B][L][d] input hidden states (embeddings of y_t), mask: [B][L] 1 = masked.

    `shape` needs n_q_heads, n_kv_heads, head_dim, rope_base, rms_eps.
    sel_override replaces step 1 with given index sets (teacher forcing in parity tests).
    rollout_layers > 0 rolls the attention out over the first layers only (the paper's "Rollout-5"
    variant, appendix table on rollout depth); 0 uses all layers (Eq. 8).
    The state is updated in place.
    """
    B, L, d = h0.shape
    res = StepResult([], [], [], [], [], [], [])
    for b in range(B):
        mb = np.asarray(mask[b]).astype(bool)
        fb = list(forced[b]) if forced is not None else []
        if sel_override is not None:
            S = np.asarray(sel_override[b], dtype=np.int64)
            m_star = S[mb[S]]
            u = S[~mb[S]]
        else:
            S, m_star, u = selection.select_rows(mb, state.conf[b], state.c[b], k, p, sigma,
                                                 forced=fb, stage2_candidates=stage2_candidates)
        x = np.asarray(h0[b], dtype=np.float64)[S]
        abars: List[np.ndarray] = []
        for l in range(state.n_layers):
            if S.size == 0:
                abars.append(np.zeros((0, L)))
                continue
            x, ab = model.layer_on_rows(x, S, state.Kc[l, b], state.Vc[l, b], w["layers"][l],
                                        shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                                        shape.rope_base, shape.rms_eps)
            abars.append(ab)
        lm_local = np.flatnonzero(mb[S]) if S.size else np.zeros(0, dtype=np.int64)
        lm_rows = S[lm_local] if S.size else np.zeros(0, dtype=np.int64)
        if lm_rows.size:
            cf, pr, lg = model.lm_head_conf(x[lm_local], w["g_final"], w["w_lm"], shape.rms_eps)
            state.conf[b, lm_rows] = cf.astype(np.float32)
            state.pred[b, lm_rows] = pr.astype(np.int32)
        else:
            lg = np.zeros((0, w["w_lm"].shape[0]))
        if S.size:
            cfun = rollout.literal if rollout_literal else rollout.chain
            depth = rollout_layers if 0 < rollout_layers < state.n_layers else state.n_layers
            state.c[b] = cfun(abars[:depth], S, L).astype(np.float32)
        res.sel.append(S); res.m_star.append(m_star); res.u.append(u)
        res.hidden.append(x); res.abar.append(abars); res.lm_rows.append(lm_rows); res.logits.append(lg)
    return res
