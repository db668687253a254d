"""Oracle: two-stage token selection of d2Cache (Section 4.1-4.2).  Test infrastructure.

Stage 1 (Eq. 3-4): certainty density D(i) over known neighbours of a masked
position, key D(i)*s^i, top-k over the masked set.
Stage 2 (last paragraph of Section 4.2): sort the remaining candidates by the
rollout influence score c_j, keep the smallest prefix whose cumulative share of
the total mass exceeds p.
The union of both stages (plus caller-forced rows) is the subset input of Eq. 5.

Readings the paper leaves open, fixed here so that exactly one answer is right:
  * equal keys / equal scores: the lower position comes first;
  * "cumulative probability": c_j divided by the sum of c over the candidates;
  * "exceeds": strictly greater; p >= 1 therefore keeps every candidate,
    p <= 0 keeps none;
  * all sums that decide an index are taken in fixed point so that the order of
    summation cannot matter: phi is tabulated as round(phi * 2^30), c_j is
    truncated to floor(c_j * 2^32).  `density` is Eq. 3 in plain fp64 and the
    tests bound the distance between the two.
"""
from __future__ import annotations

import math
from typing import Iterable, Optional, Tuple

import numpy as np

Q30 = 1 << 30
Q32 = 1 << 32


def phi(r: float, sigma: float) -> float:
    """Gaussian distance weight of Eq. 3."""
    return math.exp(-(r * r) / (2.0 * sigma * sigma))


def density(mask: np.ndarray, sigma: float) -> np.ndarray:
    """Eq. 3 as printed, fp64: D(i) = sum_j phi(|i-j|) [j not masked], for masked i (0 elsewhere)."""
    mask = np.asarray(mask).astype(bool)
    L = mask.shape[0]
    D = np.zeros(L, dtype=np.float64)
    for i in range(L):
        if not mask[i]:
            continue
        acc = 0.0
        for j in range(L):
            if not mask[j]:
                acc += phi(abs(i - j), sigma)
        D[i] = acc
    return D


def phi_table_q30(sigma: float, length: int) -> list:
    """phi(r) in 2^-30 fixed point, r = 0..length-1: floor(phi*2^30 + 0.5)."""
    return [int(math.floor(phi(float(r), float(sigma)) * Q30 + 0.5)) for r in range(length)]


def density_q30(mask: np.ndarray, sigma: float) -> list:
    """Eq. 3 with the tabulated phi: exact integer sums, one Python int per position."""
    mask = np.asarray(mask).astype(bool)
    L = mask.shape[0]
    tab = phi_table_q30(sigma, L)
    out = [0] * L
    for i in range(L):
        if mask[i]:
            out[i] = sum(tab[abs(i - j)] for j in range(L) if not mask[j])
    return out


def stage1_keys(mask: np.ndarray, conf: np.ndarray, sigma: float) -> np.ndarray:
    """fp32 key D(i)*s^i of Eq. 4 for masked i (0 elsewhere).

    D is the fixed-point sum converted once to fp32 (round to nearest) and scaled
    by 2^-30 (exact); the product with the stored fp32 confidence is one fp32 multiply.
    """
    Dq = density_q30(mask, sigma)
    D32 = np.array([np.float32(np.uint64(v)) for v in Dq], dtype=np.float32) * np.float32(2.0 ** -30)
    key = (D32 * np.asarray(conf, dtype=np.float32)).astype(np.float32)
    key[~np.asarray(mask).astype(bool)] = 0.0
    return key


SCORE_CAP = np.float32(262144.0)   # 2^18: keeps the fixed-point mass of 8192 positions inside 64 bits


def _clean_score(x: np.ndarray) -> np.ndarray:
    """Scores that are NaN, negative or infinite count as 0 (they cannot be ordered as masses);
    finite ones are capped at 2^18 (a rollout score never exceeds the sequence length)."""
    x = np.asarray(x, dtype=np.float32).copy()
    x[~((x > 0) & np.isfinite(x))] = 0.0
    return np.minimum(x, SCORE_CAP)


def stage1_select(mask: np.ndarray, conf: np.ndarray, k: int, sigma: float,
                  key: Optional[np.ndarray] = None, block: Optional[Tuple[int, int]] = None) -> np.ndarray:
    """Eq. 4: indices of the k largest keys over the masked set (all of it if it has <= k members).

    block = (lo, hi) confines the masked set to positions lo <= i < hi: the reading taken here of
    "semi-autoregressive decoding with d2Cache" (blocks decoded left to right, Section 5.1), which
    the paper does not spell out.  The density of Eq. 3 still sees the whole sequence.
    """
    mask = np.asarray(mask).astype(bool)
    if key is None:
        key = stage1_keys(mask, conf, sigma)
    key = _clean_score(key)
    members = [int(i) for i in np.flatnonzero(mask)]
    if block is not None and block[1] > block[0]:
        members = [i for i in members if block[0] <= i < block[1]]
    members.sort(key=lambda i: (-float(key[i]), i))
    return np.array(sorted(members[: max(0, int(k))]), dtype=np.int64)


def stage2_select(c: np.ndarray, candidates: np.ndarray, p: float) -> np.ndarray:
    """Top-p over the candidate positions by influence score c_j (Section 4.2, after Eq. 9)."""
    c = _clean_score(c)
    cand = [int(j) for j in np.flatnonzero(np.asarray(candidates).astype(bool))]
    p32 = float(np.float32(p))
    if not (p32 > 0.0) or not cand:
        return np.zeros(0, dtype=np.int64)
    cand.sort(key=lambda j: (-float(c[j]), j))
    q = [int(math.floor(float(c[j]) * Q32)) for j in cand]       # exact: fp32 * 2^32 fits fp64
    total = sum(q)
    threshold = p32 * float(total)
    prefix = 0
    take = len(cand)
    for m, qj in enumerate(q):
        prefix += qj
        if float(prefix) > threshold:
            take = m + 1
            break
    return np.array(sorted(cand[:take]), dtype=np.int64)


def select_rows(mask: np.ndarray, conf: np.ndarray, c: np.ndarray, k: int, p: float, sigma: float,
                forced: Iterable[int] = (), stage2_candidates: int = 0,
                key: Optional[np.ndarray] = None, block: Optional[Tuple[int, int]] = None
                ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Both stages and their union (the index set of Eq. 5), for one sequence.

    stage2_candidates = 0: candidates are the known (prompt / decoded) positions;
                        1: every position not taken by stage 1.
    Returns (S ascending, M* ascending, U ascending).
    """
    mask = np.asarray(mask).astype(bool)
    m_star = stage1_select(mask, conf, k, sigma, key=key, block=block)
    if stage2_candidates == 0:
        cand = ~mask
    else:
        cand = np.ones_like(mask)
        cand[m_star] = False
    u = stage2_select(c, cand, p)
    s = sorted(set(m_star.tolist()) | set(u.tolist()) | {int(f) for f in forced})
    return np.array(s, dtype=np.int64), m_star, u
