"""Oracle: attention rollout influence scores (Section 4.2, Eq. 6-9).  Test infrastructure.

`literal` writes the equations out with dense L x L matrices.  `chain` is the
same quantity as a row-vector recursion: c = 1^T W^(N) ... W^(1), evaluated from
the left, using only that a row of W^(l) is e_i for an unselected row and
(Abar_i + e_i)/rowsum for a selected one.  The tests hold the two against each
other and against closed forms.
"""
from __future__ import annotations

from typing import Sequence

import numpy as np


def literal(abar: Sequence[np.ndarray], sel: np.ndarray, L: int) -> np.ndarray:
    """Eq. 6-9 as printed.  abar[l]: [n][L] head-averaged attention of layer l+1 for rows `sel`."""
    sel = np.asarray(sel, dtype=np.int64)
    C = np.eye(L, dtype=np.float64)                              # C^(0) = I
    for A in abar:
        E = np.eye(L, dtype=np.float64)                          # Eq. 6: unselected rows are e_i
        if sel.size:
            E[sel, :] = A
        W = E + np.eye(L, dtype=np.float64)                      # Eq. 7: residual, then row-normalise
        W = W / np.sum(W, axis=1, keepdims=True)
        C = W @ C                                                # Eq. 8
    return np.sum(C, axis=0)                                     # Eq. 9: column sums


def chain(abar: Sequence[np.ndarray], sel: np.ndarray, L: int) -> np.ndarray:
    """c^T = 1^T W^(N) W^(N-1) ... W^(1), one vector-matrix product per layer, last layer first."""
    sel = np.asarray(sel, dtype=np.int64)
    u = np.ones(L, dtype=np.float64)
    for A in reversed(list(abar)):
        nxt = u.copy()                                           # unselected rows of W are e_i
        if sel.size:
            rowsum = np.sum(A, axis=1) + 1.0                     # row sum of (Abar_i + e_i)
            wgt = u[sel] / rowsum                                # [n]
            nxt[sel] = 0.0
            nxt += wgt @ A                                       # sum_i u_i Abar_ij / rowsum_i
            nxt[sel] += wgt                                      # the +e_i part of the same rows
        u = nxt
    return u
