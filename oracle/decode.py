"""Oracle: the scheduling function G of the decoding loop (Eq. 2 and Section 4.1).  Test infrastructure.

Which masked positions are replaced by their predictions after a step.  Only positions whose
prediction the step just refreshed (selected and still masked) are eligible.
  rule 0  the single position with the highest confidence s^i ("Vanilla" scheduling, Section 5.1);
  rule 1  the single position with the highest certainty prior D(i) * s^i (Section 4.1);
  rule 2  every eligible position whose confidence exceeds the threshold, and in any case the most
          confident one (parallel decoding, appendix on parallel decoding settings).
Equal scores: the lower position wins.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

from . import selection


def commit(mask: np.ndarray, conf: np.ndarray, eligible: Sequence[int], rule: int = 0, sigma: float = 10.0,
           threshold: float = 0.9) -> Tuple[List[int], int]:
    """Positions to commit for one sequence and the best one among them (-1 if none is eligible).

    conf is the fp32 confidence vector; scores are compared in fp32, as the stored state is.
    """
    mask = np.asarray(mask).astype(bool)
    elig = [int(i) for i in eligible if mask[int(i)]]
    if not elig:
        return [], -1
    conf = np.asarray(conf, dtype=np.float32)
    if rule == 1:
        score = selection.stage1_keys(mask, conf, sigma)             # D(i) * s^i with the density of Eq. 3
    else:
        score = conf
    clean = selection._clean_score(score)
    best = min(elig, key=lambda i: (-float(clean[i]), i))
    out = {best}
    if rule == 2:
        out |= {i for i in elig if float(conf[i]) > float(np.float32(threshold))}
    return sorted(out), best
