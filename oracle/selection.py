"""The paper's index set (OmniAttn, Eq. 2), written out.  TEST INFRASTRUCTURE ONLY.

Eq. 2 keeps the first N_sink tokens (the attention sink) and the last N_recent tokens of a
context of M tokens.  The paper counts tokens from 1; positions here count from 0, so the
set is [0, N_sink) united with [M - N_recent, M).  Where the two ranges overlap the result
is their union without repeats, which is every token once N_sink + N_recent >= M.
"""
from __future__ import annotations

import numpy as np


def sink_recent(M: int, n_sink: int, n_recent: int) -> np.ndarray:
    """Sorted 0-based positions of Eq. 2's index set, int32, no duplicates."""
    if M < 0 or n_sink < 0 or n_recent < 0:
        raise ValueError("negative size")
    keep = []
    for t in range(M):
        in_sink = t < n_sink
        in_recent = t >= M - n_recent
        if in_sink or in_recent:
            keep.append(t)
    return np.asarray(keep, dtype=np.int32)
