"""Top-k selection producer, written out from its definition.  TEST INFRASTRUCTURE ONLY.

The paper's own index set is the sink + recent rule of Eq. 2; a token-level variant replaces it
with "the k tokens of highest score".  The definition used here: order the positions 0..M-1 of a
request by score, highest first, where NaN ranks below every number and -0 below +0, equal
scores by increasing position; keep the first min(k, M) positions of that order and report them
in increasing order of position.  All NaNs are equal to one another whatever their sign bit or
payload (the sign distinction applies to numbers only, where it separates -0 from +0), so among
NaNs the lower position wins.
"""
from __future__ import annotations

import numpy as np


def topk_positions(scores, M: int, k: int) -> np.ndarray:
    """Sorted positions (int32) of the min(k, M) highest of scores[0:M]."""
    s = np.asarray(scores, dtype=np.float32)[: max(0, int(M))]
    M = s.shape[0]
    take = min(int(k), M)
    if take <= 0:
        return np.zeros(0, dtype=np.int32)
    is_num = ~np.isnan(s)
    value = np.where(is_num, s, np.float32(0)).astype(np.float64)
    positive_sign = np.where(is_num, ~np.signbit(s), True)      # the sign key orders numbers only
    # np.lexsort sorts by its LAST key first; every key ascending
    order = np.lexsort((np.arange(M), ~positive_sign, -value, ~is_num))
    return np.sort(order[:take]).astype(np.int32)


def topk_batch(scores, ctx_len, k: int):
    """(sel_idx [B, k] int32 padded with -1, sel_len [B] int32) for a batch."""
    scores = np.asarray(scores, dtype=np.float32)
    B = scores.shape[0]
    sel_idx = np.full((B, int(k)), -1, dtype=np.int32)
    sel_len = np.zeros(B, dtype=np.int32)
    for b in range(B):
        M = min(max(int(ctx_len[b]), 0), scores.shape[1])
        pos = topk_positions(scores[b], M, k)
        sel_idx[b, : len(pos)] = pos
        sel_len[b] = len(pos)
    return sel_idx, sel_len
