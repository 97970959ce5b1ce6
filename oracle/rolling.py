"""Rolling sink + recent cache of a compressed layer, written out.  TEST INFRASTRUCTURE ONLY.

The paper's layer-wise compression keeps, for a compressed layer, only the tokens of Eq. 2's
index set: the first N_sink and the last N_recent of a context.  A cache that stores nothing
else can be a short list of 64-token pages per request: enough pages for the sink, kept for
good, and a ring of pages for the recent window.  This module states where a token lives in such
a cache and replays appends on the host, with plain loops, so that the GPU's append kernel and
its addressing can be checked against it.  Nothing here is shared with the CUDA path.
"""
from __future__ import annotations

import numpy as np

PAGE = 64


def pages_per_request(n_sink: int, n_recent: int) -> tuple[int, int]:
    """(sink pages, ring pages).  The recent window of N_recent tokens can straddle one more
    page than it fills, hence the + 1."""
    sink_pages = -(-n_sink // PAGE)
    ring_pages = -(-n_recent // PAGE) + 1
    return sink_pages, ring_pages


def position(t: int, n_sink: int, n_recent: int) -> int:
    """Position in the request's short page table of the token at absolute position t."""
    sink_pages, ring_pages = pages_per_request(n_sink, n_recent)
    block, offset = divmod(t, PAGE)
    if block < sink_pages:
        return t
    slot = sink_pages
    for _ in range(block - sink_pages):        # walk the ring one block at a time
        slot += 1
        if slot == sink_pages + ring_pages:
            slot = sink_pages
    return slot * PAGE + offset


def replay_appends(pool: np.ndarray, table_row: np.ndarray, rows: np.ndarray, n_sink: int, n_recent: int) -> None:
    """Append rows[0], rows[1], ... (tokens 0, 1, ...) of one request into ``pool``
    ([pages, 64, width]) through its page-table row, in place."""
    for t in range(rows.shape[0]):
        pos = position(t, n_sink, n_recent)
        pool[table_row[pos // PAGE], pos % PAGE] = rows[t]


def selected_rows(table_row: np.ndarray, M: int, n_sink: int, n_recent: int) -> np.ndarray:
    """Physical pool rows of Eq. 2's index set for a context of M tokens, in increasing token order."""
    out = []
    for t in range(M):
        if t < n_sink or t >= M - n_recent:
            pos = position(t, n_sink, n_recent)
            out.append(int(table_row[pos // PAGE]) * PAGE + pos % PAGE)
    return np.asarray(out, dtype=np.int64)
