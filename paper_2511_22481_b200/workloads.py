"""Seeded synthetic decode workloads (inputs only; no attention arithmetic lives here).

Every workload is a batch of independent decode requests over one shared paged pool of
latent KV rows, shaped like DeepSeek-R1 MLA decode: d_qk = 576 (512 latent + 64 rope),
d_v = 512, 64-token pages.  Values are bf16 RN(0.5 * N(0,1)); the bits produced by the
seeded torch generator on the chosen device are the definition of the input, so a checker
must read back the bits it needs rather than regenerate them elsewhere.  Index structures
(page table, selection lists) come from a numpy generator and are identical on any device.

Selections follow the shapes of the OmniAttn index set (sink + recent, Eq. 2 of the paper)
extended with randomly chosen middle pages or a token-level top-k, as decode-time sparse
attention variants would produce.  Unused tails of ``sel_idx`` hold -1 on purpose: entries
at or beyond ``sel_len[b]`` must never be read as token positions.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

D_QK = 576
D_V = 512
PAGE = 64
SCALE = 1.0 / math.sqrt(192.0)


@dataclass
class Workload:
    name: str
    batch: int
    heads: int
    num_pages: int
    max_pages_per_req: int
    max_sel: int
    q: torch.Tensor            # bf16 [B, H, 576]
    kv_cache: torch.Tensor     # bf16 [num_pages, 64, 576]
    page_table: torch.Tensor   # int32 [B, max_pages_per_req]
    sel_idx: torch.Tensor      # int32 [B, max_sel]
    sel_len: torch.Tensor      # int32 [B]
    ctx_len: np.ndarray        # int64 [B]
    scale: float = SCALE
    d_qk: int = D_QK
    d_v: int = D_V
    page_size: int = PAGE
    meta: dict = field(default_factory=dict)

    @property
    def selected_tokens(self) -> int:
        return int(self.sel_len.sum().item())

    @property
    def selected_kv_bytes(self) -> int:
        return self.selected_tokens * self.d_qk * 2

    def to(self, device) -> "Workload":
        kw = dict(self.__dict__)
        for k in ("q", "kv_cache", "page_table", "sel_idx", "sel_len"):
            kw[k] = kw[k].to(device)
        return Workload(**kw)


def _normal_bf16(shape, gen: torch.Generator, device, chunk_rows: int = 1 << 16) -> torch.Tensor:
    """bf16 RN(0.5*N(0,1)), filled in fixed-size row chunks so no large fp32 temp exists."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1, shape[-1])
    for r0 in range(0, flat.shape[0], chunk_rows):
        r1 = min(flat.shape[0], r0 + chunk_rows)
        tmp = torch.randn((r1 - r0, shape[-1]), generator=gen, device=device, dtype=torch.float32)
        flat[r0:r1] = (tmp * 0.5).to(torch.bfloat16)
    return out


def _values(seed: int, batch: int, heads: int, num_pages: int, device):
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    q = _normal_bf16((batch, heads, D_QK), gen, device)
    kv = _normal_bf16((num_pages, PAGE, D_QK), gen, device)
    return q, kv


def _pack(name, seed, heads, pages_per_req, page_table_rows, selections, device, meta,
          make_values=True) -> Workload:
    batch = len(selections)
    num_pages = int(sum(pages_per_req))
    max_pages = int(max(pages_per_req))
    max_sel = max(1, max(len(s) for s in selections))
    pt = np.full((batch, max_pages), -1, dtype=np.int32)
    si = np.full((batch, max_sel), -1, dtype=np.int32)
    sl = np.zeros((batch,), dtype=np.int32)
    for b in range(batch):
        pt[b, : pages_per_req[b]] = page_table_rows[b]
        si[b, : len(selections[b])] = selections[b]
        sl[b] = len(selections[b])
    if make_values:
        q, kv = _values(seed, batch, heads, num_pages, device)
    else:
        q = kv = None
    return Workload(
        name=name, batch=batch, heads=heads, num_pages=num_pages, max_pages_per_req=max_pages,
        max_sel=max_sel, q=q, kv_cache=kv,
        page_table=torch.from_numpy(pt).to(device), sel_idx=torch.from_numpy(si).to(device),
        sel_len=torch.from_numpy(sl).to(device),
        ctx_len=np.asarray(pages_per_req, dtype=np.int64) * PAGE, meta=dict(meta, seed=seed))


def _page_tokens(pages) -> np.ndarray:
    pages = np.asarray(pages, dtype=np.int64)
    return (pages[:, None] * PAGE + np.arange(PAGE)[None, :]).reshape(-1).astype(np.int32)


def _shuffled_tables(rng: np.random.Generator, pages_per_req, shuffle: bool):
    total = int(sum(pages_per_req))
    pool = rng.permutation(total) if shuffle else np.arange(total)
    rows, off = [], 0
    for n in pages_per_req:
        rows.append(pool[off: off + n].astype(np.int32))
        off += n
    return rows


def page_sparse(name: str, seed: int, batch: int, heads: int, ctx_pages, recent_pages,
                middle_pages, device="cpu", shuffle: bool = True, make_values=True) -> Workload:
    """Page-granular selection: page 0 (sink) + randomly drawn middle pages + the last pages.

    ``ctx_pages``, ``recent_pages`` and ``middle_pages`` are ints or per-request sequences.
    Middle pages are drawn uniformly without replacement from the pages strictly between the
    sink page and the recent region, and kept in drawn order.
    """
    rng = np.random.default_rng(seed)
    as_list = lambda v: [int(v)] * batch if np.isscalar(v) else [int(x) for x in v]
    ctx_pages, recent_pages, middle_pages = as_list(ctx_pages), as_list(recent_pages), as_list(middle_pages)
    tables = _shuffled_tables(rng, ctx_pages, shuffle)
    sels = []
    for b in range(batch):
        n, r, m = ctx_pages[b], recent_pages[b], middle_pages[b]
        first_recent = max(1, n - r)
        mid_pool = np.arange(1, first_recent)
        m = min(m, len(mid_pool))
        mid = rng.choice(mid_pool, size=m, replace=False) if m > 0 else np.zeros(0, dtype=np.int64)
        pages = np.concatenate([[0], mid, np.arange(first_recent, n)]).astype(np.int64)
        sels.append(_page_tokens(pages))
    return _pack(name, seed, heads, ctx_pages, tables, sels, device,
                 dict(kind="page_sparse"), make_values)


def sink_recent(name: str, seed: int, batch: int, heads: int, ctx_tokens, n_sink: int,
                n_recent: int, device="cpu", shuffle: bool = True, make_values=True) -> Workload:
    """The paper's own selection rule (Eq. 2): the first ``n_sink`` and the last ``n_recent``
    positions of each context, as an increasing list without repeats.  ``ctx_tokens`` is an int
    or a per-request sequence of context lengths in tokens (they need not fill their last page).
    The same requests can be given to the range entry point as (ctx_len, n_sink, n_recent):
    ``meta`` carries the two sizes and ``ctx_len`` the lengths."""
    rng = np.random.default_rng(seed)
    ctx = [int(ctx_tokens)] * batch if np.isscalar(ctx_tokens) else [int(x) for x in ctx_tokens]
    pages = [max(1, -(-m // PAGE)) for m in ctx]
    tables = _shuffled_tables(rng, pages, shuffle)
    sels = []
    for m in ctx:
        head = np.arange(0, min(n_sink, m))
        tail = np.arange(max(len(head), m - n_recent), m)
        sels.append(np.concatenate([head, tail]).astype(np.int32))
    w = _pack(name, seed, heads, pages, tables, sels, device,
              dict(kind="sink_recent", n_sink=int(n_sink), n_recent=int(n_recent)), make_values)
    w.ctx_len = np.asarray(ctx, dtype=np.int64)
    return w


def token_topk(name: str, seed: int, batch: int, heads: int, ctx_pages: int, k: int,
               device="cpu", make_values=True) -> Workload:
    """Token-level selection: the k best positions of a seeded random score vector, in
    best-first order (unsorted positions, scattered over pages)."""
    rng = np.random.default_rng(seed)
    pages = [int(ctx_pages)] * batch
    tables = _shuffled_tables(rng, pages, True)
    sels = []
    for _ in range(batch):
        score = rng.standard_normal(ctx_pages * PAGE)
        order = np.argsort(-score, kind="stable")[:k]
        sels.append(order.astype(np.int32))
    return _pack(name, seed, heads, pages, tables, sels, device, dict(kind="token_topk"),
                 make_values)


def dense(name: str, seed: int, batch: int, heads: int, ctx_pages: int, device="cpu",
          shuffle=True, make_values=True) -> Workload:
    """Every token selected, in position order (the uncompressed-layer case)."""
    rng = np.random.default_rng(seed)
    pages = [int(ctx_pages)] * batch
    tables = _shuffled_tables(rng, pages, shuffle)
    sels = [np.arange(ctx_pages * PAGE, dtype=np.int32) for _ in range(batch)]
    return _pack(name, seed, heads, pages, tables, sels, device, dict(kind="dense"), make_values)


# ---------------------------------------------------------------------------------------
# The five named configurations.
# ---------------------------------------------------------------------------------------

def config1_tiny(device="cpu") -> Workload:
    """Batch 1, 16 heads, 4096-token context, identity page table; page 0 + last 256 tokens
    + 8 middle pages = 832 selected tokens; seed 0."""
    return page_sparse("config1_tiny", 0, 1, 16, 64, 4, 8, device, shuffle=False)


def config2_r1(device="cpu", middle_pages: int = 24, batch: int = 32) -> Workload:
    """Batch 32, 128 heads, 32768-token contexts over a shuffled shared pool; page 0 + last
    512 tokens + 24 middle pages = 2112 selected tokens per request; seed 1.  With
    ``middle_pages=23`` the total is the round 2048."""
    return page_sparse("config2_r1", 1, batch, 128, 512, 8, middle_pages, device)


def config3_ragged(device="cpu", batch: int = 128, make_values=True) -> Workload:
    """Batch 128, 128 heads, context lengths uniform in [4096, 65536] rounded to pages;
    one eighth of each request's pages selected (page 0 + last 8 pages + middle), never
    fewer than the 9 fixed pages; seed 2."""
    rng = np.random.default_rng(2)
    ctx_pages = rng.integers(64, 1024, size=batch, endpoint=True)
    n_sel = np.maximum(9, np.rint(ctx_pages / 8.0).astype(np.int64))
    return page_sparse("config3_ragged", 2, batch, 128, ctx_pages, 8, n_sel - 9, device,
                       make_values=make_values)


def config4_topk(device="cpu", batch: int = 16, ctx_pages: int = 2048, k: int = 2048) -> Workload:
    """Batch 16, 128 heads, 131072-token contexts; 2048 token positions per request from a
    top-k over random scores; seed 3."""
    return token_topk("config4_topk", 3, batch, 128, ctx_pages, k, device)


SWEEP_BATCHES = (1, 8, 32, 128, 256)
SWEEP_SELECTED = (512, 2048, 8192)


def config5_cell(batch: int, n_sel: int, device="cpu", dense_variant: bool = False,
                 ctx_pages: int = 1024) -> Workload:
    """One cell of the batch x selected-tokens sweep at 65536-token contexts (seeds 10-24 in
    batch-major order).  Sparse cells: page 0 + the last n_sel/4 tokens + middle pages up to
    n_sel.  ``dense_variant`` selects every token of the same pool and page table."""
    seed = 10 + SWEEP_BATCHES.index(batch) * len(SWEEP_SELECTED) + SWEEP_SELECTED.index(n_sel)
    name = "config5_B%d_N%d%s" % (batch, n_sel, "_dense" if dense_variant else "")
    if dense_variant:
        return dense(name, seed, batch, 128, ctx_pages, device)
    tot = n_sel // PAGE
    recent = tot // 4
    return page_sparse(name, seed, batch, 128, ctx_pages, recent, tot - 1 - recent, device)
