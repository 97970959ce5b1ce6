"""Helpers for the GPU parity tests: run the CUDA path through the C ABI binding, compute the
same (request, head) results with the CPU oracle on the same bits, and compare.

Tolerances (bf16 inputs, fp32 accumulation, bf16 output):
  * out: every element |gpu - oracle| <= 2e-3 + 2^-8 * |oracle|.  The second term is one bf16
         ulp of the value: the output format alone rounds by up to half of it, which exceeds
         2e-3 once |out| >= 0.5 (selections of one or two tokens).  At the benchmark shapes
         |out| < 0.1 and the tests also assert the plain max |gpu - oracle| <= 2e-3
         (``strict_abs``).
  * out: per (request, head) row max_d |gpu - oracle| <= 1e-2 * max_d |oracle| (element-wise
         relative error is meaningless next to zero crossings, so the relative bound is taken
         against the row's largest magnitude)
  * lse: |gpu - oracle| <= 2e-3
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2511_22481_b200 import binding as B

ABS_TOL = 2e-3
REL_TOL = 1e-2
LSE_TOL = 2e-3


def run_gpu(w, flags=0, num_splits=0, plan=None):
    plan = plan or B.plan_for(w, num_splits=num_splits, flags=flags)
    plan.status.zero_()
    plan.run(w.q, w.kv_cache, w.page_table, w.sel_idx, w.sel_len)
    torch.cuda.synchronize()
    return plan


def oracle_subset(w, reqs=None, heads=None):
    """Oracle results for the listed requests and heads of a (device-resident) workload.

    Index arrays go to the host whole; of the KV pool only the selected rows are copied.
    Returns (out f64 [len(reqs), len(heads), d_v], lse f64 [len(reqs), len(heads)], rows).
    """
    reqs = list(range(w.batch)) if reqs is None else list(reqs)
    heads = list(range(w.heads)) if heads is None else list(heads)
    pt = w.page_table.cpu().numpy()[reqs]
    si = w.sel_idx.cpu().numpy()[reqs]
    sl = w.sel_len.cpu().numpy()[reqs]
    rows = oracle.resolve_rows(pt, si, sl, w.page_size, w.num_pages)
    gather = torch.from_numpy(np.where(rows < 0, 0, rows)).to(w.kv_cache.device)
    krows = w.kv_cache.view(-1, w.d_qk)[gather.view(-1)].view(len(reqs), -1, w.d_qk).cpu()
    q = w.q[torch.tensor(reqs, device=w.q.device)][:, torch.tensor(heads, device=w.q.device)].cpu()
    out, lse = oracle.attend_rows(q, krows, sl, w.d_v, w.scale)
    return out, lse, rows


def compare(gpu_out, gpu_lse, ref_out, ref_lse, what="", strict_abs=False):
    g = gpu_out.to(torch.float64).cpu().numpy()
    gl = gpu_lse.to(torch.float64).cpu().numpy()
    err = np.abs(g - ref_out)
    row_ref = np.abs(ref_out).max(axis=-1)
    row_err = err.max(axis=-1)
    rel = np.where(row_ref > 0, row_err / np.where(row_ref > 0, row_ref, 1.0), row_err)
    both_inf = np.isneginf(gl) & np.isneginf(ref_lse)
    with np.errstate(invalid="ignore"):
        lse_err = np.where(both_inf, 0.0, np.abs(gl - ref_lse))
    stats = dict(max_abs=float(err.max(initial=0.0)), max_row_rel=float(rel.max(initial=0.0)),
                 max_lse=float(np.nan_to_num(lse_err, nan=np.inf).max(initial=0.0)))
    assert np.all(np.isfinite(g)), what + ": non-finite output"
    excess = float((err - (ABS_TOL + 2.0 ** -8 * np.abs(ref_out))).max(initial=-1.0))
    assert excess <= 0.0, "%s: abs err exceeds 2e-3 + ulp by %.3e (max abs %.3e)" % (what, excess, stats["max_abs"])
    if strict_abs:
        assert stats["max_abs"] <= ABS_TOL, "%s: max abs err %.3e" % (what, stats["max_abs"])
    assert stats["max_row_rel"] <= REL_TOL, "%s: max row-relative err %.3e" % (what, stats["max_row_rel"])
    assert stats["max_lse"] <= LSE_TOL, "%s: max lse err %.3e" % (what, stats["max_lse"])
    return stats


def check_workload(w, flags=0, num_splits=0, reqs=None, heads=None, what="", strict_abs=False):
    plan = run_gpu(w, flags=flags, num_splits=num_splits)
    assert int(plan.status.item()) == 0, what + ": device status %d" % int(plan.status.item())
    ref_out, ref_lse, _ = oracle_subset(w, reqs, heads)
    r = torch.arange(w.batch) if reqs is None else torch.tensor(list(reqs))
    h = torch.arange(w.heads) if heads is None else torch.tensor(list(heads))
    g = plan.out.cpu()[r][:, h]
    gl = plan.lse.cpu()[r][:, h]
    return compare(g, gl, ref_out, ref_lse, what, strict_abs), plan


# ------------------------------------------------------------------ 8-bit latent cache

def quantise_pool_q8(w, check_rows=4096, seed=0):
    """8-bit form of a workload's pool.  The pool is quantised on the device through the C ABI
    and the result is compared, bit for bit, with the oracle's quantiser on `check_rows` rows
    (all rows of a small pool), so the decode tests run on a cache the oracle vouches for."""
    from oracle import q8
    rows = w.kv_cache.view(-1, w.d_qk)
    n = rows.shape[0]
    cache = torch.empty((n, B.OMNI_Q8_ROW_BYTES), dtype=torch.uint8, device=rows.device)
    scale = torch.empty((n,), dtype=torch.float32, device=rows.device)
    B.omni_kv_quantize_q8(rows, cache, scale)
    torch.cuda.synchronize()
    pick = np.arange(n) if n <= check_rows else np.sort(np.random.default_rng(seed).choice(n, check_rows, replace=False))
    idx = torch.from_numpy(pick).to(rows.device)
    bits = rows[idx].cpu().view(torch.int16).numpy().view(np.uint16)
    want_cache, want_scale = q8.quantise_rows(bits)
    assert np.array_equal(scale[idx].cpu().numpy().view(np.uint32), want_scale.view(np.uint32)), "scales differ"
    assert np.array_equal(cache[idx].cpu().numpy(), want_cache), "codes differ"
    return cache, scale


def oracle_subset_q8(w, cache, scale, reqs=None, heads=None):
    """Oracle results over the de-quantised rows, for the listed requests and heads."""
    from oracle import q8
    reqs = list(range(w.batch)) if reqs is None else list(reqs)
    heads = list(range(w.heads)) if heads is None else list(heads)
    pt = w.page_table.cpu().numpy()[reqs]
    si = w.sel_idx.cpu().numpy()[reqs]
    sl = w.sel_len.cpu().numpy()[reqs]
    rows = oracle.resolve_rows(pt, si, sl, w.page_size, w.num_pages)
    gather = torch.from_numpy(np.where(rows < 0, 0, rows)).to(cache.device).view(-1)
    # the rows the oracle attends to are quantised by the oracle itself from the seeded bf16 pool;
    # the device-made cache must hold the same bits there, and is not otherwise used as an input
    bits = w.kv_cache.view(-1, w.d_qk)[gather].cpu().view(torch.int16).numpy().view(np.uint16)
    own_cache, own_scale = q8.quantise_rows(bits)
    live = np.asarray(rows).reshape(-1) >= 0
    assert np.array_equal(cache[gather].cpu().numpy()[live], own_cache[live]), "codes of the selected rows differ"
    assert np.array_equal(scale[gather].cpu().numpy().view(np.uint32)[live], own_scale.view(np.uint32)[live]), \
        "scales of the selected rows differ"
    krows = q8.dequantise_rows(own_cache, own_scale).reshape(len(reqs), -1, w.d_qk)
    q = w.q[torch.tensor(reqs, device=w.q.device)][:, torch.tensor(heads, device=w.q.device)].cpu().to(torch.float64).numpy()
    return q8.attend_dequantised(q, krows, sl, w.d_v, w.scale)


def check_workload_q8(w, flags=0, num_splits=0, reqs=None, heads=None, what="", strict_abs=False, quantised=None):
    cache, scale = quantised or quantise_pool_q8(w)
    plan = B.plan_for(w, num_splits=num_splits, flags=flags)
    plan.status.zero_()
    B.omni_sparse_mla_decode_q8(plan.desc, w.q, cache, scale, w.page_table, w.sel_idx, w.sel_len, plan.out, plan.lse,
                                plan.workspace, plan.status)
    torch.cuda.synchronize()
    assert int(plan.status.item()) == 0, what + ": device status %d" % int(plan.status.item())
    ref_out, ref_lse = oracle_subset_q8(w, cache, scale, reqs, heads)
    r = torch.arange(w.batch) if reqs is None else torch.tensor(list(reqs))
    h = torch.arange(w.heads) if heads is None else torch.tensor(list(heads))
    return compare(plan.out.cpu()[r][:, h], plan.lse.cpu()[r][:, h], ref_out, ref_lse, what, strict_abs), plan
