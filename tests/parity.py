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
