"""The workspace-free decode entry point, for callers that may not allocate device memory.

Some users of this library run where cudaMalloc is off limits: a plug-in inside a serving
engine that gave all free GPU memory to its KV-cache pool at start-up, or a decode loop that
cannot afford the device-wide synchronisation an allocation implies.  For them
``omni_sparse_mla_decode_static`` keeps the split-KV scratch in a fixed array inside the library.
These tests call it through the C ABI twice in a row (the array keeps the first call's
contents, so the second call shows that stale scratch does no harm) and compare each result
with ``omni_sparse_mla_decode`` on the same inputs and with the CPU oracle, under the same
tolerance as the other parity tests.  The file name sorts last so that a run that stops at the first failure has
already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2511_22481_b200 import binding as B
from paper_2511_22481_b200 import build as builder
from paper_2511_22481_b200 import workloads as W
from parity import ABS_TOL, LSE_TOL, compare, oracle_subset


def _desc(w, num_splits=0):
    return B.make_desc(w.batch, w.heads, w.num_pages, w.max_pages_per_req, w.max_sel, w.scale,
                       num_splits=num_splits)


def _static(w, desc):
    out = torch.full((w.batch, w.heads, w.d_v), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((w.batch, w.heads), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.omni_sparse_mla_decode_static(desc, w.q, w.kv_cache, w.page_table, w.sel_idx, w.sel_len, out,
                                    lse, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out, lse


def _same(out, lse, ref_out, ref_lse):
    err = (out.float() - ref_out.float()).abs()
    bound = ABS_TOL + 2.0 ** -8 * ref_out.float().abs()
    assert bool((err <= bound).all()), "max abs difference %.3e" % float(err.max())
    both_inf = torch.isneginf(lse) & torch.isneginf(ref_lse)
    diff = torch.where(both_inf, torch.zeros_like(lse), (lse - ref_lse).abs())
    assert float(torch.nan_to_num(diff, nan=float("inf")).max()) <= LSE_TOL


@pytest.mark.gpu
def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row():
    # two different problems back to back: the second call finds the first one's partials in
    # the shared scratch; both use several splits, the second has empty splits and an empty request
    first = W.config4_topk("cuda", batch=3, ctx_pages=64, k=777)
    rng = np.random.default_rng(7)
    lens = [0, 65, 300, 513]
    tables = W._shuffled_tables(rng, [16] * len(lens), True)
    second = W._pack("ragged", 7, 128, [16] * len(lens), tables,
                     [rng.permutation(16 * 64)[:n].astype(np.int32) for n in lens], "cuda", {})
    for w, splits in ((first, 3), (second, 5), (first, 0)):
        desc = _desc(w, splits)
        assert B.omni_sparse_mla_workspace_bytes(desc) <= B.OMNI_STATIC_SCRATCH_BYTES
        plan = B.plan_for(w, num_splits=splits)
        plan.run(w.q, w.kv_cache, w.page_table, w.sel_idx, w.sel_len)
        torch.cuda.synchronize()
        out, lse = _static(w, desc)
        _same(out, lse, plan.out, plan.lse)
        ref_out, ref_lse, _ = oracle_subset(w)
        compare(out.cpu(), lse.cpu(), ref_out, ref_lse, "static scratch entry point, splits=%d" % splits)


@pytest.mark.gpu
def test_static_scratch_decode_rejects_problems_beyond_its_fixed_size():
    w = W.config4_topk("cuda", batch=2, ctx_pages=32, k=300)
    big = B.make_desc(256, 128, w.num_pages, w.max_pages_per_req, 8192, w.scale, num_splits=8)
    assert B.omni_sparse_mla_workspace_bytes(big) > B.OMNI_STATIC_SCRATCH_BYTES
    out = torch.empty((256, 128, 512), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((256, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(B.OmniError) as info:
        B.omni_sparse_mla_decode_static(big, w.q, w.kv_cache, w.page_table, w.sel_idx, w.sel_len, out, lse)
    assert info.value.code == 4                              # OMNI_ERR_WORKSPACE: nothing launched


def test_static_scratch_size_matches_the_header():
    builder.build()
    assert "omni_sparse_mla_decode_static" in B.EXPORTS
    import os
    import re
    hdr = open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))),
                            "include", "omni_mla.h")).read()
    m = re.search(r"#define OMNI_STATIC_SCRATCH_BYTES \((\d+)u \* (\d+)u \* (\d+)u\)", hdr)
    assert m and int(m.group(1)) * int(m.group(2)) * int(m.group(3)) == B.OMNI_STATIC_SCRATCH_BYTES
    d = B.make_desc(1, 1, 1, 1, 1, 1.0, d_qk=1)              # bad shape is reported before any device work
    assert B.load().omni_sparse_mla_decode_static(ctypes.byref(d), *([None] * 9)) == 2
    assert B.load().omni_sparse_mla_decode_static(None, *([None] * 9)) == 1
