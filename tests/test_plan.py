"""The split-KV plan and the planned decode call.

CPU: the plan is a pure function of the descriptor and two device facts, so its choices for the
five benchmark configurations are pinned here on the description of a 148-SM B200 (33 resident
merging clusters); a change to the heuristic shows up as a failed pin, not as a silently
different launch count in the benchmark.  GPU: the planned entry point gives the same bits as
the ordinary one and rejects what it must."""
import ctypes
import math

import pytest
import torch

from paper_2511_22481_b200 import binding as B
from paper_2511_22481_b200 import build as builder

SCALE = 1.0 / math.sqrt(192.0)


def _query(batch, heads, max_pages, max_sel, flags=0, sms=148, clusters=33):
    builder.build()
    d = B.make_desc(batch, heads, batch * max_pages, max_pages, max_sel, SCALE, flags=flags)
    return B.omni_sparse_mla_plan_query(d, sms, clusters)


def test_plan_pins_of_the_four_named_configurations():
    assert _query(1, 16, 64, 832) == (13, 2)             # config 1: launch-latency bound, many small splits
    assert _query(32, 128, 512, 2112) == (2, 1)          # config 2: two splits merged inside a cluster
    assert _query(128, 128, 1024, 8192) == (1, 1)        # config 3 (max_sel = 1/8 of 65536)
    assert _query(16, 128, 2048, 2048) == (4, 2)         # config 4


def test_plan_pins_of_the_sweep():
    want = {
        (1, 512): (1, 1), (1, 2048): (32, 2), (1, 8192): (32, 2), (1, 65536): (32, 2),
        (8, 512): (1, 1), (8, 2048): (8, 2), (8, 8192): (9, 2), (8, 65536): (9, 2),
        (32, 512): (1, 1), (32, 2048): (2, 1), (32, 8192): (2, 1), (32, 65536): (9, 2),
        (128, 512): (1, 1), (128, 2048): (1, 1), (128, 8192): (1, 1), (128, 65536): (4, 2),
        (256, 512): (1, 1), (256, 2048): (1, 1), (256, 8192): (1, 1), (256, 65536): (2, 2),
    }
    got = {key: _query(key[0], 128, 1024, key[1]) for key in want}
    assert got == want


def test_plan_follows_flags_and_device_facts():
    # no cluster merge allowed: two splits would need partial results and a second launch
    s, launches = _query(32, 128, 512, 2112, flags=B.OMNI_FLAG_NO_CLUSTER_MERGE)
    assert launches == (1 if s == 1 else 2)
    # a device that cannot keep 32 merging clusters resident cannot merge config 2 in clusters
    s, launches = _query(32, 128, 512, 2112, clusters=16)
    assert (s, launches) != (2, 1)
    # the in-kernel merge never needs a second launch; validation adds one
    assert _query(16, 128, 2048, 2048, flags=B.OMNI_FLAG_FUSED_MERGE)[1] == 1
    assert _query(16, 128, 2048, 2048, flags=B.OMNI_FLAG_VALIDATE)[1] == 3
    # forced split counts are taken as given; bad inputs give 0
    builder.build()
    d = B.make_desc(4, 128, 64, 16, 1024, SCALE, num_splits=5)
    assert B.omni_sparse_mla_plan_query(d, 148, 33)[0] == 5
    assert B.omni_sparse_mla_plan_query(d, 0, 33)[0] == 0
    bad = B.make_desc(4, 128, 64, 16, 1024, SCALE, d_qk=512)
    assert B.omni_sparse_mla_plan_query(bad, 148, 33)[0] == 0


def test_plan_init_argument_checks_need_no_device():
    builder.build()
    lib = B.load()
    d = B.make_desc(1, 128, 4, 4, 64, SCALE)
    plan = B.LaunchPlan()
    assert plan.address % 64 == 0
    assert lib.omni_sparse_mla_plan_init(ctypes.byref(d), None, None, plan.ptr) == 1           # OMNI_ERR_NULL
    assert lib.omni_sparse_mla_plan_init(ctypes.byref(d), ctypes.c_void_p(256), ctypes.c_void_p(256), None) == 1
    assert lib.omni_sparse_mla_plan_init(ctypes.byref(d), ctypes.c_void_p(256), ctypes.c_void_p(256),
                                         ctypes.c_void_p(plan.address + 8)) == 3                # OMNI_ERR_ALIGN
    bad = B.make_desc(1, 128, 4, 4, 64, SCALE, page_size=32)
    assert lib.omni_sparse_mla_plan_init(ctypes.byref(bad), ctypes.c_void_p(256), ctypes.c_void_p(256), plan.ptr) == 2
    assert lib.omni_sparse_mla_plan_init(ctypes.byref(d), ctypes.c_void_p(264), ctypes.c_void_p(256), plan.ptr) == 3
    # a plan that was never completed is refused by the planned call before anything else happens
    one = ctypes.c_void_p(256)
    assert lib.omni_sparse_mla_decode_planned(plan.ptr, one, one, one, one, one, None, 0, None, None) == 2
    assert lib.omni_sparse_mla_decode_planned(None, one, one, one, one, one, None, 0, None, None) == 1


@pytest.mark.gpu
@pytest.mark.parametrize("splits,flags", [(0, 0), (1, 0), (2, 0), (3, 0), (3, B.OMNI_FLAG_FUSED_MERGE), (2, B.OMNI_FLAG_SIMT)])
def test_planned_call_gives_the_same_bits_as_the_ordinary_call(splits, flags):
    from paper_2511_22481_b200 import workloads as W
    w = W.config4_topk("cuda", batch=5, ctx_pages=48, k=900)
    ref = B.plan_for(w, num_splits=splits, flags=flags)
    ref.run(w.q, w.kv_cache, w.page_table, w.sel_idx, w.sel_len)
    plan = B.omni_sparse_mla_plan_init(ref.desc, w.q, w.kv_cache)
    out = torch.full_like(ref.out, float("nan"))
    lse = torch.full_like(ref.lse, float("nan"))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty_like(ref.workspace)
    B.omni_sparse_mla_decode_planned(plan, w.page_table, w.sel_idx, w.sel_len, out, lse, ws, status)
    call = B.bind_planned(plan, w.page_table, w.sel_idx, w.sel_len, out, lse, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(out, ref.out) and torch.equal(lse, ref.lse)
    out.fill_(float("nan"))
    call()                                             # pre-marshalled form of the same call
    torch.cuda.synchronize()
    assert torch.equal(out, ref.out) and torch.equal(lse, ref.lse)


@pytest.mark.gpu
def test_planned_call_checks_its_per_step_arguments():
    from paper_2511_22481_b200 import workloads as W
    w = W.config4_topk("cuda", batch=2, ctx_pages=32, k=300)
    ref = B.plan_for(w, num_splits=3)
    plan = B.omni_sparse_mla_plan_init(ref.desc, w.q, w.kv_cache)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.OmniError) as info:
        B.omni_sparse_mla_decode_planned(plan, w.page_table, w.sel_idx, w.sel_len, ref.out, ref.lse, small)
    assert info.value.code == 4                              # OMNI_ERR_WORKSPACE
    with pytest.raises(B.OmniError) as info:
        B.omni_sparse_mla_decode_planned(plan, w.page_table, w.sel_idx, w.sel_len, ref.out, ref.lse, None)
    assert info.value.code == 1                              # three splits need a workspace
    lib = B.load()
    code = lib.omni_sparse_mla_decode_planned(plan.ptr, ctypes.c_void_p(w.page_table.data_ptr()), None,
                                              ctypes.c_void_p(w.sel_len.data_ptr()), ctypes.c_void_p(ref.out.data_ptr()),
                                              ctypes.c_void_p(ref.lse.data_ptr()), None, 0, None, None)
    assert code == 1
