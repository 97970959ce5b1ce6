"""The C-ABI library loads, exports every function the header declares, and rejects bad
arguments on the host before touching a device (no compute calls: runs without a GPU)."""
import ctypes
import os
import re

import pytest

from paper_2511_22481_b200 import binding as B
from paper_2511_22481_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    builder.build()
    return B.load()


def _declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(omni_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_function_is_exported(lib):
    declared = _declared_functions()
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_version_and_status_strings(lib):
    assert B.omni_version() >= 1000
    seen = {B.status_string(c) for c in range(9)}
    assert len(seen) == 9 and "ok" in seen


def test_descriptor_mirror_has_the_c_layout():
    assert ctypes.sizeof(B.OmniDesc) == 48
    assert B.OmniDesc.num_pages.offset == 0 and B.OmniDesc.batch.offset == 8
    assert B.OmniDesc.softmax_scale.offset == 40 and B.OmniDesc.flags.offset == 44


def _desc(**kw):
    args = dict(batch=2, num_heads=128, num_pages=8, max_pages_per_req=4, max_sel=256, softmax_scale=0.1)
    args.update(kw)
    return B.make_desc(**args)


def test_bad_descriptors_are_rejected(lib):
    for kw in (dict(batch=0), dict(num_heads=0), dict(num_heads=129), dict(d_qk=512), dict(d_v=576),
               dict(page_size=128), dict(num_pages=0), dict(max_sel=0), dict(num_splits=-1),
               dict(num_splits=1000), dict(max_pages_per_req=0)):
        d = _desc(**kw)
        assert B.omni_sparse_mla_workspace_bytes(d) == 0, kw
        assert B.omni_sparse_mla_num_splits(d) == 0, kw
        code = lib.omni_sparse_mla_decode(ctypes.byref(d), *([ctypes.c_void_p(256)] * 7),
                                          ctypes.c_void_p(256), 1 << 30, None, None)
        assert code == 2, kw                                 # OMNI_ERR_SHAPE


def test_null_and_misaligned_pointers_are_rejected(lib):
    d = _desc()
    ok = ctypes.c_void_p(4096)
    for missing in range(7):
        ptrs = [ok] * 7
        ptrs[missing] = None
        assert lib.omni_sparse_mla_decode(ctypes.byref(d), *ptrs, ok, 1 << 30, None, None) == 1
    assert lib.omni_sparse_mla_decode(None, *([ok] * 7), ok, 1 << 30, None, None) == 1
    ptrs = [ok] * 7
    ptrs[1] = ctypes.c_void_p(4096 + 64)                      # kv_cache must be 128-byte aligned
    assert lib.omni_sparse_mla_decode(ctypes.byref(d), *ptrs, ok, 1 << 30, None, None) == 3
    ptrs = [ok] * 7
    ptrs[0] = ctypes.c_void_p(4096 + 2)                       # q must be 16-byte aligned
    assert lib.omni_sparse_mla_decode(ctypes.byref(d), *ptrs, ok, 1 << 30, None, None) == 3
    assert lib.omni_sparse_mla_combine(ctypes.byref(d), 0, ok, ok, None, ok, ok, None) == 2
    assert lib.omni_sparse_mla_combine(ctypes.byref(d), 2, None, ok, None, ok, ok, None) == 1
    assert lib.omni_sparse_mla_validate(ctypes.byref(d), ok, ok, ok, None, None) == 1
    assert lib.omni_sparse_mla_resolve_rows(ctypes.byref(d), ok, ok, ok, None, None) == 1
    assert lib.omni_sparse_mla_decode_host(ctypes.byref(d), *([ok] * 7), None, 0, ok, 0, None, None) == 1


def test_sink_recent_entry_point_checks_its_arguments(lib):
    ok = ctypes.c_void_p(4096)
    i32 = ctypes.c_int32
    call = lambda d, ptrs, ns, nr: lib.omni_sparse_mla_decode_sink_recent(
        ctypes.byref(d), ptrs[0], ptrs[1], ptrs[2], ptrs[3], i32(ns), i32(nr), ptrs[4], ptrs[5], ok, 1 << 30, None, None)
    d = _desc(max_sel=256)                                    # 4 pages of 64 tokens per request
    for missing in range(6):
        ptrs = [ok] * 6
        ptrs[missing] = None
        assert call(d, ptrs, 64, 64) == 1                     # OMNI_ERR_NULL (ctx_len included)
    assert call(d, [ok] * 6, -1, 64) == 2 and call(d, [ok] * 6, 64, -1) == 2
    # max_sel must cover min(n_sink + n_recent, longest context)
    assert call(_desc(max_sel=127), [ok] * 6, 64, 64) == 2
    assert call(_desc(max_sel=255), [ok] * 6, 1000, 1000) == 2
    ptrs = [ok] * 6
    ptrs[3] = ctypes.c_void_p(4096 + 2)                       # ctx_len must be 4-byte aligned
    assert call(d, ptrs, 64, 64) == 3
    assert B.omni_sparse_mla_num_launches(_desc(batch=0)) == 0


def test_topk_select_checks_its_arguments(lib):
    ok = ctypes.c_void_p(4096)
    i32 = ctypes.c_int32
    call = lambda scores, ctx, batch, stride, k, idx, ln: lib.omni_topk_select(
        scores, ctx, i32(batch), i32(stride), i32(k), idx, ln, None)
    for missing in range(4):
        ptrs = [ok] * 4
        ptrs[missing] = None
        assert call(ptrs[0], ptrs[1], 2, 64, 8, ptrs[2], ptrs[3]) == 1        # OMNI_ERR_NULL
    for batch, stride, k in ((0, 64, 8), (2, 0, 1), (2, 64, 0), (2, 64, 65), (2, 131073, 8)):
        assert call(ok, ok, batch, stride, k, ok, ok) == 2                    # OMNI_ERR_SHAPE
    odd = ctypes.c_void_p(4096 + 2)
    assert call(odd, ok, 2, 64, 8, ok, ok) == 3 and call(ok, ok, 2, 64, 8, odd, ok) == 3      # OMNI_ERR_ALIGN


def test_workspace_grows_with_forced_splits(lib):
    a = B.omni_sparse_mla_workspace_bytes(_desc(num_splits=1))
    b = B.omni_sparse_mla_workspace_bytes(_desc(num_splits=4))
    assert 0 < a < b and b >= 2 * 4 * 128 * 513 * 4
    assert B.omni_sparse_mla_num_splits(_desc(num_splits=4)) == 4
    assert B.omni_sparse_mla_host_staging_bytes(_desc()) >= 2 * 128 * (576 + 512) * 2


def test_binding_refuses_cpu_tensors_for_device_arguments():
    import torch
    d = _desc()
    t = torch.zeros(4, dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        B._ptr(t, torch.bfloat16, "cuda", "q")
    with pytest.raises(TypeError):
        B._ptr(t, torch.int32, "cpu", "sel_idx")
