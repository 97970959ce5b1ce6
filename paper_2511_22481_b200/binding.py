"""ctypes binding of the C ABI in ``include/omni_mla.h``.

Argument marshalling only: every function takes torch tensors (device memory and streams are
PyTorch's job here), checks dtype / device / contiguity, and passes raw pointers and sizes to
the function of the same name in ``libomni_mla.so``.  There is no Python or CPU fallback: if
the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libomni_mla.so")

OMNI_OK = 0
OMNI_DEV_BAD_INDEX = 1
OMNI_DEV_TIMEOUT = 2
OMNI_FLAG_VALIDATE = 1
OMNI_FLAG_SIMT = 2
OMNI_FLAG_FUSED_MERGE = 4
OMNI_FLAG_NO_CLUSTER_MERGE = 8

EXPORTS = (
    "omni_version", "omni_status_string", "omni_sparse_mla_num_splits", "omni_sparse_mla_num_launches",
    "omni_sparse_mla_workspace_bytes", "omni_sparse_mla_decode", "omni_sparse_mla_decode_sink_recent",
    "omni_rolling_pages_per_request", "omni_kv_append_rolling", "omni_sparse_mla_decode_rolling",
    "omni_topk_select",
    "omni_sparse_mla_combine",
    "omni_sparse_mla_validate", "omni_sparse_mla_resolve_rows",
    "omni_sparse_mla_host_staging_bytes", "omni_sparse_mla_decode_host",
    "omni_sparse_mla_set_profile_events", "omni_sparse_mla_decode_static",
    "omni_sparse_mla_plan_init", "omni_sparse_mla_decode_planned", "omni_sparse_mla_plan_query",
    "omni_selftest_bounded_wait", "omni_kv_quantize_q8", "omni_sparse_mla_decode_q8",
)


class OmniDesc(ctypes.Structure):
    """Mirror of ``omni_mla_desc_t``."""
    _fields_ = [
        ("num_pages", ctypes.c_int64),
        ("batch", ctypes.c_int32),
        ("num_heads", ctypes.c_int32),
        ("d_qk", ctypes.c_int32),
        ("d_v", ctypes.c_int32),
        ("page_size", ctypes.c_int32),
        ("max_pages_per_req", ctypes.c_int32),
        ("max_sel", ctypes.c_int32),
        ("num_splits", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float),
        ("flags", ctypes.c_int32),
    ]


class OmniError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (status %d)" % (where, status_string(code), code))


_lib = None


def load() -> ctypes.CDLL:
    """Load libomni_mla.so (built in-tree by ``paper_2511_22481_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("libomni_mla.so is not built; run `python -m paper_2511_22481_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    dp = ctypes.POINTER(OmniDesc)
    lib.omni_version.restype = ctypes.c_int
    lib.omni_version.argtypes = []
    lib.omni_status_string.restype = ctypes.c_char_p
    lib.omni_status_string.argtypes = [ctypes.c_int]
    lib.omni_sparse_mla_num_splits.restype = i32
    lib.omni_sparse_mla_num_splits.argtypes = [dp]
    lib.omni_sparse_mla_num_launches.restype = i32
    lib.omni_sparse_mla_num_launches.argtypes = [dp]
    lib.omni_sparse_mla_workspace_bytes.restype = sz
    lib.omni_sparse_mla_workspace_bytes.argtypes = [dp]
    lib.omni_sparse_mla_decode.restype = ctypes.c_int
    lib.omni_sparse_mla_decode.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.omni_sparse_mla_decode_sink_recent.restype = ctypes.c_int
    lib.omni_sparse_mla_decode_sink_recent.argtypes = [dp, vp, vp, vp, vp, i32, i32, vp, vp, vp, sz, vp, vp]
    lib.omni_sparse_mla_decode_rolling.restype = ctypes.c_int
    lib.omni_sparse_mla_decode_rolling.argtypes = [dp, vp, vp, vp, vp, i32, i32, vp, vp, vp, sz, vp, vp]
    lib.omni_kv_append_rolling.restype = ctypes.c_int
    lib.omni_kv_append_rolling.argtypes = [dp, vp, vp, vp, vp, i32, i32, vp, vp]
    lib.omni_topk_select.restype = ctypes.c_int
    lib.omni_topk_select.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp]
    lib.omni_rolling_pages_per_request.restype = i32
    lib.omni_rolling_pages_per_request.argtypes = [i32, i32]
    lib.omni_sparse_mla_combine.restype = ctypes.c_int
    lib.omni_sparse_mla_combine.argtypes = [dp, i32, vp, vp, vp, vp, vp, vp]
    lib.omni_sparse_mla_validate.restype = ctypes.c_int
    lib.omni_sparse_mla_validate.argtypes = [dp, vp, vp, vp, vp, vp]
    lib.omni_sparse_mla_resolve_rows.restype = ctypes.c_int
    lib.omni_sparse_mla_resolve_rows.argtypes = [dp, vp, vp, vp, vp, vp]
    lib.omni_sparse_mla_host_staging_bytes.restype = sz
    lib.omni_sparse_mla_host_staging_bytes.argtypes = [dp]
    lib.omni_sparse_mla_decode_host.restype = ctypes.c_int
    lib.omni_sparse_mla_decode_host.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, sz, vp, vp]
    lib.omni_sparse_mla_decode_static.restype = ctypes.c_int
    lib.omni_sparse_mla_decode_static.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.omni_kv_quantize_q8.restype = ctypes.c_int
    lib.omni_kv_quantize_q8.argtypes = [vp, ctypes.c_int64, vp, vp, vp]
    lib.omni_sparse_mla_decode_q8.restype = ctypes.c_int
    lib.omni_sparse_mla_decode_q8.argtypes = [dp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.omni_selftest_bounded_wait.restype = ctypes.c_int
    lib.omni_selftest_bounded_wait.argtypes = [ctypes.c_int64, vp, vp, vp]
    lib.omni_sparse_mla_plan_query.restype = i32
    lib.omni_sparse_mla_plan_query.argtypes = [dp, i32, i32, ctypes.POINTER(ctypes.c_int32)]
    lib.omni_sparse_mla_plan_init.restype = ctypes.c_int
    lib.omni_sparse_mla_plan_init.argtypes = [dp, vp, vp, vp]
    lib.omni_sparse_mla_decode_planned.restype = ctypes.c_int
    lib.omni_sparse_mla_decode_planned.argtypes = [vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
    lib.omni_sparse_mla_set_profile_events.restype = None
    lib.omni_sparse_mla_set_profile_events.argtypes = [vp, vp]
    _lib = lib
    return lib


def omni_version() -> int:
    return int(load().omni_version())


def status_string(code: int) -> str:
    return load().omni_status_string(int(code)).decode()


def make_desc(batch, num_heads, num_pages, max_pages_per_req, max_sel, softmax_scale,
              num_splits=0, flags=0, d_qk=576, d_v=512, page_size=64) -> OmniDesc:
    return OmniDesc(num_pages=num_pages, batch=batch, num_heads=num_heads, d_qk=d_qk, d_v=d_v,
                    page_size=page_size, max_pages_per_req=max_pages_per_req, max_sel=max_sel,
                    num_splits=num_splits, softmax_scale=softmax_scale, flags=flags)


def _ptr(t, dtype, device_type, name):
    if t is None:
        return None
    if t.dtype != dtype:
        raise TypeError("%s must be %s, got %s" % (name, dtype, t.dtype))
    if t.device.type != device_type:
        raise ValueError("%s must live on %s" % (name, device_type))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _check(code, where):
    if code != OMNI_OK:
        raise OmniError(code, where)


def omni_sparse_mla_num_splits(desc: OmniDesc) -> int:
    return int(load().omni_sparse_mla_num_splits(ctypes.byref(desc)))


def omni_sparse_mla_num_launches(desc: OmniDesc) -> int:
    return int(load().omni_sparse_mla_num_launches(ctypes.byref(desc)))


def omni_sparse_mla_plan_query(desc: OmniDesc, sm_count: int, resident_merge_clusters: int):
    """(splits per request, launches per call) on a device description; needs no GPU."""
    launches = ctypes.c_int32(0)
    splits = int(load().omni_sparse_mla_plan_query(ctypes.byref(desc), int(sm_count), int(resident_merge_clusters),
                                                   ctypes.byref(launches)))
    return splits, int(launches.value)


def omni_sparse_mla_workspace_bytes(desc: OmniDesc) -> int:
    return int(load().omni_sparse_mla_workspace_bytes(ctypes.byref(desc)))


def omni_sparse_mla_host_staging_bytes(desc: OmniDesc) -> int:
    return int(load().omni_sparse_mla_host_staging_bytes(ctypes.byref(desc)))


def omni_sparse_mla_set_profile_events(before=None, after=None) -> None:
    """before / after: torch.cuda.Event objects (already recorded once, so they exist) or None."""
    h = lambda e: None if e is None else ctypes.c_void_p(e.cuda_event)
    load().omni_sparse_mla_set_profile_events(h(before), h(after))


def omni_sparse_mla_decode(desc, q, kv_cache, page_table, sel_idx, sel_len, out, lse,
                           workspace=None, device_status=None, stream=None) -> None:
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    code = load().omni_sparse_mla_decode(
        ctypes.byref(desc), _ptr(q, torch.bfloat16, "cuda", "q"),
        _ptr(kv_cache, torch.bfloat16, "cuda", "kv_cache"),
        _ptr(page_table, torch.int32, "cuda", "page_table"),
        _ptr(sel_idx, torch.int32, "cuda", "sel_idx"), _ptr(sel_len, torch.int32, "cuda", "sel_len"),
        _ptr(out, torch.bfloat16, "cuda", "out"), _ptr(lse, torch.float32, "cuda", "lse"),
        None if workspace is None else ctypes.c_void_p(workspace.data_ptr()), ws_bytes,
        _ptr(device_status, torch.int32, "cuda", "device_status"), _stream(stream))
    _check(code, "omni_sparse_mla_decode")


def omni_sparse_mla_decode_sink_recent(desc, q, kv_cache, page_table, ctx_len, n_sink, n_recent, out, lse,
                                       workspace=None, device_status=None, stream=None) -> None:
    """Decode with Eq. 2's selection (attention sink + recent tokens) given as N_sink, N_recent and
    the context length of every request instead of an index list."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    code = load().omni_sparse_mla_decode_sink_recent(
        ctypes.byref(desc), _ptr(q, torch.bfloat16, "cuda", "q"),
        _ptr(kv_cache, torch.bfloat16, "cuda", "kv_cache"),
        _ptr(page_table, torch.int32, "cuda", "page_table"),
        _ptr(ctx_len, torch.int32, "cuda", "ctx_len"), int(n_sink), int(n_recent),
        _ptr(out, torch.bfloat16, "cuda", "out"), _ptr(lse, torch.float32, "cuda", "lse"),
        None if workspace is None else ctypes.c_void_p(workspace.data_ptr()), ws_bytes,
        _ptr(device_status, torch.int32, "cuda", "device_status"), _stream(stream))
    _check(code, "omni_sparse_mla_decode_sink_recent")


def omni_topk_select(scores, ctx_len, k, sel_idx, sel_len, stream=None) -> None:
    """Positions of the k largest scores of every request, as sel_idx / sel_len for the decode call."""
    batch, stride = scores.shape
    code = load().omni_topk_select(
        _ptr(scores, torch.float32, "cuda", "scores"), _ptr(ctx_len, torch.int32, "cuda", "ctx_len"),
        int(batch), int(stride), int(k), _ptr(sel_idx, torch.int32, "cuda", "sel_idx"),
        _ptr(sel_len, torch.int32, "cuda", "sel_len"), _stream(stream))
    _check(code, "omni_topk_select")


def omni_rolling_pages_per_request(n_sink: int, n_recent: int) -> int:
    return int(load().omni_rolling_pages_per_request(int(n_sink), int(n_recent)))


def omni_kv_append_rolling(desc, kv_cache, page_table, ctx_len, new_rows, n_sink, n_recent,
                           device_status=None, stream=None) -> None:
    """Append one latent row per request to the rolling cache of a compressed layer."""
    code = load().omni_kv_append_rolling(
        ctypes.byref(desc), _ptr(kv_cache, torch.bfloat16, "cuda", "kv_cache"),
        _ptr(page_table, torch.int32, "cuda", "page_table"), _ptr(ctx_len, torch.int32, "cuda", "ctx_len"),
        _ptr(new_rows, torch.bfloat16, "cuda", "new_rows"), int(n_sink), int(n_recent),
        _ptr(device_status, torch.int32, "cuda", "device_status"), _stream(stream))
    _check(code, "omni_kv_append_rolling")


def omni_sparse_mla_decode_rolling(desc, q, kv_cache, page_table, ctx_len, n_sink, n_recent, out, lse,
                                   workspace=None, device_status=None, stream=None) -> None:
    """Decode over the rolling cache of a compressed layer (Eq. 2's index set, any context length)."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    code = load().omni_sparse_mla_decode_rolling(
        ctypes.byref(desc), _ptr(q, torch.bfloat16, "cuda", "q"),
        _ptr(kv_cache, torch.bfloat16, "cuda", "kv_cache"),
        _ptr(page_table, torch.int32, "cuda", "page_table"),
        _ptr(ctx_len, torch.int32, "cuda", "ctx_len"), int(n_sink), int(n_recent),
        _ptr(out, torch.bfloat16, "cuda", "out"), _ptr(lse, torch.float32, "cuda", "lse"),
        None if workspace is None else ctypes.c_void_p(workspace.data_ptr()), ws_bytes,
        _ptr(device_status, torch.int32, "cuda", "device_status"), _stream(stream))
    _check(code, "omni_sparse_mla_decode_rolling")


OMNI_Q8_ROW_BYTES = 640


def omni_kv_quantize_q8(kv_rows, kv_q8, kv_scale, stream=None) -> None:
    """bf16 rows [..., 576] -> 8-bit cache rows [..., 640] (uint8) and one fp32 scale per row."""
    num_rows = kv_rows.numel() // 576
    code = load().omni_kv_quantize_q8(
        _ptr(kv_rows, torch.bfloat16, "cuda", "kv_rows"), int(num_rows), _ptr(kv_q8, torch.uint8, "cuda", "kv_q8"),
        _ptr(kv_scale, torch.float32, "cuda", "kv_scale"), _stream(stream))
    _check(code, "omni_kv_quantize_q8")


def omni_sparse_mla_decode_q8(desc, q, kv_q8, kv_scale, page_table, sel_idx, sel_len, out, lse,
                              workspace=None, device_status=None, stream=None) -> None:
    """Decode over the 8-bit latent cache (see ``omni_kv_quantize_q8``)."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    code = load().omni_sparse_mla_decode_q8(
        ctypes.byref(desc), _ptr(q, torch.bfloat16, "cuda", "q"), _ptr(kv_q8, torch.uint8, "cuda", "kv_q8"),
        _ptr(kv_scale, torch.float32, "cuda", "kv_scale"), _ptr(page_table, torch.int32, "cuda", "page_table"),
        _ptr(sel_idx, torch.int32, "cuda", "sel_idx"), _ptr(sel_len, torch.int32, "cuda", "sel_len"),
        _ptr(out, torch.bfloat16, "cuda", "out"), _ptr(lse, torch.float32, "cuda", "lse"),
        None if workspace is None else ctypes.c_void_p(workspace.data_ptr()), ws_bytes,
        _ptr(device_status, torch.int32, "cuda", "device_status"), _stream(stream))
    _check(code, "omni_sparse_mla_decode_q8")


OMNI_PLAN_BYTES = 1024


class LaunchPlan:
    """Caller-owned storage of an ``omni_mla_plan_t`` (64-byte aligned host memory)."""

    def __init__(self):
        self._raw = ctypes.create_string_buffer(OMNI_PLAN_BYTES + 64)
        base = ctypes.addressof(self._raw)
        self.address = (base + 63) & ~63
        self.ptr = ctypes.c_void_p(self.address)


def omni_sparse_mla_plan_init(desc, q, kv_cache) -> LaunchPlan:
    """Everything of a decode call that depends only on the descriptor, q and the pool, done once."""
    plan = LaunchPlan()
    code = load().omni_sparse_mla_plan_init(
        ctypes.byref(desc), _ptr(q, torch.bfloat16, "cuda", "q"),
        _ptr(kv_cache, torch.bfloat16, "cuda", "kv_cache"), plan.ptr)
    _check(code, "omni_sparse_mla_plan_init")
    return plan


def omni_sparse_mla_decode_planned(plan, page_table, sel_idx, sel_len, out, lse, workspace=None,
                                   device_status=None, stream=None) -> None:
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    code = load().omni_sparse_mla_decode_planned(
        plan.ptr, _ptr(page_table, torch.int32, "cuda", "page_table"),
        _ptr(sel_idx, torch.int32, "cuda", "sel_idx"), _ptr(sel_len, torch.int32, "cuda", "sel_len"),
        _ptr(out, torch.bfloat16, "cuda", "out"), _ptr(lse, torch.float32, "cuda", "lse"),
        None if workspace is None else ctypes.c_void_p(workspace.data_ptr()), ws_bytes,
        _ptr(device_status, torch.int32, "cuda", "device_status"), _stream(stream))
    _check(code, "omni_sparse_mla_decode_planned")


def bind_planned(plan, page_table, sel_idx, sel_len, out, lse, workspace=None, device_status=None, stream=None):
    """The planned decode call with its arguments marshalled once: returns a function of no
    arguments that makes the C call (for loops that repeat one call on fixed buffers; the
    tensors must stay alive and in place, and the stream is the one given here)."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    fn = load().omni_sparse_mla_decode_planned
    args = (plan.ptr, _ptr(page_table, torch.int32, "cuda", "page_table"),
            _ptr(sel_idx, torch.int32, "cuda", "sel_idx"), _ptr(sel_len, torch.int32, "cuda", "sel_len"),
            _ptr(out, torch.bfloat16, "cuda", "out"), _ptr(lse, torch.float32, "cuda", "lse"),
            None if workspace is None else ctypes.c_void_p(workspace.data_ptr()), ctypes.c_size_t(ws_bytes),
            _ptr(device_status, torch.int32, "cuda", "device_status"), _stream(stream))
    keep = (plan, page_table, sel_idx, sel_len, out, lse, workspace, device_status)

    def call(_keep=keep):
        code = fn(*args)
        if code != OMNI_OK:
            raise OmniError(code, "omni_sparse_mla_decode_planned")
    return call


OMNI_STATIC_SCRATCH_BYTES = 32 * 1024 * 1024


def omni_sparse_mla_decode_static(desc, q, kv_cache, page_table, sel_idx, sel_len, out, lse,
                                  device_status=None, stream=None) -> None:
    """Decode for callers that may not allocate: no workspace argument, the split-KV scratch is
    a fixed 32 MiB array inside the library (shared by all calls on a device, so calls that
    overlap on the GPU race).  Raises OmniError(OMNI_ERR_WORKSPACE) if the problem needs more."""
    code = load().omni_sparse_mla_decode_static(
        ctypes.byref(desc), _ptr(q, torch.bfloat16, "cuda", "q"),
        _ptr(kv_cache, torch.bfloat16, "cuda", "kv_cache"),
        _ptr(page_table, torch.int32, "cuda", "page_table"),
        _ptr(sel_idx, torch.int32, "cuda", "sel_idx"), _ptr(sel_len, torch.int32, "cuda", "sel_len"),
        _ptr(out, torch.bfloat16, "cuda", "out"), _ptr(lse, torch.float32, "cuda", "lse"),
        _ptr(device_status, torch.int32, "cuda", "device_status"), _stream(stream))
    _check(code, "omni_sparse_mla_decode_static")


def omni_sparse_mla_combine(desc, max_splits, part_out, part_lse, num_splits, out, lse,
                            stream=None) -> None:
    code = load().omni_sparse_mla_combine(
        ctypes.byref(desc), int(max_splits), _ptr(part_out, torch.float32, "cuda", "part_out"),
        _ptr(part_lse, torch.float32, "cuda", "part_lse"),
        _ptr(num_splits, torch.int32, "cuda", "num_splits"),
        _ptr(out, torch.bfloat16, "cuda", "out"), _ptr(lse, torch.float32, "cuda", "lse"),
        _stream(stream))
    _check(code, "omni_sparse_mla_combine")


def omni_selftest_bounded_wait(limit_cycles, device_status, waited_cycles=None, stream=None) -> None:
    """One warp waits `limit_cycles` SM clocks on a barrier nobody arrives on, then reports the time-out."""
    code = load().omni_selftest_bounded_wait(
        int(limit_cycles), _ptr(device_status, torch.int32, "cuda", "device_status"),
        _ptr(waited_cycles, torch.int64, "cuda", "waited_cycles"), _stream(stream))
    _check(code, "omni_selftest_bounded_wait")


def omni_sparse_mla_validate(desc, page_table, sel_idx, sel_len, device_status, stream=None) -> None:
    code = load().omni_sparse_mla_validate(
        ctypes.byref(desc), _ptr(page_table, torch.int32, "cuda", "page_table"),
        _ptr(sel_idx, torch.int32, "cuda", "sel_idx"), _ptr(sel_len, torch.int32, "cuda", "sel_len"),
        _ptr(device_status, torch.int32, "cuda", "device_status"), _stream(stream))
    _check(code, "omni_sparse_mla_validate")


def omni_sparse_mla_resolve_rows(desc, page_table, sel_idx, sel_len, rows, stream=None) -> None:
    code = load().omni_sparse_mla_resolve_rows(
        ctypes.byref(desc), _ptr(page_table, torch.int32, "cuda", "page_table"),
        _ptr(sel_idx, torch.int32, "cuda", "sel_idx"), _ptr(sel_len, torch.int32, "cuda", "sel_len"),
        _ptr(rows, torch.int64, "cuda", "rows"), _stream(stream))
    _check(code, "omni_sparse_mla_resolve_rows")


def omni_sparse_mla_decode_host(desc, q_host, kv_cache, page_table_host, sel_idx_host,
                                sel_len_host, out_host, lse_host, staging, workspace=None,
                                device_status=None, stream=None) -> None:
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    code = load().omni_sparse_mla_decode_host(
        ctypes.byref(desc), _ptr(q_host, torch.bfloat16, "cpu", "q_host"),
        _ptr(kv_cache, torch.bfloat16, "cuda", "kv_cache"),
        _ptr(page_table_host, torch.int32, "cpu", "page_table_host"),
        _ptr(sel_idx_host, torch.int32, "cpu", "sel_idx_host"),
        _ptr(sel_len_host, torch.int32, "cpu", "sel_len_host"),
        _ptr(out_host, torch.bfloat16, "cpu", "out_host"), _ptr(lse_host, torch.float32, "cpu", "lse_host"),
        ctypes.c_void_p(staging.data_ptr()), staging.numel() * staging.element_size(),
        None if workspace is None else ctypes.c_void_p(workspace.data_ptr()), ws_bytes,
        _ptr(device_status, torch.int32, "cuda", "device_status"), _stream(stream))
    _check(code, "omni_sparse_mla_decode_host")


# ---------------------------------------------------------------------------------------
# Convenience wrapper: owns the output, workspace and status buffers of one problem shape.
# ---------------------------------------------------------------------------------------

@dataclass
class DecodePlan:
    desc: OmniDesc
    out: torch.Tensor
    lse: torch.Tensor
    workspace: torch.Tensor
    status: torch.Tensor
    splits: int

    def run(self, q, kv_cache, page_table, sel_idx, sel_len, stream=None):
        omni_sparse_mla_decode(self.desc, q, kv_cache, page_table, sel_idx, sel_len, self.out,
                               self.lse, self.workspace, self.status, stream)
        return self.out, self.lse


def plan_for(w, num_splits=0, flags=0, device=None) -> DecodePlan:
    """Allocate outputs / workspace for a ``workloads.Workload``-shaped problem."""
    device = device or w.q.device
    desc = make_desc(w.batch, w.heads, w.num_pages, w.max_pages_per_req, w.max_sel, w.scale,
                     num_splits=num_splits, flags=flags)
    ws = omni_sparse_mla_workspace_bytes(desc)
    if ws == 0:
        raise OmniError(2, "omni_sparse_mla_workspace_bytes")
    return DecodePlan(
        desc=desc,
        out=torch.empty((w.batch, w.heads, w.d_v), dtype=torch.bfloat16, device=device),
        lse=torch.empty((w.batch, w.heads), dtype=torch.float32, device=device),
        workspace=torch.empty((ws,), dtype=torch.uint8, device=device),
        status=torch.zeros((1,), dtype=torch.int32, device=device),
        splits=omni_sparse_mla_num_splits(desc))
