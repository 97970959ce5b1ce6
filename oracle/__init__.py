"""CPU oracle for decode-phase sparse MLA attention.  TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the benchmark's cpu-baseline leg may import this
package.  The product library neither imports nor links it, and it imports nothing from
the product package.  The arithmetic lives in ``sparse_mla_oracle.c`` (plain two-pass fp64);
this module compiles that file with gcc and marshals numpy / torch-CPU arrays into it.

Follows the paper's "OmniAttn: Problem Formulation" (Eq. 1, restricted-attention side) and
Eq. 2 (sink + recent index set, see ``selection.py``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sparse_mla_oracle.c")
_LIB = os.path.join(_HERE, "libsparse_mla_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP for threads over (request, head))."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


_LIB32 = os.path.join(_HERE, "libsparse_mla_oracle_f32.so")
_lib32 = None


def build_f32(force: bool = False) -> str:
    """The same source compiled with float as its working type.  Timed by the benchmark as the
    plain fp32 CPU figure; never a reference for anything."""
    with _lock:
        stale = (not os.path.exists(_LIB32)) or os.path.getmtime(_LIB32) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB32 + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-DORACLE_REAL=float", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB32)
    return _LIB32


def attend_rows_f32_timed(q, krows, n, d_v: int, scale: float):
    """Runs the float build of oracle_attend_rows on the same arguments as ``attend_rows``
    and returns (seconds, out, lse); for timing only."""
    import time
    global _lib32
    if _lib32 is None:
        build_f32()
        lib = ctypes.CDLL(_LIB32)
        i32, f64, vp = ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        lib.oracle_attend_rows.argtypes = [i32, i32, i32, i32, i32, f64, vp, vp, vp, vp, vp, vp]
        lib.oracle_attend_rows.restype = None
        _lib32 = lib
    qb, kb, nn = bf16_bits(q), bf16_bits(krows), _i32(n)
    B, H, d_qk = qb.shape
    max_sel = kb.shape[1]
    out = np.empty((B, H, d_v), dtype=np.float64)
    lse = np.empty((B, H), dtype=np.float64)
    t0 = time.perf_counter()
    _lib32.oracle_attend_rows(B, H, d_qk, d_v, max_sel, float(scale), _p(qb), _p(kb), _p(nn), _p(out), _p(lse), None)
    return time.perf_counter() - t0, out, lse


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i32, i64, f64, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.oracle_resolve_rows.argtypes = [i32, i32, i64, i32, i32, vp, vp, vp, vp]
        lib.oracle_resolve_rows.restype = i32
        lib.oracle_attend_rows.argtypes = [i32, i32, i32, i32, i32, f64, vp, vp, vp, vp, vp, vp]
        lib.oracle_attend_rows.restype = None
        lib.oracle_sparse_mla_decode.argtypes = [i32, i32, i32, i32, i32, i64, i32, i32, f64,
                                                 vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_sparse_mla_decode.restype = i32
        lib.oracle_splitkv_combine.argtypes = [i32, i32, i32, i32, vp, vp, vp, vp, vp]
        lib.oracle_splitkv_combine.restype = None
        lib.oracle_num_threads.argtypes = []
        lib.oracle_num_threads.restype = i32
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the oracle's parallel loop will use (OMP_NUM_THREADS / affinity mask)."""
    return int(_load().oracle_num_threads())


def bf16_bits(x) -> np.ndarray:
    """Return the raw 16-bit patterns of a bf16 array as a C-contiguous uint16 ndarray.

    Accepts a torch CPU tensor of dtype bfloat16 or an ndarray that already holds bits.
    """
    if isinstance(x, np.ndarray):
        assert x.dtype == np.uint16
        return np.ascontiguousarray(x)
    import torch  # plumbing only: reinterpret the storage, no arithmetic

    assert x.dtype == torch.bfloat16 and x.device.type == "cpu"
    return np.ascontiguousarray(x.contiguous().view(torch.int16).numpy().view(np.uint16))


def _i32(a) -> np.ndarray:
    if not isinstance(a, np.ndarray):
        a = a.numpy()
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def resolve_rows(page_table, sel_idx, sel_len, page_size: int, num_pages: int):
    """Physical pool rows of every selected token: int64 [B, max_sel], -1 past sel_len.

    Raises ValueError on any contract violation (index or page id out of range).
    """
    pt, si, sl = _i32(page_table), _i32(sel_idx), _i32(sel_len)
    B, max_sel = si.shape
    rows = np.empty((B, max_sel), dtype=np.int64)
    bad = _load().oracle_resolve_rows(B, page_size, num_pages, pt.shape[1], max_sel,
                                      _p(pt), _p(si), _p(sl), _p(rows))
    if bad:
        raise ValueError("oracle: %d selection entries violate the index contract" % bad)
    return rows


def attend_rows(q, krows, n, d_v: int, scale: float, want_wsum: bool = False):
    """Attention over gathered rows.  q bf16 [B,H,d_qk]; krows bf16 [B,max_sel,d_qk]; n [B]."""
    qb, kb, nn = bf16_bits(q), bf16_bits(krows), _i32(n)
    B, H, d_qk = qb.shape
    max_sel = kb.shape[1]
    assert kb.shape == (B, max_sel, d_qk) and nn.shape == (B,)
    assert int(nn.max(initial=0)) <= max_sel
    out = np.empty((B, H, d_v), dtype=np.float64)
    lse = np.empty((B, H), dtype=np.float64)
    wsum = np.empty((B, H), dtype=np.float64) if want_wsum else None
    _load().oracle_attend_rows(B, H, d_qk, d_v, max_sel, float(scale), _p(qb), _p(kb), _p(nn),
                               _p(out), _p(lse), _p(wsum) if want_wsum else None)
    return (out, lse, wsum) if want_wsum else (out, lse)


def sparse_mla_decode(q, kv_cache, page_table, sel_idx, sel_len, d_v: int, scale: float):
    """Whole path on a host-resident pool.  Returns (out f64 [B,H,d_v], lse f64 [B,H], rows)."""
    qb, kvb = bf16_bits(q), bf16_bits(kv_cache)
    pt, si, sl = _i32(page_table), _i32(sel_idx), _i32(sel_len)
    B, H, d_qk = qb.shape
    num_pages, page_size, d2 = kvb.shape
    assert d2 == d_qk
    max_sel = si.shape[1]
    out = np.empty((B, H, d_v), dtype=np.float64)
    lse = np.empty((B, H), dtype=np.float64)
    rows = np.empty((B, max_sel), dtype=np.int64)
    bad = _load().oracle_sparse_mla_decode(B, H, d_qk, d_v, page_size, num_pages, pt.shape[1],
                                           max_sel, float(scale), _p(qb), _p(kvb), _p(pt),
                                           _p(si), _p(sl), _p(out), _p(lse), _p(rows))
    if bad:
        raise ValueError("oracle: %d selection entries violate the index contract" % bad)
    return out, lse, rows


def splitkv_combine(part_out, part_lse, num_splits):
    """LSE-weighted merge.  part_out f64 [B,S,H,d_v], part_lse f64 [B,S,H], num_splits [B]."""
    po = np.ascontiguousarray(part_out, dtype=np.float64)
    pl = np.ascontiguousarray(part_lse, dtype=np.float64)
    ns = _i32(num_splits)
    B, S, H, d_v = po.shape
    assert pl.shape == (B, S, H)
    out = np.empty((B, H, d_v), dtype=np.float64)
    lse = np.empty((B, H), dtype=np.float64)
    _load().oracle_splitkv_combine(B, H, d_v, S, _p(po), _p(pl), _p(ns), _p(out), _p(lse))
    return out, lse
