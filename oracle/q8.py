"""8-bit latent KV cache: row format, codec and attention over the de-quantised rows.
TEST INFRASTRUCTURE ONLY (same rules as the rest of this package).

The paper serves a quantised (INT8) DeepSeek-R1 (Evaluation, "Experimental Setup") and gives no
cache format, so the format is this build's reading; it is written out here and the GPU path is
checked against it:

  * a token's 576-column latent row is stored as 640 bytes: the 512 latent ("nope") columns as
    FP8 E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities; the
    largest finite magnitude is 448; exponent field 0 holds subnormals m/8 * 2^-6), followed by
    the 64 rope columns unchanged as bf16 (128 bytes);
  * one fp32 scale per row, kept in a separate array: scale = max(amax, 2^-60) / 448 with amax
    the largest |value| of the row's 512 latent columns (the floor keeps the scale and its
    reciprocal finite for all-zero rows); code = E4M3(value / scale), both divisions done in fp32,
    the result rounded to nearest, ties to even, saturating at 448;
  * the value a code stands for is exactly decode(code) * scale (an fp32 product, taken exactly
    here in fp64), and the result of the 8-bit decode call is DEFINED as Eq. 1's restricted
    attention over those exactly de-quantised rows (rope columns as stored), with K = all 576
    columns and V = the first 512, as in the bf16 path.
"""
from __future__ import annotations

import numpy as np

E4M3_MAX = 448.0
ROW_BYTES = 640
NOPE = 512
ROPE = 64


def e4m3_decode(codes) -> np.ndarray:
    """Value of every E4M3 code (uint8 array) as float64; the two NaN codes give NaN."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = c & 0x7
    sub = (m / 8.0) * 2.0 ** -6
    nor = (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64))
    v = np.where(e == 0, sub, nor)
    v = np.where((e == 15) & (m == 7), np.nan, v)
    return sign * v


def e4m3_encode(x) -> np.ndarray:
    """Nearest E4M3 code of every float32 value: ties to even, magnitudes beyond 448 saturate to
    448 (no infinities in the format), NaN gives the NaN code 0x7f, zeros keep their sign."""
    x = np.asarray(x, dtype=np.float32).astype(np.float64)
    sign = np.signbit(x)
    a = np.abs(x)
    out = np.zeros(x.shape, dtype=np.uint8)
    nan = np.isnan(a)
    a = np.where(nan, 0.0, a)
    a = np.minimum(a, E4M3_MAX)
    # spacing of the format at magnitude a: 2^(e-3) with e = floor(log2 a) clamped to [-6, 8]
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.clip(e, -6, 8)
    step = np.exp2(e - 3)
    k = a / step                                   # a in units of the local spacing (exact: powers of two)
    r = np.floor(k)
    frac = k - r
    r = r + ((frac > 0.5) | ((frac == 0.5) & (np.mod(r, 2) == 1)))
    v = r * step                                   # rounded magnitude; may have moved up one binade
    v = np.minimum(v, E4M3_MAX)
    # encode the magnitude v: subnormal below 2^-6, else exponent/mantissa fields
    with np.errstate(divide="ignore"):
        ev = np.floor(np.log2(np.where(v > 0, v, 1.0)))
    ev = np.clip(ev, -6, 8)
    is_sub = v < 2.0 ** -6
    mant = np.where(is_sub, v / 2.0 ** -9, (v / np.exp2(ev) - 1.0) * 8.0)
    field = np.where(is_sub, 0, ev + 7)
    out = (field.astype(np.int64) << 3 | np.rint(mant).astype(np.int64)).astype(np.uint8)
    out = np.where(nan, np.uint8(0x7F), out)
    return (out | np.where(sign & ~nan, np.uint8(0x80), np.uint8(0))).astype(np.uint8)


def _bf16_bits_to_f32(bits) -> np.ndarray:
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def quantise_rows(row_bits):
    """bf16 bit patterns [rows, 576] -> (cache bytes uint8 [rows, 640], scale float32 [rows])."""
    bits = np.ascontiguousarray(row_bits, dtype=np.uint16)
    assert bits.ndim == 2 and bits.shape[1] == NOPE + ROPE
    x = _bf16_bits_to_f32(bits[:, :NOPE])
    amax = np.abs(x).max(axis=1).astype(np.float32)
    scale = (np.maximum(amax, np.float32(2.0 ** -60)) / np.float32(E4M3_MAX)).astype(np.float32)
    codes = e4m3_encode((x / scale[:, None]).astype(np.float32))
    out = np.empty((bits.shape[0], ROW_BYTES), dtype=np.uint8)
    out[:, :NOPE] = codes
    out[:, NOPE:] = np.ascontiguousarray(bits[:, NOPE:]).view(np.uint8).reshape(bits.shape[0], 2 * ROPE)
    return out, scale


def dequantise_rows(cache_bytes, scale) -> np.ndarray:
    """(uint8 [rows, 640], float32 [rows]) -> the rows' 576 values, float64, exactly."""
    c = np.ascontiguousarray(cache_bytes, dtype=np.uint8)
    s = np.asarray(scale, dtype=np.float32).astype(np.float64)
    nope = e4m3_decode(c[:, :NOPE]) * s[:, None]
    rope = _bf16_bits_to_f32(np.ascontiguousarray(c[:, NOPE:]).view(np.uint16)).astype(np.float64)
    return np.concatenate([nope, rope], axis=1)


def attend_dequantised(q, krows, n, d_v: int, scale: float):
    """Eq. 1's restricted attention, two passes in fp64, over already gathered rows.
    q float64 [B, H, d_qk]; krows float64 [B, max_sel, d_qk]; n [B] valid rows per request.
    Returns (out [B, H, d_v], lse [B, H]); n = 0 gives out = 0, lse = -inf."""
    q = np.asarray(q, dtype=np.float64)
    B, H, _ = q.shape
    out = np.zeros((B, H, d_v))
    lse = np.full((B, H), -np.inf)
    for b in range(B):
        nb = int(n[b])
        if nb <= 0:
            continue
        k = np.asarray(krows[b][:nb], dtype=np.float64)
        x = scale * (q[b] @ k.T)                       # [H, nb]
        m = x.max(axis=1, keepdims=True)
        e = np.exp(x - m)
        z = e.sum(axis=1, keepdims=True)
        lse[b] = (m + np.log(z))[:, 0]
        out[b] = (e / z) @ k[:, :d_v]
    return out, lse
