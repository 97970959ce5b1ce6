"""Pins of the 8-bit cache oracle (format, quantiser, attention over de-quantised rows) against
things that are not the oracle: the published E4M3 format tables, hand-worked rows, a library
cast, and the pinned bf16 oracle in the cases where quantisation is exact."""
import numpy as np
import pytest
import torch

import oracle
from oracle import q8


def test_e4m3_code_points_from_the_format_definition():
    # 1-4-3, bias 7: a handful of code points written down from the format's definition
    table = {0x00: 0.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x38: 1.0, 0x39: 1.125,
             0x40: 2.0, 0x7E: 448.0, 0x77: 240.0, 0xB8: -1.0, 0xFE: -448.0, 0x80: -0.0}
    for code, value in table.items():
        got = q8.e4m3_decode(np.array([code], dtype=np.uint8))[0]
        assert got == value and np.signbit(got) == np.signbit(value), hex(code)
    assert np.isnan(q8.e4m3_decode(np.array([0x7F, 0xFF], dtype=np.uint8))).all()
    # all 254 finite codes are distinct, symmetric, and strictly increasing with the code
    pos = q8.e4m3_decode(np.arange(0, 0x7F, dtype=np.uint8))
    assert np.all(np.diff(pos) > 0) and pos[-1] == 448.0
    neg = q8.e4m3_decode(np.arange(0x80, 0xFF, dtype=np.uint8))
    assert np.array_equal(neg, -pos)


def test_e4m3_encode_round_trips_every_code_and_rounds_to_nearest_even():
    codes = np.array([c for c in range(256) if c & 0x7F != 0x7F], dtype=np.uint8)
    vals = q8.e4m3_decode(codes).astype(np.float32)
    assert np.array_equal(q8.e4m3_encode(vals), codes)
    # hand-worked roundings: spacing is 0.125 in [1, 2), 32 in [256, 448]
    cases = [(1.0624, 0x38), (1.0625, 0x38), (1.0626, 0x39), (1.1875, 0x3A), (1.3125, 0x3A),
             (432.0, 0x7E), (431.9, 0x7D), (464.0, 0x7E), (1e9, 0x7E), (-1e9, 0xFE),
             (2.0 ** -10, 0x00), (2.0 ** -10 * 1.01, 0x01), (3 * 2.0 ** -10, 0x02), (-0.0, 0x80)]
    for x, code in cases:
        assert q8.e4m3_encode(np.array([x], dtype=np.float32))[0] == code, (x, hex(code))
    assert q8.e4m3_encode(np.array([np.nan], dtype=np.float32))[0] & 0x7F == 0x7F


def test_e4m3_encode_matches_the_library_cast_on_random_values():
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("no float8 dtype in this torch")
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(20000) * 100, rng.standard_normal(20000), rng.standard_normal(20000) * 0.01,
                        np.linspace(-448, 448, 30001)]).astype(np.float32)
    x = x[np.abs(x) <= 448.0]                      # the library cast does not saturate; the format's range is checked by hand above
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(q8.e4m3_encode(x), lib)


def _bits(x):
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def test_quantiser_on_hand_worked_rows():
    row = np.zeros((3, 576), dtype=np.float32)
    row[0, :4] = [448.0, -224.0, 1.0, 0.4375]      # amax 448 -> scale 1: codes of the values themselves
    row[0, 512:] = np.arange(64) * 0.25            # rope columns are copied as bf16
    row[1, 7] = -3.5                               # amax 3.5 -> scale 3.5/448 = 2^-7: -3.5/scale = -448
    row[1, 8] = 1.75                               # 224
    row[1, 9] = 2.0 ** -7                          # 1.0 after scaling
    # row 2 stays all zero: amax is floored at 2^-60, every code 0
    cache, scale = q8.quantise_rows(_bits(row))
    assert cache.shape == (3, 640) and scale.dtype == np.float32
    assert scale.tolist() == [1.0, 3.5 / 448.0, float(np.float32(2.0 ** -60) / np.float32(448.0))]
    assert cache[0, :4].tolist() == [0x7E, 0xF6, 0x38, 0x2E]
    assert cache[1, 7] == 0xFE and cache[1, 8] == 0x76 and cache[1, 9] == 0x38
    assert not cache[2, :512].any() and not cache[1, :7].any()
    assert np.array_equal(cache[0, 512:].view(np.uint16), _bits(row[0, 512:]))
    back = q8.dequantise_rows(cache, scale)
    assert np.array_equal(back[0, :4], [448.0, -224.0, 1.0, 0.4375])
    assert np.array_equal(back[1, 7:10], [-3.5, 1.75, 2.0 ** -7])
    assert np.array_equal(back[0, 512:], (np.arange(64) * 0.25))


def test_quantisation_error_is_within_half_a_step_of_the_row_scale():
    rng = np.random.default_rng(2)
    rows = (rng.standard_normal((64, 576)) * 0.5).astype(np.float32)
    bits = _bits(rows)
    exact = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    cache, scale = q8.quantise_rows(bits)
    back = q8.dequantise_rows(cache, scale)
    assert np.array_equal(back[:, 512:], exact[:, 512:])
    # E4M3 keeps 4 significant bits: the error of a value is at most 1/16 of its magnitude (half a
    # step of 1/8 relative), or half a subnormal step (2^-10 in code units) near zero
    err = np.abs(back[:, :512] - exact[:, :512])
    bound = np.maximum(np.abs(exact[:, :512]) / 16.0, 2.0 ** -10 * scale[:, None].astype(np.float64)) * (1 + 1e-6)
    assert np.all(err <= bound)
    assert np.abs(back[:, :512]).max(axis=1) == pytest.approx(np.abs(exact[:, :512]).max(axis=1), rel=1e-6)


def test_attention_over_exactly_representable_rows_equals_the_bf16_oracle():
    """Rows whose latent columns are E4M3 code points times a power-of-two scale quantise without
    error, so the 8-bit definition must reproduce the pinned bf16 oracle on them."""
    rng = np.random.default_rng(3)
    B, H, n_rows = 2, 5, 37
    codes = rng.integers(0, 0x7F, (B, n_rows, 512)).astype(np.uint8) | (rng.integers(0, 2, (B, n_rows, 512)) << 7).astype(np.uint8)
    vals = q8.e4m3_decode(codes)
    vals[:, :, 0] = 448.0                                         # pins every row's amax, hence scale = 2^k exactly
    pow2 = np.exp2(rng.integers(-12, -6, (B, n_rows, 1)).astype(np.float64))
    rows = np.concatenate([vals * pow2, rng.standard_normal((B, n_rows, 64)) * 0.5], axis=2)
    row_bits = _bits(rows)                                        # exact: 4 significant bits fit bf16
    q = torch.from_numpy((rng.standard_normal((B, H, 576)) * 0.5).astype(np.float32)).to(torch.bfloat16)
    n = np.array([n_rows, 20], dtype=np.int32)
    ref_out, ref_lse = oracle.attend_rows(q, torch.from_numpy(row_bits.view(np.int16)).view(torch.bfloat16), n, 512, 0.07)
    cache, scale = q8.quantise_rows(row_bits.reshape(-1, 576))
    deq = q8.dequantise_rows(cache, scale).reshape(B, n_rows, 576)
    exact = (row_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    assert np.array_equal(deq, exact)
    out, lse = q8.attend_dequantised(q.to(torch.float64).numpy(), deq, n, 512, 0.07)
    assert np.abs(out - ref_out).max() < 1e-12 and np.abs(lse - ref_lse).max() < 1e-12


def test_attention_special_cases():
    rng = np.random.default_rng(4)
    k = rng.standard_normal((1, 9, 576))
    q = np.zeros((1, 3, 576))
    out, lse = q8.attend_dequantised(q, k, [9], 512, 0.1)
    assert np.allclose(out[0, 0], k[0, :, :512].mean(axis=0), atol=1e-15) and np.allclose(lse, np.log(9.0))
    out, lse = q8.attend_dequantised(rng.standard_normal((1, 3, 576)), k, [1], 512, 0.1)
    assert np.array_equal(out[0, 2], k[0, 0, :512])
    out, lse = q8.attend_dequantised(q, k, [0], 512, 0.1)
    assert not out.any() and np.isneginf(lse).all()
