"""Pins for the CPU oracle: every check here compares the oracle with something that is not
the oracle -- a library routine, a brute-force loop, a closed form, an invariant or a
hand-worked table -- chosen so that a dropped term, a wrong sign or index, or a transposed
operand in the oracle fails at least one of them.  No GPU needed.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle.selection import sink_recent

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
D_QK, D_V, PAGE = 576, 512, 64


def bf16(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)


def rand_bf16(rng, shape, std=0.5):
    return bf16(rng.standard_normal(shape) * std)


def f64(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float64).numpy()


def identity_problem(rng, B, H, n_pages, page=PAGE, d_qk=D_QK):
    q = rand_bf16(rng, (B, H, d_qk))
    kv = rand_bf16(rng, (B * n_pages, page, d_qk))
    pt = np.arange(B * n_pages, dtype=np.int32).reshape(B, n_pages)
    return q, kv, pt


# ----------------------------------------------------------------------------- library pin

def test_full_selection_equals_library_dense_attention():
    rng = np.random.default_rng(100)
    B, H, n_pages = 2, 5, 3
    q, kv, pt = identity_problem(rng, B, H, n_pages)
    M = n_pages * PAGE
    sel = np.tile(np.arange(M, dtype=np.int32), (B, 1))
    scale = 1.0 / math.sqrt(192.0)
    out, lse, _ = oracle.sparse_mla_decode(q, kv, pt, sel, np.full(B, M, np.int32), D_V, scale)
    K = kv.to(torch.float64).reshape(B, M, D_QK)
    s = torch.einsum("bhc,bmc->bhm", q.to(torch.float64), K) * scale
    ref = torch.einsum("bhm,bmd->bhd", torch.softmax(s, dim=-1), K[:, :, :D_V])
    ref_lse = torch.logsumexp(s, dim=-1)
    assert np.abs(out - ref.numpy()).max() < 1e-12
    assert np.abs(lse - ref_lse.numpy()).max() < 1e-12


# ----------------------------------------------------------------------------- brute force

def _brute(q, K, d_v, scale, subset):
    """Pure-Python attention of one query over the listed rows."""
    xs = [scale * sum(q[c] * K[j][c] for c in range(len(q))) for j in subset]
    z = sum(math.exp(x) for x in xs)
    out = [sum(math.exp(x) / z * K[j][d] for x, j in zip(xs, subset)) for d in range(d_v)]
    return out, math.log(z)


def test_brute_force_every_subset_of_eight_tokens():
    rng = np.random.default_rng(101)
    H, d_qk, d_v, page, M = 2, 4, 3, 4, 8
    q = rand_bf16(rng, (1, H, d_qk), std=1.0)
    kv = rand_bf16(rng, (2, page, d_qk), std=1.0)
    pt = np.array([[1, 0]], dtype=np.int32)           # logical page 0 lives in physical page 1
    qf, kvf = f64(q)[0], f64(kv)
    logical = [kvf[pt[0, t // page], t % page] for t in range(M)]
    scale = 0.7
    for r in range(1, M + 1):
        for subset in itertools.combinations(range(M), r):
            sel = np.full((1, M), -1, np.int32)
            sel[0, :r] = subset
            out, lse, _ = oracle.sparse_mla_decode(q, kv, pt, sel, np.array([r], np.int32), d_v, scale)
            for h in range(H):
                bo, bl = _brute(list(qf[h]), logical, d_v, scale, subset)
                assert np.abs(out[0, h] - np.array(bo)).max() < 1e-13
                assert abs(lse[0, h] - bl) < 1e-13


# ----------------------------------------------------------------------------- closed forms

def test_zero_query_gives_mean_of_values_and_log_count():
    rng = np.random.default_rng(102)
    q, kv, pt = identity_problem(rng, 1, 3, 2)
    q.zero_()
    sel = rng.permutation(2 * PAGE)[:50].astype(np.int32)[None]
    out, lse, _ = oracle.sparse_mla_decode(q, kv, pt, sel, np.array([50], np.int32), D_V, 0.3)
    mean = f64(kv).reshape(-1, D_QK)[sel[0]][:, :D_V].mean(axis=0)
    assert np.abs(out - mean[None, None]).max() < 1e-14
    assert np.abs(lse - math.log(50)).max() < 1e-14


def test_single_token_returns_its_value_row_and_its_score():
    rng = np.random.default_rng(103)
    q, kv, pt = identity_problem(rng, 1, 4, 2)
    t = 77
    out, lse, _ = oracle.sparse_mla_decode(q, kv, pt, np.array([[t]], np.int32),
                                           np.array([1], np.int32), D_V, 0.25)
    row = f64(kv).reshape(-1, D_QK)[t]
    assert np.array_equal(out[0], np.tile(row[:D_V], (4, 1)))      # V = FIRST d_v columns, exactly
    assert np.abs(lse[0] - 0.25 * f64(q)[0] @ row).max() < 1e-13    # K = all d_qk columns


def test_two_tokens_with_scores_ln2_apart_weigh_two_thirds_one_third():
    # q = e_0, k_0 = e_0 (+ a value marker), k_1 = 0 : scores ln2*1 and 0 -> weights 2/3, 1/3.
    q = torch.zeros(1, 1, D_QK, dtype=torch.bfloat16)
    q[0, 0, D_QK - 1] = 1.0                                         # rope column only: not part of V
    kv = torch.zeros(1, PAGE, D_QK, dtype=torch.bfloat16)
    kv[0, 0, D_QK - 1] = 1.0
    kv[0, 0, 0] = 3.0
    kv[0, 1, 0] = -6.0
    kv[0, 1, 1] = 9.0
    out, lse, _ = oracle.sparse_mla_decode(q, kv, np.zeros((1, 1), np.int32),
                                           np.array([[0, 1]], np.int32), np.array([2], np.int32),
                                           D_V, math.log(2.0))
    assert abs(out[0, 0, 0] - (2 / 3 * 3.0 + 1 / 3 * -6.0)) < 1e-15
    assert abs(out[0, 0, 1] - 3.0) < 1e-15
    assert np.abs(out[0, 0, 2:]).max() == 0.0
    assert abs(lse[0, 0] - math.log(3.0)) < 1e-15


def test_constant_added_to_every_score_shifts_lse_only():
    rng = np.random.default_rng(104)
    q, kv, pt = identity_problem(rng, 1, 2, 1)
    q[..., D_QK - 1] = 1.0
    kv[..., D_QK - 1] = 0.0
    sel = np.arange(PAGE, dtype=np.int32)[None]
    n = np.array([PAGE], np.int32)
    o0, l0, _ = oracle.sparse_mla_decode(q, kv, pt, sel, n, D_V, 0.5)
    kv[..., D_QK - 1] = 4.0
    o1, l1, _ = oracle.sparse_mla_decode(q, kv, pt, sel, n, D_V, 0.5)
    assert np.abs(o1 - o0).max() < 1e-14
    assert np.abs(l1 - l0 - 2.0).max() < 1e-13


def test_empty_selection_is_zero_output_and_minus_infinity():
    rng = np.random.default_rng(105)
    q, kv, pt = identity_problem(rng, 2, 2, 1)
    sel = np.full((2, 4), -1, np.int32)
    sel[1, :2] = [5, 9]
    out, lse, _ = oracle.sparse_mla_decode(q, kv, pt, sel, np.array([0, 2], np.int32), D_V, 0.1)
    assert np.all(out[0] == 0.0) and np.all(np.isneginf(lse[0]))
    assert np.all(np.isfinite(lse[1])) and np.abs(out[1]).max() > 0


# ----------------------------------------------------------------------------- invariants

def _small_sparse(rng, B=2, H=3, n_pages=4, n_sel=70):
    q = rand_bf16(rng, (B, H, D_QK))
    kv = rand_bf16(rng, (B * n_pages, PAGE, D_QK))
    pt = rng.permutation(B * n_pages).astype(np.int32).reshape(B, n_pages)
    sel = np.stack([rng.permutation(n_pages * PAGE)[:n_sel] for _ in range(B)]).astype(np.int32)
    return q, kv, pt, sel, np.full(B, n_sel, np.int32)


def test_softmax_weights_sum_to_one():
    rng = np.random.default_rng(106)
    q, kv, pt, sel, n = _small_sparse(rng)
    rows = oracle.resolve_rows(pt, sel, n, PAGE, kv.shape[0])
    krows = kv.reshape(-1, D_QK)[torch.from_numpy(rows)]
    _, _, wsum = oracle.attend_rows(q, krows, n, D_V, 2.0, want_wsum=True)
    assert np.abs(wsum - 1.0).max() < 1e-14


def test_all_ones_values_give_all_ones_output():
    rng = np.random.default_rng(107)
    q, kv, pt, sel, n = _small_sparse(rng)
    kv[..., :D_V] = 1.0
    out, _, _ = oracle.sparse_mla_decode(q, kv, pt, sel, n, D_V, 1.5)
    assert np.abs(out - 1.0).max() < 1e-14


def test_permuting_the_selection_changes_nothing_beyond_rounding():
    rng = np.random.default_rng(108)
    q, kv, pt, sel, n = _small_sparse(rng)
    o0, l0, _ = oracle.sparse_mla_decode(q, kv, pt, sel, n, D_V, 0.4)
    sel2 = np.stack([rng.permutation(r) for r in sel])
    o1, l1, _ = oracle.sparse_mla_decode(q, kv, pt, sel2, n, D_V, 0.4)
    assert np.abs(o1 - o0).max() < 1e-13 and np.abs(l1 - l0).max() < 1e-13


def test_relabelling_physical_pages_changes_nothing_bit_for_bit():
    rng = np.random.default_rng(109)
    q, kv, pt, sel, n = _small_sparse(rng)
    o0, l0, _ = oracle.sparse_mla_decode(q, kv, pt, sel, n, D_V, 0.4)
    relabel = rng.permutation(kv.shape[0])                  # old physical id -> new physical id
    kv2 = torch.empty_like(kv)
    kv2[torch.from_numpy(relabel)] = kv
    pt2 = relabel[pt].astype(np.int32)
    o1, l1, _ = oracle.sparse_mla_decode(q, kv2, pt2, sel, n, D_V, 0.4)
    assert np.array_equal(o0, o1) and np.array_equal(l0, l1)


def test_ignores_entries_beyond_sel_len():
    rng = np.random.default_rng(110)
    q, kv, pt, sel, n = _small_sparse(rng)
    n2 = np.array([33, 70], np.int32)
    o0, l0, _ = oracle.sparse_mla_decode(q, kv, pt, sel, n2, D_V, 0.4)
    sel2 = sel.copy()
    sel2[0, 33:] = -1
    o1, l1, _ = oracle.sparse_mla_decode(q, kv, pt, sel2, n2, D_V, 0.4)
    assert np.array_equal(o0, o1) and np.array_equal(l0, l1)


# ----------------------------------------------------------------------------- combine

def test_any_partition_merges_to_the_unsplit_result():
    rng = np.random.default_rng(111)
    q, kv, pt, sel, n = _small_sparse(rng, B=2, H=3, n_sel=70)
    full, full_lse, _ = oracle.sparse_mla_decode(q, kv, pt, sel, n, D_V, 0.9)
    for cuts in ([0, 70], [0, 1, 70], [0, 13, 13, 40, 70], [0, 64, 70, 70]):
        S = len(cuts) - 1
        po = np.zeros((2, S + 1, 3, D_V))
        pl = np.full((2, S + 1, 3), -np.inf)
        for s in range(S):
            a, b_ = cuts[s], cuts[s + 1]
            part_sel = np.full_like(sel, -1)
            part_sel[:, : b_ - a] = sel[:, a:b_]
            po[:, s], pl[:, s], _ = oracle.sparse_mla_decode(q, kv, pt, part_sel,
                                                             np.full(2, b_ - a, np.int32), D_V, 0.9)
        out, lse = oracle.splitkv_combine(po, pl, np.array([S, S + 1], np.int32))
        assert np.abs(out - full).max() < 1e-13
        assert np.abs(lse - full_lse).max() < 1e-13


def test_combine_of_two_equal_halves_is_their_average_and_lse_plus_ln2():
    po = np.zeros((1, 2, 1, 4))
    po[0, 0, 0] = [1, 2, 3, 4]
    po[0, 1, 0] = [3, 2, 1, 0]
    pl = np.full((1, 2, 1), 0.75)
    out, lse = oracle.splitkv_combine(po, pl, np.array([2], np.int32))
    assert np.allclose(out[0, 0], [2, 2, 2, 2], atol=1e-15)
    assert abs(lse[0, 0] - (0.75 + math.log(2))) < 1e-15


def test_combine_weights_follow_exp_of_lse_difference():
    po = np.zeros((1, 2, 1, 1))
    po[0, 0, 0, 0], po[0, 1, 0, 0] = 10.0, -5.0
    pl = np.array([[[math.log(3.0)], [0.0]]])               # partition functions 3 and 1
    out, lse = oracle.splitkv_combine(po, pl, np.array([2], np.int32))
    assert abs(out[0, 0, 0] - (0.75 * 10.0 + 0.25 * -5.0)) < 1e-14
    assert abs(lse[0, 0] - math.log(4.0)) < 1e-15


def test_combine_of_only_empty_partials_is_zero_and_minus_infinity():
    po = np.ones((1, 3, 2, 4))
    pl = np.full((1, 3, 2), -np.inf)
    out, lse = oracle.splitkv_combine(po, pl, np.array([3], np.int32))
    assert np.all(out == 0.0) and np.all(np.isneginf(lse))
    out, lse = oracle.splitkv_combine(po, pl, np.array([0], np.int32))
    assert np.all(out == 0.0) and np.all(np.isneginf(lse))


# ----------------------------------------------------------------------------- index resolution

def test_resolve_rows_matches_hand_worked_table():
    pt = np.array([[5, 2, 0], [1, 4, 3]], np.int32)
    cases = {0: [], 1: []}
    with open(os.path.join(GOLDEN, "resolve_rows_case.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            b, t, r = (int(x) for x in line.split())
            cases[b].append((t, r))
    max_sel = max(len(v) for v in cases.values()) + 2
    sel = np.full((2, max_sel), -1, np.int32)
    n = np.zeros(2, np.int32)
    for b, v in cases.items():
        sel[b, : len(v)] = [t for t, _ in v]
        n[b] = len(v)
    rows = oracle.resolve_rows(pt, sel, n, 4, 6)
    for b, v in cases.items():
        assert rows[b, : len(v)].tolist() == [r for _, r in v]
        assert np.all(rows[b, len(v):] == -1)


def test_histogram_construction_counts_exactly_which_rows_were_read():
    # q = 0 gives uniform weights 1/N; one-hot value rows turn the output into a histogram
    # of the physical rows that were read.  N is a power of two, so N*out is exact.
    rng = np.random.default_rng(112)
    n_pages, N = 8, 128
    kv = torch.zeros(n_pages, PAGE, D_QK, dtype=torch.bfloat16)
    rows_all = np.arange(n_pages * PAGE)
    kv.view(-1, D_QK)[torch.from_numpy(rows_all), torch.from_numpy(rows_all % D_V)] = 1.0
    q = torch.zeros(1, 2, D_QK, dtype=torch.bfloat16)
    pt = rng.permutation(n_pages).astype(np.int32)[None]
    sel = rng.permutation(n_pages * PAGE)[:N].astype(np.int32)[None]
    out, lse, rows = oracle.sparse_mla_decode(q, kv, pt, sel, np.array([N], np.int32), D_V, 1.0)
    expect = np.zeros(D_V)
    for t in sel[0]:                                        # explicit, independent arithmetic
        phys = int(pt[0, t // PAGE]) * PAGE + int(t % PAGE)
        expect[phys % D_V] += 1
    assert np.array_equal(out[0, 0] * N, expect) and np.array_equal(out[0, 1] * N, expect)
    assert np.abs(lse - math.log(N)).max() < 1e-15


def test_spike_construction_returns_the_spiked_rows_value_bits():
    rng = np.random.default_rng(113)
    q, kv, pt, sel, n = _small_sparse(rng, B=1, H=2, n_pages=4, n_sel=40)
    kv[..., D_V:] = 0.0
    q[..., D_V:] = 0.0
    j = 17
    t = int(sel[0, j])
    phys = int(pt[0, t // PAGE]) * PAGE + t % PAGE
    q[0, :, D_QK - 1] = 64.0
    kv.view(-1, D_QK)[phys, D_QK - 1] = 64.0                # score 4096*scale above the rest
    out, _, _ = oracle.sparse_mla_decode(q, kv, pt, sel, n, D_V, 1.0)
    want = f64(kv).reshape(-1, D_QK)[phys, :D_V]
    assert np.array_equal(out[0, 0], want) and np.array_equal(out[0, 1], want)   # exp(-4096) == 0


def test_contract_violations_are_reported_not_computed():
    pt = np.array([[0, 1]], np.int32)
    q = torch.zeros(1, 1, D_QK, dtype=torch.bfloat16)
    kv = torch.zeros(2, PAGE, D_QK, dtype=torch.bfloat16)
    for bad_sel in ([[-1]], [[2 * PAGE]]):
        with pytest.raises(ValueError):
            oracle.sparse_mla_decode(q, kv, pt, np.array(bad_sel, np.int32), np.array([1], np.int32), D_V, 1.0)
    with pytest.raises(ValueError):                          # page id outside the pool
        oracle.sparse_mla_decode(q, kv, np.array([[0, 7]], np.int32), np.array([[PAGE]], np.int32),
                                 np.array([1], np.int32), D_V, 1.0)
    with pytest.raises(ValueError):                          # sel_len beyond the row stride
        oracle.resolve_rows(pt, np.array([[0]], np.int32), np.array([2], np.int32), PAGE, 2)


# ----------------------------------------------------------------------------- Eq. 2 generator

def test_sink_recent_matches_hand_worked_sets():
    with open(os.path.join(GOLDEN, "eq2_index_sets.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            left, right = line.split("|")
            M, ns, nr = (int(x) for x in left.split())
            assert sink_recent(M, ns, nr).tolist() == [int(x) for x in right.split()]


def test_sink_recent_size_and_dense_limit():
    for M, ns, nr in [(100, 4, 16), (100, 60, 60), (64, 64, 0), (7, 0, 0)]:
        s = sink_recent(M, ns, nr)
        assert len(s) == min(M, ns + nr) and len(set(s.tolist())) == len(s)
        if ns + nr >= M:
            assert s.tolist() == list(range(M))


def test_sink_recent_attention_equals_dense_attention_over_a_cache_with_the_rest_evicted():
    rng = np.random.default_rng(114)
    n_pages, ns, nr = 6, 64, 128                            # page-aligned so eviction is by page
    q, kv, pt = identity_problem(rng, 1, 3, n_pages)
    M = n_pages * PAGE
    sel = sink_recent(M, ns, nr)[None]
    o_sparse, l_sparse, _ = oracle.sparse_mla_decode(q, kv, pt, sel, np.array([sel.shape[1]], np.int32), D_V, 0.2)
    kept_pages = [0, 4, 5]
    kv_small = kv[kept_pages].contiguous()
    Ms = len(kept_pages) * PAGE
    o_dense, l_dense, _ = oracle.sparse_mla_decode(q, kv_small, np.arange(3, dtype=np.int32)[None],
                                                   np.arange(Ms, dtype=np.int32)[None],
                                                   np.array([Ms], np.int32), D_V, 0.2)
    assert np.array_equal(o_sparse, o_dense) and np.array_equal(l_sparse, l_dense)


# ------------------------------------------------------------------ rolling cache layout

def test_rolling_cache_keeps_every_token_of_the_index_set():
    # Replaying the appends of a whole context and reading the index set back must return
    # exactly the rows that were appended at those positions: no slot of the ring is reused
    # while its token is still inside the recent window, whatever the context length.
    from oracle import rolling, selection
    rng = np.random.default_rng(90)
    for n_sink, n_recent in ((64, 256), (5, 100), (0, 1), (70, 0), (130, 64), (1, 63)):
        sink_pages, ring_pages = rolling.pages_per_request(n_sink, n_recent)
        pages = sink_pages + ring_pages
        table = rng.permutation(pages + 3)[:pages].astype(np.int32)         # scattered physical pages
        for M in (0, 1, 63, 64, 65, 127, 128, 129, 500, 1000):
            rows = rng.integers(1, 1 << 30, size=(M, 2)).astype(np.int64)   # two columns identify a token
            pool = np.zeros((pages + 3, 64, 2), dtype=np.int64)
            rolling.replay_appends(pool, table, rows, n_sink, n_recent)
            want = selection.sink_recent(M, n_sink, n_recent)
            got = rolling.selected_rows(table, M, n_sink, n_recent)
            assert len(got) == len(want) and len(set(got.tolist())) == len(got)
            assert np.array_equal(pool.reshape(-1, 2)[got], rows[want])


def test_rolling_cache_sizes_and_fixed_points():
    from oracle import rolling
    assert rolling.pages_per_request(64, 2048) == (1, 33)
    assert rolling.pages_per_request(0, 1) == (0, 2)
    assert rolling.pages_per_request(65, 64) == (2, 2)
    # the sink pages are never remapped; the first ring block follows them directly
    for t in range(128):
        assert rolling.position(t, 100, 64) == t
    assert rolling.position(128, 100, 64) == 128 and rolling.position(128 + 64, 100, 64) == 192
    assert rolling.position(128 + 2 * 64 + 5, 100, 64) == 128 + 5          # ring of 2 pages wraps
