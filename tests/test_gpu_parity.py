"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element on
small problems and on sampled (request, head) rows at the full benchmark sizes."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2511_22481_b200 import binding as B
from paper_2511_22481_b200 import workloads as W
from parity import check_workload, compare, oracle_subset, run_gpu

pytestmark = pytest.mark.gpu
DEV = "cuda"
IMPLS = {"simt": B.OMNI_FLAG_SIMT, "tc": 0, "tc_fused_merge": B.OMNI_FLAG_FUSED_MERGE,
         "tc_no_cluster_merge": B.OMNI_FLAG_NO_CLUSTER_MERGE}


@pytest.fixture(params=list(IMPLS))
def flags(request):
    return IMPLS[request.param]


def _custom(name, seed, heads, ctx_pages, sel_lists, shuffle=True):
    """Workload from explicit per-request selection lists."""
    rng = np.random.default_rng(seed)
    tables = W._shuffled_tables(rng, ctx_pages, shuffle)
    return W._pack(name, seed, heads, list(ctx_pages), tables,
                   [np.asarray(s, dtype=np.int32) for s in sel_lists], DEV, dict(kind="custom"))


# ------------------------------------------------------------------ small, every element

def test_config1_tiny(flags):
    stats, plan = check_workload(W.config1_tiny(DEV), flags, what="config1", strict_abs=True)
    assert stats["max_abs"] < 1e-3


@pytest.mark.parametrize("splits", [1, 2, 3, 7])
def test_forced_splits_including_empty_ones(flags, splits):
    w = W.page_sparse("small", 40, 3, 128, [8, 5, 16], 2, [1, 0, 3], DEV)
    check_workload(w, flags, num_splits=splits, what="splits=%d" % splits)


def test_ragged_lengths_and_tails(flags):
    rng = np.random.default_rng(41)
    lens = [0, 1, 2, 63, 64, 65, 127, 129, 300, 513]
    sels = [rng.permutation(16 * 64)[:n] for n in lens]
    w = _custom("ragged_tails", 41, 128, [16] * len(lens), sels)
    for s in (0, 1, 2, 4):
        stats, plan = check_workload(w, flags, num_splits=s, what="ragged tails S=%d" % s)
        assert torch.all(plan.out[0] == 0) and torch.all(torch.isneginf(plan.lse[0]))


@pytest.mark.parametrize("heads", [1, 16, 48, 64, 80, 128])
def test_head_counts(flags, heads):
    w = W.token_topk("heads%d" % heads, 42, 2, heads, 8, 200, DEV)
    for splits in (0, 2, 3):                 # 2: merged inside a cluster when the pair kernel runs
        check_workload(w, flags, num_splits=splits, what="H=%d S=%d" % (heads, splits))


def test_token_level_unsorted_selection(flags):
    w = W.config4_topk(DEV, batch=3, ctx_pages=64, k=777)
    check_workload(w, flags, num_splits=3, what="topk small")


def test_dense_selection_equals_oracle(flags):
    w = W.dense("dense_small", 43, 2, 128, 12, DEV)
    check_workload(w, flags, what="dense small")


def test_same_bits_on_repeat(flags):
    w = W.config4_topk(DEV, batch=2, ctx_pages=32, k=500)
    a = run_gpu(w, flags)
    o1, l1 = a.out.clone(), a.lse.clone()
    b = run_gpu(w, flags, plan=a)
    assert torch.equal(o1, b.out) and torch.equal(l1, b.lse)


# ------------------------------------------------------------------ index handling, bit exact

def test_resolved_rows_match_oracle_bit_for_bit():
    for w in (W.config1_tiny(DEV), W.config4_topk(DEV, batch=4, ctx_pages=128, k=1000),
              W.config3_ragged(DEV, batch=6)):
        desc = B.make_desc(w.batch, w.heads, w.num_pages, w.max_pages_per_req, w.max_sel, w.scale)
        rows = torch.empty((w.batch, w.max_sel), dtype=torch.int64, device=DEV)
        B.omni_sparse_mla_resolve_rows(desc, w.page_table, w.sel_idx, w.sel_len, rows)
        torch.cuda.synchronize()
        ref = oracle.resolve_rows(w.page_table.cpu().numpy(), w.sel_idx.cpu().numpy(),
                                  w.sel_len.cpu().numpy(), w.page_size, w.num_pages)
        assert np.array_equal(rows.cpu().numpy(), ref)


@pytest.mark.parametrize("hi", [0, 1])
def test_histogram_of_rows_read_is_exact(flags, hi):
    # q = 0 -> uniform weights 1/N (N a power of two); one-hot value rows make N*out an exact
    # histogram of the physical rows that were read.
    n_pages, N = 24, 512
    w = W.token_topk("hist", 44, 2, 128, n_pages, N, DEV)
    w.q.zero_()
    rows_all = torch.arange(n_pages * 2 * 64, device=DEV)
    col = (rows_all % 512) if hi == 0 else ((rows_all // 512) % 512)
    w.kv_cache.zero_()
    w.kv_cache.view(-1, 576)[rows_all, col] = 1.0
    for splits in (1, 4):
        plan = run_gpu(w, flags, num_splits=splits)
        ref_out, ref_lse, _ = oracle_subset(w)
        got = plan.out.to(torch.float64).cpu().numpy() * N
        assert np.array_equal(got, ref_out * N)
        assert np.abs(plan.lse.cpu().numpy() - math.log(N)).max() < 1e-5


def test_spiked_row_comes_back_bit_exact(flags):
    w = W.token_topk("spike", 45, 2, 128, 16, 300, DEV)
    w.kv_cache[..., 512:] = 0
    w.q[..., 512:] = 0
    j = 123
    rows = oracle.resolve_rows(w.page_table.cpu().numpy(), w.sel_idx.cpu().numpy(),
                               w.sel_len.cpu().numpy(), 64, w.num_pages)
    w.q[..., 575] = 64.0
    for b in range(2):
        w.kv_cache.view(-1, 576)[int(rows[b, j]), 575] = 64.0
    plan = run_gpu(w, flags, num_splits=2)
    for b in range(2):
        want = w.kv_cache.view(-1, 576)[int(rows[b, j]), :512]
        assert torch.equal(plan.out[b], want.expand(128, 512))


def test_single_token_returns_its_row_exactly(flags):
    w = _custom("one", 46, 128, [4], [[77]])
    plan = run_gpu(w, flags)
    row = int(w.page_table[0, 1].item()) * 64 + 13
    assert torch.equal(plan.out[0], w.kv_cache.view(-1, 576)[row, :512].expand(128, 512))
    ref_out, ref_lse, _ = oracle_subset(w)
    assert np.abs(plan.lse.cpu().numpy() - ref_lse).max() < 1e-4


def test_rows_outside_the_selection_are_never_used(flags):
    # every pool row that is not selected holds NaN: a kernel that pads tiles with rows of its
    # own choosing, or reads beyond a ragged tail, poisons its output
    rng = np.random.default_rng(49)
    lens = [1, 3, 63, 64, 65, 100, 128, 129, 191, 300]
    sels = [rng.permutation(12 * 64)[:n] for n in lens]
    sels[3] = np.arange(5 * 64, 6 * 64)              # one whole page in order
    sels[6] = np.arange(2 * 64, 4 * 64)              # two whole pages in order
    sels[7] = np.arange(2 * 64, 4 * 64 + 1)          # two pages and one token
    w = _custom("nan_outside", 49, 128, [12] * len(lens), sels)
    rows = oracle.resolve_rows(w.page_table.cpu().numpy(), w.sel_idx.cpu().numpy(),
                               w.sel_len.cpu().numpy(), 64, w.num_pages)
    keep = torch.zeros(w.num_pages * 64, dtype=torch.bool, device=DEV)
    keep[torch.from_numpy(rows[rows >= 0]).to(DEV)] = True
    w.kv_cache.view(-1, 576)[~keep] = float("nan")
    for s in (0, 1, 2, 3):
        check_workload(w, flags, num_splits=s, what="nan outside S=%d" % s)


@pytest.mark.parametrize("bad_value", [-3, -2, -1])
def test_out_of_range_entries_are_flagged_and_skipped(flags, bad_value):
    # every negative position breaks the contract, -2 included (the kernels use that value
    # internally as padding of the range form, never on behalf of a caller's list)
    rng = np.random.default_rng(47)
    sel = rng.permutation(8 * 64)[:200].astype(np.int32)
    w = _custom("bad", 47, 128, [8], [sel])
    good = _custom("good", 47, 128, [8], [np.delete(sel, [5, 150])])
    bad_idx = w.sel_idx.clone()
    bad_idx[0, 5] = bad_value
    bad_idx[0, 150] = 8 * 64 + 1
    w.sel_idx = bad_idx
    plan = run_gpu(w, flags)
    assert int(plan.status.item()) & B.OMNI_DEV_BAD_INDEX
    # a lone -2 must be flagged by the decode kernel as well, not only next to another bad entry
    only = w.sel_idx.clone()
    only[0, 150] = sel[150]
    w.sel_idx = only
    plan1 = run_gpu(w, flags)
    assert int(plan1.status.item()) & B.OMNI_DEV_BAD_INDEX
    w.sel_idx = bad_idx
    ref_out, ref_lse, _ = oracle_subset(good)
    compare(plan.out.cpu(), plan.lse.cpu(), ref_out, ref_lse, "skip bad entries")
    desc = B.make_desc(1, 128, w.num_pages, w.max_pages_per_req, w.max_sel, w.scale)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.omni_sparse_mla_validate(desc, w.page_table, w.sel_idx, w.sel_len, st)
    assert int(st.item()) == B.OMNI_DEV_BAD_INDEX
    st.zero_()
    B.omni_sparse_mla_validate(desc, good.page_table, good.sel_idx, good.sel_len, st)
    assert int(st.item()) == 0


# ------------------------------------------------------------------ Eq. 2 as two ranges

def _sink_recent_case(ctx_tokens, n_sink, n_recent, seed, heads=128):
    """Requests whose selection is the oracle's Eq. 2 index set, plus their context lengths."""
    from oracle import selection
    pages = [max(1, -(-m // 64)) for m in ctx_tokens]
    sels = [selection.sink_recent(m, n_sink, n_recent) for m in ctx_tokens]
    w = _custom("sink_recent", seed, heads, pages, sels)
    # positions at or beyond the context length belong to nobody: make sure they are never used
    tail = torch.ones(w.num_pages * 64, dtype=torch.bool, device=DEV)
    pt = w.page_table.cpu().numpy()
    for b, m in enumerate(ctx_tokens):
        for lp in range(pages[b]):
            lo = int(pt[b, lp]) * 64
            tail[lo:lo + max(0, min(64, m - lp * 64))] = False
    w.kv_cache.view(-1, 576)[tail] = float("nan")
    ctx = torch.tensor(ctx_tokens, dtype=torch.int32, device=DEV)
    return w, ctx


def _run_ranges(w, ctx, n_sink, n_recent, flags, num_splits=0):
    desc = B.make_desc(w.batch, w.heads, w.num_pages, w.max_pages_per_req,
                       max(1, min(n_sink + n_recent, w.max_pages_per_req * 64)), w.scale,
                       num_splits=num_splits, flags=flags)
    out = torch.full((w.batch, w.heads, 512), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((w.batch, w.heads), float("nan"), dtype=torch.float32, device=DEV)
    ws = torch.empty(B.omni_sparse_mla_workspace_bytes(desc), dtype=torch.uint8, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.omni_sparse_mla_decode_sink_recent(desc, w.q, w.kv_cache, w.page_table, ctx, n_sink, n_recent,
                                         out, lse, ws, st)
    torch.cuda.synchronize()
    return out, lse, int(st.item())


@pytest.mark.parametrize("n_sink,n_recent", [(64, 256), (5, 100), (0, 130), (70, 0), (4096, 4096)])
def test_sink_recent_ranges_match_oracle_on_the_index_set(flags, n_sink, n_recent):
    # contexts shorter than, equal to and longer than N_sink + N_recent, ragged ends, empty
    ctx_tokens = [0, 1, 63, 64, 65, 200, 321, 330, 1000, 1537]
    w, ctx = _sink_recent_case(ctx_tokens, n_sink, n_recent, seed=60)
    ref_out, ref_lse, _ = oracle_subset(w)
    for splits in (0, 1, 2, 3):
        out, lse, status = _run_ranges(w, ctx, n_sink, n_recent, flags, splits)
        assert status == 0
        compare(out.cpu(), lse.cpu(), ref_out, ref_lse, "sink+recent ranges S=%d" % splits)
        assert torch.all(out[0] == 0) and torch.all(torch.isneginf(lse[0]))


def test_sink_recent_ranges_equal_the_list_path_bit_for_bit(flags):
    # recent ranges that start on a page boundary right behind a page-aligned sink: the range path
    # walks exactly the tiles of the list path
    ctx_tokens = [4096, 832, 130, 2048]
    w, ctx = _sink_recent_case(ctx_tokens, 64, 512, seed=61)
    for splits in (1, 2):
        plan = run_gpu(w, flags, num_splits=splits)
        out, lse, status = _run_ranges(w, ctx, 64, 512, flags, splits)
        assert status == 0
        assert torch.equal(out, plan.out) and torch.equal(lse, plan.lse)


def test_sink_recent_ranges_on_unaligned_windows_stay_close_to_the_list_path(flags):
    # any other start: the range path pads the recent range to page-aligned tiles, so sums are
    # regrouped; both results are within the parity tolerance of the oracle, hence of each other
    ctx_tokens = [4133, 777, 1001, 2049]
    w, ctx = _sink_recent_case(ctx_tokens, 64, 512, seed=63)
    ref_out, ref_lse, _ = oracle_subset(w)
    for splits in (1, 2):
        out, lse, status = _run_ranges(w, ctx, 64, 512, flags, splits)
        assert status == 0
        compare(out.cpu(), lse.cpu(), ref_out, ref_lse, "unaligned ranges S=%d" % splits)
        plan = run_gpu(w, flags, num_splits=splits)
        assert (out.float() - plan.out.float()).abs().max().item() <= 2e-3


def test_sink_recent_bad_context_length_is_flagged():
    w, ctx = _sink_recent_case([100, 200], 16, 32, seed=62)
    ctx[1] = w.max_pages_per_req * 64 + 1
    out, lse, status = _run_ranges(w, ctx, 16, 32, 0)
    assert status & B.OMNI_DEV_BAD_INDEX
    assert torch.all(out[1] == 0) and torch.all(torch.isneginf(lse[1]))


# ------------------------------------------------------------------ combine entry point

def test_combine_entry_point_matches_oracle():
    g = torch.Generator(device="cpu").manual_seed(48)
    Bn, S, H = 3, 5, 16
    po = torch.randn((Bn, S, H, 512), generator=g)
    pl = torch.randn((Bn, S, H), generator=g) * 3
    pl[0, 2] = -math.inf
    pl[1, :, 3] = -math.inf
    ns = torch.tensor([5, 4, 0], dtype=torch.int32)
    ref_out, ref_lse = oracle.splitkv_combine(po.numpy().astype(np.float64), pl.numpy().astype(np.float64), ns.numpy())
    desc = B.make_desc(Bn, H, 1, 1, 1, 1.0)
    out = torch.empty((Bn, H, 512), dtype=torch.bfloat16, device=DEV)
    lse = torch.empty((Bn, H), dtype=torch.float32, device=DEV)
    B.omni_sparse_mla_combine(desc, S, po.to(DEV), pl.to(DEV), ns.to(DEV), out, lse)
    torch.cuda.synchronize()
    got = out.to(torch.float64).cpu().numpy()
    assert np.abs(got - ref_out).max() <= 2 ** -8 * np.abs(ref_out).max()       # bf16 output rounding
    gl = lse.cpu().numpy().astype(np.float64)
    assert np.array_equal(np.isneginf(gl), np.isneginf(ref_lse))
    fin = np.isfinite(ref_lse)
    assert np.abs(gl[fin] - ref_lse[fin]).max() < 1e-5
    assert torch.all(out[2] == 0) and torch.all(out[1, 3] == 0)


# ------------------------------------------------------------------ host-buffer entry point

def test_host_buffer_entry_point(flags):
    w = W.config4_topk(DEV, batch=2, ctx_pages=32, k=300)
    desc = B.make_desc(w.batch, w.heads, w.num_pages, w.max_pages_per_req, w.max_sel, w.scale, flags=flags)
    staging = torch.empty(B.omni_sparse_mla_host_staging_bytes(desc), dtype=torch.uint8, device=DEV)
    ws = torch.empty(B.omni_sparse_mla_workspace_bytes(desc), dtype=torch.uint8, device=DEV)
    pin = lambda t: t.cpu().pin_memory()
    out_h = torch.empty((w.batch, w.heads, 512), dtype=torch.bfloat16).pin_memory()
    lse_h = torch.empty((w.batch, w.heads), dtype=torch.float32).pin_memory()
    B.omni_sparse_mla_decode_host(desc, pin(w.q), w.kv_cache, pin(w.page_table), pin(w.sel_idx),
                                  pin(w.sel_len), out_h, lse_h, staging, ws)
    torch.cuda.synchronize()
    ref_out, ref_lse, _ = oracle_subset(w)
    compare(out_h, lse_h, ref_out, ref_lse, "host entry point")


@pytest.mark.parametrize("batch", [8, 9])
def test_host_buffer_entry_point_two_halves(flags, batch):
    """From 8 requests of 128 heads on, the host entry point runs the batch as two halves on two
    streams; the result must not depend on that."""
    w = W.config4_topk(DEV, batch=batch, ctx_pages=32, k=300)
    desc = B.make_desc(w.batch, w.heads, w.num_pages, w.max_pages_per_req, w.max_sel, w.scale, flags=flags)
    staging = torch.empty(B.omni_sparse_mla_host_staging_bytes(desc), dtype=torch.uint8, device=DEV)
    ws = torch.empty(max(1, B.omni_sparse_mla_workspace_bytes(desc)), dtype=torch.uint8, device=DEV)
    pin = lambda t: t.cpu().pin_memory()
    q, pt, si, sl = pin(w.q), pin(w.page_table), pin(w.sel_idx), pin(w.sel_len)
    out_h = torch.full((w.batch, w.heads, 512), float("nan"), dtype=torch.bfloat16).pin_memory()
    lse_h = torch.full((w.batch, w.heads), float("nan"), dtype=torch.float32).pin_memory()
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    for _ in range(3):                       # back-to-back calls reuse the staging buffer
        B.omni_sparse_mla_decode_host(desc, q, w.kv_cache, pt, si, sl, out_h, lse_h, staging, ws, status)
    torch.cuda.current_stream().synchronize()            # the caller's stream alone covers both halves
    assert int(status.item()) == 0
    ref_out, ref_lse, _ = oracle_subset(w)
    compare(out_h, lse_h, ref_out, ref_lse, "host entry point, two halves")


def test_host_buffer_entry_point_two_calls_in_flight(flags):
    """Two calls on two streams at once, each with its own staging area, result buffers and
    workspace (how the benchmark's end-to-end leg keeps two steps in flight): each result is the
    oracle's, whichever side streams the library picked for them."""
    ws_list = [W.config4_topk(DEV, batch=8, ctx_pages=32, k=300), W.config4_topk(DEV, batch=9, ctx_pages=32, k=280)]
    pin = lambda t: t.cpu().pin_memory()
    lanes = []
    for w in ws_list:
        desc = B.make_desc(w.batch, w.heads, w.num_pages, w.max_pages_per_req, w.max_sel, w.scale, flags=flags)
        lanes.append(dict(
            w=w, desc=desc, stream=torch.cuda.Stream(device=DEV),
            staging=torch.empty(B.omni_sparse_mla_host_staging_bytes(desc), dtype=torch.uint8, device=DEV),
            ws=torch.empty(max(1, B.omni_sparse_mla_workspace_bytes(desc)), dtype=torch.uint8, device=DEV),
            host=[pin(t) for t in (w.q, w.page_table, w.sel_idx, w.sel_len)],
            out_h=torch.full((w.batch, w.heads, 512), float("nan"), dtype=torch.bfloat16).pin_memory(),
            lse_h=torch.full((w.batch, w.heads), float("nan"), dtype=torch.float32).pin_memory(),
            status=torch.zeros(1, dtype=torch.int32, device=DEV)))
    torch.cuda.synchronize()
    for _ in range(3):
        for ln in lanes:
            q, pt, si, sl = ln["host"]
            B.omni_sparse_mla_decode_host(ln["desc"], q, ln["w"].kv_cache, pt, si, sl, ln["out_h"], ln["lse_h"],
                                          ln["staging"], ln["ws"], ln["status"], ln["stream"])
    for ln in lanes:
        ln["stream"].synchronize()                       # each caller's stream alone covers its call
        assert int(ln["status"].item()) == 0
        ref_out, ref_lse, _ = oracle_subset(ln["w"])
        compare(ln["out_h"], ln["lse_h"], ref_out, ref_lse, "host entry point, two calls in flight")


# ------------------------------------------------------------------ full benchmark sizes

def test_config2_full_size_every_row(flags):
    """Config 2 in the launch configuration the benchmark times: every (request, head) row."""
    w = W.config2_r1(DEV)
    check_workload(w, flags, what="config2", strict_abs=True)


def test_config2_2048_variant(flags):
    w = W.config2_r1(DEV, middle_pages=23)
    check_workload(w, flags, reqs=[7], heads=[1, 100], what="config2/2048", strict_abs=True)


def test_config3_ragged_full_size_sixteen_requests_all_heads(flags):
    w = W.config3_ragged(DEV)
    sl = w.sel_len.cpu().numpy()
    order = np.argsort(sl, kind="stable")
    # the shortest and the longest selections, the first and the last request, and a spread of the rest
    reqs = sorted({int(order[0]), int(order[1]), int(order[-1]), int(order[-2]), 0, 127} |
                  {int(order[i]) for i in range(5, 128, 12)})
    assert len(reqs) >= 16
    check_workload(w, flags, reqs=reqs, what="config3", strict_abs=True)


def test_config4_topk_full_size_every_row(flags):
    w = W.config4_topk(DEV)
    check_workload(w, flags, what="config4", strict_abs=True)


def _sample_requests(batch):
    """First, last and two interior requests (at most four): with more work units than the device
    runs at once, these sit in different waves of the launch."""
    return sorted({0, batch // 3, (2 * batch) // 3, batch - 1})


@pytest.mark.parametrize("batch,n", [(1, 512), (8, 8192), (32, 2048), (32, 8192), (128, 512), (128, 8192),
                                     (256, 2048), (256, 8192)])
def test_config5_sparse_cells_sampled_all_heads(batch, n):
    w = W.config5_cell(batch, n, DEV)
    check_workload(w, 0, reqs=_sample_requests(batch), what="config5 B%d N%d" % (batch, n), strict_abs=True)


@pytest.mark.parametrize("batch", [1, 8, 32])
def test_config5_dense_cells_sampled_all_heads(batch):
    """The dense arm of the sweep (all 65536 tokens): several splits per request and a separate
    merge launch from batch 8 on."""
    w = W.config5_cell(batch, 2048, DEV, dense_variant=True)
    reqs = _sample_requests(batch)[:2] if batch > 1 else [0]
    check_workload(w, 0, reqs=reqs, what="config5 dense B%d" % batch, strict_abs=True)
