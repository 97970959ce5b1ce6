"""GPU parity of the top-k selection producer (through the C ABI) against the oracle's
definition: index lists bit for bit, then the produced lists driving the decode call."""
import numpy as np
import pytest
import torch

from oracle.topk import topk_batch
from paper_2511_22481_b200 import binding as B
from paper_2511_22481_b200 import workloads as W
from parity import compare, oracle_subset, run_gpu

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _run(scores, ctx_len, k):
    s = torch.from_numpy(np.ascontiguousarray(scores, dtype=np.float32)).to(DEV)
    cl = torch.tensor(list(ctx_len), dtype=torch.int32, device=DEV)
    sel_idx = torch.full((s.shape[0], k), -7, dtype=torch.int32, device=DEV)
    sel_len = torch.full((s.shape[0],), -7, dtype=torch.int32, device=DEV)
    B.omni_topk_select(s, cl, k, sel_idx, sel_len)
    torch.cuda.synchronize()
    return sel_idx.cpu().numpy(), sel_len.cpu().numpy()


def _check(scores, ctx_len, k):
    got_idx, got_len = _run(scores, ctx_len, k)
    want_idx, want_len = topk_batch(scores, ctx_len, k)
    assert got_len.tolist() == want_len.tolist()
    for b in range(len(want_len)):
        n = int(want_len[b])
        assert np.array_equal(got_idx[b, :n], want_idx[b, :n]), "request %d" % b
        assert np.all(got_idx[b, n:] == -7)                 # entries beyond sel_len stay untouched


@pytest.mark.parametrize("stride,k", [(1, 1), (7, 3), (8, 8), (513, 64), (4097, 512), (70000, 2048),
                                       (131072, 2048), (131072, 131072)])
def test_random_scores_ragged_lengths(stride, k):
    rng = np.random.default_rng(stride + k)
    batch = 5
    scores = rng.standard_normal((batch, stride)).astype(np.float32)
    ctx = [stride, 0, max(1, stride // 3), min(stride, k), max(1, stride - 1)]
    _check(scores, ctx, k)


@pytest.mark.parametrize("batch,stride,k", [(200, 5000, 300), (80, 20000, 1000), (40, 40000, 64), (1, 131072, 2048)])
def test_cluster_widths_follow_batch_and_context(batch, stride, k):
    """The launch picks 1, 2, 4 or 8 CTAs per request from the batch and the context length."""
    rng = np.random.default_rng(batch)
    scores = np.round(rng.standard_normal((batch, stride)) * 50).astype(np.float32)
    ctx = rng.integers(0, stride + 1, batch).tolist()
    ctx[0] = stride
    _check(scores, ctx, k)


@pytest.mark.parametrize("levels", [1, 2, 6, 300])
def test_heavy_ties(levels):
    rng = np.random.default_rng(levels)
    stride, k = 20011, 1500
    scores = rng.integers(0, levels, (4, stride)).astype(np.float32) - levels / 2
    _check(scores, [stride, 9000, 1499, 1501], k)


def test_special_values():
    rng = np.random.default_rng(5)
    stride, k = 9001, 700
    scores = rng.standard_normal((3, stride)).astype(np.float32)
    pool = np.array([0.0, -0.0, np.nan, np.inf, -np.inf, 1e-45, -1e-45, 3.4e38], dtype=np.float32)
    mask = rng.random((3, stride)) < 0.4
    scores[mask] = pool[rng.integers(0, len(pool), int(mask.sum()))]
    scores[2, :] = np.nan
    _check(scores, [stride, stride, stride], k)
    _check(scores, [stride, stride, stride], stride)


def test_nans_with_mixed_sign_bits_rank_by_position():
    """k reaches into the NaNs, which carry either sign bit: all NaNs are equal, lowest positions win."""
    rng = np.random.default_rng(8)
    stride, k = 5000, 3000
    scores = rng.standard_normal((2, stride)).astype(np.float32)
    bits = scores.view(np.uint32)
    nan_at = rng.random((2, stride)) < 0.6
    neg = rng.random((2, stride)) < 0.5
    bits[nan_at & neg] = 0xFFC00000
    bits[nan_at & ~neg] = 0x7FC00001
    assert np.isnan(scores[nan_at]).all()
    _check(scores, [stride, 4321], k)


def test_keys_that_differ_only_in_low_bits():
    base = np.float32(1.0).view(np.uint32)
    rng = np.random.default_rng(6)
    bits = (base + rng.integers(0, 5, (2, 30000)).astype(np.uint32)).astype(np.uint32)
    _check(bits.view(np.float32), [30000, 12345], 4096)


@pytest.mark.parametrize("m", [4095, 4096, 4097, 9000])
def test_candidate_counts_around_the_direct_histogram_threshold(m):
    """Scores in [1, 2) share their first key digit, so exactly m keys stay candidates after the
    first pass: on both sides of the count (4096) below which a pass adds straight into the
    published histogram."""
    rng = np.random.default_rng(m)
    scores = (1.0 + rng.random((3, 9000))).astype(np.float32)
    scores[1] = np.round(scores[1] * 64) / 64              # ties inside the shared digit
    _check(scores, [m, m, m - 1], 1000)


def test_argument_checks():
    s = torch.zeros(2, 16, device=DEV)
    cl = torch.zeros(2, dtype=torch.int32, device=DEV)
    idx = torch.zeros(2, 4, dtype=torch.int32, device=DEV)
    ln = torch.zeros(2, dtype=torch.int32, device=DEV)
    with pytest.raises(B.OmniError):
        B.omni_topk_select(s, cl, 0, idx, ln)
    with pytest.raises(B.OmniError):
        B.omni_topk_select(s, cl, 17, idx, ln)
    big = torch.zeros(1, 131073, device=DEV)
    with pytest.raises(B.OmniError):
        B.omni_topk_select(big, cl[:1], 4, idx[:1], ln[:1])


def test_produced_selection_drives_the_decode_call():
    """scores -> top-k kernel -> decode kernel, against the oracle fed with the oracle's own top-k."""
    k = 600
    w = W.config4_topk(DEV, batch=3, ctx_pages=48, k=k)
    rng = np.random.default_rng(11)
    ctx = 48 * 64
    lens = [ctx, ctx - 100, 500]
    scores = np.round(rng.standard_normal((3, ctx)) * 4).astype(np.float32) / 4      # many ties
    want_idx, want_len = topk_batch(scores, lens, k)
    s = torch.from_numpy(scores).to(DEV)
    cl = torch.tensor(lens, dtype=torch.int32, device=DEV)
    w.sel_idx.fill_(0)
    B.omni_topk_select(s, cl, k, w.sel_idx, w.sel_len)
    plan = run_gpu(w, 0)
    assert int(plan.status.item()) == 0
    gpu_out, gpu_lse = plan.out.cpu().clone(), plan.lse.cpu().clone()
    assert w.sel_len.cpu().tolist() == want_len.tolist()
    # the oracle reads its own lists, not the kernel's
    w.sel_idx.copy_(torch.from_numpy(np.where(want_idx < 0, 0, want_idx)).to(DEV))
    w.sel_len.copy_(torch.from_numpy(want_len).to(DEV))
    heads = [0, 63, 127]
    ref_out, ref_lse, _ = oracle_subset(w, None, heads)
    compare(gpu_out[:, heads], gpu_lse[:, heads], ref_out, ref_lse, what="topk -> decode")
