"""The 8-bit latent cache on the GPU: the quantiser against the oracle's, bit for bit, and the
decode call against the oracle's attention over the de-quantised rows, element by element on
small problems and on sampled rows at the benchmark size, under the tolerances of the bf16 path."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import q8
from paper_2511_22481_b200 import binding as B
from paper_2511_22481_b200 import workloads as W
from parity import check_workload_q8, quantise_pool_q8

pytestmark = pytest.mark.gpu
DEV = "cuda"
IMPLS = {"default": 0, "fused_merge": B.OMNI_FLAG_FUSED_MERGE, "no_cluster_merge": B.OMNI_FLAG_NO_CLUSTER_MERGE}


@pytest.fixture(params=list(IMPLS))
def flags(request):
    return IMPLS[request.param]


def _custom(name, seed, heads, ctx_pages, sel_lists, shuffle=True):
    rng = np.random.default_rng(seed)
    tables = W._shuffled_tables(rng, ctx_pages, shuffle)
    return W._pack(name, seed, heads, list(ctx_pages), tables,
                   [np.asarray(s, dtype=np.int32) for s in sel_lists], DEV, dict(kind="custom"))


def test_quantiser_matches_the_oracle_bit_for_bit_on_special_rows():
    rng = np.random.default_rng(60)
    rows = (rng.standard_normal((777, 576)) * 0.5).astype(np.float32)
    rows[0] = 0.0                                             # all zero: floored scale, zero codes
    rows[1, :512] = 0.0                                       # zero latent part, live rope part
    rows[2] *= 1e4                                            # large magnitudes
    rows[3] *= 1e-6                                           # small magnitudes
    rows[4, :512] = np.where(rng.random(512) < 0.5, 448.0, -224.0)      # exact code points
    rows[5, 7] = 3.0e38                                       # near the top of the bf16 range
    rows[6, :512] = rng.standard_normal(512) * 2.0 ** -120    # far below the floor of the scale
    rows[7, 100] = -0.0
    t = torch.from_numpy(rows).to(torch.bfloat16).to(DEV)
    cache = torch.empty((777, 640), dtype=torch.uint8, device=DEV)
    scale = torch.empty((777,), dtype=torch.float32, device=DEV)
    B.omni_kv_quantize_q8(t, cache, scale)
    torch.cuda.synchronize()
    want_cache, want_scale = q8.quantise_rows(t.cpu().view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(scale.cpu().numpy().view(np.uint32), want_scale.view(np.uint32))
    assert np.array_equal(cache.cpu().numpy(), want_cache)


def test_small_page_sparse(flags):
    w = W.page_sparse("q8_small", 61, 3, 128, [8, 5, 16], 2, [1, 0, 3], DEV)
    for splits in (0, 1, 2, 3):
        check_workload_q8(w, flags, num_splits=splits, what="q8 page sparse S=%d" % splits)


def test_token_level_and_ragged_tails(flags):
    rng = np.random.default_rng(62)
    lens = [0, 1, 2, 63, 64, 65, 127, 129, 300, 513]
    sels = [rng.permutation(16 * 64)[:n] for n in lens]
    w = _custom("q8_ragged", 62, 128, [16] * len(lens), sels)
    quantised = quantise_pool_q8(w)
    for splits in (0, 1, 2, 4):
        stats, plan = check_workload_q8(w, flags, num_splits=splits, what="q8 ragged S=%d" % splits, quantised=quantised)
        assert torch.all(plan.out[0] == 0) and torch.all(torch.isneginf(plan.lse[0]))


@pytest.mark.parametrize("heads", [65, 80, 128])
def test_head_counts(heads):
    w = W.token_topk("q8_heads%d" % heads, 63, 2, heads, 8, 200, DEV)
    for splits in (0, 2, 3):
        check_workload_q8(w, 0, num_splits=splits, what="q8 H=%d S=%d" % (heads, splits))


def test_rows_with_very_different_scales_and_a_peaked_softmax():
    """Token scales spanning thirteen binades (the weights absorb them) and one dominant score."""
    rng = np.random.default_rng(64)
    sel = rng.permutation(12 * 64)[:500]
    w = _custom("q8_scales", 64, 128, [12], [sel])
    rows = w.kv_cache.view(-1, 576)
    factor = torch.from_numpy(np.exp2(rng.integers(-10, 3, rows.shape[0])).astype(np.float32)).to(DEV)
    rows[:, :512] = (rows[:, :512].float() * factor[:, None]).to(torch.bfloat16)
    hot = int(w.page_table[0, int(sel[123]) // 64].item()) * 64 + int(sel[123]) % 64
    rows[hot, 512:] = (w.q[0, 5, 512:].float() * 40).to(torch.bfloat16)          # head 5 attends almost only here
    check_workload_q8(w, 0, what="q8 scales")


def test_same_bits_on_repeat_and_untouched_rows_may_hold_anything():
    rng = np.random.default_rng(65)
    sel = rng.permutation(10 * 64)[:333]
    w = _custom("q8_repeat", 65, 128, [10], [sel])
    cache, scale = quantise_pool_q8(w)
    used = np.zeros(w.num_pages * 64, dtype=bool)
    pt = w.page_table.cpu().numpy()[0]
    used[pt[sel // 64] * 64 + sel % 64] = True
    unused = torch.from_numpy(~used).to(DEV)
    cache[unused] = 0x7F                                      # NaN codes
    scale[unused] = float("nan")
    _, first = check_workload_q8(w, 0, num_splits=2, what="q8 first", quantised=(cache, scale))
    out1, lse1 = first.out.clone(), first.lse.clone()
    _, second = check_workload_q8(w, 0, num_splits=2, what="q8 second", quantised=(cache, scale))
    assert torch.equal(out1, second.out) and torch.equal(lse1, second.lse)


def test_config2_full_size_sampled():
    w = W.config2_r1(DEV)
    check_workload_q8(w, 0, reqs=[0, 13, 31], what="q8 config2", strict_abs=True)


def test_argument_checks():
    w = W.token_topk("q8_args", 66, 1, 64, 4, 50, DEV)
    plan = B.plan_for(w)
    cache = torch.empty((w.num_pages * 64, 640), dtype=torch.uint8, device=DEV)
    scale = torch.ones((w.num_pages * 64,), dtype=torch.float32, device=DEV)
    with pytest.raises(B.OmniError) as info:                  # 64 heads: the 8-bit path needs the paired-CTA kernel
        B.omni_sparse_mla_decode_q8(plan.desc, w.q, cache, scale, w.page_table, w.sel_idx, w.sel_len, plan.out, plan.lse,
                                    plan.workspace, plan.status)
    assert info.value.code == 2
    lib = B.load()
    ok = ctypes.c_void_p(4096)
    assert lib.omni_kv_quantize_q8(None, 10, ok, ok, None) == 1
    assert lib.omni_kv_quantize_q8(ok, 0, ok, ok, None) == 2
    assert lib.omni_kv_quantize_q8(ctypes.c_void_p(4096 + 8), 10, ok, ok, None) == 3
