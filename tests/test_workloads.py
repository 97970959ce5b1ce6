"""Host-side checks of the seeded workload generators (index structures only)."""
import numpy as np

from paper_2511_22481_b200 import workloads as W


def _check_valid(w):
    pt = w.page_table.numpy()
    si = w.sel_idx.numpy()
    sl = w.sel_len.numpy()
    used = []
    for b in range(w.batch):
        n_pages = int(w.ctx_len[b]) // W.PAGE
        assert np.all(pt[b, :n_pages] >= 0) and np.all(pt[b, :n_pages] < w.num_pages)
        used.append(pt[b, :n_pages])
        s = si[b, : sl[b]]
        assert np.all(s >= 0) and np.all(s < w.ctx_len[b])
        assert len(np.unique(s)) == len(s)                   # a set: no duplicates
        assert np.all(si[b, sl[b]:] == -1)
    used = np.concatenate(used)
    assert len(np.unique(used)) == len(used) == w.num_pages  # pages are not shared between requests


def test_config1_counts():
    w = W.config1_tiny()
    assert (w.batch, w.heads, w.num_pages) == (1, 16, 64)
    assert w.sel_len.tolist() == [832]
    assert np.array_equal(w.page_table.numpy()[0], np.arange(64))
    s = w.sel_idx.numpy()[0]
    assert s[:64].tolist() == list(range(64))                # sink page first
    assert s[-256:].tolist() == list(range(4096 - 256, 4096))
    assert w.q.shape == (1, 16, 576) and w.kv_cache.shape == (64, 64, 576)
    _check_valid(w)


def test_config2_structure_without_values():
    w = W.page_sparse("c2", 1, 32, 128, 512, 8, 24, make_values=False)
    assert w.num_pages == 16384 and w.sel_len.tolist() == [2112] * 32
    _check_valid(w)
    w23 = W.page_sparse("c2", 1, 32, 128, 512, 8, 23, make_values=False)
    assert w23.sel_len.tolist() == [2048] * 32


def test_config3_structure_without_values():
    w = W.config3_ragged(make_values=False)
    sl = w.sel_len.numpy()
    assert w.batch == 128 and sl.min() >= 9 * 64 and sl.max() <= 128 * 64
    assert np.all(w.ctx_len >= 4096) and np.all(w.ctx_len <= 65536)
    _check_valid(w)


def test_config4_small_variant_is_unsorted_token_level():
    w = W.config4_topk(batch=2, ctx_pages=32, k=100)
    s = w.sel_idx.numpy()[0]
    assert w.sel_len.tolist() == [100, 100] and not np.all(np.diff(s) > 0)
    _check_valid(w)


def test_sweep_cells_share_inputs_with_their_dense_variant():
    a = W.config5_cell(1, 512, ctx_pages=16)
    d = W.config5_cell(1, 512, dense_variant=True, ctx_pages=16)
    assert a.sel_len.tolist() == [512] and d.sel_len.tolist() == [1024]
    assert np.array_equal(a.page_table.numpy(), d.page_table.numpy())
    assert np.array_equal(a.kv_cache.view(dtype=__import__("torch").int16).numpy(),
                          d.kv_cache.view(dtype=__import__("torch").int16).numpy())
    _check_valid(a)
    _check_valid(d)


def test_same_seed_same_bits():
    a, b = W.config1_tiny(), W.config1_tiny()
    import torch
    assert torch.equal(a.q, b.q) and torch.equal(a.kv_cache, b.kv_cache)
    assert torch.equal(a.sel_idx, b.sel_idx)


def test_sink_recent_generator_matches_the_oracle_index_set():
    from oracle import selection
    ctx = [0, 1, 63, 64, 65, 200, 1000]
    for n_sink, n_recent in ((64, 256), (5, 100), (0, 130), (70, 0), (4096, 4096)):
        w = W.sink_recent("t", 3, len(ctx), 2, ctx, n_sink, n_recent, "cpu", make_values=False)
        for b, m in enumerate(ctx):
            want = selection.sink_recent(m, n_sink, n_recent)
            got = w.sel_idx[b, : int(w.sel_len[b])].numpy()
            assert np.array_equal(got, want)
