"""Rolling cache of a compressed layer on the GPU: the append kernel against the oracle's replay,
bit for bit, and decode over the rolling layout against (i) the oracle on the rows the oracle's
own addressing selects and (ii) the same decode over an uncompressed cache holding the same
token rows, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from oracle import rolling
from paper_2511_22481_b200 import binding as B
from parity import compare

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _build(batch, tokens, n_sink, n_recent, seed, heads=128):
    g = torch.Generator(device="cpu").manual_seed(seed)
    pages_req = B.omni_rolling_pages_per_request(n_sink, n_recent)
    assert pages_req == sum(rolling.pages_per_request(n_sink, n_recent))
    num_pages = batch * pages_req + 5
    perm = torch.randperm(num_pages, generator=g)[: batch * pages_req].to(torch.int32)
    table = perm.view(batch, pages_req).contiguous()
    stream = (0.5 * torch.randn((batch, max(tokens, 1), 576), generator=g)).to(torch.bfloat16)
    q = (0.5 * torch.randn((batch, heads, 576), generator=g)).to(torch.bfloat16)
    return table, stream, q, num_pages, pages_req


def _append_all(table, stream, tokens, n_sink, n_recent, num_pages, pages_req):
    batch = table.shape[0]
    pool = torch.full((num_pages, 64, 576), float("nan"), dtype=torch.bfloat16, device=DEV)
    desc = B.make_desc(batch, 128, num_pages, pages_req, max(1, n_sink + n_recent), 0.1)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    table_d, stream_d = table.to(DEV), stream.to(DEV)
    ctx = torch.zeros(batch, dtype=torch.int32, device=DEV)
    for t in range(tokens):
        B.omni_kv_append_rolling(desc, pool, table_d, ctx, stream_d[:, t].contiguous(), n_sink, n_recent, status)
        ctx += 1
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return pool, table_d, ctx


@pytest.mark.parametrize("n_sink,n_recent", [(64, 256), (5, 100), (130, 64), (0, 130)])
@pytest.mark.parametrize("tokens", [1, 64, 65, 333, 900])
def test_append_matches_the_oracle_replay_bit_for_bit(n_sink, n_recent, tokens):
    table, stream, q, num_pages, pages_req = _build(3, tokens, n_sink, n_recent, seed=80 + tokens)
    pool, _, _ = _append_all(table, stream, tokens, n_sink, n_recent, num_pages, pages_req)
    want = np.full((num_pages, 64, 576), 0x7FC0, dtype=np.uint16)          # bf16 NaN, as the pool was filled
    bits = oracle.bf16_bits(stream)
    for b in range(3):
        rolling.replay_appends(want, table[b].numpy(), bits[b, :tokens], n_sink, n_recent)
    got = oracle.bf16_bits(pool.cpu())
    assert np.array_equal(got, want)


@pytest.mark.parametrize("n_sink,n_recent", [(64, 256), (5, 100), (130, 64)])
@pytest.mark.parametrize("tokens", [1, 65, 333, 1500])
def test_decode_over_the_rolling_cache(n_sink, n_recent, tokens):
    batch, heads = 3, 128
    table, stream, q, num_pages, pages_req = _build(batch, tokens, n_sink, n_recent, seed=85 + tokens)
    pool, table_d, ctx = _append_all(table, stream, tokens, n_sink, n_recent, num_pages, pages_req)
    max_sel = max(1, n_sink + n_recent)
    scale = 1.0 / 192 ** 0.5
    q_d = q.to(DEV)

    def run(entry, desc, kv, tab):
        out = torch.full((batch, heads, 512), float("nan"), dtype=torch.bfloat16, device=DEV)
        lse = torch.full((batch, heads), float("nan"), dtype=torch.float32, device=DEV)
        ws = torch.empty(B.omni_sparse_mla_workspace_bytes(desc), dtype=torch.uint8, device=DEV)
        st = torch.zeros(1, dtype=torch.int32, device=DEV)
        entry(desc, q_d, kv, tab, ctx, n_sink, n_recent, out, lse, ws, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        return out, lse

    for splits in (0, 1, 2):
        desc = B.make_desc(batch, heads, num_pages, pages_req, max_sel, scale, num_splits=splits)
        out, lse = run(B.omni_sparse_mla_decode_rolling, desc, pool, table_d)
        # (i) the oracle on the rows its own addressing picks out of the GPU's pool
        pool_rows = pool.view(-1, 576).cpu()
        sel = [rolling.selected_rows(table[b].numpy(), tokens, n_sink, n_recent) for b in range(batch)]
        n = np.asarray([len(s) for s in sel], dtype=np.int32)
        krows = torch.zeros((batch, max(1, int(n.max())), 576), dtype=torch.bfloat16)
        for b in range(batch):
            krows[b, : n[b]] = pool_rows[torch.from_numpy(sel[b])]
        ref_out, ref_lse = oracle.attend_rows(q, krows, n, 512, scale)
        compare(out.cpu(), lse.cpu(), ref_out, ref_lse, "rolling decode S=%d" % splits)
        # (ii) an uncompressed cache with the same token rows gives the same bits (same forced split plan)
        if splits == 0:
            continue
        dense_pages = max(1, -(-tokens // 64))
        dense = torch.full((batch * dense_pages, 64, 576), float("nan"), dtype=torch.bfloat16, device=DEV)
        dense.view(batch, dense_pages * 64, 576)[:, :tokens] = stream[:, :tokens].to(DEV)
        dense_table = torch.arange(batch * dense_pages, dtype=torch.int32, device=DEV).view(batch, dense_pages)
        ddesc = B.make_desc(batch, heads, batch * dense_pages, dense_pages,
                            max(1, min(n_sink + n_recent, dense_pages * 64)), scale, num_splits=splits)
        dout, dlse = run(B.omni_sparse_mla_decode_sink_recent, ddesc, dense, dense_table)
        assert torch.equal(out, dout) and torch.equal(lse, dlse)
