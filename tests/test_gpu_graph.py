"""A layer loop under one CUDA graph: the paper applies its compression per layer with a 0/1
pattern (sparse sink + recent selection on some layers, the full context on the others).  Here a
few "layers" (each with its own q and its own pattern bit) are captured into one CUDA graph
through the public entry points and replayed; every layer's result must equal, bit for bit, what
the same calls produce when launched one by one, and a sparse and a dense layer of the replay are
also compared with the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2511_22481_b200 import binding as B
from paper_2511_22481_b200 import workloads as W
from parity import compare, oracle_subset

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _layer_inputs(w, layers, seed):
    g = torch.Generator(device=DEV).manual_seed(seed)
    return [(0.5 * torch.randn(w.q.shape, generator=g, device=DEV, dtype=torch.float32)).to(torch.bfloat16)
            for _ in range(layers)]


def test_layer_loop_in_one_cuda_graph_matches_eager():
    pattern = [1, 0, 1, 1, 0]                      # 1: Eq. 2 selection (sink 64 + recent 512), 0: full context
    ctx_tokens = [4096, 2500, 3333, 4000]
    sparse = W.sink_recent("layers", 70, len(ctx_tokens), 128, ctx_tokens, 64, 512, DEV)
    ctx = torch.as_tensor(sparse.ctx_len, dtype=torch.int32).to(DEV)
    qs = _layer_inputs(sparse, len(pattern), 71)
    max_ctx = sparse.max_pages_per_req * 64

    def make(max_sel):
        desc = B.make_desc(sparse.batch, 128, sparse.num_pages, sparse.max_pages_per_req, max_sel, sparse.scale)
        ws = torch.empty(B.omni_sparse_mla_workspace_bytes(desc), dtype=torch.uint8, device=DEV)
        return desc, ws

    plans = {1: make(64 + 512), 0: make(max_ctx)}
    status = torch.zeros(1, dtype=torch.int32, device=DEV)

    def run_layers(outs, lses):
        for l, bit in enumerate(pattern):
            desc, ws = plans[bit]
            n_sink, n_recent = (64, 512) if bit else (max_ctx, 0)       # N_sink >= M selects the whole context
            B.omni_sparse_mla_decode_sink_recent(desc, qs[l], sparse.kv_cache, sparse.page_table, ctx,
                                                 n_sink, n_recent, outs[l], lses[l], ws, status)

    new = lambda: ([torch.empty((sparse.batch, 128, 512), dtype=torch.bfloat16, device=DEV) for _ in pattern],
                   [torch.empty((sparse.batch, 128), dtype=torch.float32, device=DEV) for _ in pattern])
    eager_out, eager_lse = new()
    run_layers(eager_out, eager_lse)               # also the warm-up: attributes and tensor maps are set up here
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    graph_out, graph_lse = new()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        run_layers(graph_out, graph_lse)
    for o in graph_out:
        o.zero_()
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for l in range(len(pattern)):
        assert torch.equal(graph_out[l], eager_out[l]) and torch.equal(graph_lse[l], eager_lse[l]), l
    # the sparse and the dense layers do differ (the pattern is not ignored)
    assert not torch.equal(eager_out[0], eager_out[1])
    # the replayed results against the oracle: layer 0 on Eq. 2's index set (the workload's own
    # selection lists are that set), layer 1 on the whole context of every request
    keep_q = sparse.q
    sparse.q = qs[0]
    ref_out, ref_lse, _ = oracle_subset(sparse)
    compare(graph_out[0].cpu(), graph_lse[0].cpu(), ref_out, ref_lse, "graph replay, compressed layer")
    dense_idx = torch.arange(max_ctx, dtype=torch.int32, device=DEV).repeat(sparse.batch, 1)
    keep = (sparse.sel_idx, sparse.sel_len, sparse.max_sel)
    sparse.q, sparse.sel_idx, sparse.sel_len = qs[1], dense_idx, ctx.clone()
    ref_out, ref_lse, _ = oracle_subset(sparse)
    compare(graph_out[1].cpu(), graph_lse[1].cpu(), ref_out, ref_lse, "graph replay, uncompressed layer")
    sparse.q, (sparse.sel_idx, sparse.sel_len, sparse.max_sel) = keep_q, keep


def test_topk_producer_and_decode_in_one_cuda_graph_match_eager():
    """scores -> top-k kernel -> decode kernel captured as one graph; replays with new scores follow them."""
    k, ctx_pages = 512, 40
    w = W.config4_topk(DEV, batch=4, ctx_pages=ctx_pages, k=k)
    ctx = ctx_pages * 64
    g = torch.Generator(device=DEV).manual_seed(72)
    scores = torch.randn(w.batch, ctx, generator=g, device=DEV)
    ctx_len = torch.tensor([ctx, ctx - 7, 300, ctx], dtype=torch.int32, device=DEV)
    desc = B.make_desc(w.batch, 128, w.num_pages, w.max_pages_per_req, k, w.scale)
    ws = torch.empty(max(1, B.omni_sparse_mla_workspace_bytes(desc)), dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)

    def chain(sel_idx, sel_len, out, lse):
        B.omni_topk_select(scores, ctx_len, k, sel_idx, sel_len)
        B.omni_sparse_mla_decode(desc, w.q, w.kv_cache, w.page_table, sel_idx, sel_len, out, lse, ws, status)

    def buffers():
        return (torch.zeros(w.batch, k, dtype=torch.int32, device=DEV), torch.zeros(w.batch, dtype=torch.int32, device=DEV),
                torch.empty((w.batch, 128, 512), dtype=torch.bfloat16, device=DEV),
                torch.empty((w.batch, 128), dtype=torch.float32, device=DEV))

    eager = buffers()
    chain(*eager)                                   # also the warm-up
    torch.cuda.synchronize()
    captured = buffers()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        chain(*captured)
    graph.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for a, b in zip(captured, eager):
        assert torch.equal(a, b)
    # new scores in the same buffer: the replay selects and attends accordingly
    scores.copy_(torch.randn(w.batch, ctx, generator=g, device=DEV))
    chain(*eager)
    graph.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for a, b in zip(captured, eager):
        assert torch.equal(a, b)
