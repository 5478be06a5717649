"""The decode step inside a CUDA graph.

The paper's rollout engine replays full-batch CUDA graphs and avoids ragged query lengths because
they would break that (Section 3.4).  The library is built for it: a call is a fixed sequence of
launches whose grids do not depend on the lengths (the planner runs on the device), it allocates
nothing and never synchronises.  This test captures attention + greedy selection once and replays
the graph after the lengths, block table, queries and logits have been overwritten in place.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_22788_b200 import api, workloads as wl
from gpu_util import DeviceBatch, assert_close, bf16_tensor

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("ql", [1, 5])
def test_capture_once_replay_with_new_lengths(ql):
    kw = dict(q_len=ql, num_q_heads=8, num_kv_heads=2, head_dim=128, page_size=64, layout="HND")
    lens_a = np.array([300, 1000, 77, 2100, 64, 5], np.int32) + ql
    lens_b = np.array([2100, 64, 900, 31, 1500, 700], np.int32) + ql
    a = wl.make_batch("a", lens_a, seed=1, extra_table_cols=40, **kw)
    b = wl.make_batch("b", lens_b, seed=2, extra_table_cols=40, **kw)
    # one device pool large enough for both batches, one block table of a common width
    pages = max(a.num_pages, b.num_pages)
    width = max(a.max_pages_per_seq, b.max_pages_per_seq)
    for x in (a, b):
        pad = np.zeros((x.num_seqs, width), np.int32)
        pad[:, :x.max_pages_per_seq] = x.block_table
        x.block_table, x.max_pages_per_seq = pad, width
        k = np.zeros((pages,) + x.k_pool.shape[1:], np.uint16); k[:x.num_pages] = x.k_pool
        v = np.zeros((pages,) + x.v_pool.shape[1:], np.uint16); v[:x.num_pages] = x.v_pool
        x.k_pool, x.v_pool, x.num_pages = k, v, pages
    d = DeviceBatch(a)
    V, B = 4096, a.num_seqs
    logits_a = wl.make_logits(B, 0, V, seed=3)
    logits_b = wl.make_logits(B, 0, V, seed=4)
    lg = bf16_tensor(logits_a)
    tgt = torch.empty((B, 1), dtype=torch.int32, device="cuda")
    acc = torch.empty((B,), dtype=torch.int32, device="cuda")
    tok = torch.empty((B, 1), dtype=torch.int32, device="cuda")
    ws2 = torch.empty(api.accept_workspace_bytes(B, 0, V), dtype=torch.uint8, device="cuda")
    attn = api.ts_verify_attn if ql > 1 else api.ts_decode_attn

    def step():
        attn(d.geom, d.q, d.k, d.v, d.bt, d.lens, d.out, d.ws)
        api.ts_accept_greedy(lg, None, tgt, acc, tok, ws2)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()                                  # first calls before capture (one-time attribute set-up)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()

    for batch, logits in ((a, logits_a), (b, logits_b), (a, logits_a)):
        d.q.copy_(bf16_tensor(batch.q)); d.k.copy_(bf16_tensor(batch.k_pool)); d.v.copy_(bf16_tensor(batch.v_pool))
        d.bt.copy_(torch.from_numpy(batch.block_table).cuda()); d.lens.copy_(torch.from_numpy(batch.kv_lens).cuda())
        lg.copy_(bf16_tensor(logits))
        d.out.fill_(float("nan")); tgt.fill_(-1)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert d.status() == 0
        ref, _ = oracle.attention_batch(batch)
        assert_close(d.out, ref, "graph replay")
        rt, _, _ = oracle.accept_greedy(logits, np.zeros((B, 0), np.int32))
        assert np.array_equal(tgt.cpu().numpy(), rt)
