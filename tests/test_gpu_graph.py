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


def test_whole_verify_step_in_one_graph():
    """Rotary append, verify attention and penalised stochastic acceptance captured together; the replay runs
    on new lengths, rows, drafts, uniforms and bitmap.  The append is checked through what attention then
    reads: the oracle attends over a host cache into which the oracle's own rotated rows were written."""
    ql, Hq, Hkv, D, P, V = 5, 8, 2, 128, 64, 4096
    gamma, B = ql - 1, 5
    f = (1.0e4 ** (-np.arange(0, D, 2, dtype=np.float64) / D)).astype(np.float32)

    def host_case(seed, lens):
        b = wl.make_batch("g", lens, q_len=ql, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, page_size=P, seed=seed,
                          layout="HND", extra_table_cols=40)
        rng = np.random.default_rng(seed)
        q_raw = wl.normal_bf16((B, ql, Hq, D), seed=seed + 1)
        k_raw = wl.normal_bf16((B, ql, Hkv, D), seed=seed + 2)
        v_new = wl.normal_bf16((B, ql, Hkv, D), seed=seed + 3)
        pos = (b.kv_lens[:, None].astype(np.int64) - ql + np.arange(ql)[None, :]).reshape(-1)
        q_rot = wl.f32_to_bf16_bits(oracle.rope(q_raw.reshape(B * ql, Hq, D), pos, f).astype(np.float32)).reshape(B, ql, Hq, D)
        k_rot = wl.f32_to_bf16_bits(oracle.rope(k_raw.reshape(B * ql, Hkv, D), pos, f).astype(np.float32)).reshape(B, ql, Hkv, D)
        ref_cache = wl.make_batch("g", lens, q_len=ql, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, page_size=P,
                                  seed=seed, layout="HND", extra_table_cols=40)
        for s in range(B):
            for t in range(ql):
                p_ = int(b.kv_lens[s]) - ql + t
                pg, off = int(b.block_table[s, p_ // P]), p_ % P
                ref_cache.k_pool[pg, :, off, :] = k_rot[s, t]
                ref_cache.v_pool[pg, :, off, :] = v_new[s, t]
                b.k_pool[pg, :, off, :] = 0x7FC0            # the device cache starts without the new rows
                b.v_pool[pg, :, off, :] = 0x7FC0
        ref_cache.q = q_rot
        logits = wl.make_logits(B, gamma, V, seed=seed + 4)
        best = np.argmax(wl.bf16_bits_to_f32(logits), -1)
        draft = np.where(rng.random((B, gamma)) < 0.7, best[:, :gamma], rng.integers(0, V, (B, gamma))).astype(np.int32)
        u = rng.random((B, gamma + 1, 2), dtype=np.float32)
        seen = np.packbits(rng.random((B, V)) < 0.05, axis=1, bitorder="little")
        return dict(b=b, ref=ref_cache, q_raw=q_raw, k_raw=k_raw, v_new=v_new, logits=logits, draft=draft, u=u, seen=seen)

    ca = host_case(11, np.array([300, 1000, 77, 2100, 64], np.int32) + ql)
    cb = host_case(12, np.array([2100, 64, 900, 31, 1500], np.int32) + ql)
    pages = max(ca["b"].num_pages, cb["b"].num_pages)
    width = max(ca["b"].max_pages_per_seq, cb["b"].max_pages_per_seq)
    for c in (ca, cb):
        for x in (c["b"], c["ref"]):
            pad = np.zeros((B, width), np.int32); pad[:, :x.max_pages_per_seq] = x.block_table
            x.block_table, x.max_pages_per_seq = pad, width
            k = np.zeros((pages,) + x.k_pool.shape[1:], np.uint16); k[:x.num_pages] = x.k_pool
            v = np.zeros((pages,) + x.v_pool.shape[1:], np.uint16); v[:x.num_pages] = x.v_pool
            x.k_pool, x.v_pool, x.num_pages = k, v, pages
    d = DeviceBatch(ca["b"])
    q_raw, k_raw, v_new = bf16_tensor(ca["q_raw"]), bf16_tensor(ca["k_raw"]), bf16_tensor(ca["v_new"])
    d_f = torch.from_numpy(f).cuda()
    lg = bf16_tensor(ca["logits"])
    dr = torch.from_numpy(ca["draft"]).cuda()
    uu = torch.from_numpy(ca["u"]).cuda()
    seen = torch.from_numpy(ca["seen"]).cuda()
    acc = torch.empty((B,), dtype=torch.int32, device="cuda")
    tok = torch.empty((B, gamma + 1), dtype=torch.int32, device="cuda")
    ws2 = torch.empty(api.sample_workspace_bytes(B, gamma, V, 20), dtype=torch.uint8, device="cuda")

    def step():
        api.ts_rope_kv_append(d.geom, q_raw, d.q, k_raw, v_new, d.k, d.v, d.bt, d.lens, d_f)
        api.ts_verify_attn(d.geom, d.q, d.k, d.v, d.bt, d.lens, d.out, d.ws)
        api.ts_accept_sample(lg, dr, uu, acc, tok, ws2, temperature=0.7, top_k=20, top_p=0.8, presence_penalty=1.5, seen=seen)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()

    for c in (ca, cb, ca):
        b = c["b"]
        d.k.copy_(bf16_tensor(b.k_pool)); d.v.copy_(bf16_tensor(b.v_pool))
        d.bt.copy_(torch.from_numpy(b.block_table).cuda()); d.lens.copy_(torch.from_numpy(b.kv_lens).cuda())
        q_raw.copy_(bf16_tensor(c["q_raw"])); k_raw.copy_(bf16_tensor(c["k_raw"])); v_new.copy_(bf16_tensor(c["v_new"]))
        lg.copy_(bf16_tensor(c["logits"])); dr.copy_(torch.from_numpy(c["draft"]).cuda())
        uu.copy_(torch.from_numpy(c["u"]).cuda()); seen.copy_(torch.from_numpy(c["seen"]).cuda())
        d.out.fill_(float("nan")); acc.fill_(-9); tok.fill_(-9)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert d.status() == 0
        ref, _ = oracle.attention_batch(c["ref"])
        # the device rotates in fp32 and the oracle in fp64: a few rotated elements land one bf16 step apart,
        # which the attention tolerance absorbs
        assert_close(d.out, ref, "graph replay: append + verify attention")
        racc, rout, _, _ = oracle.accept_sample(c["logits"], c["draft"], c["u"].astype(np.float64), temperature=0.7,
                                                top_k=20, top_p=0.8, seen=c["seen"], presence_penalty=1.5)
        assert np.array_equal(acc.cpu().numpy(), racc) and np.array_equal(tok.cpu().numpy(), rout)
