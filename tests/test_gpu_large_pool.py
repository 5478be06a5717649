"""Addressing beyond 2^31 elements: a KV pool of 5.2 GB per tensor, sequences living in its last pages.

An HBM-sized cache holds far more than 2^31 bf16 elements per pool, so page offsets must be 64-bit
everywhere (tensor-map strides, the append kernels).  The device pools are allocated whole and zeroed;
only the pages the batch uses are filled, from a compact host pool on which the oracle runs with the
block table renumbered.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_22788_b200 import api, workloads as wl
from gpu_util import MAX_ABS_TOL, REL_L2_TOL, bf16_tensor, bf16_to_f64

pytestmark = pytest.mark.gpu

NUM_PAGES = 40000            # x 8 heads x 64 tokens x 128 dims = 2.62e9 elements (> 2^31) per pool
HKV, P, D, HQ = 8, 64, 128, 32


def _free_enough():
    free, _ = torch.cuda.mem_get_info()
    return free > 14 * (1 << 30)


@pytest.mark.parametrize("q_len", [1, 5])
def test_attention_and_append_in_the_last_pages_of_a_large_pool(q_len):
    if not _free_enough():
        pytest.skip("needs 14 GB of free device memory")
    rng = np.random.default_rng(3 + q_len)
    lens = np.array([q_len, 70, 1000, 3001, 64, 2500], np.int32) + q_len
    B = len(lens)
    npg = (lens + P - 1) // P
    used = int(npg.sum())
    # physical pages: the top of the pool, shuffled; the very last page is in use
    phys = (NUM_PAGES - 1 - rng.permutation(used)).astype(np.int32)
    assert int(phys.min()) * HKV * P * D > 2 ** 31
    max_pages = int(npg.max())
    bt_phys = np.zeros((B, max_pages), np.int32)
    bt_comp = np.zeros((B, max_pages), np.int32)
    o = 0
    for s in range(B):
        bt_phys[s, :npg[s]] = phys[o:o + npg[s]]
        bt_comp[s, :npg[s]] = np.arange(o, o + npg[s])
        o += npg[s]
    k_comp = wl.normal_bf16((used, HKV, P, D), seed=41)
    v_comp = wl.normal_bf16((used, HKV, P, D), seed=42)
    q = wl.normal_bf16((B, q_len, HQ, D), seed=43)
    scale = 1.0 / np.sqrt(D)

    dk = torch.zeros((NUM_PAGES, HKV, P, D), dtype=torch.bfloat16, device="cuda")
    dv = torch.zeros_like(dk)
    idx = torch.from_numpy(phys.astype(np.int64)).cuda()
    dk[idx] = bf16_tensor(k_comp)
    dv[idx] = bf16_tensor(v_comp)

    # the step's new rows are wiped on the device and put back by ts_kv_append
    new_k = np.zeros((B, q_len, HKV, D), np.uint16)
    new_v = np.zeros((B, q_len, HKV, D), np.uint16)
    for s in range(B):
        for t in range(q_len):
            pos = int(lens[s]) - q_len + t
            new_k[s, t] = k_comp[bt_comp[s, pos // P], :, pos % P, :]
            new_v[s, t] = v_comp[bt_comp[s, pos // P], :, pos % P, :]
            dk[int(bt_phys[s, pos // P]), :, pos % P, :] = float("nan")
            dv[int(bt_phys[s, pos // P]), :, pos % P, :] = float("nan")
    ps, ts_, hs = HKV * P * D, D, P * D
    geom = api.AttnGeometry(B, q_len, HQ, HKV, D, P, NUM_PAGES, max_pages, ps, ts_, hs, scale)
    d_bt, d_lens = torch.from_numpy(bt_phys).cuda(), torch.from_numpy(lens).cuda()
    api.ts_kv_append(geom, bf16_tensor(new_k), bf16_tensor(new_v), dk, dv, d_bt, d_lens)

    dq = bf16_tensor(q)
    out = torch.full((B, q_len, HQ, D), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(api.attn_workspace_bytes(geom), dtype=torch.uint8, device="cuda")
    f = api.ts_verify_attn if q_len > 1 else api.ts_decode_attn
    f(geom, dq, dk, dv, d_bt, d_lens, out, ws)
    torch.cuda.synchronize()
    assert int(ws[:4].view(torch.int32).item()) == 0

    ref, _ = oracle.paged_attention(q, k_comp, v_comp, bt_comp, lens, num_kv_heads=HKV, page_size=P,
                                    kv_page_stride=ps, kv_token_stride=ts_, kv_head_stride=hs, scale=scale)
    got = bf16_to_f64(out)
    diff = got - ref
    assert np.isfinite(got).all()
    assert float(np.abs(diff).max()) <= MAX_ABS_TOL
    assert float(np.sqrt((diff ** 2).sum() / (ref ** 2).sum())) <= REL_L2_TOL

    # the explicit split-KV entry point over the same pool
    S = 8
    po = torch.empty((B, S, q_len, HQ, D), dtype=torch.float32, device="cuda")
    pl = torch.empty((B, S, q_len, HQ), dtype=torch.float32, device="cuda")
    ns = torch.empty((B,), dtype=torch.int32, device="cuda")
    ws2 = torch.empty(api.splitkv_workspace_bytes(geom), dtype=torch.uint8, device="cuda")
    out2 = torch.full_like(out, float("nan"))
    api.ts_decode_attn_splitkv(geom, dq, dk, dv, d_bt, d_lens, S, po, pl, ns, ws2)
    api.ts_lse_merge(geom, S, po, pl, ns, out2)
    torch.cuda.synchronize()
    assert int(ws2[:4].view(torch.int32).item()) == 0
    diff2 = bf16_to_f64(out2) - ref
    assert float(np.abs(diff2).max()) <= MAX_ABS_TOL
    assert float(np.sqrt((diff2 ** 2).sum() / (ref ** 2).sum())) <= REL_L2_TOL
    del dk, dv
    torch.cuda.empty_cache()
