"""ts_kv_append: the new tokens' K/V rows land bit-exactly where attention will read them."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_22788_b200 import api, workloads as wl
from gpu_util import DeviceBatch, assert_close, bf16_tensor

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("layout,P,D,ql", [("HND", 64, 128, 1), ("NHD", 16, 64, 3), ("HND", 128, 128, 5), ("NHD", 32, 128, 17)])
def test_append_then_attend(layout, P, D, ql):
    lens = np.array([ql, 40, 700, 131, 64, 65], np.int32) + np.array([0, ql, ql, ql, ql, ql], np.int32)
    b = wl.make_batch("ap", lens, q_len=ql, num_q_heads=8, num_kv_heads=2, head_dim=D, page_size=P, seed=3, layout=layout)
    ref, _ = oracle.attention_batch(b)                     # with the complete cache
    # plain definition of the append on the host: remember the new rows, then wipe them from the pools
    B = len(lens)
    new_k = np.zeros((B, ql, 2, D), np.uint16)
    new_v = np.zeros((B, ql, 2, D), np.uint16)
    want_k, want_v = b.k_pool.copy(), b.v_pool.copy()
    for s in range(B):
        for t in range(ql):
            pos = int(lens[s]) - ql + t
            page, off = int(b.block_table[s, pos // P]), pos % P
            for pool, new in ((b.k_pool, new_k), (b.v_pool, new_v)):
                row = pool[page, :, off, :] if layout == "HND" else pool[page, off, :, :]
                new[s, t] = row
                row[...] = 0x7FC0                      # NaN until appended
    d = DeviceBatch(b)
    api.ts_kv_append(d.geom, bf16_tensor(new_k), bf16_tensor(new_v), d.k, d.v, d.bt, d.lens)
    torch.cuda.synchronize()
    got_k = d.k.view(torch.int16).cpu().numpy().view(np.uint16)
    got_v = d.v.view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(got_k, want_k) and np.array_equal(got_v, want_v)      # bit-exact, nothing else touched
    out = d.verify() if ql > 1 else d.decode()
    assert_close(out, ref, "attention after append")
