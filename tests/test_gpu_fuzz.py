"""Seeded random geometries against the oracle: every supported head_dim, page size, pool layout, query-head
ratio and draft depth in combination, with ragged lengths around tile and page boundaries, through the three
attention entry points.  The shapes are drawn from a fixed seed, so the test is deterministic."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_22788_b200 import api, workloads as wl
from gpu_util import DeviceBatch, assert_close

pytestmark = pytest.mark.gpu


def _cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        D = int(rng.choice([64, 128]))
        P = int(rng.choice([16, 32, 64, 128]))
        hkv = int(rng.choice([1, 2, 4]))
        G = int(rng.choice([1, 2, 3, 4, 5, 7, 8]))
        ql = int(rng.choice([1, 1, 1, 2, 3, 4, 5, 6, 8, 9, 12, 16, 17]))
        rows = G * ql
        if rows > (128 if D == 128 else 96):
            continue
        B = int(rng.integers(1, 7))
        kinds = rng.integers(0, 5, B)
        lens = []
        for k in kinds:
            if k == 0:
                lens.append(int(rng.integers(0, 4)))                       # empty or shorter than the draft block
            elif k == 1:
                lens.append(int(rng.choice([63, 64, 65, 127, 128, 129, 191, 192, 193])))
            elif k == 2:
                lens.append(int(rng.integers(1, 300)))
            elif k == 3:
                lens.append(int(rng.integers(300, 2500)))
            else:
                lens.append(int(rng.choice([P - 1, P, P + 1, 4 * P, 4 * P + 1])))
        layout = str(rng.choice(["HND", "NHD"]))
        out.append((lens, ql, G * hkv, hkv, D, P, layout))
    return out


CASES = _cases(48, seed=20260801)


@pytest.mark.parametrize("case", CASES, ids=[str(i) for i in range(len(CASES))])
def test_random_geometry(case):
    lens, ql, hq, hkv, D, P, layout = case
    b = wl.make_batch("fz", lens, q_len=ql, num_q_heads=hq, num_kv_heads=hkv, head_dim=D, page_size=P,
                      seed=sum(lens) + 31 * ql + hq, layout=layout, poison=True, spare_frac=0.3, extra_table_cols=2)
    ref, _ = oracle.attention_batch(b)
    d = DeviceBatch(b)
    out = d.verify() if ql > 1 else d.decode()
    assert_close(out, ref, f"direct {case}")
    S = 1 + (sum(lens) + ql) % 7
    d.out.fill_(float("nan"))
    d.splitkv(S)                      # partials, then ts_lse_merge into d.out
    assert_close(d.out, ref, f"split-KV max_splits={S} {case}")
