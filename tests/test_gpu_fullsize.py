"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The whole batch runs on the GPU; the fp64 oracle recomputes a sample of sequences (all of them
where that takes seconds) from the same pool bits, and the usual tolerance applies to the sampled
rows: max-abs <= 1e-2, rel-L2 <= 2e-3 against the unrounded oracle.  Everything else in the output
must be finite, and the device status word must be clean.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_22788_b200 import api, workloads as wl
from gpu_util import MAX_ABS_TOL, REL_L2_TOL, bf16_tensor, bf16_to_f64, geometry

pytestmark = pytest.mark.gpu

SEED = 0


class SharedPool:
    def __init__(self, num_pages):
        shape = (num_pages, 8, 64, 128)
        self.num_pages = num_pages
        self.k_host = wl.normal_bf16(shape, seed=SEED * 1000 + 2, threads=16)
        self.v_host = wl.normal_bf16(shape, seed=SEED * 1000 + 3, threads=16)
        self.k = bf16_tensor(self.k_host)
        self.v = bf16_tensor(self.v_host)


@pytest.fixture(scope="module")
def pool():
    need = 0
    for lens, ql in ((wl.lens_bulk(SEED), 1), (wl.lens_tail(SEED), 1), (wl.lens_verify(SEED), 17),
                     (wl.lens_mixed(SEED), 1)):
        need = max(need, wl.make_batch("x", lens, q_len=ql, fill=False).num_pages)
    p = SharedPool(need)
    yield p
    del p
    torch.cuda.empty_cache()


def build(name, lens, q_len, pool):
    b = wl.make_batch(name, lens, q_len=q_len, seed=SEED, fill=False, layout="HND")
    b.num_pages = pool.num_pages
    b.q = wl.normal_bf16((b.num_seqs, q_len, 32, 128), seed=SEED * 1000 + 1)
    b.k_pool, b.v_pool = pool.k_host, pool.v_host
    return b


def run_attn(b, pool):
    geom = geometry(b)
    q = bf16_tensor(b.q)
    bt = torch.from_numpy(b.block_table).cuda()
    lens = torch.from_numpy(b.kv_lens).cuda()
    out = torch.full((b.num_seqs, b.q_len, 32, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(api.attn_workspace_bytes(geom), dtype=torch.uint8, device="cuda")
    f = api.ts_verify_attn if b.q_len > 1 else api.ts_decode_attn
    f(geom, q, pool.k, pool.v, bt, lens, out, ws)
    torch.cuda.synchronize()
    assert int(ws[:4].view(torch.int32).item()) == 0
    return out, (geom, q, bt, lens)


def check_sample(out, b, seqs, what):
    g = bf16_to_f64(out)
    assert np.isfinite(g).all(), f"{what}: non-finite output"
    ref, _ = oracle.attention_batch(b, seqs=seqs)
    diff = g[seqs] - ref
    max_abs = float(np.abs(diff).max())
    rel_l2 = float(np.sqrt((diff ** 2).sum() / (ref ** 2).sum()))
    assert max_abs <= MAX_ABS_TOL and rel_l2 <= REL_L2_TOL, f"{what}: max_abs={max_abs:.3e} rel_l2={rel_l2:.3e}"
    # per-sequence too, so that one bad short sequence cannot hide behind long ones
    for i, s in enumerate(seqs):
        r = float(np.sqrt((diff[i] ** 2).sum() / (ref[i] ** 2).sum()))
        assert r <= REL_L2_TOL * 1.15, f"{what}: seq {s} rel_l2={r:.3e}"


def sample(lens, k, rng):
    order = np.argsort(lens)
    picks = {int(order[0]), int(order[-1]), int(order[len(order) // 2])}
    while len(picks) < min(k, len(lens)):
        picks.add(int(rng.integers(0, len(lens))))
    return np.array(sorted(picks))


def test_bulk_full_size(pool):
    lens = wl.lens_bulk(SEED)
    b = build("bulk", lens, 1, pool)
    out, _ = run_attn(b, pool)
    check_sample(out, b, sample(lens, 64, np.random.default_rng(1)), "bulk")
    out2, _ = run_attn(b, pool)
    assert torch.equal(out.view(torch.int16), out2.view(torch.int16))      # bit-reproducible


def test_tail_full_size_both_entry_points(pool):
    lens = wl.lens_tail(SEED)
    b = build("tail", lens, 1, pool)
    out, (geom, q, bt, lens_d) = run_attn(b, pool)
    seqs = np.arange(len(lens))
    check_sample(out, b, seqs, "tail ts_decode_attn")
    S = 256
    po = torch.empty((len(lens), S, 1, 32, 128), dtype=torch.float32, device="cuda")
    pl = torch.empty((len(lens), S, 1, 32), dtype=torch.float32, device="cuda")
    ns = torch.empty((len(lens),), dtype=torch.int32, device="cuda")
    ws = torch.empty(api.splitkv_workspace_bytes(geom), dtype=torch.uint8, device="cuda")
    out2 = torch.full_like(out, float("nan"))
    api.ts_decode_attn_splitkv(geom, q, pool.k, pool.v, bt, lens_d, S, po, pl, ns, ws)
    api.ts_lse_merge(geom, S, po, pl, ns, out2)
    torch.cuda.synchronize()
    assert int(ws[:4].view(torch.int32).item()) == 0
    n = ns.cpu().numpy()
    assert (n > 8).all() and (n <= S).all()          # a handful of long sequences is cut into many pieces
    check_sample(out2, b, seqs, "tail split-KV + merge")


@pytest.mark.parametrize("gamma,k", [(4, 8), (8, 8), (16, 6)])
def test_verify_full_size(pool, gamma, k):
    lens = wl.lens_verify(SEED)
    b = build(f"verify{gamma}", lens, 1 + gamma, pool)
    out, _ = run_attn(b, pool)
    check_sample(out, b, sample(lens, k, np.random.default_rng(gamma)), f"verify gamma={gamma}")


def test_mixed_full_size(pool):
    lens = wl.lens_mixed(SEED)
    assert float(lens.sum()) * 4096 <= 40e9
    b = build("mixed", lens, 1, pool)
    out, _ = run_attn(b, pool)
    check_sample(out, b, sample(lens, 64, np.random.default_rng(2)), "mixed")


def test_sweep_points(pool):
    pool_lens = wl.lens_mixed(SEED)
    for c in (1, 4, 16, 64, 256):
        lens = wl.sweep_subset(pool_lens, c, 0, SEED)
        b = build(f"sweep{c}", lens, 1, pool)
        out, _ = run_attn(b, pool)
        check_sample(out, b, sample(lens, 6, np.random.default_rng(c)), f"sweep c={c}")
