"""Pins for the oracle's attention and merge (CPU only).

The oracle is checked against things other than itself: an independent dense
NumPy implementation on *unpaged* tensors, closed forms, and invariants of
softmax attention.  Each check is chosen so that a plausible slip in the C file
(wrong GQA mapping, off-by-one in the causal mask, transposed stride, dropped
normaliser, wrong page arithmetic) fails at least one of them.
"""
import math

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle
from paper_2608_22788_b200 import workloads as wl


# ----------------------------------------------------------------------------- #
# independent brute force: gather pages to dense arrays, dense masked softmax
# ----------------------------------------------------------------------------- #
def dense_attention(batch):
    B, QL, Hq, D = batch.q.shape
    G = Hq // batch.num_kv_heads
    out = np.zeros((B, QL, Hq, D))
    lse = np.full((B, QL, Hq), -np.inf)
    qf = wl.bf16_bits_to_f32(batch.q).astype(np.float64)
    for s in range(B):
        n = int(batch.kv_lens[s])
        if n == 0:
            continue
        k_bits, v_bits = wl.contiguous_kv(batch, s)
        K = wl.bf16_bits_to_f32(k_bits).astype(np.float64)   # [n, Hkv, D]
        V = wl.bf16_bits_to_f32(v_bits).astype(np.float64)
        for h in range(Hq):
            g = h // G
            S = (qf[s, :, h, :] @ K[:, g, :].T) * batch.scale           # [QL, n]
            key = np.arange(n)[None, :]
            row = np.arange(QL)[:, None]
            visible = key <= (n - QL + row)
            S = np.where(visible, S, -np.inf)
            for t in range(QL):
                if not visible[t].any():
                    continue
                m = S[t].max()
                w = np.exp(S[t] - m)
                out[s, t, h] = (w[:, None] * V[:, g, :]).sum(0) / w.sum()
                lse[s, t, h] = m + math.log(w.sum())
    return out, lse


def test_tiny_config_matches_dense_bruteforce():
    for layout in ("HND", "NHD"):
        b = wl.config_tiny(seed=0, layout=layout)
        o, l = oracle.attention_batch(b)
        ro, rl = dense_attention(b)
        assert np.abs(o - ro).max() <= 1e-12
        assert np.abs(l - rl).max() <= 1e-12


@settings(max_examples=40, deadline=None)
@given(B=st.integers(1, 4), P=st.sampled_from([1, 4, 16]), G=st.sampled_from([1, 2, 4]),
       Hkv=st.integers(1, 2), D=st.sampled_from([8, 64]), QL=st.integers(1, 5),
       layout=st.sampled_from(["HND", "NHD"]), seed=st.integers(0, 10_000), data=st.data())
def test_random_shapes_match_dense_bruteforce(B, P, G, Hkv, D, QL, layout, seed, data):
    lens = data.draw(st.lists(st.integers(QL, 70), min_size=B, max_size=B))
    b = wl.make_batch("h", lens, q_len=QL, num_q_heads=G * Hkv, num_kv_heads=Hkv, head_dim=D,
                      page_size=P, seed=seed, layout=layout, spare_frac=0.3, extra_table_cols=2)
    o, l = oracle.attention_batch(b)
    ro, rl = dense_attention(b)
    assert np.abs(o - ro).max() <= 1e-12
    assert np.abs(l - rl).max() <= 1e-12


# ----------------------------------------------------------------------------- #
# closed forms
# ----------------------------------------------------------------------------- #
def test_two_key_closed_form():
    # q = (1, 0), k0 = (0, 0), k1 = (1, 0), scale = ln 2  ->  scores (0, ln 2),
    # weights (1/3, 2/3): O = (v0 + 2 v1) / 3 and LSE = ln 3.
    b = wl.make_batch("cf", [2], num_q_heads=1, num_kv_heads=1, head_dim=2, page_size=1, seed=3,
                      scale=math.log(2.0))
    b.q[:] = wl.f32_to_bf16_bits(np.array([1.0, 0.0], np.float32)).reshape(1, 1, 1, 2)
    p0, p1 = int(b.block_table[0, 0]), int(b.block_table[0, 1])
    b.k_pool[p0] = wl.f32_to_bf16_bits(np.zeros(2, np.float32)).reshape(1, 1, 2)
    b.k_pool[p1] = wl.f32_to_bf16_bits(np.array([1.0, 0.0], np.float32)).reshape(1, 1, 2)
    v0 = wl.bf16_bits_to_f32(b.v_pool[p0]).astype(np.float64).reshape(2)
    v1 = wl.bf16_bits_to_f32(b.v_pool[p1]).astype(np.float64).reshape(2)
    o, l = oracle.attention_batch(b)
    assert np.allclose(o.reshape(2), (v0 + 2.0 * v1) / 3.0, rtol=0, atol=1e-15)
    assert abs(l.reshape(()) - math.log(3.0)) <= 1e-15


def test_length_one_returns_v_exactly():
    b = wl.make_batch("n1", [1, 1, 1], num_q_heads=4, num_kv_heads=2, head_dim=16, page_size=4, seed=5)
    o, l = oracle.attention_batch(b)
    qf = wl.bf16_bits_to_f32(b.q).astype(np.float64)
    for s in range(3):
        k, v = wl.contiguous_kv(b, s)
        kf = wl.bf16_bits_to_f32(k).astype(np.float64)
        vf = wl.bf16_bits_to_f32(v).astype(np.float64)
        for h in range(4):
            g = h // 2
            assert np.array_equal(o[s, 0, h], vf[0, g])          # exactly v_0
            assert abs(l[s, 0, h] - b.scale * float(qf[s, 0, h] @ kf[0, g])) <= 1e-14


def _set_all_keys(b, value_bits_row):
    """Overwrite every K row with the same D-vector (uint16 bits)."""
    b.k_pool[...] = value_bits_row.reshape((1, 1, 1, -1))


def test_identical_keys_give_mean_of_v_and_lse_plus_log_n():
    lens = [5, 33, 64]
    b = wl.make_batch("same", lens, num_q_heads=4, num_kv_heads=2, head_dim=8, page_size=4, seed=6,
                      layout="NHD")
    krow = wl.normal_bf16((8,), seed=99)
    _set_all_keys(b, krow)
    o, l = oracle.attention_batch(b)
    qf = wl.bf16_bits_to_f32(b.q).astype(np.float64)
    kf = wl.bf16_bits_to_f32(krow).astype(np.float64)
    for s, n in enumerate(lens):
        _, v = wl.contiguous_kv(b, s)
        vf = wl.bf16_bits_to_f32(v).astype(np.float64)
        for h in range(4):
            assert np.abs(o[s, 0, h] - vf[:, h // 2].mean(0)).max() <= 1e-14
            x = b.scale * float(qf[s, 0, h] @ kf)
            assert abs(l[s, 0, h] - (x + math.log(n))) <= 1e-13


@pytest.mark.parametrize("mode", ["zero_q", "zero_scale"])
def test_uniform_weights_give_mean_of_v(mode):
    lens = [7, 40]
    b = wl.make_batch("u", lens, num_q_heads=2, num_kv_heads=1, head_dim=8, page_size=16, seed=8,
                      scale=0.0 if mode == "zero_scale" else None)
    if mode == "zero_q":
        b.q[...] = 0
    o, l = oracle.attention_batch(b)
    for s, n in enumerate(lens):
        _, v = wl.contiguous_kv(b, s)
        vf = wl.bf16_bits_to_f32(v).astype(np.float64)
        for h in range(2):
            assert np.abs(o[s, 0, h] - vf[:, 0].mean(0)).max() <= 1e-14
            assert abs(l[s, 0, h] - math.log(n)) <= 1e-14


def test_dominant_key_selects_its_value():
    n, J = 50, 37
    b = wl.make_batch("dom", [n], num_q_heads=1, num_kv_heads=1, head_dim=4, page_size=8, seed=9, scale=1.0)
    b.q[...] = wl.f32_to_bf16_bits(np.array([8.0, 0, 0, 0], np.float32)).reshape(1, 1, 1, 4)
    b.k_pool[...] = 0
    page, off = int(b.block_table[0, J // 8]), J % 8
    b.k_pool[page, 0, off] = wl.f32_to_bf16_bits(np.array([8.0, 0, 0, 0], np.float32))
    o, l = oracle.attention_batch(b)
    _, v = wl.contiguous_kv(b, 0)
    vf = wl.bf16_bits_to_f32(v).astype(np.float64)
    # the other 49 keys carry weight e^-64 each
    assert np.abs(o[0, 0, 0] - vf[J, 0]).max() <= 1e-15
    assert abs(l[0, 0, 0] - 64.0) <= 1e-12


# ----------------------------------------------------------------------------- #
# invariants
# ----------------------------------------------------------------------------- #
def test_page_permutation_is_bitwise_invisible():
    b1 = wl.make_batch("p", [19, 70, 33], q_len=2, num_q_heads=4, num_kv_heads=2, head_dim=16,
                       page_size=8, seed=12, spare_frac=0.5)
    o1, l1 = oracle.attention_batch(b1)
    rng = np.random.default_rng(77)
    perm = rng.permutation(b1.num_pages)            # new physical id of old page i is perm[i]
    k2 = np.empty_like(b1.k_pool)
    v2 = np.empty_like(b1.v_pool)
    k2[perm] = b1.k_pool
    v2[perm] = b1.v_pool
    bt2 = perm[b1.block_table].astype(np.int32)
    o2, l2 = oracle.paged_attention(b1.q, k2, v2, bt2, b1.kv_lens, num_kv_heads=2, page_size=8,
                                    kv_page_stride=b1.kv_page_stride, kv_token_stride=b1.kv_token_stride,
                                    kv_head_stride=b1.kv_head_stride, scale=b1.scale)
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)


def test_layouts_agree_bitwise():
    a = wl.make_batch("l", [23, 64, 5], q_len=3, num_q_heads=6, num_kv_heads=3, head_dim=8,
                      page_size=8, seed=21, layout="HND")
    b = wl.make_batch("l", [23, 64, 5], q_len=3, num_q_heads=6, num_kv_heads=3, head_dim=8,
                      page_size=8, seed=21, layout="NHD")
    b.k_pool = np.ascontiguousarray(np.transpose(a.k_pool, (0, 2, 1, 3)))
    b.v_pool = np.ascontiguousarray(np.transpose(a.v_pool, (0, 2, 1, 3)))
    oa, la = oracle.attention_batch(a)
    ob, lb = oracle.attention_batch(b)
    assert np.array_equal(oa, ob) and np.array_equal(la, lb)


def test_poisoned_unused_memory_is_never_read():
    clean = wl.make_batch("c", [17, 64, 200, 513, 1], q_len=2, num_q_heads=8, num_kv_heads=2,
                          head_dim=16, page_size=16, seed=4, spare_frac=0.3, extra_table_cols=3)
    dirty = wl.make_batch("c", [17, 64, 200, 513, 1], q_len=2, num_q_heads=8, num_kv_heads=2,
                          head_dim=16, page_size=16, seed=4, spare_frac=0.3, extra_table_cols=3,
                          poison=True)
    # -1 table slots would crash or read out of bounds if touched; NaN would spread
    oc, lc = oracle.attention_batch(clean)
    od, ld = oracle.attention_batch(dirty)
    assert np.isfinite(od).all() and not np.isnan(ld).any()
    assert np.array_equal(oc, od) and np.array_equal(lc, ld)


def test_verify_row_equals_single_token_decode_on_truncated_cache():
    QL = 5
    lens = np.array([9, 40, 131], np.int32)
    b = wl.make_batch("v", lens, q_len=QL, num_q_heads=4, num_kv_heads=2, head_dim=16, page_size=16, seed=31)
    o, l = oracle.attention_batch(b)
    for t in range(QL):
        d = wl.make_batch("v", lens, q_len=QL, num_q_heads=4, num_kv_heads=2, head_dim=16, page_size=16, seed=31)
        d.q = np.ascontiguousarray(b.q[:, t:t + 1])
        d.kv_lens = (lens - QL + t + 1).astype(np.int32)
        d.q_len = 1
        od, ld = oracle.attention_batch(d)
        assert np.array_equal(od[:, 0], o[:, t])          # exact, not approximate
        assert np.array_equal(ld[:, 0], l[:, t])


def test_first_draft_row_with_no_context_sees_one_key():
    # kv_len == q_len: row t sees keys 0..t; row 0 sees exactly key 0 -> O = v_0.
    b = wl.make_batch("nc", [4], q_len=4, num_q_heads=2, num_kv_heads=1, head_dim=8, page_size=2, seed=41)
    o, _ = oracle.attention_batch(b)
    _, v = wl.contiguous_kv(b, 0)
    vf = wl.bf16_bits_to_f32(v).astype(np.float64)
    assert np.array_equal(o[0, 0, 0], vf[0, 0]) and np.array_equal(o[0, 0, 1], vf[0, 0])


def test_empty_sequence_gives_zeros_and_minus_inf():
    b = wl.make_batch("e", [0, 5], num_q_heads=2, num_kv_heads=1, head_dim=8, page_size=4, seed=2)
    o, l = oracle.attention_batch(b)
    assert np.array_equal(o[0], np.zeros_like(o[0])) and np.isneginf(l[0]).all()
    assert np.isfinite(l[1]).all()


# ----------------------------------------------------------------------------- #
# split partials and their merge
# ----------------------------------------------------------------------------- #
def _partials(b, cuts_per_seq, S):
    """Oracle partials over contiguous key ranges given by per-sequence cut lists."""
    B, QL, Hq, D = b.q.shape
    po = np.zeros((B, S, QL * Hq, D))
    pl = np.full((B, S, QL * Hq), -np.inf)
    ns = np.zeros(B, np.int32)
    for i in range(S):
        kb = np.array([c[i] if i < len(c) - 1 else 0 for c in cuts_per_seq], np.int32)
        ke = np.array([c[i + 1] if i < len(c) - 1 else 0 for c in cuts_per_seq], np.int32)
        o, l = oracle.attention_batch(b, key_begin=kb, key_end=ke)
        po[:, i] = o.reshape(B, QL * Hq, D)
        pl[:, i] = l.reshape(B, QL * Hq)
    for s, c in enumerate(cuts_per_seq):
        ns[s] = len(c) - 1
    return po, pl, ns


@pytest.mark.parametrize("QL", [1, 4])
def test_merge_of_any_partition_equals_unsplit(QL):
    lens = [QL + 0, 33, 64, 257]
    b = wl.make_batch("m", lens, q_len=QL, num_q_heads=4, num_kv_heads=2, head_dim=16, page_size=16, seed=51)
    full_o, full_l = oracle.attention_batch(b)
    rng = np.random.default_rng(5)
    S = 7
    for trial in range(6):
        cuts = []
        for n in lens:
            k = int(rng.integers(1, S + 1))
            inner = np.sort(rng.integers(0, n + 1, size=k - 1))     # repeats -> empty parts
            cuts.append([0, *inner.tolist(), n])
        po, pl, ns = _partials(b, cuts, S)
        mo, ml = oracle.lse_merge(po, pl, ns)
        B, _, Hq, D = b.q.shape
        assert np.abs(mo.reshape(full_o.shape) - full_o).max() <= 1e-12
        assert np.abs(ml.reshape(full_l.shape) - full_l).max() <= 1e-12


def test_merge_closed_form_and_empty_parts():
    # two parts with LSE ln 1 and ln 3 -> weights 1/4, 3/4; a third, empty part is ignored
    po = np.zeros((1, 3, 1, 2))
    po[0, 0, 0] = [4.0, 0.0]
    po[0, 1, 0] = [0.0, 8.0]
    po[0, 2, 0] = [np.nan, np.nan]        # must not leak: its weight is exactly zero
    pl = np.array([[[0.0], [math.log(3.0)], [-np.inf]]])
    o, l = oracle.lse_merge(po, pl, np.array([3], np.int32))
    assert np.allclose(o[0, 0], [1.0, 6.0], rtol=0, atol=1e-15)
    assert abs(l[0, 0] - math.log(4.0)) <= 1e-15
    o, l = oracle.lse_merge(po, np.full((1, 3, 1), -np.inf), np.array([3], np.int32))
    assert np.array_equal(o, np.zeros_like(o)) and np.isneginf(l).all()
    o, l = oracle.lse_merge(po, pl, np.array([0], np.int32))
    assert np.array_equal(o, np.zeros_like(o)) and np.isneginf(l).all()
