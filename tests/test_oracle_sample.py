"""Pins for the oracle's stochastic (temperature / top-k / top-p) lossless acceptance (CPU only)."""
import math

import numpy as np
import pytest

import oracle
from paper_2608_22788_b200 import workloads as wl


def _bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, np.float32))


def filtered_distribution(row_f64, temperature, top_k, top_p):
    """Independent NumPy version of steps 1-3: returns (ids in order, probabilities)."""
    v = np.asarray(row_f64, np.float64)
    idx = np.arange(len(v))
    ok = ~np.isnan(v)
    order = sorted(idx[ok], key=lambda i: (-v[i], i))[:top_k]
    z = np.array([v[i] for i in order]) / temperature
    p = np.exp(z - z.max()) if len(z) else z
    p = p / p.sum() if len(z) else p
    keep = int(np.searchsorted(np.cumsum(p), top_p - 1e-300, side="left")) + 1 if len(p) else 0
    keep = min(keep, len(p))
    p = p[:keep] / p[:keep].sum() if keep else p[:0]
    return list(order[:keep]), p


def brute_accept(logits_bits, draft, u, temperature, top_k, top_p):
    f = wl.bf16_bits_to_f32(logits_bits).astype(np.float64)
    B, R, V = f.shape
    gamma = R - 1
    acc = np.zeros(B, np.int32)
    out = np.full((B, R), -1, np.int32)
    for b in range(B):
        for i in range(R):
            ids, p = filtered_distribution(f[b, i], temperature, top_k, top_p)
            if i < gamma:
                x = int(draft[b, i])
                px = p[ids.index(x)] if x in ids else 0.0
                if u[b, i, 0] < px:
                    out[b, i] = x
                    acc[b] += 1
                    continue
                rest = [(t, q) for t, q in zip(ids, p) if t != x]
            else:
                rest = list(zip(ids, p))
            total = sum(q for _, q in rest)
            cum, y = 0.0, -1
            for t, q in rest:
                cum += q
                y = t
                if cum > u[b, i, 1] * total:
                    break
            out[b, i] = y
            break
    return acc, out


@pytest.mark.parametrize("seed", range(6))
def test_matches_numpy_bruteforce(seed):
    rng = np.random.default_rng(seed)
    B, gamma, V = 5, 4, 200
    logits = wl.make_logits(B, gamma, V, seed=seed)
    best = np.argmax(wl.bf16_bits_to_f32(logits), -1)
    draft = np.where(rng.random((B, gamma)) < 0.7, best[:, :gamma], rng.integers(0, V, (B, gamma))).astype(np.int32)
    u = rng.random((B, gamma + 1, 2))
    T, k, pnuc = [(0.7, 20, 0.8), (1.0, 5, 0.95), (0.3, 20, 1.0), (2.0, 50, 0.5), (0.7, 1, 0.8), (0.7, 20, 0.8)][seed]
    acc, out, ids, pp = oracle.accept_sample(logits, draft, u, temperature=T, top_k=k, top_p=pnuc)
    racc, rout = brute_accept(logits, draft, u, T, k, pnuc)
    assert np.array_equal(acc, racc) and np.array_equal(out, rout)
    f = wl.bf16_bits_to_f32(logits).astype(np.float64)
    for b in range(B):
        for i in range(gamma + 1):
            rid, rp = filtered_distribution(f[b, i], T, k, pnuc)
            assert ids[b, i, :len(rid)].tolist() == rid and (ids[b, i, len(rid):] == -1).all()
            assert np.abs(pp[b, i, :len(rid)] - rp).max() <= 1e-14
            assert abs(pp[b, i].sum() - 1.0) <= 1e-14


def test_closed_form_two_to_one_distribution():
    # logits (1, 0, 0) with temperature 1/ln 2  ->  p = (1/2, 1/4, 1/4)
    T = 1.0 / math.log(2.0)
    logits = _bits(np.array([[[1.0, 0.0, 0.0], [1.0, 0.0, 0.0]]]))         # gamma = 1
    _, _, ids, pp = oracle.accept_sample(logits, [[0]], np.zeros((1, 2, 2)), temperature=T, top_k=3, top_p=1.0)
    assert ids[0, 0].tolist() == [0, 1, 2] and np.allclose(pp[0, 0], [0.5, 0.25, 0.25], rtol=0, atol=1e-15)

    def run(draft, ua, us, **kw):
        u = np.array([[[ua, us], [0.0, us]]])
        acc, out, _, _ = oracle.accept_sample(logits, [[draft]], u, temperature=T, top_k=3, **kw)
        return int(acc[0]), out[0].tolist()

    assert run(0, 0.499, 0.9, top_p=1.0) == (1, [0, 2])        # accepted, bonus from (1/2,1/4,1/4) at 0.9 -> token 2
    assert run(0, 0.501, 0.4, top_p=1.0) == (0, [1, -1])       # rejected: residual (1/2, 1/2) over tokens 1, 2
    assert run(0, 0.501, 0.6, top_p=1.0) == (0, [2, -1])
    assert run(1, 0.249, 0.6, top_p=1.0) == (1, [1, 1])        # bonus: cumulative 0.5, 0.75 -> 0.6 picks token 1
    assert run(1, 0.251, 0.6, top_p=1.0) == (0, [0, -1])       # residual (2/3, 1/3) over tokens 0, 2
    assert run(1, 0.251, 0.7, top_p=1.0) == (0, [2, -1])
    # nucleus 0.7: keep tokens 0 and 1 (the tie between 1 and 2 goes to the lower index), renormalised (2/3, 1/3)
    _, _, ids, pp = oracle.accept_sample(logits, [[0]], np.zeros((1, 2, 2)), temperature=T, top_k=3, top_p=0.7)
    assert ids[0, 0].tolist() == [0, 1, -1] and np.allclose(pp[0, 0], [2 / 3, 1 / 3, 0], rtol=0, atol=1e-15)
    assert run(2, 0.0, 0.5, top_p=0.7) == (0, [0, -1])         # a draft outside the nucleus is always rejected
    assert run(1, 0.33, 0.9, top_p=0.7) == (1, [1, 1])


def test_output_distribution_equals_target_distribution():
    # losslessness: integrate over a fine lattice of (u_accept, u_sample); whatever the draft token,
    # the emitted token follows p exactly
    rng = np.random.default_rng(1)
    V, N = 7, 400
    x = rng.standard_normal((1, 2, V)).astype(np.float32) * 2
    logits = _bits(x)
    T, k, pnuc = 0.7, 5, 0.9
    ids, p = filtered_distribution(wl.bf16_bits_to_f32(logits)[0, 0].astype(np.float64), T, k, pnuc)
    grid = (np.arange(N) + 0.5) / N
    ua, us = np.meshgrid(grid, grid, indexing="ij")
    u = np.zeros((N * N, 2, 2))
    u[:, 0, 0], u[:, 0, 1] = ua.ravel(), us.ravel()
    big = np.broadcast_to(logits, (N * N, 2, V)).copy()
    for draft_tok in (ids[0], ids[-1], int(np.argmin(x[0, 0]))):
        acc, out, _, _ = oracle.accept_sample(big, np.full((N * N, 1), draft_tok), u, temperature=T, top_k=k, top_p=pnuc)
        freq = np.bincount(out[:, 0], minlength=V) / (N * N)
        want = np.zeros(V)
        want[ids] = p
        assert np.abs(freq - want).max() <= 2.5 / N


def test_top_k_one_or_tiny_nucleus_is_greedy():
    B, gamma, V = 6, 5, 3000
    logits = wl.make_logits(B, gamma, V, seed=9)
    best, _, _ = oracle.accept_greedy(logits, np.zeros((B, gamma), np.int32))
    draft, cut = wl.make_draft(best, V, seed=9)
    gt, ga, go = oracle.accept_greedy(logits, draft)
    u = np.random.default_rng(0).random((B, gamma + 1, 2))
    for kw in (dict(temperature=0.7, top_k=1, top_p=0.8), dict(temperature=1.3, top_k=20, top_p=1e-9),
               dict(temperature=1e-3, top_k=20, top_p=0.999)):
        acc, out, _, _ = oracle.accept_sample(logits, draft, u, **kw)
        assert np.array_equal(acc, ga) and np.array_equal(out, go)


def test_nan_never_a_candidate_and_masked_vocabulary():
    x = np.full((1, 1, 10), -np.inf, np.float32)
    x[0, 0, 3] = np.nan
    x[0, 0, 7] = 1.0
    x[0, 0, 8] = 1.0
    acc, out, ids, pp = oracle.accept_sample(_bits(x), np.zeros((1, 0), np.int32), np.array([[[0.0, 0.75]]]),
                                             temperature=1.0, top_k=4, top_p=1.0)
    assert ids[0, 0, :2].tolist() == [7, 8] and 3 not in ids[0, 0]
    assert np.allclose(pp[0, 0, :2], [0.5, 0.5]) and np.allclose(pp[0, 0, 2:], 0)
    assert out[0, 0] == 8 and acc[0] == 0


# ------------------------------------------------------------------------------------------------
# presence penalty
# ------------------------------------------------------------------------------------------------
def _bitmap(B, V, tokens_per_seq):
    bm = np.zeros((B, (V + 7) // 8), np.uint8)
    for b, toks in enumerate(tokens_per_seq):
        for v in toks:
            bm[b, v >> 3] |= np.uint8(1 << (v & 7))
    return bm


@pytest.mark.parametrize("seed", range(4))
def test_presence_penalty_equals_plain_run_on_prepenalised_logits(seed):
    # logits on a grid of halves and a penalty of 1.5: every penalised value is again a bf16 number, so the
    # penalised call must equal the plain call on logits lowered beforehand, row by row, with row i also
    # lowering the drafts 0 .. i-1 (built here with NumPy, independently of the oracle's own loop)
    rng = np.random.default_rng(100 + seed)
    B, gamma, V = 4, 3, 160
    grid = (rng.integers(-24, 25, (B, gamma + 1, V)) * 0.5).astype(np.float32)
    logits = _bits(grid)
    draft = rng.integers(0, V, (B, gamma)).astype(np.int32)
    draft[0, 1] = draft[0, 0]                                   # a repeated draft is penalised once
    seen_tokens = [sorted(set(rng.integers(0, V, 30).tolist())) for _ in range(B)]
    seen_tokens[1].append(int(draft[1, 0]))                     # seen and drafted: still penalised once
    bm = _bitmap(B, V, seen_tokens)
    u = rng.random((B, gamma + 1, 2))
    T, k, pnuc, pen = 0.7, 20, 0.8, 1.5
    got = oracle.accept_sample(logits, draft, u, temperature=T, top_k=k, top_p=pnuc, seen=bm, presence_penalty=pen)
    lowered = grid.copy()
    for b in range(B):
        for i in range(gamma + 1):
            present = set(seen_tokens[b]) | set(int(x) for x in draft[b, :i])
            for v in present:
                lowered[b, i, v] -= pen
    assert np.array_equal(wl.bf16_bits_to_f32(_bits(lowered)), lowered)       # exactly representable
    want = oracle.accept_sample(_bits(lowered), draft, u, temperature=T, top_k=k, top_p=pnuc)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    racc, rout = brute_accept(_bits(lowered), draft, u, T, k, pnuc)
    assert np.array_equal(got[0], racc) and np.array_equal(got[1], rout)


def test_presence_penalty_zero_or_nothing_present_changes_nothing():
    rng = np.random.default_rng(7)
    B, gamma, V = 3, 0, 500
    logits = wl.make_logits(B, gamma, V, seed=9)
    draft = np.zeros((B, 0), np.int32)
    u = rng.random((B, 1, 2))
    base = oracle.accept_sample(logits, draft, u, temperature=0.7, top_k=20, top_p=0.8)
    bm = _bitmap(B, V, [[1, 2, 3]] * B)
    same = oracle.accept_sample(logits, draft, u, temperature=0.7, top_k=20, top_p=0.8, seen=bm, presence_penalty=0.0)
    empty = oracle.accept_sample(logits, draft, u, temperature=0.7, top_k=20, top_p=0.8,
                                 seen=np.zeros_like(bm), presence_penalty=1.5)
    for a, b_, c in zip(base, same, empty):
        assert np.array_equal(a, b_) and np.array_equal(a, c)


def test_large_presence_penalty_removes_seen_tokens_from_the_kept_set():
    rng = np.random.default_rng(8)
    B, gamma, V = 2, 2, 300
    logits = wl.make_logits(B, gamma, V, seed=10)
    f = wl.bf16_bits_to_f32(logits)
    top = np.argsort(-f, axis=-1)[..., :5]                      # the five best tokens of every row
    seen_tokens = [sorted(set(top[b].reshape(-1).tolist())) for b in range(B)]
    bm = _bitmap(B, V, seen_tokens)
    draft = top[:, :gamma, 0].astype(np.int32)
    u = rng.random((B, gamma + 1, 2))
    acc, out, ids, pp = oracle.accept_sample(logits, draft, u, temperature=0.7, top_k=20, top_p=0.8,
                                             seen=bm, presence_penalty=1000.0)
    for b in range(B):
        kept = set(ids[b][ids[b] >= 0].tolist())
        assert not (kept & set(seen_tokens[b]))
        assert acc[b] == 0                                      # the drafts are seen tokens: never kept, rejected


# ------------------------------------------------------------------ sampled drafts (general proposal q)
def brute_accept_q(logits_bits, draft, u, q, temperature, top_k, top_p):
    """The general rule written independently: accept with probability min(1, p/q), else draw from
    norm(max(0, p - q)) over the whole vocabulary (dense vectors, no kept-slot bookkeeping)."""
    f = wl.bf16_bits_to_f32(logits_bits).astype(np.float64)
    B, R, V = f.shape
    gamma = R - 1
    acc = np.zeros(B, np.int32)
    out = np.full((B, R), -1, np.int32)
    for b in range(B):
        for i in range(R):
            ids, pk = filtered_distribution(f[b, i], temperature, top_k, top_p)
            p = np.zeros(V)
            p[ids] = pk
            if i < gamma:
                x = int(draft[b, i])
                qv = q[b, i].astype(np.float64)
                if u[b, i, 0] * qv[x] < p[x]:
                    out[b, i] = x
                    acc[b] += 1
                    continue
                w = np.maximum(p - qv, 0.0)
                if not w.sum() > 0:
                    w = p
            else:
                w = p
            order = [t for t in ids if w[t] > 0]            # inverse CDF runs in the kept order
            total = sum(w[t] for t in order)
            cum, y = 0.0, -1
            for t in order:
                cum += w[t]
                y = t
                if cum > u[b, i, 1] * total:
                    break
            out[b, i] = y
            break
    return acc, out


def _random_q(rng, B, gamma, V, logits, sharp):
    """Proposal distributions loosely correlated with the target: softmax of the logits plus noise."""
    f = wl.bf16_bits_to_f32(logits)[:, :gamma].astype(np.float64)
    z = sharp * f + rng.standard_normal((B, gamma, V))
    z -= z.max(-1, keepdims=True)
    q = np.exp(z)
    q /= q.sum(-1, keepdims=True)
    return q.astype(np.float32)


def _draw(rng, q):
    B, gamma, V = q.shape
    d = np.zeros((B, gamma), np.int32)
    for b in range(B):
        for i in range(gamma):
            pr = q[b, i].astype(np.float64)
            d[b, i] = rng.choice(V, p=pr / pr.sum())
    return d


@pytest.mark.parametrize("seed", range(6))
def test_sampled_drafts_match_numpy_bruteforce(seed):
    rng = np.random.default_rng(100 + seed)
    B, gamma, V = 6, 4, 160
    logits = wl.make_logits(B, gamma, V, seed=seed)
    q = _random_q(rng, B, gamma, V, logits, sharp=[1.4, 0.5, 2.5, 1.0, 1.4, 0.0][seed])
    draft = _draw(rng, q)
    u = rng.random((B, gamma + 1, 2))
    T, k, pnuc = [(0.7, 20, 0.8), (1.0, 5, 0.95), (0.3, 20, 1.0), (2.0, 50, 0.5), (0.7, 1, 0.8), (0.7, 20, 0.8)][seed]
    acc, out, _, _ = oracle.accept_sample(logits, draft, u, temperature=T, top_k=k, top_p=pnuc, draft_probs=q)
    racc, rout = brute_accept_q(logits, draft, u, q, T, k, pnuc)
    assert np.array_equal(acc, racc) and np.array_equal(out, rout)
    assert acc.max() > 0 or seed == 5


def test_one_hot_proposal_is_the_point_proposal_rule():
    rng = np.random.default_rng(7)
    B, gamma, V = 12, 5, 700
    logits = wl.make_logits(B, gamma, V, seed=3)
    best = np.argmax(wl.bf16_bits_to_f32(logits), -1)
    draft = np.where(rng.random((B, gamma)) < 0.7, best[:, :gamma], rng.integers(0, V, (B, gamma))).astype(np.int32)
    q = np.zeros((B, gamma, V), np.float32)
    np.put_along_axis(q, draft[..., None].astype(np.int64), 1.0, axis=-1)
    u = rng.random((B, gamma + 1, 2))
    kw = dict(temperature=0.7, top_k=20, top_p=0.8)
    a0, o0, _, _ = oracle.accept_sample(logits, draft, u, **kw)
    a1, o1, _, _ = oracle.accept_sample(logits, draft, u, draft_probs=q, **kw)
    assert np.array_equal(a0, a1) and np.array_equal(o0, o1)
    assert a0.min() < gamma and a0.max() > 0


def test_sampled_draft_closed_form():
    # p = (1/2, 1/4, 1/4) as above; q = (1/4, 1/2, 1/4)
    T = 1.0 / math.log(2.0)
    logits = _bits(np.array([[[1.0, 0.0, 0.0], [1.0, 0.0, 0.0]]]))
    q = np.array([[[0.25, 0.5, 0.25]]], np.float32)

    def run(draft, ua, us):
        u = np.array([[[ua, us], [0.0, us]]])
        acc, out, _, _ = oracle.accept_sample(logits, [[draft]], u, temperature=T, top_k=3, top_p=1.0, draft_probs=q)
        return int(acc[0]), out[0].tolist()

    assert run(0, 0.999, 0.1) == (1, [0, 0])        # p/q = 2: always accepted; bonus token 0 at 0.1
    assert run(2, 0.999, 0.6) == (1, [2, 1])        # p/q = 1: accepted for every u < 1
    assert run(1, 0.499, 0.8) == (1, [1, 2])        # p/q = 1/2: accepted below 1/2 ...
    assert run(1, 0.501, 0.0) == (0, [0, -1])       # ... rejected above; max(0, p - q) = (1/4, 0, 0): token 0
    assert run(1, 0.501, 0.999) == (0, [0, -1])


def test_proposal_equal_to_target_is_always_accepted():
    rng = np.random.default_rng(9)
    B, gamma, V = 8, 6, 300
    logits = wl.make_logits(B, gamma, V, seed=9)
    f = wl.bf16_bits_to_f32(logits).astype(np.float64)
    q = np.zeros((B, gamma, V), np.float32)
    # temperature 1 and powers of two would make p exact in float32; in general q = float32(p) differs
    # from p by rounding, so u is kept away from 1
    for b in range(B):
        for i in range(gamma):
            ids, p = filtered_distribution(f[b, i], 0.7, 20, 0.8)
            q[b, i, ids] = p
    draft = _draw(rng, q)
    u = rng.random((B, gamma + 1, 2)) * 0.999
    acc, out, _, _ = oracle.accept_sample(logits, draft, u, temperature=0.7, top_k=20, top_p=0.8, draft_probs=q)
    assert (acc == gamma).all() and np.array_equal(out[:, :gamma], draft)


def test_sampled_drafts_are_lossless():
    # sum over draft tokens x of q(x) * P(emit y | draft x) = p(y): the lattice over (u_accept, u_sample)
    # integrates the inner probability, the sum over x is exact
    rng = np.random.default_rng(4)
    V, N = 6, 300
    x = rng.standard_normal((1, 2, V)).astype(np.float32) * 2
    logits = _bits(x)
    T, k, pnuc = 0.9, 4, 0.95
    ids, p = filtered_distribution(wl.bf16_bits_to_f32(logits)[0, 0].astype(np.float64), T, k, pnuc)
    want = np.zeros(V)
    want[ids] = p
    qv = rng.dirichlet(np.ones(V)).astype(np.float32)
    grid = (np.arange(N) + 0.5) / N
    ua, us = np.meshgrid(grid, grid, indexing="ij")
    u = np.zeros((N * N, 2, 2))
    u[:, 0, 0], u[:, 0, 1] = ua.ravel(), us.ravel()
    big = np.broadcast_to(logits, (N * N, 2, V)).copy()
    qq = np.broadcast_to(qv, (N * N, 1, V)).copy()
    mix = np.zeros(V)
    rejected_somewhere = False
    for tok in range(V):
        acc, out, _, _ = oracle.accept_sample(big, np.full((N * N, 1), tok), u, temperature=T, top_k=k, top_p=pnuc,
                                              draft_probs=qq)
        rejected_somewhere |= bool((acc == 0).any())
        mix += float(qv[tok]) * np.bincount(out[:, 0], minlength=V) / (N * N)
    assert rejected_somewhere
    assert np.abs(mix - want).max() <= 2.5 / N


def test_unnormalised_proposal_above_target_falls_back_to_the_target():
    # q = 2 p is not a distribution; a rejection then leaves no positive residual and the token comes from p
    T = 1.0 / math.log(2.0)
    logits = _bits(np.array([[[1.0, 0.0, 0.0], [1.0, 0.0, 0.0]]]))
    q = np.array([[[1.0, 0.5, 0.5]]], np.float32)
    u = np.array([[[0.9, 0.6], [0.0, 0.0]]])
    acc, out, _, _ = oracle.accept_sample(logits, [[0]], u, temperature=T, top_k=3, top_p=1.0, draft_probs=q)
    assert int(acc[0]) == 0 and out[0].tolist() == [1, -1]      # cumulative (1/2, 3/4, 1): 0.6 picks token 1
