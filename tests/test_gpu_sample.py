"""GPU parity of ts_accept_sample against the oracle.

Token selection (top-k with ties to the lower index) is exact.  Probabilities are fp32 on the GPU
and fp64 in the oracle, so a decision is only required to agree when the uniform is not within
1e-5 of the probability (or cumulative probability) it is compared with; the test computes those
margins from the oracle's own distributions and treats a sequence with such a near-tie before its
first divergence as undecided.  With seeded uniforms that essentially never happens.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_22788_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu
MARGIN = 1e-5


def run_gpu(logits_bits, draft, u32, T, k, pnuc, seen=None, pen=0.0, q=None):
    B, R, V = logits_bits.shape
    gamma = R - 1
    lg = torch.from_numpy(np.ascontiguousarray(logits_bits).view(np.int16)).cuda().view(torch.bfloat16)
    dr = torch.from_numpy(np.ascontiguousarray(draft, dtype=np.int32).reshape(B, gamma)).cuda()
    uu = torch.from_numpy(np.ascontiguousarray(u32, dtype=np.float32)).cuda()
    acc = torch.full((B,), -5, dtype=torch.int32, device="cuda")
    out = torch.full((B, R), -5, dtype=torch.int32, device="cuda")
    ws = torch.empty(api.sample_workspace_bytes(B, gamma, V, k), dtype=torch.uint8, device="cuda")
    sd = torch.from_numpy(np.ascontiguousarray(seen)).cuda() if seen is not None else None
    qd = torch.from_numpy(np.ascontiguousarray(q, dtype=np.float32)).cuda() if q is not None else None
    api.ts_accept_sample(lg, dr, uu, acc, out, ws, temperature=T, top_k=k, top_p=pnuc, presence_penalty=pen, seen=sd,
                         draft_probs=qd)
    torch.cuda.synchronize()
    return acc.cpu().numpy(), out.cpu().numpy()


def near_tie(b, i, draft, u, ids, pp, gamma, pnuc, q=None):
    """True if some comparison at row (b, i) is within MARGIN in the oracle's arithmetic."""
    p = pp[b, i]
    kept = ids[b, i] >= 0
    ua, us = u[b, i]
    if q is not None and i < gamma:
        # sampled draft: u_accept * q(x) against p(x), then the inverse CDF over max(0, p - q); the fp32
        # differences p - q carry an absolute error of a few 1e-7, whatever their size
        x = int(draft[b, i])
        qv = q[b, i].astype(np.float64)
        px = p[ids[b, i] == x].sum()
        if abs(ua * qv[x] - px) < MARGIN:
            return True
        r = np.where(kept, np.maximum(p - qv[np.maximum(ids[b, i], 0)], 0.0), 0.0)
        if (np.abs(np.where(kept, p - qv[np.maximum(ids[b, i], 0)], 1.0)) < 1e-6).any():
            return True                                  # a slot on the edge of the residual's support
        tot = r.sum()
        if tot > 0 and (np.abs(np.cumsum(r) - us * tot) < 4e-6).any():
            return True
        return False
    # nucleus boundary (needs the unrenormalised cumulative sums: recompute is overkill; use a proxy:
    # the kept mass before renormalisation cannot be told from here, so only flag exact-looking cases)
    if i < gamma:
        x = draft[b, i]
        px = p[ids[b, i] == x].sum()
        if abs(ua - px) < MARGIN:
            return True
        skip = ids[b, i] == x
    else:
        skip = np.zeros_like(kept)
    w = np.where(kept & ~skip, p, 0.0)
    tot = w.sum()
    if tot > 0 and (np.abs(np.cumsum(w) / tot - us) < MARGIN).any():
        return True
    return False


def check(logits_bits, draft, u32, T, k, pnuc, seen=None, pen=0.0, q=None):
    B, R, V = logits_bits.shape
    gamma = R - 1
    u = np.asarray(u32, np.float32)
    racc, rout, ids, pp = oracle.accept_sample(logits_bits, draft, u.astype(np.float64), temperature=T, top_k=k, top_p=pnuc,
                                               seen=seen, presence_penalty=pen, draft_probs=q)
    gacc, gout = run_gpu(logits_bits, draft, u, T, k, pnuc, seen, pen, q)
    undecided = 0
    for b in range(B):
        if gacc[b] == racc[b] and np.array_equal(gout[b], rout[b]):
            continue
        last = min(int(racc[b]), int(gacc[b]))
        if any(near_tie(b, i, np.asarray(draft).reshape(B, gamma), u, ids, pp, gamma, pnuc, q) for i in range(last + 1)):
            undecided += 1
            continue
        raise AssertionError(f"sequence {b}: gpu accept {gacc[b]} tokens {gout[b]} vs oracle {racc[b]} {rout[b]}")
    assert undecided <= max(1, B // 50)
    return racc, rout


@pytest.mark.parametrize("gamma", [0, 4, 16])
def test_paper_sampling_regime_full_vocab(gamma):
    B, V = 16, wl.VOCAB
    rng = np.random.default_rng(gamma)
    logits = wl.make_logits(B, gamma, V, seed=30 + gamma)
    best = np.argmax(wl.bf16_bits_to_f32(logits), -1)
    draft = np.where(rng.random((B, gamma)) < 0.8, best[:, :gamma], rng.integers(0, V, (B, gamma))).astype(np.int32)
    u = rng.random((B, gamma + 1, 2), dtype=np.float32)
    acc, out = check(logits, draft, u, 0.7, 20, 0.8)
    assert (acc >= 0).all() and (acc <= gamma).all()
    if gamma:
        assert acc.max() > 0 and acc.min() < gamma          # both outcomes occur


@pytest.mark.parametrize("cfg", [(1.0, 5, 0.95), (0.3, 32, 1.0), (2.0, 32, 0.5), (0.7, 1, 0.8), (1.5, 20, 0.3)])
def test_other_parameters_and_small_vocab(cfg):
    T, k, pnuc = cfg
    B, gamma, V = 40, 3, 4096
    rng = np.random.default_rng(int(T * 10) + k)
    logits = wl.make_logits(B, gamma, V, seed=k)
    best = np.argmax(wl.bf16_bits_to_f32(logits), -1)
    draft = np.where(rng.random((B, gamma)) < 0.6, best[:, :gamma], rng.integers(0, V, (B, gamma))).astype(np.int32)
    u = rng.random((B, gamma + 1, 2), dtype=np.float32)
    check(logits, draft, u, T, k, pnuc)


def test_ties_constant_rows_and_masked_vocabulary():
    V = 65536
    x = np.random.default_rng(0).standard_normal((4, 1, V)).astype(np.float32)
    x[0, 0, :] = 1.25                               # constant row: top-k = indices 0..k-1 (slow exact path)
    x[1, 0, :] = -np.inf
    x[1, 0, [77, 40000]] = 3.0                      # two finite tokens only
    x[2, 0, 1000:1040] = 9.0                        # 40 equal maxima, more than top_k
    x[3, 0, ::2] = np.nan                           # NaN never selected
    bits = wl.f32_to_bf16_bits(x)
    u = np.random.default_rng(1).random((4, 1, 2), dtype=np.float32)
    _, out = check(bits, np.zeros((4, 0), np.int32), u, 1.0, 20, 1.0)
    assert 0 <= out[0, 0] < 20 and out[1, 0] in (77, 40000) and 1000 <= out[2, 0] < 1020 and out[3, 0] % 2 == 1


def test_greedy_limit_matches_ts_accept_greedy():
    B, gamma, V = 16, 8, 32768
    logits = wl.make_logits(B, gamma, V, seed=5)
    best, _, _ = oracle.accept_greedy(logits, np.zeros((B, gamma), np.int32))
    draft, cut = wl.make_draft(best, V, seed=5)
    _, ga, go = oracle.accept_greedy(logits, draft)
    u = np.random.default_rng(2).random((B, gamma + 1, 2), dtype=np.float32)
    acc, out = run_gpu(logits, draft, u, 0.7, 1, 0.8)
    assert np.array_equal(acc, ga) and np.array_equal(out, go) and np.array_equal(acc, cut)


def test_argument_errors():
    lg = torch.zeros((2, 1, 64), dtype=torch.bfloat16, device="cuda")
    u = torch.zeros((2, 1, 2), dtype=torch.float32, device="cuda")
    acc = torch.zeros((2,), dtype=torch.int32, device="cuda")
    out = torch.zeros((2, 1), dtype=torch.int32, device="cuda")
    ws = torch.empty(4096 * 16, dtype=torch.uint8, device="cuda")
    for kw, err in ((dict(temperature=0.0, top_k=20, top_p=0.8), "TS_ERR_INVALID_ARG"),
                    (dict(temperature=0.7, top_k=33, top_p=0.8), "TS_ERR_UNSUPPORTED"),
                    (dict(temperature=0.7, top_k=20, top_p=0.0), "TS_ERR_INVALID_ARG")):
        with pytest.raises(api.TailSieveError, match=err):
            api.ts_accept_sample(lg, None, u, acc, out, ws, **kw)


# ------------------------------------------------------------------------------------------------
# presence penalty
# ------------------------------------------------------------------------------------------------
def _bitmap(B, V, rng, density, stride=None):
    nbytes = (V + 7) // 8
    stride = stride or nbytes
    bm = np.zeros((B, stride), np.uint8)
    bits = rng.random((B, V)) < density
    bm[:, :nbytes] = np.packbits(bits, axis=1, bitorder="little")[:, :nbytes]
    return bm


@pytest.mark.parametrize("gamma,density", [(0, 0.1), (4, 0.1), (16, 0.02), (8, 0.5)])
def test_presence_penalty_paper_regime_full_vocab(gamma, density):
    # the paper's sampling table: temperature 0.7, top-k 20, top-p 0.8, presence penalty 1.5
    B, V = 16, wl.VOCAB
    rng = np.random.default_rng(50 + gamma)
    logits = wl.make_logits(B, gamma, V, seed=60 + gamma)
    f = wl.bf16_bits_to_f32(logits)
    best = np.argmax(f, -1)
    draft = np.where(rng.random((B, gamma)) < 0.8, best[:, :gamma], rng.integers(0, V, (B, gamma))).astype(np.int32)
    if gamma >= 2:
        draft[0, 1] = draft[0, 0]                    # a repeated draft: row 2 of sequence 0 sees it once
    seen = _bitmap(B, V, rng, density, stride=(V + 7) // 8 + 16)
    # make sure the penalty matters: the best tokens of half of the rows are marked as seen
    for b in range(0, B, 2):
        for v in best[b]:
            seen[b, v >> 3] |= np.uint8(1 << (v & 7))
    u = rng.random((B, gamma + 1, 2), dtype=np.float32)
    acc, out = check(logits, draft, u, 0.7, 20, 0.8, seen=seen, pen=1.5)
    plain_acc, plain_out, _, _ = oracle.accept_sample(logits, draft, u.astype(np.float64), temperature=0.7, top_k=20, top_p=0.8)
    assert not (np.array_equal(acc, plain_acc) and np.array_equal(out, plain_out))     # the penalty changed something


def test_presence_penalty_without_bitmap_counts_the_earlier_drafts():
    B, gamma, V = 24, 6, 8192
    rng = np.random.default_rng(77)
    logits = wl.make_logits(B, gamma, V, seed=78)
    best = np.argmax(wl.bf16_bits_to_f32(logits), -1)
    draft = best[:, :gamma].astype(np.int32).copy()
    draft[:, 1:] = draft[:, :1]                      # the same token drafted again and again
    logits[:, :, :] = logits[:, :1, :]               # and the same distribution at every position
    u = rng.random((B, gamma + 1, 2), dtype=np.float32)
    check(logits, draft, u, 0.7, 20, 0.8, seen=None, pen=4.0)


def test_presence_penalty_ties_negative_penalty_and_slow_path():
    # constant rows (thousands of ties, the exact fallback path) with a few seen tokens, a negative penalty
    # (a bonus: seen tokens move up), and -inf / NaN logits that a penalty must leave alone
    B, gamma, V = 6, 2, 40000
    rng = np.random.default_rng(5)
    base = np.zeros((B, gamma + 1, V), np.float32)
    base[1] = -3.0
    base[2, :, ::2] = -np.inf
    base[3, :, 5] = np.nan
    base[4] = rng.integers(-4, 5, (gamma + 1, V)).astype(np.float32)
    base[5] = 1.0
    logits = wl.f32_to_bf16_bits(base)
    seen = _bitmap(B, V, rng, 0.001)
    for b in range(B):
        for v in (0, 1, 5, 9, V - 1):
            seen[b, v >> 3] |= np.uint8(1 << (v & 7))
    draft = rng.integers(0, 16, (B, gamma)).astype(np.int32)
    u = rng.random((B, gamma + 1, 2), dtype=np.float32)
    check(logits, draft, u, 0.7, 20, 0.8, seen=seen, pen=1.5)
    check(logits, draft, u, 1.0, 8, 1.0, seen=seen, pen=-2.25)


def test_presence_penalty_argument_errors():
    B, V = 2, 4096
    lg = torch.zeros((B, 1, V), dtype=torch.bfloat16, device="cuda")
    u = torch.zeros((B, 1, 2), dtype=torch.float32, device="cuda")
    acc = torch.zeros((B,), dtype=torch.int32, device="cuda")
    out = torch.zeros((B, 1), dtype=torch.int32, device="cuda")
    ws = torch.empty(api.sample_workspace_bytes(B, 0, V, 20), dtype=torch.uint8, device="cuda")
    short = torch.zeros((B, V // 8 - 1), dtype=torch.uint8, device="cuda")
    with pytest.raises(api.TailSieveError):
        api.ts_accept_sample(lg, None, u, acc, out, ws, temperature=0.7, top_k=20, top_p=0.8, presence_penalty=1.5, seen=short)
    with pytest.raises(api.TailSieveError):
        api.ts_accept_sample(lg, None, u, acc, out, ws, temperature=0.7, top_k=20, top_p=0.8, presence_penalty=float("nan"))


# ------------------------------------------------------------------ sampled drafts (proposal distribution q)
def _proposal(rng, logits, gamma, sharp):
    """q = softmax(sharp * logits + noise) per draft position, float32, and one draw from each."""
    f = wl.bf16_bits_to_f32(logits)[:, :gamma].astype(np.float32)
    z = sharp * f + rng.standard_normal(f.shape, dtype=np.float32)
    z -= z.max(-1, keepdims=True)
    q = np.exp(z)
    q /= q.sum(-1, keepdims=True)
    B, _, V = q.shape
    c = np.cumsum(q.astype(np.float64), -1)
    draws = rng.random((B, gamma, 1)) * c[..., -1:]
    draft = np.minimum((c < draws).sum(-1), V - 1).astype(np.int32)
    return q.astype(np.float32), draft


@pytest.mark.parametrize("gamma", [4, 16])
def test_sampled_drafts_full_vocab(gamma):
    B, V = 16, wl.VOCAB
    rng = np.random.default_rng(50 + gamma)
    logits = wl.make_logits(B, gamma, V, seed=60 + gamma)
    q, draft = _proposal(rng, logits, gamma, sharp=1.0 / 0.7)
    u = rng.random((B, gamma + 1, 2), dtype=np.float32)
    acc, out = check(logits, draft, u, 0.7, 20, 0.8, q=q)
    assert acc.max() > 0 and acc.min() < gamma


@pytest.mark.parametrize("cfg", [(1.0, 5, 0.95, 1.0), (0.3, 32, 1.0, 2.0), (2.0, 32, 0.5, 0.3), (0.7, 1, 0.8, 1.4), (0.7, 20, 0.8, 0.0)])
def test_sampled_drafts_other_parameters(cfg):
    T, k, pnuc, sharp = cfg
    B, gamma, V = 48, 3, 4096
    rng = np.random.default_rng(int(T * 10) + k + 7)
    logits = wl.make_logits(B, gamma, V, seed=k + 1)
    q, draft = _proposal(rng, logits, gamma, sharp)
    u = rng.random((B, gamma + 1, 2), dtype=np.float32)
    check(logits, draft, u, T, k, pnuc, q=q)


def test_one_hot_proposal_gives_the_point_proposal_results():
    B, gamma, V = 16, 8, 32768
    rng = np.random.default_rng(8)
    logits = wl.make_logits(B, gamma, V, seed=8)
    best = np.argmax(wl.bf16_bits_to_f32(logits), -1)
    draft = np.where(rng.random((B, gamma)) < 0.8, best[:, :gamma], rng.integers(0, V, (B, gamma))).astype(np.int32)
    q = np.zeros((B, gamma, V), np.float32)
    np.put_along_axis(q, draft[..., None].astype(np.int64), 1.0, axis=-1)
    u = rng.random((B, gamma + 1, 2), dtype=np.float32)
    a0, o0 = run_gpu(logits, draft, u, 0.7, 20, 0.8)
    a1, o1 = run_gpu(logits, draft, u, 0.7, 20, 0.8, q=q)
    assert np.array_equal(a0, a1) and np.array_equal(o0, o1)


def test_sampled_drafts_with_the_presence_penalty():
    B, gamma, V = 24, 5, 8192
    rng = np.random.default_rng(12)
    logits = wl.make_logits(B, gamma, V, seed=12)
    q, draft = _proposal(rng, logits, gamma, sharp=1.4)
    seen = rng.integers(0, 256, (B, V // 8), dtype=np.uint8) & rng.integers(0, 256, (B, V // 8), dtype=np.uint8)
    u = rng.random((B, gamma + 1, 2), dtype=np.float32)
    check(logits, draft, u, 0.7, 20, 0.8, seen=seen, pen=1.5, q=q)


def test_proposal_equal_to_target_accepts_everything_and_out_of_range_draft_is_rejected():
    B, gamma, V = 8, 4, 2048
    rng = np.random.default_rng(3)
    logits = wl.make_logits(B, gamma, V, seed=3)
    u = rng.random((B, gamma + 1, 2), dtype=np.float32) * 0.99
    _, _, ids, pp = oracle.accept_sample(logits, np.zeros((B, gamma), np.int32), u.astype(np.float64), temperature=0.7,
                                         top_k=20, top_p=0.8)
    q = np.zeros((B, gamma, V), np.float32)
    draft = np.zeros((B, gamma), np.int32)
    for b in range(B):
        for i in range(gamma):
            kept = ids[b, i] >= 0
            q[b, i, ids[b, i][kept]] = pp[b, i][kept]
            draft[b, i] = ids[b, i][rng.integers(0, kept.sum())]
    acc, out = run_gpu(logits, draft, u, 0.7, 20, 0.8, q=q)
    assert (acc == gamma).all() and np.array_equal(out[:, :gamma], draft)
    bad = draft.copy()
    bad[:, 1] = V + 5
    acc, out = run_gpu(logits, bad, u, 0.7, 20, 0.8, q=q)
    assert (acc == 1).all() and (out[:, 1] >= 0).all() and (out[:, 1] < V).all() and (out[:, 2:] == -1).all()


@pytest.mark.parametrize("with_q", [False, True])
def test_long_draft_blocks_reload_the_walk_inputs(with_q):
    # gamma above 32: the walk fetches its inputs 32 steps at a time; drafts that mostly agree with the target so
    # that the walk gets past the first batch of steps
    B, gamma, V = 12, 45, 4096
    rng = np.random.default_rng(77)
    logits = wl.make_logits(B, gamma, V, seed=77)
    f = wl.bf16_bits_to_f32(logits)
    best = np.argmax(f, -1)
    # sharpen: make the row maximum dominate so that it is accepted with probability near one
    x = f.copy()
    np.put_along_axis(x, best[..., None], 30.0, axis=-1)
    logits = wl.f32_to_bf16_bits(x)
    draft = best[:, :gamma].astype(np.int32).copy()
    draft[3, 40] = (draft[3, 40] + 1) % V                  # one late rejection
    draft[5, 33] = (draft[5, 33] + 7) % V
    u = rng.random((B, gamma + 1, 2), dtype=np.float32)
    q = None
    if with_q:
        q = np.full((B, gamma, V), 0.2 / (V - 1), np.float32)
        np.put_along_axis(q, draft[..., None].astype(np.int64), 0.8, axis=-1)
    acc, out = check(logits, draft, u, 0.7, 20, 0.8, q=q)
    assert acc.max() == gamma and acc[3] == 40 and acc[5] == 33


@pytest.mark.parametrize("pen", [1.2, 0.3, 1.5, -0.7])
def test_presence_penalties_that_are_and_are_not_bf16_numbers(pen):
    # 1.5 is a bf16 number, 1.2, 0.3 and -0.7 are not: the lowered logits are then no bf16 numbers either and
    # only the exact fp32 keys order them; the row maxima are among the seen tokens, so the penalty decides
    B, gamma, V = 16, 4, 32768
    rng = np.random.default_rng(int(abs(pen) * 100))
    logits = wl.make_logits(B, gamma, V, seed=21)
    best = np.argmax(wl.bf16_bits_to_f32(logits), -1)
    draft = np.where(rng.random((B, gamma)) < 0.7, best[:, :gamma], rng.integers(0, V, (B, gamma))).astype(np.int32)
    bits = rng.random((B, V)) < 0.05
    bits[np.arange(B)[:, None], best] = True               # the row maxima are among the seen tokens
    seen = np.packbits(bits, axis=1, bitorder="little")
    u = rng.random((B, gamma + 1, 2), dtype=np.float32)
    check(logits, draft, u, 0.7, 20, 0.8, seen=seen, pen=pen)
