"""Pins for the oracle's greedy acceptance (CPU only).

Argmax is pinned to ``numpy.argmax`` on the decoded floats (first occurrence =
lowest index, the same tie rule) and to planted ties; acceptance to cases whose
answer is known by construction.
"""
import numpy as np
import pytest

import oracle
from paper_2608_22788_b200 import workloads as wl


def _bits(x):
    return wl.f32_to_bf16_bits(np.asarray(x, np.float32))


@pytest.mark.parametrize("V", [5, 1000, 4097])
def test_argmax_matches_numpy_first_occurrence(V):
    logits = wl.make_logits(3, 4, vocab=V, seed=V)
    draft = np.zeros((3, 4), np.int32)
    tgt, _, _ = oracle.accept_greedy(logits, draft)
    ref = np.argmax(wl.bf16_bits_to_f32(logits), axis=-1)
    assert np.array_equal(tgt, ref)


def test_bf16_ties_are_common_and_resolved_to_lowest_index():
    # with 150k draws quantised to bf16 the maximum is often attained more than once
    V = wl.VOCAB
    logits = wl.make_logits(4, 7, vocab=V, seed=1)
    f = wl.bf16_bits_to_f32(logits)
    tgt, _, _ = oracle.accept_greedy(logits, np.zeros((4, 7), np.int32))
    assert np.array_equal(tgt, np.argmax(f, axis=-1))
    mx = f.max(-1, keepdims=True)
    assert ((f == mx).sum(-1) > 1).any(), "expected at least one tied row in 32 rows"


@pytest.mark.parametrize("pos", [(0, 999), (998, 999), (7, 8), (15, 16), (511, 512)])
def test_planted_ties(pos):
    V = 1000
    x = np.full((1, 1, V), -3.0, np.float32)
    x[0, 0, pos[0]] = 9.0
    x[0, 0, pos[1]] = 9.0
    tgt, acc, out = oracle.accept_greedy(_bits(x), np.zeros((1, 0), np.int32))
    assert tgt[0, 0] == pos[0] and acc[0] == 0 and out[0, 0] == pos[0]


def test_signed_zero_all_equal_and_last_index():
    V = 37
    x = np.full((4, 1, V), -1.0, np.float32)
    x[0, 0, 5] = -0.0
    x[0, 0, 9] = 0.0                 # +0 == -0: index 5 wins
    x[1, 0, :] = 2.5                 # all equal -> 0
    x[2, 0, V - 1] = 4.0             # maximum at the very last index
    x[3, 0, :] = -np.inf             # fully masked vocabulary -> 0
    tgt, _, _ = oracle.accept_greedy(_bits(x), np.zeros((4, 0), np.int32))
    assert tgt[:, 0].tolist() == [5, 0, V - 1, 0]


def _rows_with_winners(winners, V):
    B, R = winners.shape
    x = np.full((B, R, V), -2.0, np.float32)
    for b in range(B):
        for i in range(R):
            x[b, i, winners[b, i]] = 3.0
    return _bits(x)


def test_draft_equal_to_target_accepts_everything():
    V, gamma = 50, 6
    rng = np.random.default_rng(0)
    win = rng.integers(0, V, size=(5, gamma + 1))
    logits = _rows_with_winners(win, V)
    tgt, acc, out = oracle.accept_greedy(logits, win[:, :gamma])
    assert np.array_equal(tgt, win)
    assert (acc == gamma).all()
    assert np.array_equal(out, win)            # draft ++ target[gamma]


def test_first_draft_token_wrong_accepts_nothing():
    V, gamma = 50, 4
    win = np.arange(10).reshape(2, 5)
    draft = win[:, :gamma].copy()
    draft[:, 0] += 1
    tgt, acc, out = oracle.accept_greedy(_rows_with_winners(win, V), draft)
    assert (acc == 0).all()
    assert np.array_equal(out[:, 0], win[:, 0]) and (out[:, 1:] == -1).all()


def test_longest_prefix_not_match_count():
    # matches at positions 0, 1, 3 but not 2: accept 2, emit draft[0:2] ++ target[2]
    V, gamma = 20, 4
    win = np.array([[3, 4, 5, 6, 7]])
    draft = np.array([[3, 4, 9, 6]])
    tgt, acc, out = oracle.accept_greedy(_rows_with_winners(win, V), draft)
    assert acc[0] == 2 and out[0].tolist() == [3, 4, 5, -1, -1]


@pytest.mark.parametrize("gamma", [0, 1, 4, 16])
def test_seeded_cut_points_are_recovered(gamma):
    V, B = 997, 16
    logits = wl.make_logits(B, gamma, vocab=V, seed=gamma)
    best = np.argmax(wl.bf16_bits_to_f32(logits), axis=-1)
    draft, cut = wl.make_draft(best, V, seed=gamma)
    tgt, acc, out = oracle.accept_greedy(logits, draft)
    assert np.array_equal(acc, cut)
    for b in range(B):
        a = int(cut[b])
        assert out[b, :a].tolist() == draft[b, :a].tolist()
        assert out[b, a] == best[b, a] and (out[b, a + 1:] == -1).all()
