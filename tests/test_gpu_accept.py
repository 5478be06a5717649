"""GPU parity tests of ts_accept_greedy against the oracle: bit-exact argmax (lowest index wins
ties), accepted length and emitted tokens."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_22788_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu


def run_gpu(logits_bits: np.ndarray, draft: np.ndarray, row_stride=None):
    B, R, V = logits_bits.shape
    gamma = R - 1
    lg = torch.from_numpy(np.ascontiguousarray(logits_bits).view(np.int16)).cuda().view(torch.bfloat16)
    dr = torch.from_numpy(np.ascontiguousarray(draft, dtype=np.int32).reshape(B, gamma)).cuda()
    tgt = torch.full((B, R), -5, dtype=torch.int32, device="cuda")
    acc = torch.full((B,), -5, dtype=torch.int32, device="cuda")
    out = torch.full((B, R), -5, dtype=torch.int32, device="cuda")
    ws = torch.empty(api.accept_workspace_bytes(B, gamma, V), dtype=torch.uint8, device="cuda")
    api.ts_accept_greedy(lg, dr, tgt, acc, out, ws, row_stride=row_stride)
    torch.cuda.synchronize()
    return tgt.cpu().numpy(), acc.cpu().numpy(), out.cpu().numpy()


def check(logits_bits, draft):
    ref = oracle.accept_greedy(logits_bits, draft)
    got = run_gpu(logits_bits, draft)
    for r, g, name in zip(ref, got, ("target_argmax", "accept_len", "out_tokens")):
        assert np.array_equal(r, g), name
    return ref


@pytest.mark.parametrize("gamma", [0, 4, 8, 16])
def test_full_vocab_seeded_cut_points(gamma):
    B, V = 16, wl.VOCAB
    logits = wl.make_logits(B, gamma, V, seed=gamma)
    best, _, _ = oracle.accept_greedy(logits, np.zeros((B, gamma), np.int32))
    draft, cut = wl.make_draft(best, V, seed=gamma)
    tgt, acc, out = check(logits, draft)
    assert np.array_equal(acc, cut)


@pytest.mark.parametrize("V", [5, 8, 1000, 4097, 151944])
def test_odd_vocab_sizes_and_ties(V):
    rng = np.random.default_rng(V)
    B, gamma = 3, 2
    x = rng.standard_normal((B, gamma + 1, V)).astype(np.float32)
    x[0, 0, :] = 1.5                                  # all equal -> 0
    x[0, 1, V - 1] = 50.0                             # maximum at the very last index
    x[1, 0, 0] = 50.0; x[1, 0, V - 1] = 50.0          # tie between first and last
    x[1, 1, V - 2] = 50.0; x[1, 1, V - 1] = 50.0      # tie at the end
    x[2, 0, :] = -np.inf                              # fully masked row -> 0
    if V > 16:
        x[2, 1, 7] = 60.0; x[2, 1, 8] = 60.0          # tie across a 16-byte vector boundary
    bits = wl.f32_to_bf16_bits(x)
    tgt, _, _ = check(bits, rng.integers(0, V, size=(B, gamma)))
    assert tgt[0, 0] == 0 and tgt[0, 1] == V - 1 and tgt[1, 0] == 0 and tgt[1, 1] == V - 2 and tgt[2, 0] == 0


@pytest.mark.parametrize("V", [4096, 20000, 151936])
def test_nan_never_wins_and_a_row_of_nan_gives_a_token_in_range(V):
    # NaN logits are outside the contract; what is promised is that they never win against a number, and
    # that a row without any number still yields index 0 (never an index at or beyond the vocabulary)
    x = np.full((3, 1, V), np.nan, np.float32)
    x[1, 0, V - 3] = -np.inf                          # the only number of the row, and the smallest there is
    x[2, 0, 1::2] = -5.0
    x[2, 0, 2001] = -4.5
    bits = wl.f32_to_bf16_bits(x)
    B = 3
    lg = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    tgt = torch.full((B, 1), -7, dtype=torch.int32, device="cuda")
    acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    out = torch.full((B, 1), -7, dtype=torch.int32, device="cuda")
    ws = torch.empty(api.accept_workspace_bytes(B, 0, V), dtype=torch.uint8, device="cuda")
    api.ts_accept_greedy(lg, None, tgt, acc, out, ws)
    torch.cuda.synchronize()
    t = tgt.cpu().numpy()[:, 0]
    assert t[0] == 0 and t[1] == V - 3 and t[2] == 2001
    assert np.array_equal(out.cpu().numpy()[:, 0], t) and (acc.cpu().numpy() == 0).all()


def test_ties_across_chunk_boundaries_and_signed_zero():
    V = wl.VOCAB
    x = np.full((2, 1, V), -1.0, np.float32)
    for i in range(0, V, 1187):                       # the same maximum all over the row
        x[0, 0, i + 3] = 7.0
    x[1, 0, :] = -3.0
    x[1, 0, 100000] = -0.0
    x[1, 0, 140000] = 0.0                             # +0 == -0: index 100000 wins
    tgt, _, _ = check(wl.f32_to_bf16_bits(x), np.zeros((2, 0), np.int32))
    assert tgt[0, 0] == 3 and tgt[1, 0] == 100000


def test_draft_equal_to_argmax_accepts_all():
    B, gamma, V = 8, 8, 32000
    logits = wl.make_logits(B, gamma, V, seed=3)
    best, _, _ = oracle.accept_greedy(logits, np.zeros((B, gamma), np.int32))
    tgt, acc, out = check(logits, best[:, :gamma])
    assert (acc == gamma).all() and np.array_equal(out, best)


def test_many_rows_decode_sampling():
    # gamma = 0 with a bulk-sized batch: plain greedy sampling of 256 tokens
    B, V = 256, 32768
    logits = wl.make_logits(B, 0, V, seed=11)
    check(logits, np.zeros((B, 0), np.int32))


def test_row_stride_padding():
    B, gamma, V, stride = 2, 1, 1000, 1024
    rng = np.random.default_rng(2)
    padded = np.full((B, gamma + 1, stride), wl.f32_to_bf16_bits(np.array([99.0], np.float32))[0], np.uint16)
    padded[:, :, :V] = wl.make_logits(B, gamma, V, seed=5)
    ref = oracle.accept_greedy(np.ascontiguousarray(padded[:, :, :V]), np.zeros((B, gamma), np.int32))
    B_, R, _ = padded.shape
    lg = torch.from_numpy(padded.view(np.int16)).cuda().view(torch.bfloat16)
    tgt = torch.empty((B, R), dtype=torch.int32, device="cuda")
    acc = torch.empty((B,), dtype=torch.int32, device="cuda")
    out = torch.empty((B, R), dtype=torch.int32, device="cuda")
    ws = torch.empty(api.accept_workspace_bytes(B, gamma, V), dtype=torch.uint8, device="cuda")
    lib = api.load_library()
    rc = lib.ts_accept_greedy(lg.data_ptr(), stride, torch.zeros((B, gamma), dtype=torch.int32, device="cuda").data_ptr(),
                              B, gamma, V, tgt.data_ptr(), acc.data_ptr(), out.data_ptr(), ws.data_ptr(), ws.numel(),
                              torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert rc == 0
    assert np.array_equal(tgt.cpu().numpy(), ref[0])


@pytest.mark.parametrize("B,gamma", [(5, 1), (37, 2), (300, 3), (9, 31), (7, 32), (3, 70), (260, 0)])
def test_block_lengths_around_the_lane_group_sizes(B, gamma):
    # the finishing kernel gives each sequence a group of 1, 2, 4 ... 32 lanes; blocks longer than 32 positions
    # take several passes; planted cut points anywhere in the block, including "all accepted"
    V = 2048
    rng = np.random.default_rng(1000 * B + gamma)
    logits = wl.make_logits(B, gamma, V, seed=B + gamma)
    best, _, _ = oracle.accept_greedy(logits, np.zeros((B, gamma), np.int32))
    draft = best[:, :gamma].copy()
    cut = rng.integers(0, gamma + 1, B)
    for b in range(B):
        if cut[b] < gamma:
            draft[b, cut[b]] = (draft[b, cut[b]] + 1 + rng.integers(0, V - 1)) % V
            later = rng.random(gamma) < 0.5                  # later positions: half still agree, half do not
            for i in range(cut[b] + 1, gamma):
                if later[i]:
                    draft[b, i] = rng.integers(0, V)
    tgt, acc, out = check(logits, draft)
    assert np.array_equal(acc, cut)
