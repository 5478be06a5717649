"""ts_accept_greedy_noalloc -- the acceptance entry point for callers that cannot allocate.

Some users of this library have no device memory to pass as a workspace and no way to get any
(all of HBM already belongs to their KV cache, or they run where cudaMalloc is not allowed).  For
them the library carries its own fixed scratch array.  This test checks, through the C ABI, that
the variant returns exactly what ts_accept_greedy returns, on two calls in a row: the second call
is smaller than the first, so it runs over whatever the first one left in the shared array.

The file name makes pytest collect it after every other test file.
"""
import numpy as np
import pytest
import torch

from paper_2608_22788_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu


def _device_logits(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _both(logits_bits, draft_np):
    B, R, V = logits_bits.shape
    gamma = R - 1
    lg = _device_logits(logits_bits)
    dr = torch.from_numpy(np.ascontiguousarray(draft_np, dtype=np.int32).reshape(B, gamma)).cuda()
    outs = []
    for use_noalloc in (False, True):
        tgt = torch.full((B, R), -9, dtype=torch.int32, device="cuda")
        acc = torch.full((B,), -9, dtype=torch.int32, device="cuda")
        tok = torch.full((B, R), -9, dtype=torch.int32, device="cuda")
        if use_noalloc:
            api.ts_accept_greedy_noalloc(lg, dr, tgt, acc, tok)
        else:
            ws = torch.empty(api.accept_workspace_bytes(B, gamma, V), dtype=torch.uint8, device="cuda")
            api.ts_accept_greedy(lg, dr, tgt, acc, tok, ws)
        torch.cuda.synchronize()
        outs.append((tgt.cpu().numpy(), acc.cpu().numpy(), tok.cpu().numpy()))
    return outs


def test_noalloc_variant_matches_workspace_variant_on_two_calls_in_a_row():
    # call 1: 16 sequences, gamma 8, full vocabulary (144 rows, several chunks per row)
    B, gamma, V = 16, 8, wl.VOCAB
    logits = wl.make_logits(B, gamma, V, seed=21)
    best = np.argmax(wl.bf16_bits_to_f32(logits), axis=-1)      # only to build a plausible draft
    draft, _ = wl.make_draft(best, V, seed=21)
    ref, got = _both(logits, draft)
    for r, g in zip(ref, got):
        assert np.array_equal(r, g)                               # integers: bit-exact
    assert (ref[1] >= 0).all() and (ref[1] <= gamma).all()

    # call 2, right after: fewer rows, smaller odd vocabulary -> runs over call 1's leftovers
    B, gamma, V = 3, 2, 4097
    logits = wl.make_logits(B, gamma, V, seed=22)
    best = np.argmax(wl.bf16_bits_to_f32(logits), axis=-1)
    draft, _ = wl.make_draft(best, V, seed=22)
    ref, got = _both(logits, draft)
    for r, g in zip(ref, got):
        assert np.array_equal(r, g)


def test_noalloc_variant_rejects_more_rows_than_its_scratch_holds():
    B, gamma, V = 1025, 0, 64
    lg = torch.zeros((B, 1, V), dtype=torch.bfloat16, device="cuda")
    tgt = torch.full((B, 1), -9, dtype=torch.int32, device="cuda")
    acc = torch.full((B,), -9, dtype=torch.int32, device="cuda")
    tok = torch.full((B, 1), -9, dtype=torch.int32, device="cuda")
    with pytest.raises(api.TailSieveError, match="TS_ERR_UNSUPPORTED"):
        api.ts_accept_greedy_noalloc(lg, None, tgt, acc, tok)
    torch.cuda.synchronize()
    assert (tgt == -9).all() and (acc == -9).all()                # nothing was launched
    # 1024 rows is still fine
    api.ts_accept_greedy_noalloc(lg[:1024], None, tgt[:1024], acc[:1024], tok[:1024])
    torch.cuda.synchronize()
    assert (tgt[:1024] == 0).all() and (acc[:1024] == 0).all()
