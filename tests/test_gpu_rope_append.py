"""ts_rope_kv_append against the oracle's rotary embedding: rotated Q and K within one bf16 rounding of
the fp64 values, V bit-exact, nothing else in the pools touched, positions up to the longest contexts."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_22788_b200 import api, workloads as wl
from gpu_util import bf16_tensor, geometry

pytestmark = pytest.mark.gpu


def _inv_freq(D, base=1.0e6):
    return (base ** (-np.arange(0, D, 2, dtype=np.float64) / D)).astype(np.float32)


def _bits(t):
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _check_rotated(got_bits, ref, x_bits, what):
    """got: bf16 bits; ref: fp64 oracle values of the same shape [..., D]; x: the unrotated input bits."""
    got = wl.bf16_bits_to_f32(got_bits).astype(np.float64)
    x = np.abs(wl.bf16_bits_to_f32(x_bits).astype(np.float64))
    D = x.shape[-1]
    pair = x[..., : D // 2] + x[..., D // 2:]
    pair = np.concatenate([pair, pair], axis=-1)
    # one bf16 rounding of the exact value (half an ulp <= 2^-9 |ref|, a whole one allowed for values next to
    # a rounding boundary) plus the fp32 arithmetic: two products, a sum and a sincos of a reduced angle
    tol = 2.0 ** -8 * np.abs(ref) + 1e-6 * pair
    err = np.abs(got - ref)
    assert np.all(err <= tol), f"{what}: worst excess {np.max(err - tol):.3e} at {np.unravel_index(np.argmax(err - tol), err.shape)}"
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    assert rel <= 2e-3, f"{what}: rel-L2 {rel:.3e}"


@pytest.mark.parametrize("layout,P,D,ql,Hq,Hkv", [("HND", 64, 128, 1, 32, 8), ("NHD", 16, 64, 3, 8, 2),
                                                  ("HND", 128, 128, 5, 16, 4), ("NHD", 32, 256, 2, 4, 4)])
def test_rope_append_matches_oracle(layout, P, D, ql, Hq, Hkv):
    # lengths include the longest contexts of the tail batch; only the pages of the new tokens exist
    lens = np.array([ql, 40, 4097, 65536 + 3, 131072, 100000], np.int32)
    B = len(lens)
    max_pages = int((lens.max() + P - 1) // P)
    num_pages = 2 * B * ql + 3
    rng = np.random.default_rng(5)
    bt = np.zeros((B, max_pages), np.int32)
    perm = rng.permutation(num_pages).astype(np.int32)
    nxt = 0
    for s in range(B):
        first, last = (int(lens[s]) - ql) // P, (int(lens[s]) - 1) // P
        for pg in range(first, last + 1):
            bt[s, pg] = perm[nxt]
            nxt += 1
    shape = (num_pages, Hkv, P, D) if layout == "HND" else (num_pages, P, Hkv, D)
    ps = Hkv * P * D
    ts, hs = (D, P * D) if layout == "HND" else (Hkv * D, D)
    k_pool = np.full(shape, 0x7FC0, np.uint16)            # NaN everywhere: whatever is written shows
    v_pool = np.full(shape, 0x7FC0, np.uint16)
    q = wl.normal_bf16((B, ql, Hq, D), seed=11)
    new_k = wl.normal_bf16((B, ql, Hkv, D), seed=12)
    new_v = wl.normal_bf16((B, ql, Hkv, D), seed=13)
    f = _inv_freq(D)
    pos = (lens[:, None].astype(np.int64) - ql + np.arange(ql)[None, :]).reshape(-1)
    ref_q = oracle.rope(q.reshape(B * ql, Hq, D), pos, f).reshape(B, ql, Hq, D)
    ref_k = oracle.rope(new_k.reshape(B * ql, Hkv, D), pos, f).reshape(B, ql, Hkv, D)

    geom = api.AttnGeometry(B, ql, Hq, Hkv, D, P, num_pages, max_pages, ps, ts, hs, 1.0)
    dq, dk, dv = bf16_tensor(q), bf16_tensor(k_pool), bf16_tensor(v_pool)
    q_out = torch.full_like(dq, float("nan"))
    d_bt, d_lens = torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda()
    d_f = torch.from_numpy(f).cuda()
    api.ts_rope_kv_append(geom, dq, q_out, bf16_tensor(new_k), bf16_tensor(new_v), dk, dv, d_bt, d_lens, d_f)
    torch.cuda.synchronize()
    _check_rotated(_bits(q_out), ref_q, q, "rotated q")

    got_k, got_v = _bits(dk), _bits(dv)
    touched = np.zeros(shape[:3] if layout == "NHD" else shape[:3], bool)
    for s in range(B):
        for t in range(ql):
            p_ = int(lens[s]) - ql + t
            page, off = int(bt[s, p_ // P]), p_ % P
            if layout == "HND":
                krow, vrow = got_k[page, :, off, :], got_v[page, :, off, :]
                touched[page, :, off] = True
            else:
                krow, vrow = got_k[page, off, :, :], got_v[page, off, :, :]
                touched[page, off, :] = True
            assert np.array_equal(vrow, new_v[s, t]), "V rows are copied bit for bit"
            _check_rotated(krow, ref_k[s, t], new_k[s, t], f"rotated k of sequence {s} token {t}")
    assert np.all(got_k[~touched] == 0x7FC0) and np.all(got_v[~touched] == 0x7FC0), "nothing else is written"

    # in place (q_out = q_in) gives the same bits
    api.ts_rope_kv_append(geom, dq, dq, bf16_tensor(new_k), bf16_tensor(new_v), dk, dv, d_bt, d_lens, d_f)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(dq), _bits(q_out))


def test_rotated_scores_depend_on_distance_only():
    # the same q and k rows placed at (m, n) and at (m + shift, n + shift): equal dot products after rotation
    D, P, Hq, Hkv = 128, 64, 4, 4
    f = _inv_freq(D, base=10000.0)
    q = wl.normal_bf16((1, 1, Hq, D), seed=21)
    k = wl.normal_bf16((1, 1, Hkv, D), seed=22)
    v = wl.normal_bf16((1, 1, Hkv, D), seed=23)
    dots = []
    for n in (5, 2005, 90005):
        lens = np.array([n + 1], np.int32)
        max_pages = n // P + 1
        bt = np.zeros((1, max_pages), np.int32)
        geom = api.AttnGeometry(1, 1, Hq, Hkv, D, P, 1, max_pages, Hkv * P * D, D, P * D, 1.0)
        dk = torch.zeros((1, Hkv, P, D), dtype=torch.bfloat16, device="cuda")
        dv = torch.zeros_like(dk)
        # the key sits at position n; rotate the query as if it sat 37 positions later by giving it its own call
        api.ts_rope_kv_append(geom, bf16_tensor(q), torch.empty_like(bf16_tensor(q)), bf16_tensor(k), bf16_tensor(v), dk, dv,
                              torch.from_numpy(bt).cuda(), torch.from_numpy(lens).cuda(), torch.from_numpy(f).cuda())
        k_rot = dk[0, :, n % P, :].float().cpu().numpy().astype(np.float64)
        lens_q = np.array([n + 38], np.int32)
        mp2 = (n + 37) // P + 1
        geom2 = api.AttnGeometry(1, 1, Hq, Hkv, D, P, 1, mp2, Hkv * P * D, D, P * D, 1.0)
        q_out = torch.empty_like(bf16_tensor(q))
        dk2 = torch.zeros_like(dk)
        api.ts_rope_kv_append(geom2, bf16_tensor(q), q_out, bf16_tensor(k), bf16_tensor(v), dk2, dv,
                              torch.zeros((1, mp2), dtype=torch.int32, device="cuda"),
                              torch.from_numpy(lens_q).cuda(), torch.from_numpy(f).cuda())
        torch.cuda.synchronize()
        q_rot = q_out[0, 0].float().cpu().numpy().astype(np.float64)
        dots.append(np.einsum("hd,hd->h", q_rot, k_rot))
    ref_q = oracle.rope(q.reshape(1, Hq, D), np.array([37]), f)[0]
    ref = np.einsum("hd,hd->h", ref_q, wl.bf16_bits_to_f32(k).astype(np.float64)[0, 0])
    for d_ in dots:
        # two bf16-rounded vectors of norm ~ sqrt(128): the dot product carries ~ 2^-9 * |q||k| / sqrt(D) of noise
        assert np.allclose(d_, ref, rtol=0, atol=0.15), (d_, ref)


def test_rejects_bad_arguments():
    D, P = 128, 64
    geom = api.AttnGeometry(1, 1, 4, 4, D, P, 1, 1, 4 * P * D, D, P * D, 1.0)
    t = torch.zeros((1, 1, 4, D), dtype=torch.bfloat16, device="cuda")
    pool = torch.zeros((1, 4, P, D), dtype=torch.bfloat16, device="cuda")
    bt = torch.zeros((1, 1), dtype=torch.int32, device="cuda")
    lens = torch.ones((1,), dtype=torch.int32, device="cuda")
    f = torch.ones((D // 2,), dtype=torch.float32, device="cuda")
    bad = api.AttnGeometry(1, 1, 4, 4, 24, P, 1, 1, 4 * P * 24, 24, P * 24, 1.0)
    with pytest.raises(api.TailSieveError):
        api.ts_rope_kv_append(bad, t, t, t, t, pool, pool, bt, lens, f)
    with pytest.raises(api.TailSieveError):
        api.ts_rope_kv_append(geom, t, t, t, t, pool, pool, bt, lens, None)
