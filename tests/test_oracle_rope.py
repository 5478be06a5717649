"""Pins for the oracle's rotary position embedding (CPU only).

The oracle is the rotation written out per pair; it is pinned to things that do not share its
formula: complex multiplication in NumPy, the position-0 identity, the pair-norm invariant, the
relative-position property of the rotated dot product, the additivity of rotations and a one-hot
row whose image is a (cos, sin) pair.
"""
import numpy as np
import pytest

import oracle
from paper_2608_22788_b200 import workloads as wl


def _inv_freq(D, base=1.0e6):
    return (base ** (-np.arange(0, D, 2, dtype=np.float64) / D)).astype(np.float32)


def _rows(rows, heads, D, seed):
    return wl.normal_bf16((rows, heads, D), seed=seed)


@pytest.mark.parametrize("D", [8, 64, 128])
def test_equals_complex_multiplication(D):
    rows, heads = 7, 3
    x = _rows(rows, heads, D, seed=D)
    pos = np.array([0, 1, 2, 17, 4095, 65537, 131071], dtype=np.int64)
    f = _inv_freq(D)
    got = oracle.rope(x, pos, f)
    xf = wl.bf16_bits_to_f32(x).astype(np.float64)
    z = xf[..., : D // 2] + 1j * xf[..., D // 2:]
    w = np.exp(1j * pos[:, None, None].astype(np.float64) * f.astype(np.float64)[None, None, :])
    ref = z * w
    assert np.allclose(got[..., : D // 2], ref.real, rtol=0, atol=1e-12)
    assert np.allclose(got[..., D // 2:], ref.imag, rtol=0, atol=1e-12)


def test_position_zero_is_the_identity():
    x = _rows(5, 2, 64, seed=1)
    got = oracle.rope(x, np.zeros(5, np.int64), _inv_freq(64))
    assert np.array_equal(got, wl.bf16_bits_to_f32(x).astype(np.float64))


def test_pair_norms_are_preserved():
    D = 128
    x = _rows(9, 4, D, seed=2)
    pos = np.arange(9, dtype=np.int64) * 12345
    got = oracle.rope(x, pos, _inv_freq(D))
    xf = wl.bf16_bits_to_f32(x).astype(np.float64)
    n_in = xf[..., : D // 2] ** 2 + xf[..., D // 2:] ** 2
    n_out = got[..., : D // 2] ** 2 + got[..., D // 2:] ** 2
    assert np.allclose(n_in, n_out, rtol=1e-12, atol=1e-12)


def test_rotated_dot_product_depends_on_the_position_difference_only():
    D = 64
    f = _inv_freq(D, base=10000.0)
    q = _rows(1, 1, D, seed=3)
    k = _rows(1, 1, D, seed=4)
    dots = []
    for m, n in ((40, 3), (1037, 1000), (70000, 69963)):
        qm = oracle.rope(q, np.array([m]), f)[0, 0]
        kn = oracle.rope(k, np.array([n]), f)[0, 0]
        dots.append(float(qm @ kn))
    q37 = oracle.rope(q, np.array([37]), f)[0, 0]
    k0 = wl.bf16_bits_to_f32(k).astype(np.float64)[0, 0]
    ref = float(q37 @ k0)
    assert np.allclose(dots, ref, rtol=0, atol=1e-9)


def test_one_hot_row_maps_to_cos_and_sin():
    D = 16
    f = _inv_freq(D, base=100.0)
    d = 3
    x = np.zeros((1, 1, D), np.float32)
    x[0, 0, d] = 1.0
    got = oracle.rope(wl.f32_to_bf16_bits(x), np.array([11]), f)[0, 0]
    angle = 11.0 * float(f[d])
    expect = np.zeros(D)
    expect[d] = np.cos(angle)
    expect[d + D // 2] = np.sin(angle)
    assert np.allclose(got, expect, rtol=0, atol=1e-15)
    # the high half of the pair turns the other way round: e_{d+D/2} -> (-sin, cos)
    x[:] = 0
    x[0, 0, d + D // 2] = 1.0
    got = oracle.rope(wl.f32_to_bf16_bits(x), np.array([11]), f)[0, 0]
    expect[:] = 0
    expect[d] = -np.sin(angle)
    expect[d + D // 2] = np.cos(angle)
    assert np.allclose(got, expect, rtol=0, atol=1e-15)


def test_heads_share_the_angle_and_rows_do_not_mix():
    D = 32
    x = _rows(4, 3, D, seed=5)
    pos = np.array([5, 6, 7, 8], dtype=np.int64)
    f = _inv_freq(D)
    full = oracle.rope(x, pos, f)
    for r in range(4):
        for h in range(3):
            one = oracle.rope(x[r:r + 1, h:h + 1], pos[r:r + 1], f)
            assert np.array_equal(one[0, 0], full[r, h])
