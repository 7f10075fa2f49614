"""Pins of the oracle's key/value producer (paper Section 2.1: W_K, W_V map a hidden state to the key
and value of the layers that still own a cache) against exact rational arithmetic, structured
weights with known answers, a library matmul, torch's bf16 rounding, and - for the optional rotary
encoding of the key - the complex-number form of the rotation and its defining properties."""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import lckv_oracle as orc
from paper_2405_10637_b200 import inputs as syn


def f64(bits_arr):
    return (np.asarray(bits_arr).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rand_bits(shape, seed, std=1.0):
    return syn.bits(syn.randn_bf16(shape, seed, std=std))


def one_bits():
    return syn.bits(torch.ones(1, dtype=torch.bfloat16))[0]


def rope_tables(n_pos, d, base=10000.0):
    """cos / sin [n_pos, d/2] float32, angle = position * base^(-2i/d)."""
    i = np.arange(d // 2, dtype=np.float64)
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * base ** (-2.0 * i / d)[None, :]
    return np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def test_projection_equals_exact_rational_sums():
    """bf16 values are dyadic rationals: the sums can be taken exactly and compared with the
    float64 result (catches a dropped term, a transposed weight, a wrong feature -> head split)."""
    B, Hkv, d, dm = 2, 2, 4, 6
    x, wk, wv = rand_bits((B, dm), 1), rand_bits((Hkv * d, dm), 2), rand_bits((Hkv * d, dm), 3)
    lens = np.array([3, 0], np.int32)
    _, _, kf, vf = orc.project_kv(x, wk, wv, lens, Hkv, d)
    X, WK, WV = f64(x), f64(wk), f64(wv)
    for b in range(B):
        for f in range(Hkv * d):
            ek = sum(Fraction(float(WK[f, c])) * Fraction(float(X[b, c])) for c in range(dm))
            ev = sum(Fraction(float(WV[f, c])) * Fraction(float(X[b, c])) for c in range(dm))
            assert abs(kf[b, f // d, f % d] - float(ek)) <= 1e-13 * (1 + abs(float(ek)))
            assert abs(vf[b, f // d, f % d] - float(ev)) <= 1e-13 * (1 + abs(float(ev)))


def test_projection_equals_library_matmul():
    B, Hkv, d, dm = 5, 3, 8, 40
    x, wk, wv = rand_bits((B, dm), 4), rand_bits((Hkv * d, dm), 5), rand_bits((Hkv * d, dm), 6)
    lens = np.zeros(B, np.int32)
    _, _, kf, vf = orc.project_kv(x, wk, wv, lens, Hkv, d)
    np.testing.assert_allclose(kf.reshape(B, -1), f64(x) @ f64(wk).T, rtol=0, atol=1e-12)
    np.testing.assert_allclose(vf.reshape(B, -1), f64(x) @ f64(wv).T, rtol=0, atol=1e-12)


def test_selector_weights_route_features_bit_exactly():
    """A weight matrix with a single one per row copies hidden-state entries: the produced bits are
    the input bits, at feature f = (head f // d, dim f % d).  The selector is not symmetric, so a
    transposed weight fails; K and V use different selectors, so swapping them fails."""
    B, Hkv, d = 3, 2, 4
    F = dm = Hkv * d
    x = rand_bits((B, dm), 7)
    perm_k = np.array([3, 0, 7, 5, 1, 6, 2, 4])
    perm_v = np.array([1, 2, 3, 4, 5, 6, 7, 0])
    wk = np.zeros((F, dm), np.uint16)
    wv = np.zeros((F, dm), np.uint16)
    wk[np.arange(F), perm_k] = one_bits()
    wv[np.arange(F), perm_v] = one_bits()
    kb, vb, _, _ = orc.project_kv(x, wk, wv, np.zeros(B, np.int32), Hkv, d)
    assert np.array_equal(kb.reshape(B, F), x[:, perm_k])
    assert np.array_equal(vb.reshape(B, F), x[:, perm_v])


def test_rounding_to_bf16_is_nearest_even_like_torch():
    """d_model = 1: each output is one product of two bf16 numbers, exact in float32; its bf16 bits
    must be what torch's round-to-nearest-even conversion gives (ties included: many products of two
    8-bit significands end in exactly half a unit)."""
    n = 4096
    x = rand_bits((1, 1), 8)
    x[0, 0] = syn.bits(torch.tensor([1.0078125], dtype=torch.bfloat16))[0]      # 1 + 2^-7
    w = rand_bits((n, 1), 9)
    w[:256, 0] = (0x3f80 + np.arange(256) % 128).astype(np.uint16)              # 1 + j 2^-7: makes ties
    kb, _, kf, _ = orc.project_kv(x, w, w, np.zeros(1, np.int32), n // 4, 4)
    prod = (f64(w)[:, 0] * f64(x)[0, 0]).astype(np.float32)
    assert np.array_equal(prod.astype(np.float64), kf.reshape(-1))               # exact in float32
    want = syn.bits(torch.from_numpy(prod).to(torch.bfloat16))
    low = prod.view(np.uint32) & 0xffff
    assert (low == 0x8000).sum() >= 16, "the case must contain exact ties"
    assert np.array_equal(kb.reshape(-1), want)


def test_rotary_position_zero_is_identity_and_values_are_never_rotated():
    B, Hkv, d, dm = 2, 2, 8, 16
    x, wk, wv = rand_bits((B, dm), 10), rand_bits((Hkv * d, dm), 11), rand_bits((Hkv * d, dm), 12)
    cos, sin = rope_tables(16, d)
    k0, v0, _, _ = orc.project_kv(x, wk, wv, np.zeros(B, np.int32), Hkv, d)
    k1, v1, _, _ = orc.project_kv(x, wk, wv, np.zeros(B, np.int32), Hkv, d, cos, sin)
    k2, v2, _, _ = orc.project_kv(x, wk, wv, np.array([5, 9], np.int32), Hkv, d, cos, sin)
    assert np.array_equal(k0, k1) and np.array_equal(v0, v1)
    assert np.array_equal(v0, v2) and not np.array_equal(k0, k2)


def test_rotary_equals_complex_multiplication_and_keeps_norms():
    """(k[i] + 1j k[i + d/2]) * exp(1j p theta_i): the rotation written with complex numbers."""
    B, Hkv, d, dm = 3, 2, 8, 12
    x, wk, wv = rand_bits((B, dm), 13), rand_bits((Hkv * d, dm), 14), rand_bits((Hkv * d, dm), 15)
    lens = np.array([1, 7, 30], np.int32)
    cos, sin = rope_tables(32, d)
    _, _, k_plain, _ = orc.project_kv(x, wk, wv, lens, Hkv, d)
    _, _, k_rot, _ = orc.project_kv(x, wk, wv, lens, Hkv, d, cos, sin)
    half = d // 2
    z = k_plain[..., :half] + 1j * k_plain[..., half:]
    e = cos[lens].astype(np.float64) + 1j * sin[lens].astype(np.float64)      # [B, half]
    zr = z * e[:, None, :]
    np.testing.assert_allclose(k_rot[..., :half], zr.real, rtol=0, atol=1e-12)
    np.testing.assert_allclose(k_rot[..., half:], zr.imag, rtol=0, atol=1e-12)
    # float32 tables: cos^2 + sin^2 = 1 to 1e-7, so pair norms are kept to that accuracy
    n0 = np.abs(z)
    np.testing.assert_allclose(np.abs(k_rot[..., :half] + 1j * k_rot[..., half:]), n0, rtol=1e-6)


def test_rotary_direction_unit_vector():
    """A key equal to the unit vector of dimension 0 turns towards dimension d/2 by +angle."""
    d, dm = 4, 4
    x = np.zeros((1, dm), np.uint16)
    x[0, 0] = one_bits()
    wk = np.zeros((d, dm), np.uint16)
    wk[np.arange(d), np.arange(d)] = one_bits()                   # identity
    cos, sin = rope_tables(4, d)
    _, _, kf, _ = orc.project_kv(x, wk, wk, np.array([1], np.int32), 1, d, cos, sin)
    want = np.array([np.cos(1.0), 0.0, np.sin(1.0), 0.0])         # theta_0 = 1: angle = position
    np.testing.assert_allclose(kf.reshape(-1), want, atol=1e-7)


def test_rotary_scores_depend_on_relative_position_only():
    """<R_m a, R_n b> = <R_{m+s} a, R_{n+s} b>: the property the encoding exists for."""
    d = 8
    eye = np.zeros((d, d), np.uint16)
    eye[np.arange(d), np.arange(d)] = one_bits()
    a, b = rand_bits((1, d), 16), rand_bits((1, d), 17)
    cos, sin = rope_tables(64, d)

    def rot(v, p):
        return orc.project_kv(v, eye, eye, np.array([p], np.int32), 1, d, cos, sin)[2].reshape(-1)

    base = rot(a, 9) @ rot(b, 4)
    for s in (1, 13, 40):
        assert abs(rot(a, 9 + s) @ rot(b, 4 + s) - base) < 1e-5
    assert abs(rot(a, 10) @ rot(b, 4) - base) > 1e-3             # and it does depend on m - n


def test_position_outside_the_table_is_refused():
    x, w = rand_bits((1, 4), 18), rand_bits((4, 4), 19)
    cos, sin = rope_tables(4, 4)
    with pytest.raises(orc.OracleError):
        orc.project_kv(x, w, w, np.array([4], np.int32), 1, 4, cos, sin)
