"""Pins for the oracle's RoPE (CPU only).

Each test checks the oracle against something that is NOT the oracle's own formula: closed forms,
the group law of rotations stated in the paper's RoPE background section, an explicit rotation-matrix
formulation built with numpy, numpy's complex exponential, and properties from Theorem 2
(Chunked RoPE Injection).
"""
import math

import numpy as np
import pytest

THETAS = [1.0e4, 5.0e5, 1.0e6]
POSITIONS = [0, 1, 13, 4096, 131071, 2**24 - 1]


def rotation_matrix(D, pos, inv_freq, style):
    """Explicit D x D block-diagonal R_pos (independent formulation: a matrix, applied by matmul)."""
    R = np.zeros((D, D), dtype=np.float64)
    for i in range(D // 2):
        a = float(pos) * float(inv_freq[i])
        i1, i2 = (i, i + D // 2) if style == 0 else (2 * i, 2 * i + 1)
        R[i1, i1] = math.cos(a)
        R[i1, i2] = -math.sin(a)
        R[i2, i1] = math.sin(a)
        R[i2, i2] = math.cos(a)
    return R


def pairs(x, style):
    D = x.shape[-1]
    if style == 0:
        return x[..., : D // 2], x[..., D // 2 :]
    return x[..., 0::2], x[..., 1::2]


def test_inv_freq_closed_form(oracle_mod):
    # pair 0 always has frequency 1; the last pair has theta^(-(D-2)/D); ratios are constant
    for theta in THETAS:
        for D in (64, 128):
            f = oracle_mod.inv_freq(D, theta)
            assert f.dtype == np.float32 and f.shape == (D // 2,)
            assert f[0] == 1.0
            assert f[-1] == pytest.approx(theta ** (-(D - 2) / D), rel=1e-6)
            ratio = f[1:].astype(np.float64) / f[:-1].astype(np.float64)
            assert np.allclose(ratio, theta ** (-2.0 / D), rtol=3e-7)
    # theta = 10000, D = 64: pair 16 is 10000^(-1/2) = 0.01, pair 8 is 0.1 (fp32-rounded)
    f = oracle_mod.inv_freq(64, 1.0e4)
    assert f[16] == np.float32(0.01) and f[8] == np.float32(0.1)


@pytest.mark.parametrize("style", [0, 1])
def test_position_zero_is_identity(oracle_mod, style):
    x = np.random.default_rng(0).standard_normal((7, 128))
    y = oracle_mod.rope_rows(x, 0, 5.0e5, style)
    assert np.array_equal(x, y)  # cos 0 = 1, sin 0 = 0: bit-identical


@pytest.mark.parametrize("style", [0, 1])
def test_quarter_turn_closed_form(oracle_mod, style):
    # With every frequency = pi/2: position 1 maps (x1, x2) -> (-x2, x1), position 2 -> (-x1, -x2),
    # position 3 -> (x2, -x1).  This fixes the DIRECTION of rotation (a flipped sign fails here).
    D = 16
    x = np.random.default_rng(1).standard_normal((5, D))
    f = np.full(D // 2, math.pi / 2, dtype=np.float32)
    x1, x2 = pairs(x, style)
    for pos, (e1, e2) in {1: (-x2, x1), 2: (-x1, -x2), 3: (x2, -x1), 4: (x1, x2)}.items():
        y1, y2 = pairs(oracle_mod.rope_rows(x, pos, 1.0, style, f), style)
        # pi/2 rounded to fp32 is off by 4.4e-8, so the match is to ~pos * 4.4e-8 * |x|
        assert np.allclose(y1, e1, atol=1e-6) and np.allclose(y2, e2, atol=1e-6)


def test_first_pair_angle_is_position_in_radians(oracle_mod):
    # frequency of pair 0 is exactly 1, so pair 0 of (1, 0) becomes (cos p, sin p)
    D = 64
    x = np.zeros((1, D))
    x[0, 0] = 1.0
    for pos in (1, 2, 100):
        y = oracle_mod.rope_rows(x, pos, 1.0e4, 0)
        assert y[0, 0] == pytest.approx(math.cos(pos), abs=1e-15)
        assert y[0, D // 2] == pytest.approx(math.sin(pos), abs=1e-15)


@pytest.mark.parametrize("theta", THETAS)
@pytest.mark.parametrize("style", [0, 1])
def test_against_explicit_rotation_matrix(oracle_mod, theta, style):
    D = 64
    x = np.random.default_rng(2).standard_normal((3, D))
    f = oracle_mod.inv_freq(D, theta)
    for pos in POSITIONS:
        y = oracle_mod.rope_rows(x, pos, theta, style)
        R = rotation_matrix(D, pos, f, style)
        assert np.allclose(y, x @ R.T, rtol=0, atol=1e-12)


@pytest.mark.parametrize("style", [0, 1])
def test_against_complex_exponential(oracle_mod, style):
    # (x1 + i x2) * exp(i * pos * f): numpy's complex arithmetic as the library routine
    D, theta = 128, 5.0e5
    x = np.random.default_rng(3).standard_normal((11, D))
    f = oracle_mod.inv_freq(D, theta).astype(np.float64)
    x1, x2 = pairs(x, style)
    for pos in POSITIONS:
        z = (x1 + 1j * x2) * np.exp(1j * pos * f)
        y1, y2 = pairs(oracle_mod.rope_rows(x, pos, theta, style), style)
        assert np.allclose(y1, z.real, rtol=0, atol=1e-12) and np.allclose(y2, z.imag, rtol=0, atol=1e-12)


@pytest.mark.parametrize("theta", THETAS)
@pytest.mark.parametrize("style", [0, 1])
def test_pair_norms_preserved(oracle_mod, theta, style):
    x = np.random.default_rng(4).standard_normal((9, 128))
    x1, x2 = pairs(x, style)
    for pos in POSITIONS:
        y1, y2 = pairs(oracle_mod.rope_rows(x, pos, theta, style), style)
        assert np.allclose(y1**2 + y2**2, x1**2 + x2**2, rtol=1e-13, atol=0)


@pytest.mark.parametrize("style", [0, 1])
def test_group_law_rotate_a_then_b_equals_a_plus_b(oracle_mod, style):
    x = np.random.default_rng(5).standard_normal((4, 128))
    for theta in THETAS:
        for a, b in [(1, 2), (13, 4083), (4096, 4096), (70000, 61071), (5, 2**24 - 6)]:
            y_ab = oracle_mod.rope_rows(oracle_mod.rope_rows(x, a, theta, style), b, theta, style)
            y = oracle_mod.rope_rows(x, a + b, theta, style)
            # the angle (a+b) f is formed exactly in double up to one rounding of a magnitude <= 2^24
            assert np.allclose(y_ab, y, rtol=0, atol=4e-8 if a + b > 2**20 else 1e-9)


@pytest.mark.parametrize("style", [0, 1])
def test_scores_depend_on_relative_position_only(oracle_mod, style):
    # <R_a q, R_b k> = <q, R_{b-a} k>, and Theorem 2(1): with N' = N - (v0 - p0),
    # <R_N q, R_{v0+j} k> = <R_N' q, R_{p0+j} k>
    rng = np.random.default_rng(6)
    D, theta = 128, 5.0e5
    q = rng.standard_normal((1, D))
    k = rng.standard_normal((1, D))
    R = lambda x, p: oracle_mod.rope_rows(x, p, theta, style)  # noqa: E731
    for a, b in [(0, 5), (100, 37), (9000, 8000), (40000, 39990)]:
        lhs = np.vdot(R(q, a), R(k, b))
        rhs = np.vdot(q, R(k, b - a)) if b >= a else np.vdot(R(q, a - b), k)
        assert lhs == pytest.approx(rhs, abs=1e-9)
    N, v0, p0 = 5000, 4200, 37
    for j in range(8):
        lhs = np.vdot(R(q, N), R(k, v0 + j))
        rhs = np.vdot(R(q, N - (v0 - p0)), R(k, p0 + j))
        assert lhs == pytest.approx(rhs, abs=1e-9)


def test_half_split_and_interleaved_differ_by_a_fixed_permutation(oracle_mod):
    D, theta = 64, 1.0e4
    x = np.random.default_rng(7).standard_normal((6, D))
    # interleaved index 2i <- half-split index i, 2i+1 <- i + D/2
    perm = np.empty(D, dtype=np.int64)
    perm[0::2] = np.arange(D // 2)
    perm[1::2] = np.arange(D // 2) + D // 2
    for pos in (1, 77, 4096):
        y_half = oracle_mod.rope_rows(x, pos, theta, 0)
        y_int = oracle_mod.rope_rows(x[:, perm], pos, theta, 1)
        assert np.array_equal(y_half[:, perm], y_int)


def test_equal_frequencies_when_theta_is_one(oracle_mod):
    # theta = 1: all pairs rotate by `pos` radians
    D = 32
    x = np.random.default_rng(8).standard_normal((2, D))
    y = oracle_mod.rope_rows(x, 3, 1.0, 0)
    c, s = math.cos(3.0), math.sin(3.0)
    assert np.allclose(y[:, : D // 2], x[:, : D // 2] * c - x[:, D // 2 :] * s, atol=1e-15)
    assert np.allclose(y[:, D // 2 :], x[:, D // 2 :] * c + x[:, : D // 2] * s, atol=1e-15)


def test_bf16_rounding_is_nearest_even_single_step(oracle_mod):
    # exact halfway cases go to the even neighbour; a value just above halfway that a float32 detour would
    # first round DOWN onto the halfway point must still round up (no double rounding)
    one = 1.0
    ulp = 2.0**-7
    cases = {
        one + ulp / 2: 0x3F80,  # tie -> even (1.0)
        one + 3 * ulp / 2: 0x3F82,  # tie -> even (1 + 2 ulp)
        one + ulp / 2 + 2.0**-40: 0x3F81,  # just above the tie; float32 would turn it into the tie
        -(one + ulp / 2 + 2.0**-40): 0xBF81,
        0.0: 0x0000,
        2.0**-133: 0x0001,  # smallest bf16 subnormal
        2.0**-134: 0x0000,  # half of it: tie -> even (0)
        3.0 * 2.0**-134: 0x0002,
    }
    x = np.array(list(cases.keys()))
    got = oracle_mod.bf16_from_double(x)
    assert [int(g) for g in got] == list(cases.values())
    # every bf16 value survives a round trip
    allbits = np.arange(0, 0x7F80, dtype=np.uint16)
    assert np.array_equal(oracle_mod.bf16_from_double(oracle_mod.bf16_to_double(allbits)), allbits)


def test_f16_decode_matches_numpy(oracle_mod):
    bits = np.arange(0, 0x7C00, dtype=np.uint16)  # all finite non-negative halves
    assert np.array_equal(oracle_mod.f16_to_double(bits.view(np.float16)), bits.view(np.float16).astype(np.float64))
