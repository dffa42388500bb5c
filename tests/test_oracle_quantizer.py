"""Pins for the oracle's lattice quantizer (constructive reading of Corollary 1)."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import swarm_oracle as o

BITS = (2, 3, 4, 5, 6, 7, 8)


def L_of(b):
    return 2 ** (b - 1) - 1


def exact_exponent(rho, M, b):
    """The rule in exact rational arithmetic (independent of float library calls)."""
    rho, M = Fraction(float(rho)), Fraction(float(M))
    if rho == 0:
        e = -126
    else:
        e = -400
        while L_of(b) * Fraction(2) ** e < rho:
            e += 1
    if M > 0:
        fm = -400                      # least fm with M < 2^fm
        while Fraction(2) ** fm <= M:
            fm += 1
        e = max(e, fm - 23)
    return min(max(e, -126), 119)


@pytest.mark.parametrize("b", BITS)
def test_exponent_rule_matches_exact_arithmetic(b):
    rng = np.random.default_rng(b)
    rhos = [0.0, 1.0, 0.5, 2.0**-126, 2.0**-130, 2.0**-149, 3.0e38, 1.7e38, 127.0, 7.0, 6.999999, 7.000001]
    rhos += [float(np.float32(L_of(b)) * np.float32(2.0) ** k) for k in (-30, -3, 0, 5, 60)]
    rhos += [float(np.nextafter(np.float32(L_of(b) * 2.0**-3), np.float32(np.inf)))]
    rhos += list(np.float32(10.0 ** rng.uniform(-44, 38, 300)))
    for rho in rhos:
        rho = float(np.float32(rho))
        for M in (0.0, rho, max(rho, 1e-3), rho * 3e5, rho * 1e9, 3.0e38):
            M = float(np.float32(min(M, 3.3e38)))
            assert o.exponent(rho, M, b) == exact_exponent(rho, M, b), (rho, M, b)


@pytest.mark.parametrize("b", BITS)
def test_exponent_covers_range_and_is_least(b):
    rng = np.random.default_rng(10 + b)
    for rho in np.float32(10.0 ** rng.uniform(-20, 20, 200)):
        e = o.exponent(float(rho), 0.0, b)
        assert Fraction(L_of(b)) * Fraction(2) ** e >= Fraction(float(rho))
        assert Fraction(L_of(b)) * Fraction(2) ** (e - 1) < Fraction(float(rho))


def test_stochastic_rounding_probability_is_exact_over_all_uniforms():
    """Enumerate all 2^16 rounding uniforms: P(round up) = floor(frac * 2^16) / 2^16 exactly."""
    for x, e in ((0.3, -2), (-0.3, -2), (5.75, 1), (-1e-3, -12), (0.1234567, -5)):
        x = float(np.float32(x))
        t = Fraction(x) / Fraction(2) ** e
        f = math.floor(t)
        thr = math.floor((t - f) * 65536)
        qs = np.array([o.enc_q(x, e, u) for u in range(65536)])
        assert set(qs.tolist()) <= {f, f + 1}
        assert int((qs == f + 1).sum()) == thr
        assert np.all(qs[:thr] == f + 1) and np.all(qs[thr:] == f)
        # unbiased up to the 16-bit granularity: mean in (x - 2^(e-16), x]
        mean = Fraction(int(qs.sum()), 65536) * Fraction(2) ** e
        assert Fraction(x) - Fraction(2) ** (e - 16) < mean <= Fraction(x)


@pytest.mark.parametrize("b", BITS)
def test_lattice_points_are_fixed_points(b):
    e = -4
    for q in (-300, -1, 0, 1, 37, 1000):
        x = q * 2.0**e
        for u in (0, 1, 12345, 65535):
            assert o.enc_q(x, e, u) == q
        for key_off in range(-L_of(b), L_of(b) + 1):
            y = (q + key_off) * 2.0**e
            assert o.dec(y, o.code(q, b), e, b) == x


@pytest.mark.parametrize("b", BITS)
def test_decode_window_theorem_exhaustive(b):
    """Every q with q - q_y in [-L, L+1] is recovered; the next ones outside wrap by 2^b."""
    e = 3
    L = L_of(b)
    for qy in (-1000, -1, 0, 5, 99999):
        for frac in (0.0, 0.375, 0.96875):   # exactly representable in fp32
            y = (qy + frac) * 2.0**e
            for delta in range(-L, L + 2):
                q = qy + delta
                assert o.dec(y, o.code(q, b), e, b) == q * 2.0**e
            # just outside the window: aliased onto the in-window point of the same colour
            assert o.dec(y, o.code(qy + L + 2, b), e, b) == (qy + L + 2 - 2**b) * 2.0**e
            assert o.dec(y, o.code(qy - L - 1, b), e, b) == (qy - L - 1 + 2**b) * 2.0**e


@pytest.mark.parametrize("b", BITS)
def test_round_trip_error_below_one_step_when_key_is_in_range(b):
    rng = np.random.default_rng(b)
    for _ in range(300):
        e = int(rng.integers(-20, 10))
        x = float(np.float32(rng.normal() * 2.0**e * 50))
        y = float(np.float32(x + rng.uniform(-1, 1) * L_of(b) * 2.0**e))
        if abs(np.float32(x) - np.float32(y)) > L_of(b) * 2.0**e:
            continue
        u = int(rng.integers(0, 65536))
        Q = o.dec(y, o.code(o.enc_q(x, e, u), b), e, b)
        assert abs(Q - x) < 2.0**e
        assert Q == o.enc_q(x, e, u) * 2.0**e


def test_far_key_gives_the_predicted_alias():
    b, e = 4, 0
    x, y = 100.25, 3.5           # 97 steps apart, window is 7
    q = o.enc_q(x, e, 0)         # thr = floor(.25 * 65536) = 16384 > 0 -> rounds up
    assert q == 101
    got = o.dec(y, o.code(q, b), e, b)
    assert got == 5.0            # 101 mod 16 = 5; window around q_y = 3 is [-4, 11]
    assert (got - q) % 16 == 0


def test_saturating_conversion_for_distant_keys():
    # key * 2^-e overflows the int32 range: conversion saturates, arithmetic wraps mod 2^32
    y, e, b = 3.0e20, -10, 8
    got = o.dec(y, 0x7F, e, b)
    qy = 2**31 - 1
    delta = (0x7F - qy) % 256
    if delta > 128:
        delta -= 256
    q = (qy + delta + 2**31) % 2**32 - 2**31
    assert got == float(np.float32(q)) * 2.0**e
    # a key that is not a number has cell 0 (as the float-to-integer conversion of the CUDA side defines it)
    for c in range(256):
        assert o.dec(float("nan"), c, e, b) == o.dec(0.0, c, e, b)


@pytest.mark.parametrize("b", BITS)
def test_packing_matches_numpy_little_bit_order(b):
    rng = np.random.default_rng(b)
    for count in (1024, 1000, 7, 1):
        codes = rng.integers(0, 2**b, count).astype(np.uint8)
        packed = o.pack_block(codes, b)
        assert packed.shape == (1024 * b // 8,)
        bits = np.zeros(1024 * b, dtype=np.uint8)
        for j in range(b):                       # bit j of code k sits at stream position k*b + j
            bits[np.arange(count) * b + j] = (codes >> j) & 1
        assert np.array_equal(packed, np.packbits(bits, bitorder="little"))
        assert np.array_equal(o.unpack_block(packed, count, b), codes)


def test_bf16_rounding_is_nearest_even():
    import torch
    rng = np.random.default_rng(0)
    v = np.float32(rng.normal(size=2000) * 10.0 ** rng.uniform(-6, 6, 2000))
    want = torch.from_numpy(v).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([o.round_bf16(float(t)) for t in v], dtype=np.float32)
    assert np.array_equal(got, want)
    assert o.round_bf16(1.0 + 2.0**-8) == 1.0            # tie -> even
    assert o.round_bf16(1.0 + 3 * 2.0**-8) == 1.0 + 2.0**-6
