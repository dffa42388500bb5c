"""Pins for the oracle's random-number layer (no GPU)."""
import math
import os

import numpy as np

from oracle import swarm_oracle as o

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answers():
    """Published known-answer vectors of Philox4x32-10 (Salmon et al., SC'11)."""
    n = 0
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        lhs, rhs = line.split("->")
        vals = [int(v, 16) for v in lhs.split()]
        want = [int(v, 16) for v in rhs.split()]
        assert o.philox(vals[:4], vals[4:6]) == want
        n += 1
    assert n == 3


def test_philox_counter_and_key_sensitivity():
    base = o.philox([1, 2, 3, 4], [5, 6])
    for pos in range(4):
        ctr = [1, 2, 3, 4]
        ctr[pos] += 1
        assert o.philox(ctr, [5, 6]) != base
    assert o.philox([1, 2, 3, 4], [6, 6]) != base
    assert o.philox([1, 2, 3, 4], [5, 7]) != base


def test_uniform_int_is_high_half_of_product():
    rng = np.random.default_rng(0)
    for word, m in zip(rng.integers(0, 2**32, 200), rng.integers(1, 2**20, 200)):
        got = o.uniform_int(int(word), int(m))
        assert got == (int(word) * int(m)) // 2**32
        assert 0 <= got < m
    assert o.uniform_int(0xFFFFFFFF, 7) == 6
    assert o.uniform_int(0, 7) == 0


def test_uniform_int_law_chi_square():
    m = 13
    counts = np.zeros(m)
    N = 0
    for c in range(5000):
        for wd in o.philox([c, 0, 0, 77], [3, 0]):
            counts[o.uniform_int(wd, m)] += 1
            N += 1
    chi2 = ((counts - N / m) ** 2 / (N / m)).sum()
    assert chi2 < 40.0          # 12 dof, p ~ 1e-4


def test_uniform_float_range_and_moments():
    assert o.uniform_float(0) == 0.0
    assert o.uniform_float(0xFFFFFFFF) == 1.0 - 2.0**-24
    assert o.uniform_float(0x80000000) == 0.5
    us = np.array([o.uniform_float(w) for c in range(4000) for w in o.philox([c, 1, 2, 3], [9, 9])])
    assert abs(us.mean() - 0.5) < 4 * math.sqrt(1 / 12 / len(us))
    assert abs(us.var() - 1 / 12) < 0.004


def test_box_muller_closed_form_and_moments():
    # u1 = 1 (w0 all ones in the top 24 bits) -> radius 0
    z0, z1 = o.normal_pair(0xFFFFFFFF, 0x12345678)
    assert z0 == 0.0 and z1 == 0.0
    # u2 = 0 -> angle 0: z1 = 0, z0 = sqrt(-2 ln u1)
    w0 = (123456 << 8)
    z0, z1 = o.normal_pair(w0, 0)
    assert z1 == 0.0
    assert z0 == np.float32(math.sqrt(-2.0 * math.log((123456 + 1) * 2.0**-24)))
    # u2 = 1/4 -> angle pi/2: z0 ~ 0, z1 = radius
    z0, z1 = o.normal_pair(w0, 0x40000000)
    assert abs(z0) < 1e-15
    assert z1 == np.float32(math.sqrt(-2.0 * math.log((123456 + 1) * 2.0**-24)))
    zs = []
    for c in range(20000):
        wd = o.philox([c, 0, 0, 1], [0, 0])
        zs.extend(o.normal_pair(wd[0], wd[1]))
        zs.extend(o.normal_pair(wd[2], wd[3]))
    zs = np.array(zs)
    N = len(zs)
    assert abs(zs.mean()) < 4 / math.sqrt(N)
    assert abs(zs.var() - 1) < 4 * math.sqrt(2 / N)
    assert abs((zs**3).mean()) < 4 * math.sqrt(15 / N)
    assert abs((zs**4).mean() - 3) < 4 * math.sqrt(96 / N)


def test_initial_models_use_stream_layout():
    """Model init of node i, coordinate k is init_std * z(stream 1, row i, event 0, k) + offset."""
    s = o.OracleSwarm(4, 10, "complete", seed=0x1234567800000042)
    s.configure(init_std=0.25, offset_std=2.0)
    key = [0x42, 0x12345678]
    for i in range(4):
        sc = o.philox([0, i, 0, 5], key)
        off = np.float32(2.0) * np.float32(o.normal_pair(sc[0], sc[1])[0])
        assert s.offset[i] == off
        for k in range(10):
            wd = o.philox([k // 4, i, 0, 1], key)
            z = (o.normal_pair(wd[0], wd[1]) + o.normal_pair(wd[2], wd[3]))[k % 4]
            assert s.X[i, k] == np.float32(np.float32(0.25) * np.float32(z)) + off
    # sample moments of a larger draw
    s2 = o.OracleSwarm(4, 20000, "complete", seed=7)
    assert abs(s2.X.std() - 0.1) < 0.002 and abs(s2.X.mean()) < 0.002


def test_sr_uniform_layout():
    """One generator call per 8 coordinates; even k -> low half, odd k -> high half of word (k%8)//2."""
    seed, owner, w = 0xABCDEF0123456789, 5, 17
    got = o.sr_uniforms(seed, owner, w, 0, 64)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for k in range(64):
        wd = o.philox([k // 8, owner, w, 10], key)[(k % 8) // 2]
        assert got[k] == ((wd & 0xFFFF) if k % 2 == 0 else (wd >> 16))
    # offsets are absolute coordinates
    assert np.array_equal(o.sr_uniforms(seed, owner, w, 24, 16), got[24:40])
