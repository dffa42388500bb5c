"""Parity of the CUDA path against the CPU oracle, through the C ABI, on identical seeded inputs.

Bar: bit-exact for codes, packed bytes, exponents, counters, pair schedules and the fp32 outputs of
the interaction (every operation there is a single IEEE operation on both sides); max relative
error 1e-6 (max |diff| / max |ref| per row) for what involves transcendental functions or long
fp32 accumulations (normals, local steps, generated data)."""
import numpy as np
import pytest

from oracle import swarm_oracle as o
from paper_1910_12308_b200 import binding as g
from tests.parity import assert_store_equal, inject, make_pair, rel_err

pytestmark = pytest.mark.gpu
TOL = 1e-6


def disjoint_pairs(orc, rng, count):
    """Random disjoint directed edges of the oracle's graph."""
    used, out = set(), []
    order = rng.permutation(orc.n)
    for a in order:
        if a in used:
            continue
        nbrs = [int(b) for b in orc.adj[a] if int(b) not in used and int(b) != a]
        if not nbrs:
            continue
        b = nbrs[int(rng.integers(len(nbrs)))]
        out.append((int(a), b))
        used.update((int(a), b))
        if len(out) == count:
            break
    return np.array(out, dtype=np.int32)


# ---- state generation ----------------------------------------------------------------------------

@pytest.mark.parametrize("topo,deg,n", [("complete", 0, 5), ("ring", 0, 9), ("regular", 4, 32), ("regular", 8, 256)])
def test_topology_matches(topo, deg, n):
    orc, gpu = make_pair(n, 8, topo, deg, seed=11)
    assert np.array_equal(gpu.get_all(g.T_ADJ), orc.adj)


def test_initial_state_matches_within_tolerance():
    orc, gpu = make_pair(6, 5003, seed=3, init_std=0.1, offset_std=0.3, drift_std=0.2, objective=1, grad_std=0.03,
                         nonblocking=1)
    for i in range(6):
        assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL
        assert rel_err(gpu.get(g.T_B, i), orc.B[i]) < TOL
        sc = gpu.get(g.T_SCALARS, i)
        assert abs(sc[0] - orc.offset[i]) <= 1e-6 * 0.3 * 4 and abs(sc[1] - orc.drift[i]) <= 1e-6 * 0.2 * 4
        assert sc[2] == orc.shift[i]


@pytest.mark.parametrize("dtype,groups", [(0, 0), (1, 2)])
def test_lsq_data_matches_within_tolerance(dtype, groups):
    orc, gpu = make_pair(4, 3000, seed=5, objective=2, lsq_m=6, lsq_batch=4, lsq_dtype=dtype, lsq_groups=groups,
                         lsq_noise_std=float(np.sqrt(0.1)))
    assert rel_err(gpu.get(g.T_XSTAR), orc.xstar) < TOL
    for grp in range(orc.groups):
        got = gpu.get(g.T_A, grp).reshape(6, 3000)
        if dtype == 0:
            assert rel_err(got, orc.A[grp]) < TOL
        else:   # bf16 storage: a 1-ulp fp32 difference before rounding may flip a bf16 rounding
            diff = np.abs(got - orc.A[grp])
            assert (diff > 0).mean() < 1e-3 and diff.max() <= 2.0**-8 * np.abs(orc.A[grp]).max()
    for i in range(4):
        assert rel_err(gpu.get(g.T_BVEC, i), orc.bvec[i]) < 5e-6 if dtype else rel_err(gpu.get(g.T_BVEC, i), orc.bvec[i]) < TOL


# ---- pair schedule -------------------------------------------------------------------------------

@pytest.mark.parametrize("topo,deg,n,P", [("ring", 0, 64, 32), ("regular", 4, 32, 16), ("complete", 0, 16, 8),
                                          ("regular", 8, 256, 128), ("complete", 0, 8, 1), ("ring", 0, 5, 7)])
def test_pair_schedule_is_bit_exact(topo, deg, n, P):
    orc, gpu = make_pair(n, 8, topo, deg, seed=2)
    for _ in range(12):
        assert np.array_equal(gpu.sample_pairs(P), orc.sample_pairs(P))
    assert gpu.get_state()[0] == 12


# ---- blocking interaction ------------------------------------------------------------------------

@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8, 32])
@pytest.mark.parametrize("d", [1, 7, 1024, 1030, 2049, 5000])
def test_blocking_interaction_bit_exact(bits, d):
    n = 6
    orc, gpu = make_pair(n, d, "complete", seed=100 + d, offset_std=0.05)
    inject(orc, gpu)
    rng = np.random.default_rng(d + bits)
    for rnd in range(4):
        pairs = disjoint_pairs(orc, rng, int(rng.integers(1, 4)))
        assert orc.interact(pairs, bits) == 0
        assert gpu.interact(pairs, bits) == 0
        assert_store_equal(orc, gpu, bits)


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
def test_blocking_interaction_special_values(bits):
    """Identical models, zeros, huge and tiny magnitudes, and widely separated models."""
    n, d = 4, 3000
    orc, gpu = make_pair(n, d, "complete", seed=1)
    rng = np.random.default_rng(bits)
    X = orc.X
    X[1] = X[0]                                   # rho = 0: magnitude clamp only
    X[2] = 0.0
    X[3] = 0.0
    X[3, 5] = 1e-40                               # subnormal range
    inject(orc, gpu)
    for pairs in ([[0, 1], [2, 3]], [[0, 2], [1, 3]]):
        assert orc.interact(pairs, bits) == 0 and gpu.interact(pairs, bits) == 0
        assert_store_equal(orc, gpu, bits)
    X[0] = (rng.normal(size=d) * 1e30).astype(np.float32)
    X[1] = (rng.normal(size=d) * 1e-30).astype(np.float32)
    X[2] = (rng.normal(size=d) * 1e37).astype(np.float32)
    X[3] = X[2] * np.float32(1 + 2.0**-20)
    X[2, 100:200] = np.float32(2.0) ** rng.integers(-126, 100, 100)      # exact powers of two
    inject(orc, gpu, what=("X",))
    for pairs in ([[0, 1], [2, 3]], [[1, 2], [3, 0]]):
        assert orc.interact(pairs, bits) == 0 and gpu.interact(pairs, bits) == 0
        assert_store_equal(orc, gpu, bits)


def test_blocking_interaction_on_ring_and_many_rounds():
    n, d, bits = 8, 2500, 4
    orc, gpu = make_pair(n, d, "ring", seed=8, offset_std=0.1)
    inject(orc, gpu)
    for rnd in range(12):
        pairs = orc.sample_pairs(4)
        assert np.array_equal(gpu.sample_pairs(4), pairs)
        assert orc.interact(pairs, bits) == 0 and gpu.interact(pairs, bits) == 0
    assert_store_equal(orc, gpu, bits)
    assert abs(gpu.potential() - orc.potential()) <= 1e-9 * orc.potential()


# ---- non-blocking interaction --------------------------------------------------------------------

@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("d", [5, 1024, 3001])
def test_publish_and_nonblocking_interaction_bit_exact(bits, d):
    n = 6
    cfg = dict(objective=1, nonblocking=1, grad_std=0.03, drift_std=0.1, offset_std=0.02)
    orc, gpu = make_pair(n, d, "regular", 4, seed=40 + d, **cfg)
    inject(orc, gpu)
    assert orc.publish(bits) == 0 and gpu.publish(bits) == 0
    assert_store_equal(orc, gpu, bits)
    rng = np.random.default_rng(bits * 1000 + d)
    for rnd in range(5):
        nodes = rng.permutation(n)[: int(rng.integers(1, n + 1))]
        assert orc.local_steps(nodes, 2, 0.05) == 0 and gpu.local_steps(nodes, 2, 0.05) == 0
        for i in nodes:
            assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL
        inject(orc, gpu, what=("X",))                      # teacher forcing after the transcendental step
        pairs = disjoint_pairs(orc, rng, int(rng.integers(1, 4)))
        assert orc.interact(pairs, bits, o.NONBLOCKING) == 0
        assert gpu.interact(pairs, bits, g.NONBLOCKING) == 0
        assert_store_equal(orc, gpu, bits)


def test_nonblocking_auto_publish_and_mode_switch():
    n, d = 4, 2100
    cfg = dict(objective=1, nonblocking=1, grad_std=0.0, drift_std=0.0, offset_std=0.05)
    orc, gpu = make_pair(n, d, "complete", seed=7, **cfg)
    inject(orc, gpu)
    seq = [([[0, 1]], 8, 1), ([[2, 3], [1, 0]], 8, 1), ([[0, 2]], 8, 0), ([[3, 1]], 4, 1), ([[1, 2]], 4, 1),
           ([[0, 3]], 32, 0), ([[2, 0]], 4, 1)]
    for pairs, bits, mode in seq:
        assert orc.interact(pairs, bits, mode) == 0 and gpu.interact(pairs, bits, mode) == 0
        assert_store_equal(orc, gpu, bits)


def test_nonblocking_far_key_alias_matches():
    """A key outside the decode window is defined behaviour (a lattice point of the same colour
    near the key); both sides must produce the same alias, including saturated conversions."""
    n, d, bits = 4, 1500, 4
    cfg = dict(objective=1, nonblocking=1, grad_std=0.0, drift_std=0.0)
    orc, gpu = make_pair(n, d, "complete", seed=9, **cfg)
    orc.publish(bits)
    orc.B[0] += np.float32(3.0)                  # move one snapshot far from what its buffer encodes
    orc.X[0] = orc.B[0]
    orc.B[1, :700] = np.float32(1e30)            # key * 2^-e overflows int32
    orc.X[1] = orc.B[1]
    inject(orc, gpu)
    for pairs in ([[0, 2]], [[1, 3]], [[2, 0], [3, 1]]):
        assert orc.interact(pairs, bits, o.NONBLOCKING) == 0 and gpu.interact(pairs, bits, g.NONBLOCKING) == 0
        assert_store_equal(orc, gpu, bits)


# ---- launches with more pairs / nodes than fit the kernel parameters --------------------------------

@pytest.mark.parametrize("mode,bits", [(0, 4), (1, 2), (2, 8)])
def test_launch_of_128_pairs_on_256_nodes(mode, bits):
    """The 256-node workload's launch shape (random 8-regular graph, up to 128 disjoint pairs from the
    sampler, every node stepping before the launch) at a short model: descriptor lists longer than 64
    entries travel through device memory instead of the kernel parameters."""
    n, d = 256, 2100
    cfg = dict(objective=1, nonblocking=mode, grad_std=0.02, drift_std=0.1, offset_std=0.05)
    orc, gpu = make_pair(n, d, "regular", 8, seed=5, **cfg)
    inject(orc, gpu)
    for rnd in range(3):
        nodes = np.arange(n, dtype=np.int32)
        assert orc.local_steps(nodes, 2, 0.05) == 0 and gpu.local_steps(nodes, 2, 0.05) == 0
        for i in range(0, n, 17):
            assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL
        inject(orc, gpu, what=("X",))
        pairs = orc.sample_pairs(128)
        assert np.array_equal(gpu.sample_pairs(128), pairs) and len(pairs) > 64
        assert orc.interact(pairs, bits, mode) == 0 and gpu.interact(pairs, bits, mode) == 0
        assert_store_equal(orc, gpu, bits)


# ---- magnitude / distance ratios around the kernels' conversion-free range ----------------------

def _ranged_models(n, d, rng):
    """Models whose 1024-blocks have magnitude-to-distance ratios 2^2 ... 2^30 (both signs, some blocks
    exactly on powers of two): scaled values x * 2^-e run from a few units up to the 2^23 limit of the
    exponent rule, across the 2^21 bound below which the kernels use float adds instead of conversions."""
    nblk = (d + 1023) // 1024
    X = np.zeros((n, d), dtype=np.float32)
    for k in range(nblk):
        lo, hi = k * 1024, min(d, (k + 1) * 1024)
        ratio = 2.0 ** (2 + 2 * (k % 15))
        base = (-1.0) ** k * (0.37 if k % 3 else 0.5) * 2.0 ** (k % 7 - 3)
        noise = rng.normal(size=(n, hi - lo))
        X[:, lo:hi] = (base * (1.0 + noise / ratio)).astype(np.float32)
        if k % 4 == 1:                      # mixed signs inside the block
            X[:, lo:hi:2] *= np.float32(-1.0)
    return X


@pytest.mark.parametrize("bits", [2, 4, 5, 8])
def test_blocking_interaction_across_magnitude_ratios(bits):
    n, d = 6, 16 * 1024 + 37
    orc, gpu = make_pair(n, d, "complete", seed=5)
    rng = np.random.default_rng(900 + bits)
    orc.X[:] = _ranged_models(n, d, rng)
    inject(orc, gpu)
    for rnd in range(4):
        pairs = disjoint_pairs(orc, rng, 3)
        assert orc.interact(pairs, bits) == 0 and gpu.interact(pairs, bits) == 0
        assert_store_equal(orc, gpu, bits)


@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("bits", [2, 4, 7, 8])
def test_one_way_interactions_across_magnitude_ratios(bits, mode):
    """Single-buffer and two-register interactions on the same wide-ranged models, with and without pending
    local updates, including keys that moved away from what the buffers encode."""
    n, d = 6, 16 * 1024 + 37
    cfg = dict(objective=1, nonblocking=mode, grad_std=0.0, drift_std=0.0)
    orc, gpu = make_pair(n, d, "complete", seed=6, **cfg)
    rng = np.random.default_rng(950 + 10 * bits + mode)
    orc.X[:] = _ranged_models(n, d, rng)
    orc.B[:] = orc.X
    inject(orc, gpu)
    publish = (lambda s_: s_.publish(bits)) if mode == 1 else (lambda s_: s_.register_publish(bits))
    assert publish(orc) == 0 and publish(gpu) == 0
    assert_store_equal(orc, gpu, bits)
    for rnd in range(5):
        if rnd >= 2:                         # pending updates of very different relative sizes
            scale = np.float32(2.0 ** -(4 * rnd))
            orc.X[:] = (orc.X * (1.0 + scale * rng.normal(size=orc.X.shape))).astype(np.float32)
        if rnd == 4:                         # a snapshot far from its published encoding
            orc.B[0, 2048:4096] *= np.float32(1.5)
            orc.X[0] = orc.B[0]
        inject(orc, gpu, what=("X", "B"))
        pairs = disjoint_pairs(orc, rng, 3)
        assert orc.interact(pairs, bits, mode) == 0 and gpu.interact(pairs, bits, mode) == 0
        assert_store_equal(orc, gpu, bits)


def _large_scale_models(n, d, rng):
    """Models whose block ranges exceed the decoding window at step 1, so that lattice exponents are positive
    (1 ... 40), with magnitudes from the range itself up to 2^20 times it; every block also holds zeros, subnormals
    and tiny negative values, whose scaled values x * 2^-e are inexact products that round to -0 or to a subnormal."""
    nblk = (d + 1023) // 1024
    X = np.zeros((n, d), dtype=np.float32)
    tiny = np.array([0.0, -0.0, 1e-45, -1e-45, 3e-42, -3e-42, 1e-39, -1e-39, -2e-38, 1e-30, -1e-30], dtype=np.float32)
    for k in range(nblk):
        lo, hi = k * 1024, min(d, (k + 1) * 1024)
        spread = 2.0 ** (3 + 3 * (k % 13))
        base = (-1.0) ** k * spread * 2.0 ** (2 * (k % 11))
        X[:, lo:hi] = (base + spread * rng.normal(size=(n, hi - lo))).astype(np.float32)
        idx = rng.choice(hi - lo, size=min(24, hi - lo), replace=False)
        X[:, lo + idx] = tiny[rng.integers(0, len(tiny), size=(n, len(idx)))]
    return X


@pytest.mark.parametrize("mode", [0, 1, 2])
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_interactions_with_positive_lattice_exponents(bits, mode):
    """Blocks whose lattice step is 2, 4, ... 2^40: the scaled value is then no longer an exact product for tiny
    coordinates, and the kernels must round it exactly as the definition does before taking the floor."""
    n, d = 6, 14 * 1024 + 301
    cfg = dict(objective=1, nonblocking=mode, grad_std=0.0, drift_std=0.0)
    orc, gpu = make_pair(n, d, "complete", seed=8, **cfg)
    rng = np.random.default_rng(700 + 10 * bits + mode)
    orc.X[:] = _large_scale_models(n, d, rng)
    if mode:
        orc.B[:] = orc.X
    inject(orc, gpu)
    if mode:
        publish = (lambda s_: s_.publish(bits)) if mode == 1 else (lambda s_: s_.register_publish(bits))
        assert publish(orc) == 0 and publish(gpu) == 0
        assert_store_equal(orc, gpu, bits)
    assert int(orc.exps.max()) > 0 or mode == 0
    for rnd in range(4):
        if mode and rnd >= 1:                # pending updates, tiny coordinates included
            orc.X[:] = (orc.X * (1.0 + np.float32(2.0 ** -(3 * rnd)) * rng.normal(size=orc.X.shape))).astype(np.float32)
            inject(orc, gpu, what=("X",))
        pairs = disjoint_pairs(orc, rng, 3)
        assert orc.interact(pairs, bits, mode) == 0 and gpu.interact(pairs, bits, mode) == 0
        assert_store_equal(orc, gpu, bits)
    assert int(orc.exps.max()) > 3


# ---- two-register protocol -----------------------------------------------------------------------

@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("d", [5, 1024, 3001])
def test_register_protocol_bit_exact(bits, d):
    n = 6
    cfg = dict(objective=1, nonblocking=2, grad_std=0.03, drift_std=0.1, offset_std=0.2)
    orc, gpu = make_pair(n, d, "regular", 4, seed=70 + d, **cfg)
    inject(orc, gpu)
    assert orc.register_publish(bits) == 0 and gpu.register_publish(bits) == 0
    assert_store_equal(orc, gpu, bits)
    rng = np.random.default_rng(bits * 100 + d)
    for rnd in range(6):
        nodes = rng.permutation(n)[: int(rng.integers(1, n + 1))]
        assert orc.local_steps(nodes, 2, 0.05) == 0 and gpu.local_steps(nodes, 2, 0.05) == 0
        for i in nodes:
            assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL
        inject(orc, gpu, what=("X",))
        pairs = disjoint_pairs(orc, rng, int(rng.integers(1, 4)))
        assert orc.interact(pairs, bits, o.REGISTERS) == 0
        assert gpu.interact(pairs, bits, g.REGISTERS) == 0
        assert_store_equal(orc, gpu, bits)


@pytest.mark.parametrize("bits", [3, 8])
def test_register_protocol_with_8_bit_prefix_reads(bits):
    """Readers consume only the low-byte plane of their partner's own register (in range and aliasing alike)."""
    n, d = 6, 3001
    cfg = dict(objective=1, nonblocking=2, grad_std=0.03, drift_std=0.1, offset_std=0.2)
    orc, gpu = make_pair(n, d, "complete", seed=31, **cfg)
    inject(orc, gpu)
    assert orc.set_own_prefix(8) == 0 and gpu.set_own_prefix(8) == 0 and gpu.get_own_prefix() == 8
    assert gpu.set_own_prefix(12) == g.EINVAL
    rng = np.random.default_rng(bits)
    for rnd in range(8):
        nodes = rng.permutation(n)[:3]
        assert orc.local_steps(nodes, 2, 0.05) == 0 and gpu.local_steps(nodes, 2, 0.05) == 0
        inject(orc, gpu, what=("X",))
        pairs = disjoint_pairs(orc, rng, int(rng.integers(1, 4)))
        assert orc.interact(pairs, bits, o.REGISTERS) == 0
        assert gpu.interact(pairs, bits, g.REGISTERS) == 0
        assert_store_equal(orc, gpu, bits)
    # garbage in the high-byte planes of everybody else changes nothing for a prefix reader
    before = gpu.get(g.T_X, 0).copy()
    ref_pairs = [[0, 1]]
    orc_x = orc.X.copy()
    for i in range(1, n):
        row = gpu.get(g.T_OWN, i).reshape(-1, 2, 1024)
        row[:, 1, :] ^= 0x5A
        gpu.set(g.T_OWN, i, row.reshape(-1))
    assert orc.interact(ref_pairs, bits, o.REGISTERS) == 0 and gpu.interact(ref_pairs, bits, g.REGISTERS) == 0
    assert np.array_equal(gpu.get(g.T_X, 0).view(np.uint32), orc.X[0].view(np.uint32))
    gpu.configure(**cfg)
    assert gpu.get_own_prefix() == 16


@pytest.mark.parametrize("bits", [2, 5, 8])
def test_register_protocol_with_a_prefix_per_reader(bits):
    """Launches that mix 8-bit and 16-bit readers (each pair states its own prefix), near partners and far ones,
    in range and aliasing alike; more than 64 pairs per launch too (descriptors through the staging ring)."""
    n, d = 10, 3001
    cfg = dict(objective=1, nonblocking=2, grad_std=0.03, drift_std=0.1, offset_std=0.2)
    orc, gpu = make_pair(n, d, "complete", seed=33, **cfg)
    inject(orc, gpu)
    rng = np.random.default_rng(bits)
    for rnd in range(8):
        nodes = rng.permutation(n)[:4]
        assert orc.local_steps(nodes, 2, 0.05) == 0 and gpu.local_steps(nodes, 2, 0.05) == 0
        inject(orc, gpu, what=("X",))
        pairs = disjoint_pairs(orc, rng, int(rng.integers(1, 6)))
        prefixes = rng.choice([8, 16], size=len(pairs)).astype(np.int32)
        assert orc.interact_prefixed(pairs, prefixes, bits) == 0
        assert gpu.interact_prefixed(pairs, prefixes, bits) == 0
        assert_store_equal(orc, gpu, bits)
    # an 8-bit reader does not touch its partner's high bytes, the 16-bit reader in the same launch does
    valid = (np.arange(orc.nblk * 1024) < d).reshape(-1, 1024)       # not the padding behind coordinate d
    for i in range(n):
        row = gpu.get(g.T_OWN, i).reshape(-1, 2, 1024).copy()
        row[:, 1, :][valid] ^= 0x3C
        gpu.set(g.T_OWN, i, row.reshape(-1))
        orc.own_bytes[i] = row.reshape(-1)
    pairs, prefixes = [[0, 1], [2, 3]], [8, 16]
    x0 = orc.X[0].copy()
    assert orc.interact_prefixed(pairs, prefixes, bits) == 0 and gpu.interact_prefixed(pairs, prefixes, bits) == 0
    assert_store_equal(orc, gpu, bits)
    assert gpu.get_own_prefix() == 16
    # argument checks: nothing runs, nothing changes
    w_before = [tuple(gpu.get(g.T_COUNTERS, i)) for i in range(n)]
    assert gpu.interact_prefixed([[4, 5]], [12], bits) == g.EINVAL
    assert gpu._L.swarm_interact_prefixed(gpu._h, None, None, 1, bits) == g.EINVAL
    assert gpu.interact_prefixed([[4, 4]], [8], bits) == g.EPAIR
    assert [tuple(gpu.get(g.T_COUNTERS, i)) for i in range(n)] == w_before
    plain = g.Swarm(4, 64)
    plain.configure(objective=1, nonblocking=1)
    assert plain.interact_prefixed([[0, 1]], [8], 8) == g.ESTATE


def test_prefix_per_reader_in_a_launch_of_100_pairs():
    n, d, bits = 200, 1500, 4
    cfg = dict(objective=1, nonblocking=2, grad_std=0.03, offset_std=0.02)
    orc, gpu = make_pair(n, d, "regular", 6, seed=35, **cfg)
    inject(orc, gpu)
    rng = np.random.default_rng(5)
    for rnd in range(3):
        pairs = disjoint_pairs(orc, rng, 100)
        assert len(pairs) > 64
        prefixes = rng.choice([8, 16], size=len(pairs)).astype(np.int32)
        assert orc.interact_prefixed(pairs, prefixes, bits) == 0
        assert gpu.interact_prefixed(pairs, prefixes, bits) == 0
        assert_store_equal(orc, gpu, bits)


def test_register_protocol_mode_switches_and_far_snapshots():
    n, d = 4, 2100
    cfg = dict(objective=1, nonblocking=2, grad_std=0.0, drift_std=0.0, offset_std=0.05)
    orc, gpu = make_pair(n, d, "complete", seed=17, **cfg)
    inject(orc, gpu)
    seq = [([[0, 1]], 8, 2), ([[2, 3], [1, 0]], 8, 2), ([[0, 2]], 8, 1), ([[3, 1]], 8, 2), ([[1, 2]], 4, 2),
           ([[0, 3]], 4, 0), ([[2, 0]], 4, 2), ([[1, 3]], 32, 0), ([[3, 2]], 4, 2)]
    for pairs, bits, mode in seq:
        assert orc.interact(pairs, bits, mode) == 0 and gpu.interact(pairs, bits, mode) == 0
        assert_store_equal(orc, gpu, bits)
    # a snapshot moved outside the 16-bit window of its partner's own register: both sides alias alike
    orc.B[0] += np.float32(1000.0)
    orc.X[0] = orc.B[0]
    orc.B[1, :500] = np.float32(1e30)
    orc.X[1] = orc.B[1]
    inject(orc, gpu)
    for pairs in ([[0, 2]], [[1, 3]], [[2, 0], [3, 1]]):
        assert orc.interact(pairs, 4, o.REGISTERS) == 0 and gpu.interact(pairs, 4, g.REGISTERS) == 0
        assert_store_equal(orc, gpu, 4)
    plain = g.Swarm(4, 64)
    plain.configure(objective=1, nonblocking=1)
    assert plain.interact([[0, 1]], 8, g.REGISTERS) == -4 and plain.register_publish(8) == -4


# ---- local steps ---------------------------------------------------------------------------------

@pytest.mark.parametrize("d,H", [(3, 1), (4099, 3)])
def test_synthetic_gradient_steps_within_tolerance(d, H):
    cfg = dict(objective=1, grad_std=float(np.sqrt(1e-3)), drift_std=float(np.sqrt(0.05)))
    orc, gpu = make_pair(5, d, seed=21, **cfg)
    inject(orc, gpu)
    for rnd in range(3):
        assert orc.local_steps([4, 1, 2], H, 0.05) == 0 and gpu.local_steps([4, 1, 2], H, 0.05) == 0
        for i in range(5):
            assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL
        assert [gpu.get(g.T_COUNTERS, i)[1] for i in range(5)] == orc.ls.tolist()
    # untouched nodes are bit-identical
    assert np.array_equal(gpu.get(g.T_X, 0), orc.X[0]) and np.array_equal(gpu.get(g.T_X, 3), orc.X[3])


def test_gradient_noise_accuracy():
    """The local-step kernel draws its normals with the hardware approximations of lg2/sqrt/sin/cos.
    With x0 = 0, lr = grad_std = 1 and no drift the model after one step is -z, which exposes the
    absolute error of the normals: it must stay at a few 1e-6 (including u1 next to 1, where the
    radius comes from a series)."""
    cfg = dict(objective=1, grad_std=1.0, drift_std=0.0, init_std=0.0)
    orc, gpu = make_pair(2, 400_000, seed=77, **cfg)
    assert orc.local_steps([0, 1], 1, 1.0) == 0 and gpu.local_steps([0, 1], 1, 1.0) == 0
    for i in range(2):
        got, ref = gpu.get(g.T_X, i), orc.X[i]
        err = np.abs(got - ref)
        print("normal abs error: max %.3e mean %.3e" % (err.max(), err.mean()))
        assert err.max() < 1e-5
        assert np.abs(ref).max() > 4.0
        # exact zeros of the reference (u1 = 1 or angle 0) aside, tiny normals keep their sign and scale
        tiny = (np.abs(ref) < 1e-3) & (ref != 0)
        assert tiny.sum() > 100 and np.all(np.sign(got[tiny]) == np.sign(ref[tiny]))


@pytest.mark.parametrize("d,m,batch,dtype,groups", [(4096, 64, 16, 0, 0), (5000, 12, 5, 0, 0), (9000, 32, 64, 1, 2),
                                                   (300, 8, 3, 1, 0)])
def test_least_squares_steps_within_tolerance(d, m, batch, dtype, groups):
    cfg = dict(objective=2, lsq_m=m, lsq_batch=batch, lsq_dtype=dtype, lsq_groups=groups,
               lsq_noise_std=float(np.sqrt(0.1)))
    orc, gpu = make_pair(4, d, seed=31, **cfg)
    inject(orc, gpu)
    for rnd in range(3):
        nodes = [0, 3, 1] if rnd else [2]
        assert orc.local_steps(nodes, 2, 0.05) == 0 and gpu.local_steps(nodes, 2, 0.05) == 0
        for i in range(4):
            assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL, (rnd, i)
        inject(orc, gpu, what=("X",))


@pytest.mark.parametrize("n,groups,d,m,batch", [(20, 1, 9000, 40, 64), (6, 3, 40000, 16, 7), (32, 2, 33000, 128, 64),
                                                (4, 0, 1500, 9, 33)])
def test_batched_tensor_core_least_squares_steps(n, groups, d, m, batch):
    """bf16 data: nodes that share a data matrix and a step counter are batched into tensor-core units of up
    to 16 (here: more than 16 per matrix, ragged units, mixed counters, batches below the 64-row tile,
    several k-chunks)."""
    cfg = dict(objective=2, lsq_m=m, lsq_batch=batch, lsq_dtype=1, lsq_groups=groups, lsq_noise_std=0.3)
    orc, gpu = make_pair(n, d, seed=51, **cfg)
    inject(orc, gpu)
    rng = np.random.default_rng(n)
    schedule = [list(range(n)), sorted(rng.permutation(n)[: max(1, n // 2)].tolist()), list(range(n))[::-1]]
    for nodes in schedule:
        assert orc.local_steps(nodes, 3, 0.05) == 0 and gpu.local_steps(nodes, 3, 0.05) == 0
        gpu.sync()
        for i in range(n):
            assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL, i
            assert gpu.get(g.T_COUNTERS, i)[1] == orc.ls[i]
        inject(orc, gpu, what=("X",))


@pytest.mark.parametrize("H,objective", [(1, 2), (4, 2), (5, 2), (7, 2), (9, 2), (4, 3), (6, 3)])
def test_tensor_core_steps_folded_four_at_a_time(H, objective):
    """bf16 data: up to four consecutive steps of a unit share one pass for the scores (against the model before
    the first of them, corrected step by step through blocks of the data's Gram matrix) and one pass for the
    updates. Every split of H into groups (4, 4 + 1, 4 + 3, 4 + 4 + 1) must give the oracle's H separate steps.
    Fewer rows than a minibatch draws, so that minibatches share rows and the corrections are large; a step size
    ten times the usual one; the second data matrix rewritten through swarm_set_tensor (its Gram matrix follows)."""
    n, d = 20, 17000
    cfg = dict(objective=objective, lsq_m=48, lsq_batch=64, lsq_dtype=1, lsq_groups=2, lsq_noise_std=0.3, init_std=0.5)
    orc, gpu = make_pair(n, d, seed=97, **cfg)
    orc.A[1] = (2.0 * orc.A[1][::-1]).astype(np.float32)          # exact in bf16
    inject(orc, gpu)
    lr = 0.5
    for nodes in (list(range(n)), [3, 17, 4, 11, 12]):
        assert orc.local_steps(nodes, H, lr) == 0 and gpu.local_steps(nodes, H, lr) == 0
        gpu.sync()
        for i in range(n):
            assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL, i
            assert gpu.get(g.T_COUNTERS, i)[1] == orc.ls[i]
        inject(orc, gpu, what=("X",))


@pytest.mark.parametrize("d,batch,H,objective", [(700, 5, 2, 2), (4096, 16, 3, 2), (4096, 16, 5, 3), (6000, 8, 4, 2),
                                                 (6000, 9, 4, 2), (8192, 8, 7, 3), (3000, 16, 10, 2)])
def test_short_model_steps_taken_two_per_round(d, batch, H, objective):
    """fp32 data, short models: where a minibatch fits the rows a thread keeps in flight (16 rows up to a row
    pitch of 4096, 8 above) the cluster kernel takes two steps per round, the second step's inner products
    corrected through the data's Gram matrix; an odd H ends with a round of one step, H > 8 crosses the window in
    which minibatches are drawn ahead, batch 9 at the longer pitch stays one step per round. Fewer data rows than
    two minibatches draw, so that the corrections are large, and a step size ten times the usual one."""
    n, m = 6, 20
    cfg = dict(objective=objective, lsq_m=m, lsq_batch=batch, lsq_dtype=0, lsq_groups=0, lsq_noise_std=0.3, init_std=0.5)
    orc, gpu = make_pair(n, d, seed=131, **cfg)
    orc.A[2] = (2.0 * orc.A[2][::-1]).astype(np.float32)          # rewritten data: the Gram matrix follows
    inject(orc, gpu)
    lr = 0.5
    for nodes in (list(range(n)), [4, 2]):
        assert orc.local_steps(nodes, H, lr) == 0 and gpu.local_steps(nodes, H, lr) == 0
        gpu.sync()
        for i in range(n):
            assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL, i
            assert gpu.get(g.T_COUNTERS, i)[1] == orc.ls[i]
        inject(orc, gpu, what=("X",))


@pytest.mark.parametrize("d,m,dtype,groups", [(700, 48, 1, 2), (9000, 130, 1, 3), (70000, 300, 1, 1), (3000, 129, 1, 0),
                                              (4096, 20, 0, 0), (8000, 70, 0, 2)])
def test_gram_matrices_of_the_data(d, m, dtype, groups):
    """The Gram matrices that the folded local steps read, against A A^T in double from the oracle's copy of the
    data: bf16 data on the tensor cores (one, two and three 128-row tiles, ragged last tiles, off-diagonal tiles,
    rows shorter and longer than one accumulation run of 8192 coordinates), fp32 data of short models on the CUDA
    cores; and again after one matrix has been rewritten."""
    n = 6
    cfg = dict(objective=2, lsq_m=m, lsq_batch=8, lsq_dtype=dtype, lsq_groups=groups, lsq_noise_std=0.1)
    orc, gpu = make_pair(n, d, seed=77, **cfg)
    inject(orc, gpu)
    ngroups = groups if groups else n

    def check():
        for grp in range(ngroups):
            A = orc.A[grp].astype(np.float64)
            want = A @ A.T
            got = gpu.get(g.T_GRAM, grp).reshape(m, m)
            assert np.array_equal(got, got.T), grp
            # tensor cores: runs of 128 fp32 accumulations in tensor memory, each off by up to 2^-24 of the running
            # sum in one direction, then double; CUDA cores: fp32 runs of 1024 products rounded to nearest, then double
            assert np.abs(got - want).max() < (8e-6 if dtype == 1 else 1e-6) * np.abs(want).max(), grp
    check()
    last = ngroups - 1
    orc.A[last] = (0.5 * orc.A[last][::-1]).astype(np.float32)        # exact in bf16
    gpu.set(g.T_A, last, orc.A[last])
    check()
    assert gpu._L.swarm_get_tensor(gpu._h, g.T_GRAM, ngroups, np.empty(m * m, np.float32).ctypes.data, m * m * 4) == g.ERANGE
    assert gpu._L.swarm_set_tensor(gpu._h, g.T_GRAM, 0, np.zeros(m * m, np.float32).ctypes.data, m * m * 4) == g.EINVAL


def test_tensor_core_steps_one_at_a_time_when_the_gram_matrix_is_not_kept():
    """A data matrix of 8200 rows: its Gram matrix (269 MB) is above what the library keeps, so the steps take
    one pair of passes each; same results within the tolerance."""
    n, d = 4, 1024
    cfg = dict(objective=2, lsq_m=8200, lsq_batch=64, lsq_dtype=1, lsq_groups=1, lsq_noise_std=0.3)
    orc, gpu = make_pair(n, d, seed=98, **cfg)
    inject(orc, gpu)
    launches = gpu.kernel_launches()
    assert orc.local_steps([0, 1, 2, 3], 3, 0.2) == 0 and gpu.local_steps([0, 1, 2, 3], 3, 0.2) == 0
    gpu.sync()
    assert gpu.kernel_launches() - launches == 9                           # three kernels per step
    for i in range(n):
        assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL, i


@pytest.mark.parametrize("d,m,batch,dtype,groups", [(4096, 64, 16, 0, 0), (20000, 24, 40, 0, 2), (33000, 64, 64, 1, 2),
                                                   (700, 12, 5, 1, 0)])
def test_logistic_regression_steps_within_tolerance(d, m, batch, dtype, groups):
    """Second objective on the least-squares data: residual sigmoid(<a, x>) - y, through the cluster kernel
    (short models), the general kernels and the tensor-core kernels."""
    cfg = dict(objective=3, lsq_m=m, lsq_batch=batch, lsq_dtype=dtype, lsq_groups=groups, lsq_noise_std=0.2,
               init_std=0.5)
    orc, gpu = make_pair(4, d, seed=83, **cfg)
    labels = gpu.get_all(g.T_BVEC)
    assert set(np.unique(labels).tolist()) <= {0.0, 1.0}
    assert (labels != orc.bvec).mean() < 0.02                     # a score next to zero may flip a class
    inject(orc, gpu)
    for rnd in range(3):
        nodes = [0, 3, 1] if rnd else [2, 0]
        assert orc.local_steps(nodes, 2, 0.5) == 0 and gpu.local_steps(nodes, 2, 0.5) == 0
        gpu.sync()
        for i in range(4):
            assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL, (rnd, i)
        inject(orc, gpu, what=("X",))


def test_geometric_step_counts_match():
    cfg = dict(objective=1, grad_std=0.03, drift_std=0.1)
    orc, gpu = make_pair(12, 3000, seed=61, **cfg)
    inject(orc, gpu)
    for rnd in range(4):
        nodes = list(range(12)) if rnd % 2 == 0 else [5, 1, 9]
        rc_o, steps_o = orc.local_steps_geometric(nodes, 3, 0.05)
        rc_g, steps_g = gpu.local_steps_geometric(nodes, 3, 0.05)
        assert rc_o == 0 and rc_g == 0
        assert np.array_equal(steps_o, steps_g)                    # integer draws: bit-exact
        for i in range(12):
            assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < TOL
            assert gpu.get(g.T_COUNTERS, i)[1] == orc.ls[i]
        inject(orc, gpu, what=("X",))
    assert gpu.local_steps_geometric([0], 0, 0.1)[0] == -1


# ---- mean model and potential ----------------------------------------------------------------------

@pytest.mark.parametrize("n,d", [(2, 1), (3, 1027), (8, 4096), (17, 2500), (64, 3000)])
def test_mean_model_and_potential(n, d):
    orc, gpu = make_pair(n, d, seed=n, offset_std=0.5)
    inject(orc, gpu)
    mu = gpu.mean_model().cpu().numpy()
    assert np.array_equal(mu, orc.mean_model())
    assert abs(gpu.potential() - orc.potential()) <= 1e-12 * orc.potential()
    # models far from the origin but close together: the subtraction must stay benign
    orc.X[:] = (1000.0 + 1e-3 * np.random.default_rng(0).normal(size=(n, d))).astype(np.float32)
    inject(orc, gpu, what=("X",))
    assert abs(gpu.potential() - orc.potential()) <= 1e-9 * orc.potential()
    orc.X[:] = orc.X[0]
    inject(orc, gpu, what=("X",))
    assert gpu.potential() == 0.0 and orc.potential() == 0.0


# ---- error behaviour -------------------------------------------------------------------------------

def test_rejected_calls_change_nothing():
    orc, gpu = make_pair(6, 2000, "ring", seed=4, objective=1, grad_std=0.1)
    inject(orc, gpu)
    before = gpu.get_all(g.T_X)
    launches = gpu.kernel_launches()
    assert gpu.interact([[0, 1], [1, 2]], 8) == -3
    assert gpu.interact([[0, 0]], 8) == -3
    assert gpu.interact([[0, 3]], 8) == -3
    assert gpu.interact([[0, 6]], 8) == -2
    assert gpu.interact([[0, 1]], 1) == -1 and gpu.interact([[0, 1]], 9) == -1 and gpu.interact([[0, 1]], 16) == -1
    assert gpu.interact([[0, 1]], 8, 3) == -1
    assert gpu.interact([[0, 1]], 8, g.REGISTERS) == -4
    assert gpu.interact([[0, 1]], 32, g.NONBLOCKING) == -1
    assert gpu.interact([[0, 1]], 8, g.NONBLOCKING) == -4
    assert gpu.publish(8) == -4
    assert gpu.local_steps([0, 0], 1, 0.1) == -1
    assert gpu.local_steps([6], 1, 0.1) == -2
    assert gpu.local_steps([0], -1, 0.1) == -1
    assert gpu.kernel_launches() == launches
    assert np.array_equal(gpu.get_all(g.T_X), before)
    assert [tuple(gpu.get(g.T_COUNTERS, i)) for i in range(6)] == [(0, 0, 0)] * 6
    gpu2 = g.Swarm(4, 16)
    assert gpu2.local_steps([0], 1, 0.1) == -4
    for bad in (dict(topology="ring", n=2), dict(topology="regular", n=8, degree=3)):
        with pytest.raises(g.SwarmError):
            g.Swarm(bad["n"], 16, bad["topology"], bad.get("degree", 0))
    assert gpu.interact([], 8) == 0 and gpu.local_steps([], 3, 0.1) == 0
