"""swarm_run_sequence (sequential gossip, Section 3 "Sequential model"; one kernel launch for short models)
against the step-by-step calls it must reproduce bit for bit, and against the oracle."""
import numpy as np
import pytest

from oracle import swarm_oracle as o
from paper_1910_12308_b200 import binding as g
from parity import inject, make_pair

pytestmark = pytest.mark.gpu

ROWS = (g.T_X, g.T_CODES, g.T_EXPS, g.T_COUNTERS, g.T_CLOCKS)
LSQ = dict(objective=2, lsq_m=64, lsq_batch=16, lsq_dtype=0, lsq_groups=0, lsq_noise_std=0.3)


def assert_contexts_equal(a, b):
    for i in range(a.n):
        for which in ROWS:
            assert np.array_equal(a.get(which, i).view(np.uint8), b.get(which, i).view(np.uint8)), \
                f"tensor {which} of node {i} differs"
    assert a.get_state() == b.get_state() and a.get_buffer_mode() == b.get_buffer_mode()


def random_sequence(n, steps, seed):
    rng = np.random.default_rng(seed)
    return [[int(v) for v in rng.choice(n, size=2, replace=False)] for _ in range(steps)]


@pytest.mark.parametrize("responders", [True, False])
@pytest.mark.parametrize("d,bits,steps", [(4096, 8, 150), (1500, 3, 40), (8192, 4, 30), (5000, 8, 70), (700, 6, 10),
                                           (900, 2, 12), (2100, 5, 12), (3000, 7, 12)])
def test_sequence_equals_the_steps_one_by_one(d, bits, steps, responders):
    n = 8
    two = g.Swarm(n, d, "complete", 0, 21)
    one = g.Swarm(n, d, "complete", 0, 21)
    cfg = dict(LSQ, objective=2 if d != 1500 else 3)
    two.configure(**cfg)
    one.configure(**cfg)
    seq = random_sequence(n, steps, d)
    for a, b in seq:
        assert two.local_steps([a, b] if responders else [a], 2, 0.05) == 0
        assert two.interact([[a, b]], bits) == 0
    assert one.run_sequence(seq, 2, 0.05, bits, responders) == 0
    assert_contexts_equal(one, two)
    # and the contexts keep agreeing when used further
    for sw in (one, two):
        assert sw.local_steps([0, 1], 1, 0.05) == 0 and sw.interact([[0, 1]], bits) == 0
    assert_contexts_equal(one, two)


def test_sequence_is_one_launch_for_the_8_node_case():
    sw = g.Swarm(8, 4096, "complete", 0, 0)
    sw.configure(**LSQ)
    seq = random_sequence(8, 64, 1)
    before = sw.kernel_launches()
    assert sw.run_sequence(seq, 2, 0.05, 8) == 0
    assert sw.kernel_launches() - before == 1


def test_sequence_against_the_oracle_within_a_few_lattice_steps():
    """Least-squares steps differ from the oracle's double accumulation in the last fp32 bits, so codes may
    round differently: models agree to a few lattice steps, and the swarm contracts alike."""
    n, d = 8, 4096
    orc, gpu = make_pair(n, d, "complete", seed=6, **LSQ)
    inject(orc, gpu)
    seq = random_sequence(n, 40, 9)
    for a, b in seq:
        assert orc.local_steps([a, b], 2, 0.05) == 0 and orc.interact([[a, b]], 8) == 0
    assert gpu.run_sequence(seq, 2, 0.05, 8) == 0
    step = 2.0 ** float(orc.exps.max())
    for i in range(n):
        assert np.abs(gpu.get(g.T_X, i).astype(np.float64) - orc.X[i]).max() <= 4 * step
        w, ls, pb = gpu.get(g.T_COUNTERS, i)
        assert (w, ls, pb) == (orc.w[i], orc.ls[i], orc.pbits[i])
        assert tuple(gpu.get(g.T_CLOCKS, i)) == (orc.wo[i], orc.tau[i])
    assert gpu.potential() == pytest.approx(orc.potential(), rel=0.05)


@pytest.mark.parametrize("H,lr", [(0, 0.05), (2, 0.0)])
@pytest.mark.parametrize("d,bits", [(4096, 8), (1500, 3), (8192, 4), (700, 2)])
def test_sequence_of_pure_interactions_matches_the_oracle_bit_for_bit(d, bits, H, lr):
    """Without local steps (H = 0), or with steps of size zero, a sequence is a chain of blocking interactions on
    shared nodes: everything in it is exact or a single rounding, so the single launch must reproduce the oracle's
    models, codes, exponents and counters bit for bit."""
    n = 8
    orc, gpu = make_pair(n, d, "complete", seed=8, **LSQ)
    inject(orc, gpu)
    seq = random_sequence(n, 90, d + bits)
    for a, b in seq:
        if H > 0:
            assert orc.local_steps([a, b], H, lr) == 0
        assert orc.interact([[a, b]], bits) == 0
    before = gpu.kernel_launches()
    assert gpu.run_sequence(seq, H, lr, bits, True) == 0
    assert gpu.kernel_launches() - before == 2          # 64 steps per launch
    for i in range(n):
        assert np.array_equal(gpu.get(g.T_X, i).view(np.uint32), orc.X[i].view(np.uint32)), i
        nbytes = orc.nblk * 128 * bits
        assert np.array_equal(gpu.get(g.T_CODES, i)[:nbytes], orc.codes[i, :nbytes]), i
        assert np.array_equal(gpu.get(g.T_EXPS, i), orc.exps[i]), i
        assert tuple(gpu.get(g.T_COUNTERS, i)) == (orc.w[i], orc.ls[i], orc.pbits[i])
        assert tuple(gpu.get(g.T_CLOCKS, i)) == (orc.wo[i], orc.tau[i])
    assert gpu.potential() == pytest.approx(orc.potential(), rel=1e-9)


def test_sequence_falls_back_to_single_steps_elsewhere():
    n, d = 6, 3000
    for cfg, bits in ((dict(objective=1, grad_std=0.05, drift_std=0.2), 8), (dict(LSQ), 32),
                      (dict(LSQ, lsq_dtype=1), 8)):
        two = g.Swarm(n, d, "complete", 0, 4)
        one = g.Swarm(n, d, "complete", 0, 4)
        two.configure(**cfg)
        one.configure(**cfg)
        seq = random_sequence(n, 6, 2)
        for a, b in seq:
            assert two.step([[a, b]], 2, 0.05, bits, g.BLOCKING, True) == 0
        assert one.run_sequence(seq, 2, 0.05, bits) == 0
        assert_contexts_equal(one, two)


def test_sequence_errors_leave_everything_untouched():
    sw = g.Swarm(6, 2000, "ring", 0, 3)
    sw.configure(**LSQ)
    before = [sw.get(g.T_X, i) for i in range(6)]
    assert sw.run_sequence([[0, 1], [1, 2], [0, 3]], 2, 0.05, 8) == g.EPAIR      # (0, 3) is no edge of the ring
    assert sw.run_sequence([[0, 1], [1, 7]], 2, 0.05, 8) == g.ERANGE
    assert sw.run_sequence([[0, 1]], 2, 0.05, 9) == g.EINVAL
    assert sw.run_sequence([[0, 1]], -1, 0.05, 8) == g.EINVAL
    assert sw.run_sequence([], 2, 0.05, 8) == 0
    for i in range(6):
        assert np.array_equal(sw.get(g.T_X, i), before[i])
        assert tuple(sw.get(g.T_COUNTERS, i)) == (0, 0, 0)
    sw.configure(**dict(LSQ, nonblocking=1))
    assert sw.track_staleness(True) == 0
    assert sw.run_sequence([[0, 1]], 2, 0.05, 8) == g.ESTATE
