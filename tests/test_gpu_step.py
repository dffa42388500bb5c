"""swarm_step (Algorithm 1's whole step; local steps fused into the blocking and single-buffer interaction
kernels) against the oracle and against the two-call sequence it must reproduce bit for bit."""
import numpy as np
import pytest

from oracle import swarm_oracle as o
from paper_1910_12308_b200 import binding as g
from parity import assert_store_equal, inject, make_pair

pytestmark = pytest.mark.gpu

ROWS = (g.T_X, g.T_B, g.T_CODES, g.T_EXPS, g.T_OWN, g.T_OEXPS, g.T_COUNTERS, g.T_CLOCKS)


def assert_contexts_equal(a, b):
    for i in range(a.n):
        for which in ROWS:
            try:
                ra = a.get(which, i)
            except g.SwarmError:
                continue
            rb = b.get(which, i)
            assert np.array_equal(ra.view(np.uint8), rb.view(np.uint8)), f"tensor {which} of node {i} differs"
    assert a.get_state() == b.get_state() and a.get_buffer_mode() == b.get_buffer_mode()


def stepped(pairs, responders):
    return [p[0] for p in pairs] + ([p[1] for p in pairs] if responders else [])


@pytest.mark.parametrize("responders", [True, False])
@pytest.mark.parametrize("mode,bits", [(0, 4), (0, 8), (0, 32), (0, 5), (1, 8), (1, 3), (2, 8), (2, 4)])
@pytest.mark.parametrize("d", [1030, 5000])
def test_fused_step_equals_local_steps_then_interact(mode, bits, d, responders):
    n = 6
    cfg = dict(objective=1, nonblocking=mode, grad_std=0.05, drift_std=0.3, offset_std=0.2)
    two = g.Swarm(n, d, "complete", 0, 11)
    one = g.Swarm(n, d, "complete", 0, 11)
    two.configure(**cfg)
    one.configure(**cfg)
    rng = np.random.default_rng(d + bits)
    for rnd in range(4):
        perm = rng.permutation(n)
        pairs = [[int(perm[0]), int(perm[1])], [int(perm[2]), int(perm[3])]][: 1 + rnd % 2]
        H = 1 + rnd % 3
        assert two.local_steps(stepped(pairs, responders), H, 0.05) == 0
        assert two.interact(pairs, bits, mode) == 0
        launches = one.kernel_launches()
        assert one.step(pairs, H, 0.05, bits, mode, responders) == 0
        if rnd > 0:
            # one kernel does the whole step; the two-register exchange keeps its local steps in a kernel of their own
            assert one.kernel_launches() - launches == (2 if mode == g.REGISTERS else 1)
        assert_contexts_equal(one, two)


@pytest.mark.parametrize("mode,bits", [(0, 4), (1, 8), (2, 6)])
def test_fused_step_against_the_oracle_with_noise_free_gradients(mode, bits):
    """grad_std = 0 keeps the local step free of transcendental arithmetic, so the whole step is bit-exact."""
    n, d = 6, 4100
    orc, gpu = make_pair(n, d, "complete", seed=3, objective=1, nonblocking=mode, grad_std=0.0, drift_std=0.4,
                         offset_std=0.2)
    inject(orc, gpu)
    rng = np.random.default_rng(bits)
    for rnd in range(5):
        perm = rng.permutation(n)
        pairs = [[int(perm[0]), int(perm[1])], [int(perm[2]), int(perm[3])]]
        assert orc.local_steps(stepped(pairs, True), 2, 0.1) == 0
        assert orc.interact(pairs, bits, mode) == 0
        assert gpu.step(pairs, 2, 0.1, bits, mode, True) == 0
        assert_store_equal(orc, gpu, bits)


def test_step_after_a_blocking_exchange_refreshes_snapshots_like_the_two_calls():
    n, d = 4, 3000
    cfg = dict(objective=1, nonblocking=1, grad_std=0.05, drift_std=0.3, offset_std=0.2)
    two = g.Swarm(n, d, "complete", 0, 5)
    one = g.Swarm(n, d, "complete", 0, 5)
    for sw in (two, one):
        sw.configure(**cfg)
        assert sw.interact([[0, 1], [2, 3]], 8, g.BLOCKING) == 0      # leaves the snapshots stale
    assert two.local_steps([0, 2], 2, 0.05) == 0 and two.interact([[0, 2]], 8, g.NONBLOCKING) == 0
    assert one.step([[0, 2]], 2, 0.05, 8, g.NONBLOCKING, True) == 0
    assert_contexts_equal(one, two)


def test_step_with_least_squares_is_the_two_calls_in_sequence():
    n, d = 4, 2500
    cfg = dict(objective=2, nonblocking=0, lsq_m=32, lsq_batch=8, lsq_dtype=0, lsq_groups=0, lsq_noise_std=0.1)
    two = g.Swarm(n, d, "complete", 0, 9)
    one = g.Swarm(n, d, "complete", 0, 9)
    two.configure(**cfg)
    one.configure(**cfg)
    for pairs in ([[0, 1]], [[2, 3], [1, 0]]):
        assert two.local_steps(stepped(pairs, True), 2, 0.05) == 0 and two.interact(pairs, 8) == 0
        assert one.step(pairs, 2, 0.05, 8, g.BLOCKING, True) == 0
        assert_contexts_equal(one, two)


def test_step_errors_leave_the_models_untouched():
    gpu = g.Swarm(4, 2000, "ring", 0, 1)
    assert gpu.step([[0, 1]], 2, 0.1, 8) == g.ESTATE               # no objective configured
    assert gpu.step([[0, 1]], 0, 0.1, 8) == 0                      # H = 0 is a plain interaction
    gpu.configure(objective=1, grad_std=0.1)
    before = [gpu.get(g.T_X, i) for i in range(4)]
    assert gpu.step([[0, 2]], 2, 0.1, 8) == g.EPAIR                # not an edge of the ring
    assert gpu.step([[0, 1]], 2, 0.1, 9) == g.EINVAL
    assert gpu.step([[0, 1]], -1, 0.1, 8) == g.EINVAL
    assert gpu.step([[0, 1]], 2, 0.1, 8, g.NONBLOCKING) == g.ESTATE
    for i in range(4):
        assert np.array_equal(gpu.get(g.T_X, i), before[i])
    assert gpu.get(g.T_COUNTERS, 0)[1] == 0
