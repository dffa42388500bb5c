"""CUDA path against the oracle: auxiliary potentials Gamma-hat, A_t, B_t of the staleness analysis
(appendix, "Notation and Auxiliary Potential Functions")."""
import numpy as np
import pytest

from oracle import swarm_oracle as o
from paper_1910_12308_b200 import binding as g
from parity import assert_store_equal, inject, make_pair

pytestmark = pytest.mark.gpu

# double sums in another order than the oracle's
REL = 1e-11


def assert_records_equal(orc, gpu):
    for i in range(orc.n):
        assert np.array_equal(gpu.get(g.T_MU_RECORD, i).view(np.uint32), orc.mu_hist[i].view(np.uint32)), f"mean record[{i}]"
        assert float(gpu.get(g.T_A_RECORD, i)[0]) == pytest.approx(float(orc.a_hist[i]), rel=REL), f"A term[{i}]"


@pytest.mark.parametrize("mode,d", [(o.NONBLOCKING, 2100), (o.REGISTERS, 5000), (o.NONBLOCKING, 70001)])
def test_aux_potentials_follow_the_oracle_along_a_trajectory(mode, d):
    n = 6
    orc, gpu = make_pair(n, d, "complete", seed=5, objective=1, nonblocking=mode, grad_std=0.05, drift_std=0.3,
                         offset_std=0.2)
    inject(orc, gpu)
    assert orc.track_staleness(True) == 0 and gpu.track_staleness(True) == 0
    assert_records_equal(orc, gpu)
    for q, w in zip(gpu.aux_potentials(), orc.aux_potentials()):
        assert q == pytest.approx(w, rel=REL, abs=1e-300)
    rng = np.random.default_rng(1)
    for step in range(6):
        if step % 2 == 0:
            a, b = rng.choice(n, size=2, replace=False)
            pairs = [[int(a), int(b)]]
        else:
            perm = rng.permutation(n)
            pairs = [[int(perm[0]), int(perm[1])], [int(perm[2]), int(perm[3])]]
        nodes = [p[0] for p in pairs]
        orc.local_steps(nodes, 2, 0.05)
        gpu.local_steps(nodes, 2, 0.05)
        inject(orc, gpu, what=("X",))                     # normals differ in the last bit: teacher forcing
        assert orc.interact(pairs, 8, mode) == 0
        assert gpu.interact(pairs, 8, mode) == 0
        assert_store_equal(orc, gpu, bits=8)
        assert_records_equal(orc, gpu)
        got, want = gpu.aux_potentials(), orc.aux_potentials()
        for q, w in zip(got, want):
            assert q == pytest.approx(w, rel=REL)
        assert got[0] <= 2 * got[1] + 2 * got[2]
    assert min(got) > 0.0


def test_tracking_state_rules():
    gpu = g.Swarm(4, 3000, "complete", seed=0)
    gpu.configure(objective=1, nonblocking=0)
    assert gpu.track_staleness(True) == g.ESTATE
    with pytest.raises(g.SwarmError):
        gpu.aux_potentials()
    gpu.configure(objective=1, nonblocking=1, offset_std=0.1)
    assert gpu.track_staleness(True) == 0
    gh, a, b = gpu.aux_potentials()
    assert b == 0.0 and gh == pytest.approx(a, rel=1e-12) and gh == pytest.approx(gpu.potential(), rel=1e-5)
    assert gpu.interact([[0, 1]], 8, g.BLOCKING) == g.ESTATE
    assert gpu.track_staleness(False) == 0
    assert gpu.interact([[0, 1]], 8, g.BLOCKING) == 0
    assert gpu.track_staleness(True) == g.ESTATE        # snapshots are stale after a blocking exchange
    gpu.configure(objective=1, nonblocking=1)           # a new configuration drops the records
    with pytest.raises(g.SwarmError):
        gpu.get(g.T_MU_RECORD, 0)


def test_more_initiators_than_one_descriptor_slice():
    n, d = 160, 1500
    orc, gpu = make_pair(n, d, "ring", seed=2, objective=1, nonblocking=1, offset_std=0.2, drift_std=0.1)
    inject(orc, gpu)
    orc.track_staleness(True); gpu.track_staleness(True)
    pairs = [[2 * t, 2 * t + 1] for t in range(n // 2)]          # 80 initiators in one launch
    orc.local_steps(list(range(0, n, 2)), 1, 0.1)
    gpu.local_steps(list(range(0, n, 2)), 1, 0.1)
    inject(orc, gpu, what=("X",))
    assert orc.interact(pairs, 4, o.NONBLOCKING) == 0
    assert gpu.interact(pairs, 4, o.NONBLOCKING) == 0
    assert_records_equal(orc, gpu)
    for q, w in zip(gpu.aux_potentials(), orc.aux_potentials()):
        assert q == pytest.approx(w, rel=REL)
