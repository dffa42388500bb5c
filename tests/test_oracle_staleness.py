"""Pins for the auxiliary potentials of the staleness analysis (appendix, "Notation and Auxiliary
Potential Functions"): Gamma-hat_t = sum_i ||X^_i - mu_t||^2, A_t = sum_i ||X_{t-tau_i} - mu_{t-tau_i}||^2,
B_t = sum_i ||mu_t - mu_{t-tau_i}||^2, and the inequality Gamma-hat <= 2 A + 2 B that ties them."""
import numpy as np
import pytest

from oracle import swarm_oracle as o


def make(mode, n=6, d=1500, seed=3, **kw):
    s = o.OracleSwarm(n, d, "complete", seed=seed)
    cfg = dict(objective=1, nonblocking=mode, grad_std=0.05, drift_std=0.3, offset_std=0.2)
    cfg.update(kw)
    s.configure(**cfg)
    return s


class History:
    """The definitions, written out with numpy in double from the trajectory alone."""

    def __init__(self, s):
        self.s = s
        mu = s.X.astype(np.float64).mean(axis=0)
        self.mu_then = [mu.copy() for _ in range(s.n)]
        self.x_then = [s.B[i].astype(np.float64).copy() for i in range(s.n)]

    def after_interaction(self, initiator):
        mu = self.s.X.astype(np.float64).mean(axis=0)
        self.mu_then[initiator] = mu
        self.x_then[initiator] = self.s.X[initiator].astype(np.float64).copy()   # X^ <- X at an initiation

    def potentials(self):
        mu = self.s.X.astype(np.float64).mean(axis=0)
        gh = sum(np.sum((self.x_then[i] - mu) ** 2) for i in range(self.s.n))
        a = sum(np.sum((self.x_then[i] - self.mu_then[i]) ** 2) for i in range(self.s.n))
        b = sum(np.sum((mu - self.mu_then[i]) ** 2) for i in range(self.s.n))
        return gh, a, b


@pytest.mark.parametrize("mode", [o.NONBLOCKING, o.REGISTERS])
def test_aux_potentials_match_their_definitions_along_a_trajectory(mode):
    s = make(mode)
    assert s.track_staleness(True) == 0
    ref = History(s)
    rng = np.random.default_rng(0)
    for step in range(25):
        a, b = rng.choice(s.n, size=2, replace=False)
        s.local_steps([int(a)], 2, 0.05)
        assert s.interact([[int(a), int(b)]], 8, mode) == 0
        ref.after_interaction(int(a))
        got = s.aux_potentials()
        want = ref.potentials()
        # the oracle rounds the mean model to fp32 (it is the mean-model routine's output): 1e-6 relative
        for g, w in zip(got, want):
            assert g == pytest.approx(w, rel=2e-6, abs=1e-9)
        assert got[0] <= 2.0 * got[1] + 2.0 * got[2] + 1e-12      # Cauchy-Schwarz bound on Gamma-hat
        assert np.array_equal(s.B[int(a)], s.X[int(a)])            # the snapshot is the model after an initiation
    # the trajectory really exercises all three: none of them is trivially zero
    assert min(got) > 0.0


def test_fresh_tracking_makes_b_zero_and_gamma_hat_equal_a():
    s = make(o.NONBLOCKING)
    s.track_staleness(True)
    gh, a, b = s.aux_potentials()
    assert b == 0.0 and gh == pytest.approx(a, rel=1e-13) and gh > 0.0
    assert s.tau.tolist() == [0] * s.n
    # before anything moved the snapshots are the models: Gamma-hat is the potential with the fp32 mean
    assert gh == pytest.approx(s.potential(), rel=1e-6)


def test_local_steps_move_gamma_hat_and_b_but_not_a():
    s = make(o.NONBLOCKING)
    s.track_staleness(True)
    gh0, a0, b0 = s.aux_potentials()
    s.local_steps(list(range(s.n)), 3, 0.1)
    gh1, a1, b1 = s.aux_potentials()
    assert a1 == a0 and b1 > 0.0 and gh1 != gh0
    # B_t = n * ||mu_t - mu_0||^2 while no node has initiated since tracking started
    mu0 = s.mu_hist[0].astype(np.float64)
    mu1 = s.mean_model().astype(np.float64)
    assert b1 == pytest.approx(s.n * np.sum((mu1 - mu0) ** 2), rel=1e-12)


def test_launch_with_several_pairs_records_one_common_mean():
    s = make(o.NONBLOCKING, n=8)
    s.track_staleness(True)
    s.local_steps(list(range(8)), 2, 0.05)
    assert s.interact([[0, 1], [2, 3], [4, 5]], 8, o.NONBLOCKING) == 0
    mu = s.mean_model()
    for i in (0, 2, 4):
        assert np.array_equal(s.mu_hist[i], mu)
        assert s.a_hist[i] == pytest.approx(np.sum((s.B[i].astype(np.float64) - mu) ** 2), rel=1e-12)
    assert not np.array_equal(s.mu_hist[1], mu)   # responders keep their record
    assert s.tau.tolist()[:6] == [2, 3, 1, 3, 0, 3]


def test_tracking_needs_snapshots_and_refuses_blocking_exchanges():
    s = make(0)
    assert s.track_staleness(True) == -4
    with pytest.raises(ValueError):
        s.aux_potentials()
    s = make(o.NONBLOCKING)
    assert s.track_staleness(True) == 0
    assert s.interact([[0, 1]], 8, o.BLOCKING) == -4
    assert s.track_staleness(False) == 0
    assert s.interact([[0, 1]], 8, o.BLOCKING) == 0
    assert s.track_staleness(True) == -4          # snapshots are stale after a blocking exchange
