"""Pins for the local SGD steps (Section 3 "The Communication Procedure": H sequential stochastic
gradients, each taken at the running iterate) on the two synthetic objectives."""
import numpy as np
import pytest

from oracle import swarm_oracle as o


def lsq(n=3, d=24, m=10, batch=4, dtype=0, groups=0, noise=0.0, seed=1):
    s = o.OracleSwarm(n, d, "complete", seed=seed)
    s.configure(objective=2, lsq_m=m, lsq_batch=batch, lsq_dtype=dtype, lsq_groups=groups, lsq_noise_std=noise)
    return s


def test_lsq_data_recipe():
    s = lsq(n=4, d=4000, m=6, noise=float(np.sqrt(0.1)), seed=2)
    A = s.A
    assert A.shape == (4, 6, 4000)
    assert abs(A.std() * np.sqrt(4000) - 1) < 0.02          # N(0, 1/d)
    assert abs(s.xstar.std() - 1) < 0.05
    assert np.all(np.abs(s.shift) <= 1)
    clean = np.einsum("grk,k->gr", A.astype(np.float64), s.xstar.astype(np.float64))
    resid = s.bvec - clean - s.shift[:, None]
    assert abs(resid.std() - np.sqrt(0.1)) < 0.15            # 24 samples of the label noise
    s = lsq(n=4, d=64, m=6, groups=2, dtype=1)
    assert s.A.shape == (2, 6, 64)
    import torch
    a = torch.from_numpy(s.A.copy())
    assert torch.equal(a, a.to(torch.bfloat16).to(torch.float32))   # stored values are bf16-representable


def test_lsq_single_step_by_hand():
    """H = 1, batch 1: x' = x - lr * (<a, x> - b) * a for the sampled row a."""
    s = lsq(n=2, d=5, m=3, batch=1)
    x0 = s.X[1].astype(np.float64).copy()
    row = int(s.minibatch_rows(1, 0)[0])
    a = s.A[1, row].astype(np.float64)
    assert s.local_steps([1], 1, 0.25) == 0
    want = x0 - 0.25 * (a @ x0 - float(s.bvec[1, row])) * a
    assert np.array_equal(s.X[1], want.astype(np.float32))
    assert s.ls.tolist() == [0, 1]
    fresh = o.OracleSwarm(2, 5, "complete", seed=1)
    assert np.array_equal(s.X[0], fresh.X[0])                 # other node untouched


def test_lsq_step_is_minus_lr_times_minibatch_gradient_by_finite_differences():
    s = lsq(n=2, d=8, m=12, batch=5, noise=0.3)
    rows = s.minibatch_rows(0, 0)
    x0 = s.X[0].astype(np.float64).copy()
    A = s.A[0].astype(np.float64)[rows]
    b = s.bvec[0].astype(np.float64)[rows]

    def f(x):                                  # minibatch objective (1/2B) sum (a_s x - b_s)^2
        return 0.5 * ((A @ x - b) ** 2).mean()
    g = np.zeros(8)
    for k in range(8):
        h = np.zeros(8)
        h[k] = 1e-6
        g[k] = (f(x0 + h) - f(x0 - h)) / 2e-6
    s.local_steps([0], 1, 0.1)
    assert np.abs((s.X[0] - x0) / -0.1 - g).max() < 1e-5 * max(1.0, np.abs(g).max())


def test_lsq_rows_are_uniform_with_replacement_and_shared_inside_a_data_group():
    s = lsq(n=4, d=8, m=7, batch=6, groups=2)
    counts = np.zeros(7)
    repeats = 0
    for ev in range(2000):
        r = s.minibatch_rows(0, ev)
        assert r.min() >= 0 and r.max() < 7
        counts[r] += 1
        repeats += int(r[0] == r[1]) + int(r[2] == r[3]) + int(r[3] == r[4])
        assert np.array_equal(r, s.minibatch_rows(1, ev))        # same group, same event
    assert abs(repeats / 6000 - 1 / 7) < 0.02                    # draws are independent: two agree with probability 1/m
    assert not np.array_equal(s.minibatch_rows(0, 0), s.minibatch_rows(2, 0))
    exp = counts.sum() / 7
    assert ((counts - exp) ** 2 / exp).sum() < 30
    # restated from the counter layout: word t of stream 8, row id = data group, event = step counter
    wd = o.philox([1, 1, 5, 8], [1, 0])
    assert s.minibatch_rows(3, 5)[4] == o.uniform_int(wd[0], 7)


def test_lsq_sgd_converges_on_a_consistent_system():
    """No label noise, no shift: the system A x = b is consistent (m < d), so randomized row-action
    SGD drives the residual to zero (Kaczmarz-type convergence)."""
    s = lsq(n=2, d=40, m=8, batch=4, noise=0.0)
    s.shift[:] = 0
    A = s.A.astype(np.float64)
    s.bvec[:] = np.einsum("grk,k->gr", A, s.xstar.astype(np.float64)).astype(np.float32)
    r0 = np.linalg.norm(A[0] @ s.X[0] - s.bvec[0])
    s.local_steps([0], 4000, 0.5)
    r1 = np.linalg.norm(A[0] @ s.X[0] - s.bvec[0])
    assert r1 < 1e-4 * r0
    assert int(s.ls[0]) == 4000 and int(s.ls[1]) == 0


def test_each_local_step_uses_the_running_iterate():
    s1, s2 = lsq(seed=4), lsq(seed=4)
    s1.local_steps([2], 3, 0.2)
    for _ in range(3):
        s2.local_steps([2], 1, 0.2)
    assert np.array_equal(s1.X, s2.X)
    assert s1.ls.tolist() == [0, 0, 3]


def test_sequential_steps_equal_their_closed_form_through_the_gram_matrix():
    """A step moves the model along its sampled rows only, x_q = x_0 - (lr/B) sum_{p<q} A_p^T r_p, so the inner
    products of step q are A_q x_0 - (lr/B) sum_{p<q} (A_q A_p^T) r_p: H sequential steps of the oracle against
    that recursion over blocks of A A^T, written out in double (rows repeat inside and across minibatches here:
    10 rows, 4 draws a step)."""
    H, lr = 4, 0.3
    s = lsq(n=3, d=200, m=10, batch=4, noise=0.2, seed=9)
    node = 1
    A = s.A[node].astype(np.float64)
    x0 = s.X[node].astype(np.float64)
    rows = [s.minibatch_rows(node, q) for q in range(H)]
    assert len({tuple(r.tolist()) for r in rows}) == H
    gram = A @ A.T
    scale = lr / 4
    resid = []
    for q in range(H):
        score = A[rows[q]] @ x0
        for p in range(q):
            score -= scale * gram[np.ix_(rows[q], rows[p])] @ resid[p]
        resid.append(score - s.bvec[node, rows[q]].astype(np.float64))
    closed = x0 - scale * sum(A[rows[q]].T @ resid[q] for q in range(H))
    assert s.local_steps([node], H, lr) == 0
    assert np.abs(s.X[node] - closed).max() < 3e-7 * np.abs(closed).max()      # the oracle rounds x to fp32 per step
    assert np.abs(closed - x0).max() > 1e-3 * np.abs(closed).max()
    # without the correction terms the result is the one of H steps all taken at x_0: visibly different
    naive = x0 - scale * sum(A[rows[q]].T @ (A[rows[q]] @ x0 - s.bvec[node, rows[q]]) for q in range(H))
    assert np.abs(naive - closed).max() > 1e-4 * np.abs(closed).max()


def test_synthetic_gradient_moments_and_op_order():
    n, d = 2, 40000
    s = o.OracleSwarm(n, d, "complete", seed=6)
    s.configure(objective=1, grad_std=float(np.sqrt(1e-3)), drift_std=float(np.sqrt(0.05)))
    x0 = s.X.copy()
    lr = 0.05
    s.local_steps([1], 1, lr)
    upd = (s.X[1].astype(np.float64) - x0[1])
    c = float(s.drift[1])
    assert abs(upd.mean() + lr * c) < 5 * lr * np.sqrt(1e-3 / d) + 1e-8
    assert abs(upd.var() - lr**2 * 1e-3) < 0.03 * lr**2 * 1e-3
    assert np.array_equal(s.X[0], x0[0])
    # element 0 restated from the counter layout with the unfused fp32 operation order
    wd = o.philox([0, 1, 0, 9], [6, 0])
    z = np.float32(o.normal_pair(wd[0], wd[1])[0])
    p = np.float32(s.cfg.grad_std) * z
    g = np.float32(c) + p
    st = np.float32(lr) * g
    assert s.X[1, 0] == x0[1, 0] - st
    # second step draws fresh noise (event counter advanced)
    x1 = s.X[1].copy()
    s.local_steps([1], 1, lr)
    assert abs(np.corrcoef(s.X[1] - x1, x1 - x0[1])[0, 1]) < 0.03


def test_local_step_validation():
    s = o.OracleSwarm(3, 8, "complete")
    assert s.local_steps([0], 1, 0.1) == -1          # no objective configured
    s.configure(objective=1, grad_std=0.1)
    assert s.local_steps([0, 0], 1, 0.1) == -1       # node listed twice
    assert s.local_steps([3], 1, 0.1) == -2
    assert s.local_steps([], 2, 0.1) == 0
    assert s.local_steps([1], 0, 0.1) == 0 and int(s.ls[1]) == 0


def test_geometric_step_counts_have_the_stated_moments():
    """Section 3 (sequential model): H_i geometric with mean H; the analysis uses E[H_i^2] = 2H^2 - H."""
    for H in (1, 2, 4):
        s = o.OracleSwarm(64, 4, "complete", seed=H)
        s.configure(objective=1, grad_std=0.0)
        draws = []
        for _ in range(120):
            rc, steps = s.local_steps_geometric(list(range(64)), H, 0.0)
            assert rc == 0
            draws.extend(steps.tolist())
        draws = np.array(draws, dtype=np.float64)
        N = len(draws)
        assert draws.min() >= 1
        if H == 1:
            assert np.all(draws == 1)
            continue
        var = H * H - H                                  # variance of the geometric law
        assert abs(draws.mean() - H) < 5 * np.sqrt(var / N)
        assert abs((draws**2).mean() - (2 * H * H - H)) < 0.08 * (2 * H * H - H)
        # appendix lemmas on the step count: sum_K Pr[H_i = K] K^3 <= 6 H^3 and sum_K Pr[H_i = K] K^4 <= 24 H^4.
        # Closed forms of the geometric law with success probability 1/H: E[K^3] = 6H^3 - 6H^2 + H and
        # E[K^4] = 24H^4 - 36H^3 + 14H^2 - H; the sample moments must sit at those and under the bounds
        m3, m4 = 6 * H**3 - 6 * H**2 + H, 24 * H**4 - 36 * H**3 + 14 * H**2 - H
        assert abs((draws**3).mean() - m3) < 0.15 * m3 and (draws**3).mean() <= 6 * H**3
        assert abs((draws**4).mean() - m4) < 0.30 * m4 and (draws**4).mean() <= 24 * H**4
        assert abs((draws == 1).mean() - 1 / H) < 5 * np.sqrt((1 / H) * (1 - 1 / H) / N)
        assert abs((draws == 2).mean() - (1 - 1 / H) / H) < 5 * np.sqrt(0.25 / N)


def test_geometric_steps_equal_that_many_plain_steps():
    s1, s2 = lsq(seed=9), lsq(seed=9)
    rc, steps = s1.local_steps_geometric([0, 2], 3, 0.1)
    assert rc == 0 and s1.ls.tolist() == [int(steps[0]), 0, int(steps[1])]
    s2.local_steps([0], int(steps[0]), 0.1)
    s2.local_steps([2], int(steps[1]), 0.1)
    assert np.array_equal(s1.X, s2.X)
    # the draw restated from the counter layout: first trial whose word maps to 0 under uniform_int(., mean)
    t = 0
    while o.uniform_int(o.philox([t // 4, 2, 0, 11], [9, 0])[t % 4], 3) != 0:
        t += 1
    assert steps[1] == t + 1
    assert s1.local_steps_geometric([0], 0, 0.1)[0] == -1


def logistic(n=3, d=24, m=10, batch=4, seed=1, noise=0.2):
    s = o.OracleSwarm(n, d, "complete", seed=seed)
    s.configure(objective=3, lsq_m=m, lsq_batch=batch, lsq_dtype=0, lsq_groups=0, lsq_noise_std=noise)
    return s


def test_logistic_labels_and_gradient_by_finite_differences():
    """Logistic regression as second workload: labels are the sign of the noisy linear score, the step is
    minus lr times the minibatch gradient of (1/B) sum log(1 + e^{a.x}) - y a.x."""
    s = logistic(n=2, d=8, m=40, batch=6, seed=3)
    assert set(np.unique(s.bvec).tolist()) <= {0.0, 1.0} and 0 < s.bvec.mean() < 1
    score = s.A[0].astype(np.float64) @ s.xstar.astype(np.float64) + float(s.shift[0])
    sure = np.abs(score) > 0.9                               # label noise (std 0.2) cannot flip these
    assert sure.sum() >= 3 and np.array_equal(s.bvec[0][sure], (score[sure] > 0).astype(np.float32))
    # without label noise the class is exactly the sign of the score (threshold 0, not 1/2)
    clean = logistic(n=2, d=8, m=400, batch=6, seed=4, noise=0.0)
    sc = clean.A[1].astype(np.float64) @ clean.xstar.astype(np.float64) + float(clean.shift[1])
    away = np.abs(sc) > 1e-4
    assert ((sc > 0) & (sc < 0.5)).sum() >= 10
    assert np.array_equal(clean.bvec[1][away], (sc[away] > 0).astype(np.float32))
    rows = s.minibatch_rows(0, 0)
    x0 = s.X[0].astype(np.float64).copy()
    A, y = s.A[0].astype(np.float64)[rows], s.bvec[0].astype(np.float64)[rows]

    def f(x):
        z = A @ x
        return (np.log1p(np.exp(z)) - y * z).mean()
    g = np.zeros(8)
    for k in range(8):
        h = np.zeros(8)
        h[k] = 1e-6
        g[k] = (f(x0 + h) - f(x0 - h)) / 2e-6
    s.local_steps([0], 1, 0.1)
    assert np.abs((s.X[0] - x0) / -0.1 - g).max() < 1e-5 * max(1.0, np.abs(g).max())


def test_logistic_sgd_reduces_the_loss():
    s = logistic(n=2, d=30, m=64, batch=16, seed=5, noise=0.0)
    A, y = s.A[1].astype(np.float64), s.bvec[1].astype(np.float64)

    def loss(x):
        z = A @ x
        return (np.log1p(np.exp(z)) - y * z).mean()
    l0 = loss(s.X[1].astype(np.float64))
    s.local_steps([1], 400, 0.5)
    assert loss(s.X[1].astype(np.float64)) < 0.6 * l0
    pred = (A @ s.X[1].astype(np.float64)) > 0
    assert (pred == (y > 0.5)).mean() > 0.85


def test_step_on_explicit_rows_is_the_step_the_counter_would_draw():
    """local_step_on_rows with the rows of minibatch_rows is local_steps; with one explicit row it is the
    by-hand update x' = x - lr (<a, x> - b) a; the counter advances either way."""
    s1, s2 = lsq(n=3, d=40, m=12, batch=5, noise=0.2, seed=6), lsq(n=3, d=40, m=12, batch=5, noise=0.2, seed=6)
    for step in range(3):
        rows = s1.minibatch_rows(2, step)
        assert s1.local_steps([2], 1, 0.1) == 0
        assert s2.local_step_on_rows(2, rows, 0.1) == 0
    assert np.array_equal(s1.X, s2.X) and s1.ls.tolist() == s2.ls.tolist() == [0, 0, 3]
    x0 = s2.X[1].astype(np.float64).copy()
    a = s2.A[1, 7].astype(np.float64)
    assert s2.local_step_on_rows(1, [7], 0.25) == 0
    assert np.array_equal(s2.X[1], (x0 - 0.25 * (a @ x0 - float(s2.bvec[1, 7])) * a).astype(np.float32))
    # two explicit rows: the mean of the two single-row gradients
    x0 = s2.X[0].astype(np.float64).copy()
    A = s2.A[0].astype(np.float64)
    g = 0.5 * sum((A[r] @ x0 - float(s2.bvec[0, r])) * A[r] for r in (3, 3))   # a row may repeat (drawn with replacement)
    assert s2.local_step_on_rows(0, [3, 3], 0.5) == 0
    assert np.array_equal(s2.X[0], (x0 - 0.5 * g).astype(np.float32))
    assert s2.local_step_on_rows(0, [12], 0.1) == -2 and s2.local_step_on_rows(3, [0], 0.1) == -1
