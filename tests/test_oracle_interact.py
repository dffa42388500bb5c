"""Pins for the interaction step (Algorithm 1 / Section 3) and for mu, Gamma (Section 4)."""
import numpy as np
import pytest

from oracle import swarm_oracle as o


def gamma_np(X):
    X = X.astype(np.float64)
    return float(((X - X.mean(axis=0)) ** 2).sum())


def test_gamma_and_mean_closed_forms():
    s = o.OracleSwarm(2, 1500, "complete", seed=1)
    X = s.X.astype(np.float64)
    assert abs(s.potential() - ((X[0] - X[1]) ** 2).sum() / 2) < 1e-9      # n = 2
    s = o.OracleSwarm(7, 300, "complete", seed=2)
    X = s.X.astype(np.float64)
    pair_sum = sum(((X[i] - X[j]) ** 2).sum() for i in range(7) for j in range(i + 1, 7))
    assert abs(pair_sum - 7 * s.potential()) < 1e-8 * pair_sum             # equality case, lambda_2 = n
    assert np.array_equal(s.mean_model(), X.mean(axis=0).astype(np.float32))
    assert abs(s.potential() - gamma_np(s.X)) < 1e-9 * s.potential()


def test_exact_averaging_by_hand():
    s = o.OracleSwarm(3, 2, "complete", seed=0)
    s.X[:] = np.array([[1.0, 2.0], [3.0, -2.0], [10.0, 0.5]], dtype=np.float32)
    # mu = (14/3, 1/6); Gamma = sum of squared deviations
    assert abs(s.potential() - (((1 - 14 / 3) ** 2 + (3 - 14 / 3) ** 2 + (10 - 14 / 3) ** 2)
                                + ((2 - 1 / 6) ** 2 + (-2 - 1 / 6) ** 2 + (0.5 - 1 / 6) ** 2))) < 1e-12
    assert s.interact([[0, 1]], 32) == 0
    assert s.X.tolist() == [[2.0, 0.0], [2.0, 0.0], [10.0, 0.5]]
    assert s.w.tolist() == [0, 0, 0] and s.pbits.tolist() == [0, 0, 0]


@pytest.mark.parametrize("n", [2, 5])
def test_exact_averaging_preserves_mean_and_drops_gamma(n):
    s = o.OracleSwarm(n, 3000, "complete", seed=n)
    mu0, g0 = s.X.astype(np.float64).mean(axis=0), s.potential()
    diff2 = ((s.X[0].astype(np.float64) - s.X[1]) ** 2).sum()
    s.interact([[0, 1]], 32)
    assert np.abs(s.X.astype(np.float64).mean(axis=0) - mu0).max() < 1e-8
    assert abs((s.potential() - g0) + diff2 / 2) < 1e-6 * diff2       # fp32 rounding of the average only
    assert np.array_equal(s.X[0], s.X[1])
    if n == 2:
        assert s.potential() == 0.0


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 7, 8])
def test_quantized_interaction_satisfies_the_gamma_change_identity(bits):
    """Delta = -||Xi-Xj||^2/2 + <Xi-mu + Xj-mu, Si+Sj> + (n-2)/n^2 ||Si+Sj||^2
               + ||(n-1)/n Si - Sj/n||^2 + ||(n-1)/n Sj - Si/n||^2,   Si = Sj = X' - (Xi+Xj)/2."""
    n, d = 6, 2500
    s = o.OracleSwarm(n, d, "complete", seed=bits)
    X0 = s.X.astype(np.float64).copy()
    mu0, g0 = X0.mean(axis=0), s.potential()
    s.interact([[3, 1]], bits)
    assert np.array_equal(s.X[3], s.X[1])
    S = s.X[3].astype(np.float64) - (X0[3] + X0[1]) / 2
    mu1 = s.X.astype(np.float64).mean(axis=0)
    assert np.abs(mu1 - (mu0 + 2 * S / n)).max() < 1e-12
    delta = (-((X0[3] - X0[1]) ** 2).sum() / 2 + ((X0[3] - mu0 + X0[1] - mu0) * 2 * S).sum()
             + (n - 2) / n**2 * ((2 * S) ** 2).sum() + 2 * (((n - 2) / n * S) ** 2).sum())
    assert abs((s.potential() - g0) - delta) < 1e-9 * abs(g0)
    # per-coordinate error of each decoded model is below one lattice step
    for blk in range(s.nblk):
        sl = slice(blk * 1024, min(d, (blk + 1) * 1024))
        step = 2.0 ** int(s.exps[3, blk])
        assert np.abs(S[sl]).max() < step
        rho = np.abs(X0[3, sl] - X0[1, sl]).max()
        assert (2 ** (bits - 1) - 1) * step >= rho
        assert s.exps[3, blk] == s.exps[1, blk]
    assert s.w.tolist() == [0, 1, 0, 1, 0, 0]
    assert s.pbits.tolist() == [0, bits, 0, bits, 0, 0]


@pytest.mark.parametrize("bits", [2, 8])
def test_quantized_average_is_unbiased_over_write_counters(bits):
    n, d, trials = 2, 256, 600
    s = o.OracleSwarm(n, d, "complete", seed=5)
    X0 = s.X.copy()
    exact = (X0[0].astype(np.float64) + X0[1]) / 2
    acc = np.zeros(d)
    for t in range(trials):
        s.X[:] = X0
        s.w[:] = [2 * t, 2 * t + 1]          # fresh rounding uniforms each trial
        s.interact([[0, 1]], bits)
        acc += s.X[0]
    step = 2.0 ** int(s.exps[0, 0])
    err = acc / trials - exact
    # each decoded value has variance <= step^2/4; the average of two independent ones step^2/8
    assert np.abs(err).max() < 5 * step / np.sqrt(8 * trials) + step * 2.0**-16
    assert abs(err.mean()) < 5 * step / np.sqrt(8 * trials * d) + step * 2.0**-16


def test_codes_in_buffer_are_the_encodings_of_the_pre_interaction_models():
    n, d, bits = 4, 1500, 4
    seed = 9
    s = o.OracleSwarm(n, d, "ring", seed=seed)
    s.w[:] = [3, 0, 7, 0]
    X0 = s.X.copy()
    s.interact([[2, 1]], bits)
    for node, w in ((2, 7), (1, 0)):
        u = o.sr_uniforms(seed, node, w, 0, d)
        for blk in range(s.nblk):
            e = int(s.exps[node, blk])
            k0, k1 = blk * 1024, min(d, (blk + 1) * 1024)
            codes = np.array([o.code(o.enc_q(float(X0[node, k]), e, int(u[k])), bits) for k in range(k0, k1)],
                             dtype=np.uint8)
            want = o.pack_block(codes, bits)
            got = s.packed_codes(node, bits)[blk * 512:(blk + 1) * 512]
            assert np.array_equal(got, want)
    assert s.w.tolist() == [3, 1, 8, 0]


def test_tail_block_and_identical_models():
    s = o.OracleSwarm(2, 1030, "complete", seed=3)
    s.X[1] = s.X[0]
    x0 = s.X[0].copy()
    s.interact([[0, 1]], 8)
    # rho = 0: the step is set by the magnitude clamp alone, every value is within one step
    for blk in range(2):
        sl = slice(blk * 1024, min(1030, (blk + 1) * 1024))
        M = np.abs(x0[sl]).max()
        e = int(s.exps[0, blk])
        assert e == max(int(np.frexp(M)[1]) - 23, -126)
        assert np.abs(s.X[0, sl].astype(np.float64) - x0[sl]).max() < 2.0**e
    assert np.all(s.packed_codes(0, 8)[1030:] == 0)
    s.X[:] = 0
    s.interact([[1, 0]], 2)
    assert np.all(s.X == 0) and np.all(s.exps == -126) and np.all(s.packed_codes(0, 2) == 0)


def test_pair_validation():
    s = o.OracleSwarm(6, 8, "ring", seed=0)
    assert s.interact([[0, 1], [2, 3]], 8) == 0
    assert s.interact([[0, 1], [1, 2]], 8) == -3      # not disjoint
    assert s.interact([[0, 0]], 8) == -3
    assert s.interact([[0, 3]], 8) == -3              # not adjacent on the ring
    assert s.interact([[0, 6]], 8) == -2
    assert s.interact([[0, 1]], 1) == -1             # one bit leaves no decoding window (L = 0)
    assert s.interact([[0, 1]], 9) == -1 and s.interact([[0, 1]], 16) == -1
    assert s.interact([[0, 1]], 8, o.NONBLOCKING) == -4


# ---- non-blocking mode ---------------------------------------------------------------------

def make_nb(n=4, d=2100, bits=8, seed=1, topo="complete"):
    s = o.OracleSwarm(n, d, topo, seed=seed)
    s.configure(objective=1, nonblocking=1, grad_std=0.03, drift_std=0.2)
    return s


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 7, 8])
def test_publish_encodes_base_with_the_spread_of_all_bases(bits):
    s = make_nb(bits=bits)
    assert np.array_equal(s.B, s.X)
    assert s.publish(bits) == 0
    L = 2 ** (bits - 1) - 1
    for blk in range(s.nblk):
        sl = slice(blk * 1024, min(s.d, (blk + 1) * 1024))
        spread = (s.B[:, sl].max(axis=0) - s.B[:, sl].min(axis=0)).max()
        e = int(s.exps[0, blk])
        assert np.all(s.exps[:, blk] == e)
        assert L * 2.0**e >= spread > L * 2.0 ** (e - 1)
        # any node can decode any other node's buffer with its own base as key
        for i, j in ((0, 1), (3, 2)):
            codes = o.unpack_block(s.packed_codes(j, bits)[blk * 128 * bits:(blk + 1) * 128 * bits],
                                   sl.stop - sl.start, bits)
            Q = np.array([o.dec(float(s.B[i, sl.start + k]), int(codes[k]), e, bits) for k in range(len(codes))])
            assert np.abs(Q - s.B[j, sl]).max() < 2.0**e
    assert s.w.tolist() == [1] * s.n and s.pbits.tolist() == [bits] * s.n


@pytest.mark.parametrize("bits", [4, 8])
def test_nonblocking_interaction_is_one_way(bits):
    s = make_nb(bits=bits)
    s.local_steps([0, 1, 2, 3], 2, 0.05)
    X0, B0 = s.X.copy(), s.B.copy()
    assert s.interact([[0, 2]], bits, o.NONBLOCKING) == 0        # publishes first
    # responder's model and snapshot are not touched; bystanders neither
    assert np.array_equal(s.X[1:], X0[1:]) and np.array_equal(s.B[1:], B0[1:])
    # initiator: new model = average of the two decoded buffers minus its pending update
    D = B0[0] - X0[0]
    avg = s.X[0] + D                                             # fp32: exact enough to compare at step level
    want = (B0[0].astype(np.float64) + B0[2]) / 2
    for blk in range(s.nblk):
        sl = slice(blk * 1024, min(s.d, (blk + 1) * 1024))
        assert np.abs(avg[sl] - want[sl]).max() < 1.01 * 2.0 ** 1 * 2.0 ** int(np.max(s.exps[:, blk]))
    assert np.array_equal(s.B[0], s.X[0])
    assert s.w.tolist() == [2, 1, 2, 1]
    # the responder's buffer now decodes (with the responder's own base as key) to the average
    e = s.exps[2]
    for blk in range(s.nblk):
        sl = slice(blk * 1024, min(s.d, (blk + 1) * 1024))
        codes = o.unpack_block(s.packed_codes(2, bits)[blk * 128 * bits:(blk + 1) * 128 * bits],
                               sl.stop - sl.start, bits)
        Q = np.array([o.dec(float(s.B[2, sl.start + k]), int(codes[k]), int(e[blk]), bits) for k in range(len(codes))])
        assert np.abs(Q - avg[sl]).max() < 2.0 ** int(e[blk]) * 1.001
        assert s.exps[0, blk] == s.exps[2, blk]


def test_nonblocking_without_pending_update_matches_blocking_average_of_decoded_buffers():
    """With D = 0 both modes average the same two decoded vectors."""
    bits = 8
    s = make_nb(bits=bits)
    s.publish(bits)
    own = np.zeros(s.d, dtype=np.float32)
    oth = np.zeros(s.d, dtype=np.float32)
    for blk in range(s.nblk):
        sl = slice(blk * 1024, min(s.d, (blk + 1) * 1024))
        for row, node in ((own, 1), (oth, 3)):
            codes = o.unpack_block(s.packed_codes(node, bits)[blk * 1024:(blk + 1) * 1024], sl.stop - sl.start, bits)
            row[sl] = [o.dec(float(s.B[1, sl.start + k]), int(codes[k]), int(s.exps[node, blk]), bits)
                       for k in range(len(codes))]
    s.interact([[1, 3]], bits, o.NONBLOCKING)
    assert np.array_equal(s.X[1], np.float32(0.5) * (own + oth))


def test_nonblocking_write_scales_both_written_vectors_below_2_to_23():
    """The exponent of a one-way write must keep both vectors it encodes (the new model and the average) below
    2^23 lattice steps, or their scaled values stop being exact. Here the average is exactly 1 and the new model
    just below 1, with a pending update of 2^-20: the distance alone would allow a step of 2^-26, the new model
    alone one of 2^-23, the average needs 2^-22."""
    s = make_nb(n=4, d=1024)
    s.X[:] = np.float32(1.0)
    s.B[:] = np.float32(1.0)
    assert s.publish(8) == 0
    assert s.exps[:, 0].tolist() == [-22] * 4                       # zero spread: only the magnitude rule acts
    s.X[0] = np.float32(1.0 - 2.0**-20)                             # pending update D = B - X = 2^-20
    assert s.interact([[0, 1]], 8, o.NONBLOCKING) == 0
    assert np.all(s.X[0] == np.float32(1.0 - 2.0**-20))             # average 1 minus D
    e = int(s.exps[0, 0])
    assert int(s.exps[1, 0]) == e
    assert 1.0 * 2.0**-e < 2.0**23 and 1.0 * 2.0**-(e - 1) >= 2.0**23   # least step that keeps the average exact


def test_nonblocking_swarm_contracts_gamma():
    """Statistical sanity only: repeated one-way interactions pull the models together (coordinates
    whose key distance left the decode window stay aliased: the quantization-failure event)."""
    s = make_nb(n=8, d=1024, bits=8, seed=3)
    s.configure(objective=1, nonblocking=1, offset_std=0.05, grad_std=0.0, drift_std=0.0)
    g0 = s.potential()
    for _ in range(200):
        pairs = s.sample_pairs(1)
        s.interact(pairs, 8, o.NONBLOCKING)
    # every node has adopted some average by now
    assert s.potential() < 0.01 * g0


def test_blocking_then_nonblocking_refreshes_the_base():
    s = make_nb()
    s.interact([[0, 1]], 8, o.BLOCKING)
    assert int(s.b_stale[0]) == 1
    s.interact([[2, 3]], 8, o.NONBLOCKING)
    assert int(s.b_stale[0]) == 0
    assert np.array_equal(s.B[0], s.X[0]) and np.array_equal(s.B[1], s.X[1])
