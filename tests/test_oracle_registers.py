"""Pins for the two-register protocol: Algorithm 1 with its chain of three decodes
(Section 3, "The Communication Registers" and "The Communication Procedure")."""
import numpy as np
import pytest

from oracle import swarm_oracle as o


def make(n=4, d=2100, seed=1, topo="complete", **kw):
    s = o.OracleSwarm(n, d, topo, seed=seed)
    cfg = dict(objective=1, nonblocking=2, grad_std=0.03, drift_std=0.2)
    cfg.update(kw)
    s.configure(**cfg)
    return s


def decode_own(s, reader, owner):
    """Q(X^_owner) as `reader` obtains it: own register of `owner` decoded with reader's snapshot as key."""
    out = np.zeros(s.d, dtype=np.float32)
    for k in range(s.d):
        out[k] = o.dec(float(s.B[reader, k]), int(s.own[owner, k]), int(s.oexps[owner, k // 1024]), 16)
    return out


def decode_current(s, key, owner, bits):
    out = np.zeros(s.d, dtype=np.float32)
    for blk in range(s.nblk):
        k0, k1 = blk * 1024, min(s.d, (blk + 1) * 1024)
        codes = o.unpack_block(s.packed_codes(owner, bits)[blk * 128 * bits:(blk + 1) * 128 * bits], k1 - k0, bits)
        e = int(s.exps[owner, blk])
        out[k0:k1] = [o.dec(float(key[k0 + t]), int(codes[t]), e, bits) for t in range(k1 - k0)]
    return out


def steps(exps, d):
    return np.repeat(2.0 ** exps.astype(np.float64), 1024)[:d]


@pytest.mark.parametrize("bits", [2, 3, 4, 6, 8])
def test_register_publish_chain_decodes_every_snapshot(bits):
    s = make(offset_std=0.3)
    assert s.register_publish(bits) == 0
    assert int(s.p_mode[0]) == 2 and s.wo.tolist() == [1] * 4 and s.w.tolist() == [1] * 4
    for blk in range(s.nblk):
        assert np.all(s.oexps[:, blk] == s.oexps[0, blk])            # one step per block for the own registers
    for reader, owner in ((0, 1), (3, 2), (2, 2)):
        qhat = decode_own(s, reader, owner)
        assert np.all(np.abs(qhat.astype(np.float64) - s.B[owner]) < steps(s.oexps[owner], s.d))
        assert np.array_equal(qhat, decode_own(s, owner, owner))    # every in-range reader sees the same point
        cur = decode_current(s, qhat, owner, bits)
        assert np.all(np.abs(cur.astype(np.float64) - s.B[owner]) < steps(s.exps[owner], s.d))
    # the current register is scaled by the distance to its own key: far finer than the own register's range
    assert np.all(s.exps.astype(int) <= s.oexps.astype(int) - (bits - 2))


@pytest.mark.parametrize("bits", [4, 8])
def test_register_interaction_follows_algorithm_1(bits):
    s = make(offset_std=0.1)
    s.local_steps([0, 1, 2, 3], 2, 0.05)
    s.register_publish(bits)
    s.local_steps([1], 2, 0.05)
    X0, B0, own0, codes0 = s.X.copy(), s.B.copy(), s.own.copy(), s.codes.copy()
    Qa = decode_current(s, decode_own(s, 1, 1), 1, bits)            # Q(X_a)  <- Dec(Q(X^_a), Enc(X_a))
    qhat_b = decode_own(s, 1, 3)                                    # Q(X^_b) <- Dec(X^_a, Enc(X^_b))
    Qb = decode_current(s, qhat_b, 3, bits)                         # Q(X_b)  <- Dec(Q(X^_b), Enc(X_b))
    assert s.interact([[1, 3]], bits, o.REGISTERS) == 0
    avg = np.float32(0.5) * (Qa + Qb)
    D = B0[1] - X0[1]
    assert np.array_equal(s.X[1], avg - D)                          # X_a <- Q(X_a)/2 + Q(X_b)/2 - eta h
    assert np.array_equal(s.B[1], s.X[1])
    # one-way: the responder's model, snapshot and own register are untouched; bystanders entirely
    for i in (0, 2, 3):
        assert np.array_equal(s.X[i], X0[i]) and np.array_equal(s.B[i], B0[i]) and np.array_equal(s.own[i], own0[i])
    for i in (0, 2):
        assert np.array_equal(s.codes[i], codes0[i])
    # registers written: both of a hold its new model, the current register of b holds the average,
    # decodable by b with its own (unchanged) Q(X^_b)
    qa_new = decode_own(s, 1, 1)
    assert np.all(np.abs(qa_new.astype(np.float64) - s.X[1]) < steps(s.oexps[1], s.d))
    assert np.all(np.abs(decode_current(s, qa_new, 1, bits).astype(np.float64) - s.X[1]) < steps(s.exps[1], s.d))
    assert np.array_equal(decode_own(s, 3, 3), qhat_b)
    assert np.all(np.abs(decode_current(s, qhat_b, 3, bits).astype(np.float64) - avg) < steps(s.exps[3], s.d))
    assert s.wo.tolist() == [1, 2, 1, 1] and s.w.tolist() == [1, 2, 1, 2]
    assert s.tau.tolist() == [1, 0, 1, 1]
    # the own register's step is that of an 8-bit code of the guard distance 2 max|Q(X_a) - Q(X_b)| + max|eta h|,
    # whatever the width of the current registers: 127 steps cover the distance, 127 half-steps would not
    for blk in range(s.nblk):
        k = slice(blk * 1024, min(s.d, (blk + 1) * 1024))
        guard = 2.0 * float(np.abs(Qa[k] - Qb[k]).max()) + float(np.abs(D[k]).max())
        step = 2.0 ** int(s.oexps[1, blk])
        assert 127 * step >= guard > 127 * step / 2


def test_registers_remove_the_aliasing_plateau_of_the_single_buffer_form():
    """With per-node offsets far larger than the per-coordinate spread, the single-buffer form stalls at a
    large Gamma (keys leave the decode window for good); the register chain keeps every current-register
    decode inside its window, so the swarm contracts to its quantisation floor."""
    results = {}
    for mode, nb in ((o.NONBLOCKING, 1), (o.REGISTERS, 2)):
        s = make(n=8, d=1024, seed=3, nonblocking=nb, offset_std=0.3, grad_std=0.0, drift_std=0.0)
        g0 = s.potential()
        for _ in range(600):
            s.interact(s.sample_pairs(1), 8, mode)
        results[mode] = s.potential() / g0
    assert results[o.NONBLOCKING] > 0.05          # the documented plateau
    assert results[o.REGISTERS] < 1e-4


def test_staleness_clocks_and_mode_switches():
    s = make(n=5, d=64)
    s.interact([[0, 1], [2, 3]], 8, o.REGISTERS)
    assert s.tau.tolist() == [1, 2, 0, 2, 2]
    assert int(s.p_mode[0]) == 2
    s.interact([[4, 0]], 8, o.NONBLOCKING)           # other convention: buffers are re-published first
    assert int(s.p_mode[0]) == 1 and s.tau.tolist() == [2, 3, 1, 3, 0]
    w_before = s.w.copy()
    s.interact([[1, 2]], 8, o.REGISTERS)
    assert int(s.p_mode[0]) == 2
    assert np.all(s.w >= w_before + 1)               # register_publish rewrote every current register
    s.interact([[3, 4]], 8, o.BLOCKING)
    assert int(s.p_mode[0]) == 0 and int(s.b_stale[0]) == 1
    plain = o.OracleSwarm(4, 16, "complete")
    plain.configure(objective=1, nonblocking=1)
    assert plain.interact([[0, 1]], 8, o.REGISTERS) == -4
    assert plain.register_publish(8) == -1


# ---- variable rate: a reader consumes a prefix of the partner's own register (Corollary 1, second case) ----

def test_colours_nest_so_a_prefix_is_a_shorter_code():
    """The b-bit colour of a lattice point is the low b bits of its 16-bit colour; decoding the prefix gives
    the full decode exactly when the key lies within the prefix's own window."""
    rng = np.random.default_rng(0)
    e = -7
    step = 2.0 ** e
    for _ in range(400):
        q = int(rng.integers(-10**6, 10**6))
        c16 = o.code(q, 16)
        for b in (8, 4):
            assert o.code(q, b) == c16 & ((1 << b) - 1)
        L8 = 127
        for off in (0, 1, -1, L8, -L8, L8 + 1, -(L8 + 1), L8 + 2, 300, -5000):
            key = (q - off) * step + 0.25 * step           # key cell = q - off, i.e. q = cell + off
            full = o.dec(key, c16, e, 16)
            short = o.dec(key, c16 & 0xFF, e, 8)
            assert full == q * step
            if -L8 <= off <= L8 + 1:                        # q inside [cell - L, cell + L + 1]
                assert short == full
            else:
                assert short != full and (short - full) / step % 256 == 0


def far_reader():
    """Nodes 0 and 1 start close together and node 2 a fixed offset away; after one interaction of 0 with 1
    the own register of 0 has a finer step, and node 2 sits more than 127 but less than 32767 of those steps
    away."""
    s = make(n=3, d=1500, seed=4, offset_std=0.0, drift_std=0.0, grad_std=0.0, init_std=0.001)
    s.X[2] += np.float32(0.05)
    s.B[:] = s.X
    s.register_publish(8)
    s.interact([[0, 1]], 8, o.REGISTERS)
    dist_steps = np.abs(s.B[2].astype(np.float64) - s.B[0]) / steps(s.oexps[0], s.d)
    assert dist_steps.min() > 200 and dist_steps.max() < 30000
    return s


def test_prefix_reader_within_range_matches_the_full_register_and_fails_beyond():
    near16, near8 = make(offset_std=0.05), make(offset_std=0.05)
    assert near8.set_own_prefix(8) == 0 and near8.own_prefix == 8 and near16.own_prefix == 16
    # nodes that keep talking to the same partner stay within the guard distance of each other's snapshots
    # (that distance sets the own register's step): the 8-bit prefix is all such a reader needs
    for pairs in ([[0, 1], [2, 3]], [[1, 0], [3, 2]], [[0, 1], [3, 2]], [[1, 0], [2, 3]]):
        for s in (near16, near8):
            s.local_steps([p[0] for p in pairs], 2, 0.05)
            assert s.interact(pairs, 8, o.REGISTERS) == 0
    assert np.array_equal(near16.X, near8.X) and np.array_equal(near16.own_bytes, near8.own_bytes)
    assert np.array_equal(near16.codes, near8.codes)
    # beyond 127 steps the 8-bit prefix aliases (by whole multiples of 256 steps); the full register does not
    far16, far8 = far_reader(), far_reader()
    far8.set_own_prefix(8)
    for s in (far16, far8):
        assert s.interact([[2, 0]], 8, o.REGISTERS) == 0
    mid = 0.5 * (far16.B[0].astype(np.float64) + 0.05 + far16.B[0])          # about half way between 2 and 0
    assert np.abs(far16.X[2] - mid).max() < 0.01
    assert np.abs(far8.X[2].astype(np.float64) - far16.X[2]).max() > 0.005


def test_prefix_reader_never_touches_the_high_bytes_of_its_partner():
    ref, scr = make(offset_std=0.05), make(offset_std=0.05)
    for s in (ref, scr):
        s.set_own_prefix(8)
        s.local_steps([1], 2, 0.05)
        s.register_publish(8)
    planes = scr.own_bytes.reshape(scr.n, scr.nblk, 2, 1024)
    planes[:, :, 1, :] ^= 0xA5                               # garbage in every high byte, own and partner's
    for s in (ref, scr):
        assert s.interact([[1, 3]], 8, o.REGISTERS) == 0
    assert np.array_equal(ref.X, scr.X) and np.array_equal(ref.codes, scr.codes)
    assert np.array_equal(ref.own[1], scr.own[1])                            # a's register is rewritten in full
    # with the full register the same garbage changes what the reader decodes
    full = make(offset_std=0.05)
    full.local_steps([1], 2, 0.05)
    full.register_publish(8)
    full.own_bytes.reshape(full.n, full.nblk, 2, 1024)[3, :, 1, :] ^= 0xA5
    assert full.interact([[1, 3]], 8, o.REGISTERS) == 0
    assert not np.array_equal(full.X[1], ref.X[1])


def test_own_prefix_argument_checks():
    s = make()
    assert s.set_own_prefix(12) == -1 and s.set_own_prefix(8) == 0
    s.configure(objective=1, nonblocking=2)
    assert s.own_prefix == 16                                # a new configuration goes back to the full register
    plain = o.OracleSwarm(4, 16, "complete")
    plain.configure(objective=1, nonblocking=1)
    assert plain.set_own_prefix(8) == -4


# ---- the prefix is the reader's: each interaction of a launch states its own (Corollary 1, second case;
# ---- "Counting Communication Cost": a reader uses the first bits in proportion to its distance) ----

def decode_own_prefix(s, reader, owner, prefix):
    mask = (1 << prefix) - 1
    return np.array([o.dec(float(s.B[reader, k]), int(s.own[owner, k]) & mask, int(s.oexps[owner, k // 1024]), prefix)
                     for k in range(s.d)], dtype=np.float32)


def near_and_far_readers():
    """Nodes 0, 1 and 3, 4 are close pairs that have just met (fine own registers); node 2 sits 0.05 away from
    all of them: hundreds of own-register steps, far outside an 8-bit window, well inside the 16-bit one."""
    s = make(n=5, d=1500, seed=4, offset_std=0.0, drift_std=0.0, grad_std=0.0, init_std=0.001)
    s.X[2] += np.float32(0.05)
    s.B[:] = s.X
    s.register_publish(8)
    assert s.interact([[0, 1], [3, 4]], 8, o.REGISTERS) == 0
    dist_steps = np.abs(s.B[2].astype(np.float64) - s.B[0]) / steps(s.oexps[0], s.d)
    assert dist_steps.min() > 200 and dist_steps.max() < 30000
    near_steps = np.abs(s.B[4].astype(np.float64) - s.B[3]) / steps(s.oexps[3], s.d)
    assert near_steps.max() < 100
    return s


def test_a_launch_mixes_readers_with_different_prefixes():
    launch = [[2, 0], [4, 3]]                          # a far reader and a near reader
    ref, default = near_and_far_readers(), near_and_far_readers()
    assert ref.interact_prefixed(launch, [16, 16], 8) == 0
    assert default.interact(launch, 8, o.REGISTERS) == 0             # the context's default prefix is 16
    for name in ("X", "B", "own_bytes", "codes", "exps", "oexps", "w", "wo", "tau"):
        assert np.array_equal(getattr(ref, name), getattr(default, name)), name
    # the near reader needs 8 bits only: same launch, same result, half of its partner's register read
    mixed = near_and_far_readers()
    assert mixed.interact_prefixed(launch, [16, 8], 8) == 0
    for name in ("X", "B", "own_bytes", "codes", "exps", "oexps", "w", "wo", "tau"):
        assert np.array_equal(getattr(ref, name), getattr(mixed, name)), name
    # the prefix travels with its pair, wherever the pair stands in the list
    swapped = near_and_far_readers()
    assert swapped.interact_prefixed(launch[::-1], [8, 16], 8) == 0
    for name in ("X", "B", "own_bytes", "codes", "exps", "oexps", "w", "wo"):
        assert np.array_equal(getattr(ref, name), getattr(swapped, name)), name
    # the other way round the far reader aliases; the near reader's interaction is not affected by it
    wrong = near_and_far_readers()
    before = near_and_far_readers()
    short, full = decode_own_prefix(before, 2, 0, 8), decode_own_prefix(before, 2, 0, 16)
    st = steps(before.oexps[0], before.d)
    q = np.round(full.astype(np.float64) / st)
    cell = np.floor(before.B[2].astype(np.float64) / st)
    inside = (q - cell >= -127) & (q - cell <= 128)                  # the 8-bit window around the reader's cell
    assert not inside.any()
    assert np.array_equal(short == full, inside)
    off = (short.astype(np.float64) - full) / st
    assert np.all(off % 256 == 0) and np.all(off != 0)
    assert wrong.interact_prefixed(launch, [8, 16], 8) == 0
    for i in (3, 4, 0, 1):
        assert np.array_equal(wrong.X[i], ref.X[i]) and np.array_equal(wrong.B[i], ref.B[i])
    assert np.array_equal(wrong.own_bytes[4], ref.own_bytes[4]) and np.array_equal(wrong.codes[3], ref.codes[3])
    # node 2's update restated from unit decodes with the short prefix
    Qa = decode_current(before, decode_own_prefix(before, 2, 2, 8), 2, 8)
    Qb = decode_current(before, short, 0, 8)
    assert np.array_equal(wrong.X[2], np.float32(0.5) * (Qa + Qb) - (before.B[2] - before.X[2]))
    assert np.abs(wrong.X[2].astype(np.float64) - ref.X[2]).max() > 0.005


def test_context_default_prefix_is_the_prefix_of_every_pair():
    launch = [[1, 0], [4, 3]]
    a, b = near_and_far_readers(), near_and_far_readers()
    assert a.set_own_prefix(8) == 0
    assert a.interact(launch, 8, o.REGISTERS) == 0
    assert b.interact_prefixed(launch, [8, 8], 8) == 0 and b.own_prefix == 16
    for name in ("X", "B", "own_bytes", "codes", "exps", "oexps"):
        assert np.array_equal(getattr(a, name), getattr(b, name)), name
    assert b.interact_prefixed(launch, [8, 12], 8) == -1
    with pytest.raises(ValueError):
        b.interact_prefixed(launch, [8], 8)
