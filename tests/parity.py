"""Helpers for the GPU parity tests: build an oracle swarm and a CUDA swarm from the same seeded
recipe, compare them, and copy the oracle's state into the CUDA context (teacher forcing)."""
import numpy as np

from oracle import swarm_oracle as o
from paper_1910_12308_b200 import binding as g


def rel_err(got, ref):
    """max |got - ref| / max |ref| over a row (the floating-point parity measure)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    scale = np.abs(ref).max()
    return float(np.abs(got - ref).max() / scale) if scale > 0 else float(np.abs(got).max())


def make_pair(n, d, topology="complete", degree=0, seed=0, **cfg):
    orc = o.OracleSwarm(n, d, topology, degree, seed)
    gpu = g.Swarm(n, d, topology, degree, seed)
    if cfg:
        orc.configure(**cfg)
        gpu.configure(**cfg)
    return orc, gpu


def inject(orc, gpu, what=("X", "B", "P", "counters", "data")):
    """Copy the oracle's state into the CUDA context."""
    for i in range(orc.n):
        if "X" in what:
            gpu.set(g.T_X, i, orc.X[i])
        if "B" in what and orc.B is not None:
            gpu.set(g.T_B, i, orc.B[i])
        if "P" in what:
            gpu.set(g.T_CODES, i, orc.codes[i])
            gpu.set(g.T_EXPS, i, orc.exps[i])
        if "P" in what and orc.own_bytes is not None:
            gpu.set(g.T_OWN, i, orc.own_bytes[i])
            gpu.set(g.T_OEXPS, i, orc.oexps[i])
        if "counters" in what:
            gpu.set(g.T_COUNTERS, i, [orc.w[i], orc.ls[i], orc.pbits[i]])
            gpu.set(g.T_CLOCKS, i, [orc.wo[i], orc.tau[i]])
        if "data" in what:
            gpu.set(g.T_SCALARS, i, [orc.offset[i], orc.drift[i], orc.shift[i]])
            if orc.groups:
                gpu.set(g.T_BVEC, i, orc.bvec[i])
    if "data" in what and orc.groups:
        for grp in range(orc.groups):
            gpu.set(g.T_A, grp, orc.A[grp])
    if "counters" in what:
        gpu.set_state(int(orc.launch[0]), int(orc.b_stale[0]))
        gpu.set_buffer_mode(int(orc.p_mode[0]))


def assert_store_equal(orc, gpu, bits=None, nodes=None, check_B=True):
    """Bit-exact comparison of models, snapshots, buffers, exponents and counters."""
    nodes = range(orc.n) if nodes is None else nodes
    for i in nodes:
        gx = gpu.get(g.T_X, i)
        assert np.array_equal(gx.view(np.uint32), orc.X[i].view(np.uint32)), f"X[{i}] differs"
        if check_B and orc.B is not None:
            assert np.array_equal(gpu.get(g.T_B, i).view(np.uint32), orc.B[i].view(np.uint32)), f"B[{i}] differs"
        w, ls, pb = gpu.get(g.T_COUNTERS, i)
        assert (w, ls, pb) == (orc.w[i], orc.ls[i], orc.pbits[i]), f"counters[{i}]"
        assert tuple(gpu.get(g.T_CLOCKS, i)) == (orc.wo[i], orc.tau[i]), f"clocks[{i}]"
        if orc.own_bytes is not None and int(orc.p_mode[0]) == 2:
            assert np.array_equal(gpu.get(g.T_OWN, i), orc.own_bytes[i]), f"own register[{i}] differs"
            assert np.array_equal(gpu.get(g.T_OEXPS, i), orc.oexps[i]), f"own exponents[{i}] differ"
        if bits is not None and 2 <= bits <= 8 and orc.pbits[i] == bits:
            nbytes = orc.nblk * 128 * bits
            assert np.array_equal(gpu.get(g.T_CODES, i)[:nbytes], orc.codes[i, :nbytes]), f"codes[{i}] differ"
            assert np.array_equal(gpu.get(g.T_EXPS, i), orc.exps[i]), f"exps[{i}] differ"
    launch, stale = gpu.get_state()
    assert (launch, stale) == (int(orc.launch[0]), int(orc.b_stale[0]))
    assert gpu.get_buffer_mode() == int(orc.p_mode[0])
