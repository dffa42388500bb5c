"""Parity at the sizes of the benchmark configurations, in the launch shapes the benchmark uses.
The oracle runs either the whole launch (where it finishes in seconds) or a sample of the pairs."""
import numpy as np
import pytest

from oracle import swarm_oracle as o
from paper_1910_12308_b200 import binding as g
from tests.parity import rel_err

pytestmark = pytest.mark.gpu


def ring_matching(n, parity, flip_bits):
    pairs = []
    for t in range(n // 2):
        a, b = (2 * t + parity) % n, (2 * t + 1 + parity) % n
        pairs.append((b, a) if (flip_bits >> t) & 1 else (a, b))
    return np.array(pairs, dtype=np.int32)


def test_config2_full_launch_bit_exact():
    """n = 64, d = 2^20, ring, 32 disjoint pairs per launch, 4-bit, averaging only."""
    n, d, bits = 64, 1 << 20, 4
    gpu = g.Swarm(n, d, "ring", seed=2)
    gpu.configure(offset_std=float(np.sqrt(0.1)))
    orc = o.OracleSwarm(n, d, "ring", seed=2)
    for i in range(n):                       # the CUDA-generated state is the common input
        orc.X[i] = gpu.get(g.T_X, i)
    assert abs(float(orc.X.std()) - np.sqrt(0.01 + 0.1)) < 0.1
    for launch in range(2):
        pairs = ring_matching(n, launch & 1, 0x5A5A5A5A >> launch)
        assert gpu.interact(pairs, bits) == 0
        assert orc.interact(pairs, bits, threads=8) == 0
    for i in range(n):
        assert np.array_equal(gpu.get(g.T_X, i).view(np.uint32), orc.X[i].view(np.uint32))
        assert np.array_equal(gpu.get(g.T_CODES, i)[: orc.nblk * 128 * bits], orc.packed_codes(i, bits))
        assert np.array_equal(gpu.get(g.T_EXPS, i), orc.exps[i])
    assert abs(gpu.potential() - orc.potential()) <= 1e-9 * orc.potential()


@pytest.mark.parametrize("d,bits,mode", [(11_689_512, 8, 1), (25_557_032, 4, 0), (25_557_032, 8, 0)])
def test_large_model_sampled_pair_bit_exact(d, bits, mode):
    """ResNet-18 / ResNet-50 sized vectors (ragged tail blocks of 552 and 40 coordinates): the CUDA
    path runs a full launch, the oracle recomputes one of its pairs."""
    n = 4
    cfg = dict(objective=1, nonblocking=mode, grad_std=float(np.sqrt(1e-3)), drift_std=float(np.sqrt(0.05)))
    gpu = g.Swarm(n, d, "complete", seed=3)
    gpu.configure(**cfg)
    orc = o.OracleSwarm(n, d, "complete", seed=3)
    orc.configure(objective=1, nonblocking=mode, grad_std=0.0, drift_std=0.0, init_std=0.0)
    assert gpu.local_steps([0, 1, 2, 3], 2, 0.05) == 0
    if mode == 1:
        assert gpu.publish(bits) == 0
        assert gpu.local_steps([0, 1, 2, 3], 1, 0.05) == 0
    for i in range(n):
        orc.X[i] = gpu.get(g.T_X, i)
        if mode == 1:
            orc.B[i] = gpu.get(g.T_B, i)
            orc.codes[i] = gpu.get(g.T_CODES, i)
            orc.exps[i] = gpu.get(g.T_EXPS, i)
            orc.pbits[i] = bits
            orc.p_mode[0] = 1                 # buffers were published in the single-buffer convention
        orc.w[i] = gpu.get(g.T_COUNTERS, i)[0]
    assert gpu.interact([[2, 0], [1, 3]], bits, mode) == 0
    assert orc.interact([[1, 3]], bits, mode) == 0            # one of the launch's pairs
    for i in (1, 3):
        assert np.array_equal(gpu.get(g.T_X, i).view(np.uint32), orc.X[i].view(np.uint32))
        assert np.array_equal(gpu.get(g.T_CODES, i)[: orc.nblk * 128 * bits], orc.packed_codes(i, bits))
        assert np.array_equal(gpu.get(g.T_EXPS, i), orc.exps[i])
        if mode == 1:
            assert np.array_equal(gpu.get(g.T_B, i).view(np.uint32), orc.B[i].view(np.uint32))
    # tail padding of the communication buffer stays zero
    assert not gpu.get(g.T_CODES, 1)[d * bits // 8: orc.nblk * 128 * bits].any()


@pytest.mark.parametrize("workload", ["regular32_resnet18_b8_nb", "complete16_resnet50_b4", "regular256_d1m_b2_lsq_nb"])
def test_full_store_launch_checked_on_the_pair_with_the_highest_node(workload):
    """The benchmark's store and launch shape at full size (32 x 11.7 M, 16 x 25.6 M and 256 x 1 M coordinates: row
    offsets beyond 2^31 bytes, up to 128 pairs per launch from the benchmark's own schedule); the oracle recomputes
    the pair that contains the last node, and that node's local steps. The objective is the synthetic one in all three (the least-squares data
    of the 256-node workload is covered at 32 nodes below), with the oracle's own initial state switched off: its
    rows for the checked pair are copies of the CUDA state."""
    import bench
    wl = bench.WORKLOADS[workload]
    n, d, bits, mode = wl["n"], wl["d"], wl["bits"], wl["mode"]
    cfg = dict(objective=1, nonblocking=mode, grad_std=float(np.sqrt(1e-3)), drift_std=float(np.sqrt(0.05)))
    gpu = g.Swarm(n, d, wl["topology"], wl["degree"], wl["seed"])
    gpu.configure(**cfg)
    sched = bench.PairSchedule(wl, gpu.get_all(g.T_ADJ))
    pairs = sched.next()
    assert len(pairs) >= wl["pairs"] * 3 // 4
    if mode == 1:
        assert gpu.publish(bits) == 0
    sample = [p for p in pairs.tolist() if n - 1 in p] or [pairs[-1].tolist()]
    a, b = sample[0]
    last = max(a, b)
    x_before = gpu.get(g.T_X, last).copy()
    assert gpu.local_steps(pairs.reshape(-1), 2, 0.05) == 0       # pending updates for the one-way exchange
    orc = o.OracleSwarm(n, d, wl["topology"], wl["degree"], wl["seed"])
    orc.configure(objective=1, nonblocking=mode, grad_std=cfg["grad_std"], drift_std=cfg["drift_std"], init_std=0.0)
    # the last node's two local steps, recomputed from its row before the steps
    orc.X[last] = x_before
    orc.drift[last] = gpu.get(g.T_SCALARS, last)[1]
    assert orc.local_steps([last], 2, 0.05) == 0
    assert rel_err(gpu.get(g.T_X, last), orc.X[last]) < 1e-6
    for i in (a, b):
        orc.X[i] = gpu.get(g.T_X, i)
        orc.w[i] = gpu.get(g.T_COUNTERS, i)[0]
        if mode == 1:
            orc.B[i] = gpu.get(g.T_B, i)
            orc.codes[i] = gpu.get(g.T_CODES, i)
            orc.exps[i] = gpu.get(g.T_EXPS, i)
    if mode == 1:
        orc.pbits[:] = bits
        orc.p_mode[0] = 1
    assert gpu.interact(pairs, bits, mode) == 0
    assert orc.interact([[a, b]], bits, mode) == 0
    for i in (a, b):
        assert np.array_equal(gpu.get(g.T_X, i).view(np.uint32), orc.X[i].view(np.uint32)), i
        assert np.array_equal(gpu.get(g.T_CODES, i)[: orc.nblk * 128 * bits], orc.packed_codes(i, bits)), i
        assert np.array_equal(gpu.get(g.T_EXPS, i), orc.exps[i]), i
        if mode == 1:
            assert np.array_equal(gpu.get(g.T_B, i).view(np.uint32), orc.B[i].view(np.uint32)), i
    # a bystander of the launch with a high node id kept its rows unless it was in a pair
    touched = set(pairs.reshape(-1).tolist())
    idle = [i for i in range(n - 1, -1, -1) if i not in touched]
    if idle:
        assert gpu.get(g.T_COUNTERS, idle[0])[0] == (1 if mode == 1 else 0)


def test_config1_trajectory_teacher_forced():
    """n = 8, d = 4096, least squares 64 x 4096, H = 2, batch 16, lr = 0.05, 8-bit, one pair per
    interaction, seed 0: local steps within tolerance, interactions bit-exact."""
    from tests.parity import assert_store_equal, inject, make_pair
    cfg = dict(objective=2, lsq_m=64, lsq_batch=16, lsq_dtype=0, lsq_groups=0, lsq_noise_std=float(np.sqrt(0.1)))
    orc, gpu = make_pair(8, 4096, "complete", seed=0, **cfg)
    inject(orc, gpu)
    for t in range(40):
        pairs = orc.sample_pairs(1)
        assert np.array_equal(gpu.sample_pairs(1), pairs)
        nodes = pairs.reshape(-1)
        assert orc.local_steps(nodes, 2, 0.05) == 0 and gpu.local_steps(nodes, 2, 0.05) == 0
        for i in nodes:
            assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < 1e-6
        inject(orc, gpu, what=("X",))
        assert orc.interact(pairs, 8) == 0 and gpu.interact(pairs, 8) == 0
    assert_store_equal(orc, gpu, 8)
    assert abs(gpu.potential() - orc.potential()) <= 1e-9 * orc.potential()


def test_config5_shape_tensor_core_steps_and_two_bit_interaction():
    """d = 2^20, bf16 least-squares data shared by groups of 16 nodes, batch 64 (the tensor-core path with
    128 k-chunks per unit), then a 2-bit non-blocking launch of 16 pairs: reduced in n and in the rows per
    data matrix (32 nodes, 2 matrices of 64 rows) so that the oracle finishes in under a minute."""
    from tests.parity import assert_store_equal, inject, make_pair
    n, d = 32, 1 << 20
    cfg = dict(objective=2, nonblocking=1, lsq_m=64, lsq_batch=64, lsq_dtype=1, lsq_groups=2,
               lsq_noise_std=float(np.sqrt(0.1)))
    orc, gpu = make_pair(n, d, "regular", 8, seed=5, **cfg)
    inject(orc, gpu)
    nodes = list(range(n))
    assert orc.local_steps(nodes, 2, 0.05) == 0 and gpu.local_steps(nodes, 2, 0.05) == 0
    gpu.sync()
    for i in range(n):
        assert rel_err(gpu.get(g.T_X, i), orc.X[i]) < 1e-6, i
    inject(orc, gpu, what=("X",))
    pairs = orc.sample_pairs(16)
    assert np.array_equal(gpu.sample_pairs(16), pairs) and len(pairs) >= 8
    assert orc.interact(pairs, 2, o.NONBLOCKING, threads=8) == 0 and gpu.interact(pairs, 2, g.NONBLOCKING) == 0
    assert_store_equal(orc, gpu, 2)
    assert abs(gpu.potential() - orc.potential()) <= 1e-9 * orc.potential()


def test_config5_full_size_tensor_core_steps_on_the_last_data_matrix():
    """The 256-node store at full size (16 data matrices of 512 x 2^20 bf16: row offsets up to 16 GiB into the
    data): all nodes take the workload's four local steps on the tensor cores, as in the benchmark (one group of four:
    one pass for the scores, one for the updates); the oracle recomputes the 16 nodes of the last data matrix step by
    step from the rows that matrix's minibatches drew, read back row by row."""
    import bench
    wl = bench.WORKLOADS["regular256_d1m_b2_lsq_nb"]
    n, d, cfg = wl["n"], wl["d"], wl["cfg"]
    m, batch, groups = cfg["lsq_m"], cfg["lsq_batch"], cfg["lsq_groups"]
    per = n // groups
    gpu = g.Swarm(n, d, wl["topology"], wl["degree"], wl["seed"])
    gpu.configure(**cfg)
    unit = list(range(n - per, n))
    x0 = [gpu.get(g.T_X, i).copy() for i in unit]
    # the rows that the last matrix's first four minibatches draw, from the oracle's own sampler: they depend on
    # the seed, the matrix id, the step counter, m and the batch size only, so a short-model oracle gives them
    tiny = o.OracleSwarm(n, 8, wl["topology"], wl["degree"], wl["seed"])
    tiny.configure(**dict(cfg, nonblocking=0))
    H = wl["H"]
    assert H == 4
    drawn = [tiny.minibatch_rows(n - 1, step) for step in range(H)]
    assert all(len(r) == batch and r.max() < m for r in drawn) and not np.array_equal(drawn[0], drawn[1])
    assert len(set(np.concatenate(drawn).tolist())) < H * batch       # minibatches share rows: the corrections matter
    assert gpu.local_steps(np.arange(n), H, wl["lr"]) == 0
    gpu.sync()
    # a 16-node oracle whose one data matrix holds exactly those rows (4 x 64) and the labels that go with them
    orc = o.OracleSwarm(per, d, "complete", seed=1)
    orc.configure(objective=2, lsq_m=H * batch, lsq_batch=batch, lsq_dtype=1, lsq_groups=1, init_std=0.0)
    for step in range(H):
        for s_idx, r in enumerate(drawn[step]):
            orc.A[0, step * batch + s_idx] = gpu.get_data_rows(groups - 1, int(r), 1)[0]
    for j, node in enumerate(unit):
        labels = gpu.get(g.T_BVEC, node)
        for step in range(H):
            orc.bvec[j, step * batch:(step + 1) * batch] = labels[drawn[step]]
        orc.X[j] = x0[j]
    for step in range(H):
        for j in range(per):
            assert orc.local_step_on_rows(j, np.arange(step * batch, (step + 1) * batch), wl["lr"]) == 0
    for j, node in enumerate(unit):
        got = gpu.get(g.T_X, node)
        assert not np.array_equal(got, x0[j])
        assert rel_err(got, orc.X[j]) < 1e-6, node
    assert gpu._L.swarm_get_data_rows(gpu._h, groups, 0, 1, x0[0].ctypes.data, d * 4) == g.ERANGE
    assert gpu._L.swarm_get_data_rows(gpu._h, 0, m, 1, x0[0].ctypes.data, d * 4) == g.ERANGE


@pytest.mark.parametrize("workload", ["regular32_resnet18_b8_nb", "complete16_resnet50_b4", "complete16_resnet50_b8"])
def test_one_call_step_equals_the_two_calls_at_the_full_store(workload):
    """The benchmark runs these workloads through swarm_step (local steps inside the interaction kernel). At the
    full store and with the benchmark's own launch lists, three such steps must leave every model, snapshot, buffer
    and counter of the swarm bit-identical to swarm_local_steps + swarm_interact, which the tests above tie to the
    oracle."""
    import bench
    wl = bench.WORKLOADS[workload]
    n, d, bits, mode = wl["n"], wl["d"], wl["bits"], wl["mode"]
    one = g.Swarm(n, d, wl["topology"], wl["degree"], wl["seed"])
    two = g.Swarm(n, d, wl["topology"], wl["degree"], wl["seed"])
    one.configure(**wl["cfg"])
    two.configure(**wl["cfg"])
    sched = bench.PairSchedule(wl, one.get_all(g.T_ADJ))
    for _ in range(3):
        pairs = sched.next()
        assert two.local_steps(pairs.reshape(-1), wl["H"], wl["lr"]) == 0
        assert two.interact(pairs, bits, mode) == 0
        before = one.kernel_launches()
        assert one.step(pairs, wl["H"], wl["lr"], bits, mode, True) == 0
    assert one.kernel_launches() - before == 1
    rows = (g.T_X, g.T_CODES, g.T_EXPS, g.T_COUNTERS) + ((g.T_B,) if mode else ())
    for i in range(n):
        for which in rows:
            assert np.array_equal(one.get(which, i).view(np.uint8), two.get(which, i).view(np.uint8)), (which, i)
    assert one.potential() == two.potential()
