"""Checkpoint / resume through swarm_get_tensor / swarm_set_tensor, and work on a non-default stream."""
import numpy as np
import pytest

from paper_1910_12308_b200 import binding as g

pytestmark = pytest.mark.gpu

ROWS = (g.T_X, g.T_B, g.T_CODES, g.T_EXPS, g.T_OWN, g.T_OEXPS, g.T_COUNTERS, g.T_CLOCKS)


def snapshot(sw):
    state = {which: sw.get_all(which) for which in ROWS}
    state["ctx"] = sw.get_state() + (sw.get_buffer_mode(),)
    return state


def restore(sw, state):
    for which in ROWS:
        for i in range(sw.n):
            sw.set(which, i, state[which][i])
    launch, stale, mode = state["ctx"]
    sw.set_state(launch, stale)
    sw.set_buffer_mode(mode)


def run(sw, rounds):
    for _ in range(rounds):
        pairs = sw.sample_pairs(3)
        assert sw.local_steps(pairs.reshape(-1), 2, 0.05) == 0
        assert sw.interact(pairs, 8, g.REGISTERS) == 0
    pairs = sw.sample_pairs(2)
    assert sw.interact(pairs, 4, g.NONBLOCKING) == 0
    assert sw.interact(sw.sample_pairs(2), 8, g.BLOCKING) == 0


def test_checkpoint_and_resume_reproduce_the_run_bit_for_bit():
    cfg = dict(objective=1, nonblocking=2, grad_std=0.03, drift_std=0.1, offset_std=0.05)
    a = g.Swarm(8, 3000, "regular", 4, seed=5)
    a.configure(**cfg)
    run(a, 3)
    saved = snapshot(a)
    run(a, 4)
    want = snapshot(a)
    b = g.Swarm(8, 3000, "regular", 4, seed=5)     # same seed and workload, fresh context
    b.configure(**cfg)
    restore(b, saved)
    run(b, 4)
    got = snapshot(b)
    for which in ROWS:
        assert np.array_equal(got[which].view(np.uint8), want[which].view(np.uint8)), which
    assert got["ctx"] == want["ctx"]
    assert abs(a.potential() - b.potential()) == 0.0


def test_non_default_stream():
    import torch
    stream = torch.cuda.Stream()
    ref = g.Swarm(6, 5000, "ring", seed=9)
    sw = g.Swarm(6, 5000, "ring", seed=9, stream=stream)
    for s in (ref, sw):
        s.configure(objective=1, grad_std=0.02, offset_std=0.1)
    with torch.cuda.stream(stream):
        out = torch.empty(5000, device="cuda")
        for s in (ref, sw):
            for r in range(5):
                pairs = [[0, 1], [2, 3]] if r % 2 == 0 else [[1, 2], [4, 5]]
                assert s.local_steps([0, 1, 2, 3, 4, 5], 1, 0.05) == 0
                assert s.interact(pairs, 4) == 0
        mu = sw.mean_model(out)
        sw.sync()
    assert np.array_equal(sw.get_all(g.T_X), ref.get_all(g.T_X))
    assert np.array_equal(mu.cpu().numpy(), ref.mean_model().cpu().numpy())
    assert sw.potential() == ref.potential()


def test_asynchronous_row_read_arrives_after_sync():
    import torch
    sw = g.Swarm(4, 3000, "complete", 0, 2)
    sw.configure(objective=1, grad_std=0.1, offset_std=0.2)
    out = torch.zeros(3000, dtype=torch.float32).pin_memory()
    exps = torch.zeros(sw.nblk, dtype=torch.int8).pin_memory()
    assert sw.interact([[0, 1]], 8) == 0
    assert sw.get_async(g.T_X, 1, out) == 0 and sw.get_async(g.T_EXPS, 1, exps) == 0
    sw.sync()
    assert np.array_equal(out.numpy(), sw.get(g.T_X, 1)) and np.array_equal(exps.numpy(), sw.get(g.T_EXPS, 1))
    small = torch.zeros(3, dtype=torch.uint32).pin_memory() if hasattr(torch, "uint32") else np.zeros(3, np.uint32)
    assert sw.get_async(g.T_COUNTERS, 0, small) == g.EINVAL          # host-side rows have no asynchronous form
    assert sw.get_async(g.T_X, 9, out) == g.ERANGE
    assert sw.get_async(g.T_X, 0, exps) == g.EINVAL                  # size mismatch


def test_queued_row_reads_keep_the_value_of_their_point_in_the_stream():
    """A queued read returns the row as it was when queued, even if later launches change it before the
    synchronising call; any synchronising call delivers (here the potential), destinations need not be pinned,
    and more rows than the context's ring holds are still all delivered."""
    sw = g.Swarm(4, 5000, "complete", 0, 3)
    sw.configure(offset_std=0.2)
    before = sw.get(g.T_X, 0).copy()
    first = np.zeros(5000, dtype=np.float32)                         # pageable memory
    assert sw.get_async(g.T_X, 0, first) == 0
    assert sw.interact([[0, 1]], 8) == 0                             # changes row 0 after the read was queued
    second = np.zeros(5000, dtype=np.float32)
    assert sw.get_async(g.T_X, 0, second) == 0
    sw.potential()                                                   # synchronises: both rows are there
    assert np.array_equal(first, before)
    assert np.array_equal(second, sw.get(g.T_X, 0)) and not np.array_equal(first, second)
    # 80 rows of 20,000 bytes exceed the 1 MiB ring: the call that finds it full delivers the queued ones first
    outs = [np.zeros(5000, dtype=np.float32) for _ in range(80)]
    rows = [sw.get(g.T_X, i % 4) for i in range(4)]
    for i, o_ in enumerate(outs):
        assert sw.get_async(g.T_X, i % 4, o_) == 0
    sw.sync()
    for i, o_ in enumerate(outs):
        assert np.array_equal(o_, rows[i % 4])
