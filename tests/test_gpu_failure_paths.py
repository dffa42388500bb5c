"""Failure paths that can be exercised on a healthy GPU: a bounded device wait that runs out (made to run out
by a zero poll budget, never by a fault or a hang) and a device allocation that fails inside swarm_configure."""
import numpy as np
import pytest

from paper_1910_12308_b200 import binding as g

pytestmark = pytest.mark.gpu

CUDA_ERROR_LAUNCH_TIMEOUT = 702     # cudaErrorLaunchTimeout, what an expired wait is reported as
LSQ_BF16 = dict(objective=2, lsq_m=32, lsq_batch=16, lsq_dtype=1, lsq_groups=2, lsq_noise_std=0.1)


@pytest.mark.parametrize("d", [700, 20000])
def test_expired_device_wait_returns_an_error_status_and_touches_no_model(d):
    n = 8
    sw = g.Swarm(n, d, "complete", seed=21)
    sw.configure(**LSQ_BF16)
    before = sw.get_all(g.T_X)
    assert sw.set_wait_limit(0) == 0            # every wait on a tensor-core commit gives up at once
    assert sw.local_steps(np.arange(n), 2, 0.05) == 0       # the launch itself succeeds
    with pytest.raises(g.SwarmError) as err:
        sw.sync()
    assert err.value.code == g.ECUDA
    assert sw.last_cuda_error() == CUDA_ERROR_LAUNCH_TIMEOUT
    # the step that gave up wrote nothing, and the kernels queued behind it returned at once: a row read still
    # delivers the row (and reports the expired wait, like every synchronising call from now on)
    for i in range(n):
        row = np.empty_like(before[i])
        assert sw._L.swarm_get_tensor(sw._h, g.T_X, i, row.ctypes.data, row.nbytes) == g.ECUDA
        assert np.array_equal(row, before[i])
    assert sw.set_wait_limit(1 << 32) == g.EINVAL
    # every synchronising call keeps reporting it ...
    with pytest.raises(g.SwarmError):
        sw.potential()
    # ... until the context is rebuilt from its seed
    assert sw.set_wait_limit(-1) == 0
    sw.configure(**LSQ_BF16)
    assert np.array_equal(sw.get_all(g.T_X), before)
    assert sw.local_steps(np.arange(n), 2, 0.05) == 0
    sw.sync()
    after = sw.get_all(g.T_X)
    assert not np.array_equal(after, before)
    # a fresh context takes the same steps to the same models
    fresh = g.Swarm(n, d, "complete", seed=21)
    fresh.configure(**LSQ_BF16)
    assert fresh.local_steps(np.arange(n), 2, 0.05) == 0
    assert np.array_equal(fresh.get_all(g.T_X), after)


def test_configure_out_of_memory_leaves_the_default_configuration():
    import torch
    L = g.load()
    blocks, state = {}, {"budget": None}

    def alloc(nbytes, _user):
        if state["budget"] is not None:
            if state["budget"] == 0:
                return None
            state["budget"] -= 1
        t = torch.empty(int(nbytes), dtype=torch.uint8, device="cuda")
        blocks[t.data_ptr()] = t
        return t.data_ptr()

    def free(ptr, _user):
        blocks.pop(ptr, None)

    a_cb, f_cb = g.ALLOC_FN(alloc), g.FREE_FN(free)
    assert L.swarm_set_allocator(a_cb, f_cb, None) == 0
    n, d = 8, 3000
    want = dict(objective=2, nonblocking=2, lsq_m=32, lsq_batch=16, lsq_dtype=1, lsq_groups=2, lsq_noise_std=0.1)
    try:
        sw = g.Swarm(n, d, "complete", seed=5, torch_memory=False)
        default_x = sw.get_all(g.T_X)
        needed = 11      # snapshots, own registers + exponents, data, labels, x*, two scratch arrays, tensor-core scratch x 2, Gram matrices
        for k in range(needed + 1):
            state["budget"] = k
            if k < needed:
                with pytest.raises(g.SwarmError) as err:
                    sw.configure(**want)
                assert err.value.code == g.ENOMEM, k
                state["budget"] = None
                # the context is in the state swarm_init leaves: no objective, no snapshots, models from the seed
                assert sw.local_steps([0, 1], 1, 0.05) == g.ESTATE
                assert sw.interact([[0, 1]], 8, g.NONBLOCKING) == g.ESTATE
                assert sw.interact([[0, 1]], 8, g.REGISTERS) == g.ESTATE
                assert sw.publish(8) == g.ESTATE
                assert np.array_equal(sw.get_all(g.T_X), default_x)
                assert sw.interact([[0, 1]], 8, g.BLOCKING) == 0
                sw.sync()
            else:
                sw.configure(**want)
                state["budget"] = None
                assert sw.local_steps([0, 1], 1, 0.05) == 0
                assert sw.interact([[0, 1]], 8, g.REGISTERS) == 0
                sw.sync()
        sw.close()
    finally:
        state["budget"] = None
        if g._alloc_cb is not None:
            L.swarm_set_allocator(g._alloc_cb, g._free_cb, None)
        else:
            L.swarm_set_allocator(g.ALLOC_FN(), g.FREE_FN(), None)
