"""The allocation-free potential entry point against the context-based one.

Some users of the library hold a fixed device-memory pool, or run inside another component's step, and may
not allocate; for them `swarm_potential_static` keeps its scratch in a fixed array inside the library. This
test calls it through the C ABI twice in a row on different states and compares with `swarm_potential`.
Collected last on purpose."""
import numpy as np
import pytest

from paper_1910_12308_b200 import binding as g

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,d", [(8, 5000), (3, 1), (16, 1 << 20)])
def test_static_potential_matches_context_potential_twice_in_a_row(n, d):
    import torch
    sw = g.Swarm(n, d, "complete", seed=77)
    sw.configure(offset_std=0.2)
    x_ptr, pitch = sw.model_ptr()
    out = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    stream = torch.cuda.current_stream()
    sw.set_stream(stream)
    before = torch.cuda.memory_allocated()
    for call in range(2):
        want = sw.potential()
        assert g.potential_static(x_ptr, n, d, pitch, out.data_ptr(), stream) == 0
        torch.cuda.synchronize()
        got = float(out.item())
        assert want > 0
        assert abs(got - want) <= 1e-12 * want, (call, got, want)
        # second call sees a different state and a scratch array that still holds the first call's sums
        assert sw.interact([[0, 1]], 8) == 0
    assert torch.cuda.memory_allocated() == before


def test_static_potential_on_a_plain_tensor_and_size_limit():
    import torch
    torch.manual_seed(0)
    n, d = 5, 1003                       # pitch not a multiple of 4: element-wise path
    x = (torch.randn(n, d, device="cuda") * 3 + 100).contiguous()
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    assert g.potential_static(x.data_ptr(), n, d, d, out.data_ptr(), torch.cuda.current_stream()) == 0
    torch.cuda.synchronize()
    xd = x.double()
    want = float(((xd - xd.mean(0)) ** 2).sum().item())
    assert abs(float(out.item()) - want) <= 1e-9 * want
    # beyond the fixed capacity: rejected before anything is launched, output untouched
    out.fill_(-5.0)
    assert g.potential_static(x.data_ptr(), n, g.STATIC_MAX_D + 1, g.STATIC_MAX_D + 1, out.data_ptr(), None) == -1
    assert g.potential_static(0, n, d, d, out.data_ptr(), None) == -1
    assert g.potential_static(x.data_ptr(), 1, d, d, out.data_ptr(), None) == -1
    assert g.potential_static(x.data_ptr(), n, d, d - 1, out.data_ptr(), None) == -1
    torch.cuda.synchronize()
    assert float(out.item()) == -5.0


@pytest.mark.parametrize("offset,d,pitch", [(1, 1000, 1004), (2, 4099, 4100), (3, 17, 20), (4, 1000, 1004), (1, 1000, 1001)])
def test_static_potential_on_a_view_that_starts_off_a_16_byte_boundary(offset, d, pitch):
    """A slice of a larger tensor: the pitch may be a multiple of four floats while the first row starts one,
    two or three floats past a 16-byte boundary. Such rows are read element by element; offset 4 is aligned
    again and takes the 128-bit loads."""
    import torch
    torch.manual_seed(offset)
    n = 7
    store = (torch.randn(n * pitch + 8, device="cuda") * 2 - 30).contiguous()
    assert store.data_ptr() % 16 == 0
    view = store[offset: offset + n * pitch].view(n, pitch)[:, :d]
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    for _ in range(2):
        assert g.potential_static(store.data_ptr() + 4 * offset, n, d, pitch, out.data_ptr(),
                                  torch.cuda.current_stream()) == 0
        torch.cuda.synchronize()
        xd = view.double()
        want = float(((xd - xd.mean(0)) ** 2).sum().item())
        assert abs(float(out.item()) - want) <= 1e-9 * want
    # addresses that cannot be a float or a double are refused before anything is launched
    assert g.potential_static(store.data_ptr() + 2, n, d, pitch, out.data_ptr(), None) == -1
    assert g.potential_static(store.data_ptr(), n, d, pitch, out.data_ptr() + 4, None) == -1
