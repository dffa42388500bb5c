"""CPU-side checks of the boundary: the library loads, exports every symbol the header declares,
and fails loudly (no fallback) when no device is present."""
import ctypes as C
import os
import re

import pytest

from paper_1910_12308_b200 import binding as g

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "swarm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(swarm_[a-z_]+)\s*\(", text)) - {"swarm_alloc_fn", "swarm_free_fn"})


def test_library_exports_every_declared_symbol():
    L = g.load()
    names = declared_symbols()
    assert len(names) >= 20
    for name in names:
        assert hasattr(L, name), name
    assert sorted(g.EXPORTS) == names


def test_error_strings():
    L = g.load()
    for code in range(0, -7, -1):
        assert L.swarm_strerror(code)
    assert L.swarm_strerror(-99) == b"unknown error"


def test_argument_validation_needs_no_device():
    L = g.load()
    h = C.c_void_p()
    assert L.swarm_init(C.byref(h), 1, 16, g.SwarmTopology(0, 0), 0) == -1        # n < 2
    assert L.swarm_init(C.byref(h), 4, 0, g.SwarmTopology(0, 0), 0) == -1         # d < 1
    assert L.swarm_init(None, 4, 16, g.SwarmTopology(0, 0), 0) == -1
    assert L.swarm_interact(None, None, 0, 8, 0) == -1
    assert L.swarm_potential(None, None) == -1
    assert L.swarm_step(None, None, 0, 1, 0.1, 8, 0, 1) == -1
    assert L.swarm_run_sequence(None, None, 0, 1, 0.1, 8, 1) == -1
    assert L.swarm_set_own_prefix(None, 8) == -1 and L.swarm_get_own_prefix(None, None) == -1
    assert L.swarm_track_staleness(None, 1) == -1 and L.swarm_aux_potentials(None, None) == -1
    assert L.swarm_get_tensor_async(None, 0, 0, None, 0) == -1
    out = C.c_double()
    assert L.swarm_potential_static(None, 4, 16, 16, C.addressof(out), None) == -1


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("device present")
    L = g.load()
    h = C.c_void_p()
    assert L.swarm_init(C.byref(h), 4, 16, g.SwarmTopology(0, 0), 0) == -6        # CUDA error, not a CPU path
    assert not h.value
    with pytest.raises(RuntimeError):
        g.Swarm(4, 16)


def test_product_package_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_1910_12308_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower().replace("test oracle", ""), os.path.join(dirpath, f)
