"""Thin ctypes binding of the C ABI declared in include/swarm.h.

Argument marshalling only: every step of the method runs in the CUDA library. PyTorch supplies
device memory (through the allocator hook) and the stream. There is no CPU path: the binding
raises at import if the shared library is missing and cannot be built.
"""
import atexit
import ctypes as C
import os
import sys
import weakref

import numpy as np

from . import build as _build

_HERE = os.path.dirname(os.path.abspath(__file__))

BLOCKING, NONBLOCKING, REGISTERS = 0, 1, 2
TOPO_COMPLETE, TOPO_RING, TOPO_REGULAR = 0, 1, 2
OBJ_NONE, OBJ_SYNTH, OBJ_LSQ, OBJ_LOGISTIC = 0, 1, 2, 3
F32, BF16 = 0, 1
OK, EINVAL, ERANGE, EPAIR, ESTATE, ENOMEM, ECUDA = 0, -1, -2, -3, -4, -5, -6
(T_X, T_B, T_CODES, T_EXPS, T_ADJ, T_A, T_BVEC, T_XSTAR, T_SCALARS, T_COUNTERS, T_OWN, T_OEXPS, T_CLOCKS, T_MU_RECORD,
 T_A_RECORD, T_GRAM) = range(16)
TOPOLOGY = {"complete": TOPO_COMPLETE, "ring": TOPO_RING, "regular": TOPO_REGULAR}

EXPORTS = [
    "swarm_set_allocator", "swarm_init", "swarm_local_steps", "swarm_local_steps_geometric", "swarm_interact", "swarm_interact_prefixed", "swarm_step", "swarm_run_sequence", "swarm_mean_model",
    "swarm_potential", "swarm_track_staleness", "swarm_aux_potentials", "swarm_configure", "swarm_sample_pairs", "swarm_publish", "swarm_register_publish", "swarm_set_own_prefix", "swarm_get_own_prefix", "swarm_get_buffer_mode",
    "swarm_set_buffer_mode", "swarm_get_tensor", "swarm_get_data_rows", "swarm_get_tensor_async",
    "swarm_set_tensor", "swarm_get_state", "swarm_set_state", "swarm_model_ptr", "swarm_set_stream",
    "swarm_sync", "swarm_set_wait_limit", "swarm_potential_static", "swarm_kernel_launches", "swarm_last_cuda_error", "swarm_strerror", "swarm_destroy",
]


class SwarmPair(C.Structure):
    _fields_ = [("a", C.c_int32), ("b", C.c_int32)]


class SwarmTopology(C.Structure):
    _fields_ = [("kind", C.c_int32), ("degree", C.c_int32)]


class SwarmConfig(C.Structure):
    _fields_ = [
        ("objective", C.c_int32), ("nonblocking", C.c_int32),
        ("init_std", C.c_float), ("offset_std", C.c_float),
        ("grad_std", C.c_float), ("drift_std", C.c_float),
        ("lsq_m", C.c_int32), ("lsq_batch", C.c_int32), ("lsq_dtype", C.c_int32), ("lsq_groups", C.c_int32),
        ("lsq_noise_std", C.c_float),
    ]


ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_size_t, C.c_void_p)
FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)

_lib = None


class SwarmError(RuntimeError):
    def __init__(self, code, what=""):
        self.code = code
        msg = load().swarm_strerror(code).decode()
        super().__init__(f"{what}: {msg} ({code})" if what else f"{msg} ({code})")


def library_path():
    """The in-tree library; SWARM_B200_LIBRARY names another build of it to load instead (for comparing builds)."""
    return os.environ.get("SWARM_B200_LIBRARY") or os.path.join(_HERE, "libswarm_b200.so")


def load():
    """Load (building first if the sources are newer) the CUDA library. Never falls back."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path) or os.environ.get("SWARM_REBUILD"):
        path = _build.build()
    L = C.CDLL(path)
    vp, i32, i64, u32, u64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64, C.c_float
    sig = {
        "swarm_set_allocator": (C.c_int, [ALLOC_FN, FREE_FN, vp]),
        "swarm_init": (C.c_int, [C.POINTER(vp), i32, i64, SwarmTopology, u64]),
        "swarm_local_steps": (C.c_int, [vp, C.POINTER(i32), i32, i32, f32]),
        "swarm_local_steps_geometric": (C.c_int, [vp, C.POINTER(i32), i32, i32, f32, C.POINTER(i32)]),
        "swarm_interact": (C.c_int, [vp, C.POINTER(SwarmPair), i32, i32, i32]),
        "swarm_interact_prefixed": (C.c_int, [vp, C.POINTER(SwarmPair), C.POINTER(i32), i32, i32]),
        "swarm_step": (C.c_int, [vp, C.POINTER(SwarmPair), i32, i32, f32, i32, i32, i32]),
        "swarm_run_sequence": (C.c_int, [vp, C.POINTER(SwarmPair), i32, i32, f32, i32, i32]),
        "swarm_mean_model": (C.c_int, [vp, vp]),
        "swarm_potential": (C.c_int, [vp, C.POINTER(C.c_double)]),
        "swarm_track_staleness": (C.c_int, [vp, i32]),
        "swarm_aux_potentials": (C.c_int, [vp, C.POINTER(C.c_double)]),
        "swarm_configure": (C.c_int, [vp, C.POINTER(SwarmConfig)]),
        "swarm_sample_pairs": (C.c_int, [vp, i32, C.POINTER(SwarmPair), C.POINTER(i32)]),
        "swarm_publish": (C.c_int, [vp, i32]),
        "swarm_register_publish": (C.c_int, [vp, i32]),
        "swarm_set_own_prefix": (C.c_int, [vp, i32]),
        "swarm_get_own_prefix": (C.c_int, [vp, C.POINTER(i32)]),
        "swarm_get_buffer_mode": (C.c_int, [vp, C.POINTER(i32)]),
        "swarm_set_buffer_mode": (C.c_int, [vp, i32]),
        "swarm_get_tensor": (C.c_int, [vp, i32, i32, vp, C.c_size_t]),
        "swarm_get_tensor_async": (C.c_int, [vp, i32, i32, vp, C.c_size_t]),
        "swarm_get_data_rows": (C.c_int, [vp, i32, i32, i32, vp, C.c_size_t]),
        "swarm_set_tensor": (C.c_int, [vp, i32, i32, vp, C.c_size_t]),
        "swarm_get_state": (C.c_int, [vp, C.POINTER(u32), C.POINTER(i32)]),
        "swarm_set_state": (C.c_int, [vp, u32, i32]),
        "swarm_model_ptr": (C.c_int, [vp, C.POINTER(vp), C.POINTER(i64)]),
        "swarm_potential_static": (C.c_int, [vp, i32, i64, i64, vp, vp]),
        "swarm_set_stream": (C.c_int, [vp, vp]),
        "swarm_sync": (C.c_int, [vp]),
        "swarm_set_wait_limit": (C.c_int, [vp, i64]),
        "swarm_kernel_launches": (i64, [vp]),
        "swarm_last_cuda_error": (C.c_int, [vp]),
        "swarm_strerror": (C.c_char_p, [C.c_int]),
        "swarm_destroy": (None, [vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype = res
        fn.argtypes = args
    _lib = L
    return L


# ---- torch-backed device memory ---------------------------------------------------------------
_torch_blocks = {}
_alloc_cb = None
_free_cb = None


def use_torch_allocator():
    """Route the library's device allocations through PyTorch's caching allocator."""
    global _alloc_cb, _free_cb
    import torch

    def _alloc(nbytes, _user):
        try:
            t = torch.empty(int(nbytes), dtype=torch.uint8, device="cuda")
        except Exception:
            return None
        _torch_blocks[t.data_ptr()] = t
        return t.data_ptr()

    def _free(ptr, _user):
        _torch_blocks.pop(ptr, None)

    _alloc_cb, _free_cb = ALLOC_FN(_alloc), FREE_FN(_free)
    rc = load().swarm_set_allocator(_alloc_cb, _free_cb, None)
    if rc != 0:
        raise SwarmError(rc, "swarm_set_allocator")


# Contexts still alive at interpreter exit are destroyed before the interpreter and the framework that
# backs the allocator callbacks are torn down (a destroy during finalisation would call back into them).
_live = weakref.WeakSet()


@atexit.register
def _close_all():
    for sw in list(_live):
        try:
            sw.close()
        except Exception:
            pass


def _pairs_array(pairs):
    pairs = np.ascontiguousarray(pairs, dtype=np.int32).reshape(-1, 2)
    return pairs, pairs.ctypes.data_as(C.POINTER(SwarmPair))


class Swarm:
    """One swarm context on the current CUDA device. Methods mirror the C entry points."""

    def __init__(self, n, d, topology="complete", degree=0, seed=0, torch_memory=True, stream=None):
        L = load()
        if torch_memory:
            import torch
            if not torch.cuda.is_available():
                raise RuntimeError("swarm: no CUDA device; this library has no CPU path")
            if _alloc_cb is None:
                use_torch_allocator()
        kind = TOPOLOGY[topology] if isinstance(topology, str) else int(topology)
        h = C.c_void_p()
        rc = L.swarm_init(C.byref(h), n, d, SwarmTopology(kind, degree), seed)
        if rc != 0:
            raise SwarmError(rc, "swarm_init")
        self._h, self._L = h, L
        _live.add(self)
        self.n, self.d, self.seed = n, d, seed
        self.nblk = (d + 1023) // 1024
        self.cfg = SwarmConfig(OBJ_NONE, 0, 0.1, 0.0, 0.0, 0.0, 0, 0, 0, 0, 0.0)
        self.degree = {TOPO_COMPLETE: n - 1, TOPO_RING: 2}.get(kind, degree)
        if stream is not None:
            self.set_stream(stream)

    # -- lifetime
    def close(self):
        if getattr(self, "_h", None):
            self._L.swarm_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            if sys is None or sys.is_finalizing():
                return
            self.close()
        except Exception:
            pass

    def _check(self, rc, what):
        if rc != 0:
            raise SwarmError(rc, what)

    # -- the five core calls
    def local_steps(self, nodes, H, lr):
        nodes = np.ascontiguousarray(nodes, dtype=np.int32)
        return self._L.swarm_local_steps(self._h, nodes.ctypes.data_as(C.POINTER(C.c_int32)), len(nodes), H, lr)

    def local_steps_geometric(self, nodes, mean_h, lr):
        """Returns (rc, steps taken per listed node)."""
        nodes = np.ascontiguousarray(nodes, dtype=np.int32)
        steps = np.zeros(len(nodes), dtype=np.int32)
        rc = self._L.swarm_local_steps_geometric(self._h, nodes.ctypes.data_as(C.POINTER(C.c_int32)), len(nodes), mean_h,
                                                 lr, steps.ctypes.data_as(C.POINTER(C.c_int32)))
        return rc, steps

    def interact(self, pairs, bits, mode=BLOCKING):
        arr, ptr = _pairs_array(pairs)
        return self._L.swarm_interact(self._h, ptr, len(arr), bits, mode)

    def interact_prefixed(self, pairs, prefixes, bits):
        """Two-register interactions; the initiator of pairs[p] reads prefixes[p] (8 or 16) bits of its
        responder's own register. Returns the C code."""
        arr, ptr = _pairs_array(pairs)
        pf = np.ascontiguousarray(prefixes, dtype=np.int32)
        if len(pf) != len(arr):
            raise ValueError("one prefix per pair")
        return self._L.swarm_interact_prefixed(self._h, ptr, pf.ctypes.data_as(C.POINTER(C.c_int32)), len(arr), bits)

    def step(self, pairs, H, lr, bits, mode=BLOCKING, step_responders=True):
        """H local steps of the nodes in `pairs` (initiators only if step_responders is false), then the
        interactions, in one call; returns the C code."""
        arr, ptr = _pairs_array(pairs)
        return self._L.swarm_step(self._h, ptr, len(arr), H, lr, bits, mode, 1 if step_responders else 0)

    def run_sequence(self, pairs, H, lr, bits, step_responders=True):
        """One interaction per time step, pairs[t] at step t, local steps before each (sequential gossip);
        a single kernel launch for short models with fp32 least-squares data. Returns the C code."""
        arr, ptr = _pairs_array(pairs)
        return self._L.swarm_run_sequence(self._h, ptr, len(arr), H, lr, bits, 1 if step_responders else 0)

    def mean_model(self, out=None):
        import torch
        if out is None:
            out = torch.empty(self.d, dtype=torch.float32, device="cuda")
        self._check(self._L.swarm_mean_model(self._h, out.data_ptr()), "swarm_mean_model")
        return out

    def potential(self):
        g = C.c_double()
        self._check(self._L.swarm_potential(self._h, C.byref(g)), "swarm_potential")
        return g.value

    def set_own_prefix(self, bits):
        """Bits (8 or 16) of a partner's own register that a reader consumes; returns the C code."""
        return int(self._L.swarm_set_own_prefix(self._h, bits))

    def get_own_prefix(self):
        v = C.c_int32()
        self._check(self._L.swarm_get_own_prefix(self._h, C.byref(v)), "swarm_get_own_prefix")
        return v.value

    def track_staleness(self, enable=True):
        """Start (or stop) recording what the auxiliary potentials need; returns the C code."""
        return int(self._L.swarm_track_staleness(self._h, 1 if enable else 0))

    def aux_potentials(self):
        """(Gamma-hat, A_t, B_t) of the staleness analysis."""
        out = (C.c_double * 3)()
        self._check(self._L.swarm_aux_potentials(self._h, out), "swarm_aux_potentials")
        return float(out[0]), float(out[1]), float(out[2])

    # -- auxiliary
    def configure(self, **kw):
        for k, v in kw.items():
            if not hasattr(self.cfg, k):
                raise KeyError(k)
            setattr(self.cfg, k, v)
        self._check(self._L.swarm_configure(self._h, C.byref(self.cfg)), "swarm_configure")

    def sample_pairs(self, max_pairs):
        out = np.zeros((max(max_pairs, 1), 2), dtype=np.int32)
        cnt = C.c_int32()
        self._check(self._L.swarm_sample_pairs(self._h, max_pairs, out.ctypes.data_as(C.POINTER(SwarmPair)),
                                               C.byref(cnt)), "swarm_sample_pairs")
        return out[: cnt.value].copy()

    def publish(self, bits):
        return self._L.swarm_publish(self._h, bits)

    def register_publish(self, bits):
        return self._L.swarm_register_publish(self._h, bits)

    def get_buffer_mode(self):
        m = C.c_int32()
        self._check(self._L.swarm_get_buffer_mode(self._h, C.byref(m)), "swarm_get_buffer_mode")
        return m.value

    def set_buffer_mode(self, mode):
        self._check(self._L.swarm_set_buffer_mode(self._h, mode), "swarm_set_buffer_mode")

    def set_stream(self, stream):
        ptr = getattr(stream, "cuda_stream", stream)
        self._check(self._L.swarm_set_stream(self._h, ptr), "swarm_set_stream")

    def sync(self):
        self._check(self._L.swarm_sync(self._h), "swarm_sync")

    def set_wait_limit(self, polls):
        """Polls after which a device-side wait gives up (negative = default, 0 = at once); returns the C code."""
        return int(self._L.swarm_set_wait_limit(self._h, polls))

    def last_cuda_error(self):
        return int(self._L.swarm_last_cuda_error(self._h))

    def kernel_launches(self):
        return int(self._L.swarm_kernel_launches(self._h))

    def model_ptr(self):
        p, pitch = C.c_void_p(), C.c_int64()
        self._check(self._L.swarm_model_ptr(self._h, C.byref(p), C.byref(pitch)), "swarm_model_ptr")
        return p.value, pitch.value

    def model_tensor(self):
        """The live models as an (n, pitch) float32 torch tensor over the library's own memory (contexts whose
        device memory comes from PyTorch only): for callers that read or restore models in place, on the
        context's stream. Valid until the next configure / close."""
        import torch
        ptr, pitch = self.model_ptr()
        block = _torch_blocks.get(ptr)
        if block is None:
            raise RuntimeError("swarm: the models of this context are not backed by a torch allocation")
        return block[: self.n * pitch * 4].view(torch.float32).view(self.n, pitch)

    # -- state access
    def _row_spec(self, which):
        m = self.cfg.lsq_m
        return {
            T_X: (np.float32, self.d), T_B: (np.float32, self.d), T_CODES: (np.uint8, self.nblk * 1024),
            T_EXPS: (np.int8, self.nblk), T_ADJ: (np.int32, self.degree), T_A: (np.float32, m * self.d),
            T_BVEC: (np.float32, m), T_XSTAR: (np.float32, self.d), T_SCALARS: (np.float32, 3),
            T_COUNTERS: (np.uint32, 3), T_OWN: (np.uint8, self.nblk * 2048), T_OEXPS: (np.int8, self.nblk),
            T_CLOCKS: (np.uint32, 2), T_MU_RECORD: (np.float32, self.d), T_A_RECORD: (np.float64, 1),
            T_GRAM: (np.float32, m * m),
        }[which]

    def get(self, which, node=0):
        dt, count = self._row_spec(which)
        out = np.empty(count, dtype=dt)
        self._check(self._L.swarm_get_tensor(self._h, which, node, out.ctypes.data, out.nbytes), "swarm_get_tensor")
        return out

    def get_data_rows(self, matrix, row0, nrows):
        """Rows row0 .. row0 + nrows - 1 of a least-squares data matrix as an (nrows, d) float array."""
        out = np.empty((nrows, self.d), dtype=np.float32)
        self._check(self._L.swarm_get_data_rows(self._h, matrix, row0, nrows, out.ctypes.data, out.nbytes),
                    "swarm_get_data_rows")
        return out

    def get_async(self, which, node, out):
        """Queue the read of a row into `out` (a pinned torch tensor or array of the row's size) without
        waiting; the data is there after sync(). Returns the C code."""
        ptr = out.data_ptr() if hasattr(out, "data_ptr") else out.ctypes.data
        nbytes = out.numel() * out.element_size() if hasattr(out, "numel") else out.nbytes
        return int(self._L.swarm_get_tensor_async(self._h, which, node, ptr, nbytes))

    def set(self, which, node, values):
        dt, count = self._row_spec(which)
        arr = np.ascontiguousarray(values, dtype=dt).reshape(-1)
        if arr.size != count:
            raise ValueError(f"expected {count} elements, got {arr.size}")
        self._check(self._L.swarm_set_tensor(self._h, which, node, arr.ctypes.data, arr.nbytes), "swarm_set_tensor")

    def get_all(self, which):
        return np.stack([self.get(which, i) for i in range(self.n)])

    def get_state(self):
        launch, stale = C.c_uint32(), C.c_int32()
        self._check(self._L.swarm_get_state(self._h, C.byref(launch), C.byref(stale)), "swarm_get_state")
        return launch.value, stale.value

    def set_state(self, launch, b_stale):
        self._check(self._L.swarm_set_state(self._h, launch, b_stale), "swarm_set_state")


STATIC_MAX_D = 33554432


def potential_static(x_ptr, n, d, pitch, out_ptr, stream=None):
    """Gamma of n caller-held rows (device pointer x_ptr, row pitch in elements) into the device double at
    out_ptr, through the entry point that allocates nothing (for callers that must not allocate: fixed
    memory pools, hooks inside another component's step). Asynchronous on `stream`; returns the C code."""
    ptr = getattr(stream, "cuda_stream", stream)
    return load().swarm_potential_static(x_ptr, n, d, pitch, out_ptr, ptr)
