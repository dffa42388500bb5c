"""ctypes/numpy view of the CPU oracle (oracle/swarm_oracle.cpp).

Test infrastructure only. Importable from tests/, from the smoke check and from the
CPU-baseline leg of the benchmark; never from the product package.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

_lib = None


class OracleConfig(C.Structure):
    _fields_ = [
        ("objective", C.c_int32), ("nonblocking", C.c_int32),
        ("init_std", C.c_float), ("offset_std", C.c_float),
        ("grad_std", C.c_float), ("drift_std", C.c_float),
        ("lsq_m", C.c_int32), ("lsq_batch", C.c_int32), ("lsq_dtype", C.c_int32), ("lsq_groups", C.c_int32),
        ("lsq_noise_std", C.c_float),
    ]


def lib():
    global _lib
    if _lib is not None:
        return _lib
    L = C.CDLL(_build.build())
    u32p, i32p, f32p = C.POINTER(C.c_uint32), C.POINTER(C.c_int32), C.POINTER(C.c_float)
    u8p, i8p, u16p = C.POINTER(C.c_uint8), C.POINTER(C.c_int8), C.POINTER(C.c_uint16)
    vp = C.c_void_p
    sig = {
        "orc_philox": (None, [u32p, u32p, u32p]),
        "orc_uniform_int": (C.c_uint32, [C.c_uint32, C.c_uint32]),
        "orc_uniform_float": (C.c_float, [C.c_uint32]),
        "orc_normal_pair": (None, [C.c_uint32, C.c_uint32, f32p]),
        "orc_exponent": (C.c_int, [C.c_float, C.c_float, C.c_int]),
        "orc_enc_q": (C.c_int32, [C.c_float, C.c_int, C.c_uint32]),
        "orc_code": (C.c_uint32, [C.c_int32, C.c_int]),
        "orc_dec": (C.c_float, [C.c_float, C.c_uint32, C.c_int, C.c_int]),
        "orc_round_bf16": (C.c_float, [C.c_float]),
        "orc_sr_uniforms": (None, [C.c_uint64, C.c_uint32, C.c_uint32, C.c_int64, C.c_int64, u16p]),
        "orc_pack_block": (None, [u8p, C.c_int, C.c_int, u8p]),
        "orc_unpack_block": (None, [u8p, C.c_int, C.c_int, u8p]),
        "orc_create": (vp, [C.c_int32, C.c_int64, C.c_int32, C.c_int32, C.c_uint64]),
        "orc_destroy": (None, [vp]),
        "orc_configure": (C.c_int, [vp, C.POINTER(OracleConfig)]),
        "orc_degree": (C.c_int32, [vp]),
        "orc_nblk": (C.c_int64, [vp]),
        "orc_groups": (C.c_int32, [vp]),
        "orc_adj": (i32p, [vp]),
        "orc_X": (f32p, [vp]), "orc_B": (f32p, [vp]),
        "orc_codes": (u8p, [vp]), "orc_exps": (i8p, [vp]), "orc_pbits": (i32p, [vp]),
        "orc_w": (u32p, [vp]), "orc_ls": (u32p, [vp]), "orc_launch": (u32p, [vp]),
        "orc_b_stale": (i32p, [vp]),
        "orc_A": (f32p, [vp]), "orc_bvec": (f32p, [vp]), "orc_xstar": (f32p, [vp]),
        "orc_offset": (f32p, [vp]), "orc_drift": (f32p, [vp]), "orc_shift": (f32p, [vp]),
        "orc_minibatch_rows": (C.c_int, [vp, C.c_int32, C.c_uint32, i32p]),
        "orc_sample_pairs": (C.c_int, [vp, C.c_int32, i32p, i32p]),
        "orc_local_steps": (C.c_int, [vp, i32p, C.c_int32, C.c_int32, C.c_float]),
        "orc_local_step_on_rows": (C.c_int, [vp, C.c_int32, i32p, C.c_int32, C.c_float]),
        "orc_local_steps_geometric": (C.c_int, [vp, i32p, C.c_int32, C.c_int32, C.c_float, i32p]),
        "orc_interact": (C.c_int, [vp, i32p, C.c_int32, C.c_int32, C.c_int32, C.c_int32]),
        "orc_interact_prefixed": (C.c_int, [vp, i32p, i32p, C.c_int32, C.c_int32, C.c_int32, C.c_int32]),
        "orc_publish": (C.c_int, [vp, C.c_int32]),
        "orc_register_publish": (C.c_int, [vp, C.c_int32]),
        "orc_own": (u8p, [vp]), "orc_set_own_prefix": (C.c_int, [vp, C.c_int32]), "orc_get_own_prefix": (C.c_int32, [vp]), "orc_oexps": (i8p, [vp]), "orc_wo": (u32p, [vp]), "orc_tau": (u32p, [vp]),
        "orc_p_mode": (i32p, [vp]),
        "orc_mean_model": (None, [vp, f32p]),
        "orc_potential": (C.c_double, [vp]),
        "orc_track_staleness": (C.c_int, [vp, C.c_int32]),
        "orc_mu_hist": (f32p, [vp]), "orc_a_hist": (C.POINTER(C.c_double), [vp]),
        "orc_aux_potentials": (C.c_int, [vp, C.POINTER(C.c_double)]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype = res
        fn.argtypes = args
    _lib = L
    return L


def _view(ptr, shape, dtype):
    if not ptr:
        return None
    n = int(np.prod(shape))
    arr = np.ctypeslib.as_array(ptr, shape=(n,))
    return arr.view(dtype).reshape(shape)


# ---- scalar-level entry points (unit pins) -------------------------------------------------

def philox(ctr, key):
    c = (C.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (C.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    o = (C.c_uint32 * 4)()
    lib().orc_philox(c, k, o)
    return [int(v) for v in o]


def uniform_int(word, m):
    return int(lib().orc_uniform_int(word, m))


def uniform_float(word):
    return float(lib().orc_uniform_float(word))


def normal_pair(w0, w1):
    o = (C.c_float * 2)()
    lib().orc_normal_pair(w0, w1, o)
    return float(o[0]), float(o[1])


def exponent(rho, M, bits):
    return int(lib().orc_exponent(float(rho), float(M), bits))


def enc_q(x, e, u16):
    return int(lib().orc_enc_q(float(x), e, u16))


def code(q, bits):
    return int(lib().orc_code(q, bits))


def dec(y, c, e, bits):
    return float(lib().orc_dec(float(y), c, e, bits))


def round_bf16(v):
    return float(lib().orc_round_bf16(float(v)))


def sr_uniforms(seed, owner, w, k0, count):
    out = np.zeros(count, dtype=np.uint16)
    lib().orc_sr_uniforms(seed, owner, w, k0, count, out.ctypes.data_as(C.POINTER(C.c_uint16)))
    return out


def pack_block(codes, bits):
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.zeros(1024 * bits // 8, dtype=np.uint8)
    lib().orc_pack_block(codes.ctypes.data_as(C.POINTER(C.c_uint8)), len(codes), bits,
                         out.ctypes.data_as(C.POINTER(C.c_uint8)))
    return out


def unpack_block(packed, count, bits):
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    out = np.zeros(count, dtype=np.uint8)
    lib().orc_unpack_block(packed.ctypes.data_as(C.POINTER(C.c_uint8)), count, bits,
                           out.ctypes.data_as(C.POINTER(C.c_uint8)))
    return out


# ---- swarm state ---------------------------------------------------------------------------

TOPOLOGY = {"complete": 0, "ring": 1, "regular": 2}
BLOCKING, NONBLOCKING, REGISTERS = 0, 1, 2


class OracleSwarm:
    """n node models of dimension d on a graph; every array attribute is a live numpy
    view of the oracle's own storage (writes go straight into the oracle)."""

    def __init__(self, n, d, topology="complete", degree=0, seed=0):
        self.n, self.d, self.seed = n, d, seed
        kind = TOPOLOGY[topology] if isinstance(topology, str) else int(topology)
        self._h = lib().orc_create(n, d, kind, degree, seed)
        if not self._h:
            raise ValueError("oracle: invalid n/d/topology")
        self.nblk = int(lib().orc_nblk(self._h))
        self.degree = int(lib().orc_degree(self._h))
        self.cfg = OracleConfig(0, 0, 0.1, 0.0, 0.0, 0.0, 0, 0, 0, 0, 0.0)

    def close(self):
        if self._h:
            lib().orc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def configure(self, **kw):
        for k, v in kw.items():
            if not hasattr(self.cfg, k):
                raise KeyError(k)
            setattr(self.cfg, k, v)
        rc = lib().orc_configure(self._h, C.byref(self.cfg))
        if rc != 0:
            raise ValueError(f"oracle configure rc={rc}")

    # live views
    @property
    def adj(self):
        return _view(lib().orc_adj(self._h), (self.n, self.degree), np.int32)

    @property
    def X(self):
        return _view(lib().orc_X(self._h), (self.n, self.d), np.float32)

    @property
    def B(self):
        return _view(lib().orc_B(self._h), (self.n, self.d), np.float32)

    @property
    def codes(self):
        return _view(lib().orc_codes(self._h), (self.n, self.nblk * 1024), np.uint8)

    @property
    def exps(self):
        return _view(lib().orc_exps(self._h), (self.n, self.nblk), np.int8)

    @property
    def pbits(self):
        return _view(lib().orc_pbits(self._h), (self.n,), np.int32)

    @property
    def w(self):
        return _view(lib().orc_w(self._h), (self.n,), np.uint32)

    @property
    def ls(self):
        return _view(lib().orc_ls(self._h), (self.n,), np.uint32)

    @property
    def launch(self):
        return _view(lib().orc_launch(self._h), (1,), np.uint32)

    @property
    def b_stale(self):
        return _view(lib().orc_b_stale(self._h), (1,), np.int32)

    @property
    def own_bytes(self):
        """Own registers as stored: per node and block 1024 low bytes, then 1024 high bytes (live view)."""
        return _view(lib().orc_own(self._h), (self.n, self.nblk * 2048), np.uint8)

    @property
    def own(self):
        """16-bit colours per coordinate, assembled from the two byte planes (a copy)."""
        raw = self.own_bytes
        if raw is None:
            return None
        planes = raw.reshape(self.n, self.nblk, 2, 1024).astype(np.uint16)
        return (planes[:, :, 0, :] | (planes[:, :, 1, :] << 8)).reshape(self.n, self.nblk * 1024)[:, : self.d]

    def set_own_prefix(self, bits):
        return int(lib().orc_set_own_prefix(self._h, bits))

    @property
    def own_prefix(self):
        return int(lib().orc_get_own_prefix(self._h))

    @property
    def oexps(self):
        return _view(lib().orc_oexps(self._h), (self.n, self.nblk), np.int8)

    @property
    def wo(self):
        return _view(lib().orc_wo(self._h), (self.n,), np.uint32)

    @property
    def tau(self):
        return _view(lib().orc_tau(self._h), (self.n,), np.uint32)

    @property
    def p_mode(self):
        return _view(lib().orc_p_mode(self._h), (1,), np.int32)

    @property
    def groups(self):
        return int(lib().orc_groups(self._h))

    @property
    def A(self):
        g = self.groups
        return _view(lib().orc_A(self._h), (g, self.cfg.lsq_m, self.d), np.float32) if g else None

    @property
    def bvec(self):
        return _view(lib().orc_bvec(self._h), (self.n, self.cfg.lsq_m), np.float32) if self.groups else None

    @property
    def xstar(self):
        return _view(lib().orc_xstar(self._h), (self.d,), np.float32) if self.groups else None

    @property
    def offset(self):
        return _view(lib().orc_offset(self._h), (self.n,), np.float32)

    @property
    def drift(self):
        return _view(lib().orc_drift(self._h), (self.n,), np.float32)

    @property
    def shift(self):
        return _view(lib().orc_shift(self._h), (self.n,), np.float32)

    def packed_codes(self, node, bits):
        """The bytes of node's communication buffer that are meaningful at `bits`."""
        return self.codes[node, : self.nblk * 1024 * bits // 8]

    # operations
    def minibatch_rows(self, node, event):
        rows = np.zeros(self.cfg.lsq_batch, dtype=np.int32)
        rc = lib().orc_minibatch_rows(self._h, node, event, rows.ctypes.data_as(C.POINTER(C.c_int32)))
        if rc != 0:
            raise ValueError(rc)
        return rows

    def sample_pairs(self, max_pairs):
        out = np.zeros((max_pairs, 2), dtype=np.int32)
        cnt = C.c_int32(0)
        rc = lib().orc_sample_pairs(self._h, max_pairs, out.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(cnt))
        if rc != 0:
            raise ValueError(rc)
        return out[: cnt.value].copy()

    def local_steps(self, nodes, H, lr):
        nodes = np.ascontiguousarray(nodes, dtype=np.int32)
        return int(lib().orc_local_steps(self._h, nodes.ctypes.data_as(C.POINTER(C.c_int32)), len(nodes), H, lr))

    def local_step_on_rows(self, node, rows, lr):
        """One least-squares step of `node` on the listed rows of its data matrix (its counter advances by one)."""
        rows = np.ascontiguousarray(rows, dtype=np.int32)
        return int(lib().orc_local_step_on_rows(self._h, node, rows.ctypes.data_as(C.POINTER(C.c_int32)), len(rows), lr))

    def local_steps_geometric(self, nodes, mean_h, lr):
        """Returns (rc, steps taken per listed node)."""
        nodes = np.ascontiguousarray(nodes, dtype=np.int32)
        steps = np.zeros(len(nodes), dtype=np.int32)
        rc = int(lib().orc_local_steps_geometric(self._h, nodes.ctypes.data_as(C.POINTER(C.c_int32)), len(nodes), mean_h,
                                                 lr, steps.ctypes.data_as(C.POINTER(C.c_int32))))
        return rc, steps

    def interact(self, pairs, bits, mode=BLOCKING, threads=1):
        pairs = np.ascontiguousarray(pairs, dtype=np.int32).reshape(-1, 2)
        return int(lib().orc_interact(self._h, pairs.ctypes.data_as(C.POINTER(C.c_int32)), len(pairs), bits, mode,
                                      threads))

    def interact_prefixed(self, pairs, prefixes, bits, threads=1):
        """Two-register interactions in which the initiator of pairs[p] reads prefixes[p] (8 or 16) bits of its
        responder's own register."""
        pairs = np.ascontiguousarray(pairs, dtype=np.int32).reshape(-1, 2)
        prefixes = np.ascontiguousarray(prefixes, dtype=np.int32)
        if len(prefixes) != len(pairs):
            raise ValueError("one prefix per pair")
        return int(lib().orc_interact_prefixed(self._h, pairs.ctypes.data_as(C.POINTER(C.c_int32)),
                                               prefixes.ctypes.data_as(C.POINTER(C.c_int32)), len(pairs), bits,
                                               REGISTERS, threads))

    def publish(self, bits):
        return int(lib().orc_publish(self._h, bits))

    def register_publish(self, bits):
        return int(lib().orc_register_publish(self._h, bits))

    def mean_model(self):
        out = np.zeros(self.d, dtype=np.float32)
        lib().orc_mean_model(self._h, out.ctypes.data_as(C.POINTER(C.c_float)))
        return out

    def potential(self):
        return float(lib().orc_potential(self._h))

    def track_staleness(self, enable=True):
        return int(lib().orc_track_staleness(self._h, 1 if enable else 0))

    @property
    def mu_hist(self):
        return _view(lib().orc_mu_hist(self._h), (self.n, self.d), np.float32)

    @property
    def a_hist(self):
        return _view(lib().orc_a_hist(self._h), (self.n,), np.float64)

    def aux_potentials(self):
        """(Gamma-hat, A_t, B_t) of the staleness analysis; tracking must be on."""
        out = (C.c_double * 3)()
        rc = int(lib().orc_aux_potentials(self._h, out))
        if rc != 0:
            raise ValueError(rc)
        return float(out[0]), float(out[1]), float(out[2])
