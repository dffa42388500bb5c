"""Benchmark of the pairwise gossip interaction path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one launch of the hot path over one batch of disjoint pairs: (local steps, if the
workload has them) -> fused quantize / exchange / average over all pairs of the launch. The metric is
gossip interactions per second (pairs processed / time); the roofline object reports the fused
interaction kernel against the measured HBM copy bandwidth. With N > 1 every rank runs an independent
replica of the workload on its own GPU (the method is single-GPU: no data-path collective).
Averaging-only workloads add a "sustained" object at N = 1: the same launches kept up for about two seconds (long
enough for the board to settle at its power limit), beside a plain device copy kept up for as long.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "gossip interactions/sec and fused-interaction HBM GB/s (% of B200 peak) at 1 GPU"
UNIT = "interactions/s"

# Synthetic workloads shaped like the paper's (flat model vectors, 8..256 nodes, 2..8-bit codes).
WORKLOADS = {
    # n = 64 nodes, d = 2^20, ring, 32 disjoint pairs per launch, 4-bit codes, averaging only.
    "ring64_d1m_b4": dict(n=64, d=1 << 20, topology="ring", degree=0, pairs=32, bits=4, mode=0, H=0, lr=0.0, seed=2,
                          cfg=dict(offset_std=float(np.sqrt(0.1)))),
    # the same store with the launches drawn by the library's pair sampler (Algorithm 1's draw with rejection of
    # pairs that touch a node already paired in the launch: 27-28 of the 32 possible pairs on average)
    "ring64_d1m_b4_sampled": dict(n=64, d=1 << 20, topology="ring", degree=0, pairs=32, bits=4, mode=0, H=0, lr=0.0, seed=2,
                                  sampler=True, cfg=dict(offset_std=float(np.sqrt(0.1)))),
    # the same with code widths that do not divide a byte (codes regrouped into aligned words by warp shuffles)
    "ring64_d1m_b3": dict(n=64, d=1 << 20, topology="ring", degree=0, pairs=32, bits=3, mode=0, H=0, lr=0.0, seed=2,
                          cfg=dict(offset_std=float(np.sqrt(0.1)))),
    "ring64_d1m_b7": dict(n=64, d=1 << 20, topology="ring", degree=0, pairs=32, bits=7, mode=0, H=0, lr=0.0, seed=2,
                          cfg=dict(offset_std=float(np.sqrt(0.1)))),
    # identity quantizer (Corollary 2): plain averaging, 16 bytes per coordinate pair
    "ring64_d1m_identity": dict(n=64, d=1 << 20, topology="ring", degree=0, pairs=32, bits=32, mode=0, H=0, lr=0.0,
                                seed=2, cfg=dict(offset_std=float(np.sqrt(0.1)))),
    # n = 16 nodes, d = 25,557,032 (ResNet-50 sized), complete graph, 8 pairs, synthetic-gradient steps.
    "complete16_resnet50_b8": dict(n=16, d=25_557_032, topology="complete", degree=0, pairs=8, bits=8, mode=0, H=2,
                                   lr=0.05, seed=4, cfg=dict(objective=1, grad_std=float(np.sqrt(1e-3)),
                                                             drift_std=float(np.sqrt(0.05)))),
    "complete16_resnet50_b4": dict(n=16, d=25_557_032, topology="complete", degree=0, pairs=8, bits=4, mode=0, H=2,
                                   lr=0.05, seed=4, cfg=dict(objective=1, grad_std=float(np.sqrt(1e-3)),
                                                             drift_std=float(np.sqrt(0.05)))),
    # reduced copy of the workload above (4 nodes, 2 pairs) for profiler captures that must stay small
    "complete4_resnet50_b8": dict(n=4, d=25_557_032, topology="complete", degree=0, pairs=2, bits=8, mode=0, H=2,
                                  lr=0.05, seed=4, cfg=dict(objective=1, grad_std=float(np.sqrt(1e-3)),
                                                            drift_std=float(np.sqrt(0.05)))),
    # n = 32 nodes, d = 11,689,512 (ResNet-18 sized), random 4-regular graph, non-blocking, 8-bit.
    "regular32_resnet18_b8_nb": dict(n=32, d=11_689_512, topology="regular", degree=4, pairs=16, bits=8, mode=1, H=3,
                                     lr=0.05, seed=3, cfg=dict(objective=1, nonblocking=1,
                                                               grad_std=float(np.sqrt(1e-3)))),
    # the same workload through the two-register protocol (Algorithm 1's chain of three decodes)
    "regular32_resnet18_b8_reg": dict(n=32, d=11_689_512, topology="regular", degree=4, pairs=16, bits=8, mode=2, H=3,
                                      lr=0.05, seed=3, cfg=dict(objective=1, nonblocking=2,
                                                                grad_std=float(np.sqrt(1e-3)))),
    "regular8_resnet18_b8_reg": dict(n=8, d=11_689_512, topology="regular", degree=4, pairs=4, bits=8, mode=2, H=3,
                                     lr=0.05, seed=3, cfg=dict(objective=1, nonblocking=2,
                                                               grad_std=float(np.sqrt(1e-3)))),
    # ring of 64 nodes through the two-register protocol: every reader consumes all 16 bits of its partner's own
    # register (the default), or only the 8-bit prefix (ring neighbours keep meeting, so their snapshots stay within
    # the 8-bit window of each other's own registers): bytes moved per interaction 22 d + 2 d bits/8 against 21 d + ...
    "ring64_d1m_b8_reg": dict(n=64, d=1 << 20, topology="ring", degree=0, pairs=32, bits=8, mode=2, H=2, lr=0.05, seed=2,
                              cfg=dict(objective=1, nonblocking=2, grad_std=float(np.sqrt(1e-3)))),
    "ring64_d1m_b8_reg_p8": dict(n=64, d=1 << 20, topology="ring", degree=0, pairs=32, bits=8, mode=2, H=2, lr=0.05,
                                 seed=2, prefix=8, cfg=dict(objective=1, nonblocking=2, grad_std=float(np.sqrt(1e-3)))),
    # reduced copy (8 nodes, 4 pairs) for profiler captures that must stay small
    "regular8_resnet18_b8_nb": dict(n=8, d=11_689_512, topology="regular", degree=4, pairs=4, bits=8, mode=1, H=3,
                                    lr=0.05, seed=3, cfg=dict(objective=1, nonblocking=1,
                                                              grad_std=float(np.sqrt(1e-3)))),
    # n = 256 nodes, d = 2^20, least squares on bf16 data (512 x 2^20 per data group, 16 groups of 16 nodes),
    # random 8-regular graph, 128 pairs per launch, 2-bit codes, non-blocking, H = 4 steps of batch 64.
    # every node takes its H steps in every launch (all nodes compute between interactions), which keeps the
    # step counters of a data group equal so that its 16 nodes share minibatches and are batched.
    "regular256_d1m_b2_lsq_nb": dict(n=256, d=1 << 20, topology="regular", degree=8, pairs=128, bits=2, mode=1, H=4,
                                     lr=0.05, seed=5, step_all=True,
                                     cfg=dict(objective=2, nonblocking=1, lsq_m=512, lsq_batch=64, lsq_dtype=1,
                                              lsq_groups=16, lsq_noise_std=float(np.sqrt(0.1)))),
    # reduced copy (2 data groups) for profiler captures that must stay small
    "regular32_d1m_b2_lsq_nb": dict(n=32, d=1 << 20, topology="regular", degree=8, pairs=16, bits=2, mode=1, H=4,
                                    lr=0.05, seed=5, step_all=True,
                                    cfg=dict(objective=2, nonblocking=1, lsq_m=512, lsq_batch=64, lsq_dtype=1,
                                             lsq_groups=2, lsq_noise_std=float(np.sqrt(0.1)))),
    # small case the CPU checker finishes in seconds
    "complete8_d4096_b8_lsq": dict(n=8, d=4096, topology="complete", degree=0, pairs=1, bits=8, mode=0, H=2, lr=0.05,
                                   seed=0, sequence=True, cfg=dict(objective=2, lsq_m=64, lsq_batch=16, lsq_dtype=0, lsq_groups=0,
                                                    lsq_noise_std=float(np.sqrt(0.1)))),
}
DEFAULT_WORKLOAD = "ring64_d1m_b4"


def stepping_nodes(wl, pairs):
    """Nodes that take local steps before this launch's interactions."""
    if wl.get("step_all"):
        return np.arange(wl["n"], dtype=np.int32)
    return pairs.reshape(-1)


def interaction_bytes(d, bits, mode, prefix=16):
    """Algorithmic bytes one interaction must move: blocking reads two models, writes two models and
    two packed buffers; non-blocking reads model + snapshot + two buffers and writes the same."""
    nblk = (d + 1023) // 1024
    if mode == 0 and bits == 32:
        return d * 16
    if mode == 0:
        return d * 16 + 2 * d * bits // 8 + 2 * nblk
    if mode == 1:
        return d * 16 + 4 * d * bits // 8 + 4 * nblk
    # two registers: model + snapshot read and written; own registers: the 8-bit prefix of the initiator's,
    # `prefix` bits of the responder's read, the initiator's 16 bits written; two current registers read and written
    return d * 16 + d * (3 + prefix // 8) + 4 * d * bits // 8 + 7 * nblk


class PairSchedule:
    """Deterministic full matchings for the launch shapes of the workloads (host-side list making
    only; the library validates disjointness and adjacency). With `sampler` (an object with sample_pairs(P): the
    CUDA context or the oracle) the launches are the method's own draws instead."""

    def __init__(self, wl, adj, sampler=None):
        self.wl, self.adj, self.rng = wl, adj, np.random.default_rng(wl["seed"])
        self.step = 0
        self.sampler = sampler if wl.get("sampler") else None

    def next(self):
        wl, n, P = self.wl, self.wl["n"], self.wl["pairs"]
        if self.sampler is not None:
            self.step += 1
            return np.ascontiguousarray(self.sampler.sample_pairs(P), dtype=np.int32)
        if wl["topology"] == "ring":
            parity = self.step & 1
            flips = self.rng.integers(0, 2, P)
            pairs = []
            for t in range(P):
                a, b = (2 * t + parity) % n, (2 * t + 1 + parity) % n
                pairs.append((b, a) if flips[t] else (a, b))
        elif wl["topology"] == "complete":
            perm = self.rng.permutation(n)
            pairs = [(int(perm[2 * t]), int(perm[2 * t + 1])) for t in range(P)]
        else:   # greedy random matching on the graph
            used, pairs = set(), []
            for a in self.rng.permutation(n):
                if int(a) in used:
                    continue
                free = [int(b) for b in self.adj[a] if int(b) not in used]
                if not free:
                    continue
                b = free[int(self.rng.integers(len(free)))]
                used.update((int(a), b))
                pairs.append((int(a), b))
                if len(pairs) == P:
                    break
        self.step += 1
        return np.array(pairs, dtype=np.int32)


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self.power = []
        self._halt = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {
            nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
            nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonHwPowerBrakeSlowdown: "hw_power_brake",
        }
        while not self._halt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.005)

    def stop(self):
        self._halt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        watts = float(np.median(self.power)) if self.power else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w": watts}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def aggregate_over_ranks(ms_local, pairs_local, dist=None, device="cpu"):
    """Whole-job figure for independent replicas: time = max over ranks, work = sum over ranks.
    Returns (ms_max, pairs_total). `dist` is an initialised torch.distributed module or None."""
    if dist is None:
        return ms_local, pairs_local
    import torch
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    p = torch.tensor([pairs_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(p, op=dist.ReduceOp.SUM)
    return float(t.item()), float(p.item())


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# ---------------------------------------------------------------------------------------------------
# CPU checker timing (reported baseline; also the whole of --impl reference)
# ---------------------------------------------------------------------------------------------------
def oracle_sample(wl, max_pairs):
    """A bounded sample of the workload for the CPU checker: the same d, objective and code width, but only
    as many nodes as the sampled pairs need (complete graph among them, one data matrix), because the
    checker's cost per interaction does not depend on n while its set-up (Philox normals in double) does."""
    p = max(1, min(wl["pairs"], max_pairs))
    if wl["n"] * wl["d"] <= (1 << 27):
        return dict(wl), wl["pairs"]
    small = dict(wl, n=2 * p, topology="complete", degree=0, pairs=p)
    cfg = dict(wl["cfg"])
    if cfg.get("lsq_groups", 0) > 0:
        cfg["lsq_groups"] = 1
    small["cfg"] = cfg
    return small, p


def time_oracle(wl, budget_s, max_launches, threads=None):
    from oracle import swarm_oracle as o
    cores = len(os.sched_getaffinity(0))
    wl, P = oracle_sample(wl, cores if threads is None else threads)
    T = min(P, cores) if threads is None else threads
    orc = o.OracleSwarm(wl["n"], wl["d"], wl["topology"], wl["degree"], wl["seed"])
    if wl["cfg"]:
        orc.configure(**wl["cfg"])
    sched = PairSchedule(wl, orc.adj, orc)
    done, t_total, launches = 0, 0.0, 0
    while launches < max_launches and (t_total < budget_s or launches == 0):
        pairs = sched.next()[:P]
        t0 = time.perf_counter()
        if wl["H"] > 0:
            orc.local_steps(stepping_nodes(wl, pairs), wl["H"], wl["lr"])
        rc = orc.interact(pairs, wl["bits"], wl["mode"], threads=T)
        t_total += time.perf_counter() - t0
        assert rc == 0
        done += len(pairs)
        launches += 1
    return done / t_total, T, launches, t_total, wl


def run_reference(args, wl, name):
    """Times the CPU checker as it stands. Every step is a bounded sample of one launch: the first
    p pairs of the launch's pair list at full d, p chosen from a calibration interaction so that K
    steps end within a few minutes."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    K, W = args.steps, args.warmup
    from oracle import swarm_oracle as o
    cores = len(os.sched_getaffinity(0))
    orc = o.OracleSwarm(wl["n"], wl["d"], wl["topology"], wl["degree"], wl["seed"])
    if wl["cfg"]:
        orc.configure(**wl["cfg"])
    sched = PairSchedule(wl, orc.adj, orc)

    def step(p, T):
        pairs = sched.next()[:p]
        if wl["H"] > 0:
            orc.local_steps(stepping_nodes(wl, pairs), wl["H"], wl["lr"])
        assert orc.interact(pairs, wl["bits"], wl["mode"], threads=T) == 0
        return len(pairs)
    t0 = time.perf_counter()
    step(1, 1)                                     # calibration (also the first warm-up step)
    t1 = time.perf_counter() - t0
    budget = 150.0
    p = int(max(1, min(wl["pairs"], cores, budget / (K * t1))))
    T = p
    for _ in range(min(W, 3) - 1):
        step(p, T)
    t0 = time.perf_counter()
    done = sum(step(p, T) for _ in range(K))
    dt = time.perf_counter() - t0
    value = done / dt
    sample = (f"each step = the first {p} of the launch's {wl['pairs']} pairs at full d on {T} host threads "
              f"(std::thread over disjoint pairs); {K} steps")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K,
        "warmup": min(W, 3), "ms_per_step": 1e3 * dt / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": name, **{k: wl[k] for k in ("n", "d", "topology", "pairs", "bits", "mode", "H")}},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": T, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---------------------------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------------------------
KERNEL_SOURCES = ("swarm_interact.cu", "swarm_blocks.cuh", "swarm_dev.cuh", "swarm_internal.h")
# the five workloads of the measurement table: small least squares, ring averaging, ResNet-18-sized non-blocking,
# ResNet-50-sized blocking at two code widths, 256 nodes with tensor-core least squares
TABLE_WORKLOADS = ("complete8_d4096_b8_lsq", "ring64_d1m_b4", "regular32_resnet18_b8_nb", "complete16_resnet50_b4",
                   "complete16_resnet50_b8", "regular256_d1m_b2_lsq_nb")


def kernel_source_hash():
    """sha256 over the sources that define the interaction kernels: profiler counters recorded under profiles/
    carry the hash of the sources they were captured from and are dropped once it no longer matches."""
    import hashlib
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_1910_12308_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def profiler_counters(name):
    """Counters of the dominant kernel of workload `name` from profiles/kernel_counters.json ({} when there is no
    capture of the kernels as they are now)."""
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "kernel_counters.json")))[name]
    except Exception:
        return {}
    return rec if rec.get("source_sha256_16") == kernel_source_hash() else {}


def traffic_of(name, pairs_per_launch):
    """ncu dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, or None."""
    rec = profiler_counters(name)
    if "dram_bytes_per_launch" in rec:
        return rec["dram_bytes_per_launch"]
    if "dram_bytes_per_pair" in rec:       # launches whose number of pairs varies: every pair streams its own rows once
        return rec["dram_bytes_per_pair"] * pairs_per_launch
    return None


def kernel_name(wl, fused=False):
    base = ("interact_identity_kernel" if wl["bits"] == 32 else
            ["interact_blocking_kernel", "interact_nonblocking_kernel", "interact_registers_kernel"][wl["mode"]])
    return base + (" (local steps fused)" if fused else "")


class Runner:
    """One workload on the current device: context, pair schedule and the timed loop over the C ABI."""

    def __init__(self, g, torch, wl, name, seed_shift, stream, args):
        self.g, self.torch, self.wl, self.name, self.stream = g, torch, wl, name, stream
        self.sw = g.Swarm(wl["n"], wl["d"], wl["topology"], wl["degree"], wl["seed"] + seed_shift, stream=stream)
        if wl["cfg"]:
            self.sw.configure(**wl["cfg"])
        self.sched = PairSchedule(wl, self.sw.get_all(g.T_ADJ), self.sw)
        # elementwise (synthetic) objective: the nodes of the pairs step inside the interaction kernel (swarm_step),
        # unless two calls per step are asked for
        self.fused = bool(wl["H"] > 0 and wl["cfg"].get("objective") == 1 and not wl.get("step_all")
                          and wl["mode"] != 2 and not args.unfused)
        # sequential gossip on short models: the whole timed region is one swarm_run_sequence call
        self.sequence = bool(wl.get("sequence")) and wl["pairs"] == 1 and wl["mode"] == 0 and not args.stepwise

    def step(self, pairs):
        """One step through the public binding (what a user calls)."""
        sw, wl = self.sw, self.wl
        if self.fused:
            rc = sw.step(pairs, wl["H"], wl["lr"], wl["bits"], wl["mode"], True)
            assert rc == 0, rc
            return
        if wl["H"] > 0:
            rc = sw.local_steps(stepping_nodes(wl, pairs), wl["H"], wl["lr"])
            assert rc == 0, rc
        if wl.get("prefix"):
            rc = sw.interact_prefixed(pairs, np.full(len(pairs), wl["prefix"], dtype=np.int32), wl["bits"])
        else:
            rc = sw.interact(pairs, wl["bits"], wl["mode"])
        assert rc == 0, rc

    def timed(self, launches, barrier, probe_every=8):
        """Times len(launches) steps with CUDA events on the context's stream, models resident in HBM. Arguments
        are marshalled before the timed region; the loop only crosses the C ABI. Returns (ms for all steps,
        average ms of the interaction kernel, kernels launched)."""
        import ctypes as C
        g, torch, wl, sw, stream = self.g, self.torch, self.wl, self.sw, self.stream
        L, h = sw._L, sw._h
        H, lr, bits, mode = wl["H"], wl["lr"], wl["bits"], wl["mode"]
        K = len(launches)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ok, ev_mid = 0, []
        l0 = sw.kernel_launches()
        if self.sequence:
            seq = np.ascontiguousarray(np.concatenate(launches), dtype=np.int32)
            ptr = seq.ctypes.data_as(C.POINTER(g.SwarmPair))
            ev0.record(stream)
            ok |= L.swarm_run_sequence(h, ptr, len(seq), H, lr, bits, 1)
            ev1.record(stream)
        else:
            prefixes = np.full(wl["n"], wl.get("prefix", 16), dtype=np.int32)
            pf_ptr = prefixes.ctypes.data_as(C.POINTER(C.c_int32))

            def interact(pp, npp):
                if wl.get("prefix"):
                    return L.swarm_interact_prefixed(h, pp, pf_ptr, npp, bits)
                return L.swarm_interact(h, pp, npp, bits, mode)
            calls = []
            for pairs in launches:
                pa = np.ascontiguousarray(pairs, dtype=np.int32)
                na = np.ascontiguousarray(stepping_nodes(wl, pairs), dtype=np.int32)
                calls.append((pa, pa.ctypes.data_as(C.POINTER(g.SwarmPair)), len(pa), na,
                              na.ctypes.data_as(C.POINTER(C.c_int32)), len(na)))
            self.calls = calls
            probes = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                      for _ in range(0, K, probe_every)] if (H > 0 and not self.fused) else []
            ev0.record(stream)
            for i, (_, pp, npp, _, nn, ncount) in enumerate(calls):
                if self.fused:
                    ok |= L.swarm_step(h, pp, npp, H, lr, bits, mode, 1)
                elif H > 0:
                    ok |= L.swarm_local_steps(h, nn, ncount, H, lr)
                    if i % probe_every == 0:       # the interaction kernel is bracketed by events on every 8th step
                        e_a, e_b = probes[i // probe_every]
                        e_a.record(stream)
                        ok |= interact(pp, npp)
                        e_b.record(stream)
                        ev_mid.append((e_a, e_b))
                    else:
                        ok |= interact(pp, npp)
                else:
                    ok |= interact(pp, npp)
            ev1.record(stream)
        barrier()
        assert ok == 0, "a call in the timed region failed"
        ms = ev0.elapsed_time(ev1)
        if ev_mid:
            kern_ms = sum(a.elapsed_time(b) for a, b in ev_mid) / len(ev_mid)
            kern_pairs = float(np.mean([len(launches[i]) for i in range(0, K, probe_every)]))
        else:
            kern_ms, kern_pairs = ms / K, float(np.mean([len(p) for p in launches]))
        return ms, kern_ms, kern_pairs, sw.kernel_launches() - l0

    def kernel_bytes(self, pairs_per_launch):
        """Algorithmic bytes one launch of the interaction kernel moves."""
        wl = self.wl
        b = interaction_bytes(wl["d"], wl["bits"], wl["mode"], wl.get("prefix", 16)) * pairs_per_launch
        if self.fused and wl["mode"] != 0:
            b += 8 * wl["d"] * pairs_per_launch             # the responder's model is read and written too
        return b

    def end_to_end(self, launches, seconds, barrier):
        """The same steps through the public binding with host buffers inside the timed region: every step's pair
        list comes from pinned host memory, a result of every step (the block exponents that the first initiator
        published) is read back to pinned host memory, and the potential is read (synchronising, which also delivers
        the queued rows) every 1000 interactions, at least every 32 steps. Runs for at least `seconds` and at least
        len(launches) steps.
        Returns (pairs processed, ms, host-to-device bytes per step, device-to-host bytes per step)."""
        g, torch, wl, sw, stream = self.g, self.torch, self.wl, self.sw, self.stream
        nblk = (wl["d"] + 1023) // 1024
        pinned = [torch.from_numpy(np.ascontiguousarray(p, dtype=np.int32).copy()).pin_memory() for p in launches]
        chunk = 64 if self.sequence else 1        # sequential gossip: 64 time steps per call (one kernel launch)
        if self.sequence:
            flat = torch.from_numpy(np.ascontiguousarray(np.concatenate(launches), dtype=np.int32).copy()).pin_memory()
            nchunks_have = max(1, len(flat) // chunk)
        ring = torch.empty((32, nblk), dtype=torch.int8).pin_memory()     # results of the last 32 steps
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def one(i):
            if self.sequence:
                c0 = (i % nchunks_have) * chunk
                pairs = flat[c0:c0 + chunk].numpy()
                rc = sw.run_sequence(pairs, wl["H"], wl["lr"], wl["bits"], True)
                assert rc == 0, rc
                first = int(pairs[-1, 0])
                done = len(pairs)
            else:
                pairs = pinned[i % len(pinned)].numpy()
                self.step(pairs)
                first = int(pairs[0, 0])
                done = len(pairs)
            rc = sw.get_async(g.T_EXPS, first, ring[i % 32])
            assert rc == 0, rc
            return done, pairs.nbytes

        # warm the path: first launch of the row-read kernel, first queued read, first potential
        one(0)
        sw.potential()
        barrier()
        t0 = time.perf_counter()
        for i in range(32):
            one(1 + i)
        sw.sync()
        per_step = max((time.perf_counter() - t0) / 32, 1e-7)
        steps = max(-(-len(launches) // chunk), int(seconds / per_step) + 1)
        steps = min((steps + 31) // 32 * 32, 200000)          # whole groups of 32: the last potential read ends the run
        barrier()
        done = h2d = d2h = checksum = since = reads = 0
        t0 = time.perf_counter()
        ev0.record(stream)
        for i in range(steps):
            dn, nb = one(i + 33)
            done += dn
            since += dn
            h2d += nb
            d2h += nblk
            if since >= 1000 or i % 32 == 31:
                sw.potential()
                since = 0
                reads += 1
                d2h += 8
                checksum += int(ring.sum())
        ev1.record(stream)
        self.potential_reads_per_step = reads / steps
        barrier()
        ms = max(ev0.elapsed_time(ev1), (time.perf_counter() - t0) * 1e3)
        return done, ms, h2d / steps, d2h / steps, steps

    def close(self):
        self.sw.close()


def table_entry(g, torch, wl, name, args, stream, peak, local_rank):
    """A short run (at least 0.25 s of timed steps) of one workload: interactions/s of the whole step, the
    interaction kernel's time, its algorithmic GB/s and fraction of the measured copy bandwidth, clocks. Workloads
    whose local steps can run inside the interaction kernel are run both ways: the whole-step rate is the one-call
    form's (swarm_step), the interaction kernel's own figures come from the two-call form."""
    if (wl["H"] > 0 and wl["cfg"].get("objective") == 1 and not wl.get("step_all") and wl["mode"] != 2
            and not args.unfused):
        two_calls = argparse.Namespace(**dict(vars(args), unfused=True))
        entry = table_entry_one(g, torch, wl, name, two_calls, stream, peak, local_rank)
        one_call = table_entry_one(g, torch, wl, name, args, stream, peak, local_rank)
        entry["two_calls_per_step"] = {k: entry[k] for k in ("interactions_per_s", "ms_per_step", "gpu_launches", "steps")}
        for k in ("interactions_per_s", "ms_per_step", "gpu_launches", "steps", "seconds", "clocks"):
            entry[k] = one_call[k]
        entry["step_kernel"] = one_call["kernel"]
        entry["step_kernel_ms"] = one_call["interaction_kernel_ms"]
        return entry
    return table_entry_one(g, torch, wl, name, args, stream, peak, local_rank)


def table_entry_one(g, torch, wl, name, args, stream, peak, local_rank):
    r = Runner(g, torch, wl, name, 0, stream, args)

    def barrier():
        torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)             # NVML set up before the warm-up: no idle gap before the timed steps
    warm = [r.sched.next() for _ in range(5)]
    for p in warm:
        r.step(p)
    barrier()
    probe = [r.sched.next() for _ in range(8)]
    ms, _, _, _ = r.timed(probe, barrier)
    K = int(min(20000, max(16, 0.25 / max(ms / len(probe) * 1e-3, 1e-7))))
    launches = [r.sched.next() for _ in range(K)]
    sampler.start()
    ms, kern_ms, kern_pairs, nl = r.timed(launches, barrier)
    clocks = sampler.stop()
    pairs_total = sum(len(p) for p in launches)
    entry = {"interactions_per_s": pairs_total / (ms * 1e-3), "steps": K, "seconds": ms * 1e-3, "ms_per_step": ms / K,
             "pairs_per_launch": pairs_total / K, "gpu_launches": int(nl), "clocks": clocks,
             "config": {k: wl[k] for k in ("n", "d", "topology", "pairs", "bits", "mode", "H")}}
    if r.sequence:
        entry.update({"kernel": "lsq_sequence_kernel", "single_launch_sequence": True, "bound": "latency",
                      "us_per_whole_step": 1e3 * ms / K})
    else:
        gbs = r.kernel_bytes(kern_pairs) / (kern_ms * 1e-3) / 1e9
        entry.update({"kernel": kernel_name(wl, r.fused), "interaction_kernel_ms": kern_ms,
                      "interaction_only_per_s": kern_pairs / (kern_ms * 1e-3), "algorithmic_GBps": gbs,
                      "frac": gbs / peak, "frac_of_8000": gbs / 8000.0})
    r.close()
    del r
    torch.cuda.empty_cache()
    return entry


def run_ours(args, wl, name):
    import torch
    from paper_1910_12308_b200 import binding as g

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench: no CUDA device (the library has no CPU path)")
    torch.cuda.set_device(local_rank)
    use_dist = world > 1
    dist = None
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    stream = torch.cuda.current_stream()
    r = Runner(g, torch, wl, name, 1000 * rank, stream, args)
    sw, fused, sequence = r.sw, r.fused, r.sequence
    K, W = args.steps, args.warmup
    launches = [r.sched.next() for _ in range(K + W)]
    npairs_total = sum(len(p) for p in launches[W:])

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: W untimed steps, then exactly K timed steps. The clock sampler is set up (NVML
    # initialisation takes tens of milliseconds) before the warm-up, so that the device does not sit idle between the
    # warm-up and the timed region; it starts sampling when the timed region starts.
    sampler = ClockSampler(local_rank)
    for pairs in launches[:W]:
        r.step(pairs)
    barrier()
    sampler.start()
    ms_local, kern_ms, kern_pairs, gpu_launches = r.timed(launches[W:], barrier)
    clocks = sampler.stop()
    ms, pairs_all = aggregate_over_ranks(ms_local, npairs_total, dist if use_dist else None, "cuda")
    value = pairs_all / (ms * 1e-3)

    # fused interaction kernel: average launch duration inside the timed region
    per_launch_bytes = r.kernel_bytes(kern_pairs)
    achieved = per_launch_bytes / (kern_ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak()

    # ---- end to end through the public binding with host buffers (see Runner.end_to_end)
    e2e_pairs, e2e_ms, h2d, d2h, e2e_steps = r.end_to_end(launches[W:], args.e2e_seconds, barrier)
    e2e_ms, e2e_pairs_all = aggregate_over_ranks(e2e_ms, e2e_pairs, dist if use_dist else None, "cuda")
    e2e = {"value": e2e_pairs_all / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(round(h2d)),
           "d2h_bytes_per_step": int(round(d2h)), "steps": e2e_steps, "seconds": e2e_ms * 1e-3,
           "calls_per_step": ("swarm_run_sequence (64 time steps per call)" if sequence else
                              ("swarm_step" if fused else ("swarm_local_steps, swarm_interact" if wl["H"] > 0
                                                           else "swarm_interact")))
           + ", swarm_get_tensor_async; swarm_potential every 1000 interactions (%.3f reads per step)"
           % r.potential_reads_per_step}

    traffic = traffic_of(name, kern_pairs)
    roofline = {"bound": "hbm", "kernel": kernel_name(wl, fused),
                "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "what": "algorithmic bytes per launch / CUDA-event time of the launch (not DRAM traffic)",
                "peak_kind": peak_kind, "frac_of_8000": achieved / 8000.0, "traffic": traffic,
                "algorithmic_bytes_per_launch": per_launch_bytes, "kernel_ms": kern_ms}
    if traffic is not None:
        # what reached DRAM in the profiler's capture, at the launch time measured here
        roofline["dram_GBps"] = traffic / (kern_ms * 1e-3) / 1e9
        roofline["dram_frac"] = roofline["dram_GBps"] / peak
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": name, **{k: wl[k] for k in ("n", "d", "topology", "pairs", "bits", "mode", "H")},
                   "fused_local_steps": bool(fused), "single_launch_sequence": bool(sequence),
                   "l2": ("inputs larger than L2: the models a launch touches (%.0f MB) exceed the 126 MB L2, so every "
                          "launch reads them from HBM; part of the lines it rewrites is still in L2 when it ends"
                          % (2 * kern_pairs * wl["d"] * 4 / 1e6)) if wl["d"] * kern_pairs * 8 > 126e6 else
                         "L2 flushed by nothing: the working set fits in L2 (latency-bound workload, no HBM roofline)",
                   "replicas": world},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(gpu_launches), "roofline": roofline,
    }
    counters = profiler_counters(name)
    if wl["mode"] == 2 and not fused and "warp_instructions_per_block" in counters:
        # the two-register kernel is bound by instruction issue where it does not reach the HBM rate: also report it
        # against the issue rate (148 SMs x 4 schedulers x SM clock) with its warp instructions per 1024-block
        nblk = (wl["d"] + 1023) // 1024
        instr = counters["warp_instructions_per_block"] * nblk * kern_pairs
        rate = instr / (kern_ms * 1e-3) / 1e12
        issue_peak = 148 * 4 * (clocks["sm_max_mhz"] or 1965) * 1e6 / 1e12
        out["roofline"]["issue"] = {"achieved": rate, "peak": issue_peak, "unit": "T warp-instructions/s",
                                    "frac": rate / issue_peak, "warp_instructions_per_launch": instr}
    # the same launches for about two seconds: long enough for the board to settle at its power limit, which the
    # timed region above (a burst of K launches) is not; reported beside the burst figure, with the clock seen
    if not sequence and wl["H"] == 0 and not fused and rank == 0 and world == 1:
        L, h, ok = sw._L, sw._h, 0
        bits, mode = wl["bits"], wl["mode"]
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = max(1, int(2.0 / max(ms_local * 1e-3, 1e-6)))
        # An averaging-only swarm contracts: kept going for hundreds of thousands of interactions it reaches
        # consensus, where the lattice steps are set by the magnitude rule and the kernels take the defining form of
        # the lattice arithmetic (another instruction stream than the workload's). The workload is 10^4 interactions
        # from the initial state, so the models are put back to that state every 10^4 interactions (one
        # device-to-device copy on the same stream, inside the timed loop and counted in its time).
        sw.configure(**wl["cfg"])
        xt = sw.model_tensor()
        x_init = xt.clone()
        restore_every = max(1, int(round(1e4 / max(kern_pairs, 1))))
        barrier()
        sampler2 = ClockSampler(local_rank)
        sampler2.start()
        done_launches = 0
        ev0.record(stream)
        for _ in range(reps):
            for (_, pp, npp, _, _, _) in r.calls:
                ok |= L.swarm_interact(h, pp, npp, bits, mode)
                done_launches += 1
                if done_launches % restore_every == 0:
                    xt.copy_(x_init)
        ev1.record(stream)
        barrier()
        assert ok == 0
        clk2 = sampler2.stop()
        s_ms = ev0.elapsed_time(ev1) / (reps * K)
        s_gbs = per_launch_bytes / (s_ms * 1e-3) / 1e9
        out["sustained"] = {"launches": reps * K, "seconds": ev0.elapsed_time(ev1) * 1e-3,
                            "value": npairs_total * reps / (ev0.elapsed_time(ev1) * 1e-3), "unit": UNIT,
                            "kernel_ms": s_ms, "achieved": s_gbs, "frac": s_gbs / peak, "clocks": clk2,
                            "models_restored_every_launches": restore_every}
        del x_init
        # yardstick under the same conditions: a plain device copy (library kernel) kept up for as long
        a = torch.empty(1 << 28, dtype=torch.float32, device="cuda")
        b = torch.empty_like(a)
        for _ in range(3):
            b.copy_(a)
        barrier()
        one = 2.0 * a.numel() * 4
        creps = max(1, int(2.0 / (one / (peak * 1e9))))
        sampler3 = ClockSampler(local_rank)
        sampler3.start()
        ev0.record(stream)
        for _ in range(creps):
            b.copy_(a)
        ev1.record(stream)
        barrier()
        clk3 = sampler3.stop()
        copy_gbs = one * creps / (ev0.elapsed_time(ev1) * 1e-3) / 1e9
        out["sustained"]["copy_gbs_same_duration"] = copy_gbs
        out["sustained"]["frac_of_sustained_copy"] = s_gbs / copy_gbs
        out["sustained"]["copy_clocks"] = clk3
        del a, b

    # mean model and potential (one HBM pass over all n models each), timed on their own
    reps = 20
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    mu = torch.empty(wl["d"], dtype=torch.float32, device="cuda")
    L, h = sw._L, sw._h
    for name_k, call in (("mean_model", lambda: L.swarm_mean_model(h, mu.data_ptr())),
                         ("potential", lambda: sw.potential())):
        for _ in range(3):
            call()
        barrier()
        ev0.record(stream)
        for _ in range(reps):
            call()
        ev1.record(stream)
        barrier()
        t_ms = ev0.elapsed_time(ev1) / reps
        out.setdefault("aux_kernels", {})[name_k] = {
            "ms": t_ms, "GB/s": 4.0 * wl["n"] * wl["d"] / (t_ms * 1e-3) / 1e9, "bytes": 4 * wl["n"] * wl["d"]}
    r.close()
    del r, mu
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_table:
        # short runs of the five workloads of the measurement table, in the same process and on the same board
        table = {}
        for nm in TABLE_WORKLOADS:
            if nm == name and wl["H"] == 0 and not args.stepwise:
                table[nm] = {"interactions_per_s": value, "steps": K, "seconds": ms * 1e-3, "ms_per_step": ms / K,
                             "pairs_per_launch": npairs_total / K, "kernel": kernel_name(wl),
                             "interaction_kernel_ms": kern_ms, "algorithmic_GBps": achieved, "frac": achieved / peak,
                             "frac_of_8000": achieved / 8000.0, "clocks": clocks, "same_as": "the timed region above"}
                if sequence:
                    table[nm] = {"interactions_per_s": value, "steps": K, "seconds": ms * 1e-3, "bound": "latency",
                                 "kernel": "lsq_sequence_kernel", "us_per_whole_step": 1e3 * ms / K, "clocks": clocks,
                                 "same_as": "the timed region above"}
                continue
            table[nm] = table_entry(g, torch, WORKLOADS[nm], nm, args, stream, peak, local_rank)
        out["workloads"] = table
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, T, nl, tt, swl = time_oracle(wl, budget_s=10.0, max_launches=40)
        v1, _, nl1, tt1, _ = time_oracle(wl, budget_s=3.0, max_launches=1, threads=1)
        what = ("the workload itself" if swl["n"] == wl["n"]
                else f"a {swl['n']}-node sample of the workload (same d, objective, bits)")
        out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": T, "kind": "oracle",
                               "sample": f"{nl} launches of {swl['pairs']} pairs at full d ({tt:.1f} s) on {T} host "
                                         f"threads, {what}; local steps included where the workload has them",
                               "single_thread_value": v1}
    if use_dist:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-seconds", type=float, default=0.3,
                    help="least duration of the end-to-end loop (it always runs at least --steps steps)")
    ap.add_argument("--no-table", action="store_true",
                    help="skip the short runs of the other workloads of the measurement table (\"workloads\" object)")
    ap.add_argument("--stepwise", action="store_true",
                    help="sequential small-model workload: two calls per step instead of one swarm_run_sequence "
                         "call for the whole timed region")
    ap.add_argument("--unfused", action="store_true",
                    help="synthetic-objective workloads: swarm_local_steps + swarm_interact per step instead of one "
                         "swarm_step call (local steps inside the interaction kernel, the default: one trip of the "
                         "models through HBM instead of two)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    wl = WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl, args.workload)
    else:
        run_ours(args, wl, args.workload)


if __name__ == "__main__":
    main()
