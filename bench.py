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


def interaction_bytes(d, bits, mode):
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
    # the 16 bits of the responder's (default prefix) read, the initiator's 16 bits written; two current
    # registers read and written
    return d * 16 + d * 5 + 4 * d * bits // 8 + 7 * nblk


class PairSchedule:
    """Deterministic full matchings for the launch shapes of the workloads (host-side list making
    only; the library validates disjointness and adjacency)."""

    def __init__(self, wl, adj):
        self.wl, self.adj, self.rng = wl, adj, np.random.default_rng(wl["seed"])
        self.step = 0

    def next(self):
        wl, n, P = self.wl, self.wl["n"], self.wl["pairs"]
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
    sched = PairSchedule(wl, orc.adj)
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
    sched = PairSchedule(wl, orc.adj)

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
def run_ours(args, wl, name):
    import torch
    from paper_1910_12308_b200 import binding as g

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench: no CUDA device (the library has no CPU path)")
    torch.cuda.set_device(local_rank)
    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    stream = torch.cuda.current_stream()
    sw = g.Swarm(wl["n"], wl["d"], wl["topology"], wl["degree"], wl["seed"] + 1000 * rank, stream=stream)
    if wl["cfg"]:
        sw.configure(**wl["cfg"])
    adj = sw.get_all(g.T_ADJ)
    sched = PairSchedule(wl, adj)
    K, W = args.steps, args.warmup
    launches = [sched.next() for _ in range(K + W)]
    npairs_total = sum(len(p) for p in launches[W:])

    # elementwise (synthetic) objective, on request: the nodes of the pairs step inside the interaction kernel
    fused = (wl["H"] > 0 and wl["cfg"].get("objective") == 1 and not wl.get("step_all") and args.fused)

    # sequential gossip on short models: the whole timed region is one swarm_run_sequence call
    sequence = bool(wl.get("sequence")) and wl["pairs"] == 1 and wl["mode"] == 0 and not args.stepwise

    def step(pairs):
        if fused:
            rc = sw.step(pairs, wl["H"], wl["lr"], wl["bits"], wl["mode"], True)
            assert rc == 0, rc
            return
        if wl["H"] > 0:
            rc = sw.local_steps(stepping_nodes(wl, pairs), wl["H"], wl["lr"])
            assert rc == 0, rc
        rc = sw.interact(pairs, wl["bits"], wl["mode"])
        assert rc == 0, rc

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    # arguments are marshalled once, outside the timed region; the loop only crosses the C ABI
    import ctypes as C
    L, h = sw._L, sw._h
    calls = []
    for pairs in launches[W:]:
        pa = np.ascontiguousarray(pairs, dtype=np.int32)
        na = np.ascontiguousarray(stepping_nodes(wl, pairs), dtype=np.int32)
        calls.append((pa, pa.ctypes.data_as(C.POINTER(g.SwarmPair)), len(pa), na,
                      na.ctypes.data_as(C.POINTER(C.c_int32)), len(na)))
    H, lr, bits, mode = wl["H"], wl["lr"], wl["bits"], wl["mode"]
    probe_every = 8                       # the interaction kernel is bracketed by events on every 8th step
    probes = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(0, K, probe_every)] if (H > 0 and not fused) else []
    # ---- device-resident timing
    for pairs in launches[:W]:
        step(pairs)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    l0 = sw.kernel_launches()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev_mid = []
    ok = 0
    ev0.record(stream)
    if sequence:
        seq = np.ascontiguousarray(np.concatenate(launches[W:]), dtype=np.int32)
        ok |= L.swarm_run_sequence(h, seq.ctypes.data_as(C.POINTER(g.SwarmPair)), len(seq), H, lr, bits, 1)
        calls = []
        probes = []
    for i, (_, pp, npp, _, nn, ncount) in enumerate(calls):
        if fused:
            ok |= L.swarm_step(h, pp, npp, H, lr, bits, mode, 1)
        elif H > 0:
            ok |= L.swarm_local_steps(h, nn, ncount, H, lr)
            if i % probe_every == 0:
                e_a, e_b = probes[i // probe_every]
                e_a.record(stream)
                ok |= L.swarm_interact(h, pp, npp, bits, mode)
                e_b.record(stream)
                ev_mid.append((e_a, e_b))
            else:
                ok |= L.swarm_interact(h, pp, npp, bits, mode)
        else:
            ok |= L.swarm_interact(h, pp, npp, bits, mode)
    ev1.record(stream)
    barrier()
    assert ok == 0, "a call in the timed region failed"
    clocks = sampler.stop()
    gpu_launches = sw.kernel_launches() - l0
    ms_local = ev0.elapsed_time(ev1)
    ms, pairs_all = aggregate_over_ranks(ms_local, npairs_total, dist if use_dist else None, "cuda")
    value = pairs_all / (ms * 1e-3)

    # fused interaction kernel: average launch duration inside the timed region
    if ev_mid:
        kern_ms = sum(a.elapsed_time(b) for a, b in ev_mid) / len(ev_mid)
    else:
        kern_ms = ms_local / K
    per_launch_bytes = interaction_bytes(wl["d"], wl["bits"], wl["mode"]) * npairs_total / K
    if fused and wl["mode"] != 0:
        per_launch_bytes += 8 * wl["d"] * npairs_total / K      # the responder's model is read and written too
    achieved = per_launch_bytes / (kern_ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak()

    # ---- end to end through the C ABI with host buffers: pair lists come from pinned host memory,
    # the step's result (block exponents of the first initiator) is read back into pinned memory every step
    # (asynchronously, consumed in batches of 32), the potential every 32 steps (synchronising).
    e2e_steps = min(K, 2000)
    pinned = [torch.from_numpy(p.copy()).pin_memory() for p in launches[W:W + e2e_steps]]
    barrier()
    d2h = 0
    nblk = (wl["d"] + 1023) // 1024
    ring = torch.empty((32, nblk), dtype=torch.int8).pin_memory()     # results of the last 32 steps
    checksum = 0
    t0 = time.perf_counter()
    ev0.record(stream)
    for i, pt in enumerate(pinned):
        pairs = pt.numpy()
        step(pairs)
        # the step's result is read back every step, queued behind the step on the same stream; the host
        # consumes the last 32 results at each synchronising potential read
        rc = sw.get_async(g.T_EXPS, int(pairs[0, 0]), ring[i % 32])
        assert rc == 0, rc
        d2h += nblk
        if i % 32 == 31:
            sw.potential()
            d2h += 8
            checksum += int(ring.sum())
    ev1.record(stream)
    barrier()
    checksum += int(ring.sum())
    e2e_ms = ev0.elapsed_time(ev1)
    wall_ms = (time.perf_counter() - t0) * 1e3
    e2e_ms = max(e2e_ms, wall_ms)
    e2e_pairs = sum(len(p) for p in launches[W:W + e2e_steps])
    e2e_ms, e2e_pairs_all = aggregate_over_ranks(e2e_ms, e2e_pairs, dist if use_dist else None, "cuda")
    e2e = {"value": e2e_pairs_all / (e2e_ms * 1e-3), "unit": UNIT,
           "h2d_bytes_per_step": int(np.mean([len(p) * 16 for p in launches[W:W + e2e_steps]])),
           "d2h_bytes_per_step": int(d2h / e2e_steps)}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": name, **{k: wl[k] for k in ("n", "d", "topology", "pairs", "bits", "mode", "H")},
                   "fused_local_steps": bool(fused), "single_launch_sequence": bool(sequence),
                   "l2": "inputs larger than L2: every launch streams all models it touches from HBM",
                   "replicas": world},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(gpu_launches),
        "roofline": {"bound": "hbm", "kernel": ("interact_identity_kernel" if wl["bits"] == 32 else
                                ["interact_blocking_kernel", "interact_nonblocking_kernel", "interact_registers_kernel"][wl["mode"]])
                     + (" (local steps fused)" if fused else ""),
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": peak_kind, "frac_of_8000": achieved / 8000.0, "traffic": traffic_of(name, npairs_total / K),
                     "algorithmic_bytes_per_launch": per_launch_bytes, "kernel_ms": kern_ms},
    }
    if wl["mode"] == 2 and not fused:
        # the two-register kernel is bound by instruction issue, not by HBM: report it against the issue rate
        # (148 SMs x 4 schedulers x SM clock) with its warp instructions per 1024-block from the ncu capture
        nblk = (wl["d"] + 1023) // 1024
        instr = REGISTER_KERNEL_INSTR_PER_BLOCK * nblk * npairs_total / K
        rate = instr / (kern_ms * 1e-3) / 1e12
        issue_peak = 148 * 4 * (clocks["sm_max_mhz"] or 1965) * 1e6 / 1e12
        hbm = out["roofline"]
        out["roofline"] = {"bound": "alu", "kernel": hbm["kernel"], "achieved": rate, "peak": issue_peak,
                           "unit": "T warp-instructions/s", "frac": rate / issue_peak, "traffic": traffic_of(name, npairs_total / K),
                           "warp_instructions_per_launch": instr, "kernel_ms": kern_ms,
                           "hbm": {k: hbm[k] for k in ("achieved", "peak", "unit", "frac", "peak_kind", "frac_of_8000",
                                                       "algorithmic_bytes_per_launch")}}
    # the same launches for about two seconds: long enough for the board to settle at its power limit, which the
    # timed region above (a burst of K launches) is not; reported beside the burst figure, with the clock seen
    if calls and H == 0 and not fused and rank == 0 and world == 1:
        reps = max(1, int(2.0 / max(ms_local * 1e-3, 1e-6)))
        sampler2 = ClockSampler(local_rank)
        sampler2.start()
        ev0.record(stream)
        for _ in range(reps):
            for (_, pp, npp, _, _, _) in calls:
                ok |= L.swarm_interact(h, pp, npp, bits, mode)
        ev1.record(stream)
        barrier()
        assert ok == 0
        clk2 = sampler2.stop()
        s_ms = ev0.elapsed_time(ev1) / (reps * K)
        s_gbs = per_launch_bytes / (s_ms * 1e-3) / 1e9
        out["sustained"] = {"launches": reps * K, "seconds": ev0.elapsed_time(ev1) * 1e-3,
                            "value": npairs_total * reps / (ev0.elapsed_time(ev1) * 1e-3), "unit": UNIT,
                            "kernel_ms": s_ms, "achieved": s_gbs, "frac": s_gbs / peak, "clocks": clk2}
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


# ncu dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel (see profiles/);
# None until a capture of the current kernel exists.
TRAFFIC = {"ring64_d1m_b4": 512.1e6}
# the same per pair of a launch, for workloads whose launches differ in their number of pairs: captured on a reduced
# copy (8 nodes, 3 pairs per launch) for the single-buffer kernel and on the full workload (14 pairs) for the
# two-register kernel; traffic is proportional to the pairs of a launch (every pair streams its own rows once)
TRAFFIC_PER_PAIR = {"regular32_resnet18_b8_nb": 214.8e6, "regular32_resnet18_b8_reg": 288.1e6}
# smsp__inst_executed.sum per 1024-coordinate block of interact_registers_kernel<8> (see profiles/)
REGISTER_KERNEL_INSTR_PER_BLOCK = 3607


def traffic_of(name, pairs_per_launch):
    if name in TRAFFIC:
        return TRAFFIC[name]
    if name in TRAFFIC_PER_PAIR:
        return TRAFFIC_PER_PAIR[name] * pairs_per_launch
    return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--stepwise", action="store_true",
                    help="sequential small-model workload: two calls per step instead of one swarm_run_sequence "
                         "call for the whole timed region")
    ap.add_argument("--fused", action="store_true",
                    help="synthetic-objective workloads: one swarm_step call per step (local steps inside the "
                         "interaction kernel) instead of swarm_local_steps + swarm_interact; measured slower, "
                         "because the step is bound by instruction issue, not by HBM")
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
