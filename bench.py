#!/usr/bin/env python
"""Benchmark of the Benes routing hot path on B200.

One "step" = one pass of the whole path over one synthetic input: benes_route
(all levels) followed by benes_apply_ex of a payload through the 2n-1 stages.
Default workload: a single uniform random permutation of N = 2^26 (uint32,
Fisher-Yates seed 2) with a 2^26-element uint64 payload.

--gpus N: one process per GPU, every rank routes its own permutation (seed
2 + rank): batch replicas, no collective on the data path, weak scaling.  Under
torchrun the ranks come from the environment; started plainly with --gpus N > 1
this script starts the N ranks itself.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "routed_perm_elements_per_s"
UNIT = "elements/s"

WORKLOADS = {
    # name: (log2n, batch, payload bytes, seed, description)
    "c4": (26, 1, 8, 2, "C4: 1 x N=2^26 uniform random permutation (Fisher-Yates seed 2), route + uint64 payload apply"),
    "c3": (20, 1, 4, 1, "C3: 1 x N=2^20 uniform random permutation (seed 1), route + fp32 payload apply"),
    "c2": (8, 16384, 4, 0, "C2: 16384 x N=2^8 uniform random permutations (seeds 0..16383), route + uint32 payload apply"),
    "c1": (10, 1, 4, 0, "C1: 1 x N=2^10 uniform random permutation (seed 0), route + uint32 identity payload apply"),
    "r25": (25, 1, 8, 2, "profiling case: 1 x N=2^25 uniform random permutation (seed 2), route + uint64 payload apply"),
    "r22": (22, 1, 8, 2, "profiling case: 1 x N=2^22 uniform random permutation (seed 2), route + uint64 payload apply"),
    "c5s": (24, 1, 4, 3, "C5: 1 x N=2^24 Sattolo single-cycle permutation (seed 3), route + uint32 payload apply"),
    "m10": (10, 16384, 4, 0, "mid-size batch: 16384 x N=2^10 uniform random permutations, route + uint32 payload apply"),
    "m12": (12, 4096, 4, 0, "mid-size batch: 4096 x N=2^12 uniform random permutations, route + uint32 payload apply"),
    "m16": (16, 256, 4, 0, "mid-size batch: 256 x N=2^16 uniform random permutations, route + uint32 payload apply"),
    "m17": (17, 128, 4, 0, "mid-size batch: 128 x N=2^17 uniform random permutations, route + uint32 payload apply"),
    "c5i": (24, 1, 4, 0, "C5: 1 x N=2^24 identity, route + uint32 payload apply"),
    "c5h": (24, 1, 4, 0, "C5: 1 x N=2^24 cyclic shift by 1, route + uint32 payload apply"),
    "c5b": (24, 1, 4, 0, "C5: 1 x N=2^24 bit reversal, route + uint32 payload apply"),
    "c5t": (24, 1, 4, 0, "C5: 1 x N=2^24 index map of a 4096x4096 transpose, route + uint32 payload apply"),
}
STRUCTURED = {"c5i": "identity", "c5h": "shift1", "c5b": "bitrev", "c5t": "transpose"}
L2_BYTES = 126 << 20
# workloads whose summary rides along in the default (C4) line: the rest of the metric's range (C3,
# C2) and the remaining configurations (C1, the five structured permutations of C5)
SIDE_WORKLOADS = ("c3", "c2", "c1", "c5s", "c5i", "c5h", "c5b", "c5t")


def algorithmic_bytes_per_element(kind: str, ebytes: int, kappa: int) -> float:
    """Useful bytes one launch of a kernel kind moves per permutation element."""
    k = float(1 << max(kappa, 1))
    return {
        # per switch, visited once: P[j^1] read (4 B), owner word read and written (8 B),
        # Q[.] read (4 B) -> 8 B per element; one 16-byte walk record per ruler output
        "walk": 8.0 + 16.0 / k,
        # build 16 B + (m-2) passes of 24 B + last 8 B per element, m ~ 20 on average
        "full_label": 16.0 + 18 * 24.0 + 8.0,
        # payload pair in, pair out, one switch bit per pair
        "apply": 2.0 * ebytes + 1.0 / 16.0,
        "apply_fused": 2.0 * ebytes + 1.0 / 16.0,
        # P read (4 B), record written (8 B), Q scattered (4 B)
        "inverse": 16.0,
        # record (8 B) and Q (4 B) read, record (8 B) and Q' (4 B) written, two stage bits
        "split": 24.0 + 1.0 / 8.0,
        # owner word per switch, contracted word per switch, one stage bit
        "colour": 2.0 + 4.0 + 1.0 / 16.0,
        "combine": (16.0 + 16.0 + 8.0) / k, "list_walk": 20.0 / k, "list_label": 16.0 / k / 16.0,
        "list_resolve": 24.0 / k,
        "fused": 4.0 + (2 * 15 - 1) / 16.0,
    }[kind]


FALLBACK_HBM_GBS = 6650.0
# which source file holds the kernels of a profile kind (its hash guards the stored ncu counters)
KIND_SOURCE = {"walk": "route_sampled.cu", "colour": "route_sampled.cu", "fused": "route_fused.cu",
               "split": "route_levels.cu", "inverse": "route_levels.cu", "apply_fused": "apply_fused.cu"}


def binding_packed_level0(n: int, kappa: int) -> bool:
    """Whether level 0 of a permutation of 2^n uses packed 8-byte records (the library's rule)."""
    return kappa != 0 and 3 * n - kappa + 1 < 64


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def source_hash(fname: str) -> str:
    with open(os.path.join(ROOT, "paper_1912_04050_b200", "csrc", fname), "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:16]


def stored_dram_traffic(kind: str, workload: str):
    """DRAM bytes per launch (read + write) of one kernel kind on one workload, from the
    ncu counters kept as text beside the other profile summaries; None if there are none,
    or if the kernel's source file has changed since they were taken."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    try:
        with open(path) as f:
            rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    except OSError:
        return None
    for row in rows:
        rec = dict(kv.split("=", 1) for kv in row)
        if rec.get("kind") == kind and rec.get("workload") == workload:
            src = KIND_SOURCE.get(kind)
            if src is None or rec.get("source_sha") != source_hash(src):
                return None
            return float(rec["dram_bytes_per_launch"])
    return None


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi during the timed region."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            pass
    return local_rank


def max_over_ranks(values, dist, device):
    """Every rank's timings -> the slowest rank's (all ranks get the same list)."""
    import torch
    vals = torch.tensor(values, dtype=torch.float64, device=device)
    if dist:
        dist.all_reduce(vals, op=dist.ReduceOp.MAX)
    return vals.tolist()


def whole_job_value(elems_per_rank: int, world: int, ms_per_step: float) -> float:
    """Elements all ranks routed per second (replicas: every rank does elems_per_rank per step)."""
    return world * elems_per_rank / (ms_per_step * 1e-3)


def make_inputs(name: str, rank: int):
    import numpy as np
    from paper_1912_04050_b200 import inputs
    n, batch, ebytes, seed, _ = WORKLOADS[name]
    if name == "c5s":
        perm = inputs.sattolo_perm(n, seed + rank)
    elif name in STRUCTURED:
        perm = inputs.structured_perms(n)[STRUCTURED[name]]
    elif batch == 1:
        perm = inputs.random_perm(n, seed + rank)
    else:
        perm = inputs.random_perm_batch(n, batch, seed0=seed + rank * batch)
    if ebytes == 8:
        x = inputs.payload_u64(batch << n, seed)
    elif name == "c3":
        x = inputs.payload_f32(batch << n, seed)
    else:
        x = np.tile(inputs.identity_perm(n), batch)
    return perm.reshape(-1), x


# ---- ranks ----------------------------------------------------------------------------------
def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(world: int, argv, extra_env=None) -> int:
    """Start `world` copies of this script, one per GPU, with the rendezvous variables
    torchrun would set (127.0.0.1, a free port).  Returns the first non-zero exit code."""
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   LOCAL_WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=env))
    rc = 0
    for p in procs:
        p.wait()
        rc = rc or p.returncode
    return rc


def init_ranks(args, backend: str):
    """(rank, local_rank, world, dist or None) from the environment; checks --gpus against it."""
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        raise SystemExit("bench.py: --gpus %d but WORLD_SIZE=%d" % (args.gpus, world))
    dist = None
    if world > 1:
        import torch
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group(backend)
    return rank, local_rank, world, dist


def run_rank_check(args):
    """The rank plumbing alone, on the CPU (gloo): every rank builds its inputs, pretends to
    need (rank + 1) ms per step, and rank 0 prints the line skeleton.  Used by the tests."""
    rank, _, world, dist = init_ranks(args, "gloo")
    n, batch, _, _, desc = WORKLOADS[args.workload]
    perm, _ = make_inputs(args.workload, rank)
    ms_step, = max_over_ranks([1.0 + rank], dist, "cpu")
    digest = hashlib.sha256(perm.tobytes()).hexdigest()[:16]
    digests = [None] * world
    if dist:
        dist.all_gather_object(digests, digest)
    else:
        digests = [digest]
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": whole_job_value(batch << n, world, ms_step), "unit": UNIT,
                          "n_gpus": world, "ms_per_step": ms_step, "scaling": "weak",
                          "config": {"workload": desc}, "rank_inputs": digests}), flush=True)
    if dist:
        dist.barrier()
        dist.destroy_process_group()


# ---- CPU oracle legs -------------------------------------------------------------------------
def oracle_step(perm, x, n, threads):
    import oracle
    if threads > 1:
        bits = oracle.route_parallel(perm, n, threads)
        return oracle.apply_parallel(bits, x, n, threads)
    bits = oracle.route(perm, n)
    return oracle.apply(bits, x, n)


def oracle_inputs(name: str, n: int, batch: int):
    import numpy as np
    from paper_1912_04050_b200 import inputs
    _, _, ebytes, seed, _ = WORKLOADS[name]
    if name == "c5s":
        perm = inputs.sattolo_perm(n, seed)
    elif name in STRUCTURED:
        perm = inputs.structured_perms(n)[STRUCTURED[name]]
    else:
        perm = inputs.random_perm_batch(n, batch, seed0=seed) if batch > 1 else inputs.random_perm(n, seed)
    x = inputs.payload_u64(batch << n, seed) if ebytes == 8 else np.tile(inputs.identity_perm(n), batch)
    return perm, x.reshape(batch, -1) if batch > 1 else x


def run_reference(args):
    """The CPU oracle as it stands, one thread, on the host cores.  A step of the full C4
    workload takes about a minute, so each step runs a bounded sample: the largest N (same
    generator and seed) for which steps + warm-up finish within about three minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_full, batch_full, ebytes, seed, desc = WORKLOADS[args.workload]
    total = args.steps + args.warmup
    budget_s = 170.0
    if batch_full > 1:
        n, batch = n_full, batch_full
        perm, x = oracle_inputs(args.workload, n, batch)
        t0 = time.perf_counter(); oracle_step(perm[:256], x[:256], n, 1); t256 = time.perf_counter() - t0
        while batch > 256 and t256 * (batch / 256.0) * total > budget_s:
            batch //= 2
        perm, x = perm[:batch], x[:batch]
        sample = "first %d of the %d permutations of N=2^%d, route + apply per step" % (batch, batch_full, n)
    else:
        batch = 1
        n_cal = min(n_full, 20)
        perm, x = oracle_inputs(args.workload, n_cal, 1)
        t0 = time.perf_counter(); oracle_step(perm, x, n_cal, 1); t_cal = time.perf_counter() - t0
        n = n_cal
        # time per element grows slowly with N (cache misses): allow 15 % per doubling
        while n < n_full and t_cal * (2.3 ** (n + 1 - n_cal)) * total <= budget_s:
            n += 1
        perm, x = oracle_inputs(args.workload, n, 1)
        sample = ("one uniform random permutation of N=2^%d (same generator and seed as the N=2^%d "
                  "workload; the largest size whose %d steps fit in about %d s), route + %d-byte payload "
                  "apply per step" % (n, n_full, total, int(budget_s), ebytes))
    times = []
    for i in range(total):
        t0 = time.perf_counter()
        out = oracle_step(perm, x, n, 1)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
    assert out.shape == x.shape
    elems = batch << n
    ms = 1e3 * sum(times) / len(times)
    value = elems / (ms * 1e-3)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
        "config": {"workload": desc, "reference_sample": sample, "sample_log2n": n, "sample_batch": batch},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "nproc": os.cpu_count(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def time_cpu_baseline(name: str):
    """The oracle, once, on the benched workload itself (same generator, seed and size):
    single thread (the oracle is sequential by definition), then on all host cores over
    independent units only (permutations of a batch; for one permutation the sub-networks
    below level ceil(log2 cores), the levels above them on one thread)."""
    import numpy as np
    n, batch, ebytes, _, _ = WORKLOADS[name]
    perm, x = oracle_inputs(name, n, batch)
    cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    out1 = oracle_step(perm, x, n, 1)
    dt1 = time.perf_counter() - t0
    t0 = time.perf_counter()
    outp = oracle_step(perm, x, n, cores)
    dtp = time.perf_counter() - t0
    assert np.array_equal(out1, outp)
    what = ("all %d permutations of N=2^%d" % (batch, n)) if batch > 1 else ("the whole N=2^%d permutation" % n)
    return {"value": (batch << n) / dt1, "unit": UNIT, "cores": 1, "kind": "oracle", "nproc": cores,
            "sample": "%s (same generator and seed as the GPU run), route + %d-byte payload apply, once, one thread"
                      % (what, ebytes),
            "seconds": dt1,
            "all_cores": {"value": (batch << n) / dtp, "unit": UNIT, "cores": cores, "seconds": dtp,
                          "how": ("permutations spread over the threads" if batch > 1 else
                                  "levels above the split on one thread, the independent sub-networks "
                                  "below it on %d threads" % cores)}}


# ---- GPU legs --------------------------------------------------------------------------------
class GpuCase:
    """Device-resident inputs and outputs of one workload on the current device."""

    def __init__(self, name: str, rank: int, stream):
        import numpy as np
        import torch
        from paper_1912_04050_b200 import binding
        self.name, self.stream, self.binding = name, stream, binding
        self.n, self.batch, self.ebytes, _, self.desc = WORKLOADS[name]
        self.perm_h, self.x_h = make_inputs(name, rank)
        self.elems = self.batch << self.n
        self.view = {4: np.int32, 8: np.int64}[self.ebytes]
        self.d_perm = torch.from_numpy(self.perm_h.view(np.int32)).cuda()
        self.d_x = torch.from_numpy(self.x_h.view(self.view)).cuda()
        self.d_bits = torch.empty(binding.benes_switch_words(self.n, self.batch), dtype=torch.int32, device="cuda")
        self.d_out = torch.empty_like(self.d_x)
        self.input_bytes = self.perm_h.nbytes + self.x_h.nbytes

    def step(self):
        b = self.binding
        b.benes_route(self.d_perm, self.n, self.batch, self.d_bits, self.stream)
        b.benes_apply_ex(self.d_bits, self.d_x, self.d_out, self.ebytes, self.n, self.batch, self.stream)

    def check(self):
        """the routed payload must equal the gather (on the device)"""
        import torch
        idx = self.d_perm.view(self.batch, -1).to(torch.int64) & 0xFFFFFFFF
        ok = torch.equal(self.d_out.view(self.batch, -1), torch.gather(self.d_x.view(self.batch, -1), 1, idx))
        assert ok, "routed payload wrong (%s)" % self.name


class L2Flush:
    """Writes a buffer twice the size of the L2 between timed iterations of small workloads."""

    def __init__(self):
        import torch
        self.buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")

    def __call__(self):
        self.buf.fill_(1)


def time_steps(case: GpuCase, steps: int, flush):
    """Per-step device times (ms).  Inputs above the L2 size run back to back inside one
    event pair; smaller ones are timed step by step with the L2 flushed in between."""
    import torch
    s = case.stream
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s)
        for _ in range(steps):
            case.step()
        e1.record(s)
        torch.cuda.synchronize()
        return [e0.elapsed_time(e1) / steps] * steps
    pairs = []
    for _ in range(steps):
        flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s)
        case.step()
        e1.record(s)
        pairs.append((e0, e1))
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in pairs]


PROBE_MODES = {
    # name: (mode, record bytes, records = elements >> shift, what it stands for)
    "load4": (0, 4, 0, "4-byte load from an array of one word per element (the inverse entry of a hop)"),
    "load16": (1, 16, 1, "16-byte load of a wide switch record"),
    "load16_cas": (2, 16, 1, "16-byte load + compare-and-swap on its owner word (a visit of a wide record)"),
    "and64": (3, 8, 1, "64-bit atomic AND on an 8-byte record (a visit of a packed record)"),
    "store4": (4, 16, 1, "4-byte store into a 16-byte record"),
}


def probe_random_access(binding, stream, log2_elems: int):
    """Independent random accesses, one per switch of a level of 2^log2_elems outputs, on
    arrays of that level's sizes: G operations/s per access pattern (best of 3)."""
    import torch
    switches = 1 << (log2_elems - 1)
    table = torch.empty(switches * 16, dtype=torch.uint8, device="cuda")
    sink = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = {}
    for name, (mode, rbytes, shift, what) in PROBE_MODES.items():
        best = None
        for _ in range(3):
            table.fill_(255)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            binding.benes_probe_random_access(table, log2_elems - shift, rbytes, mode, switches, sink, stream)
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            best = ms if best is None else min(best, ms)
        out[name] = {"g_ops_per_s": switches / (best * 1e-3) / 1e9, "ms": best, "ops": switches,
                     "table_bytes": (1 << (log2_elems - shift)) * rbytes, "what": what}
    del table
    return out


def side_workload(name: str, rank: int, stream, flush, steps: int = 10):
    """Short summary of another configuration (device-resident, L2 flushed between steps)."""
    import torch
    case = GpuCase(name, rank, stream)
    with torch.cuda.stream(stream):
        for _ in range(3):
            case.step()
        torch.cuda.synchronize()
        case.check()
        ms = time_steps(case, steps, flush)
        r0, r1, r2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        flush()
        r0.record(stream)
        case.binding.benes_route(case.d_perm, case.n, case.batch, case.d_bits, stream)
        r1.record(stream)
        case.binding.benes_apply_ex(case.d_bits, case.d_x, case.d_out, case.ebytes, case.n, case.batch, stream)
        r2.record(stream)
        torch.cuda.synchronize()
        # the same step as a plan (benes_plan_create: captured once into a CUDA graph with a
        # scratch buffer of its own; benes_plan_launch replays it with one call): what a caller
        # with fixed buffers gets for the 2-50 short dependent launches of these sizes
        graph_ms = None
        if case.elems <= (1 << 22):
            plan = case.binding.Plan(case.d_perm, case.n, case.batch, case.d_bits, case.d_x, case.d_out, case.ebytes)
            pairs = []
            for _ in range(steps):
                flush()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                plan.launch(stream)
                e1.record(stream)
                pairs.append((e0, e1))
            torch.cuda.synchronize()
            case.check()
            graph_ms = statistics.median(a.elapsed_time(b) for a, b in pairs)
            plan.destroy()
    med = statistics.median(ms)
    elems = case.elems
    del case
    torch.cuda.empty_cache()
    out = {"workload": WORKLOADS[name][4], "ms_per_step": med, "best_ms": min(ms), "steps": steps,
           "value": elems / (med * 1e-3), "unit": UNIT, "l2": "flushed between steps",
           "route_ms": r0.elapsed_time(r1), "apply_ms": r1.elapsed_time(r2)}
    if graph_ms is not None:
        out["plan_replay"] = {"ms_per_step": graph_ms, "value": elems / (graph_ms * 1e-3), "unit": UNIT,
                              "api": "benes_plan_create once, benes_plan_launch per step"}
    return out


def run_gpu(args):
    import numpy as np
    import torch
    from paper_1912_04050_b200 import binding
    from paper_1912_04050_b200 import build as cuda_build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    rank, local_rank, world, dist = init_ranks(args, "nccl")
    torch.cuda.set_device(local_rank)
    if rank == 0:
        cuda_build.build()
    if dist:
        dist.barrier()
    binding.load()
    if args.kappa is not None:
        binding.benes_set_option(binding.OPT_SAMPLE_LOG2K, args.kappa)

    if args.cluster is not None:
        binding.benes_set_option(binding.OPT_CLUSTER, args.cluster)
    if args.apply_fused is not None:
        binding.benes_set_option(binding.OPT_APPLY_FUSED, args.apply_fused)
    if args.walk_pairs is not None:
        binding.benes_set_option(binding.OPT_WALK_PAIRS, args.walk_pairs)

    name = args.workload
    stream = torch.cuda.Stream()
    if args.probe_only:
        n0, b0 = WORKLOADS[name][0], WORKLOADS[name][1]
        with torch.cuda.stream(stream):
            print(json.dumps({"random_access_probe": probe_random_access(binding, stream, n0 + (b0.bit_length() - 1))}),
                  flush=True)
        return
    case = GpuCase(name, rank, stream)
    n, batch, ebytes, elems = case.n, case.batch, case.ebytes, case.elems
    flush = None if case.input_bytes > L2_BYTES else L2Flush()
    warmup = max(args.warmup, 3)

    def fence():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        for _ in range(warmup):
            case.step()
        fence()
        case.check()

        # ---- timed region: device-resident inputs, K steps, nothing but the library's launches
        sampler = ClockSampler(gpu_index(local_rank))
        if rank == 0:
            sampler.start()
            time.sleep(0.3)
        binding.benes_profile_enable(False)
        fence()
        l0 = binding.benes_launch_count()
        step_ms = time_steps(case, args.steps, flush)
        fence()
        launches = binding.benes_launch_count() - l0
        # ---- the same K steps once more with the library's per-kind event brackets on (two event
        # records per group of launches, about 170 per C4 step): the per-kernel times of the
        # roofline and the breakdown come from this region, whose steps are a few per cent slower
        binding.benes_profile_reset()
        binding.benes_profile_enable(not args.no_brackets)
        fence()
        bracketed_ms = time_steps(case, args.steps, flush)
        fence()
        binding.benes_profile_enable(False)
        kinds = {}
        for k in range(binding.PROFILE_KINDS):
            cnt, ms = binding.benes_profile_read(k)
            kinds[binding.benes_profile_kind_name(k)] = {"launches": cnt, "ms": ms}
        spans = binding.benes_profile_spans()
        per_level = {}
        for kname, _, ms in spans[:len(spans) // args.steps]:       # first timed step
            per_level.setdefault(kname, []).append(round(ms, 3))
        binding.benes_profile_reset()
        clocks = sampler.stop() if rank == 0 else None

        # route-only / apply-only split (one extra pass, not part of `value`)
        r0, r1, r2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        r0.record(stream)
        binding.benes_route(case.d_perm, n, batch, case.d_bits, stream)
        r1.record(stream)
        binding.benes_apply_ex(case.d_bits, case.d_x, case.d_out, ebytes, n, batch, stream)
        r2.record(stream)
        fence()
        route_ms, apply_ms = r0.elapsed_time(r1), r1.elapsed_time(r2)

        # ---- end to end: host buffers through the C ABI, copies inside the timed region ----
        perm_p = torch.from_numpy(case.perm_h.view(np.int32)).pin_memory()
        x_p = torch.from_numpy(case.x_h.view(case.view)).pin_memory()
        bits_p = torch.empty(case.d_bits.numel(), dtype=torch.int32).pin_memory()
        out_p = torch.empty_like(x_p).pin_memory()

        def e2e_step():
            # one call: permutation and payload in, switch words and routed payload out
            binding.benes_route_apply_host(perm_p, x_p, out_p, ebytes, n, batch, bits_p, stream)

        e2e_step()
        fence()
        e2e_steps = max(1, min(args.steps, 5))
        t0 = time.perf_counter()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for _ in range(e2e_steps):
            e2e_step()
        g1.record(stream)
        fence()
        e2e_ms = max(g0.elapsed_time(g1), 1e3 * (time.perf_counter() - t0)) / e2e_steps
        assert torch.equal(out_p, case.d_out.cpu()), "end-to-end payload differs from the device-resident run"
        del perm_p, x_p, out_p

        probe = None
        if rank == 0 and n >= 20 and not args.no_probe:
            probe = probe_random_access(binding, stream, n + (batch.bit_length() - 1))

    ms_step = sum(step_ms) / len(step_ms)
    ms_step, e2e_ms, route_ms, apply_ms = max_over_ranks([ms_step, e2e_ms, route_ms, apply_ms], dist, "cuda")

    if rank == 0:
        peak, peak_kind = measured_peaks()
        kappa = binding.benes_get_option(binding.OPT_SAMPLE_LOG2K)
        top = max(kinds, key=lambda k: kinds[k]["ms"])
        dom = kinds[top]
        roofline = None
        if dom["launches"] and dom["ms"] > 0:
            per_launch_s = dom["ms"] * 1e-3 / dom["launches"]
            bpe = algorithmic_bytes_per_element(top, ebytes, kappa)
            achieved = bpe * elems / per_launch_s / 1e9
            roofline = {
                "bound": "hbm", "kernel": top,
                "achieved": achieved, "peak": peak, "peak_source": peak_kind + " (STREAM-style copy)",
                "unit": "GB/s", "frac": achieved / peak,
                "traffic": stored_dram_traffic(top, name),
                "algorithmic_bytes_per_launch": bpe * elems,
                "avg_launch_ms": per_launch_s * 1e3, "launches_timed": dom["launches"],
            }
            traffic = roofline["traffic"]
            if traffic:
                # what the DRAM actually moved for this kernel (ncu counters of the same workload)
                roofline["dram_gbs"] = traffic / per_launch_s / 1e9
                roofline["dram_frac"] = traffic / per_launch_s / 1e9 / peak
                roofline["dram_frac_of_nominal_8tbs"] = traffic / per_launch_s / 1e9 / 8000.0
            if top == "walk" and per_level.get("walk") and probe:
                # The walk is a chain of dependent random accesses: per switch one record visit
                # (load + claim) and one 4-byte inverse entry.  Level 0 is the launch whose block
                # is furthest above the L2.  The time the same accesses take when they are
                # independent (measured in this run on arrays of the same sizes) is the floor.
                visit = "load16_cas" if per_level["walk"][0] and not binding_packed_level0(n, kappa) else "and64"
                floor_ms = probe[visit]["ms"] + probe["load4"]["ms"]
                roofline["random_access"] = {
                    "launch": "level 0", "ms": per_level["walk"][0],
                    "floor_ms": floor_ms, "frac": floor_ms / per_level["walk"][0],
                    "floor": "independent accesses of the same kinds and counts on arrays of the same "
                             "sizes (benes_probe_random_access, this run): %s %.3f ms + load4 %.3f ms"
                             % (visit, probe[visit]["ms"], probe["load4"]["ms"])}
        bits_bytes = case.d_bits.numel() * 4
        line = {
            "metric": METRIC, "value": whole_job_value(elems, world, ms_step), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u32", "data": "synthetic",
            "config": {"workload": case.desc, "log2n": n, "batch_per_gpu": batch, "payload_bytes": ebytes,
                       "parallelism": "replicas x%d, no collective" % world,
                       "l2": ("inputs larger than L2 (perm %d MiB, payload %d MiB)"
                              % (case.perm_h.nbytes >> 20, case.x_h.nbytes >> 20)) if flush is None
                             else "L2 flushed between timed steps (a 252 MiB buffer is written)",
                       "fused_log2m": binding.benes_fused_log2m(),
                       "ruler_spacing_log2": kappa},
            "clocks": clocks,
            "e2e": {"value": world * elems / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                    "api": "benes_route_apply_host (pinned host buffers; switch words returned too)",
                    "h2d_bytes_per_step": case.perm_h.nbytes + case.x_h.nbytes,
                    "d2h_bytes_per_step": bits_bytes + case.x_h.nbytes},
            "gpu_launches": launches,
            "roofline": roofline,
            "breakdown": {"ms_per_step_with_event_brackets": sum(bracketed_ms) / len(bracketed_ms),
                          "route_ms": route_ms, "apply_ms": apply_ms,
                          "route_elements_per_s": elems / (route_ms * 1e-3),
                          "apply_elements_per_s": elems / (apply_ms * 1e-3),
                          "kernel_ms_per_step": {k: v["ms"] / args.steps for k, v in kinds.items()},
                          "first_step_ms_by_level": {k: v for k, v in per_level.items()
                                                     if k in ("walk", "colour", "split", "list_label", "list_walk")},
                          "kernel_launches_per_step": {k: v["launches"] // args.steps for k, v in kinds.items()}},
        }
        if probe:
            line["random_access_probe"] = probe
        if world == 1 and name == "c4" and not args.no_side_workloads:
            del case
            torch.cuda.empty_cache()
            fl = flush or L2Flush()
            line["other_workloads"] = {w: side_workload(w, rank, stream, fl) for w in SIDE_WORKLOADS}
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = time_cpu_baseline(name)
        print(json.dumps(line), flush=True)
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-side-workloads", action="store_true")
    ap.add_argument("--no-probe", action="store_true", help="skip the random-access probe")
    ap.add_argument("--no-brackets", action="store_true",
                    help="time the steps without the library's per-kind event brackets (no roofline then)")
    ap.add_argument("--probe-only", action="store_true",
                    help="run only the random-access probe for the workload's size (for profiling it)")
    ap.add_argument("--kappa", type=int, default=None,
                    help="ruler spacing (log2) of the loop labelling; 0 = full pointer jumping")
    ap.add_argument("--cluster", type=int, default=None,
                    help="1: blocks of 2^16 finished by clusters of two CTAs; 0: blocks of 2^15 in one CTA")
    ap.add_argument("--apply-fused", type=int, default=None,
                    help="0: one payload-apply kernel per stage; 1: several stages per pass (default)")
    ap.add_argument("--walk-pairs", type=int, default=None,
                    help="ruler walks per thread: 0 one, 1 two where it pays (default), 2 two wherever possible")
    ap.add_argument("--rank-check", action="store_true",
                    help="run only the rank plumbing on the CPU (gloo); used by the tests")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly: be the launcher (NCCL's own log stays on for the ranks)
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.rank_check:
        run_rank_check(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
