#!/usr/bin/env python
"""Benchmark of the Benes routing hot path on B200.

One "step" = one pass of the whole path over one synthetic input: benes_route
(all levels) followed by benes_apply_ex of a payload through the 2n-1 stages.
Default workload: a single uniform random permutation of N = 2^26 (uint32,
Fisher-Yates seed 2) with a 2^26-element uint64 payload.  With --gpus N every
rank routes its own permutation (seed 2 + rank): batch replicas, no collective
on the data path, weak scaling.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
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
    "r25": (25, 1, 8, 2, "profiling case: 1 x N=2^25 uniform random permutation (seed 2), route + uint64 payload apply"),
    "c5s": (24, 1, 4, 3, "C5: 1 x N=2^24 Sattolo single-cycle permutation (seed 3), route + uint32 payload apply"),
    "m10": (10, 16384, 4, 0, "mid-size batch: 16384 x N=2^10 uniform random permutations, route + uint32 payload apply"),
    "m12": (12, 4096, 4, 0, "mid-size batch: 4096 x N=2^12 uniform random permutations, route + uint32 payload apply"),
    "m16": (16, 256, 4, 0, "mid-size batch: 256 x N=2^16 uniform random permutations, route + uint32 payload apply"),
    "c5i": (24, 1, 4, 0, "C5: 1 x N=2^24 identity, route + uint32 payload apply"),
    "c5h": (24, 1, 4, 0, "C5: 1 x N=2^24 cyclic shift by 1, route + uint32 payload apply"),
    "c5b": (24, 1, 4, 0, "C5: 1 x N=2^24 bit reversal, route + uint32 payload apply"),
    "c5t": (24, 1, 4, 0, "C5: 1 x N=2^24 index map of a 4096x4096 transpose, route + uint32 payload apply"),
}
STRUCTURED = {"c5i": "identity", "c5h": "shift1", "c5b": "bitrev", "c5t": "transpose"}

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


# DRAM bytes per launch per element of the dominant kernel measured with ncu
# (dram__bytes_read.sum + dram__bytes_write.sum); see profiles/.  None until captured
# for the kernel as it stands.
NCU_DRAM_BYTES_PER_ELEMENT = {
    # mean over the 10 k_walk launches of one route at N = 2^25 (profiles/k_walk_n2p25.md),
    # scaled by the elements of a launch; the top level of a larger N moves somewhat more
    "walk": 32.8,
}
FALLBACK_HBM_GBS = 6650.0
RANDOM_GATHER_PEAK_G = 64.7


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


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


# --------------------------------------------------------------------------------------------
def run_reference(args):
    """The CPU oracle as it stands, on the host cores, on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import oracle
    from paper_1912_04050_b200 import inputs
    n_full, batch_full, ebytes, seed, desc = WORKLOADS[args.workload]
    total = args.steps + args.warmup
    n = min(n_full, 22 if total <= 12 else 20)
    if batch_full > 1:
        n, batch = n_full, min(batch_full, 4096)
        perm = inputs.random_perm_batch(n, batch, seed0=seed)
        sample = "first %d of the %d permutations of N=2^%d" % (batch, batch_full, n)
    else:
        batch = 1
        perm = inputs.random_perm(n, seed)
        sample = ("one uniform random permutation of N=2^%d (same generator and seed as the "
                  "N=2^%d workload), route + %d-byte payload apply per step" % (n, n_full, ebytes))
    x = inputs.payload_u64(batch << n, seed) if ebytes == 8 else np.tile(inputs.identity_perm(n), batch)
    x = x.reshape(batch, -1)
    times = []
    for i in range(total):
        t0 = time.perf_counter()
        bits = oracle.route(perm, n)
        out = oracle.apply(bits, x, n)
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
        "config": {"workload": desc, "reference_sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def time_cpu_baseline(name: str):
    """Oracle on a bounded sample (about 10-30 s of single-core work)."""
    import numpy as np
    import oracle
    from paper_1912_04050_b200 import inputs
    n_full, batch_full, ebytes, seed, _ = WORKLOADS[name]
    if batch_full > 1:
        n, batch = n_full, batch_full
        perm = inputs.random_perm_batch(n, batch, seed0=seed)
        sample = "all %d permutations of N=2^%d, route + apply, once" % (batch, n)
    else:
        n, batch = min(n_full, 23), 1
        perm = inputs.random_perm(n, seed)
        sample = ("one uniform random permutation of N=2^%d (same generator and seed), route + "
                  "%d-byte payload apply, once, single thread" % (n, ebytes))
    x = inputs.payload_u64(batch << n, seed) if ebytes == 8 else np.tile(inputs.identity_perm(n), batch)
    x = x.reshape(batch, -1)
    t0 = time.perf_counter()
    bits = oracle.route(perm, n)
    oracle.apply(bits, x, n)
    dt = time.perf_counter() - t0
    return {"value": (batch << n) / dt, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
            "seconds": dt}


# --------------------------------------------------------------------------------------------
def run_gpu(args):
    import numpy as np
    import torch
    from paper_1912_04050_b200 import binding
    from paper_1912_04050_b200 import build as cuda_build

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        cuda_build.build()
    if dist:
        dist.barrier()
    binding.load()
    if args.kappa is not None:
        binding.benes_set_option(binding.OPT_SAMPLE_LOG2K, args.kappa)

    name = args.workload
    n, batch, ebytes, seed, desc = WORKLOADS[name]
    perm_h, x_h = make_inputs(name, rank)
    elems = batch << n
    view = {4: np.int32, 8: np.int64}
    d_perm = torch.from_numpy(perm_h.view(np.int32)).cuda()
    d_x = torch.from_numpy(x_h.view(view[ebytes])).cuda()
    d_bits = torch.empty(binding.benes_switch_words(n, batch), dtype=torch.int32, device="cuda")
    d_out = torch.empty_like(d_x)
    stream = torch.cuda.Stream()

    def step():
        binding.benes_route(d_perm, n, batch, d_bits, stream)
        binding.benes_apply_ex(d_bits, d_x, d_out, ebytes, n, batch, stream)

    def fence():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            step()
        fence()
        # correctness guard: the routed payload must equal the gather (cheap, on device)
        idx = d_perm.view(batch, -1).to(torch.int64) & 0xFFFFFFFF
        assert torch.equal(d_out.view(batch, -1), torch.gather(d_x.view(batch, -1), 1, idx)), "routed payload wrong"
        del idx

        # ---- timed region: device-resident inputs ----
        sampler = ClockSampler(gpu_index(local_rank))
        if rank == 0:
            sampler.start()
            time.sleep(0.3)
        binding.benes_profile_reset()
        binding.benes_profile_enable(True)
        fence()
        l0 = binding.benes_launch_count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        fence()
        launches = binding.benes_launch_count() - l0
        ms_total = e0.elapsed_time(e1)
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

        # route-only / apply-only split (one extra untimed-for-value pass each)
        r0.record(stream)
        binding.benes_route(d_perm, n, batch, d_bits, stream)
        r1.record(stream)
        binding.benes_apply_ex(d_bits, d_x, d_out, ebytes, n, batch, stream)
        e1b = torch.cuda.Event(enable_timing=True)
        e1b.record(stream)
        fence()
        route_ms, apply_ms = r0.elapsed_time(r1), r1.elapsed_time(e1b)

        # ---- end to end: host buffers through the C ABI, copies inside the timed region ----
        perm_p = torch.from_numpy(perm_h.view(np.int32)).pin_memory()
        x_p = torch.from_numpy(x_h.view(view[ebytes])).pin_memory()
        bits_p = torch.empty(d_bits.numel(), dtype=torch.int32).pin_memory()
        out_p = torch.empty_like(x_p).pin_memory()

        def e2e_step():
            binding.benes_route_host(perm_p, n, batch, bits_p, stream)
            binding.benes_apply_host(bits_p, x_p, out_p, ebytes, n, batch, stream)

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
        assert torch.equal(out_p, d_out.cpu()), "end-to-end payload differs from the device-resident run"

    ms_step = ms_total / args.steps
    ms_step, e2e_ms, route_ms, apply_ms = max_over_ranks([ms_step, e2e_ms, route_ms, apply_ms], dist, "cuda")

    if rank == 0:
        peak, peak_kind = measured_peaks()
        kappa = binding.benes_get_option(binding.OPT_SAMPLE_LOG2K)
        top = max(kinds, key=lambda k: kinds[k]["ms"])
        dom = kinds[top]
        roofline = None
        if dom["launches"]:
            per_launch_s = dom["ms"] * 1e-3 / dom["launches"]
            bpe = algorithmic_bytes_per_element(top, ebytes, kappa)
            achieved = bpe * elems / per_launch_s / 1e9
            roofline = {
                "bound": "hbm", "kernel": top,
                "achieved": achieved, "peak": peak, "peak_source": peak_kind + " (STREAM-style copy)",
                "unit": "GB/s", "frac": achieved / peak,
                "traffic": (NCU_DRAM_BYTES_PER_ELEMENT[top] * elems
                            if top in NCU_DRAM_BYTES_PER_ELEMENT else None),
                "algorithmic_bytes_per_launch": bpe * elems,
                "avg_launch_ms": per_launch_s * 1e3, "launches_timed": dom["launches"],
            }
            if top == "walk" and per_level.get("walk"):
                # the walk is a chain of dependent random accesses: per switch one 16-byte
                # record and one 4-byte inverse entry (the claim hits the record's sector),
                # i.e. one access per element.  Level 0 is the launch whose block (12 B per
                # output) is furthest above the L2, so its accesses all go to DRAM.
                acc = float(elems) / (per_level["walk"][0] * 1e-3) / 1e9
                roofline["random_access"] = {
                    "launch": "level 0", "ms": per_level["walk"][0],
                    "achieved": acc, "unit": "G accesses/s", "peak": RANDOM_GATHER_PEAK_G,
                    "peak_source": "stand-alone test on this GPU: independent random 4-byte gathers "
                                   "from a 256 MiB array", "frac": acc / RANDOM_GATHER_PEAK_G,
                    # the claim (a compare-and-swap on the record) counted as a third
                    # memory operation per switch, i.e. 1.5 per element
                    "achieved_with_claims": 1.5 * acc,
                    "frac_with_claims": 1.5 * acc / RANDOM_GATHER_PEAK_G}
        bits_bytes = d_bits.numel() * 4
        line = {
            "metric": METRIC, "value": whole_job_value(elems, world, ms_step), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u32", "data": "synthetic",
            "config": {"workload": desc, "log2n": n, "batch_per_gpu": batch, "payload_bytes": ebytes,
                       "parallelism": "replicas x%d, no collective" % world,
                       "l2": "inputs larger than L2 (perm %d MiB, words %d MiB)" % (elems * 4 >> 20, elems * 8 >> 20),
                       "fused_log2m": binding.benes_fused_log2m(),
                       "ruler_spacing_log2": kappa},
            "clocks": clocks,
            "e2e": {"value": world * elems / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": perm_h.nbytes + bits_bytes + x_h.nbytes,
                    "d2h_bytes_per_step": bits_bytes + x_h.nbytes},
            "gpu_launches": launches,
            "roofline": roofline,
            "breakdown": {"route_ms": route_ms, "apply_ms": apply_ms,
                          "route_elements_per_s": elems / (route_ms * 1e-3),
                          "apply_elements_per_s": elems / (apply_ms * 1e-3),
                          "kernel_ms_per_step": {k: v["ms"] / args.steps for k, v in kinds.items()},
                          "first_step_ms_by_level": {k: v for k, v in per_level.items()
                                                     if k in ("walk", "colour", "split", "list_label", "list_walk")},
                          "kernel_launches_per_step": {k: v["launches"] // args.steps for k, v in kinds.items()}},
        }
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
    ap.add_argument("--kappa", type=int, default=None,
                    help="ruler spacing (log2) of the loop labelling; 0 = full pointer jumping")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
