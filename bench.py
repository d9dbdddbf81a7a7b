#!/usr/bin/env python
"""Benchmark of the MoE decode layer on VQ + shared-basis low-rank expert weights.

A step is ONE call of the whole layer (router, top-k, grouping, gate/up, SwiGLU, down, weighted
sum) on one batch of tokens.  Steps rotate over L distinct synthetic layers so that every call
reads its weights from HBM, not from L2.  Metric: microseconds per MoE layer per token.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload qwen3|qwen3_b16|dsv2lite|dsv2lite_b8|mixtral|...] [--mode full|paper|dense]

N > 1 (launched with torch.distributed.run) runs independent replicas, one per GPU: the path
has no exchange step, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import warnings
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

# DRAM bytes (read + write) per launch of the dominant kernels come from the ncu captures
# summarised under profiles/; the table profiles/dram_traffic.md lists them with their source.
def ncu_traffic_table():
    """{(workload, mode, kernel): (bytes per launch, source)} parsed from profiles/dram_traffic.md."""
    table = {}
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.md")) as f:
            for line in f:
                cells = [c.strip() for c in line.strip().strip("|").split("|")]
                if len(cells) >= 5 and cells[0] not in ("workload", "") and not set(cells[0]) <= set("-: "):
                    try:
                        table[(cells[0], cells[1], cells[2].strip("`"))] = (float(cells[3]), cells[4])
                    except ValueError:
                        pass
    except OSError:
        pass
    return table


L2_BYTES = 126 * 1024 * 1024
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


# a stage the configuration does not have captures an empty graph: expected, not worth a warning per layer
warnings.filterwarnings("ignore", message="The CUDA Graph is empty")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4800)
    ap.add_argument("--warmup", type=int, default=240)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen3")
    ap.add_argument("--mode", default="full", choices=["full", "paper", "dense"])
    ap.add_argument("--layers", type=int, default=0, help="distinct layers to rotate over (0 = auto)")
    ap.add_argument("--no-extras", action="store_true", help="skip the secondary measurements")
    ap.add_argument("--ablate", default="", choices=["", "z", "launch", "both"],
                    help="switch a mechanism off (Section 5.4): z = shared projections recomputed per expert, "
                         "launch = one gate/up and one down launch per work group")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--flags", type=int, default=0,
                    help="extra MOE_VQLR_FLAG_* bits for the handles of the main workload (A/B runs of the kernel paths)")
    return ap.parse_args()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def max_over_ranks(value: float, world: int, device="cuda") -> float:
    """Maximum of a per-rank scalar over all ranks (replicas report the slowest rank's time)."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self._stop = threading.Event()
        self._thr = None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}",
                                      "--format=csv,noheader,nounits"], capture_output=True,
                                     text=True, timeout=5).stdout.strip()
                if out:
                    self.rows.append([c.strip() for c in out.splitlines()[0].split(",")])
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thr.join(timeout=6)

    def summary(self) -> dict:
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except Exception:
                continue
            for name, v in zip(names, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on the host cores
# ------------------------------------------------------------------------------------------
def oracle_timing(workload: str, mode: str, budget_s: float, max_steps: int, warmup: int = 1):
    """Times full oracle layer calls (fp64, dense reconstruction) on a numpy-generated layer of
    the same shape; stops after `max_steps` calls or when `budget_s` of CPU time is used."""
    import oracle
    from paper_2609_21137_b200 import synth
    shp = synth.shape(workload, mode=mode)
    layer = synth.make_layer(shp, seed=0)
    orc = oracle.OracleLayer.from_synth(layer)
    for _ in range(warmup):
        orc.decode_layer(layer.x)
    times = []
    t_start = time.perf_counter()
    while len(times) < max_steps and (time.perf_counter() - t_start) < budget_s:
        t0 = time.perf_counter()
        orc.decode_layer(layer.x)
        times.append(time.perf_counter() - t0)
    mean_s = sum(times) / len(times)
    return dict(us_per_layer_per_token=mean_s * 1e6 / shp.T, calls=len(times), cores=oracle.threads(),
                T=shp.T, mean_s=mean_s)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    r = oracle_timing(args.workload, args.mode, budget_s=150.0, max_steps=max(1, args.steps),
                      warmup=min(max(args.warmup, 1), 2))
    sample = (f"{r['calls']} full fp64 oracle layer calls of the {args.workload} shape (mode {args.mode}, "
              f"T={r['T']}, seed 0) on the host cores; {args.steps} steps requested, capped at 150 s")
    line = {"impl": "reference", "metric": "us_per_moe_layer_per_token", "value": r["us_per_layer_per_token"],
            "unit": "us", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": r["mean_s"] * 1e3, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{args.workload} T={r['T']} mode={args.mode}"},
            "cpu_baseline": {"value": r["us_per_layer_per_token"], "unit": "us", "cores": r["cores"],
                             "kind": "oracle", "sample": sample},
            "e2e": {"value": r["us_per_layer_per_token"], "unit": "us", "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------
class Workload:
    """L distinct layers of one shape on the GPU, with per-layer token batches."""

    def __init__(self, name: str, mode: str, n_layers: int, device, flags: int = 0):
        import torch
        from paper_2609_21137_b200 import accounting, binding, devsynth, synth
        self.torch = torch
        self.shp = synth.shape(name, mode=mode)
        self.name, self.mode, self.device = name, mode, device
        shp = self.shp
        probe = accounting.layer_bytes(H=shp.H, I=shp.I, E=shp.E, d=shp.d, K=shp.K, r=shp.r, T=shp.T,
                                       mode=mode, n_active=shp.k + shp.S, up_only=shp.act == "relu2", idx12=shp.idx12)
        if n_layers <= 0:       # enough distinct layers that one rotation touches > 2.5x L2
            n_layers = max(4, min(64, -(-int(2.5 * L2_BYTES) // max(probe.total, 1))))
        self.layers, self.xs, self.outs = [], [], []
        for i in range(n_layers):
            kw = devsynth.make_device_layer(shp, seed=1000 + i, device=device)
            x = kw.pop("x")
            self.layers.append(binding.MoeVqlrLayer(flags=flags, **kw))
            self.xs.append(x)
            self.outs.append(torch.empty_like(x))
        torch.cuda.synchronize(device)
        # routing of every layer (distinct activated experts) for the byte accounting
        self.bytes = []
        for lay, x in zip(self.layers, self.xs):
            _, dbg = lay.decode(x, debug=True)
            n_act = int((dbg["counts"] > 0).sum().item()) + shp.S
            self.bytes.append(accounting.layer_bytes(H=shp.H, I=shp.I, E=shp.E, d=shp.d, K=shp.K, r=shp.r,
                                                     T=shp.T, mode=mode, n_active=n_act,
                                                     up_only=shp.act == "relu2", idx12=shp.idx12))
        torch.cuda.synchronize(device)
        self.mean_bytes = sum(b.total for b in self.bytes) / len(self.bytes)
        self.mean_active = sum(b.n_active for b in self.bytes) / len(self.bytes)

    def step(self, i: int):
        j = i % len(self.layers)
        self.layers[j].decode(self.xs[j], out=self.outs[j])

    def launches(self) -> int:
        return sum(l.launch_count for l in self.layers)

    def capture(self, n_calls: int, stage: str = None):
        """CUDA graph of `n_calls` consecutive layer calls (layer i % L each), or of one stage's
        kernel per layer.  Returns (graph, kernel launches inside it)."""
        torch = self.torch
        g = torch.cuda.CUDAGraph()
        n0 = self.launches()
        with torch.cuda.graph(g):
            for i in range(n_calls):
                j = i % len(self.layers)
                if stage is None:
                    self.layers[j].decode(self.xs[j], out=self.outs[j])
                else:
                    self.layers[j].run_stage(stage, self.xs[j], self.outs[j])
        return g, self.launches() - n0

    def prepare(self, steps: int):
        """Graphs for a timed region of exactly `steps` calls: whole rotations plus a remainder."""
        L = len(self.layers)
        self.g_full, self.n_full = self.capture(L)
        self.rem = steps % L
        self.g_rem, self.n_rem = self.capture(self.rem) if self.rem else (None, 0)
        self.reps = steps // L

    def warm(self, warmup: int):
        L = len(self.layers)
        for _ in range(max(1, -(-warmup // L))):
            self.g_full.replay()

    def timed_region(self):
        """Enqueue exactly reps * L + rem calls; returns kernel launches enqueued."""
        for _ in range(self.reps):
            self.g_full.replay()
        if self.g_rem is not None:
            self.g_rem.replay()
        return self.reps * self.n_full + self.n_rem

    def timed_regions(self, regions: int):
        """`regions` timed regions of exactly reps * L + rem calls each, every one bracketed by its own
        pair of CUDA events on the launching stream; returns (list of ms, launches per region)."""
        torch = self.torch
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(regions)]
        n = 0
        for e0, e1 in ev:
            e0.record()
            n = self.timed_region()
            e1.record()
        torch.cuda.synchronize(self.device)
        return [e0.elapsed_time(e1) for e0, e1 in ev], n

    def run_cold_l2(self, samples: int = 48):
        """One layer call at a time with the L2 flushed before it (a 256 MB buffer is overwritten):
        device time of the isolated call in microseconds, per sample."""
        torch = self.torch
        flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=self.device)
        graphs = []
        for j in range(len(self.layers)):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self.layers[j].decode(self.xs[j], out=self.outs[j])
            graphs.append(g)
        for g in graphs:
            g.replay()
        out = []
        for i in range(samples):
            flush.fill_(i & 0xFF)
            torch.cuda.synchronize(self.device)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graphs[i % len(graphs)].replay()
            e1.record()
            torch.cuda.synchronize(self.device)
            out.append(e0.elapsed_time(e1) * 1e3)
        del flush
        return out

    def run_timed(self, steps: int, warmup: int):
        """Device time of `steps` back-to-back calls in milliseconds (CUDA events on the stream)."""
        torch = self.torch
        self.prepare(steps)
        self.warm(warmup)
        torch.cuda.synchronize(self.device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        n = self.timed_region()
        e1.record()
        torch.cuda.synchronize(self.device)
        return e0.elapsed_time(e1), n

    def run_stage_profile(self, rotations: int = 8) -> dict:
        """Average device time per launch (ms) of each stage's kernel, timed back to back over
        the rotating layers inside a captured graph (workspace state comes from full calls)."""
        torch = self.torch
        L = len(self.layers)
        out = {}
        for stage in ("router_z", "gateup", "zdown", "down", "combine"):
            g, n = self.capture(L, stage=stage)
            if n == 0:
                out[stage] = 0.0
                continue
            for _ in range(2):
                g.replay()
            torch.cuda.synchronize(self.device)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(rotations):
                g.replay()
            e1.record()
            torch.cuda.synchronize(self.device)
            out[stage] = e0.elapsed_time(e1) / (rotations * n)
        return out

    def run_e2e(self, steps: int, warmup: int):
        """Host buffers in and out through moe_vqlr_decode_layer_host; ms for `steps` calls."""
        torch = self.torch
        shp = self.shp
        xh = [x.cpu().pin_memory() for x in self.xs]
        oh = [torch.empty((shp.T, shp.H), dtype=torch.bfloat16).pin_memory() for _ in self.xs]
        # every handle's first host call captures its graphs: do that for ALL layers before the clock
        # starts, then the requested warm-up
        for j in range(len(self.layers)):
            self.layers[j].decode_host(xh[j], oh[j])
        for i in range(warmup):
            j = i % len(self.layers)
            self.layers[j].decode_host(xh[j], oh[j])
        torch.cuda.synchronize(self.device)
        t0 = time.perf_counter()
        for i in range(steps):
            j = (warmup + i) % len(self.layers)
            self.layers[j].decode_host(xh[j], oh[j])
        torch.cuda.synchronize(self.device)
        ms = (time.perf_counter() - t0) * 1e3
        nbytes = shp.T * shp.H * 2
        return ms, nbytes, nbytes

    def close(self):
        for lay in self.layers:
            lay.close()
        self.g_full = self.g_rem = None
        self.layers, self.xs, self.outs = [], [], []
        self.torch.cuda.empty_cache()


def percentiles(values):
    v = sorted(values)
    def q(p):
        if len(v) == 1:
            return v[0]
        pos = p * (len(v) - 1)
        lo = int(pos)
        hi = min(lo + 1, len(v) - 1)
        return v[lo] + (v[hi] - v[lo]) * (pos - lo)
    return {"median": q(0.5), "p2_5": q(0.025), "p97_5": q(0.975), "min": v[0], "max": v[-1], "n": len(v)}


def stage_roofline(wl, workload, mode, peak, peak_kind, lookup_peak=None):
    """Roofline block of the dominant kernel of a workload: every stage's kernel is replayed alone,
    back to back over the rotating layers inside a captured graph and timed with CUDA events; the
    dominant one is the byte-carrying stage that takes longest."""
    shp = wl.shp
    stage_ms = wl.run_stage_profile()
    gu_bytes = sum(b.gateup_kernel for b in wl.bytes) / len(wl.bytes)
    dn_bytes = sum(b.down_kernel for b in wl.bytes) / len(wl.bytes)
    stage_bytes = {"gateup": gu_bytes, "down": dn_bytes}
    gu_look = sum(b.n_active * b.lookups_per_expert_gateup for b in wl.bytes) / len(wl.bytes)
    dn_look = sum(b.n_active * b.lookups_per_expert_down for b in wl.bytes) / len(wl.bytes)
    stage_lookups = {"gateup": gu_look, "down": dn_look}
    kernel_names = {"gateup": "k_gateup_mma", "down": "k_down_mma"}
    if stage_ms.get("down", 0.0) == 0.0 and stage_ms.get("zdown", 0.0) == 0.0:
        # the fused expert kernel ran as the "gateup" stage: it streams gate/up and the down indices (or the
        # dense down matrix); the low-rank factor of a compressed down projection is read by the weighted sum
        lr_down = 2 * shp.H * shp.r if mode == "full" else 0
        n_act = sum(b.n_active for b in wl.bytes) / len(wl.bytes)
        stage_bytes = {"gateup": gu_bytes + dn_bytes - n_act * lr_down}
        stage_lookups = {"gateup": gu_look + dn_look}
        kernel_names = {"gateup": "k_expert_fused"}
    dominant = max(stage_bytes, key=lambda st: stage_ms.get(st, 0.0))
    dom_ms = stage_ms[dominant]
    achieved = stage_bytes[dominant] / (dom_ms * 1e-3) / 1e9 if dom_ms > 0 else 0.0
    traffic, source = ncu_traffic_table().get((workload, mode, kernel_names[dominant]), (None, None))
    # the same kernel against the bound that does hold it: the measured rate of random 16-byte shared-memory
    # code-word reads (probe kernel, this run) x SMs x clock
    second = None
    if lookup_peak and stage_lookups.get(dominant, 0) > 0 and dom_ms > 0:
        got = stage_lookups[dominant] / (dom_ms * 1e-3) / 1e9
        second = {"bound": "shared-memory code-word reads", "achieved": got, "peak": lookup_peak, "unit": "Glookup/s",
                  "frac": got / lookup_peak, "lookups_per_launch": stage_lookups[dominant],
                  "peak_kind": "probe kernel of this run: lookups per clock per SM x SMs x SM clock under load"}
    return {"second_bound": second, "bound": "hbm", "kernel": kernel_names[dominant], "achieved": achieved, "peak": peak,
            "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
            "traffic": traffic, "traffic_source": source,
            "algorithmic_bytes_per_launch": stage_bytes[dominant], "us_per_launch": dom_ms * 1e3,
            "how": "each stage's kernel replayed back to back over the rotating layers in a captured graph, CUDA events",
            "stage_us": {k_: v * 1e3 for k_, v in stage_ms.items()}}


def measure(name, mode, steps, warmup, device, n_layers=0):
    wl = Workload(name, mode, n_layers, device)
    ms, launches = wl.run_timed(steps, warmup)
    us_layer = ms * 1e3 / steps
    res = dict(workload=name, mode=mode, T=wl.shp.T, layers=len(wl.layers), us_per_layer=us_layer,
               us_per_layer_per_token=us_layer / wl.shp.T, algorithmic_bytes=wl.mean_bytes,
               distinct_experts=wl.mean_active, gbs=wl.mean_bytes / (us_layer * 1e-6) / 1e9,
               launches=launches)
    return wl, res, ms


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_21137_b200 import accounting  # noqa: F401

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(device)

    peak, peak_kind = measured_peak()
    from paper_2609_21137_b200 import binding as _b
    ablate_flags = {"": 0, "z": _b.FLAG_ABLATE_Z_PER_EXPERT, "launch": _b.FLAG_ABLATE_PER_EXPERT_LAUNCH,
                    "both": _b.FLAG_ABLATE_Z_PER_EXPERT | _b.FLAG_ABLATE_PER_EXPERT_LAUNCH}[args.ablate]
    wl = Workload(args.workload, args.mode, args.layers, device, flags=ablate_flags | args.flags)

    # ---- the timed regions: W warm-up steps, then R regions of exactly K steps each -----------
    # A region of few steps lasts well under a millisecond and one sample of it is noisy, so the
    # region is repeated (about a second of device time, 5..400 regions, each with its own pair of
    # CUDA events) and the median region is the value, with the 2.5 / 97.5 percentiles beside it.
    wl.prepare(args.steps)
    wl.warm(args.warmup)
    barrier()
    with ClockSampler(local_rank) as clocks:
        first_ms, launches = wl.timed_regions(1)
        regions = int(max(5, min(400, 1000.0 / max(first_ms[0], 1e-3))))
        barrier()
        region_ms, launches = wl.timed_regions(regions)
        barrier()
        t_end = time.time() + 0.8      # keep the same load running so the sampler sees its clocks
        while time.time() < t_end:
            wl.g_full.replay()
            torch.cuda.synchronize(device)
    per_step_us = percentiles([m * 1e3 / args.steps for m in region_ms])
    ms = max_over_ranks(per_step_us["median"] * args.steps / 1e3, world, device)
    shp = wl.shp
    ms_per_step = ms / args.steps
    us_per_layer_token = ms_per_step * 1e3 / (shp.T * world)
    layer_gbs = wl.mean_bytes / (ms_per_step * 1e-3) / 1e9
    timing = {"regions": regions, "steps_per_region": args.steps,
              "us_per_step": {k_: v for k_, v in per_step_us.items()},
              "first_region_us_per_step": first_ms[0] * 1e3 / args.steps,
              "how": "every region is exactly `steps` layer calls between two CUDA events on the launching stream; "
                     "value = median region (max over ranks), percentiles over the regions of rank 0"}

    # ---- per-stage profile for the roofline of the dominant kernel -------------------------
    lookup_peak = None          # G lookups/s of the whole GPU at the probe's rate
    if any(b.lookups for b in wl.bytes):
        from paper_2609_21137_b200 import binding as _bind
        _rate = _bind.probe_lookup_rate(shp.K, replicated=shp.K * 128 <= 72 * 1024)
        _sms = torch.cuda.get_device_properties(device).multi_processor_count
        lookup_peak = _rate * _sms * ((clocks.summary().get("sm_mhz") or 1965.0) * 1e6) / 1e9
    roofline = stage_roofline(wl, args.workload, args.mode, peak, peak_kind, lookup_peak)
    roofline["layer"] = {"algorithmic_bytes": wl.mean_bytes, "gbs": layer_gbs, "frac_of_measured": layer_gbs / peak,
                         "frac_of_nominal_8TBs": layer_gbs / NOMINAL_HBM_GBS}

    # ---- one isolated call with a cold L2 ---------------------------------------------------
    cold = None
    if rank == 0 and not args.no_extras:
        cs = percentiles(wl.run_cold_l2())
        cold = {"us_per_layer": cs, "how": "a 256 MB buffer is overwritten before every call (L2 is 126 MB); one call "
                                           "(its kernels captured as one graph) between two CUDA events; 48 samples over the layers"}

    # ---- second bound: shared-memory lookup rate (measured live by a probe kernel) ----------
    lookup_bound = None
    mean_lookups = sum(b.lookups for b in wl.bytes) / len(wl.bytes)
    if mean_lookups > 0:
        from paper_2609_21137_b200 import binding
        n_books = 1
        repl = shp.K * 128 * n_books <= 72 * 1024
        rate = binding.probe_lookup_rate(shp.K, replicated=repl)
        sm_mhz = (clocks.summary().get("sm_mhz") or 1965.0)
        sms = torch.cuda.get_device_properties(device).multi_processor_count
        t_us = mean_lookups / (rate * sms * sm_mhz)          # lookups / (lookups per us)
        lookup_bound = {"what": "random 16-byte shared-memory code-word reads; the compressed projections cannot run faster than this",
                        "lookups_per_layer": mean_lookups, "measured_lookups_per_clk_per_sm": rate,
                        "replicated_codebook": bool(repl), "sms": sms, "sm_mhz": sm_mhz,
                        "us_per_layer_at_that_rate": t_us, "frac_of_lookup_bound": t_us / (ms_per_step * 1e3),
                        "hbm_us_per_layer_at_measured_peak": wl.mean_bytes / peak / 1e3}

    # ---- end to end through host buffers --------------------------------------------------
    e2e_steps = min(args.steps, 400)
    e2e_ms, h2d, d2h = wl.run_e2e(e2e_steps, max(3, min(args.warmup, 20)))
    e2e_ms = max_over_ranks(e2e_ms, world, device)
    e2e = {"value": e2e_ms * 1e3 / e2e_steps / (shp.T * world), "unit": "us", "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": e2e_steps,
           "how": "moe_vqlr_decode_layer_host with pinned host buffers, one call after the other, wall clock around "
                  "the loop; every handle made one call before the clock started (its first call captures graphs)"}
    n_layers = len(wl.layers)
    specialized = {"layers_with_kernels_compiled_for_their_shape": sum(1 for l in wl.layers if l.specialized()),
                   "of": len(wl.layers),
                   "note": next((l.specialization_note() for l in wl.layers if not l.specialized()), "")}
    wl.close()

    extras = []
    roofline_b16 = None
    if rank == 0 and world == 1 and not args.no_extras:
        todo = [("qwen3", "paper"), ("qwen3", "dense"), ("qwen3_b16", "full"), ("qwen3_b16", "paper"),
                ("qwen3_b16", "dense"), ("qwen3_deployed", "paper"), ("qwen3_deployed_b16", "paper")]
        todo = [t_ for t_ in todo if t_ != (args.workload, args.mode)]
        for name, mode in todo:
            try:
                w2, r2, _ = measure(name, mode, 960, 96, device)
                r2["frac_of_measured"] = r2["gbs"] / peak
                r2["frac_of_nominal_8TBs"] = r2["gbs"] / NOMINAL_HBM_GBS
                if (name, mode) == ("qwen3_b16", "full"):      # the metric names batch 1 AND batch 16
                    roofline_b16 = stage_roofline(w2, name, mode, peak, peak_kind, lookup_peak)
                    roofline_b16["layer"] = {"us_per_layer": r2["us_per_layer"], "algorithmic_bytes": r2["algorithmic_bytes"],
                                             "gbs": r2["gbs"], "frac_of_measured": r2["frac_of_measured"],
                                             "distinct_experts": r2["distinct_experts"]}
                w2.close()
                extras.append(r2)
            except Exception as exc:   # an extra must never take the headline down
                extras.append({"workload": name, "mode": mode, "error": str(exc)[:200]})

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        r = oracle_timing(args.workload, args.mode, budget_s=20.0, max_steps=64)
        cpu = {"value": r["us_per_layer_per_token"], "unit": "us", "cores": r["cores"], "kind": "oracle",
               "sample": f"{r['calls']} full fp64 oracle layer calls of the same shape (numpy-seeded layer, T={r['T']})"}

    if rank == 0:
        line = {"metric": "us_per_moe_layer_per_token", "value": us_per_layer_token, "unit": "us",
                "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
                "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic",
                "config": {"workload": f"{args.workload} T={shp.T} mode={args.mode}"
                                       + (f" ablate={args.ablate}" if args.ablate else "")
                                       + (f" flags={args.flags}" if args.flags else ""),
                           "shape": f"H={shp.H} I={shp.I} E={shp.E} k={shp.k} S={shp.S} K={shp.K} r={shp.r}",
                           "distinct_layers": n_layers,
                           "l2": f"rotation over {n_layers} distinct layers touches "
                                 f"{n_layers * wl.mean_bytes / 1e6:.0f} MB per pass, larger than the 126 MB L2",
                           "launch": "each rotation over the layers is one captured CUDA graph; kernels of a call are linked by programmatic dependent launch",
                           "specialized": specialized,
                           "parallelism": "replicas only" if world > 1 else "single GPU"},
                "tokens_per_s_per_layer": shp.T * world / (ms_per_step * 1e-3),
                "hbm_gbs": layer_gbs, "hbm_frac_of_measured": layer_gbs / peak,
                "hbm_frac_of_nominal_8TBs": layer_gbs / NOMINAL_HBM_GBS,
                "algorithmic_bytes_per_layer": wl.mean_bytes, "distinct_experts_per_layer": wl.mean_active,
                "gpu_launches": launches, "clocks": clocks.summary(), "timing": timing, "roofline": roofline,
                "roofline_b16": roofline_b16, "cold_l2": cold, "e2e": e2e,
                "lookup_bound": lookup_bound, "cpu_baseline": cpu, "extras": extras}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
