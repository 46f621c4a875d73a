#!/usr/bin/env python
"""Benchmark of the DynamicKV compression pass: prefix tokens/s through all layers.

One step = one whole pass of Algorithm 1 (score, per-head top-k, gather for every layer; rebudget
and shrink every m layers) over one synthetic prompt batch, through the C ABI of libdkv.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  Under torchrun each rank runs an independent replica of the whole
workload on its own GPU (the path has no cross-GPU exchange); the time is the max over ranks.
`--impl reference` times the CPU oracle on a bounded sample of the same workload instead.
"""
from __future__ import annotations

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

from paper_2412_14838_b200 import synth  # noqa: E402

METRIC = "prefix tokens/s through 32-layer KV compression at 32K ctx; HBM GB/s vs 8 TB/s"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "mistral32k"
NOMINAL_HBM_GBS = 8000.0

# DRAM traffic of one full scoring launch (dram__bytes_read.sum + dram__bytes_write.sum): sweep 2 of four layers
# followed by sweep 1 of the next four, taken with ncu on the 8-layer cut of the mistral32k shape (same per-layer
# shape and group size, so the figure needs no scaling; see profiles/score_tc_kernel_mistral32k_8layers.md).
# "live" is a single-pass capture without ncu's cache flush, i.e. with whatever the previous launch left in L2, as
# in a real pass; "cold" is the --set full capture, where every replay starts from flushed caches.  Both hold for
# the kernel source they were measured on, for that per-layer shape and for four-layer groups only: any other
# source hash, shape or grouping reports null.
NCU_TRAFFIC = {
    "kernel_sha256": "303acb3e0fa3bf64ba7b5cb1069bb408c1cc9088dab894f6a69887c302ea26de",
    "shape": (8, 128, 1, 32768, 32),          # Hkv, D, Bt, S, ws
    "layers_per_launch": 4,
    "live_bytes_per_launch": 478_000_384 + 28_855_296,
    "cold_bytes_per_launch": 540_321_280 + 6_633_728,
}


def ncu_traffic(w, score_launches=None):
    import hashlib
    src = os.path.join(ROOT, "paper_2412_14838_b200", "csrc", "score_tc.cuh")
    try:
        with open(src, "rb") as f:
            sha = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        return None
    if sha != NCU_TRAFFIC["kernel_sha256"] or (w.Hkv, w.D, w.Bt, w.S, w.ws) != NCU_TRAFFIC["shape"]:
        return None
    g = NCU_TRAFFIC["layers_per_launch"]
    if w.L % g or score_launches is None or round(score_launches) != w.L // g + 1:
        return None                             # the pass was not run in full four-layer groups
    return NCU_TRAFFIC
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return json.load(f), "measured"
    except Exception:
        return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


# ------------------------------------------------------------------------------------ CPU oracle leg
def oracle_sample(w, layers: int, inputs=None):
    """Time the oracle, as it stands, on the first `layers` layers of the workload.

    Returns (seconds, threads used).  Input generation is outside the timed part."""
    from oracle import dynamickv as O
    if inputs is None:
        inputs = [synth.layer_inputs(w, l) for l in range(layers)]

    def layer_fn(l):
        t = inputs[l]
        return {"q": synth.bf16_bits_to_f64(t["q"]), "k": synth.bf16_bits_to_f64(t["k"]),
                "k_rows": t["k"], "v_rows": t["v"]}

    t0 = time.perf_counter()
    O.run_prefill_pass(layer_fn, layers, ws=w.ws, pool=w.pool, N=w.N, Bl=w.Bl, m=w.m)
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    return dt, int(cores)


def cpu_baseline(w, layers: int):
    dt, cores = oracle_sample(w, layers)
    if dt < 5.0 and layers < w.L:
        # a quick host: take more update blocks, aiming at about 10 s of oracle time
        blocks = int(min(w.L // layers, max(2, round(10.0 / max(dt, 1e-3)))))
        layers = layers * blocks
        dt, cores = oracle_sample(w, layers)
    value = w.Bt * w.S / (dt * w.L / layers)
    return {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"layers 0..{layers - 1} of {w.L} (whole update blocks) of workload {w.name}: {dt:.2f} s, "
                      f"scaled by {w.L}/{layers} to a whole pass"}


def run_reference(args, w):
    # one update block per step when few steps are asked for, one layer per step otherwise,
    # so that the whole run stays within a few minutes
    layers = min(w.m, w.L) if args.steps <= 5 else 1
    inputs = [synth.layer_inputs(w, l) for l in range(layers)]
    cores = 1
    for _ in range(min(args.warmup, 1)):
        oracle_sample(w, layers, inputs)
    times = []
    for _ in range(args.steps):
        dt, cores = oracle_sample(w, layers, inputs)
        times.append(dt)
    measured = float(np.mean(times))                 # seconds one step really took
    per_pass = measured * w.L / layers               # the same rate over all L layers
    value = w.Bt * w.S / per_pass
    base = {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"each step = layers 0..{layers - 1} of {w.L} of workload {w.name} ({measured:.2f} s measured, "
                      f"ms_per_step is that time); value = tokens of a whole pass / (step time x {w.L}/{layers})"}
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": measured * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w), "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def workload_config(w):
    return {"workload": w.name, "layers": w.L, "q_heads": w.Hq, "kv_heads": w.Hkv, "head_dim": w.D, "batch": w.Bt,
            "prefix_len": w.S, "window": w.ws, "pool": w.pool, "avg_budget": w.N, "layer_max": w.Bl,
            "update_interval": w.m, "recipe": w.recipe, "seed": synth.BASE_SEED,
            "l2": ("inputs (K+V of all layers, %.2f GB) exceed L2; no flush needed" if 2 * w.L * w.k_bytes_per_layer() > 256e6
                   else "inputs (K+V of all layers, %.2f GB) fit L2 and are NOT flushed between steps: a parity-size "
                        "workload, not a bench line") % (2 * w.L * w.k_bytes_per_layer() / 1e9)}


# ------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    BAD = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown"}
    NOTE = {0x4: "sw_power_cap"}

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz, self.err = [], set(), None, None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            p = torch.cuda.get_device_properties(device_index)
            bus = "%08x:%02x:%02x.0" % (p.pci_domain_id, p.pci_bus_id, p.pci_device_id)
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByPciBusId(bus.encode())
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception as e:      # NVML missing: report that instead of a number
            self.err = repr(e)

    def _loop(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in {**self.BAD, **self.NOTE}.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception as e:
                self.err = repr(e)
                return
            time.sleep(0.005)

    def __enter__(self):
        if self.err is None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if self.err is not None and not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "error": self.err}
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------ replicas
def max_over_ranks(x: float, device: str = "cuda") -> float:
    """The slowest rank's time: every rank runs an independent replica, the job ends with the last one."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_replica: int, world: int, seconds_per_step: float) -> float:
    """Aggregate tokens/s of `world` independent replicas that all took `seconds_per_step` (the max)."""
    return world * tokens_per_replica / seconds_per_step


# ------------------------------------------------------------------------------------ GPU leg
def run_gpu(args, w):
    import torch
    import torch.distributed as dist
    from paper_2412_14838_b200 import binding as B
    from paper_2412_14838_b200 import build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    B.load()

    # inputs: the same seeded bits on every rank (independent replicas of one workload)
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda()
    q, k, v = [], [], []
    want_e2e = not args.no_e2e
    hq, hk, hv = [], [], []
    for l in range(w.L):
        t = synth.layer_inputs(w, l)
        q.append(to_dev(t["q"])); k.append(to_dev(t["k"])); v.append(to_dev(t["v"]))
        if want_e2e:
            for dst, name in ((hq, "q"), (hk, "k"), (hv, "v")):
                dst.append(torch.from_numpy(t[name].view(np.int16)).pin_memory())
    shape = (w.Bt, w.Hkv, w.Blc + w.ws, w.D)
    kb = [torch.zeros(shape, dtype=torch.int16, device="cuda") for _ in range(w.L)]
    vb = [torch.zeros(shape, dtype=torch.int16, device="cuda") for _ in range(w.L)]
    ctx = B.dkv_create(B.config_of(w))
    stream = torch.cuda.current_stream()

    def one_pass():
        B.dkv_run_prefill_pass(ctx, q, k, v, kb, vb, stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_pass()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # a short burst first (the clocks have not yet met the power cap), reported beside the sustained figure
    burst_steps = min(20, args.steps)
    ev0.record(stream)
    for _ in range(burst_steps):
        one_pass()
    ev1.record(stream)
    barrier()
    burst_ms = max_over_ranks(ev0.elapsed_time(ev1)) / burst_steps
    launches0 = B.dkv_launch_count(ctx)
    with ClockSampler(local) as clocks:
        ev0.record(stream)
        for _ in range(args.steps):
            one_pass()
        ev1.record(stream)
        barrier()
    ms = ev0.elapsed_time(ev1)
    launches = B.dkv_launch_count(ctx) - launches0
    ms = max_over_ranks(ms)
    ms_per_step = ms / args.steps
    tokens = w.Bt * w.S
    value = whole_job_value(tokens, world, ms_per_step * 1e-3)

    # per-kernel durations: the same steps again, each step's launches bracketed by CUDA events
    prof_steps = min(args.steps, 20)
    B.dkv_profile(ctx, True)
    for _ in range(prof_steps):
        one_pass()
    prof = B.dkv_profile_read(ctx)
    B.dkv_profile(ctx, False)
    peaks, peak_kind = measured_peaks()
    peak = float(peaks["hbm_gbs"])
    # the scoring kernel: every launch sweeps a group of layers (sweep 2 of one group, sweep 1 of the next), so
    # the algorithmic bytes of a launch are the pass's K bytes over the launches of a pass
    score_ms = (prof["score_stats"][0] + prof["score_emit"][0]) / prof_steps
    score_launches = (prof["score_stats"][1] + prof["score_emit"][1]) / prof_steps
    score_launch_ms = score_ms / score_launches
    k_bytes = w.k_bytes_per_layer()
    launch_bytes = k_bytes * w.L / score_launches
    achieved = launch_bytes / (score_launch_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "window scoring (softmax statistics sweep + emit sweep + pooling)",
                "achieved": achieved, "peak": peak, "peak_source": f"MEASURED_PEAKS.json hbm_gbs ({peak_kind})",
                "unit": "GB/s", "frac": achieved / peak,
                "algorithmic_bytes_per_launch": launch_bytes, "avg_launch_ms": score_launch_ms,
                "launches_per_pass": score_launches, "scoring_ms_per_layer": score_ms / w.L,
                "traffic": (ncu_traffic(w, score_launches) or {}).get("live_bytes_per_launch"),
                "traffic_cold_cache": (ncu_traffic(w, score_launches) or {}).get("cold_bytes_per_launch"),
                "traffic_note": "DRAM bytes of a full launch (sweep 2 of 4 layers + sweep 1 of the next 4); the first "
                                "and last launch of a pass run one sweep only, so avg launches carry 8/9 of that",
                "whole_pass": {"algorithmic_bytes": w.algorithmic_bytes(),
                               "achieved_gbs": w.algorithmic_bytes() / (ms_per_step * 1e-3) / 1e9,
                               "frac_of_measured_peak": w.algorithmic_bytes() / (ms_per_step * 1e-3) / 1e9 / peak,
                               "frac_of_8TBs": w.algorithmic_bytes() / (ms_per_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
                "step_ms_per_pass": {n: round(t / prof_steps, 4) for n, (t, _) in prof.items() if t > 0}}

    # the one-sweep scoring entry point (normalisers given, as a prefill attention kernel would hand them over):
    # reported beside the headline, never part of it.  The normalisers are prepared outside the timed region.
    one_sweep = None
    if not args.no_one_sweep:
        lse = []
        hidden = (torch.arange(w.S, device="cuda")[None, :] > (w.P + torch.arange(w.ws, device="cuda"))[:, None])
        for l in range(w.L):
            qf = q[l].view(torch.bfloat16).float().view(w.Bt, w.Hkv, w.G * w.ws, w.D)
            kf = k[l].view(torch.bfloat16).float().view(w.Bt, w.Hkv, w.S, w.D)
            logits = torch.matmul(qf, kf.transpose(-1, -2)).view(w.Bt, w.Hq, w.ws, w.S) / float(np.sqrt(w.D))
            lse.append(torch.logsumexp(logits.masked_fill(hidden, float("-inf")), dim=-1).contiguous())
            del logits
        B.dkv_reset(ctx, stream)
        for l in range(w.L):
            B.dkv_score_lse(ctx, l, q[l], k[l], lse[l], None, stream)
        barrier()
        ev0.record(stream)
        for _ in range(prof_steps):
            for l in range(w.L):
                B.dkv_score_lse(ctx, l, q[l], k[l], lse[l], None, stream)
        ev1.record(stream)
        barrier()
        one_ms = max_over_ranks(ev0.elapsed_time(ev1)) / (prof_steps * w.L)
        one_sweep = {"api": "dkv_score_lse", "avg_launch_ms": one_ms, "algorithmic_bytes_per_launch": k_bytes,
                     "achieved": k_bytes / (one_ms * 1e-3) / 1e9, "unit": "GB/s",
                     "frac": k_bytes / (one_ms * 1e-3) / 1e9 / peak}

    # the pass scored in one sweep (dkv_run_prefill_pass_lse), normalisers prepared outside the timed region;
    # reported beside the headline, never part of it
    one_sweep_pass = None
    if one_sweep is not None:
        def lse_pass():
            B.dkv_run_prefill_pass_lse(ctx, q, k, v, lse, kb, vb, stream)
        for _ in range(3):
            lse_pass()
        barrier()
        ev0.record(stream)
        for _ in range(prof_steps):
            lse_pass()
        ev1.record(stream)
        barrier()
        lp_ms = max_over_ranks(ev0.elapsed_time(ev1)) / prof_steps
        one_sweep_pass = {"api": "dkv_run_prefill_pass_lse", "ms_per_step": lp_ms, "steps": prof_steps,
                          "value": whole_job_value(tokens, world, lp_ms * 1e-3), "unit": UNIT,
                          "whole_pass_frac_of_measured_peak": w.algorithmic_bytes() / (lp_ms * 1e-3) / 1e9 / peak}
        del lse

    # decoding over the compressed cache the pass leaves behind: one new query per sample, all layers in one
    # launch, then layer by layer; algorithmic bytes = the valid K and V rows, once
    one_pass()
    barrier()
    counts_now = np.zeros((w.Bt, w.L), dtype=np.int32)
    B.dkv_get_counts(ctx, counts_now)
    dq = [to_dev(synth.decode_queries(w, l)) for l in range(w.L)]
    dout = [torch.zeros((w.Bt, w.Hq, 1, w.D), dtype=torch.float32, device="cuda") for _ in range(w.L)]
    dec_bytes = int((counts_now.astype(np.int64) + w.ws).sum()) * w.Hkv * w.D * 2 * 2
    dec = {}
    for label, per_call in (("all_layers_one_launch", w.L), ("layer_by_layer", 1)):
        def dec_step():
            for l0 in range(0, w.L, per_call):
                B.dkv_decode_attend(ctx, l0, per_call, 1, dq[l0:l0 + per_call], kb[l0:l0 + per_call], vb[l0:l0 + per_call],
                                    dout[l0:l0 + per_call], stream)
        for _ in range(3):
            dec_step()
        barrier()
        ev0.record(stream)
        for _ in range(prof_steps):
            dec_step()
        ev1.record(stream)
        barrier()
        d_ms = max_over_ranks(ev0.elapsed_time(ev1)) / prof_steps
        dec[label] = {"ms": d_ms, "achieved": dec_bytes / (d_ms * 1e-3) / 1e9, "frac": dec_bytes / (d_ms * 1e-3) / 1e9 / peak}
    decode = {"api": "dkv_decode_attend", "queries_per_sample": 1, "algorithmic_bytes": dec_bytes, "unit": "GB/s",
              "bound": "hbm", "peak": peak, "note": "the buffers of a pass fit L2, so repeated calls are served from it",
              **dec}

    # end to end: host buffers in, compacted buffers + counts out, copies inside the timed region
    e2e = None
    if want_e2e:
        okb = [torch.zeros(shape, dtype=torch.int16).pin_memory() for _ in range(w.L)]
        ovb = [torch.zeros(shape, dtype=torch.int16).pin_memory() for _ in range(w.L)]
        counts = np.zeros((w.Bt, w.L), dtype=np.int32)
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        B.dkv_run_prefill_pass_host(ctx, hq, hk, hv, okb, ovb, counts)      # warm-up (allocates staging)
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            B.dkv_run_prefill_pass_host(ctx, hq, hk, hv, okb, ovb, counts)
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) / e2e_steps
        dt = max_over_ranks(dt)
        # in: q and k in full and, of v, the rows the gather reads in place from the pinned buffers (count + ws per
        # head at gather time); out: the counts and the valid rows of every head's K and V buffers.  The library
        # counts them from the copies it issues and the rows it gathers; the full tensors are given beside them.
        h2d, d2h = B.dkv_host_pass_bytes(ctx)
        h2d_full = sum(t.numel() * 2 for t in hq) + sum(t.numel() * 2 for t in hk) + sum(t.numel() * 2 for t in hv)
        assert d2h == int((counts.astype(np.int64) + w.ws).sum()) * w.Hkv * w.D * 2 * 2 + counts.nbytes
        e2e = {"value": whole_job_value(tokens, world, dt), "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
               "ms_per_step": dt * 1e3, "steps": e2e_steps, "api": "dkv_run_prefill_pass_host (pinned host buffers)",
               "host_input_bytes": int(h2d_full),
               "note": ("of V only the gathered rows cross the bus (read in place from pinned memory by the gather kernel)"
                        if h2d < h2d_full else "q, k and v copied in full")}

    B.dkv_destroy(ctx)
    out = None
    if rank == 0:
        base = None
        if world == 1 and not args.no_cpu_baseline:
            base = cpu_baseline(w, min(w.m, w.L))
        out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "bf16 in, f32 accumulate", "data": "synthetic",
               "config": workload_config(w), "parallelism": f"{world} independent replica(s)",
               "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
               "burst": {"steps": burst_steps, "ms_per_step": burst_ms,
                         "value": whole_job_value(tokens, world, burst_ms * 1e-3),
                         "note": "the first timed steps, before the clocks meet the power cap; `value` is the "
                                 "sustained figure over all `steps`"},
               "one_sweep_scoring": one_sweep, "one_sweep_pass": one_sweep_pass, "decode_attention": decode,
               "cpu_baseline": base}
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="dkv", choices=["dkv", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--layers", type=int, default=0, help="profiling aid: keep only the first N layers of the workload")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-one-sweep", action="store_true", help="skip the timing of dkv_score_lse")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    if args.layers:
        w = w.with_(name=f"{w.name}[:{args.layers}]", L=args.layers)
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) != 0:
            return 0
        print(json.dumps(run_reference(args, w)))
        return 0
    if args.warmup < 3:
        args.warmup = 3
    out = run_gpu(args, w)
    if out is not None:
        print(json.dumps(out))
    return 0


if __name__ == "__main__":
    sys.exit(main())
