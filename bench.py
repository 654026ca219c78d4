#!/usr/bin/env python
"""Benchmark of the MonarchAttention forward pass (one JSON line on stdout).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C5] [--impl ours|reference]

A step is one whole forward call (all T rounds of Eq. 7-10 and the Monarch multiply of Eq. 4) on
one batch of the named configuration.  `value` is forward tokens/s (batch*N tokens per call) with
inputs resident in HBM; `e2e` is the same metric through the host-buffer entry point with the
host<->device copies inside the timed region.  Under torchrun every rank runs the same
configuration on its own batch (heads are independent: no collective on the data path) and the
time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2505_18698_b200 import workloads as wl  # noqa: E402

METRIC = "MonarchAttention fwd tokens/s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = f"/tmp/ma_clocks_{os.getpid()}.csv"

    def start(self):
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100", "-i", str(self.gpu)], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "samples": len(sm),
                "power_w_max": max(power), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- reference arm
def _oracle_head(args):
    """One whole head through the fp64 oracle (runs in a worker process, one BLAS thread)."""
    from oracle import monarch_oracle
    Q, K, V, b, T = args
    monarch_oracle.monarch_attention_head(Q, K, V, b, T)
    return 1


def _one_blas_thread():
    """One BLAS thread per worker process: the host cores are the workers."""
    try:
        from threadpoolctl import threadpool_limits
        threadpool_limits(1)
    except Exception:
        pass


def host_cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return max(1, os.cpu_count() or 1)


def oracle_sample(w: wl.Workload, budget_s: float):
    """Times the fp64 oracle, as it stands, on whole heads of the workload, one head per host core
    at a time (the (batch, head) units are independent), until the budget is used; returns
    (tokens_per_s, heads_done, seconds, cores).  The rate over the sample is extrapolated to the
    workload's token count: the sample cycles through the workload's own heads."""
    import multiprocessing as mp
    cores = host_cores()
    n_heads = min(w.heads, max(cores, 4))
    Q, K, V = wl.make_qkv(1, n_heads, w.N, w.d, w.dtype, w.rank, w.s, w.seed)
    done = 0
    with mp.get_context("fork").Pool(cores, initializer=_one_blas_thread) as pool:
        pool.map(_oracle_head, [(Q[0, 0, :w.b * 2], K[0, 0, :w.b * 2], V[0, 0, :w.b * 2], w.b, 1)] * cores)
        t0 = time.perf_counter()
        while True:
            jobs = [(Q[0, (done + i) % n_heads], K[0, (done + i) % n_heads], V[0, (done + i) % n_heads],
                     w.b, w.T) for i in range(cores)]
            done += sum(pool.map(_oracle_head, jobs))
            el = time.perf_counter() - t0
            if el >= budget_s:
                break
    tokens = w.tokens * done / w.BH
    return tokens / el, done, el, cores


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warm = max(1, args.steps), max(0, args.warmup)
    budget = min(15.0, 120.0 / (steps + warm))
    vals, heads, cores = [], 0, 1
    for i in range(warm + steps):
        v, heads, _, cores = oracle_sample(w, budget)
        if i >= warm:
            vals.append(v)
    value = float(np.mean(vals))
    sample = (f"{heads} head evaluations of {w.name} (its {w.BH} (batch, head) units in turn) per step on "
              f"{cores} host cores, fp64 numpy oracle; tokens/s extrapolated from the sample")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": 1e3 * w.tokens / value,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, 1),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(w, world, strong=False):
    return {"workload": f"{w.name}: batch={w.batch} heads={w.heads} N={w.N} d={w.d} b={w.b} "
                        f"T={w.T} {w.dtype}, rank-{w.rank} component x{w.s}, seed {w.seed}",
            "per_gpu_batch": w.batch if not strong else None,
            "global_batch": w.batch * (1 if strong else world), "seq_len": w.N,
            "parallelism": (f"the configuration's {w.BH} (batch,head) units split over {world} rank(s), "
                            "no collective" if strong else
                            f"every rank runs the configuration on its own batch, {world} rank(s), "
                            "no collective"),
            "l2": "3 rotating input/output sets (>= 3x the call's footprint) so no step re-reads "
                  "data left in the 126 MB L2 by the previous one"}


# ----------------------------------------------------------------------------- ours
def time_config(w, steps, warmup, torch, binding, n_sets=3, dist=None, units=None, path=None):
    """Device-timed steps of workload w (or, with `units` = (lo, hi), of that slice of its
    (batch, head) units: strong scaling).  `path`: None = the library's own choice through
    monarch_attn_fwd; a path constant = that kernel through monarch_attn_fwd_ex with a workspace
    allocated once.  Returns dict with ms_per_step etc."""
    sets = []
    for r in range(n_sets):
        seed = w.seed + 1000 * r + 17 * int(os.environ.get("RANK", "0"))
        if units is None:
            Q, K, V = wl.make_qkv(w.batch, w.heads, w.N, w.d, w.dtype, w.rank, w.s, seed)
        else:      # this rank's units as one batch entry with (hi - lo) heads
            Q, K, V = wl.make_qkv(1, units[1] - units[0], w.N, w.d, w.dtype, w.rank, w.s, seed)
        Qd, Kd, Vd = (binding.to_device(x, w.dtype) for x in (Q, K, V))
        sets.append((Qd, Kd, Vd, torch.empty_like(Qd)))
    if path is None:
        def call(s):
            binding.monarch_attn_fwd(s[0], s[1], s[2], w.b, w.T, Y=s[3])
        status_of = None
    else:
        q0 = sets[0][0]
        need = binding.monarch_attn_workspace_bytes(q0.shape[0], q0.shape[1], w.N, w.d, w.b, w.T, q0.dtype, path)
        if need == 0:
            raise SystemExit(f"--path: that kernel does not take workload {w.name}")
        ws = torch.zeros(need, dtype=torch.uint8, device=q0.device)
        status_of = ws

        def call(s):
            binding.monarch_attn_fwd_ex(s[0], s[1], s[2], w.b, w.T, path=path, workspace=ws, Y=s[3])
    call(sets[0])                                   # sizes the library's workspace
    torch.cuda.synchronize()
    launches = binding.monarch_attn_last_launch_count()
    for i in range(warmup):
        call(sets[i % n_sets])
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
        torch.cuda.synchronize()
    # the K timed steps: one event before the first, one after the last (an event record between
    # steps costs 2.5 - 4.5 us of device time per step and keeps consecutive launches from
    # overlapping their tails; measured)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        call(sets[(warmup + i) % n_sets])
    e1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    total_ms = e0.elapsed_time(e1)
    # per-step statistics from a second, shorter loop with an event after every step (each step of
    # this loop carries that event's overhead)
    n_stat = min(steps, 50)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_stat + 1)]
    evs[0].record()
    for i in range(n_stat):
        call(sets[i % n_sets])
        evs[i + 1].record()
    torch.cuda.synchronize()
    per = [evs[i].elapsed_time(evs[i + 1]) for i in range(n_stat)]
    assert binding.monarch_attn_device_status(status_of) == 0
    # host time of one call with an idle stream (argument checks, cached tensor maps, launch)
    host = []
    for i in range(20):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        call(sets[i % n_sets])
        host.append((time.perf_counter() - t0) * 1e6)
    torch.cuda.synchronize()
    host_us = statistics.median(host)
    # Launch-bound sizes (the fastest step of the loop is not much longer than the host needs to
    # issue a call): the same calls captured in a CUDA graph and replayed, so that the number is the
    # device's, not the host's.  (The fastest step, not the mean: the mean of a host-bound loop
    # moves with whatever else the host does.)
    loop_ms = total_ms / steps
    timing = "cuda events around K calls issued from Python"
    if min(per) < 0.025:
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for i in range(steps):
                        call(sets[i % n_sets])
            torch.cuda.synchronize()
            graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(5):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            graph_ms = e0.elapsed_time(e1) / (5 * steps)
            if graph_ms < loop_ms:
                total_ms, timing = graph_ms * steps, (f"cuda events around 5 replays of a CUDA graph of {steps} "
                                                      f"captured calls (the Python call loop is host-bound at "
                                                      f"{loop_ms * 1e3:.1f} us per call)")
        except Exception:
            pass
    return {"total_ms": total_ms, "ms_per_step": total_ms / steps, "min_ms": min(per),
            "median_ms": statistics.median(per), "launches_per_step": launches, "sets": sets,
            "host_us_per_call": host_us, "loop_ms_per_step": loop_ms, "timing": timing}


def time_e2e(w, steps, warmup, torch, binding, dist=None):
    Q, K, V = wl.make_workload_inputs(w)
    td = binding.torch_dtype(w.dtype)
    Qh, Kh, Vh = (torch.from_numpy(x).to(td).pin_memory() for x in (Q, K, V))
    Yh = torch.empty_like(Qh).pin_memory()
    for _ in range(max(warmup, 1)):
        binding.monarch_attn_fwd_host(Qh, Kh, Vh, Yh, w.b, w.T)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        binding.monarch_attn_fwd_host(Qh, Kh, Vh, Yh, w.b, w.T)
    e1.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    nbytes = Qh.numel() * Qh.element_size()
    return e0.elapsed_time(e1) / steps, 3 * nbytes, nbytes


def ncu_traffic_bytes(name):
    """DRAM bytes of ONE step of workload `name` (dram__bytes_read.sum + dram__bytes_write.sum of its
    kernel launches, from the ncu captures summarised under profiles/): read from
    profiles/traffic.json, which is written when a capture is summarised; None if not captured."""
    try:
        d = json.load(open(os.path.join(ROOT, "profiles", "traffic.json")))
        e = d["workloads"].get(name)
        return None if e is None else float(e["dram_read_bytes"]) + float(e["dram_write_bytes"])
    except Exception:
        return None


def roofline(w, ms, peaks, which):
    t_hbm = w.algorithmic_bytes() / (peaks["hbm_gbs"] * 1e9)
    t_tc = w.algorithmic_flops() / (peaks["bf16_tflops_sustained"] * 1e12) if w.dtype != "f32" else 0.0
    if t_tc > t_hbm:
        ach = w.algorithmic_flops() / (ms * 1e-3) / 1e12
        return {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"],
                "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops_sustained"],
                "traffic": ncu_traffic_bytes(w.name), "of": which + " (sustained)",
                "scope": "one launch = one step (the tensor path is a single persistent kernel)"}
    ach = w.algorithmic_bytes() / (ms * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": ach / peaks["hbm_gbs"], "traffic": ncu_traffic_bytes(w.name), "of": which,
            "scope": "one step (one launch on the tcgen05 and fused paths, 2T on the tile and generic paths)"}


def sdpa_ms(w, torch, sets, iters=5):
    import torch.nn.functional as F
    if w.dtype == "f32":
        return None
    q, k, v, _ = sets[0]
    try:
        for _ in range(2):
            F.scaled_dot_product_attention(q, k, v)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            s = sets[i % len(sets)]
            F.scaled_dot_product_attention(s[0], s[1], s[2])
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters
    except Exception:
        return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="C5", choices=sorted(wl.WORKLOADS) + sorted(wl.EXTRA_WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="weak: every rank runs the whole configuration on its own batch; strong: the "
                         "configuration's (batch, head) units are split over the ranks")
    ap.add_argument("--path", default="auto",
                    choices=["auto", "generic", "tensor", "tensor_tmem", "tensor_basic", "fused_f32",
                             "fused_jsplit", "fused_small", "tile_mma"],
                    help="auto: the kernel the library picks (monarch_attn_fwd); else that kernel by name "
                         "through monarch_attn_fwd_ex (for profiling one kernel against another)")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the other configurations, SDPA context and the CPU baseline")
    args = ap.parse_args()
    w = {**wl.WORKLOADS, **wl.EXTRA_WORKLOADS}[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import __graft_entry__ as entry
    entry.build()
    from paper_2505_18698_b200 import binding
    binding.load_library()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")

    from paper_2505_18698_b200 import distributed as D
    rank, local, world = D.env_world()
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        D.init("nccl")
    steps, warmup = max(1, args.steps), max(3, args.warmup)
    peaks, which = load_peaks()

    strong = args.scaling == "strong" and world > 1
    units = wl.shard_units(w.BH, world, rank) if strong else None
    if strong and units[1] == units[0]:
        raise SystemExit(f"--scaling strong: {w.name} has only {w.BH} units for {world} ranks")
    sampler = ClockSampler(local)
    sampler.start()
    path = None if args.path == "auto" else getattr(binding, "MA_PATH_" + args.path.upper())
    res = time_config(w, steps, warmup, torch, binding, dist=dist, units=units, path=path)
    clocks = sampler.stop()
    ms = D.max_over_ranks(res["total_ms"] / steps, device="cuda")
    e2e_ms, h2d, d2h = time_e2e(w, max(3, min(steps, 20)), 3, torch, binding, dist)
    e2e_ms = D.max_over_ranks(e2e_ms, device="cuda")
    # weak: every rank processed the whole configuration; strong: the ranks shared one
    job_tokens = w.tokens if strong else world * w.tokens

    line = {
        "metric": METRIC, "value": job_tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "strong" if strong else "weak", "vs_baseline": None, "dtype": w.dtype,
        "data": "synthetic", "config": workload_config(w, world, strong),
        "clocks": clocks,
        "e2e": {"value": world * w.tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "note": "every rank moves the whole configuration through its own host buffers"},
        "gpu_launches": res["launches_per_step"] * steps,
        "roofline": roofline(w, ms, peaks, which) if not strong else None,
        "min_ms": res["min_ms"], "median_ms": res["median_ms"],
        "host_us_per_call": res["host_us_per_call"], "timing": res["timing"],
    }
    if path is not None:
        line["config"]["path"] = args.path

    if rank == 0 and not args.no_extras and world == 1:
        line["context"] = {"sdpa_dense_attention_ms": sdpa_ms(w, torch, res["sets"]),
                           "paper_speedups_over_flashattention2_on_A40":
                               {"N=256": 1.4, "N=4096": 4.5, "N=16384": 8.2}}
        del res
        torch.cuda.empty_cache()
        per = {}
        for name in sorted(wl.WORKLOADS):
            if name == w.name:
                continue
            ww = wl.WORKLOADS[name]
            r = time_config(ww, 50, 5, torch, binding)
            rl = roofline(ww, r["ms_per_step"], peaks, which)
            per[name] = {"ms_per_step": r["ms_per_step"], "min_ms": r["min_ms"], "timing": r["timing"],
                         "tokens_per_s": ww.tokens / (r["ms_per_step"] * 1e-3),
                         "bound": rl["bound"], "frac": rl["frac"],
                         "sdpa_dense_attention_ms": sdpa_ms(ww, torch, r["sets"])}
            del r
            torch.cuda.empty_cache()
        line["other_configs"] = per
        v, heads, secs, threads = oracle_sample(w, 3.0)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"{heads} head evaluations of {w.name} (its {w.BH} (batch, head) "
                                          f"units in turn) in {secs:.1f} s on {threads} host cores, fp64 "
                                          f"numpy oracle; tokens/s extrapolated from the sample"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
