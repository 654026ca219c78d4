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
def oracle_sample(w: wl.Workload, budget_s: float):
    """Times the fp64 oracle, as it stands, on whole heads of the workload until the budget is
    used; returns (tokens_per_s, heads_done, seconds, threads)."""
    from oracle import monarch_oracle
    Q, K, V = wl.make_qkv(1, min(w.heads, 16), w.N, w.d, w.dtype, w.rank, w.s, w.seed)
    monarch_oracle.monarch_attention_head(Q[0, 0, :w.b * 2], K[0, 0, :w.b * 2], V[0, 0, :w.b * 2],
                                          w.b, 1)   # import/warm-up
    done, t0 = 0, time.perf_counter()
    while True:
        h = done % Q.shape[1]
        monarch_oracle.monarch_attention_head(Q[0, h], K[0, h], V[0, h], w.b, w.T)
        done += 1
        el = time.perf_counter() - t0
        if el >= budget_s or done >= w.BH:
            break
    tokens = w.tokens * done / w.BH
    return tokens / el, done, el, 1


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    steps, warm = max(1, args.steps), max(0, args.warmup)
    budget = min(20.0, 150.0 / (steps + warm))
    vals, heads = [], 0
    for i in range(warm + steps):
        v, heads, _, threads = oracle_sample(w, budget)
        if i >= warm:
            vals.append(v)
    value = float(np.mean(vals))
    sample = f"{heads} of {w.BH} (batch, head) units of {w.name} per step, fp64 numpy oracle"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": 1e3 * w.tokens / value,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, 1),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(w, world):
    return {"workload": f"{w.name}: batch={w.batch} heads={w.heads} N={w.N} d={w.d} b={w.b} "
                        f"T={w.T} {w.dtype}, rank-{w.rank} component x{w.s}, seed {w.seed}",
            "per_gpu_batch": w.batch, "global_batch": w.batch * world, "seq_len": w.N,
            "parallelism": f"(batch,head) units sharded, {world} rank(s), no collective",
            "l2": "3 rotating input/output sets (>= 3x the call's footprint) so no step re-reads "
                  "data left in the 126 MB L2 by the previous one"}


# ----------------------------------------------------------------------------- ours
def time_config(w, steps, warmup, torch, binding, n_sets=3, dist=None):
    """Device-timed steps of workload w.  Returns dict with ms_per_step etc."""
    sets = []
    for r in range(n_sets):
        Q, K, V = wl.make_qkv(w.batch, w.heads, w.N, w.d, w.dtype, w.rank, w.s,
                              w.seed + 1000 * r + 17 * int(os.environ.get("RANK", "0")))
        Qd, Kd, Vd = (binding.to_device(x, w.dtype) for x in (Q, K, V))
        sets.append((Qd, Kd, Vd, torch.empty_like(Qd)))
    binding.monarch_attn_fwd(sets[0][0], sets[0][1], sets[0][2], w.b, w.T, Y=sets[0][3])  # sizes ws
    torch.cuda.synchronize()
    launches = binding.monarch_attn_last_launch_count()
    for i in range(warmup):
        s = sets[i % n_sets]
        binding.monarch_attn_fwd(s[0], s[1], s[2], w.b, w.T, Y=s[3])
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
        torch.cuda.synchronize()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    evs[0].record()
    for i in range(steps):
        s = sets[(warmup + i) % n_sets]
        binding.monarch_attn_fwd(s[0], s[1], s[2], w.b, w.T, Y=s[3])
        evs[i + 1].record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    total_ms = evs[0].elapsed_time(evs[-1])
    per = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]
    assert binding.monarch_attn_device_status() == 0
    return {"total_ms": total_ms, "ms_per_step": total_ms / steps, "min_ms": min(per),
            "median_ms": statistics.median(per), "launches_per_step": launches, "sets": sets}


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


# DRAM bytes of ONE launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum,
# ncu; see the summaries under profiles/ named for each kernel and workload).
NCU_TRAFFIC_BYTES = {"C5": 185.5e6 + 31.7e6, "C4": 174.9e6 + 20.7e6, "C3": 132.7e6 + 42.5e6, "C2": 75.5e6 + 4.0e6,
                     "S1": 62.0e6 + 2.4e6, "S3": (100.7e6 + 31.8e6) + (101.8e6 + 13.0e6)}   # S3: both launches of a step


def roofline(w, ms, peaks, which):
    t_hbm = w.algorithmic_bytes() / (peaks["hbm_gbs"] * 1e9)
    t_tc = w.algorithmic_flops() / (peaks["bf16_tflops_sustained"] * 1e12) if w.dtype != "f32" else 0.0
    if t_tc > t_hbm:
        ach = w.algorithmic_flops() / (ms * 1e-3) / 1e12
        return {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"],
                "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops_sustained"],
                "traffic": NCU_TRAFFIC_BYTES.get(w.name), "of": which + " (sustained)",
                "scope": "one launch = one step (the tensor path is a single persistent kernel)"}
    ach = w.algorithmic_bytes() / (ms * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": ach / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES.get(w.name), "of": which,
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

    sampler = ClockSampler(local)
    sampler.start()
    res = time_config(w, steps, warmup, torch, binding, dist=dist)
    clocks = sampler.stop()
    ms = D.max_over_ranks(res["total_ms"] / steps, device="cuda")
    e2e_ms, h2d, d2h = time_e2e(w, max(3, min(steps, 20)), 3, torch, binding, dist)
    e2e_ms = D.max_over_ranks(e2e_ms, device="cuda")

    line = {
        "metric": METRIC, "value": world * w.tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": workload_config(w, world),
        "clocks": clocks,
        "e2e": {"value": world * w.tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": res["launches_per_step"] * steps,
        "roofline": roofline(w, ms, peaks, which),
        "min_ms": res["min_ms"], "median_ms": res["median_ms"],
    }

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
            per[name] = {"ms_per_step": r["ms_per_step"], "min_ms": r["min_ms"],
                         "tokens_per_s": ww.tokens / (r["ms_per_step"] * 1e-3),
                         "bound": rl["bound"], "frac": rl["frac"],
                         "sdpa_dense_attention_ms": sdpa_ms(ww, torch, r["sets"])}
            del r
            torch.cuda.empty_cache()
        line["other_configs"] = per
        v, heads, secs, threads = oracle_sample(w, 12.0)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"{heads} of {w.BH} (batch, head) units of {w.name} in "
                                          f"{secs:.1f} s, fp64 numpy oracle"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
