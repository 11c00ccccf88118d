"""Benchmark of the Fira optimizer step on B200.

    python bench.py --gpus 1 --steps K --warmup W [--workload llama-7b]
    python bench.py --impl reference ...      # the fp64 CPU oracle on a bounded sample

One "step" is one fira_step() over every 2-D weight matrix of the workload (all
phases of Algorithm 1's loop body).  The metric is the step time in milliseconds
per full model (lower is better).  Prints one JSON line on rank 0.

With --gpus N > 1 the path does not shard (one GPU per model, no collective): every
rank steps its own replica and the reported time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fira_step_time_ms_per_model"
UNIT = "ms"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama-7b")
    ap.add_argument("--layers", type=int, default=None, help="override the layer count")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--refresh", default="full", choices=["none", "layer", "full"],
                    help="time the projection refresh (separately from the step)")
    return ap.parse_args()


# ----------------------------------------------------------------------------- roofline numbers
def flops_and_bytes(wl):
    """Algorithmic work of one step: 4 m n r flops (two products) and the minimum
    bytes (G once, W read + write, fp32 M and V read + write, projection once)."""
    e = 2 if wl.dtype == "bf16" else 4
    fl = by = 0
    for (m, n) in wl.shapes:
        l, d = max(m, n), min(m, n)
        fl += 4 * m * n * wl.r
        by += 3 * e * m * n + 16 * wl.r * l + e * wl.r * d
    return fl, by


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# fp32 CUDA-core peak: 148 SMs x 128 FMA lanes x 2 flop x 1.965 GHz (maximum SM clock)
ALU_FP32_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12

# dram__bytes_read.sum + dram__bytes_write.sum of one launch, from an ncu capture of 2 layers of
# the llama-7b list (every layer has the same shapes, so the traffic of a full launch is this times
# the layer ratio).  None: the kernel has changed since its counters were taken.
NCU_DRAM_BYTES_2_LAYERS = {"k_tc_project": 1.855e9 + 0.971e9, "k_tc_back_project": 1.999e9 + 0.781e9}

# kernel name -> (pipe that does its arithmetic, share of the step's 4 m n r flops)
KERNEL_PIPE = {
    "k_project": ("alu", 0.5), "k_back_project<norm>": ("alu", 0.5), "k_back_project<update>": ("alu", 0.5),
    "k_tc_project": ("tensor", 0.5), "k_tc_back_project": ("tensor", 0.5),
}


def kernel_min_bytes(name, wl):
    """The kernel's share of the step's minimum bytes: the projection product reads G and the
    projection once and moves the fp32 moments in and out; the back-projection reads and writes W.
    (What the two exchange through scratch memory -- N, R, X -- and the second pass over G are not
    algorithmic bytes.)"""
    e = 2 if wl.dtype == "bf16" else 4
    by = 0
    for (m, n) in wl.shapes:
        l, d = max(m, n), min(m, n)
        if "back_project" in name:
            by += 2 * e * m * n
        elif "project" in name:
            by += e * m * n + e * wl.r * d + 16 * wl.r * l
    return by


def time_adam_dense(dev, dtype, numel=64 * 1024 * 1024, tensors=2, iters=10):
    """fira_adam_dense on `tensors` flat tensors of `numel` elements (far larger than L2):
    achieved bytes per second against the measured copy bandwidth."""
    import torch
    from paper_2410_01623_b200 import binding as fb
    hp = fb.make_hparams()
    W = [torch.zeros(numel, dtype=dtype, device=dev) for _ in range(tensors)]
    G = [torch.ones(numel, dtype=dtype, device=dev) for _ in range(tensors)]
    M = [torch.zeros(numel, device=dev) for _ in range(tensors)]
    V = [torch.zeros(numel, device=dev) for _ in range(tensors)]
    for t in range(3):
        fb.adam_dense(hp, W, G, M, V, t)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for t in range(iters):
        fb.adam_dense(hp, W, G, M, V, 3 + t)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    es = 2 if dtype == torch.bfloat16 else 4
    gbs = tensors * numel * (3 * es + 16) / (ms * 1e-3) / 1e9
    peak = measured_peaks()["hbm_gbs"]
    return {"ms": ms, "elements": tensors * numel, "bytes_per_element": 3 * es + 16, "GB/s": gbs,
            "frac_of_hbm_peak": gbs / peak}


class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, reasons, mx = [], set(), None
        try:
            for line in open(self.path):
                p = [x.strip() for x in line.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1]))
                    mx = float(p[2])
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), p[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=mx, samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ----------------------------------------------------------------------------- reference arm
def oracle_sample_indices(wl):
    """One whole layer (all three shapes) when the model has several."""
    per_layer = 7 if len(wl.shapes) >= 7 else len(wl.shapes)
    return list(range(per_layer)), len(wl.shapes) / per_layer


def time_oracle(wl, steps, warmup):
    """Times oracle.fira_oracle.fira_step as it stands on the host cores, on one layer
    of the workload; returns (ms per full model, cores, sample description)."""
    import numpy as np
    from oracle import fira_oracle as fo
    from paper_2410_01623_b200 import workloads as wk
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    idxs, scale = oracle_sample_indices(wl)
    hp = fo.Hyper(lr=wl.lr, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, alpha=wl.alpha, gamma=wl.gamma)
    store = "bf16" if wl.dtype == "bf16" else "f32"
    import torch
    data = []
    for i in idxs:
        m, n = wl.shapes[i]
        W = wk.initial_weight(wl, i).to(dtype=torch.float64).numpy()
        G = wk.gradient(wl, i, 1).to(dtype=torch.float64).numpy()
        P = wk.random_projection(wl, i).to(dtype=torch.float64).numpy()
        data.append([W, G, P, fo.new_state(m, n, wl.r)])
    times = []
    start = time.perf_counter()
    for s in range(warmup + steps):
        t0 = time.perf_counter()
        for row in data:
            row[0], _ = fo.fira_step(row[0], row[1], row[2], row[3], hp, store=store)
        dt = time.perf_counter() - t0
        if s >= warmup or time.perf_counter() - start > 120:
            times.append(dt)
        if time.perf_counter() - start > 120:           # keep the whole run within minutes
            break
    ms_model = 1e3 * statistics.mean(times) * scale
    sample = (f"{len(idxs)} matrices (one layer) x {len(times)} steps, scaled x{scale:g} to the "
              f"{len(wl.shapes)}-matrix model")
    return ms_model, cores, sample


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2410_01623_b200 import workloads as wk
    wl = wk.workload(args.workload, args.layers)
    steps = max(1, min(args.steps, 3))
    warmup = min(args.warmup, 1)
    ms, cores, sample = time_oracle(wl, steps, warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": ms, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(wl, args),
        "cpu_baseline": {"value": ms, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": ms, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(wl, args):
    return {"workload": wl.name, "matrices": len(wl.shapes), "layers": wl.layers, "r": wl.r,
            "storage": wl.dtype, "parallelism": "replicas only" if args.gpus > 1 else "1 gpu",
            "l2": "inputs larger than L2 (no flush needed)" if sum(m * n for m, n in wl.shapes) * 2 > 126e6
                  else "L2 flushed between steps"}


def max_over_ranks(ms: float, world: int, device) -> float:
    """The job's time is the slowest rank's: every rank steps its own replica (the path
    has no exchange step), so the only collective is this MAX over the ranks' times."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ----------------------------------------------------------------------------- our arm
def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    import torch
    import torch.distributed as dist
    from paper_2410_01623_b200 import binding as fb
    from paper_2410_01623_b200 import build as fbuild
    from paper_2410_01623_b200 import workloads as wk

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        fbuild.build()
    if world > 1:
        dist.barrier()

    wl = wk.workload(args.workload, args.layers)
    nmat = len(wl.shapes)
    hp = fb.make_hparams(lr=wl.lr, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, alpha=wl.alpha,
                         gamma=wl.gamma, T=wl.T)
    f = fb.Fira(wl.shapes, wl.r, wl.torch_dtype, hp, dev)
    W = [wk.initial_weight(wl, i, dev) for i in range(nmat)]
    G = [wk.gradient(wl, i, 1, dev) for i in range(nmat)]
    # projections: the refresh is outside the timed step, so seeded orthonormal bases
    # (one per distinct projected extent) are set; the refresh is timed on its own below
    cache = {}
    for i, (m, n) in enumerate(wl.shapes):
        d = min(m, n)
        if d not in cache:
            cache[d] = wk.random_projection(wl, i, dev)
        f.set_projection(i, cache[d])
    cache.clear()
    flush = None
    if sum(m * n for m, n in wl.shapes) * 2 <= 126e6:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        f.step(W, G)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    f.enable_phase_timing(True)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(args.steps)]
    barrier()
    for s in range(args.steps):
        if flush is not None:
            flush.fill_(s & 255)
        ev[s][0].record()
        f.step(W, G)
        ev[s][1].record()
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = sum(a.elapsed_time(b) for a, b in ev)
    phases, nrec = f.phase_times()
    f.enable_phase_timing(False)
    launches = f.last_step_launches() * args.steps
    status = f.poll()
    ms_step = max_over_ranks(ms_total, world, dev) / args.steps

    # ---- the same list with rows padded to a 16-byte multiple (leading dimension = n rounded up to
    # 8 elements), for lists that have matrices whose rows TMA cannot address in place: what a
    # caller gains by padding its rows (the library then works on W and G where they are)
    aligned = None
    if rank == 0 and wl.dtype == "bf16" and any(n % 8 for _, n in wl.shapes):
        lds = [(n + 7) // 8 * 8 for _, n in wl.shapes]
        hp2 = fb.make_hparams(lr=wl.lr, beta1=wl.beta1, beta2=wl.beta2, eps=wl.eps, alpha=wl.alpha,
                              gamma=wl.gamma, T=wl.T, flags=fb.FLAG_ROW_PADDING_WRITABLE)
        f2 = fb.Fira(wl.shapes, wl.r, wl.torch_dtype, hp2, dev, lds=lds)
        W2, G2 = [], []
        for i, (m, n) in enumerate(wl.shapes):
            wb = torch.zeros(m, lds[i], dtype=wl.torch_dtype, device=dev)
            gb = torch.zeros(m, lds[i], dtype=wl.torch_dtype, device=dev)
            wb[:, :n].copy_(W[i]); gb[:, :n].copy_(G[i])
            W2.append(wb[:, :n]); G2.append(gb[:, :n])
            f2.set_projection(i, f.get_projection(i))
        for _ in range(args.warmup):
            f2.step(W2, G2)
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(args.steps):
            f2.step(W2, G2)
        a1.record()
        torch.cuda.synchronize()
        aligned = {"ms_per_step": a0.elapsed_time(a1) / args.steps, "steps": args.steps,
                   "what": "same list, leading dimension padded to a multiple of 8 elements and "
                           "FIRA_FLAG_ROW_PADDING_WRITABLE set (worked on in place, no staging copies)"}
        del f2, W2, G2

    # ---- plain Adam for unprojected parameters (fira_adam_dense): HBM-bound, timed on its own
    adam_dense = None
    if args.refresh != "none" and rank == 0:
        adam_dense = time_adam_dense(dev, wl.torch_dtype)

    # ---- refresh, timed separately (one layer, scaled, unless --refresh full)
    refresh = None
    if args.refresh != "none" and rank == 0:
        which = list(range(nmat)) if args.refresh == "full" else list(range(min(7, nmat)))
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        f.refresh_projection(G, which=which, seed=1)
        torch.cuda.synchronize()
        dt = (time.perf_counter() - t0) * 1e3
        refresh = {"ms": dt * (nmat / len(which)), "measured_on": f"{len(which)} of {nmat} matrices",
                   "rounds": 4, "iters": "library default (4 rounds)"}

    # ---- end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        try:
            e2e = run_e2e(f, wl, W, G, dev, world, min(args.steps, 3))
        except Exception as exc:  # host memory for the pinned copies may be missing
            e2e = {"value": None, "unit": UNIT, "error": str(exc)[:200]}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    fl, by = flops_and_bytes(wl)
    # the step's roofline: the slower of the two products at the tensor peak and the minimum bytes at
    # the copy bandwidth; the sustained tensor figure applies to a kernel timed inside a long step,
    # the burst figure is given beside it
    t_hbm = by / (peaks["hbm_gbs"] * 1e9)
    pipe_peak = peaks["bf16_tflops_sustained"] if wl.dtype == "bf16" else ALU_FP32_TFLOPS
    roof_ms = max(fl / (pipe_peak * 1e12), t_hbm) * 1e3
    roof_ms_burst = max(fl / ((peaks["bf16_tflops"] if wl.dtype == "bf16" else ALU_FP32_TFLOPS) * 1e12), t_hbm) * 1e3
    top = max(phases, key=lambda p: p[1]) if phases else ("", 0.0)
    pipe, share = KERNEL_PIPE.get(top[0], ("hbm", None))
    kbytes = kernel_min_bytes(top[0], wl)
    kflops = fl * share if share else 0.0
    if pipe == "tensor":
        ppeak, peak_kind = peaks["bf16_tflops_sustained"], f"cuBLAS bf16 sustained, {peaks['source']}"
    elif pipe == "alu":
        ppeak, peak_kind = ALU_FP32_TFLOPS, "fp32 FMA: 148 SMs x 128 lanes x 2 x 1.965 GHz (derived)"
    else:
        ppeak, peak_kind = None, None
    # which roof bounds THIS kernel on THIS workload: its flop time against its byte time
    if ppeak is not None and kflops / (ppeak * 1e12) >= kbytes / (peaks["hbm_gbs"] * 1e9):
        bound, peak, unit, ach = pipe, ppeak, "TFLOP/s", kflops / (top[1] * 1e-3) / 1e12
    else:
        bound, peak, unit = "hbm", peaks["hbm_gbs"], "GB/s"
        ach = kbytes / (top[1] * 1e-3) / 1e9 if kbytes else None
        peak_kind = f"copy bandwidth, {peaks['source']}"
    # DRAM bytes per launch from an ncu capture of 2 of the 32 layers, scaled by the layer count
    traffic = None
    if wl.name == "llama-7b" and NCU_DRAM_BYTES_2_LAYERS.get(top[0]):
        traffic = NCU_DRAM_BYTES_2_LAYERS[top[0]] * (nmat / 14.0)
    roofline = {"kernel": top[0], "bound": bound, "achieved": ach, "peak": peak, "unit": unit,
                "frac": (ach / peak) if ach else None, "traffic": traffic, "peak_kind": peak_kind,
                "frac_of_burst_peak": (ach / peaks["bf16_tflops"]) if (ach and bound == "tensor") else None,
                "kernel_ms": top[1], "kernel_share": top[1] / max(sum(p[1] for p in phases), 1e-9),
                "kernel_algorithmic_bytes": kbytes, "kernel_algorithmic_flops": kflops,
                "step_roofline_ms": roof_ms, "step_frac_of_roofline": roof_ms / ms_step,
                "step_roofline_ms_burst": roof_ms_burst, "step_frac_of_roofline_burst": roof_ms_burst / ms_step,
                "phases_ms": {k: round(v, 4) for k, v in phases}, "phase_steps": nrec}
    if refresh is not None:
        # Eq. 7 by subspace iteration: 2 q + 1 big products of 2 m n r flops each (q rounds)
        q = refresh["rounds"]
        rfl = (2 * q + 1) * fl / 2
        rpeak = peaks["bf16_tflops_sustained"] if wl.dtype == "bf16" else ALU_FP32_TFLOPS
        refresh["achieved_tflops"] = rfl / (refresh["ms"] * 1e-3) / 1e12
        refresh["frac"] = refresh["achieved_tflops"] / rpeak
        refresh["peak_tflops"] = rpeak

    cpu = None
    if not args.no_cpu_baseline:
        ms_cpu, cores, sample = time_oracle(wl, 1, 0)
        cpu = {"value": ms_cpu, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample}

    line = {
        "metric": METRIC, "value": ms_step, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
        "config": workload_config(wl, args), "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
        "roofline": roofline, "cpu_baseline": cpu, "refresh": refresh, "adam_dense": adam_dense, "aligned_pitch": aligned, "device_status": status,
        "engines": sorted({f.diagnostics(i)["engine"] for i in range(0, nmat, max(1, nmat // 8))}),
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_e2e(f, wl, W, G, dev, world, steps):
    """The same step through fira_step_host: weights and gradients start in page-locked
    host memory; every step copies G and W to the device, steps, and copies W back."""
    import torch
    import torch.distributed as dist
    nmat = len(wl.shapes)
    Wh = [w.to("cpu").pin_memory() for w in W]
    Gh = [g.to("cpu").pin_memory() for g in G]
    staging = torch.empty(f.staging_bytes(), dtype=torch.uint8, device=dev)
    h2d = sum(w.numel() * w.element_size() for w in Wh) + sum(g.numel() * g.element_size() for g in Gh)
    d2h = sum(w.numel() * w.element_size() for w in Wh)
    f.step_host(Wh, Gh, staging)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        f.step_host(Wh, Gh, staging)
    b.record()
    torch.cuda.synchronize()
    return {"value": max_over_ranks(a.elapsed_time(b), world, dev) / steps, "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "steps": steps}


if __name__ == "__main__":
    main()
