#!/usr/bin/env python
"""Benchmark of the ZGR step on synthetic LLaMA-7B-shaped bf16 parameters (one B200 per process).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama_7b] [--bits 16|32]
    python bench.py --impl reference ...        # the CPU oracle on a bounded sample, same JSON line

A "step" is the whole hot path once: for each of the Q perturbation queries of the workload,
perturb(+eps), perturb(-2 eps), restore_update(lr/Q) -- 3Q in-place sweeps over every weight tensor.
`value` = model parameters stepped per second (parameters x steps / time, all ranks), measured with
CUDA events with weights, subspaces and work tables resident in HBM.  `e2e` repeats the measurement
with the per-step inputs coming from the host through the C ABI: every guided tensor's subspace is
copied from pinned host memory, layer by layer on a copy stream while the step's first sweep works through the
earlier layers (zgr_perturb_layers), that sweep also keeps the norm bookkeeping, and the per-tensor norms are
read back to the host (zgr_get_stats).  The weights themselves stay in HBM in both: keeping the model on
the device and never materialising z is the point of the method.

The path does not shard (one GPU holds the model; the only cross-rank quantities would be two loss
scalars), so --gpus N runs N independent replicas and reports their sum ("replicas only").
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "zgr_step_params_per_sec"
UNIT = "params/s"


# DRAM traffic per launch of the dominant kernel from one ncu capture (a small case, scaled by the elements
# processed), valid only for the kernel sources it was taken from.
NCU_TRAFFIC = {"kernel": "sweep_umma_kernel(k=32)", "workload": "llama_7b", "bytes_per_launch": 26.75e9,
               "sources": ["paper_2601_12917_b200/csrc/zgr_umma.cu", "paper_2601_12917_b200/csrc/zgr_device.cuh",
                           "paper_2601_12917_b200/csrc/zgr_internal.h"],
               "sha1": "6b5749836414c60e4212f96ea4d0513a440a50e2"}


def _code_only(text: str) -> str:
    """Source text without comments and white space: the digest below follows the code, not its commentary."""
    import re
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"//[^\n]*", "", text)
    return re.sub(r"\s+", "", text)


def ncu_traffic(kernel: str, workload: str):
    import hashlib
    if kernel != NCU_TRAFFIC["kernel"] or workload != NCU_TRAFFIC["workload"]:
        return None
    h = hashlib.sha1()
    try:
        for src in NCU_TRAFFIC["sources"]:
            with open(os.path.join(ROOT, src), "r") as f:
                h.update(_code_only(f.read()).encode())
    except OSError:
        return None
    if h.hexdigest() != NCU_TRAFFIC["sha1"]:
        return None                   # the kernel has changed since the counters were taken
    return NCU_TRAFFIC["bytes_per_launch"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ------------------------------------------------------------------------------------------ oracle legs
def oracle_sample(wl, rows: int, sweeps: int, bits: int):
    """Time `sweeps` oracle sweeps over a slab (rows x cols of the workload's first attention matrix,
    with its rank).  Returns (seconds, elements, threads)."""
    import numpy as np
    import oracle
    from paper_2601_12917_b200 import synth
    spec = next(t for t in wl.tensors if t.rank > 0 and t.rows == t.cols)
    rows = min(rows, spec.rows)
    dt = {"f32": oracle.F32, "f16": oracle.F16, "bf16": oracle.BF16}[wl.dtype]
    w = synth.weights_host(synth.TensorSpec("slab", rows, spec.cols, spec.rank), 0).ravel()
    U = synth.subspace(rows, spec.rank, 0)
    q = sc = None
    if wl.dtc:
        q, sc = synth.dtc_payload(spec.rank, spec.cols, 0)
    t = oracle.OracleTensor(theta=oracle.encode(w, dt), rows=rows, cols=spec.cols, dtype=dt, U=U, q=q, scale=sc)
    a, b = oracle.mix_scalars(wl.alpha, wl.params, wl.coeffs, wl.scale_mode)
    coeff = [wl.eps, -2 * wl.eps, wl.eps]
    t0 = time.perf_counter()
    for s in range(sweeps):
        oracle.sweep_tensor(t, 1 + s // 3, 1, bits, a, b, coeff[s % 3])
    return time.perf_counter() - t0, rows * spec.cols, oracle.num_threads(), f"{rows}x{spec.cols} slab of a rank-{spec.rank} {wl.dtype} matrix"


def cpu_baseline(wl, bits: int):
    """The oracle as it stands, timed on this machine's host cores on a bounded sample of the workload:
    whole sweeps over a slab of one matrix, repeated until about ten seconds of CPU work are done."""
    import oracle
    oracle.build()
    rows = 4096 if wl.params > (1 << 28) else 1024
    sweeps_per_step = 3 * wl.queries
    secs, n, threads, what = oracle_sample(wl, rows, 1, bits)       # also the warm-up
    reps = int(min(48, max(1, round(15.0 / max(secs * threads, 1e-3)))))
    secs, n, threads, what = oracle_sample(wl, rows, reps, bits)
    return {"value": n * reps / secs / sweeps_per_step, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{reps} sweeps over a {what} in {secs:.2f} s, scaled by 1/{sweeps_per_step} sweeps per step"}


def run_reference(args, wl):
    """`--impl reference`: the CPU oracle, K steps of 3Q sweeps over a bounded slab."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    sweeps_per_step = 3 * wl.queries
    rows = 1024
    for _ in range(args.warmup):
        oracle_sample(wl, 64, 1, args.bits)
    t0 = time.perf_counter()
    total = 0.0
    n = 0
    for _ in range(args.steps):
        secs, n, threads, what = oracle_sample(wl, rows, sweeps_per_step, args.bits)
        total += secs
    value = n * args.steps / total
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": wl.name, "sample": what, "queries": wl.queries, "bits_per_normal": args.bits},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": f"{args.steps} steps of {sweeps_per_step} sweeps over a {what}"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    def __init__(self, index):
        self.path = f"/tmp/zgr_clocks_{os.getpid()}.csv"
        self.proc = None
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(index), "--query-gpu=clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
                 "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap",
                 "--format=csv,noheader,nounits", "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
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
        self.f.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for ln in open(self.path):
                parts = [x.strip() for x in ln.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0])); mx.append(float(parts[1]))
                except ValueError:
                    continue
                for nm, v in zip(names, parts[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            os.remove(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------------------------------ GPU arm
def reduce_over_ranks(ms_local: float, units_local: float, dist=None):
    """(max over ranks of the elapsed time, sum over ranks of the units processed)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return ms_local, units_local
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    u = torch.tensor([units_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def run_step_deferred(z, wl, t: int):
    """The same step in 2Q+1 sweeps: the restore of query q-1 rides on the perturbation of query q, and one
    final multi-seed pass undoes the last perturbation and applies all Q projected-gradient updates."""
    Q = wl.queries
    seeds = [wl.seed(t, q) for q in range(Q)]
    z.sweep_multi([seeds[0]], [wl.eps])
    z.sweep_multi([seeds[0]], [-2.0 * wl.eps])
    for q in range(1, Q):
        z.sweep_multi([seeds[q - 1], seeds[q]], [wl.eps, wl.eps])
        z.sweep_multi([seeds[q]], [-2.0 * wl.eps])
    losses = [wl.losses(t, q) for q in range(Q)]
    z.restore_update_multi(seeds, [l[0] for l in losses], [l[1] for l in losses], wl.lr / Q)


def run_step(z, wl, t: int, schedule: str = "sequential", keep_norms: bool = False):
    """keep_norms: the first perturbation of the step also keeps the norm bookkeeping (zgr_enable_stats)."""
    if schedule == "deferred":
        return run_step_deferred(z, wl, t)
    for q in range(wl.queries):
        seed = wl.seed(t, q)
        lp, lm = wl.losses(t, q)
        if keep_norms and q == 0:
            z.enable_stats(True)
            z.perturb(seed, wl.eps)
            z.enable_stats(False)
        else:
            z.perturb(seed, wl.eps)
        z.perturb(seed, -2.0 * wl.eps)
        z.restore_update(seed, lp, lm, wl.lr / wl.queries)


def roofline_of(kernels, eb, peak, peak_kind):
    """Roofline entry of the kernel that took the most time: algorithmic bytes (read + write of every weight it
    covers) per launch over its average CUDA-event duration."""
    top = max(kernels, key=lambda k: k["ms_total"]) if kernels else None
    if not top:
        return None, None
    per_launch_ms = top["ms_total"] / top["launches"]
    achieved = 2 * eb * top["elements"] / (per_launch_ms * 1e-3) / 1e9
    kname = f"sweep_{top['path']}_kernel(k={top['kpad']})"
    return top, {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                 "peak_kind": f"of {peak_kind}", "kernel": kname, "launches": top["launches"], "ms_per_launch": per_launch_ms,
                 "algorithmic_bytes_per_launch": 2 * eb * top["elements"],
                 "share_of_kernel_time": top["ms_total"] / sum(k["ms_total"] for k in kernels)}


def measure_other(name, device, bits, steps, peak, peak_kind):
    """A short resident measurement of another of the paper-shaped configurations (parity-test cases of their
    own, shown here so that every sweep kernel has a driver-visible figure): 1 warm-up step, `steps` timed."""
    import torch
    from paper_2601_12917_b200 import synth, zgr
    wl = synth.workload(name)
    free, _ = torch.cuda.mem_get_info()
    if free < wl.params * synth.DTYPE_BYTES[wl.dtype] * 1.3 + 4e9:
        return {"workload": name, "skipped": "not enough free device memory"}
    dm = synth.materialise(wl, device, seed=0)
    z = zgr.from_device_model(dm, bits)
    stream = torch.cuda.current_stream()
    run_step(z, wl, 0)
    torch.cuda.synchronize()
    z.profile(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for t in range(steps):
        run_step(z, wl, 1 + t)
    ev1.record(stream)
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1)
    kernels = z.profile_read()
    z.profile(False)
    _, roof = roofline_of(kernels, synth.DTYPE_BYTES[wl.dtype], peak, peak_kind)
    out = {"workload": name, "storage": wl.dtype, "params": wl.params, "rank": wl.rank, "queries": wl.queries, "dtc": wl.dtc,
           "steps": steps, "ms_per_step": ms / steps, "value": wl.params * steps / (ms * 1e-3), "unit": UNIT, "roofline": roof}
    z.close()
    del z, dm
    torch.cuda.empty_cache()
    return out


def layer_table(wl):
    """Tensor index one past each layer: the embedding, every Transformer block, and what follows the last block."""
    ends, prev, seen_block = [], None, False
    for l, t in enumerate(wl.tensors):
        prefix = t.name.split(".")[0]
        is_block = prefix.startswith("l") and prefix[1:].isdigit()
        seen_block = seen_block or is_block
        key = prefix if is_block else ("after the blocks" if seen_block else "before the blocks")
        if prev is not None and key != prev:
            ends.append(l)
        prev = key
    ends.append(len(wl.tensors))
    return ends


def measure_overlap(device, bits):
    """Sec. 3.3 / 3.4 on the DTC configuration: the compressed coefficients of layer l + 1 travel from pinned host
    memory on a copy stream while layer l is swept (zgr_perturb_layers).  Reports the per-layer transmission time
    T_t against the per-layer sweep time T_cc, and what the delivery adds to the sweep."""
    import torch
    from paper_2601_12917_b200 import synth, zgr
    wl = synth.workload("llama_13b")
    free, _ = torch.cuda.mem_get_info()
    if free < wl.params * 2 * 1.3 + 4e9:
        return {"workload": wl.name, "skipped": "not enough free device memory"}
    dm = synth.materialise(wl, device, seed=0)
    z = zgr.from_device_model(dm, bits)
    ends = layer_table(wl)
    deliveries = [(l, dm.q[l].cpu().pin_memory(), dm.scale[l].cpu().pin_memory(), None) for l in range(len(wl.tensors)) if dm.q[l] is not None]
    payload = sum(q.numel() + 4 * sc.numel() for _, q, sc, _ in deliveries)
    stream, copy_stream = torch.cuda.current_stream(), torch.cuda.Stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, reps=3):
        fn(0)
        z.restore_update(0, 2.0, 2.0, 0.0)
        torch.cuda.synchronize()
        total = 0.0
        for i in range(reps):
            ev0.record(stream)
            fn(1 + i)
            ev1.record(stream)
            torch.cuda.synchronize()
            total += ev0.elapsed_time(ev1)
            z.restore_update(1 + i, 2.0, 2.0, 0.0)
        torch.cuda.synchronize()
        return total / reps

    one_launch = timed(lambda s: z.perturb(s, wl.eps))
    layerwise = timed(lambda s: z.perturb_layers(s, wl.eps, ends, copy_stream=copy_stream))
    delivered = timed(lambda s: z.perturb_layers(s, wl.eps, ends, deliveries, copy_stream=copy_stream))
    # the transmission alone
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(copy_stream):
        c0.record(copy_stream)
        for l, q, sc, _ in deliveries:
            dm.q[l].copy_(q, non_blocking=True)
            dm.scale[l].copy_(sc, non_blocking=True)
        c1.record(copy_stream)
    torch.cuda.synchronize()
    copy_ms = c0.elapsed_time(c1)
    n_layers = len(ends)
    out = {"workload": wl.name, "layers": n_layers, "omega": 1.0, "payload_bytes": payload, "transmission_ms": copy_ms,
           "sweep_ms_one_launch_per_kernel": one_launch, "sweep_ms_layerwise": layerwise, "sweep_ms_layerwise_with_delivery": delivered,
           "per_layer": {"T_t_ms": copy_ms / n_layers, "T_cc_ms": layerwise / n_layers},
           "transmission_hidden": 1.0 - max(0.0, delivered - layerwise) / copy_ms,
           "omega_that_still_hides": min(1.0, layerwise / copy_ms),
           "what": "H2D of the int8 coefficients and scales of layer l+1 on a copy stream while layer l is swept; T_t <= T_cc per layer means the transmission is hidden"}
    z.close()
    del z, dm
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="zgr", choices=["zgr", "reference"])
    ap.add_argument("--workload", default="llama_7b")
    ap.add_argument("--layers", type=int, default=None, help="shrink the model (profiling captures only)")
    ap.add_argument("--bits", type=int, default=16, choices=[16, 32], help="random bits per normal")
    ap.add_argument("--schedule", default="sequential", choices=["sequential", "deferred"],
                    help="sequential: 3Q single-seed sweeps per step (the headline); deferred: 2Q+1 sweeps with multi-seed passes")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="skip the short runs of the other configurations")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    from paper_2601_12917_b200 import synth
    wl = synth.workload(args.workload, layers=args.layers)
    if args.impl == "reference":
        run_reference(args, wl)
        return

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(wl, args.bits)        # before the first CUDA call

    import torch
    import torch.distributed as dist
    from paper_2601_12917_b200 import zgr
    zgr.lib()                                     # fail loudly if the CUDA library is missing
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    device = torch.device("cuda", local_rank)

    dm = synth.materialise(wl, device, seed=rank)
    z = zgr.from_device_model(dm, args.bits)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for t in range(args.warmup):
        run_step(z, wl, t, args.schedule)
    barrier()

    # ---- timed region: K steps, device-resident inputs ----
    cvd = [x for x in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if x]
    sampler = ClockSampler(cvd[local_rank] if local_rank < len(cvd) else local_rank)
    time.sleep(0.3)
    launches0 = z.launch_count()
    z.profile(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    for t in range(args.steps):
        run_step(z, wl, args.warmup + t, args.schedule)
    ev1.record(stream)
    barrier()
    ms_local = ev0.elapsed_time(ev1)
    kernels = z.profile_read()
    z.profile(False)
    launches = z.launch_count() - launches0
    clocks = sampler.stop()
    ms, units = reduce_over_ranks(ms_local, float(wl.params) * args.steps, dist if world > 1 else None)
    value = units / (ms * 1e-3)

    # ---- roofline of the dominant kernel ----
    peak, peak_kind = load_peaks()
    eb = synth.DTYPE_BYTES[wl.dtype]
    top, roofline = roofline_of(kernels, eb, peak, peak_kind)
    if top:
        per_launch_ms = roofline["ms_per_launch"]
        roofline["traffic"] = ncu_traffic(roofline["kernel"], wl.name) if args.layers is None else None
        # second bound of the same kernel: the special-function pipe that the Gaussian transform runs on.
        # 16 lanes per clock per SM x 148 SMs x 1.965 GHz; the transform costs four operations per pair of
        # normals (lg2, sqrt, sin, cos), i.e. 2 per element, in both generator modes.
        sfu_peak = 16 * 148 * 1.965e9 / 2.0
        roofline["sfu"] = {"bound": "alu", "achieved": top["elements"] / (per_launch_ms * 1e-3), "peak": sfu_peak,
                           "unit": "elements/s", "frac": top["elements"] / (per_launch_ms * 1e-3) / sfu_peak,
                           "peak_kind": "nominal: 16 special-function lanes/clk/SM x 148 SMs x 1.965 GHz / 2 operations per element"}

    # ---- end to end: per-step inputs from pinned host memory, result read back ----
    e2e = None
    if not args.no_e2e:
        guided = [l for l, U in enumerate(dm.U) if U is not None]
        host_U = {l: dm.U[l].cpu().pin_memory() for l in guided}
        h2d = sum(h.numel() * 4 for h in host_U.values())
        d2h = 3 * 8 * len(dm.theta)
        n_e2e = max(1, min(args.steps, 3))

        ends = layer_table(wl)
        copy_stream = torch.cuda.Stream()
        deliveries = [(l, None, None, None, host_U[l]) for l in guided]

        def e2e_step(t):
            # The step's first sweep runs layer by layer: the subspaces of a layer arrive from pinned host memory
            # on the copy stream while earlier layers are swept, and that sweep also keeps the norm bookkeeping.
            if args.schedule == "sequential":
                seed0 = wl.seed(t, 0)
                lp, lm = wl.losses(t, 0)
                z.enable_stats(True)
                z.perturb_layers(seed0, wl.eps, ends, deliveries, copy_stream=copy_stream)
                z.enable_stats(False)
                z.perturb(seed0, -2.0 * wl.eps)
                z.restore_update(seed0, lp, lm, wl.lr / wl.queries)
                for q in range(1, wl.queries):
                    seed = wl.seed(t, q)
                    lp, lm = wl.losses(t, q)
                    z.perturb(seed, wl.eps)
                    z.perturb(seed, -2.0 * wl.eps)
                    z.restore_update(seed, lp, lm, wl.lr / wl.queries)
            else:
                z.update_subspaces(guided, [host_U[l] for l in guided])
                run_step(z, wl, t, args.schedule, keep_norms=True)
            return z.get_stats(wl.seed(t, 0))      # the norms kept by the step's first sweep: one small launch and a 7 KB read

        e2e_step(10_000)
        barrier()
        ev0.record(stream)
        for t in range(n_e2e):
            e2e_step(20_000 + t)
        ev1.record(stream)
        barrier()
        ms_e, units_e = reduce_over_ranks(ev0.elapsed_time(ev1), float(wl.params) * n_e2e, dist if world > 1 else None)
        e2e = {"value": units_e / (ms_e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e,
               "ms_per_step": ms_e / n_e2e, "what": "subspaces H2D from pinned memory (layer by layer on a copy stream, under the step's first sweep) + step + per-tensor norms D2H, through the C ABI"}

    # ---- the other configurations, briefly (single process only; the headline above is unaffected) ----
    others = overlap = None
    z.close()
    if world == 1 and not args.no_others and args.layers is None and wl.name == "llama_7b":
        del dm
        torch.cuda.empty_cache()
        others = [measure_other(name, device, args.bits, 3, peak, peak_kind) for name in ("roberta_large", "opt_1p3b", "llama_13b")]
        full = measure_other("llama_7b", device, 32, 3, peak, peak_kind)      # the headline workload with 32 random bits per normal
        full["bits_per_normal"] = 32
        others.append(full)
        overlap = measure_overlap(device, args.bits)

    if rank == 0:
        sweeps = 3 * wl.queries if args.schedule == "sequential" else 2 * wl.queries + 1
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32",     # the arithmetic type of the path; the weights are stored as config.storage
                "data": "synthetic",
                "config": {"workload": wl.name, "storage": wl.dtype, "params": wl.params, "tensors": len(wl.tensors), "rank": wl.rank,
                           "queries": wl.queries, "schedule": args.schedule, "sweeps_per_step": sweeps, "bits_per_normal": args.bits, "alpha": wl.alpha, "eps": wl.eps,
                           "lr": wl.lr, "scale_mode": "unit", "l2": "inputs larger than L2 (no flush needed)", "parallelism": "replicas only"},
                "sweep_params_per_s": value * sweeps, "hbm_gbs_all_sweeps": value * sweeps * 2 * eb / 1e9,
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu,
                "kernels": kernels, "other_configs": others, "overlap": overlap}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
