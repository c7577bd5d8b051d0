"""Benchmark of the APOLLO optimizer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama7b] [--impl ours|reference]

One "step" is one whole apollo_step (projection pass, finalize, update pass) over the
LLaMA-7B-shaped list of 224 linear weights with rank 256 (bf16 W and G, fp32 states).
Prints one JSON line.  With N > 1 (torchrun) every rank steps its own replica of the model;
no collective runs inside the step.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

import torch

from paper_2412_05270_b200 import workloads as WL

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


def step_bytes(wl: WL.Workload, state_elem: int = 4):
    """Algorithmic HBM bytes of one step: G read by both passes, W read and written,
    M and V (state_elem bytes per entry) read and written (B_2p), and the single-read-of-G
    variant (B_min)."""
    e = 2 if wl.dtype == "bf16" else 4
    two_pass = minimal = flops = update = 0
    for rows, cols in wl.shapes:
        n = max(rows, cols)
        two_pass += 4 * e * rows * cols + 4 * state_elem * wl.rank * n
        minimal += 3 * e * rows * cols + 4 * state_elem * wl.rank * n
        update += 3 * e * rows * cols
        flops += 2 * wl.rank * rows * cols
    return two_pass, minimal, update, flops


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_value(params_per_rank: int, world: int, ms_per_step: float) -> float:
    """Parameters per second over all replicas (every rank steps its own copy of the list)."""
    return world * params_per_rank / (ms_per_step * 1e-3)


# DRAM bytes per parameter of update_kernel<bf16> from its ncu capture (profiles/update_kernel_*.md);
# set to None when the kernel changes until the counters are taken again.
UPDATE_TRAFFIC_BYTES_PER_PARAM = 5.89


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.monotonic(), [x.strip() for x in line.split(",")]))

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, t0=None, t1=None):
        """Median SM clock and the throttle reasons seen between host times t0 and t1 (the timed region).
        nvidia-smi needs 0.1-0.2 s to deliver its first sample, so the sampler is started before the
        warm-up; if the region was too short to catch a sample, the samples since the start are used
        and "window" says so."""
        inside = [r for t, r in self.rows if t0 is None or (t0 <= t <= t1)]
        window = "timed region"
        if not inside:
            inside, window = [r for _, r in self.rows], "warm-up and timed region"
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in inside:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "window": window}


def cpu_baseline(wl: WL.Workload, budget_s: float = 12.0):
    """Times the oracle, as it stands, on the host cores over the leading matrices of the list."""
    import oracle
    sys.path.insert(0, str(ROOT / "tests"))
    from parity import oracle_of
    oracle.build()
    cores = os.cpu_count() or 1
    done_params, elapsed, used = 0, 0.0, []
    for i in range(min(7, len(wl.shapes))):
        mo = oracle_of(wl, [i])[i]
        W = WL.make_weight(wl, i).float().numpy()
        G = WL.make_grad(wl, i, 0).float().numpy()
        t0 = time.perf_counter()
        mo.step(W, G, float(wl.lr), float(wl.wd))
        elapsed += time.perf_counter() - t0
        done_params += W.size
        used.append(f"{W.shape[0]}x{W.shape[1]}")
        if elapsed > budget_s:
            break
    return {"value": done_params / elapsed, "unit": "params/s", "cores": cores, "kind": "oracle",
            "sample": f"one step of matrices {', '.join(used)} of {wl.name} (rank {wl.rank}); {elapsed:.1f} s",
            "seconds": elapsed, "params": done_params}


def run_reference(args, wl, rank, world):
    """The reference arm: the CPU oracle on a bounded sample of the workload."""
    if rank != 0:
        return
    base = None
    for _ in range(max(1, min(args.steps, 2))):
        base = cpu_baseline(wl, budget_s=10.0)
    line = {
        "impl": "reference", "metric": "apollo_step_params_per_s", "value": base["value"], "unit": "params/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * base["seconds"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "rank": wl.rank, "mode": wl.mode, "sample": base["sample"]},
        "cpu_baseline": {k: base[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": base["value"], "unit": "params/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, wl, rank, world, local_rank):
    import torch.distributed as dist
    from paper_2412_05270_b200 import binding as B

    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    n = len(wl.shapes)
    Ws = [WL.make_weight(wl, i, device=dev) for i in range(n)]
    Gs = [WL.make_grad(wl, i, 0, device=dev) for i in range(n)]
    opt = B.Apollo(wl.shapes, B.config_for(wl, B.FLAG_BF16_STATES if args.bf16_states else 0), device=dev)
    opt.set_timing(True)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        for _ in range(args.warmup):
            opt.step(Ws, Gs, wl.lr, wl.wd, check=False)
        barrier()
        t_region0 = time.monotonic()
        start.record(stream)
        launches = 0
        for _ in range(args.steps):
            opt.step(Ws, Gs, wl.lr, wl.wd, check=False)
            launches += opt.last_launches()      # P is regenerated only in steps that open an epoch
        stop.record(stream)
        barrier()
        t_region1 = time.monotonic()
    ms_total = start.elapsed_time(stop)
    assert opt.status() == B.OK
    phases = [opt.timing(k) for k in range(min(args.steps, 64))]
    proj_ms = sum(p[0] for p in phases) / len(phases)
    fin_ms = sum(p[1] for p in phases) / len(phases)
    upd_ms = sum(p[2] for p in phases) / len(phases)

    # end to end: gradients arrive from pinned host memory every step, the limiter norms go back
    e2e = None
    if not args.no_e2e:
        e2e_steps = max(1, min(args.steps, 3))
        g_bytes = sum(g.numel() * g.element_size() for g in Gs)
        host_G = [torch.empty(g.shape, dtype=g.dtype, pin_memory=True).copy_(g) for g in Gs]
        norms_dev = torch.empty((n, 4), dtype=torch.float32, device=dev)
        norms_host = torch.empty((n, 4), dtype=torch.float32, pin_memory=True)
        barrier()
        s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s2.record(stream)
        # layer-wise, as the gradients would arrive during a backward pass: the copy of the next layer's
        # gradients (copy stream) runs under the optimizer step of the current layer (apollo_step_range)
        copy_stream = torch.cuda.Stream(device=dev)
        layers = [(a, min(a + 7, n)) for a in range(0, n, 7)]
        landed = [torch.cuda.Event() for _ in layers]
        consumed = [torch.cuda.Event() for _ in layers]
        for e2e_step in range(e2e_steps):
            with torch.cuda.stream(copy_stream):
                for k, (a, b) in enumerate(layers):
                    if e2e_step > 0:
                        copy_stream.wait_event(consumed[k])      # the previous step has read this layer's G
                    for i in range(a, b):
                        Gs[i].copy_(host_G[i], non_blocking=True)
                    landed[k].record(copy_stream)
            for k, (a, b) in enumerate(layers):
                stream.wait_event(landed[k])
                opt.step_range(a, Ws[a:b], Gs[a:b], wl.lr, wl.wd, close_step=(k == len(layers) - 1), stream=stream)
                consumed[k].record(stream)
            for i in range(n):
                B._check(opt.lib.apollo_get_limiter(opt.ctx, i, norms_dev[i].data_ptr(), stream.cuda_stream), "limiter")
            norms_host.copy_(norms_dev, non_blocking=True)
            stream.synchronize()
        e2.record(stream)
        barrier()
        e2e_ms = s2.elapsed_time(e2) / e2e_steps
        del host_G
    ms_total, e2e_ms = max_over_ranks([ms_total, e2e_ms if not args.no_e2e else 0.0], device=dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    ms_step = ms_total / args.steps
    two_pass, minimal, update_bytes, flops = step_bytes(wl, 2 if args.bf16_states else 4)
    value = whole_job_value(wl.params, world, ms_step)
    hbm, tc = peaks["hbm_gbs"] * 1e9, peaks["bf16_tflops_sustained"] * 1e12
    t_roof = max(two_pass / hbm, flops / tc)
    upd_gbs = update_bytes / (upd_ms * 1e-3) / 1e9
    line = {
        "metric": "apollo_step_params_per_s", "value": value, "unit": "params/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": {"workload": wl.name, "matrices": n, "params": wl.params, "rank": wl.rank, "mode": wl.mode,
                   "T": wl.T, "lr": wl.lr, "wd": wl.wd, "states": "bf16" if args.bf16_states else "f32", "replicas": world,
                   "l2": "inputs (W, G: %.1f GB) exceed L2, no flush" % (2 * wl.params * 2 / 1e9)},
        "roofline": {"bound": "hbm", "kernel": "update_kernel", "achieved": upd_gbs, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": upd_gbs / peaks["hbm_gbs"],
                     "traffic": (UPDATE_TRAFFIC_BYTES_PER_PARAM * wl.params
                                 if UPDATE_TRAFFIC_BYTES_PER_PARAM and wl.dtype == "bf16" else None),
                     "peak_source": peaks["source"], "bytes_per_launch": update_bytes, "ms_per_launch": upd_ms},
        "step_roofline": {"bytes_two_pass": two_pass, "bytes_min": minimal, "gemm_flops": flops,
                          "t_roofline_ms": 1e3 * t_roof, "frac": 1e3 * t_roof / ms_step,
                          "frac_vs_8TBs": 1e3 * max(two_pass / 8e12, flops / tc) / ms_step,
                          "phase_ms": {"projection": proj_ms, "finalize": fin_ms, "update": upd_ms}},
        "clocks": clocks.summary(t_region0, t_region1),
        "gpu_launches": launches,
    }
    if not args.no_e2e:
        line["e2e"] = {"value": whole_job_value(wl.params, world, e2e_ms), "unit": "params/s",
                       "h2d_bytes_per_step": g_bytes, "d2h_bytes_per_step": n * 16, "ms_per_step": e2e_ms}
    if args.adamw:
        # the non-projected parameters of the same model (embedding and head 32000 x hidden, norms):
        # 22 bytes per bf16 parameter (read g, p, m, v; write p, m, v)
        hidden = wl.shapes[0][0]
        sizes = [32000 * hidden, 32000 * hidden] + [hidden] * 65
        Pn = [torch.zeros(k, dtype=torch.bfloat16, device=dev) for k in sizes]
        Gn = [torch.full((k,), 1e-3, dtype=torch.bfloat16, device=dev) for k in sizes]
        Mn = [torch.zeros(k, dtype=torch.float32, device=dev) for k in sizes]
        Vn = [torch.zeros(k, dtype=torch.float32, device=dev) for k in sizes]
        for t in range(3):
            B.adamw_step(Pn, Gn, Mn, Vn, t, 1e-3, wd=0.01)
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        for t in range(10):
            B.adamw_step(Pn, Gn, Mn, Vn, 3 + t, 1e-3, wd=0.01)
        a1.record(stream)
        torch.cuda.synchronize()
        ms = a0.elapsed_time(a1) / 10
        nbytes = 22 * sum(sizes)
        line["adamw"] = {"params": sum(sizes), "ms_per_step": ms, "achieved": nbytes / (ms * 1e-3) / 1e9,
                         "unit": "GB/s", "frac": nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "bytes_per_param": 22}
    if world == 1 and not args.no_cpu:
        base = cpu_baseline(wl)
        line["cpu_baseline"] = {k: base[k] for k in ("value", "unit", "cores", "kind", "sample")}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="llama7b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="keep only the first LAYERS layers (profiling aid)")
    ap.add_argument("--adamw", action="store_true", help="also time the fused AdamW of the non-projected parameters")
    ap.add_argument("--bf16-states", action="store_true", help="keep M and V in bfloat16 (a variant, not the headline)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    wl = WL.workload(args.workload)
    if args.layers > 0:
        wl.shapes = wl.shapes[:7 * args.layers]
        wl.name = f"{wl.name}[first {args.layers} layers]"
    if args.impl == "reference":
        run_reference(args, wl, rank, world)
    else:
        run_ours(args, wl, rank, world, local_rank)


if __name__ == "__main__":
    main()
