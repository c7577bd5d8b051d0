"""Benchmark of the APOLLO optimizer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama7b] [--impl ours|reference]

One "step" is one whole apollo_step (projection pass, finalize, update pass) over the
LLaMA-7B-shaped list of 224 linear weights with rank 256 (bf16 W and G, fp32 states).
Prints one JSON line.  With N > 1 (torchrun) every rank steps its own replica of the model;
no collective runs inside the step.  The same line carries, under "also", the step of the
other named lists (LLaMA-1B at rank 512, 7B APOLLO-Mini, 350M) and, under "sustained", the 7B
step repeated for several seconds (the board then runs at its power cap).
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


# DRAM bytes per parameter of update_kernel<bf16> from its ncu capture on the first two layers of the list;
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


def oracle_sample_step(wl: WL.Workload, mats, state):
    """One oracle step over the matrices `mats` (fresh gradients each call); returns seconds and parameters."""
    import oracle
    sys.path.insert(0, str(ROOT / "tests"))
    from parity import oracle_of
    if not state:
        oracle.build()
        state["orc"] = oracle_of(wl, mats)
        state["W"] = {i: WL.make_weight(wl, i).float().numpy() for i in mats}
        state["t"] = 0
    elapsed, params = 0.0, 0
    for i in mats:
        G = WL.make_grad(wl, i, state["t"]).float().numpy()
        t0 = time.perf_counter()
        res = state["orc"][i].step(state["W"][i], G, float(wl.lr), float(wl.wd))
        elapsed += time.perf_counter() - t0
        state["W"][i] = res.W
        params += G.size
    state["t"] += 1
    return elapsed, params


def run_reference(args, wl, rank, world):
    """The reference arm: the CPU oracle, as it stands, on the host cores.  One step of this arm is one oracle
    step over a bounded sample of the list (one square and one tall matrix), so that warm-up plus timed steps
    end within a few minutes; parameters per second is the metric, and the estimate for the whole list is the
    sample's time scaled by the parameter counts."""
    if rank != 0:
        return
    mats = [0, 6] if len(wl.shapes) >= 7 else [0]
    state = {}
    for _ in range(args.warmup):
        oracle_sample_step(wl, mats, state)
    seconds, params = 0.0, 0
    for _ in range(args.steps):
        dt, p = oracle_sample_step(wl, mats, state)
        seconds += dt
        params += p
    per_step_s = seconds / max(args.steps, 1)
    sample_params = params // max(args.steps, 1)
    value = params / seconds
    sample = (f"per step: one oracle step of matrices {', '.join('%dx%d' % tuple(wl.shapes[i]) for i in mats)} of "
              f"{wl.name} (rank {wl.rank}), {sample_params} parameters, {per_step_s:.2f} s")
    base = {"value": value, "unit": "params/s", "cores": os.cpu_count() or 1, "kind": "oracle", "sample": sample}
    line = {
        "impl": "reference", "metric": "apollo_step_params_per_s", "value": value, "unit": "params/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * per_step_s, "ms_per_full_step_estimate": 1e3 * per_step_s * wl.params / sample_params,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "rank": wl.rank, "mode": wl.mode, "sample": sample,
                   "step": "one oracle step over the sample; ms_per_step is the sample's, "
                           "ms_per_full_step_estimate scales it by parameters to the whole list"},
        "cpu_baseline": base,
        "e2e": {"value": value, "unit": "params/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


RANGE_SIZE = 0      # --range-size: step the list in ranges of this many matrices (apollo_step_range), 0 = apollo_step


def one_step(opt, Ws, Gs, wl):
    """One optimizer step: apollo_step over the whole list, or range by range (projection, finalize and update of
    a few matrices back to back, as a layer-wise update during the backward pass would issue them)."""
    if RANGE_SIZE <= 0:
        opt.step(Ws, Gs, wl.lr, wl.wd, check=False)
        return opt.last_launches()
    n, launches = len(Ws), 0
    for a in range(0, n, RANGE_SIZE):
        b = min(a + RANGE_SIZE, n)
        opt.step_range(a, Ws[a:b], Gs[a:b], wl.lr, wl.wd, close_step=(b == n))
        launches += opt.last_launches()
    return launches


def time_steps(opt, Ws, Gs, wl, steps, warmup, stream, barrier, clocks):
    """`warmup` untimed steps, then `steps` timed ones between two CUDA events on `stream`.  Returns the
    total milliseconds, the kernel launches inside the timed region, the per-phase means and the clocks
    sampled during the region."""
    for _ in range(warmup):
        one_step(opt, Ws, Gs, wl)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t0 = time.monotonic()
    start.record(stream)
    launches = 0
    for _ in range(steps):
        launches += one_step(opt, Ws, Gs, wl)
    stop.record(stream)
    barrier()
    t1 = time.monotonic()
    if RANGE_SIZE > 0:          # the per-phase events are recorded by whole-list steps only
        return start.elapsed_time(stop), launches, {"projection": 0.0, "finalize": 0.0, "update": 1e-9}, clocks.summary(t0, t1)
    phases = [opt.timing(k) for k in range(min(steps, 64))]
    phase_ms = {name: sum(p[k] for p in phases) / len(phases) for k, name in enumerate(("projection", "finalize", "update"))}
    return start.elapsed_time(stop), launches, phase_ms, clocks.summary(t0, t1)


def step_roofline(wl, ms_step, phase_ms, peaks, state_elem=4):
    """Where the step stands against its bytes and FLOPs.  bytes_min counts G once (the method's own traffic:
    G, W read, W written, moments read and written); bytes_two_pass counts the second read of G that this
    implementation's two passes make.  frac_vs_min is the fraction of the step's roofline; frac_schedule is
    how close the two-pass schedule runs to its own bytes."""
    two_pass, minimal, update_bytes, flops = step_bytes(wl, state_elem)
    hbm, tc = peaks["hbm_gbs"] * 1e9, peaks["bf16_tflops_sustained"] * 1e12
    t_min = max(minimal / hbm, flops / tc)
    t_2p = max(two_pass / hbm, flops / tc)
    return {"bytes_min": minimal, "bytes_two_pass": two_pass, "gemm_flops": flops,
            "t_roofline_ms": 1e3 * t_min, "frac_vs_min": 1e3 * t_min / ms_step,
            "frac_vs_min_8TBs": 1e3 * max(minimal / 8e12, flops / tc) / ms_step,
            "t_two_pass_ms": 1e3 * t_2p, "frac_schedule": 1e3 * t_2p / ms_step,
            "frac_schedule_8TBs": 1e3 * max(two_pass / 8e12, flops / tc) / ms_step,
            "phase_ms": phase_ms}, update_bytes


def run_ours(args, wl, rank, world, local_rank):
    import torch.distributed as dist
    from paper_2412_05270_b200 import binding as B

    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    flags = (B.FLAG_BF16_STATES if args.bf16_states else 0) | (B.FLAG_KEEP_P if args.keep_p else 0)
    state_elem = 2 if args.bf16_states else 4
    stream = torch.cuda.current_stream()
    peaks = measured_peaks()
    tuning = None
    if args.tuning:
        tuning = B.make_tuning(**{k: int(v) for k, v in (kv.split("=") for kv in args.tuning.split(","))})

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def make(w):
        k = len(w.shapes)
        Ws = [WL.make_weight(w, i, device=dev) for i in range(k)]
        Gs = [WL.make_grad(w, i, 0, device=dev) for i in range(k)]
        opt = B.Apollo(w.shapes, B.config_for(w, flags), device=dev, tuning=tuning)
        opt.set_timing(True)
        return opt, Ws, Gs

    n = len(wl.shapes)
    opt, Ws, Gs = make(wl)
    with ClockSampler(local_rank) as clocks:
        ms_total, launches, phase_ms, clock_summary = time_steps(opt, Ws, Gs, wl, args.steps, args.warmup, stream,
                                                                 barrier, clocks)
        assert opt.status() == B.OK

        # the same step repeated for several seconds: the board settles at its power cap
        sustained = None
        if args.sustain_s > 0:
            k = max(10, int(args.sustain_s * 1e3 / (ms_total / args.steps)))
            ms_s, _, phase_s, clock_s = time_steps(opt, Ws, Gs, wl, k, 0, stream, barrier, clocks)
            sustained = {"steps": k, "seconds": ms_s * 1e-3, "ms_per_step": ms_s / k, "phase_ms": phase_s,
                         "clocks": clock_s}
            assert opt.status() == B.OK

        # gradients at a different address every step (a framework that frees and reallocates them): the step
        # then re-encodes the tensor maps of the moved matrices and uploads its descriptor table again
        moved = None
        if not args.no_moved and args.layers == 0:
            Gs2 = [g.clone() for g in Gs]
            both = (Gs, Gs2)
            for k in range(3):
                opt.step(Ws, both[k & 1], wl.lr, wl.wd, check=False)
            m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            h0 = time.perf_counter()
            m0.record(stream)
            for k in range(args.steps):
                opt.step(Ws, both[k & 1], wl.lr, wl.wd, check=False)
            m1.record(stream)
            barrier()
            h0 = time.perf_counter()
            opt.step(Ws, both[args.steps & 1], wl.lr, wl.wd, check=False)      # one call on an idle stream: its host cost
            host_ms = (time.perf_counter() - h0) * 1e3
            barrier()
            moved = {"ms_per_step": m0.elapsed_time(m1) / args.steps, "host_ms_per_call": host_ms,
                     "what": "every gradient at another address than in the step before; host_ms_per_call is one "
                             "apollo_step call on an idle stream (tensor maps of all matrices encoded again)"}
            assert opt.status() == B.OK
            del Gs2, both

    # end to end: gradients arrive from pinned host memory every step, the limiter norms go back
    e2e_ms = 0.0
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
    workspace = opt.workspace_bytes
    opt.close()
    del opt, Ws, Gs
    torch.cuda.empty_cache()

    # the other lists the metric names, in the same process, each with its own clock window
    also = {}
    for name in ([] if args.no_also or args.layers > 0 else [x for x in args.also.split(",") if x and x != wl.name]):
        w2 = WL.workload(name)
        o2, W2, G2 = make(w2)
        with ClockSampler(local_rank) as c2:
            ms2, _, ph2, cs2 = time_steps(o2, W2, G2, w2, args.steps, args.warmup, stream, barrier, c2)
        assert o2.status() == B.OK
        roof2, _ = step_roofline(w2, ms2 / args.steps, ph2, peaks, state_elem)
        also[name] = {"ms_per_step": ms2 / args.steps, "params": w2.params, "rank": w2.rank, "mode": w2.mode,
                      "value": whole_job_value(w2.params, world, ms2 / args.steps), "workspace_bytes": o2.workspace_bytes,
                      "step_roofline": roof2, "clocks": cs2}
        o2.close()
        del o2, W2, G2
        torch.cuda.empty_cache()

    ranked = [ms_total, e2e_ms] + ([sustained["ms_per_step"]] if sustained else []) + [a["ms_per_step"] for a in also.values()]
    ranked = max_over_ranks(ranked, device=dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    ms_total, e2e_ms = ranked[0], ranked[1]
    at = 2
    if sustained:
        sustained["ms_per_step"] = ranked[at]; at += 1
    for a in also.values():
        a["ms_per_step"] = ranked[at]; at += 1
        a["value"] = whole_job_value(a["params"], world, a["ms_per_step"])

    ms_step = ms_total / args.steps
    roof, update_bytes = step_roofline(wl, ms_step, phase_ms, peaks, state_elem)
    value = whole_job_value(wl.params, world, ms_step)
    upd_ms = phase_ms["update"]
    upd_gbs = update_bytes / (upd_ms * 1e-3) / 1e9
    traffic = UPDATE_TRAFFIC_BYTES_PER_PARAM * wl.params if UPDATE_TRAFFIC_BYTES_PER_PARAM and wl.dtype == "bf16" else None
    line = {
        "metric": "apollo_step_params_per_s", "value": value, "unit": "params/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": {"workload": wl.name, "matrices": n, "params": wl.params, "rank": wl.rank, "mode": wl.mode,
                   "T": wl.T, "lr": wl.lr, "wd": wl.wd, "states": "bf16" if args.bf16_states else "f32", "replicas": world,
                   "p_storage": "kept" if args.keep_p else "per_step", "workspace_bytes": workspace,
                   "tuning": args.tuning or "default", "range_size": RANGE_SIZE,
                   "l2": "inputs (W, G: %.1f GB) exceed L2, no flush" % (2 * wl.params * 2 / 1e9)},
        "roofline": {"bound": "hbm", "kernel": "update_kernel", "achieved": upd_gbs, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": upd_gbs / peaks["hbm_gbs"], "traffic": traffic,
                     "traffic_source": "ncu capture of the first 2 layers, scaled by parameters (not measured in this run)"
                     if traffic else None,
                     "peak_source": peaks["source"], "bytes_per_launch": update_bytes, "ms_per_launch": upd_ms},
        "step_roofline": roof,
        "clocks": clock_summary,
        "gpu_launches": launches,
    }
    if sustained:
        sustained["value"] = whole_job_value(wl.params, world, sustained["ms_per_step"])
        sustained["frac_vs_min"] = roof["t_roofline_ms"] / sustained["ms_per_step"]
        sustained["frac_schedule"] = roof["t_two_pass_ms"] / sustained["ms_per_step"]
        line["sustained"] = sustained
    if moved:
        line["moved_gradients"] = moved
    if also:
        line["also"] = also
    if not args.no_e2e:
        line["e2e"] = {"value": whole_job_value(wl.params, world, e2e_ms), "unit": "params/s",
                       "h2d_bytes_per_step": g_bytes, "d2h_bytes_per_step": n * 16, "ms_per_step": e2e_ms,
                       "note": "bound by the host-to-device copy of the gradients; the weights stay on the device"}
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
    ap.add_argument("--keep-p", action="store_true",
                    help="keep every matrix's projection for its epoch (APOLLO_FLAG_KEEP_P) instead of regenerating it every step")
    ap.add_argument("--range-size", type=int, default=0,
                    help="step the list in ranges of this many matrices with apollo_step_range (measurement aid; 0: apollo_step)")
    ap.add_argument("--tuning", default="", help="apollo_tuning fields, e.g. p_generator=1,scratch_mb=64 (measurement aid)")
    ap.add_argument("--also", default="llama1b,llama7b_mini,llama350m", help="other lists timed in the same run")
    ap.add_argument("--no-also", action="store_true")
    ap.add_argument("--sustain-s", type=float, default=3.0, help="seconds of back-to-back steps for the sustained figure (0: skip)")
    ap.add_argument("--no-moved", action="store_true", help="skip the run with gradients at changing addresses")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    global RANGE_SIZE
    RANGE_SIZE = args.range_size
    if RANGE_SIZE > 0:
        args.no_e2e = args.no_moved = args.no_also = True
        args.sustain_s = 0.0
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
