#!/usr/bin/env python
"""Throughput of the FLuRKA attention forward pass (tokens/s = B*H*N per second) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config c3] [--impl reference]

One step = one whole forward pass (down-projection, key side, query side) over one synthetic batch.
Under torchrun every rank runs its own batch on its own GPU (the path shards over B*H with no
collective), timing is the maximum over ranks, and rank 0 prints one JSON line.
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
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2306_15799_b200 import configs, synth  # noqa: E402

METRIC = "flurka_attn_fwd_tokens_per_s"
UNIT = "tokens/s"
L2_BYTES = 126 * 1024 * 1024


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.tmp = None

    def start(self):
        try:
            self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.tmp, stderr=subprocess.DEVNULL)
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
        self.tmp.flush()
        self.tmp.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.tmp.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def recorded_traffic(stage: str, w):
    """DRAM bytes per launch of a stage kernel from the committed ncu capture (profiles/dram_traffic.json),
    or None when there is no capture for this workload or the kernel source changed since it was taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as fh:
        table = json.load(fh)
    for e in table.get("entries", []):
        if e["stage"] != stage or e["workload"] != w.name:
            continue
        src = os.path.join(ROOT, "paper_2306_15799_b200", "csrc", e["source"])
        with open(src, "rb") as fh:
            if hashlib.sha256(fh.read()).hexdigest() != e["sha256"]:
                return None
        return e["dram_bytes_per_launch"]
    return None


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def rank_workload(w, rank):
    """Weak scaling over B*H: every rank draws its own batch of the same shape from a rank-offset seed."""
    return configs.shrink(w, seed=w.seed + 7919 * rank)


def max_over_ranks(values, world, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (the slowest rank sets the job's time)."""
    if world <= 1:
        return list(values)
    import torch.distributed as dist
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def job_tokens_per_s(w, world, ms_per_step):
    """Whole-job throughput: the tokens all ranks processed in one step over the slowest rank's time."""
    return w.tokens * world / (ms_per_step * 1e-3)


def is_fused(w):
    return isinstance(w, configs.FusedWorkload)


def host_inputs(w):
    return synth.make_fused_inputs(w) if is_fused(w) else synth.make_inputs(w)


def oracle_sample(w, inputs, heads):
    """Times the fp64 oracle (as it stands) on `heads` heads of the workload. Returns seconds."""
    import oracle
    f64 = lambda t: t.double().numpy()
    E, F = f64(inputs["E"]), f64(inputs["F"])
    W = f64(inputs["W"]) if inputs["W"] is not None else None
    t0 = time.perf_counter()
    for i in range(heads):
        b, h = divmod(i % (w.B * w.H), w.H)
        if is_fused(w):
            cols = slice(h * w.d, (h + 1) * w.d)
            oracle.fused_head(f64(inputs["Xq"][b]), f64(inputs["Xk"][b]), f64(inputs["Xv"][b]), E, F,
                              f64(inputs["Wq"][:, cols]), f64(inputs["Wk"][:, cols]), f64(inputs["Wv"][:, cols]), W, w.variant)
        else:
            oracle.head(f64(inputs["Q"][b, h]), f64(inputs["K"][b, h]), f64(inputs["V"][b, h]), E, F, W, w.variant)
    return time.perf_counter() - t0


def run_reference(args, w):
    """--impl reference: the CPU oracle on the machine's host cores, a bounded sample per step."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    import oracle
    oracle.build()
    small = configs.shrink(w, B=1, H=1)          # one head per step; E, F, W keep their full size
    inputs = host_inputs(small)
    for _ in range(args.warmup):
        oracle_sample(small, inputs, 1)
    t = 0.0
    for _ in range(args.steps):
        t += oracle_sample(small, inputs, 1)
    ms = 1e3 * t / max(args.steps, 1)
    value = small.N / (ms * 1e-3)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "sample": "one head (N=%d tokens) per step" % small.N},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                         "sample": "one head of %s per step, fp64 C + OpenMP" % w.name},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def measure(w, args, binding, rank, world, local, with_e2e=True):
    """Times `args.steps` forward passes of workload `w` on this rank's GPU: CUDA events on the launch
    stream around every step, a second pass with the library's per-stage events, the clocks sampled
    meanwhile, and (optionally) the host-buffer entry point end to end."""
    import torch.distributed as dist

    # every rank draws its own batch (weak scaling over B*H); same recipe, rank-offset seed
    wr = rank_workload(w, rank)
    host = host_inputs(wr)
    fused = is_fused(w)
    laid_out = dict(host)
    if args.layout == "bnhd" and not fused:
        for n in ("Q", "K", "V"):
            laid_out[n] = host[n].transpose(1, 2).contiguous()
    # one X serves as queries, keys and values when the workload says so: pinned, copied and counted once
    names = [n for n in laid_out if not (fused and w.shared_x and n in ("Xk", "Xv"))]
    pinned = {n: (laid_out[n].pin_memory() if laid_out[n] is not None else None) for n in names}
    dev = {n: (t.cuda(non_blocking=True) if t is not None else None) for n, t in pinned.items()}
    if fused and w.shared_x:
        dev["Xk"] = dev["Xv"] = dev["Xq"]
    out = torch.empty((w.B, w.N, w.H, w.d), dtype=dev["E"].dtype, device="cuda") if fused else torch.empty_like(dev["Q"])
    in_bytes = sum(t.numel() * t.element_size() for n, t in dev.items() if t is not None and n in names)
    flush = None
    if in_bytes < 2 * L2_BYTES:
        flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()

    def step():
        if fused:
            binding.flurka_forward_fused(dev["Xq"], dev["Xk"], dev["Xv"], dev["E"], dev["F"], dev["Wq"], dev["Wk"],
                                         dev["Wv"], dev["W"], w.variant, w.H, out=out, stream=stream)
        else:
            binding.flurka_forward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], w.variant,
                                   out=out, stream=stream, layout=args.layout)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # the clock sampler runs from the warm-up to the end of the stage-timing pass; a steady load of
    # untimed steps before the timed region gives nvidia-smi something to see (steps last < 1 ms)
    sampler = ClockSampler(local)
    sampler.start()
    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            step()
        t_load = time.perf_counter()
        while not args.no_load and time.perf_counter() - t_load < 0.6:
            for _ in range(20):
                step()
            stream.synchronize()
    barrier()

    # ---- timed region: K steps, CUDA events on the launch stream around each step
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    barrier()
    with torch.cuda.stream(stream):
        for i in range(args.steps):
            if flush is not None:
                flush.zero_()
            starts[i].record(stream)
            step()
            stops[i].record(stream)
    barrier()
    step_ms = [s.elapsed_time(e) for s, e in zip(starts, stops)]
    res = {"step_ms": step_ms, "total_ms": sum(step_ms), "in_bytes": in_bytes,
           "out_bytes": out.numel() * out.element_size(), "flushed": flush is not None,
           "launches": binding.flurka_last_launches() * args.steps,
           "path": {1: "simt", 2: "tensor"}.get(binding.flurka_last_path(), "?")}

    # ---- per-stage durations (same inputs, events inside the library between the stages)
    binding.flurka_set_stage_timing(True)
    stage_ms = [0.0, 0.0, 0.0]
    with torch.cuda.stream(stream):
        for _ in range(args.steps):
            if flush is not None:
                flush.zero_()
            step()
            ms3 = binding.flurka_last_stage_ms()
            stage_ms = [a + b for a, b in zip(stage_ms, ms3)]
    binding.flurka_set_stage_timing(False)
    res["stage_ms"] = [x / args.steps for x in stage_ms]
    torch.cuda.synchronize()
    res["clocks"] = sampler.stop()

    # ---- end to end: host buffers in, host buffer out, through the host entry point
    res["e2e_ms"] = None
    if with_e2e:
        host_out = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        e2e_steps = max(1, min(args.steps, 5))

        def e2e_step():
            if fused:
                # the entry point with un-projected inputs takes device buffers: the copies are made here,
                # on the launch stream, from and to pinned host memory
                with torch.cuda.stream(stream):
                    for n in names:
                        if pinned[n] is not None:
                            dev[n].copy_(pinned[n], non_blocking=True)
                    step()
                    host_out.copy_(out, non_blocking=True)
                stream.synchronize()
            else:
                binding.flurka_forward_host(pinned["Q"], pinned["K"], pinned["V"], pinned["E"], pinned["F"], pinned["W"],
                                            w.variant, out=host_out, stream=stream, layout=args.layout)

        e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        torch.cuda.synchronize()
        res["e2e_ms"] = 1e3 * (time.perf_counter() - t0) / e2e_steps
    res["status"] = binding.flurka_last_status()
    res["host_inputs"] = (wr, host)
    return res


def backward_work(w):
    """Algorithmic FLOPs and compulsory bytes of one backward pass (all heads): the forward's stage 1 and
    key side again, the query side's four products (S, dO a^T, dQ, da), the key side's four, and the four
    products with E, F, K, V that give dK, dV, dE, dF; bytes: Q, K, V, dO in, dQ, dK, dV out, E, F in, dE, dF out."""
    N, d, k, m, BH, s = w.N, w.d, w.k, w.m, w.B * w.H, w.elem_bytes
    perf = w.variant == configs.PERFORMER
    p = m if perf else d
    flops = BH * (12 * N * k * d + (8 * N * p * d if perf else 0) + (12 * k * p * d if perf else 0))
    byts = 7 * BH * N * d * s + 4 * k * N * s
    return flops, byts


def measure_backward(w, args, binding, rank, world):
    """Times flurka_backward on workload `w` (device-resident inputs, CUDA events on the launch stream, the
    same warm-up and L2 rules as the forward)."""
    wr = rank_workload(w, rank)
    host = host_inputs(wr)
    dev = {n: (t.cuda() if t is not None else None) for n, t in host.items()}
    gen = torch.Generator().manual_seed(wr.seed + 17)
    dO = torch.randn(host["Q"].shape, generator=gen, dtype=torch.float32).to(host["Q"].dtype).cuda()
    in_bytes = sum(t.numel() * t.element_size() for t in dev.values() if t is not None) + dO.numel() * dO.element_size()
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda") if in_bytes < 2 * L2_BYTES else None
    stream = torch.cuda.Stream()
    grads = None

    def step():
        return binding.flurka_backward(dev["Q"], dev["K"], dev["V"], dev["E"], dev["F"], dev["W"], dO, w.variant,
                                       stream=stream, out=grads)

    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        grads = step()
        for _ in range(max(args.warmup, 3)):
            step()
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    with torch.cuda.stream(stream):
        for i in range(args.steps):
            if flush is not None:
                flush.zero_()
            starts[i].record(stream)
            step()
            stops[i].record(stream)
    torch.cuda.synchronize()
    step_ms = [a.elapsed_time(b) for a, b in zip(starts, stops)]
    return {"step_ms": step_ms, "total_ms": sum(step_ms), "launches": binding.flurka_last_launches() * args.steps,
            "path": {1: "simt", 2: "tensor", 3: "tensor stage 1 and projections, cuda-core query side"}.get(binding.flurka_last_path(), "?"),
            "status": binding.flurka_last_status(), "flushed": flush is not None}


def backward_block(w, rb, peaks, steps, world):
    ms = rb["total_ms"] / steps
    flops, byts = backward_work(w)
    t_t, t_h = flops / (peaks["bf16_tflops"] * 1e12), byts / (peaks["hbm_gbs"] * 1e9)
    return {"value": job_tokens_per_s(w, world, ms), "unit": UNIT, "ms_per_step": ms,
            "step_ms_min": min(rb["step_ms"]), "step_ms_median": statistics.median(rb["step_ms"]),
            "path": rb["path"], "gpu_launches": rb["launches"], "device_status": rb["status"],
            "path_roofline": {"flops": flops, "bytes": byts, "t_tensor_us": t_t * 1e6, "t_hbm_us": t_h * 1e6,
                              "frac": max(t_t, t_h) / (ms * 1e-3),
                              "peak_source": "of " + peaks["source"] + " (burst GEMM figure)"}}


def stage_work(w):
    """Algorithmic FLOPs, bytes and exponentials of the three stages (all heads), and their names."""
    N, d, k, m, BH, s = w.N, w.d, w.k, w.m, w.B * w.H, w.elem_bytes
    perf = w.variant == configs.PERFORMER
    p = m if perf else d
    flops = [4 * N * k * d * BH,
             (2 * k * d * m + 2 * k * m * d) * BH if perf else 2 * k * d * d * BH,
             (2 * N * d * m + 2 * N * m * d) * BH if perf else 2 * N * d * d * BH]
    byts = [2 * BH * N * d * s + 2 * k * N * s + 2 * BH * k * d * 4,
            2 * BH * k * d * 4 + m * d * s + BH * p * (d * 2 + 4),
            2 * BH * N * d * s + m * d * s + BH * p * (d * 2 + 4)]
    exps = [0, k * p * BH, N * p * BH]
    names = ["down_projection", "key_side", "query_side"]
    if is_fused(w):
        # stage 0 = contraction of the un-projected inputs and the three linear maps; its bytes: X, E, F, the
        # maps, K' and V'; the query side then reads Xq W^Q from the workspace
        dm, Hd = w.dm, w.H * w.d
        names[0] = "contraction_and_linear_maps"
        flops[0] = (4 * N * k * dm + 2 * N * dm * Hd + 4 * k * dm * Hd) * w.B
        byts[0] = w.B * N * dm * s * (1 if w.shared_x else 3) + 2 * k * N * s + 3 * dm * Hd * s + 2 * BH * k * d * 4
    return names, flops, byts, exps


def rooflines(w, res, peaks, steps, world, exp_rate):
    """The `roofline` object (dominant kernel) and the `path_roofline` object (whole forward) of a run.

    Both follow one definition: time at the roofline = max(FLOPs / measured dense bf16 peak, bytes / measured
    HBM bandwidth); frac = that time / measured time.  The GEMM denominator is the burst figure; the fraction
    against the seconds-long (power-capped) figure is given beside it."""
    ms_per_step = res["total_ms"] / steps
    names, sflops, sbytes, sexps = stage_work(w)
    stage_ms = res["stage_ms"]
    dom = max(range(3), key=lambda i: stage_ms[i])
    dt = stage_ms[dom] * 1e-3
    tf, tf_s, hbm = peaks["bf16_tflops"] * 1e12, peaks["bf16_tflops_sustained"] * 1e12, peaks["hbm_gbs"] * 1e9
    t_tensor, t_hbm = sflops[dom] / tf, sbytes[dom] / hbm
    if t_hbm >= t_tensor:
        roofline = {"bound": "hbm", "achieved": sbytes[dom] / dt / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    else:
        roofline = {"bound": "tensor", "achieved": sflops[dom] / dt / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    roofline["frac"] = max(t_tensor, t_hbm) / dt
    roofline["frac_sustained"] = max(sflops[dom] / tf_s, t_hbm) / dt
    roofline["frac_tensor"] = t_tensor / dt
    roofline["frac_hbm"] = t_hbm / dt
    roofline["traffic"] = recorded_traffic(names[dom], w)
    roofline["kernel"] = names[dom]
    roofline["peak_source"] = "of " + peaks["source"] + " (burst GEMM figure)"
    roofline["stage_ms"] = dict(zip(names, stage_ms))
    if sexps[dom] and exp_rate:
        # a third limit the FLOP / byte roofline does not count: the exponentials of this stage against the
        # rate a loop of nothing but independent ex2.approx chains reaches on this GPU (measured in this run)
        roofline["exp"] = {"achieved_gexp_s": sexps[dom] / dt / 1e9, "measured_peak_gexp_s": exp_rate,
                           "frac": sexps[dom] / dt / 1e9 / exp_rate}
    flops, byts = w.flops(), w.compulsory_bytes()
    t_t, t_h = flops / tf, byts / hbm
    path = {"flops": flops, "bytes": byts, "t_tensor_us": t_t * 1e6, "t_hbm_us": t_h * 1e6,
            "frac": max(t_t, t_h) / (ms_per_step * 1e-3),
            "frac_sustained": max(flops / tf_s, t_h) / (ms_per_step * 1e-3),
            "tensor_peak_tflops": peaks["bf16_tflops"], "peak_source": "of " + peaks["source"] + " (burst GEMM figure)"}
    return roofline, path


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="", help="workload (default: c3, followed by a c4 block under `also`)")
    ap.add_argument("--impl", default="flurka", choices=["flurka", "reference"])
    ap.add_argument("--path", default="auto", choices=["auto", "simt", "tensor"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="default run: skip the second target configuration (c4)")
    ap.add_argument("--no-backward", action="store_true", help="skip the backward-pass block under `also`")
    ap.add_argument("--heads", default="", help="B,H override: a smaller batch of the same workload (profiling)")
    ap.add_argument("--no-load", action="store_true", help="skip the sustained-load phase before timing (profiling)")
    ap.add_argument("--layout", default="bhnd", choices=["bhnd", "bnhd"],
                    help="Q, K, V, out as [B,H,N,d] (default) or [B,N,H,d]")
    args = ap.parse_args()
    default_run = args.config == ""
    w = configs.get(args.config or "c3")
    if args.heads:
        b, h = (int(x) for x in args.heads.split(","))
        w = configs.shrink(w, name="%s_B%d_H%d" % (w.name, b, h), B=b, H=h)

    if args.impl == "reference":
        run_reference(args, w)
        return

    from paper_2306_15799_b200 import binding, build

    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the CUDA library has no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    binding.load()
    binding.flurka_set_path({"auto": binding.PATH_AUTO, "simt": binding.PATH_SIMT, "tensor": binding.PATH_TENSOR}[args.path])

    res = measure(w, args, binding, rank, world, local)
    total_ms, e2e_ms = max_over_ranks([res["total_ms"], res["e2e_ms"]], world, device="cuda")
    res["total_ms"] = total_ms
    ms_per_step = total_ms / args.steps
    wr, host = res.pop("host_inputs")

    also = None
    if default_run and not args.no_also and not args.heads:
        # the second configuration the roofline target is stated on, timed the same way (no end-to-end
        # leg, no oracle leg); every rank runs it, the slowest one counts
        w4 = configs.get("c4")
        r4 = measure(w4, args, binding, rank, world, local, with_e2e=False)
        r4.pop("host_inputs")
        r4["total_ms"] = max_over_ranks([r4["total_ms"]], world, device="cuda")[0]
        also = (w4, r4)

    bwd = None
    if not args.no_backward and not is_fused(w):
        # the backward pass of the same workload (gradients of Q, K, V, E, F), timed the same way
        bwd = measure_backward(w, args, binding, rank, world)
        bwd["total_ms"] = max_over_ranks([bwd["total_ms"]], world, device="cuda")[0]

    if rank == 0:
        peaks = measured_peaks()
        exp_rate = binding.flurka_measure_ex2_rate()          # Gexp/s of a bare ex2.approx loop on this GPU, now
        tokens = w.tokens * world
        value = job_tokens_per_s(w, world, ms_per_step)
        roofline, path_roofline = rooflines(w, res, peaks, args.steps, world, exp_rate)
        clocks = res["clocks"]
        step_ms = res["step_ms"]

        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.io == "bf16" else "f32",
            "data": "synthetic",
            "config": {"workload": w.name, "variant": "performer" if w.variant == configs.PERFORMER else "rnn",
                       "B": w.B, "H": w.H, "N": w.N, "d": w.d, "k": w.k, "m": w.m, "io": w.io, "path": res["path"],
                       "layout": "bnhd" if is_fused(w) else args.layout, **({"dm": w.dm, "shared_x": w.shared_x} if is_fused(w) else {}),
                       "parallelism": "replicated batches over B*H, no collective" if world > 1 else "single GPU",
                       "l2": "inputs (%.0f MB) exceed L2" % (res["in_bytes"] / 1e6) if not res["flushed"]
                             else "L2 flushed between steps (252 MiB write)"},
            "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"]},
            "e2e": {"value": tokens / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": res["in_bytes"], "d2h_bytes_per_step": res["out_bytes"]},
            "gpu_launches": res["launches"],
            "roofline": roofline,
            "path_roofline": path_roofline,
            "step_ms_min": min(step_ms), "step_ms_median": statistics.median(step_ms),
            "device_status": res["status"],
        }
        if also is not None:
            w4, r4 = also
            rf4, pr4 = rooflines(w4, r4, peaks, args.steps, world, exp_rate)
            ms4 = r4["total_ms"] / args.steps
            line["also"] = {w4.name: {
                "value": job_tokens_per_s(w4, world, ms4), "unit": UNIT, "ms_per_step": ms4,
                "step_ms_min": min(r4["step_ms"]), "step_ms_median": statistics.median(r4["step_ms"]),
                "config": {"workload": w4.name, "variant": "performer", "B": w4.B, "H": w4.H, "N": w4.N, "d": w4.d,
                           "k": w4.k, "m": w4.m, "io": w4.io, "path": r4["path"], "layout": args.layout,
                           "l2": "inputs (%.0f MB) exceed L2" % (r4["in_bytes"] / 1e6)},
                "clocks": {"sm_mhz": r4["clocks"]["sm_mhz"], "sm_max_mhz": r4["clocks"]["sm_max_mhz"],
                           "reasons": r4["clocks"]["reasons"]},
                "gpu_launches": r4["launches"], "roofline": rf4, "path_roofline": pr4, "device_status": r4["status"]}}
        if bwd is not None:
            line.setdefault("also", {})["backward_" + w.name] = backward_block(w, bwd, peaks, args.steps, world)
        if not args.no_cpu_baseline and world == 1:
            import oracle
            oracle.build()
            t1 = oracle_sample(wr, host, 1)                        # warm + calibrate
            heads = max(1, int(25.0 / max(t1, 1e-3)))              # 10 to 25 s of CPU work (the first, cold pass over-estimates)
            tt = oracle_sample(wr, host, heads)
            line["cpu_baseline"] = {"value": heads * w.N / tt, "unit": UNIT, "cores": oracle.threads(),
                                    "kind": "oracle",
                                    "sample": "%d head passes over the %d heads of %s, all %d rows each, %.1f s" % (heads, w.B * w.H, w.name, w.N, tt)}
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
