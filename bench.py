#!/usr/bin/env python
"""Benchmark of the gated N-D long convolution (HyenaND FFT hot path) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one forward of the whole path (gate+pad, forward transforms of k*v
and h, spectral product, inverse, crop, output gate) over one synthetic batch of
the chosen workload.  Rank 0 prints ONE JSON line.  `value` is B*C*L elements
per second over all ranks with inputs resident in HBM; `e2e` is the same metric
through hyenand_forward_host (host buffers, copies inside the timed region).
With more than one GPU every rank runs its own batch of the same shape (weak
scaling, no collective on the data path).

--impl reference times the CPU oracle (fp64, radix-2 FFT path) on a bounded
sample of the same workload on the host cores; it is a deliberately plain
program, reported as a baseline only.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2607_19378_b200 import workloads as W  # noqa: E402

ALL_WORKLOADS = {**W.WORKLOADS, **W.EXTRA_WORKLOADS}
METRIC = "hyenand_forward_throughput"
UNIT = "Gelem/s"
DEFAULT_WORKLOAD = "volume3d"
FP32_LANES_PER_SM = 128


# ---- roofline bookkeeping ----------------------------------------------------------------

def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured", float(d.get("sm_max_mhz", 1965.0))
    return 6650.0, "fallback", 1965.0


def fp32_peak_tflops(sm_count: int, sm_max_mhz: float) -> float:
    # 2 flops (FMA) x 128 FP32 lanes x SMs x max SM clock
    return 2.0 * FP32_LANES_PER_SM * sm_count * sm_max_mhz * 1e6 / 1e12


def padded_dims(w: W.Workload):
    """Transform size per axis: the grid itself with periodic boundaries, else the next power of two >= 2L-1."""
    return [L if w.circular else 1 << max(0, (2 * L - 2).bit_length()) for L in w.dims]


def op_algorithmic(w: W.Workload):
    """Minimal bytes (q,k,v,h,y once) and nominal flops (2.5 P log2 P per real transform:
    k*v forward and the inverse per slice, h forward per filter) of one forward."""
    s = 4 if w.dtype == "f32" else 2
    E = w.elements
    hcount = w.C if w.h_shared else w.B * w.C
    hbytes = hcount * math.prod(w.taps) * s
    P = math.prod(padded_dims(w))
    transforms = 2 * w.B * w.C + hcount
    flops = transforms * 2.5 * P * math.log2(P) if P > 1 else 0.0
    return 4 * E * s + hbytes, flops, P


# ---- clocks ---------------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc = None
        self.lines = []
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self, t0: float, t1: float):
        """Median SM clock and the throttle reasons seen between wall-clock t0 and t1."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.12)
        self.proc.terminate()
        try:
            text, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            return out
        import datetime
        sm, reasons, smax = [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in text.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                if not (t0 - 0.05 <= ts <= t1 + 0.05):
                    continue
                sm.append(float(parts[1]))
                smax = float(parts[2])
                for n, val in zip(names, parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=smax, reasons=sorted(reasons), samples=len(sm))
        return out


# ---- our arm ----------------------------------------------------------------------------------

def time_workload(w: W.Workload, steps: int, warmup: int, dist, device, want_kernels: bool,
                  sampler_device=None):
    """Device-resident timing of `steps` forwards.  Returns a dict of raw measurements."""
    from paper_2607_19378_b200 import hyenand as hn
    q, k, v, h = W.make_inputs(w, device=device)
    y = torch.empty_like(q)
    plan = hn.Plan(w.dims, w.B, w.C, causal=w.causal, dtype=w.torch_dtype, circular=w.circular)
    stream = torch.cuda.current_stream()
    for _ in range(max(warmup, 3)):
        plan.forward(q, k, v, h, y)
    torch.cuda.synchronize()
    sampler = ClockSampler(sampler_device) if sampler_device is not None else None
    if sampler is not None:
        time.sleep(0.6)                       # let nvidia-smi start sampling
        for _ in range(3):                    # re-warm after the pause
            plan.forward(q, k, v, h, y)
        torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps - 1)]
    e0.record(stream)
    for i in range(steps):
        plan.forward(q, k, v, h, y)
        if i < steps - 1:
            marks[i].record(stream)               # per-step times for the median and the minimum
    e1.record(stream)
    torch.cuda.synchronize()
    t1 = time.time()
    if dist is not None:
        dist.barrier()
    ms = e0.elapsed_time(e1) / steps
    seq = [e0] + marks + [e1]
    per_step = sorted(a.elapsed_time(b) for a, b in zip(seq[:-1], seq[1:]))
    kernels = []
    if want_kernels:
        # Per-kernel durations: the same K forwards once more, every launch bracketed by CUDA events on its
        # stream; a plan with several lanes enqueues its groups one after the other meanwhile (mode 2), so a
        # kernel's duration is not stretched by another lane's kernels sharing the GPU.
        hn.hyenand_plan_set_timing(plan.handle, 2)
        for i in range(steps):
            plan.forward(q, k, v, h, y)
        torch.cuda.synchronize()
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if sampler is not None else None
    if want_kernels:
        for kid in range(hn.hyenand_plan_kernel_count(plan.handle)):
            name, launches, nbytes, flops = hn.hyenand_plan_kernel_info(plan.handle, kid, w.h_shared)
            tot_ms, n = hn.hyenand_plan_kernel_time(plan.handle, kid)
            if n > 0:
                kernels.append({"name": name, "launches_per_step": n / steps, "ms_per_step": tot_ms / steps,
                                "ms_per_launch": tot_ms / n, "bytes_per_launch": nbytes / launches,
                                "flops_per_launch": flops / launches})
        hn.hyenand_plan_set_timing(plan.handle, False)
    status = hn.hyenand_plan_device_status(plan.handle)
    damage = hn.hyenand_plan_guard_damage(plan.handle)
    if status != 0 or damage != 0:
        raise SystemExit(f"{w.name}: device status {status} (a bounded wait gave up) / {damage} damaged guard bytes: "
                         "the timing is void")
    group, lanes = hn.hyenand_plan_groups(plan.handle)
    res = {"ms": ms, "ms_median": per_step[len(per_step) // 2], "ms_min": per_step[0], "clocks": clocks, "kernels": kernels,
           "device_status": status, "guard_damage": damage, "slices_per_group": group, "lanes": lanes,
           "launches": hn.hyenand_plan_launches(plan.handle, w.h_shared),
           "path": hn.hyenand_plan_path(plan.handle),
           "workspace_bytes": hn.hyenand_plan_workspace_bytes(plan.handle)}
    return res, plan, (q, k, v, h, y)


def time_e2e(w: W.Workload, plan, tensors, steps: int, dist):
    q, k, v, h, y = tensors
    host = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in (q, k, v, h, y)]
    for dst, src in zip(host[:4], (q, k, v, h)):
        dst.copy_(src)
    torch.cuda.synchronize()
    plan.forward_host(*host)                          # allocates the staging buffers, warms up
    plan.forward_host(*host)
    if dist is not None:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        plan.forward_host(*host)                      # returns after y is back on the host
    dt = (time.perf_counter() - t0) / steps
    if dist is not None:
        dist.barrier()
    h2d = sum(t.numel() * t.element_size() for t in host[:4])
    d2h = host[4].numel() * host[4].element_size()
    return dt * 1e3, h2d, d2h


def cufft_composition(w: W.Workload, tensors, reps: int = 3):
    """Reference point only (never on the product path): the same operator written as a composition of
    library calls -- torch.fft (cuFFT) real transforms in fp32 on the padded grid, spectral product,
    inverse, crop, gate -- on the same device-resident inputs, in chunks of slices that bound its memory.
    Returns its time per forward and its error against our result."""
    q, k, v, h, y = tensors
    nd = len(w.dims)
    P = padded_dims(w)
    S = w.B * w.C
    axes = tuple(range(1, nd + 1))
    qf, kf, vf = (t.reshape(S, *w.dims) for t in (q, k, v))
    hf = h.reshape(-1, *h.shape[-nd:])                        # [S or C, K...]
    per_slice = 4 * 6 * int(torch.tensor(P).prod())           # bytes of fp32 work arrays per slice, roughly
    chunk = max(1, min(S, int(4e9) // max(per_slice, 1)))
    out = torch.empty_like(qf)
    crop0 = [0 if (w.causal or w.circular) else L - 1 for L in w.dims]

    def run():
        for s0 in range(0, S, chunk):
            s1 = min(S, s0 + chunk)
            u = kf[s0:s1].float() * vf[s0:s1].float()
            if w.h_shared:
                idx = torch.arange(s0, s1, device=q.device) % w.C
                hh = hf[idx].float()
            else:
                hh = hf[s0:s1].float()
            Y = torch.fft.irfftn(torch.fft.rfftn(u, s=P, dim=axes) * torch.fft.rfftn(hh, s=P, dim=axes), s=P, dim=axes)
            sl = (slice(None),) + tuple(slice(c, c + L) for c, L in zip(crop0, w.dims))
            out[s0:s1] = (qf[s0:s1].float() * Y[sl]).to(out.dtype)

    run()
    if q.is_cuda:
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            run()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
    else:                                                     # host tensors: only the unit test comes here
        t0 = time.perf_counter()
        for _ in range(reps):
            run()
        ms = (time.perf_counter() - t0) / reps * 1e3
    a, b = out.reshape(-1)[:1 << 24].double(), y.reshape(-1)[:1 << 24].double()
    diff = float((a - b).norm() / b.norm().clamp_min(1e-300))
    return {"kind": "torch.fft (cuFFT) composition, fp32, same inputs", "ms_per_step": ms,
            "value": w.elements / (ms * 1e-3) / 1e9, "unit": UNIT, "slices_per_chunk": chunk,
            "rel_l2_vs_ours_first_16M": diff}


def cpu_oracle_sample(w: W.Workload, budget_s: float = 15.0):
    """Times the oracle (as it stands) on a bounded sample of slices of the workload."""
    import oracle
    threads = oracle.threads()
    mode = w.mode

    def run(n_slices):
        ws = w.scaled(B=1, C=n_slices)
        q, k, v, h = W.make_inputs(ws, device="cpu")
        t0 = time.perf_counter()
        oracle.conv_fft(q, k, v, h, mode)
        return time.perf_counter() - t0, ws.elements

    S = w.B * w.C
    n = min(S, threads)
    dt, elems = run(n)
    if dt < budget_s / 3 and n < S:
        n2 = min(S, max(n, int(n * (budget_s / max(dt, 1e-3)) // threads * threads)))
        if n2 > n:
            n = n2
            dt, elems = run(n)
    return {"value": elems / dt / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{n} of {S} (b,c) slices of {w.name}, oracle FFT path (fp64, radix-2), {dt:.1f} s"}


def roofline_of(kern, hbm_gbs, peak_src, fp32_tf, traffic):
    t_h = kern["bytes_per_launch"] / (hbm_gbs * 1e9)
    t_a = kern["flops_per_launch"] / (fp32_tf * 1e12)
    dur = kern["ms_per_launch"] * 1e-3
    if t_h >= t_a:
        ach = kern["bytes_per_launch"] / dur / 1e9
        return {"kernel": kern["name"], "bound": "hbm", "achieved": ach, "peak": hbm_gbs, "unit": "GB/s",
                "frac": ach / hbm_gbs, "traffic": traffic, "peak_source": f"of {peak_src}"}
    ach = kern["flops_per_launch"] / dur / 1e12
    return {"kernel": kern["name"], "bound": "alu", "achieved": ach, "peak": fp32_tf, "unit": "TFLOP/s",
            "frac": ach / fp32_tf, "traffic": traffic,
            "peak_source": "derived: 2 x 128 FP32 lanes x SMs x max SM clock"}


def load_traffic(workload: str, kernel: str):
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    try:
        with open(path) as f:
            return json.load(f).get(workload, {}).get(kernel)
    except Exception:
        return None


def workload_for_rank(w: W.Workload, rank: int, world: int) -> W.Workload:
    """Weak scaling: every rank runs a full batch of the same shape, drawn from its own seed."""
    from dataclasses import replace
    return w if world == 1 else replace(w, seed=w.seed + 100 * rank)


def max_over_ranks(values, dist, device):
    """Element-wise maximum of per-rank timings (the slowest rank defines the step time)."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def aggregate_throughput(elements_per_rank: int, world: int, ms: float) -> float:
    """Whole-job Gelem/s: all ranks' elements over the slowest rank's time."""
    return elements_per_rank * world / (ms * 1e-3) / 1e9


def spawn_command(args, port: int):
    """argv that runs this benchmark as args.gpus ranks on this node (one process per GPU)."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__),
           "--gpus", str(args.gpus), "--steps", str(args.steps), "--warmup", str(args.warmup),
           "--workload", args.workload, "--impl", args.impl]
    if args.batch is not None:
        cmd += ["--batch", str(args.batch)]
    if args.channels is not None:
        cmd += ["--channels", str(args.channels)]
    for flag, on in (("--no-all", args.no_all), ("--no-cpu", args.no_cpu), ("--no-cufft", args.no_cufft)):
        if on:
            cmd.append(flag)
    return cmd


def main_ours(args):
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # called without a launcher: start the ranks ourselves
        if torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"--gpus {args.gpus} but only {torch.cuda.device_count()} CUDA device(s) are visible")
        import socket
        with socket.socket() as sock:
            sock.bind(("127.0.0.1", 0))
            port = sock.getsockname()[1]
        raise SystemExit(subprocess.call(spawn_command(args, port)))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} does not match WORLD_SIZE={world}")
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    w = ALL_WORKLOADS[args.workload].scaled(B=args.batch, C=args.channels)
    w = workload_for_rank(w, rank, world)
    hbm_gbs, peak_src, sm_max = measured_peaks()
    props = torch.cuda.get_device_properties(local)
    fp32_tf = fp32_peak_tflops(props.multi_processor_count, sm_max)

    res, plan, tensors = time_workload(w, args.steps, args.warmup, dist, device, True, sampler_device=local)
    ms = res["ms"]
    e2e_ms, h2d, d2h = time_e2e(w, plan, tensors, max(2, min(args.steps, 5)), dist)
    ms, e2e_ms = max_over_ranks([ms, e2e_ms], dist, device)
    plan.close()
    cufft_ref = None
    if world == 1 and not args.no_cufft:
        try:
            cufft_ref = cufft_composition(w, tensors)
        except Exception as exc:                              # reference point only: never fails the bench
            cufft_ref = {"unavailable": repr(exc)[:200]}
    del tensors
    torch.cuda.empty_cache()

    total_elems = w.elements * world
    nbytes, flops, P = op_algorithmic(w)
    t_hbm = nbytes / (hbm_gbs * 1e9) * 1e3
    t_alu = flops / (fp32_tf * 1e12) * 1e3
    kernels = sorted(res["kernels"], key=lambda kk: -kk["ms_per_step"])
    dom = kernels[0] if kernels else None
    out = {
        "metric": METRIC, "value": aggregate_throughput(w.elements, world, ms), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
        "ms_per_step_median": res["ms_median"], "ms_per_step_min": res["ms_min"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "io_dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "dims": list(w.dims), "B": w.B, "C": w.C, "causal": w.causal, "circular": w.circular,
                   "h_shared_over_batch": w.h_shared, "padded_points_per_slice": P,
                   "l2": "inputs larger than L2 (no flush needed)" if nbytes > 126e6 else "fits L2; latency-bound",
                   "path": res["path"], "slices_per_group": res["slices_per_group"], "lanes": res["lanes"],
                   "per_gpu_batch": "fixed (each rank runs the full workload)"},
        "device_status": res["device_status"], "guard_damage": res["guard_damage"],
        "kernel_timing": "CUDA events around every launch in a second pass of the same K forwards, lanes serialised",
        "clocks": res["clocks"],
        "e2e": {"value": aggregate_throughput(w.elements, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": res["launches"] * args.steps,
        "roofline": roofline_of(dom, hbm_gbs, peak_src, fp32_tf, load_traffic(w.name, dom["name"])) if dom else None,
        "op_roofline": {"t_hbm_ms": t_hbm, "t_fp32_ms": t_alu, "roofline_ms": max(t_hbm, t_alu),
                        "frac": max(t_hbm, t_alu) / ms, "hbm_peak_gbs": hbm_gbs, "hbm_peak_source": peak_src,
                        "fp32_peak_tflops": fp32_tf, "min_bytes": nbytes, "nominal_flops": flops},
        "kernels": [{"name": kk["name"], "launches_per_step": kk["launches_per_step"],
                     "ms_per_step": round(kk["ms_per_step"], 5),
                     "share": kk["ms_per_step"] / max(sum(x["ms_per_step"] for x in kernels), 1e-12),
                     "GBps_algorithmic": kk["bytes_per_launch"] / (kk["ms_per_launch"] * 1e-3) / 1e9,
                     "TFLOPs_nominal": kk["flops_per_launch"] / (kk["ms_per_launch"] * 1e-3) / 1e12}
                    for kk in kernels],
        "workspace_bytes": res["workspace_bytes"],
    }
    if cufft_ref is not None:
        out["cufft_reference"] = cufft_ref
    if world == 1 and rank == 0:
        if not args.no_all:
            table = []
            for name, ww in W.WORKLOADS.items():
                if name == w.name:
                    r_ms, path = ms, res["path"]
                else:
                    r, p2, tens = time_workload(ww, max(3, min(args.steps, 10)), 3, None, device, False)
                    r_ms, path = r["ms"], r["path"]
                    p2.close()
                    del tens, p2
                    torch.cuda.empty_cache()
                nb, fl, _ = op_algorithmic(ww)
                th, ta = nb / (hbm_gbs * 1e9) * 1e3, fl / (fp32_tf * 1e12) * 1e3
                table.append({"workload": name, "ms": r_ms, "gelem_s": ww.elements / (r_ms * 1e-3) / 1e9,
                              "t_hbm_ms": th, "t_fp32_ms": ta, "roofline_frac": max(th, ta) / r_ms, "path": path})
            out["all_workloads"] = table
            # the rows built around the hot path, each timed on its own benchmark mode (few steps: reported, not the headline)
            import copy
            rows = []
            for op, wl, fn in (("conv (circular mode)", "periodic2d", None), ("mixer", "volume3d", measure_mixer),
                               ("synth", "volume3d", measure_synth), ("backward", "volume3d", measure_backward)):
                try:
                    if fn is None:
                        r, p2, tens = time_workload(ALL_WORKLOADS[wl], 5, 3, None, device, False)
                        p2.close()
                        del tens, p2
                        nb, fl, _ = op_algorithmic(ALL_WORKLOADS[wl])
                        th, ta = nb / (hbm_gbs * 1e9) * 1e3, fl / (fp32_tf * 1e12) * 1e3
                        rows.append({"op": op, "workload": wl, "ms": r["ms"], "roofline_frac": max(th, ta) / r["ms"]})
                    else:
                        a2 = copy.copy(args)
                        a2.workload, a2.steps, a2.warmup, a2.batch, a2.channels = wl, 3, 3, None, None
                        if not hasattr(a2, "hidden"):
                            a2.hidden, a2.layers = 32, 2
                        d = fn(a2, sample_clocks=False)
                        frac = d.get("op_roofline", d.get("roofline", {})).get("frac")
                        rows.append({"op": op, "workload": wl, "ms": d["ms_per_step"], "roofline_frac": frac})
                    torch.cuda.empty_cache()
                except Exception as exc:                          # reported rows: never fail the benchmark line
                    rows.append({"op": op, "workload": wl, "unavailable": repr(exc)[:200]})
            out["next_rows"] = rows
        if not args.no_cpu:
            out["cpu_baseline"] = cpu_oracle_sample(w)
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


# ---- the full operator of Eq. 2 (pointwise stages + long convolution) ------------------------------------

def measure_mixer(args, sample_clocks=True):
    """`--op mixer`: times hyenand_mixer_forward (Eq. 2) on the workload, inputs resident in HBM.  The long
    convolution inside runs on an fp32 plan; its kernels are timed by the library, the pointwise stages are the
    remainder."""
    from paper_2607_19378_b200 import hyenand as hn
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    w = ALL_WORKLOADS[args.workload].scaled(B=args.batch, C=args.channels)
    q, k, v, h = W.make_inputs(w, device=device)
    g_in = torch.ones(w.C, device=device)
    g_out = torch.ones(w.C, device=device)
    y = torch.empty_like(q)
    mx = hn.Mixer(w.dims, w.B, w.C, mode=w.mode, dtype=w.torch_dtype, eps=1e-6)
    for _ in range(max(args.warmup, 3)):
        mx.forward(q, k, v, h, g_in, g_out, y)
    torch.cuda.synchronize()
    sampler = ClockSampler(0) if sample_clocks else None
    if sampler is not None:
        time.sleep(0.6)
    for _ in range(3):
        mx.forward(q, k, v, h, g_in, g_out, y)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    for _ in range(args.steps):
        mx.forward(q, k, v, h, g_in, g_out, y)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    inner = hn.hyenand_mixer_plan(mx.handle)
    hn.hyenand_plan_set_timing(inner, 2)
    for _ in range(args.steps):
        mx.forward(q, k, v, h, g_in, g_out, y)
    torch.cuda.synchronize()
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if sampler is not None else None
    conv_ms = 0.0
    kernels = []
    for kid in range(hn.hyenand_plan_kernel_count(inner)):
        name = hn.hyenand_plan_kernel_info(inner, kid, w.h_shared)[0]
        tot, n = hn.hyenand_plan_kernel_time(inner, kid)
        if n > 0:
            kernels.append({"name": name, "ms_per_step": tot / args.steps, "launches_per_step": n / args.steps})
            conv_ms += tot / args.steps
    hn.hyenand_plan_set_timing(inner, 0)
    status = hn.hyenand_plan_device_status(inner)
    damage = hn.hyenand_mixer_guard_damage(mx.handle)
    if status != 0 or damage != 0:
        raise SystemExit(f"mixer: device status {status} / {damage} damaged guard bytes: the timing is void")
    mx.close()
    hbm_gbs, peak_src, sm_max = measured_peaks()
    fp32_tf = fp32_peak_tflops(torch.cuda.get_device_properties(0).multi_processor_count, sm_max)
    nbytes, flops, P = op_algorithmic(w)
    t_hbm, t_alu = nbytes / (hbm_gbs * 1e9) * 1e3, flops / (fp32_tf * 1e12) * 1e3
    return {
        "metric": "hyenand_mixer_throughput", "value": w.elements / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
        "dtype": "f32", "io_dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "op": "Eq. 2: RMSNorm(Sigmoid(v) * (K conv RMSNorm(l2(q) * SiLU(k))))",
                   "dims": list(w.dims), "B": w.B, "C": w.C, "mode": w.mode},
        "stages": {"long_convolution_ms": conv_ms, "pointwise_and_widening_ms": ms - conv_ms, "conv_kernels": kernels},
        "op_roofline": {"t_hbm_ms": t_hbm, "t_fp32_ms": t_alu, "roofline_ms": max(t_hbm, t_alu),
                        "frac": max(t_hbm, t_alu) / ms,
                        "note": "minimal bytes and transform flops of the long convolution; the pointwise stages add no minimal traffic"},
        "clocks": clocks, "device_status": status, "guard_damage": damage}


# ---- backward pass ------------------------------------------------------------------------------------------

def measure_backward(args, sample_clocks=True):
    """`--op backward`: times hyenand_backward (dq, dk, dv, dh) on the workload, inputs resident in HBM.  Roofline:
    the minimal traffic of the gradient (q, k, v, h, dy in; dq, dk, dv, dh out) and the transforms a direct spectral
    formulation needs (k v, dy q and h forward; dq, du, dh inverse), charged like the forward's."""
    from paper_2607_19378_b200 import hyenand as hn
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    w = ALL_WORKLOADS[args.workload].scaled(B=args.batch, C=args.channels)
    q, k, v, h = W.make_inputs(w, device=device)
    dy = torch.randn(q.shape, device=device, generator=torch.Generator(device=device).manual_seed(w.seed)).to(q.dtype)
    bw = hn.Backward(w.dims, w.B, w.C, mode=w.mode, dtype=w.torch_dtype)
    for _ in range(max(args.warmup, 3)):
        bw(q, k, v, h, dy)
    torch.cuda.synchronize()
    sampler = ClockSampler(0) if sample_clocks else None
    if sampler is not None:
        time.sleep(0.6)
    bw(q, k, v, h, dy)
    torch.cuda.synchronize()
    outs = [torch.empty_like(q), torch.empty_like(q), torch.empty_like(q), torch.empty_like(h)]
    stride = 0 if w.h_shared else w.C * h[0, 0].numel()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    for _ in range(args.steps):
        hn.hyenand_backward(bw.handle, q, k, v, h, stride, dy, *outs)
    e1.record()
    torch.cuda.synchronize()
    t1 = time.time()
    ms = e0.elapsed_time(e1) / args.steps
    clocks = sampler.stop(t0, t1) if sampler is not None else None
    damage = hn.hyenand_backward_guard_damage(bw.handle)
    if damage != 0:
        raise SystemExit(f"backward: {damage} damaged guard bytes: the timing is void")
    bw.close()
    hbm_gbs, peak_src, sm_max = measured_peaks()
    fp32_tf = fp32_peak_tflops(torch.cuda.get_device_properties(0).multi_processor_count, sm_max)
    sbytes = 4 if w.dtype == "f32" else 2
    hcount = w.C if w.h_shared else w.B * w.C
    nbytes = 7 * w.elements * sbytes + 2 * hcount * math.prod(w.taps) * sbytes
    P = math.prod(padded_dims(w))
    transforms = 5 * w.B * w.C + hcount
    flops = transforms * 2.5 * P * math.log2(P) if P > 1 else 0.0
    t_hbm, t_alu = nbytes / (hbm_gbs * 1e9) * 1e3, flops / (fp32_tf * 1e12) * 1e3
    return {
        "metric": "hyenand_backward_throughput", "value": w.elements / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
        "dtype": "f32", "io_dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "op": "dq, dk, dv, dh of y = q * (h conv (k v))", "dims": list(w.dims), "B": w.B,
                   "C": w.C, "mode": w.mode, "h_shared_over_batch": w.h_shared},
        "op_roofline": {"t_hbm_ms": t_hbm, "t_fp32_ms": t_alu, "roofline_ms": max(t_hbm, t_alu), "frac": max(t_hbm, t_alu) / ms,
                        "min_bytes": nbytes, "nominal_flops": flops,
                        "note": "six transforms per slice (five when the kernel is shared over the batch) at 2.5 P log2 P"},
        "clocks": clocks, "guard_damage": damage}


# ---- kernel synthesis ---------------------------------------------------------------------------------------

def measure_synth(args, sample_clocks=True):
    """`--op synth`: times hyenand_synthesize_kernel for the workload's kernel grid (SIREN of `--hidden` units and
    `--layers` hidden layers, FiLM-modulated per batch entry when the kernel is per sample).  Bound: FP32 ALUs
    (one fused multiply-add per weight and tap), reported against the derived FP32 peak."""
    from paper_2607_19378_b200 import hyenand as hn
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = ALL_WORKLOADS[args.workload].scaled(B=args.batch, C=args.channels)
    N, Hf, J = w.ndim, args.hidden, args.layers
    Bk = 1 if w.h_shared else w.B
    g = torch.Generator(device=dev).manual_seed(w.seed)
    r = lambda *shape: torch.rand(shape, generator=g, device=dev) * 2 - 1
    W1, b1, om = r(Hf, N) / math.sqrt(N), r(Hf) * 0.5, (r(Hf) + 1) * 15 + 1
    Wh, bh = r(max(J - 1, 1), Hf, Hf) * math.sqrt(6 / Hf), r(max(J - 1, 1), Hf) * 0.3
    Wout, bout = r(w.C, Hf) * math.sqrt(6 / Hf), r(w.C) * 0.1
    gamma, beta = (1 + 0.3 * r(Bk, J, Hf), 0.3 * r(Bk, J, Hf)) if not w.h_shared else (None, None)
    window = (r(w.C) + 1.5) if w.causal else torch.exp(r(N, w.C))
    h = torch.empty((Bk, w.C) + w.taps, dtype=w.torch_dtype, device=dev)
    mode = {"linear": 0, "causal": 1, "circular": 2}[w.mode]
    code = hn.HYENAND_F32 if w.dtype == "f32" else hn.HYENAND_BF16

    def run():
        hn.hyenand_synthesize_kernel(w.dims, mode, Bk, w.C, Hf, J, W1, b1, om, Wh if J > 1 else None, bh if J > 1 else None,
                                     Wout, bout, gamma, beta, window, code, h)
    for _ in range(max(args.warmup, 3)):
        run()
    torch.cuda.synchronize()
    sampler = ClockSampler(0) if sample_clocks else None
    if sampler is not None:
        time.sleep(0.6)
    for _ in range(3):
        run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    for _ in range(args.steps):
        run()
    e1.record()
    torch.cuda.synchronize()
    t1 = time.time()
    ms = e0.elapsed_time(e1) / args.steps
    clocks = sampler.stop(t0, t1) if sampler is not None else None
    taps = Bk * math.prod(w.taps)
    flops = 2.0 * taps * (Hf * (N + 1) + (J - 1) * Hf * (Hf + 1) + w.C * (Hf + 1))
    hbm_gbs, peak_src, sm_max = measured_peaks()
    fp32_tf = fp32_peak_tflops(torch.cuda.get_device_properties(0).multi_processor_count, sm_max)
    out_bytes = taps * w.C * (4 if w.dtype == "f32" else 2)
    ach = flops / (ms * 1e-3) / 1e12
    return {
        "metric": "hyenand_kernel_synthesis_throughput", "value": taps * w.C / (ms * 1e-3) / 1e9, "unit": "Gtap/s (taps x channels)",
        "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
        "dtype": "f32", "io_dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "op": "K(x) = window * SIREN(coordinates; FiLM)", "dims": list(w.dims), "taps": list(w.taps),
                   "kernels": Bk, "C": w.C, "hidden": Hf, "layers": J, "mode": w.mode},
        "roofline": {"kernel": "synth", "bound": "alu", "achieved": ach, "peak": fp32_tf, "unit": "TFLOP/s", "frac": ach / fp32_tf,
                     "traffic": None, "peak_source": "derived: 2 x 128 FP32 lanes x SMs x max SM clock",
                     "flops": "2 per weight and tap (fused multiply-adds of the three layer kinds); sines and exponentials not counted",
                     "t_hbm_ms_for_the_output": out_bytes / (hbm_gbs * 1e9) * 1e3,
                     "contractions_on": ("tensor cores (tcgen05.mma, tf32 operands split in two, three products: the "
                                         "fraction is the equivalent FP32 rate against the ALU peak)")
                                        if 16 < Hf <= 64 and not os.environ.get("HYENAND_SYNTH_ALU") else "FP32 ALUs"},
        "synth_device_status": hn.hyenand_synth_device_status(),
        "clocks": clocks}


# ---- reference arm: the CPU oracle ----------------------------------------------------------------

def main_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    w = ALL_WORKLOADS[args.workload].scaled(B=args.batch, C=args.channels)
    threads = oracle.threads()
    mode = w.mode
    S = w.B * w.C
    # size one step at roughly 2 s of oracle time: probe with one slice per thread first
    n = min(S, threads)
    ws = w.scaled(B=1, C=n)
    q, k, v, h = W.make_inputs(ws, device="cpu")
    t0 = time.perf_counter()
    oracle.conv_fft(q, k, v, h, mode)
    probe = time.perf_counter() - t0
    if probe < 1.0 and n < S:
        n = min(S, max(n, int(n * (2.0 / max(probe, 1e-3)) // threads * threads)))
        ws = w.scaled(B=1, C=n)
        q, k, v, h = W.make_inputs(ws, device="cpu")
    warm = max(0, min(args.warmup, 1 if probe > 5 else args.warmup))
    steps = args.steps if probe * args.steps < 240 else max(1, int(240 / probe))
    for _ in range(warm):
        oracle.conv_fft(q, k, v, h, mode)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.conv_fft(q, k, v, h, mode)
    dt = (time.perf_counter() - t0) / steps
    val = ws.elements / dt / 1e9
    sample = f"{n} of {S} (b,c) slices of {w.name} per step, oracle FFT path (fp64, radix-2)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": steps, "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "dims": list(w.dims), "B": w.B, "C": w.C, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(ALL_WORKLOADS))
    ap.add_argument("--batch", type=int, default=None, help="override B (profiling on a smaller case)")
    ap.add_argument("--channels", type=int, default=None, help="override C (profiling on a smaller case)")
    ap.add_argument("--no-all", action="store_true", help="skip the table over the other workloads")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--no-cufft", action="store_true", help="skip the torch.fft (cuFFT) composition reference point")
    ap.add_argument("--op", default="conv", choices=["conv", "mixer", "synth", "backward"],
                    help="conv: the gated long convolution (default, the benchmark line); mixer: the full operator of Eq. 2; "
                         "synth: the kernel synthesis K(x); backward: dq, dk, dv, dh")
    ap.add_argument("--hidden", type=int, default=32, help="--op synth: width of the SIREN")
    ap.add_argument("--layers", type=int, default=2, help="--op synth: hidden layers of the SIREN")
    a = ap.parse_args()
    if a.impl == "reference":
        main_reference(a)
    elif a.op == "mixer":
        print(json.dumps(measure_mixer(a)))
    elif a.op == "synth":
        print(json.dumps(measure_synth(a)))
    elif a.op == "backward":
        print(json.dumps(measure_backward(a)))
    else:
        main_ours(a)
