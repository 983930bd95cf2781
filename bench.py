#!/usr/bin/env python
"""Benchmark: one step = the 53 convolutions of ResNet-50 v1 at batch 64, the
depthwise case and the classifier-head Gemm, each launched once through the C ABI.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--repack]

Prints ONE JSON line.  `value` is TFLOP/s over the whole step with inputs resident
in HBM; `e2e` repeats the measurement with host (pinned) inputs copied in and the
outputs copied back inside the timed region.  `--impl reference` times the fp64
CPU oracle on a bounded sample of the same workload.  The weights are constants of
the graph, so their packed / TF32-rounded copies are made once at set-up
(onnx_conv2d_prepack) and the timed region runs onnx_conv2d_run_prepacked;
`--repack` times onnx_conv2d_run instead, which redoes that copy at every call.
With `--gpus N` and no launcher (WORLD_SIZE unset) the script starts its N ranks itself.

    python bench.py --layers [--only SUBSTR] [--repack]

prints one JSON line per distinct layer shape of the step and per configuration 1-4
(warm and L2-cold device time, TFLOP/s, GB/s, the roofline bound and the fraction of
it reached), then one summary line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2008_08272_b200 import workloads as wl  # noqa: E402

METRIC = "Conv/Gemm TFLOP/s (fp32 I/O, TF32 MMA)"
WORKLOAD = "resnet50_v1_53conv_sweep_b64+depthwise_256x28x28+gemm_head_64x1000x2048"
TF32_OVER_BF16 = 1125.0 / 2250.0     # nominal dense ratio, applied to the measured bf16 peak
SAMPLE_IMAGES = 16
SAMPLE_TEXT = ("first 16 images of each of the 54 convolutions plus the full head Gemm "
               "(1/4 of a step's convolution work)")

# DRAM traffic of the implicit-GEMM convolution kernel per benchmark step (its 17 launches), from the
# ncu captures summarised in profiles/tc_conv_kernel_dram_traffic_per_layer_shape.md.  Valid only for
# the kernel source those captures ran: the hash below is checked at run time.
NCU_TRAFFIC = {"mma_implicit": {"bytes_per_step": 596.8e6,
                                "sources": ["paper_2008_08272_b200/csrc/tc_conv.cu",
                                            "paper_2008_08272_b200/csrc/tc_conv_plan.h"],
                                "sha1": "bf5bedd99ba31432e2988109cf48ec0f4b731c63"}}


def ncu_traffic(family):
    """Measured DRAM bytes per step for `family`, or None when no capture matches the current source."""
    import hashlib
    rec = NCU_TRAFFIC.get(family)
    if rec is None:
        return None
    h = hashlib.sha1()
    try:
        for f in rec["sources"]:
            with open(os.path.join(ROOT, f), "rb") as fh:
                h.update(fh.read())
    except OSError:
        return None
    return rec["bytes_per_step"] if h.hexdigest() == rec["sha1"] else None
FP32_FMA_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12   # 148 SMs x 128 FMA lanes x 2 flop x max clock


def tf32_peak_for(peaks, clocks=None, isolated=False):
    """(TFLOP/s, text): the measured bf16 GEMM rate x the nominal TF32/bf16 ratio 0.5.  The burst figure
    for launches timed alone or for a region that ran at the maximum SM clock; the sustained one (taken
    under the power cap) when the clock record shows the region was power-limited."""
    burst = isolated
    if not isolated and clocks and clocks.get("sm_mhz") and clocks.get("sm_max_mhz"):
        burst = clocks["sm_mhz"] >= 0.95 * clocks["sm_max_mhz"] and "sw_power_cap" not in clocks.get("reasons", [])
    key = "bf16_burst" if burst else "bf16_sustained"
    why = ("launch timed alone" if isolated else "timed region ran at the maximum SM clock, no power cap") if burst \
        else "timed region under the power cap or below the maximum clock"
    return peaks[key] * TF32_OVER_BF16, f"{peaks['source']} bf16 {'burst' if burst else 'sustained'} x nominal tf32/bf16 ratio 0.5 ({why})"


def roof_of(flops, nbytes, seconds, tensor_peak_tflops, hbm_gbs):
    """Roofline of one launch or one family: the binding roof, what was achieved against it, the fraction."""
    t_tensor = flops / (tensor_peak_tflops * 1e12)
    t_hbm = nbytes / (hbm_gbs * 1e9)
    if t_tensor >= t_hbm:
        ach = flops / seconds / 1e12
        return {"bound": "tensor", "achieved": ach, "peak": tensor_peak_tflops, "unit": "TFLOP/s",
                "frac": ach / tensor_peak_tflops}
    ach = nbytes / seconds / 1e9
    return {"bound": "hbm", "achieved": ach, "peak": hbm_gbs, "unit": "GB/s", "frac": ach / hbm_gbs}


def step_ops(batch: int = 64):
    """The ops of one step, in launch order."""
    convs = wl.resnet50_v1_convs(batch) + [wl.config5_depthwise(batch)]
    gemm = wl.GemmCase("r50_head_gemm", (batch, 2048), (1000, 2048), (1000,), transB=True,
                       seed=wl.SEED_BASE + 1000 * 5 + 54)
    return convs, gemm


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"],
                    bf16_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """SM clock and throttle-reason samples while the timed region runs (read-only NVML queries from a
    thread every few milliseconds; falls back to an nvidia-smi loop if NVML cannot be loaded)."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.thread = None
        self.stop_flag = False
        self.sm, self.reasons, self.max_mhz = [], set(), None

    def _nvml_loop(self, nv, handle):
        bits = {"hw_slowdown": nv.nvmlClocksEventReasonHwSlowdown if hasattr(nv, "nvmlClocksEventReasonHwSlowdown")
                else nv.nvmlClocksThrottleReasonHwSlowdown,
                "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown",
                                               getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0)),
                "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown",
                                               getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0)),
                "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap",
                                        getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0))}
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons",
                              getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons", None))
        while not self.stop_flag:
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(handle, nv.NVML_CLOCK_SM)))
                if get_reasons is not None:
                    r = int(get_reasons(handle))
                    for name, bit in bits.items():
                        if bit and (r & bit):
                            self.reasons.add(name)
            except Exception:
                break
            time.sleep(0.002)

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            # NVML enumerates all GPUs of the machine; honour CUDA_VISIBLE_DEVICES when it is a plain index list
            vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            idx = self.gpu
            if vis and all(t.strip().isdigit() for t in vis.split(",")):
                idx = int(vis.split(",")[self.gpu])
            handle = nv.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = float(nv.nvmlDeviceGetMaxClockInfo(handle, nv.NVML_CLOCK_SM))
            import threading
            self.thread = threading.Thread(target=self._nvml_loop, args=(nv, handle), daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.thread is not None:
            self.stop_flag = True
            self.thread.join(timeout=2)
            return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.max_mhz,
                    "samples": len(self.sm), "reasons": sorted(self.reasons), "source": "nvml"}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["clock query unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons), "source": "nvidia-smi"}


def run_reference(args):
    """The fp64 CPU oracle, as it stands, on a bounded sample of the step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    convs, gemm = step_ops()
    sample = SAMPLE_TEXT
    prepared = []
    for c in convs:
        X, W, B = wl.conv_inputs(wl.with_batch(c, SAMPLE_IMAGES))
        prepared.append((c, X, W, B))
    A, Bm, C = wl.gemm_inputs(gemm)
    flops = sum(wl.with_batch(c, SAMPLE_IMAGES).flops for c in convs) + gemm.flops

    def one():
        for c, X, W, B in prepared:
            oracle.conv2d(X, W, B, pads=c.pads, strides=c.strides, dilations=c.dilations, group=c.group,
                          relu=c.relu, want_s=False)
        oracle.gemm(A, Bm, C, transB=True, want_s=False)

    for _ in range(min(args.warmup, 1)):
        one()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one()
    dt = (time.perf_counter() - t0) / args.steps
    value = flops / dt / 1e12
    cores = oracle.threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch": 64, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def max_over_ranks(value: float, world: int, device=None) -> float:
    """The slowest rank's figure (every rank gets it): the replicas run independently, so the job's
    step time is the maximum of theirs.  Uses the default process group (NCCL on GPUs, gloo on CPU)."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def ranks_reporting(world: int, device=None) -> int:
    """How many ranks of the job are really there: every rank contributes one to a sum."""
    if world <= 1:
        return 1
    import torch
    import torch.distributed as dist
    t = torch.ones(1, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(round(float(t.item())))


def spawn_ranks(n: int, argv) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks (one per GPU, rendezvous on
    127.0.0.1), pass rank 0's output through, fail if any rank fails."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=env,
                                      stdout=subprocess.PIPE if r == 0 else subprocess.DEVNULL, text=True))
    out, _ = procs[0].communicate()
    codes = [procs[0].returncode] + [p.wait() for p in procs[1:]]
    sys.stdout.write(out or "")
    sys.stdout.flush()
    return 0 if all(c == 0 for c in codes) else 1


def run_cpu_dry_run(args):
    """The rank logic of a multi-GPU run with the kernels left out (gloo on CPU): every rank joins, the
    slowest rank's time is the job's, rank 0 prints a line whose n_gpus is the number of ranks that
    reported.  For testing the launch path on a machine without GPUs; the line says what it is."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("gloo")
    seen = ranks_reporting(world)
    if seen != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but {seen} rank(s) reported")
    ms = max_over_ranks(10.0 + rank, world)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"cpu_dry_run": True, "n_gpus": seen, "ms_per_step": ms, "value": None,
                          "note": "no kernel ran: launch-path test only"}))
    return 0


def job_tflops(world: int, flops_per_replica_step: float, ms_per_step: float) -> float:
    """Whole-job throughput of `world` independent replicas that each do one step in ms_per_step."""
    return world * flops_per_replica_step / (ms_per_step * 1e-3) / 1e12


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2008_08272_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if ranks_reporting(world, dev) != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but {world} rank(s) are running: launch one rank per GPU "
                         "(python bench.py --gpus N starts them itself when WORLD_SIZE is unset)")
    binding.load(build_if_missing=False)

    convs, gemm = step_ops(args.batch)
    if args.only:
        # profiling aid: a subset of the step's convolutions (name substring), e.g. one layer under ncu
        convs = [c for c in convs if args.only in c.name]
        if not convs:
            raise SystemExit(f"--only {args.only!r} matches no convolution of the step")
    # ---- inputs: seeded host arrays (pinned, reused by the e2e leg) and resident device copies
    host, devt, descs, packed = [], [], [], []
    for c in convs:
        X, W, B = wl.conv_inputs(c)
        hx, hw, hb = (torch.from_numpy(t).pin_memory() for t in (X, W, B))
        host.append((hx, hw, hb))
        d = binding.Conv2dDesc(c.x_shape, c.w_shape, pads=c.pads, strides=c.strides, dilations=c.dilations,
                               group=c.group, has_bias=True, fuse_relu=c.relu)
        ws = torch.empty(max(d.workspace_bytes, 16), dtype=torch.uint8, device=dev)
        y = torch.empty(d.y_shape, dtype=torch.float32, device=dev)
        devt.append([hx.to(dev), hw.to(dev), hb.to(dev), y, ws])
        packed.append(None if args.repack else d.prepack(devt[-1][1]))
        descs.append(d)
    A, Bm, C = wl.gemm_inputs(gemm)
    g_host = tuple(torch.from_numpy(t).pin_memory() for t in (A, Bm, C))
    g_dev = [t.to(dev) for t in g_host]
    gm, gn, gk = gemm.mnk
    g_y = torch.empty((gm, gn), dtype=torch.float32, device=dev)
    g_ws = torch.empty(max(binding.gemm_workspace_bytes(False, True, gm, gn, gk), 16), dtype=torch.uint8, device=dev)
    y_host = torch.empty(max(int(np.prod(d.y_shape)) for d in descs), dtype=torch.float32).pin_memory()
    torch.cuda.synchronize()

    flops_per_step = sum(c.flops for c in convs) + gemm.flops
    bytes_per_op = [c.algorithmic_bytes for c in convs] + [4 * (gm * gk + gn * gk + gn + gm * gn)]
    flops_per_op = [c.flops for c in convs] + [gemm.flops]
    families = [d.kernel_family for d in descs] + ["gemm"]
    n_ops = len(flops_per_op)

    def run_conv(i):
        x, w, b, y, ws = devt[i]
        if args.repack:
            descs[i].run(x, w, b, Y=y, workspace=ws)
        else:
            descs[i].run_prepacked(x, w, packed[i], b, None, Y=y, workspace=ws)

    def launch_all(events=None):
        for i, d in enumerate(descs):
            run_conv(i)
            if events is not None:
                events[i + 1].record()
        binding.onnx_gemm(g_dev[0], g_dev[1], g_dev[2], transB=True, Y=g_y, workspace=g_ws)
        if events is not None:
            events[n_ops].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing
    for _ in range(args.warmup):
        launch_all()
    barrier()
    run_step = launch_all
    graph_launches = None
    if not args.no_graph:
        # One step (its 66 launches with their programmatic dependencies) captured once into a CUDA graph
        # and replayed: the library calls' host work (argument checks, tensor-map encoding, launch) then
        # costs nothing inside the timed region and the launches follow each other more closely (2.05 ->
        # 1.99 ms per step).  The kernels, their arguments and their order are the same; --no-graph
        # launches them call by call instead.
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        cuda_graph = torch.cuda.CUDAGraph()
        l0 = binding.launch_count()
        with torch.cuda.stream(side):
            with torch.cuda.graph(cuda_graph, stream=side):
                launch_all()
        graph_launches = int(binding.launch_count() - l0)
        torch.cuda.current_stream().wait_stream(side)
        run_step = cuda_graph.replay
        for _ in range(3):
            run_step()
        barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = binding.launch_count()
    barrier()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for s in range(args.steps):
        run_step()
    t_end.record()
    barrier()
    launches = graph_launches * args.steps if graph_launches is not None else binding.launch_count() - launches0
    ms_total = t_start.elapsed_time(t_end)
    assert binding.last_device_status() == 0, "a device-side wait timed out"
    ms_total = max_over_ranks(ms_total, world, dev)
    ms_per_step = ms_total / args.steps
    value = job_tflops(world, flops_per_step, ms_per_step)

    # Per-op durations: the same K steps again, now with an event after every op.  (Events between
    # kernels forbid the early start of the next kernel that back-to-back launches get, so this pass is
    # a little slower than the timed one; it only feeds the per-family roofline figures.)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(n_ops + 1)] for _ in range(args.steps)]
    for s in range(args.steps):
        ev[s][0].record()
        launch_all(ev[s])
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    # grouped by kernel family
    per_op_ms = [statistics.fmean(ev[s][i].elapsed_time(ev[s][i + 1]) for s in range(args.steps))
                 for i in range(n_ops)]
    fam_time, fam_flops, fam_bytes, fam_count = {}, {}, {}, {}
    for i, f in enumerate(families):
        fam_time[f] = fam_time.get(f, 0.0) + per_op_ms[i]
        fam_flops[f] = fam_flops.get(f, 0) + flops_per_op[i]
        fam_bytes[f] = fam_bytes.get(f, 0) + bytes_per_op[i]
        fam_count[f] = fam_count.get(f, 0) + 1
    top = max(fam_time, key=fam_time.get)
    peaks = measured_peaks()
    tensor_peak, tensor_src = tf32_peak_for(peaks, clocks)

    def family_roof(f):
        secs = fam_time[f] * 1e-3
        if f.startswith("mma") or f == "gemm":
            r = roof_of(fam_flops[f], fam_bytes[f], secs, tensor_peak, peaks["hbm_gbs"])
            r["peak_source"] = tensor_src if r["bound"] == "tensor" else f"{peaks['source']} HBM copy"
        elif f == "simt_depthwise":
            gbs = fam_bytes[f] / secs / 1e9
            r = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                 "frac": gbs / peaks["hbm_gbs"], "peak_source": f"{peaks['source']} HBM copy"}
        else:
            tf = fam_flops[f] / secs / 1e12
            r = {"bound": "alu", "achieved": tf, "peak": FP32_FMA_PEAK_TFLOPS, "unit": "TFLOP/s",
                 "frac": tf / FP32_FMA_PEAK_TFLOPS,
                 "peak_source": "derived: 148 SMs x 128 fp32 FMA/clk x 2 x 1.965 GHz"}
        return r

    roof = family_roof(top)
    only_full = (not args.only) and args.batch == 64
    roof.update({"kernel": top, "launches_per_step": fam_count[top], "ms_per_step": fam_time[top],
                 "basis": "all launches of this kernel family in one step (flops or bytes summed, time summed)",
                 "traffic": ncu_traffic(top) if only_full else None, "traffic_unit": "bytes per step"})
    families_out = {}
    for f in fam_time:
        r = family_roof(f)
        families_out[f] = {"ops": fam_count[f], "ms": round(fam_time[f], 4),
                           "tflops": round(fam_flops[f] / (fam_time[f] * 1e-3) / 1e12, 3),
                           "gbs": round(fam_bytes[f] / (fam_time[f] * 1e-3) / 1e9, 1),
                           "bound": r["bound"], "frac": round(r["frac"], 4)}
    # the step against its own roofline: every op at max(flops / tensor peak, bytes / HBM bandwidth)
    step_roof_ms = sum(max(fl / (tensor_peak * 1e12), by / (peaks["hbm_gbs"] * 1e9))
                       for fl, by in zip(flops_per_op, bytes_per_op)) * 1e3

    # ---- end to end: pinned host inputs in, results out, every step
    e2e_steps = max(1, min(args.steps, 2))
    h2d = sum(t.numel() * 4 for trip in host for t in trip) + sum(t.numel() * 4 for t in g_host)
    d2h = sum(int(np.prod(d.y_shape)) * 4 for d in descs) + gm * gn * 4

    # Three streams: host->device copies, kernels, device->host reads.  Every op has its own device buffers,
    # so the only ordering needed is per op: copy-in -> run -> read-out, and the next step's copy-in / run
    # of the same op after this step's run / read-out.  PCIe carries both directions at once.
    s_run = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    n_ops = len(descs) + 1
    ev_in = [torch.cuda.Event() for _ in range(n_ops)]
    ev_run = [torch.cuda.Event() for _ in range(n_ops)]
    ev_out = [torch.cuda.Event() for _ in range(n_ops)]
    first = [True]

    def e2e_op(i, dev_in, host_in, run, y):
        if not first[0]:
            s_in.wait_event(ev_run[i])            # the previous step's kernel has read these inputs
        with torch.cuda.stream(s_in):
            for dt_, ht_ in zip(dev_in, host_in):
                dt_.copy_(ht_, non_blocking=True)
            ev_in[i].record(s_in)
        s_run.wait_event(ev_in[i])
        if not first[0]:
            s_run.wait_event(ev_out[i])           # the previous step's result has left the device
        run()
        ev_run[i].record(s_run)
        s_out.wait_event(ev_run[i])
        with torch.cuda.stream(s_out):
            y_host[: y.numel()].copy_(y.view(-1), non_blocking=True)
            ev_out[i].record(s_out)

    def e2e_step():
        for i, d in enumerate(descs):
            x, w, b, y, ws = devt[i]
            e2e_op(i, (x, w, b), host[i], lambda i=i: run_conv(i), y)
        e2e_op(n_ops - 1, g_dev, g_host,
               lambda: binding.onnx_gemm(g_dev[0], g_dev[1], g_dev[2], transB=True, Y=g_y, workspace=g_ws), g_y)
        first[0] = False

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    s_in.wait_stream(s_run)
    s_out.wait_stream(s_run)
    for _ in range(e2e_steps):
        e2e_step()
    s_run.wait_stream(s_in)
    s_run.wait_stream(s_out)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    e2e_ms = max_over_ranks(e2e_ms, world, dev)
    e2e_value = job_tflops(world, flops_per_step, e2e_ms)

    # ---- CPU baseline: the oracle on a bounded sample (rank 0, single GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        sample_flops, t_cpu = 0, 0.0
        for i, c in enumerate(convs):
            hx, hw, hb = host[i]
            X1 = hx[:SAMPLE_IMAGES].numpy()
            t0 = time.perf_counter()
            oracle.conv2d(X1, hw.numpy(), hb.numpy(), pads=c.pads, strides=c.strides, dilations=c.dilations,
                          group=c.group, relu=c.relu, want_s=False)
            t_cpu += time.perf_counter() - t0
            sample_flops += wl.with_batch(c, SAMPLE_IMAGES).flops
        t0 = time.perf_counter()
        oracle.gemm(A, Bm, C, transB=True, want_s=False)
        t_cpu += time.perf_counter() - t0
        sample_flops += gemm.flops
        cpu = {"value": sample_flops / t_cpu / 1e12, "unit": "TFLOP/s", "cores": oracle.threads(),
               "kind": "oracle", "seconds": round(t_cpu, 3),
               "sample": SAMPLE_TEXT}

    if world > 1:
        dist.destroy_process_group()
    if rank != 0:
        return 0
    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "tf32" if any(f.startswith("mma") for f in families) else "f32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD if not args.only and args.batch == 64 else
                   f"SUBSET only={args.only!r} batch={args.batch} (profiling aid, not the benchmark)",
                   "batch_per_gpu": args.batch, "ops_per_step": n_ops,
                   "gflop_per_step": round(flops_per_step / 1e9, 3),
                   "l2": "inputs larger than L2: every op has its own X/W/Y buffers, ~8 GB touched per step",
                   "weights": ("re-packed / re-rounded by every run call (--repack)" if args.repack else
                               "constant weights pre-packed once, outside the timed region (onnx_conv2d_prepack)"),
                   "launch": ("call by call on one stream (--no-graph)" if args.no_graph else
                              "one CUDA graph per step (the step's library calls captured once), replayed"),
                   "parallelism": f"replicas x{world} (batch split, no collective)"},
        "pct_of_nominal_tf32_peak_1125": round(100 * value / world / 1125.0, 2),
        "roofline": roof, "kernel_families": families_out,
        "step_roofline": {"ms": round(step_roof_ms, 4), "frac": round(step_roof_ms / ms_per_step, 4),
                          "basis": "sum over ops of max(flops / tensor peak, algorithmic bytes / HBM bandwidth)",
                          "tensor_peak_tflops": tensor_peak, "hbm_gbs": peaks["hbm_gbs"]},
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "ms_per_step": e2e_ms, "steps": e2e_steps,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "pipeline": "copy-in, kernels and read-out on three streams, ordered per op by events"},
        "gpu_launches": int(launches), "clocks": clocks, "cpu_baseline": cpu,
    }
    if args.per_op:
        # every op's own duration inside the step (event after each op), in the step's order
        names = [c.name for c in convs] + ["head_gemm"]
        line["per_op_us"] = [[names[i], families[i], round(per_op_ms[i] * 1e3, 1)] for i in range(n_ops)]
    print(json.dumps(line))
    return 0


def run_probe_tf32():
    """TF32 tcgen05.mma issue-rate ceiling (operands resident in shared memory, every SM busy): one JSON line."""
    import torch
    from paper_2008_08272_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(0)
    binding.load(build_if_missing=False)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    max_mhz = measured_clock_max_mhz()
    out = {"probe": "tcgen05.mma kind::tf32, 128 x N x 8, operands resident in shared memory", "sms": sms,
           "sm_max_mhz": max_mhz, "shapes": {}}
    for n in (64, 128, 256):
        cyc = min(binding.probe_tf32_mma_rate(n, 4096) for _ in range(3))
        mac = 128.0 * n * 8 / cyc
        out["shapes"][str(n)] = {"cycles_per_instruction": round(cyc, 2), "ideal": n // 2,
                                 "mac_per_clk_per_sm": round(mac, 1),
                                 "tflops_at_max_clock": round(2 * mac * sms * max_mhz * 1e6 / 1e12, 1)}
    print(json.dumps(out))
    return 0


def run_model(args):
    """Chained ResNet-50 v1 inference at --batch images (synthetic weights): 53 convolutions with fused
    bias/Relu and fused residual Add, the two pools and the classifier Gemm, enqueued back to back on one
    stream.  Device time per forward pass over --steps passes after --warmup; one JSON line.  This is the
    figure comparable in kind (not in hardware) with the inference times of the paper's Table 1."""
    import torch
    from paper_2008_08272_b200 import binding
    from paper_2008_08272_b200.resnet50_chain import Resnet50Chain
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    binding.load(build_if_missing=False)
    net = Resnet50Chain(args.batch, dev)
    x = torch.rand((args.batch, 3, 224, 224), device=dev)
    for _ in range(max(args.warmup, 3)):
        net.forward(x)
    torch.cuda.synchronize()
    l0 = binding.launch_count()
    net.forward(x)
    per_pass = int(binding.launch_count() - l0)
    run = lambda: net.forward(x)
    if args.graph:
        # the whole pass captured once into a CUDA graph and replayed: the 56 library calls per pass (argument
        # checks, tensor-map encoding, launches) then cost the host nothing, which is what bounds batch 1
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                net.forward(x)
        torch.cuda.current_stream().wait_stream(side)
        run = graph.replay
        for _ in range(3):
            run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        run()
    e1.record()
    torch.cuda.synchronize()
    assert binding.last_device_status() == 0
    ms = e0.elapsed_time(e1) / args.steps
    out = {"metric": "ResNet-50 v1 chained inference, device time per forward pass", "value": ms, "unit": "ms",
           "higher_is_better": False, "batch": args.batch, "images_per_s": round(args.batch / ms * 1e3, 1),
           "tflops": round(net.flops / (ms * 1e-3) / 1e12, 1), "steps": args.steps, "data": "synthetic",
           "gpu_launches_per_pass": per_pass, "cuda_graph": bool(args.graph),
           "paper_table1_context": "7.540 s for one image on a 2.3 GHz POWER9 CPU, unoptimised scalar loops"}
    net.close()
    print(json.dumps(out))
    return 0


def run_pool():
    """ResNet-50's MaxPool (3x3, stride 2, pad 1 on [64,64,112,112]) and GlobalAveragePool ([64,2048,7,7]):
    device time per launch with L2 flushed before each (ten flush+run pairs minus ten flushes), against
    the measured HBM copy bandwidth.  One JSON line."""
    import torch
    from paper_2008_08272_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    binding.load(build_if_missing=False)
    peaks = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def timed(fn, reps=10):
        def once(with_run):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(reps):
                flush.zero_()
                if with_run:
                    fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e3 / reps
        fn()
        return min(once(True) for _ in range(3)) - min(once(False) for _ in range(3))

    out = {"metric": "pooling operators, device time per launch (L2 flushed)", "unit": "us", "data": "synthetic",
           "hbm_peak_gbs": peaks["hbm_gbs"], "ops": {}}
    x = torch.rand((64, 64, 112, 112), device=dev)
    y = torch.empty((64, 64, 56, 56), device=dev)
    us = timed(lambda: binding.onnx_maxpool2d(x, (3, 3), pads=(1, 1, 1, 1), strides=(2, 2), Y=y))
    nbytes = 4 * (x.numel() + y.numel())
    out["ops"]["maxpool_3x3_s2_64x64x112x112"] = {"us": round(us, 1), "gbs": round(nbytes / us / 1e3, 1),
                                                  "frac_of_hbm_peak": round(nbytes / us / 1e3 / peaks["hbm_gbs"], 3)}
    x2 = torch.rand((64, 2048, 7, 7), device=dev)
    y2 = torch.empty((64, 2048, 1, 1), device=dev)
    us = timed(lambda: binding.onnx_global_average_pool(x2, Y=y2))
    nbytes = 4 * (x2.numel() + y2.numel())
    out["ops"]["global_average_pool_64x2048x7x7"] = {"us": round(us, 1), "gbs": round(nbytes / us / 1e3, 1),
                                                     "frac_of_hbm_peak": round(nbytes / us / 1e3 / peaks["hbm_gbs"], 3)}
    print(json.dumps(out))
    return 0


def run_gemm():
    """ONNX Gemm (Sec. 3.4.3's MatMul + Add target) at a few sizes and attribute sets: device time per
    launch with L2 flushed before each (ten flush+run pairs minus ten flushes), TFLOP/s against the measured
    bf16 burst peak x the nominal TF32/bf16 ratio 0.5, and GB/s against the measured copy bandwidth.  One JSON line."""
    import torch
    from paper_2008_08272_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    binding.load(build_if_missing=False)
    peaks = measured_peaks()
    tf32_peak = peaks["bf16_burst"] * 0.5
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def timed(fn, reps=10):
        def once(with_run):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(reps):
                flush.zero_()
                if with_run:
                    fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e3 / reps
        fn()
        return min(once(True) for _ in range(3)) - min(once(False) for _ in range(3))

    cases = [  # (M, N, K, transA, transB, C shape or None)
        (64, 1000, 2048, False, True, (1000,)),        # ResNet-50 classifier head, batch 64
        (1024, 1024, 1024, False, False, None),
        (4096, 4096, 4096, False, False, (4096,)),
        (4096, 4096, 4096, False, True, None),
        (4096, 4096, 4096, True, False, None),
        (8192, 8192, 8192, False, False, None),
        (8192, 1024, 512, False, False, (8192, 1)),    # wide output, short reduction: store-bound
        (2048, 2048, 16, False, False, (2048,)),       # thin contraction (K < 32): the exact fp32 SIMT kernel
    ]
    g = torch.Generator(device="cpu").manual_seed(20)
    out = {"metric": "ONNX Gemm, device time per launch (L2 flushed)", "unit": "us", "dtype": "tf32",
           "data": "synthetic", "tf32_peak_tflops": tf32_peak,
           "tf32_peak_source": peaks["source"] + " bf16 burst x nominal tf32/bf16 ratio 0.5",
           "hbm_peak_gbs": peaks["hbm_gbs"], "ops": {}}
    for M, N, K, ta, tb, cs in cases:
        A = torch.randn((K, M) if ta else (M, K), generator=g).to(dev)
        B = torch.randn((N, K) if tb else (K, N), generator=g).to(dev)
        C = torch.randn(cs, generator=g).to(dev) if cs else None
        Y = torch.empty((M, N), device=dev)
        need = binding.gemm_workspace_bytes(ta, tb, M, N, K)
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
        us = timed(lambda: binding.onnx_gemm(A, B, C, transA=ta, transB=tb, Y=Y, workspace=ws))
        if binding.last_device_status() != 0:
            raise SystemExit("device status set during the Gemm sweep")
        flops = 2.0 * M * N * K
        nbytes = 4.0 * (M * K + K * N + M * N)
        name = f"{M}x{N}x{K}" + ("_tA" if ta else "") + ("_tB" if tb else "") + ("_C" + "x".join(map(str, cs)) if cs else "")
        out["ops"][name] = {"us": round(us, 1), "tflops": round(flops / us / 1e6, 1),
                            "frac_of_tf32_peak": round(flops / us / 1e6 / tf32_peak, 3),
                            "gbs": round(nbytes / us / 1e3, 1)}
        del A, B, C, Y, ws
    print(json.dumps(out))
    return 0


def run_layers(args):
    """Per-layer measurements: every distinct convolution shape of the step (with its multiplicity), the
    depthwise case, the head Gemm, and configurations 1-4 at their stated sizes.  For each: device time
    warm (twenty back-to-back launches between two events) and L2-cold (ten L2-flush + launch pairs minus
    ten flushes: the event clock ticks every ~2 us), TFLOP/s and algorithmic GB/s of the cold time, the
    roofline time max(flops / TF32 peak, bytes / HBM bandwidth) and the fraction of it reached.
    Denominators: MEASURED_PEAKS.json's copy bandwidth, and its bf16 burst GEMM rate x 0.5 (launches
    timed alone run at the maximum clock).  One JSON line per layer, then a summary line."""
    import torch
    from paper_2008_08272_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    binding.load(build_if_missing=False)
    peaks = measured_peaks()
    tensor_peak, tensor_src = tf32_peak_for(peaks, isolated=True)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def timed(fn):
        def span(n, with_flush, with_run):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(n):
                if with_flush:
                    flush.zero_()
                if with_run:
                    fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) * 1e3 / n
        for _ in range(3):
            fn()
        warm = min(span(20, False, True) for _ in range(3))
        cold = min(span(10, True, True) for _ in range(3)) - min(span(10, True, False) for _ in range(3))
        return warm, cold

    def emit(name, group, shape, family, mult, flops, nbytes, warm, cold, launches):
        roof_us = max(flops / (tensor_peak * 1e12), nbytes / (peaks["hbm_gbs"] * 1e9)) * 1e6
        tiny = flops < 1e8                    # configurations 1 and 2: a few microseconds of launch latency
        rec = {"layer": name, "group": group, "shape": shape, "family": family, "count_in_step": mult,
               "launches": launches, "us_warm": round(warm, 2), "us_cold": round(cold, 2),
               "tflops": round(flops / cold / 1e6, 2), "gbs": round(nbytes / cold / 1e3, 1),
               "bound": "launch" if tiny else ("tensor" if flops / (tensor_peak * 1e12) >= nbytes / (peaks["hbm_gbs"] * 1e9) else "hbm"),
               "roofline_us": round(roof_us, 2), "frac": None if tiny else round(roof_us / cold, 3),
               "gflop": round(flops / 1e9, 3), "mbytes": round(nbytes / 1e6, 2)}
        print(json.dumps(rec), flush=True)
        return rec

    def conv_line(c, group, mult):
        X, W, B = wl.conv_inputs(c)
        x, w, b = (torch.from_numpy(t).to(dev) for t in (X, W, B))
        d = binding.Conv2dDesc(c.x_shape, c.w_shape, pads=c.pads, strides=c.strides, dilations=c.dilations,
                               group=c.group, has_bias=True, fuse_relu=c.relu)
        ws = torch.empty(max(d.workspace_bytes, 16), dtype=torch.uint8, device=dev)
        y = torch.empty(d.y_shape, dtype=torch.float32, device=dev)
        pk = None if args.repack else d.prepack(w)
        fn = (lambda: d.run(x, w, b, Y=y, workspace=ws)) if args.repack else \
             (lambda: d.run_prepacked(x, w, pk, b, None, Y=y, workspace=ws))
        l0 = binding.launch_count()
        fn()
        launches = int(binding.launch_count() - l0)
        warm, cold = timed(fn)
        if binding.last_device_status() != 0:
            raise SystemExit(f"device status set while timing {c.name}")
        rec = emit(c.name, group, {"x": list(c.x_shape), "w": list(c.w_shape), "strides": list(c.strides),
                                   "pads": list(c.pads), "group": c.group},
                   d.kernel_family, mult, c.flops, c.algorithmic_bytes, warm, cold, launches)
        d.close()
        return rec

    def gemm_line(g, group, mult):
        A, Bm, C = wl.gemm_inputs(g)
        a, bm, cc = (torch.from_numpy(t).to(dev) for t in (A, Bm, C))
        m, n, k = g.mnk
        y = torch.empty((m, n), dtype=torch.float32, device=dev)
        ws = torch.empty(max(binding.gemm_workspace_bytes(g.transA, g.transB, m, n, k), 16), dtype=torch.uint8, device=dev)
        fn = lambda: binding.onnx_gemm(a, bm, cc, alpha=g.alpha, beta=g.beta, transA=g.transA, transB=g.transB,
                                       fuse_relu=g.relu, Y=y, workspace=ws)
        l0 = binding.launch_count()
        fn()
        launches = int(binding.launch_count() - l0)
        warm, cold = timed(fn)
        nbytes = 4 * (m * k + k * n + (int(np.prod(g.c_shape)) if g.c_shape is not None else 0) + m * n)
        return emit(g.name, group, {"M": m, "N": n, "K": k, "transA": g.transA, "transB": g.transB,
                                    "c_shape": list(g.c_shape) if g.c_shape is not None else None},
                    "gemm", mult, g.flops, nbytes, warm, cold, launches)

    convs, head = step_ops(args.batch)
    seen, order = {}, []
    for c in convs:
        key = (c.x_shape, c.w_shape, c.strides, c.pads, c.group)
        if key in seen:
            seen[key][1] += 1
        else:
            seen[key] = [c, 1]
            order.append(key)
    want = lambda name: (not args.only) or any(t in name for t in args.only.split(","))
    step_us, step_roof = 0.0, 0.0
    for key in order:
        c, mult = seen[key]
        if want(c.name):
            r = conv_line(c, "step", mult)
            step_us += r["us_cold"] * mult
            step_roof += r["roofline_us"] * mult
    if want(head.name):
        r = gemm_line(head, "step", 1)
        step_us += r["us_cold"]
        step_roof += r["roofline_us"]
    if args.batch == 64:
        if want("cfg1"):
            conv_line(wl.config1_mnist_conv(), "config1", 0)
        if want("cfg2"):
            gemm_line(wl.config2_gemm_head(), "config2", 0)
        if want("cfg3"):
            conv_line(wl.config3_stage2_3x3(), "config3", 0)
        for c4 in wl.config4_stem_and_projection():
            if want(c4.name):
                conv_line(c4, "config4", 0)
    print(json.dumps({"summary": "sum over the step's ops of the L2-cold times (count_in_step weighted)",
                      "us": round(step_us, 1), "roofline_us": round(step_roof, 1),
                      "frac": round(step_roof / step_us, 3) if step_us else None,
                      "subset": args.only or None, "batch": args.batch,
                      "weights": "re-packed every call" if args.repack else "pre-packed once",
                      "tf32_peak_tflops": tensor_peak, "tf32_peak_source": tensor_src,
                      "hbm_peak_gbs": peaks["hbm_gbs"], "hbm_peak_source": f"{peaks['source']} HBM copy"}))
    return 0


def measured_clock_max_mhz():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh).get("sm_max_mhz", 1965.0))
    except (OSError, ValueError):
        return 1965.0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only", default="", help="profiling aid: run only the convolutions whose name contains this")
    ap.add_argument("--batch", type=int, default=64, help="images per convolution (the benchmark proper uses 64)")
    ap.add_argument("--model", action="store_true",
                    help="time a chained ResNet-50 v1 forward pass (all operators, one stream) instead of the step")
    ap.add_argument("--graph", action="store_true", help="with --model: replay the pass from a captured CUDA graph")
    ap.add_argument("--no-graph", action="store_true",
                    help="bench step: launch the step's library calls one by one instead of replaying a CUDA graph of them")
    ap.add_argument("--pool", action="store_true",
                    help="time the two pooling operators at ResNet-50 batch-64 sizes instead of the step")
    ap.add_argument("--gemm", action="store_true",
                    help="time ONNX Gemm at a few sizes and attribute sets instead of the step")
    ap.add_argument("--probe-tf32", action="store_true",
                    help="measure the issue-rate ceiling of the TF32 tensor-core instruction instead of the step")
    ap.add_argument("--per-op", action="store_true",
                    help="add every op's duration inside the step (an event after each op) to the JSON line")
    ap.add_argument("--repack", action="store_true",
                    help="time onnx_conv2d_run (weights re-packed at every call) instead of the pre-packed form")
    ap.add_argument("--layers", action="store_true",
                    help="per-layer mode: one JSON line per distinct layer shape of the step and per configuration 1-4")
    ap.add_argument("--cpu-dry-run", action="store_true",
                    help="exercise the multi-rank launch path on CPU (gloo), no kernels; for tests")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        return spawn_ranks(args.gpus, sys.argv[1:])
    if args.cpu_dry_run:
        return run_cpu_dry_run(args)
    if args.impl == "reference":
        return run_reference(args)
    if args.layers:
        return run_layers(args)
    if args.probe_tf32:
        return run_probe_tf32()
    if args.pool:
        return run_pool()
    if args.gemm:
        return run_gemm()
    if args.model:
        return run_model(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
