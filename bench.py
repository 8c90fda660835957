#!/usr/bin/env python
"""Benchmark of the 3D complex DFT hot path (one JSON line on stdout).

A "step" is one whole 3D complex-to-complex transform of a seeded synthetic cube through the C-ABI
library (`dft3d_execute`: three per-axis tensor-core passes).  Default workload: the 1024^3 cube the
headline metric is quoted on, input U(-1,1), in the FFT formulation (GEMM - twiddle - GEMM per axis);
the KDFT formulation (dense N x N matrix per axis) of the same cube is timed in the same run and
reported under "kdft".  `value` is GFLOP/s in the 5*P*log2(P) convention (P points), with the input
already resident in HBM; `e2e` is the same metric through `dft3d_execute_host` with pinned HOST
buffers (H2D and D2H copies inside the timed region).

python bench.py [--gpus N] [--steps K] [--warmup W] [--mode fft|kdft] [--n 1024 | --shape a,b,c] [--impl reference]
Under torchrun every rank transforms its own cube (independent problems, no collective): weak scaling.
"""
import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

SMI_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--mode", choices=["kdft", "fft"], default=None)
    ap.add_argument("--n", type=int, default=1024)
    ap.add_argument("--shape", type=str, default=None, help="n0,n1,n2 instead of a cube (profiling on smaller cases)")
    ap.add_argument("--no-kdft", action="store_true", help="FFT mode only: skip the KDFT timing of the same cube")
    ap.add_argument("--split", choices=["default", "fp16", "tf32"], default="default",
                    help="operand split of the tensor-core products (default: the library's choice per formulation)")
    ap.add_argument("--axes", type=str, default=None,
                    help="transform only these axes, e.g. 1,2 with --shape 1,8192,8192 for the paper's 2D workload")
    ap.add_argument("--destroy-input", action="store_true",
                    help="plans use the input cube as their workspace (DFT3D_DESTROY_INPUT): for sizes where input + "
                         "output leave no room for one, e.g. 2048^3; the input is not regenerated between steps")
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    ap.add_argument("--config", type=str, default=None,
                    help="c1..c5 or all: the five configurations the parity tests cover, one JSON line each (time, "
                         "GFLOP/s in both conventions, issued tensor flops, roofline fraction, oracle seconds)")
    ap.add_argument("--md", type=str, default=None, help="with --config: also write the lines as a markdown table here")
    ap.add_argument("--traffic-from-ncu", nargs="+", default=None, metavar="KERNEL:POINTS:CSV",
                    help="no GPU work: read dram__bytes_read/write.sum per launch of KERNEL from an `ncu --csv` log of a "
                         "case with POINTS points per launch and write profiles/dram_bytes_per_point.json")
    return ap.parse_args()


def conv_flops(n):
    """5*P*log2(P); n is the cube edge or a shape tuple."""
    P = float(n) ** 3 if not isinstance(n, tuple) else float(n[0]) * n[1] * n[2]
    return 5.0 * P * math.log2(P)


TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_bytes_per_point.json")


def dram_bytes_per_point(kernel):
    """DRAM bytes per point and launch of `kernel` as ncu measured them (dram__bytes_read.sum + dram__bytes_write.sum
    of a capture divided by the points of that launch; traffic grows in proportion to the points).  The file is
    written by `bench.py --traffic-from-ncu` from the ncu logs; None when it has no entry for the kernel."""
    try:
        with open(TRAFFIC_FILE) as f:
            entry = json.load(f).get(kernel)
    except (OSError, ValueError):
        return None, None
    return (entry["bytes_per_point"], entry["case"]) if entry else (None, None)


def traffic_from_ncu(specs):
    """Parses `ncu --csv --metrics dram__bytes_read.sum,dram__bytes_write.sum ...` logs: mean bytes per launch of every
    launch whose kernel name starts with KERNEL, divided by POINTS."""
    import csv
    out = {}
    if os.path.exists(TRAFFIC_FILE):
        with open(TRAFFIC_FILE) as f:
            out = json.load(f)
    for spec in specs:
        kernel, points, path = spec.split(":", 2)
        per_launch = {}
        with open(path) as f:
            rows = [r for r in csv.reader(f) if len(r) > 10]
        hdr = rows[0]
        ki, mi, vi, ii = hdr.index("Kernel Name"), hdr.index("Metric Name"), hdr.index("Metric Value"), hdr.index("ID")
        for r in rows[1:]:
            base = r[ki].replace("void ", "").split("<")[0].split("(")[0]
            if base == kernel and r[mi] in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
                per_launch[r[ii]] = per_launch.get(r[ii], 0.0) + float(r[vi].replace(",", ""))
        if not per_launch:
            raise SystemExit("no launch of %s in %s" % (kernel, path))
        mean = sum(per_launch.values()) / len(per_launch)
        out[kernel] = {"bytes_per_point": mean / float(points), "launches": len(per_launch),
                       "points_per_launch": int(points), "case": os.path.basename(path)}
    with open(TRAFFIC_FILE, "w") as f:
        json.dump(out, f, indent=1, sort_keys=True)
        f.write("\n")
    print(json.dumps(out))


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + SMI_QUERY, "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        clocks, maxc, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    clocks.append(float(parts[1]))
                    maxc.append(float(parts[2]))
                    power.append(float(parts[3]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not clocks:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        load = sorted(c for c, p in zip(clocks, power) if p >= 0.5 * max(power)) or sorted(clocks)
        return {"sm_mhz": load[len(load) // 2], "sm_max_mhz": max(maxc), "power_w_max": max(power),
                "samples": len(clocks), "reasons": sorted(reasons)}


def oracle_planes(n):
    """Planes of the bounded oracle sample: about 3e10 complex MACs per transformed axis (1.5 s or more on the box's
    cores); both legs that time the oracle (the cpu_baseline of the GPU arm and --impl reference) use this one."""
    return max(1, min(n, int(3.0e10 / (float(n) ** 3))))


def oracle_sample(n, planes, seed):
    """Times the oracle, as it stands, on `planes` n0-planes of the workload: once along the last axis (its
    contiguous branch) and once along axis 1 (its strided branch, which axis 0 uses too), and extrapolates by the
    exact operation count (n complex MACs per point and axis) to a full transform: one contiguous and two strided
    axis passes over n/planes times as many planes."""
    import numpy as np
    from oracle import oracle
    from paper_2002_03260_b200 import inputs
    oracle.build()
    x = inputs.cube((planes, n, n), "uniform", seed, device="cpu").numpy().astype(np.complex128)
    t0 = time.perf_counter()
    oracle.dft_axis(x, 2)
    t1 = time.perf_counter()
    oracle.dft_axis(x, 1)
    t2 = time.perf_counter()
    dt_contig, dt_strided = t1 - t0, t2 - t1
    full_seconds = (dt_contig + 2.0 * dt_strided) * (n / planes)
    return {"value": conv_flops(n) / full_seconds * 1e-9, "unit": "GFLOP/s (5*P*log2P)", "cores": oracle.num_threads(),
            "kind": "oracle",
            "sample": "float64 direct summation over %d of %d n0-planes: last axis %.2f s, axis 1 %.2f s; extrapolated by "
                      "the exact operation count (%d complex MACs per point and axis; one contiguous and two strided "
                      "axis passes) to %.0f s per transform" % (planes, n, dt_contig, dt_strided, n, full_seconds),
            "seconds_measured": dt_contig + dt_strided,
            "seconds_per_transform_extrapolated": full_seconds}


def run_reference(args):
    """--impl reference: the oracle on the host cores, each step the same bounded sample of the workload that the
    GPU arm's cpu_baseline leg times."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n = args.n
    planes = oracle_planes(n)
    measured, full = [], []
    res = None
    for i in range(args.warmup + args.steps):
        res = oracle_sample(n, planes, 1003)
        if i >= args.warmup:
            measured.append(res["seconds_measured"])
            full.append(res["seconds_per_transform_extrapolated"])
    sec = sum(full) / len(full)
    value = conv_flops(n) / sec * 1e-9
    line = {"impl": "reference", "metric": "3D C2C DFT GFLOP/s (5*P*log2P) at %d^3" % n, "value": value,
            "unit": "GFLOP/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            # a step is the bounded sample that actually ran; the whole-transform figure is extrapolated from it
            "ms_per_step": sum(measured) / len(measured) * 1e3,
            "ms_per_transform_extrapolated": sec * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": "%d^3 complex64 cube, U(-1,1), float64 direct-summation oracle" % n,
                       "step": "%d of %d n0-planes, one contiguous-axis and one strided-axis pass" % (planes, n)},
            "cpu_baseline": {"value": value, "unit": "GFLOP/s", "cores": res["cores"], "kind": "oracle",
                             "sample": res["sample"]},
            "e2e": {"value": value, "unit": "GFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


CONFIGS = {
    # name: (shape, input recipe, what runs) -- the five configurations the parity tests cover
    "c1": ((64, 64, 64), "uniform:1001", [("kdft", -1, False)]),
    "c2": ((512, 512, 512), "normal:1002", [("kdft", -1, False), ("kdft", +1, False)]),
    "c3": ((1024, 1024, 1024), "uniform:1003", [("fft", -1, False), ("kdft", -1, False)]),
    "c4": ((256, 256, 256), "normal:1004", [("kdft", -1, True)]),
    "c5": ((2048, 2048, 2048), "exponentials:2005:1005", [("fft", -1, False), ("kdft", -1, False)]),
}


def run_configs(args):
    """--config: per configuration and formulation one JSON line: median and minimum time of a transform (CUDA events,
    3 warm-up + `reps` timed transforms, one event pair each), GFLOP/s in the 5*P*log2(P) convention and by the
    matrix-product flops the formulation defines (KDFT 8*n_a, FFT 8*(N1+N2) real flops per point and axis), the flops
    the tensor cores actually issue (three split products; the FFT kernels' R*R core), the roofline fraction, and the
    oracle's seconds on the host cores (whole transform where that takes under two minutes, else extrapolated from a
    sample and labelled so)."""
    import numpy as np
    import torch
    import paper_2002_03260_b200 as dft
    from paper_2002_03260_b200 import inputs
    from oracle import oracle
    oracle.build()
    torch.cuda.set_device(0)
    peaks, peak_kind = measured_peaks()
    names = sorted(CONFIGS) if args.config == "all" else [args.config]
    lines = []
    for name in names:
        shape, recipe, runs = CONFIGS[name]
        P = float(shape[0]) * shape[1] * shape[2]
        if P * 8 * 2.3 > torch.cuda.mem_get_info()[0]:
            sys.stderr.write("bench: %s does not fit this device, skipped\n" % name)
            continue
        kind = recipe.split(":")
        if kind[0] == "exponentials":
            x = inputs.exponentials(shape, 16, int(kind[1]), 1e-3, int(kind[2]), device="cuda")[0]
        else:
            x = inputs.cube(shape, kind[0], int(kind[1]), device="cuda")
        y = torch.empty_like(x)
        stream = torch.cuda.current_stream()
        # the oracle beside it: whole transform up to 512^3, a sample beyond
        n = shape[0]
        if P <= 512 ** 3:
            xh = x.cpu().numpy()
            nodes_o = inputs.sorted_nodes(shape, 2004) if runs[0][2] else None
            t0 = time.perf_counter()
            oracle.dft3d(xh, nodes=nodes_o)
            osec, okind = time.perf_counter() - t0, "whole transform"
            del xh
        else:
            smp = oracle_sample(n, oracle_planes(n), 1003)
            osec, okind = smp["seconds_per_transform_extrapolated"], "extrapolated from " + smp["sample"].split(";")[0]
        for mode, sign, with_nodes in runs:
            nodes = inputs.sorted_nodes(shape, 2004) if with_nodes else None
            limit = 4 * 2 ** 30 if (mode == "kdft" and P * 8 > 32 * 2 ** 30) else 0
            plan = dft.Plan(*shape, mode=dft.DFT3D_KDFT if mode == "kdft" else dft.DFT3D_FFT, sign=sign, nodes=nodes,
                            workspace_limit=limit)
            reps = 200 if P <= 64 ** 3 else (20 if P <= 1024 ** 3 else 3)
            for _ in range(3):
                plan.execute(x, y)
            torch.cuda.synchronize()
            sampler = ClockSampler(0)
            sampler.start()
            pairs = []
            for _ in range(reps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                plan.execute(x, y)
                e1.record(stream)
                pairs.append((e0, e1))
            torch.cuda.synchronize()
            clk = sampler.stop()
            plan.status()
            ms = sorted(a.elapsed_time(b) for a, b in pairs)
            med, mn = ms[len(ms) // 2], ms[0]
            f16 = plan.split == dft.DFT3D_SPLIT_FP16
            if mode == "kdft":
                gemm = 8.0 * sum(shape) * P
                issued = 3.0 * gemm
                peak = peaks["bf16_tflops_sustained"] * (1.0 if f16 else 1.1 / 2.25)
                roof = {"bound": "tensor", "achieved": issued / (med * 1e-3) * 1e-12, "peak": peak, "unit": "TFLOP/s",
                        "peak_source": "%s bf16 sustained%s" % (peak_kind, "" if f16 else " x 1.1/2.25 (TF32)")}
            else:
                splits = [plan.fft_split(a) for a in range(3)]
                gemm = 8.0 * sum(a + b for a, b in splits) * P
                issued = 3.0 * 8.0 * sum(2 * b for a, b in splits) * P
                roof = {"bound": "hbm", "achieved": 48.0 * P / (med * 1e-3) * 1e-9, "peak": peaks["hbm_gbs"],
                        "unit": "GB/s", "peak_source": "%s STREAM-style copy" % peak_kind}
            roof["frac"] = roof["achieved"] / roof["peak"]
            line = {"config": name, "shape": list(shape), "formulation": mode, "sign": sign, "nonuniform": with_nodes,
                    "split": "fp16" if f16 else "tf32", "launches": plan.launches, "reps": reps,
                    "ms_median": med, "ms_min": mn,
                    "gflops_5PlogP": conv_flops(shape) / (med * 1e-3) * 1e-9,
                    "gflops_gemm": gemm / (med * 1e-3) * 1e-9, "tflops_issued_tensor": issued / (med * 1e-3) * 1e-12,
                    "roofline": roof, "clocks": clk,
                    "oracle_seconds": osec, "oracle_kind": okind, "oracle_cores": oracle.num_threads()}
            print(json.dumps(line), flush=True)
            lines.append(line)
            plan.destroy()
        del x, y
        torch.cuda.empty_cache()
    if args.md:
        with open(args.md, "w") as f:
            f.write("| config | shape | formulation | split | launches | median ms | min ms | GFLOP/s (5P log2 P) | GFLOP/s "
                    "(matrix-product flops) | issued tensor TFLOP/s | roofline | SM MHz | oracle s (cores) |\n")
            f.write("|---|---|---|---|---|---|---|---|---|---|---|---|---|\n")
            for d in lines:
                r = d["roofline"]
                f.write("| %s | %s | %s%s%s | %s | %d | %.4g | %.4g | %.4g | %.4g | %.4g | %.2f of %s (%.4g of %.4g %s) | %s | %.4g (%d), %s |\n"
                        % (d["config"], "x".join(str(v) for v in d["shape"]), d["formulation"],
                           " inverse" if d["sign"] > 0 else "", " nonuniform" if d["nonuniform"] else "", d["split"],
                           d["launches"], d["ms_median"], d["ms_min"], d["gflops_5PlogP"], d["gflops_gemm"],
                           d["tflops_issued_tensor"], r["frac"], r["bound"], r["achieved"], r["peak"], r["unit"],
                           d["clocks"].get("sm_mhz"), d["oracle_seconds"], d["oracle_cores"], d["oracle_kind"]))


def main():
    args = parse_args()
    if args.traffic_from_ncu:
        traffic_from_ncu(args.traffic_from_ncu)
        return
    if args.impl == "reference":
        run_reference(args)
        return
    if args.config:
        run_configs(args)
        return
    import torch
    import torch.distributed as dist
    import paper_2002_03260_b200 as dft
    from paper_2002_03260_b200 import inputs, replicas

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the transform has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    n = args.n
    mode = args.mode or "fft"
    shape = (n, n, n) if not args.shape else tuple(int(v) for v in args.shape.split(","))
    x = inputs.cube(shape, "uniform", replicas.rank_seed(1003, rank), device="cuda")
    y = torch.empty_like(x)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def time_mode(mode_name, steps, warmup, sample_clocks):
        """W warm-up steps, then K timed steps between barriers; CUDA events on the launching stream; max over ranks."""
        flags = {"default": 0, "fp16": dft.DFT3D_SPLIT_FP16, "tf32": dft.DFT3D_SPLIT_TF32}[args.split]
        if args.destroy_input:
            flags |= dft.DFT3D_DESTROY_INPUT
        axes = tuple(int(v) for v in args.axes.split(",")) if args.axes else None
        plan_ = dft.Plan(*shape, mode=dft.DFT3D_KDFT if mode_name == "kdft" else dft.DFT3D_FFT, sign=dft.DFT3D_FORWARD,
                         flags=flags, axes=axes)
        for _ in range(warmup):
            plan_.execute(x, y)
        barrier()
        sampler = ClockSampler(local_rank)
        if sample_clocks and rank == 0:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            plan_.execute(x, y)
        e1.record(stream)
        barrier()
        clk = sampler.stop() if (sample_clocks and rank == 0) else None
        plan_.status()
        return plan_, replicas.max_over_ranks(e0.elapsed_time(e1), "cuda") / steps, clk

    plan, ms_step, clocks = time_mode(mode, args.steps, args.warmup, True)
    launches = plan.launches
    psplit, pws = plan.split, plan.workspace_bytes
    if args.no_e2e:
        plan.destroy()     # its workspace (half a cube at 2048^3) would sit beside the KDFT leg's
        plan = None
    kdft_info = None
    if mode == "fft" and not args.no_kdft:
        ksteps = max(1, min(args.steps, 10 if n <= 1024 else 3))
        kplan, kms, kclk = time_mode("kdft", ksteps, 3, True)
        kdft_info = {"ms_per_step": kms, "steps": ksteps, "warmup": 3, "launches_per_step": kplan.launches,
                     "split": "fp16" if kplan.split == dft.DFT3D_SPLIT_FP16 else "tf32", "clocks": kclk}
        ksplit = kplan.split
        kplan.destroy()

    # ---- end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        xh = x.cpu().pin_memory()
        yh = torch.empty_like(xh).pin_memory()
        plan.execute_host(xh, yh)   # warm-up, allocates the staging buffers
        barrier()
        # one call at a time: upload, transform, download, one after the other (the latency of a single transform)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        plan.execute_host(xh, yh)
        e1.record(stream)
        barrier()
        ms_single = replicas.max_over_ranks(e0.elapsed_time(e1), "cuda")
        # a stream of cubes: the download of one result runs under the upload of the next input.  Every step's
        # upload (from pinned host memory) and download are inside the timed region; two pinned inputs take turns
        e2e_steps = max(2, min(args.steps, 6))
        nbytes = x.numel() * 8
        try:
            xh2 = xh.clone().pin_memory()
            plan.execute_host_batch([xh, xh2], [yh, yh])   # warm-up, allocates the second pair of staging buffers
            streamed = True
        except (RuntimeError, MemoryError, dft.Dft3dError) as err:   # no room for the second buffers: single calls
            sys.stderr.write("bench: streamed e2e leg unavailable (%s); timing single calls\n" % err)
            streamed = False
        barrier()
        e0.record(stream)
        if streamed:
            plan.execute_host_batch([xh, xh2] * (e2e_steps // 2) + [xh] * (e2e_steps % 2), [yh] * e2e_steps)
        else:
            for _ in range(e2e_steps):
                plan.execute_host(xh, yh)
        e1.record(stream)
        barrier()
        ms_e2e = replicas.max_over_ranks(e0.elapsed_time(e1), "cuda") / e2e_steps
        e2e = {"value": world * conv_flops(shape) / ms_e2e * 1e-6, "unit": "GFLOP/s", "ms_per_step": ms_e2e,
               "h2d_bytes_per_step": nbytes, "d2h_bytes_per_step": nbytes, "steps": e2e_steps,
               "call": ("dft3d_execute_host_batch (pinned host buffers; the download of cube i overlaps the upload of "
                        "cube i+1; the first upload and the last download are inside the timed region)") if streamed
                       else "dft3d_execute_host (pinned host buffers), one call per step",
               "single_call_ms": ms_single,
               "single_call": "dft3d_execute_host: upload, transform, download one after the other"}
        xh2 = None
        del xh, yh

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        P = float(shape[0]) * shape[1] * shape[2]
        taxes = tuple(int(v) for v in args.axes.split(",")) if args.axes else (0, 1, 2)
        nsum = float(sum(shape[a] for a in taxes))   # lengths of the transformed axes

        def kdft_roofline(ms, nlaunch, split):
            # dominant kernel: the KDFT axis kernel (the fp16 split adds one small reduction over the input).
            # Algorithmic flops per point per axis = 8*n_a (4 real multiply-adds per complex MAC); the tensor cores
            # issue them three times (split products hi*hi, lo*hi, hi*lo).
            algo_flops = 8.0 * nsum * P
            issued = 3.0 * algo_flops
            ach = issued / (ms * 1e-3) * 1e-12
            if split == dft.DFT3D_SPLIT_FP16:
                paired = max(shape[a] for a in taxes) >= 2048 and os.environ.get("DFT3D_KDFT_PAIR", "1") != "0"
                kernel = "kdft_f16x2_axis_kernel" if paired else "kdft_f16_axis_kernel"   # CTA pairs from 2048 points up
                peak = peaks["bf16_tflops_sustained"]
                src = "%s bf16 sustained (fp16 and bf16 share the tensor rate)" % peak_kind
                axis_launches = nlaunch - 1
            else:
                kernel, peak = "kdft_axis_kernel", peaks["bf16_tflops_sustained"] * (1.1 / 2.25)
                src = "%s bf16 sustained x nominal TF32/bf16 ratio (1.1/2.25)" % peak_kind
                axis_launches = nlaunch
            return {"bound": "tensor", "kernel": kernel, "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                    "frac": ach / peak,
                    "traffic": (dram_bytes_per_point(kernel)[0] or 0.0) * P or None,
                    "traffic_note": "DRAM bytes per launch, ncu capture (%s) scaled by points (algorithmic: 16 B/point)"
                                    % dram_bytes_per_point(kernel)[1],
                    "peak_source": src,
                    "flops": "issued tensor flops = 3 split products x 8*n_a flops per point per axis",
                    "useful_gemm_tflops": algo_flops / (ms * 1e-3) * 1e-12, "avg_launch_ms": ms / axis_launches}

        if mode == "kdft":
            roofline = kdft_roofline(ms_step, launches, psplit)
        else:
            # only kernel: fft_axis_kernel, one launch per axis; algorithmic traffic 16 B per point per axis
            algo_bytes = len(taxes) * 16.0 * P
            achieved = algo_bytes / (ms_step * 1e-3) * 1e-9
            fkernel = "fft_f16_axis_kernel" if psplit == dft.DFT3D_SPLIT_FP16 else "fft_axis_kernel"
            roofline = {"bound": "hbm", "kernel": fkernel, "achieved": achieved, "peak": peaks["hbm_gbs"],
                        "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                        "traffic": (dram_bytes_per_point(fkernel)[0] or 0.0) * P or None,
                        "traffic_note": "DRAM bytes per launch, ncu capture (%s) scaled by points"
                                        % dram_bytes_per_point(fkernel)[1],
                        "bytes_per_point_algorithmic": 16.0 * len(taxes),
                        "peak_source": "%s STREAM-style copy" % peak_kind, "avg_launch_ms": ms_step / launches,
                        "bytes": "8 B read + 8 B written per point per axis pass"}
        if kdft_info is not None:
            kdft_info["value"] = world * conv_flops(shape) / kdft_info["ms_per_step"] * 1e-6
            kdft_info["unit"] = "GFLOP/s"
            kdft_info["roofline"] = kdft_roofline(kdft_info["ms_per_step"], kdft_info["launches_per_step"], ksplit)
        cpu = None
        if not args.no_cpu_baseline:
            cpu = oracle_sample(n, oracle_planes(n), 1003) if not args.shape else None
        wl = "%d^3" % n if not args.shape else "x".join(str(v) for v in shape)
        line = {"metric": "3D C2C DFT GFLOP/s (5*P*log2P) at %s" % wl,
                "value": world * conv_flops(shape) / ms_step * 1e-6, "unit": "GFLOP/s", "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "fp16x3" if psplit == dft.DFT3D_SPLIT_FP16 else "tf32x3", "data": "synthetic",
                "config": {"workload": "%s forward 3D complex64 DFT %s, re/im iid U(-1,1), seed 1003+rank" % (mode.upper(), wl),
                           "mode": mode, "shape": list(shape), "axes": list(taxes),
                           "l2": "input and output (%.2f GiB each) are larger than L2" % (P * 8 / 2**30),
                           "per_rank": "one independent cube per GPU",
                           "destroy_input": bool(args.destroy_input), "workspace_bytes": pws},
                "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches * args.steps,
                "clocks": clocks, "kdft": kdft_info}
        print(json.dumps(line))
    if plan is not None:
        plan.destroy()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
