#!/usr/bin/env python
"""Benchmark of the binary-convolution hot path.

One step = one pass of the whole path over one batch: the backbone-shaped sequence at
batch 256 (fp32 224x224x4 input -> bias + sign + 8x channel replication -> 18 fused
binary 3x3 / 1x1 convolutions with integer thresholds, packed activations resident on
the device).  Prints ONE JSON line (rank 0).

    python bench.py --gpus 1 --steps 20 --warmup 5
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference        # the CPU oracle on the host cores

With N > 1 every rank runs its own batch (images are independent, weights are
replicated, no collective on the data path): weak scaling, time = max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2010_00704_b200 import synth, workloads as wl  # noqa: E402

METRIC = "binary conv throughput (2*M*N*K bit-ops/s), backbone-shaped stack"
UNIT = "TOPS"
WORKLOAD = ("backbone18 @ batch 256: 224x224x4 fp32 -> pack(32ch) -> 18 fused binary conv layers (pack + layer 1 in one kernel; "
            "weights of the wide layers prepared once at set-up)")


# ----------------------------------------------------------------------------- helpers

def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def reduce_max(value: float, device=None) -> float:
    """Max over ranks of a host scalar (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(units_per_rank: float, world: int, max_seconds: float) -> float:
    """Whole-job throughput: the units all ranks processed divided by the slowest rank's time."""
    return units_per_rank * world / max_seconds


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                    "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    "source": "measured"}
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        def pump():
            for line in self.proc.stdout:
                self.rows.append(line.strip())
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in self.rows:
            f = [c.strip() for c in row.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "power_w_max": float(max(power)),
                "samples": len(sm), "reasons": sorted(reasons)}


def backbone_inputs(batch: int, rank: int = 0):
    """Seeded synthetic tensors of the backbone workload (host side)."""
    layers = wl.BACKBONE18
    H, W, C, R = wl.BACKBONE18_INPUT
    rng = synth.rng_for(5, 500 + rank)
    x = synth.real_input(rng, (batch, H, W, C))
    bias = synth.real_input(synth.rng_for(5, 499), (C * R,))
    ws = [synth.random_bits(synth.rng_for(5, i + 1), (l.C_out, l.k, l.k, l.C_in // 8)) for i, l in enumerate(layers)]
    ts = [synth.thresholds(synth.rng_for(5, 100 + i), l.K, l.C_out) for i, l in enumerate(layers)]
    return x, bias, ws, ts


# ----------------------------------------------------------------------------- CPU oracle legs

def oracle_backbone_seconds(n_images: int, x, bias, ws, ts):
    """Time the CPU oracle, as it stands, on the first n_images images of the workload."""
    import oracle
    layers = wl.BACKBONE18
    _, _, _, R = wl.BACKBONE18_INPUT
    wpm = [synth.unpack_bits(w) for w in ws]
    t0 = time.perf_counter()
    cur = oracle.binarize(x[:n_images], bias, R)
    for l, w, t in zip(layers, wpm, ts):
        cur = oracle.threshold(oracle.conv2d(cur, w, l.stride, l.pad), t)
    return time.perf_counter() - t0


def checker_backbone_seconds(n_images: int, x, bias, ws, ts):
    """Time the bit-packed CPU checker (xor + popcount loops; not the oracle) on the first n_images images."""
    import oracle
    layers = wl.BACKBONE18
    _, _, _, R = wl.BACKBONE18_INPUT
    cur = synth.pack_bits(oracle.binarize(x[:n_images], bias, R))       # untimed: the checker starts from packed bits
    t0 = time.perf_counter()
    for l, w, t in zip(layers, ws, ts):
        acc = oracle.checker_conv2d(cur, w, (n_images, l.H, l.W, l.C_in, l.C_out, l.k, l.k), l.stride, l.pad)
        cur = synth.pack_bits(np.where(acc >= t, 1, -1).astype(np.int8))
    return time.perf_counter() - t0


def cpu_baseline(target_seconds: float = 15.0):
    import oracle
    oracle.build()
    cap = 192
    x, bias, ws, ts = backbone_inputs(cap)
    t1 = oracle_backbone_seconds(2, x, bias, ws, ts) / 2
    n = int(max(1, min(cap, target_seconds / max(t1, 1e-3))))
    secs = oracle_backbone_seconds(n, x, bias, ws, ts)
    ops = wl.chain_ops(wl.BACKBONE18, n)
    c1 = checker_backbone_seconds(2, x, bias, ws, ts) / 2
    nc = int(max(1, min(cap, 5.0 / max(c1, 1e-3))))
    csecs = checker_backbone_seconds(nc, x, bias, ws, ts)
    return {"value": ops / secs / 1e12, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"first {n} images of the batch through pack + 18 layers ({secs:.1f} s)",
            "images_per_s": n / secs,
            "packed_checker": {"value": wl.chain_ops(wl.BACKBONE18, nc) / csecs / 1e12, "unit": UNIT, "cores": oracle.threads(),
                               "kind": "bit-packed xor + popcount loops (the tests' full-coverage checker, not the oracle)",
                               "sample": f"first {nc} images through the 18 layers ({csecs:.1f} s)", "images_per_s": nc / csecs}}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    import oracle
    oracle.build()
    x, bias, ws, ts = backbone_inputs(16)
    t1 = oracle_backbone_seconds(1, x, bias, ws, ts)
    budget = 150.0 / max(1, args.steps + args.warmup)
    n = int(max(1, min(16, budget / max(t1, 1e-3))))
    for _ in range(args.warmup):
        oracle_backbone_seconds(n, x, bias, ws, ts)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_backbone_seconds(n, x, bias, ws, ts)
    secs = time.perf_counter() - t0
    ops = wl.chain_ops(wl.BACKBONE18, n) * args.steps
    value = ops / secs / 1e12
    sample = f"{n} images of the batch-256 workload per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8 (+-1) / int32",
        "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
        "images_per_s": n * args.steps / secs,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- instruction probes

PROBES_SRC = os.path.join(ROOT, "bench_probes.cu")
PROBES_LIB = os.path.join(ROOT, "bench_probes.so")


def build_probes() -> str:
    """Compile bench_probes.cu (instruction-throughput probes) into bench_probes.so beside this file."""
    csrc = os.path.join(ROOT, "paper_2010_00704_b200", "csrc")
    deps = [PROBES_SRC, os.path.join(csrc, "tc_common.cuh"), os.path.join(csrc, "bcnn_common.cuh")]
    if not os.path.exists(PROBES_LIB) or os.path.getmtime(PROBES_LIB) < max(os.path.getmtime(d) for d in deps):
        tmp = PROBES_LIB + f".tmp{os.getpid()}"
        subprocess.run([os.environ.get("NVCC", "nvcc"), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3",
                        "-std=c++17", "-shared", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"), "-I", csrc,
                        "-o", tmp, PROBES_SRC, "-lcudart"], check=True)
        os.replace(tmp, PROBES_LIB)
    return PROBES_LIB


def run_probes():
    """Instruction peaks measured in this process (TOP/s, 1 MAC = 2 ops); see bench_probes.cu."""
    import ctypes
    lib = ctypes.CDLL(build_probes())
    dbl, i32 = ctypes.c_double, ctypes.c_int
    out = {}
    ms, macs, derr = dbl(0), dbl(0), i32(0)
    for n in (256, 128, 64, 32):
        st = lib.probe_tcgen05_i8(n, 4000 * (256 // n), ctypes.byref(ms), ctypes.byref(macs), ctypes.byref(derr))
        if st != 0 or derr.value != 0:
            raise SystemExit(f"tcgen05 probe failed: status {st}, device error {derr.value}")
        out[f"tcgen05_i8_n{n}"] = 2 * macs.value / (ms.value / 1e3) / 1e12
    for mode, name in ((0, "mma_sync_b1_and_popc"), (1, "mma_sync_b1_xor_popc"), (2, "mma_sync_s8")):
        st = lib.probe_mma_sync(mode, 2000 if mode < 2 else 20000, ctypes.byref(ms), ctypes.byref(macs))
        if st != 0:
            raise SystemExit(f"mma.sync probe failed: status {st}")
        out[name] = 2 * macs.value / (ms.value / 1e3) / 1e12
    st = lib.probe_popc(20000, ctypes.byref(ms), ctypes.byref(macs))
    if st != 0:
        raise SystemExit(f"popc probe failed: status {st}")
    out["xor_popc"] = 2 * macs.value / (ms.value / 1e3) / 1e12
    return out


def roofline_traffic(summary_name: str, sources):
    """DRAM bytes per launch from a tracked ncu summary under profiles/ (a line `traffic_bytes_per_launch: N`), or
    None when there is none or when the kernel's sources changed after the capture (the summary's `source_sha` line
    is the sha1 of the concatenated source files)."""
    import hashlib
    path = os.path.join(ROOT, "profiles", summary_name)
    if not os.path.exists(path):
        return None
    fields = {}
    for line in open(path):
        if ":" in line:
            k, v = line.split(":", 1)
            fields[k.strip()] = v.strip()
    h = hashlib.sha1()
    for src in sources:
        h.update(open(os.path.join(ROOT, "paper_2010_00704_b200", "csrc", src), "rb").read())
    if fields.get("source_sha") != h.hexdigest():
        return None
    try:
        return int(fields["traffic_bytes_per_launch"])
    except (KeyError, ValueError):
        return None


# ----------------------------------------------------------------------------- GPU arm

def timed_launches(fn, steps: int, warmup: int, flush=None):
    """CUDA-event time of each of `steps` calls of fn (ms), after `warmup` untimed ones; `flush` (a device buffer
    larger than L2) is overwritten before every timed call."""
    import torch
    for _ in range(warmup):
        fn()
    ts = []
    for _ in range(steps):
        if flush is not None:
            flush.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b))
    return ts


def bound_and_frac(ops: float, nbytes: float, ms: float, tensor_peak: float, hbm_gbs: float):
    """The roof that bounds a launch (the slower of ops / tensor peak and bytes / HBM peak) and the fraction of it
    reached: floor time / measured time."""
    t_tensor = ops / (tensor_peak * 1e12) * 1e3
    t_hbm = nbytes / (hbm_gbs * 1e9) * 1e3
    bound = "tensor" if t_tensor >= t_hbm else "hbm"
    return bound, max(t_tensor, t_hbm) / ms


def other_configs(tensor_peak: float, hbm_gbs: float, steps: int = 20, warmup: int = 5):
    """The other benchmark workloads (single 3x3 layer, GEMM sweep int32 + fused - plain calls and the calls on
    prepared weights -, stem / down-sampling layers, block stack), AUTO engine, 20 launches each with L2 flushed in
    between: median and min time, TOP/s and the fraction of
    the bounding roof (tensor pipe or HBM, on algorithmic bytes: packed inputs + weights + output)."""
    import torch
    from paper_2010_00704_b200 import binding
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    rng = np.random.default_rng(synth.seed_for(2, 77))
    rows = []

    def add(name, fn, ops, nbytes):
        ts = timed_launches(fn, steps, warmup, flush)
        med, mn = float(np.median(ts)), float(min(ts))
        bound, frac = bound_and_frac(ops, nbytes, med, tensor_peak, hbm_gbs)
        rows.append({"name": name, "ms_median": med, "ms_min": mn, "tops": ops / (med / 1e3) / 1e12, "bound": bound,
                     "frac": frac, "algorithmic_bytes": int(nbytes)})

    def conv_case(tag, l, B, fused=True):
        x = torch.from_numpy(synth.random_bits(rng, (l.in_bytes(B),))).cuda()
        Wb = torch.from_numpy(synth.random_bits(rng, (l.w_bytes(),))).cuda()
        if fused:
            thr = torch.from_numpy(synth.thresholds(rng, l.K, l.C_out)).cuda()
            out = torch.empty(l.out_bits_bytes(B), dtype=torch.uint8, device="cuda")
            fn = lambda: binding.bcnn_conv2d_b1_fused(x, Wb, thr, out, B, l.H, l.W, l.C_in, l.C_out, l.k, l.k, l.stride, l.pad)
            ob = l.out_bits_bytes(B)
        else:
            out = torch.empty(l.M(B) * l.C_out, dtype=torch.int32, device="cuda")
            fn = lambda: binding.bcnn_conv2d_b1(x, Wb, out, B, l.H, l.W, l.C_in, l.C_out, l.k, l.k, l.stride, l.pad)
            ob = 4 * l.M(B) * l.C_out
        add(f"{tag} {l.name} B={B} M={l.M(B)} N={l.C_out} K={l.K} {'fused' if fused else 'int32'}", fn, l.ops(B),
            l.in_bytes(B) + l.w_bytes() + ob)

    conv_case("single3x3:", wl.SINGLE_3X3, wl.SINGLE_3X3_BATCH, fused=False)
    for mn_ in wl.GEMM_SWEEP_MN:
        for k in wl.GEMM_SWEEP_K:
            M = N = mn_
            A = torch.from_numpy(synth.random_bits(rng, (M, k // 8))).cuda()
            Wb = torch.from_numpy(synth.random_bits(rng, (N, k // 8))).cuda()
            thr = torch.from_numpy(synth.thresholds(rng, k, N)).cuda()
            out32 = torch.empty(M * N, dtype=torch.int32, device="cuda")
            outb = torch.empty(M * N // 8, dtype=torch.uint8, device="cuda")
            ops = wl.gemm_ops(M, N, k)
            add(f"gemm M=N={M} K={k} int32", lambda: binding.bcnn_gemm_b1(A, Wb, out32, M, N, k), ops, (M + N) * k // 8 + 4 * M * N)
            add(f"gemm M=N={M} K={k} fused", lambda: binding.bcnn_gemm_b1_fused(A, Wb, thr, outb, M, N, k), ops,
                (M + N) * k // 8 + M * N // 8)
            # the same products on prepared weights (expanded once by bcnn_prepare_weights, outside the timed call)
            prep = torch.empty(binding.bcnn_prepared_weights_bytes(N, k), dtype=torch.uint8, device="cuda")
            binding.bcnn_prepare_weights(Wb, prep, N, k)
            add(f"gemm M=N={M} K={k} int32, prepared weights", lambda: binding.bcnn_gemm_b1_prepared(A, prep, None, out32, M, N, k),
                ops, (M + N) * k // 8 + 4 * M * N)
            add(f"gemm M=N={M} K={k} fused, prepared weights", lambda: binding.bcnn_gemm_b1_prepared(A, prep, thr, outb, M, N, k),
                ops, (M + N) * k // 8 + M * N // 8)
            del A, Wb, thr, out32, outb, prep
    for l in wl.STEM_DOWN:
        conv_case("stem/down:", l, wl.STEM_DOWN_BATCH)
    for l in wl.BLOCK_STACK:
        conv_case("block stack:", l, wl.BLOCK_STACK_BATCH)
    return rows


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2010_00704_b200 import build, binding
    from paper_2010_00704_b200.chain import FusedChain

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    build.build()
    binding.load()
    peaks = load_peaks()
    probes = run_probes() if rank == 0 else None

    layers = wl.BACKBONE18
    B = wl.BACKBONE18_BATCH
    H, W, C, R = wl.BACKBONE18_INPUT
    x, bias, ws, ts = backbone_inputs(B, rank)
    chain = FusedChain(layers, B, ws, ts, real_input_shape=(H, W, C), bias=bias, replicate=R, device=device)
    x_host = torch.from_numpy(x.reshape(-1)).pin_memory()
    chain.x_real.copy_(x_host, non_blocking=True)
    torch.cuda.synchronize()
    ops_step = wl.chain_ops(layers, B)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timed region (CUDA graph replay of the fused stem + 17 layers); an event after every
    # step gives the per-step times too
    chain.capture()
    for _ in range(max(args.warmup, 3)):
        chain.run()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    marks[0].record()
    for s in range(args.steps):
        chain.run()
        marks[s + 1].record()
    barrier()
    ms_total = reduce_max(marks[0].elapsed_time(marks[-1]), device)
    step_ms = [marks[s].elapsed_time(marks[s + 1]) for s in range(args.steps)]
    clocks = sampler.stop() if rank == 0 else None
    err = binding.bcnn_device_error()
    if err != 0:
        raise SystemExit(f"device-side error code {err}: {binding.status_string(err)}")
    ms_step = ms_total / args.steps
    value = aggregate_throughput(ops_step * args.steps, world, ms_total / 1e3) / 1e12

    # ---- sustained leg: the same graph replayed back to back for at least two seconds (warm, power-limited GPU)
    n_sus = max(args.steps, int(np.ceil(args.sustain_seconds * 1e3 / ms_step)))
    sampler_s = ClockSampler(local_rank)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    if rank == 0:
        sampler_s.start()
    e0.record()
    for _ in range(n_sus):
        chain.run()
    e1.record()
    barrier()
    ms_sus = reduce_max(e0.elapsed_time(e1), device)
    clocks_sus = sampler_s.stop() if rank == 0 else None
    value_sus = aggregate_throughput(ops_step * n_sus, world, ms_sus / 1e3) / 1e12

    # ---- end to end: pinned host input -> device, whole path, result back to the host
    out_host = torch.empty(chain.outs[-1].numel(), dtype=torch.uint8).pin_memory()
    def e2e_step():
        # host -> device copy of this step's input (copy stream, overlapping the previous step's kernels),
        # fused stem + 17 layers, packed result back to the host
        chain.run_from_host(x_host, out_host)
    for _ in range(3):
        e2e_step()
    barrier()
    e0.record()
    for _ in range(args.steps):
        e2e_step()
    e1.record()
    barrier()
    ms_e2e = reduce_max(e0.elapsed_time(e1), device)
    e2e_value = aggregate_throughput(ops_step * args.steps, world, ms_e2e / 1e3) / 1e12

    # ---- per-kernel pass: the same launches, one CUDA-event pair around each; clocks sampled during it
    nl = len(layers)
    per = np.zeros((args.steps, nl + 1))
    evs = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(nl + 1)]
           for _ in range(args.steps)]
    fused_stem = chain.fuse_stem
    sampler_k = ClockSampler(local_rank)
    if rank == 0:
        sampler_k.start()
    # the same kernel-by-kernel launches, unrecorded, for about 0.7 s first, so that the clock sampler sees the state
    # the recorded launches run in
    t_lead = time.perf_counter()
    while time.perf_counter() - t_lead < 0.7:
        chain.enqueue()
        torch.cuda.current_stream().synchronize()
    for s in range(args.steps):
        a, b = evs[s][0]
        a.record()
        chain.enqueue_pack(chain.x_real)          # the pack kernel, or the fused stem (pack + first layer)
        b.record()
        cur = chain.in_bits
        for i, (l, w, t, o) in enumerate(zip(layers, chain.w, chain.thr, chain.outs)):
            if i == 0 and fused_stem:
                cur = o
                continue
            a, b = evs[s][i + 1]
            a.record()
            cur = chain.enqueue_layer(i, cur)
            b.record()
    torch.cuda.synchronize()
    clocks_k = sampler_k.stop() if rank == 0 else None
    for s in range(args.steps):
        for i in range(nl + 1):
            if not (i == 1 and fused_stem):
                per[s, i] = evs[s][i][0].elapsed_time(evs[s][i][1])
    per_ms = per.mean(axis=0)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    # Tensor peak: the tcgen05.mma kind::i8 rate measured in this process by the tensor-memory-resident probe
    # (N = 256 instructions back to back).  Beside it, 2 x the measured bf16 GEMM peaks (the nominal 2:1 ratio of
    # the dense 8-bit and 16-bit pipes): burst for launches timed alone at the maximum clock, sustained for a warm,
    # power-limited GPU.  Which of the two applies to the per-launch times is decided by the clocks sampled
    # while those launches ran.
    tensor_peak = probes["tcgen05_i8_n256"]
    peak_alt = {"2x_bf16_burst": 2.0 * peaks["bf16_tflops"], "2x_bf16_sustained": 2.0 * peaks["bf16_tflops_sustained"]}
    def regime_of(c):
        if not c or not c.get("sm_mhz") or not c.get("sm_max_mhz"):
            return "unknown"
        return "burst" if c["sm_mhz"] >= 0.95 * c["sm_max_mhz"] else "sustained"
    regime = regime_of(clocks_k)
    alt_key = "2x_bf16_sustained" if regime == "sustained" else "2x_bf16_burst"
    engines = [chain.engine_name(i) for i in range(nl)]   # "stem": the first layer runs inside the stem kernel (slot 0 of per_ms)
    kernel_of = {"tc_i8": "conv_tc_i8_kernel (tcgen05 kind::i8)", "mma_s8": "conv_mma_s8_kernel (mma.sync u8)",
                 "mma_b1": "conv_mma_b1_kernel (mma.sync b1)",
                 "tc_ws": "conv_tc_ws_kernel (tcgen05 kind::i8, weights resident in shared memory)",
                 "tc_pw": "conv_tc_pw_kernel (tcgen05 kind::i8, pointwise layers, bulk-copied rows)",
                 "tc_pre": "conv_tc_pre_kernel (tcgen05 kind::i8, prepared weights streamed by TMA)",
                 "tc_c3": "conv_tc_c3_kernel (tcgen05 kind::i8, 3x3 layers on 32/64 channels, halo tiles by TMA)",
                 "tc_pn": "conv_tc_pn_kernel (tcgen05 kind::i8, pointwise layers with K = 256 / 512, resident weight slices)",
                 "lop3": "conv_k32_kernel (CUDA-core xor + popc)"}
    lay_ms = [float(per_ms[0]) if engines[i] == "stem" else float(per_ms[i + 1]) for i in range(nl)]
    per_layer = []
    for i, l in enumerate(layers):
        nbytes = l.in_bytes(B) + l.w_bytes() + l.out_bits_bytes(B)
        bound, frac = bound_and_frac(l.ops(B), nbytes, lay_ms[i], tensor_peak, peaks["hbm_gbs"])
        per_layer.append({"layer": l.name + (" (with the pack, one kernel)" if engines[i] == "stem" else ""), "engine": engines[i],
                          "ms": lay_ms[i], "tops": l.ops(B) / (lay_ms[i] / 1e3) / 1e12, "bound": bound, "frac": frac})
    groups = []
    for en in sorted(set(engines) - {"stem"}):
        idx = [i for i, e in enumerate(engines) if e == en]
        g_ms = float(sum(per_ms[i + 1] for i in idx))
        g_ops = float(sum(layers[i].ops(B) for i in idx))
        # the CUDA-core kernel sits on the population-count unit: its peak is the xor + popc rate of the probe
        g_bound, g_peak = ("alu", probes["xor_popc"]) if en == "lop3" else ("tensor", tensor_peak)
        groups.append({"kernel": kernel_of[en], "launches_per_step": len(idx), "ms_per_step": g_ms,
                       "share_of_step": g_ms / float(per_ms.sum()), "bound": g_bound,
                       "achieved": g_ops / (g_ms / 1e3) / 1e12, "peak": g_peak, "unit": "TOP/s",
                       "frac": g_ops / (g_ms / 1e3) / 1e12 / g_peak})
    groups.sort(key=lambda g: -g["ms_per_step"])
    # the roofline entry describes the dominant kernel's costliest launch: algorithmic ops of that
    # layer / its average launch duration (CUDA events around each launch, averaged over the steps)
    dom_engine = [e for e in kernel_of if kernel_of[e] == groups[0]["kernel"]][0]
    # (layers of equal shape time within noise of each other: the first one within 7 % of the slowest stands for them)
    dom_idx = [i for i, e in enumerate(engines) if e == dom_engine]
    slowest = max(per_ms[i + 1] for i in dom_idx)
    top = next(i for i in dom_idx if per_ms[i + 1] >= 0.93 * slowest)
    lt = layers[top]
    top_tops = lt.ops(B) / (per_ms[top + 1] / 1e3) / 1e12
    src_of = {"tc_ws": ["conv_tc_ws.cu", "tc_common.cuh"], "tc_i8": ["conv_tc_i8.cu", "tc_common.cuh"],
              "tc_pw": ["conv_tc_pw.cu", "tc_slot.cuh", "tc_common.cuh"], "tc_pre": ["conv_tc_pre.cu", "tc_common.cuh"],
              "tc_c3": ["conv_tc_c3.cu", "tc_slot.cuh", "tc_common.cuh"],
              "tc_pn": ["conv_tc_pn.cu", "tc_slot.cuh", "tc_common.cuh"]}
    roofline = {
        "kernel": groups[0]["kernel"], "launch": f"{lt.name}: M={lt.M(B)} N={lt.C_out} K={lt.K}",
        "bound": "tensor", "achieved": top_tops, "peak": tensor_peak, "unit": "TOP/s", "frac": top_tops / tensor_peak,
        "peak_source": "tcgen05.mma kind::i8 (M=128, N=256, K=32, A in tensor memory) issued back to back, measured in this "
                       f"process by bench_probes.cu; peak_alt = 2 x the {peaks['source']} bf16 GEMM peaks (MEASURED_PEAKS.json), "
                       f"of {peaks['source']}",
        "peak_alt": peak_alt, "frac_alt": {k: top_tops / v for k, v in peak_alt.items()},
        "regime": regime, "frac_of_regime_peak": top_tops / peak_alt[alt_key],
        "regime_source": "median SM clock sampled while the per-launch events ran: burst when within 5 % of the maximum",
        "clocks_during_launch_timing": clocks_k,
        "launch_ms": float(per_ms[top + 1]),
        "launch_ms_x_sm_mhz": (float(per_ms[top + 1]) * clocks_k["sm_mhz"]) if clocks_k and clocks_k.get("sm_mhz") else None,
        "ops_per_launch": int(lt.ops(B)),
        "traffic": roofline_traffic(f"conv_{dom_engine}_{lt.name}.txt", src_of.get(dom_engine, [])),
        "kernels": groups,
        "instruction_peaks_tops": probes,
    }
    # pack: 16 bytes read, 4 written per pixel; the fused stem writes the first layer's 4 bytes instead
    pack_bytes = B * H * W * C * 4 + B * H * W * (layers[0].C_out if fused_stem else C * R) // 8
    pack = {"kernel": "stem_c4r8_k32_kernel (pack + first 1x1 layer, table look-up)" if fused_stem else "pack_c4r8_kernel",
            "ms": float(per_ms[0]), "bound": "hbm",
            "achieved": pack_bytes / (per_ms[0] / 1e3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": pack_bytes / (per_ms[0] / 1e3) / 1e9 / peaks["hbm_gbs"], "algorithmic_bytes": pack_bytes}

    configs = other_configs(tensor_peak, peaks["hbm_gbs"]) if world == 1 and not args.no_configs else None
    err = binding.bcnn_device_error()
    if err != 0:
        raise SystemExit(f"device-side error code {err}: {binding.status_string(err)}")
    cpu = cpu_baseline() if world == 1 and not args.no_cpu_baseline else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "ms_per_step_median": float(np.median(step_ms)),
        "ms_per_step_min": float(min(step_ms)), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "b1 (sign bits) with int32 accumulation", "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch_per_gpu": B, "layers": nl,
                   "cache": "inputs larger than L2 (205.5 MB fp32 input read every step)",
                   "launch": f"CUDA graph replay of {chain.launches_per_run} kernels"},
        "images_per_s": B * world * args.steps / (ms_total / 1e3),
        "clocks": clocks,
        "value_sustained": value_sus,
        "sustained": {"value": value_sus, "unit": UNIT, "steps": n_sus, "seconds": ms_sus / 1e3, "ms_per_step": ms_sus / n_sus,
                      "images_per_s": B * world * n_sus / (ms_sus / 1e3), "clocks": clocks_sus, "regime": regime_of(clocks_sus)},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(x_host.numel() * 4),
                "d2h_bytes_per_step": int(out_host.numel()), "ms_per_step": ms_e2e / args.steps,
                "api": "FusedChain.run_from_host: pinned host input, copy stream overlapping the previous step",
                "images_per_s": B * world * args.steps / (ms_e2e / 1e3)},
        "gpu_launches": int(args.steps * chain.launches_per_run),
        "roofline": roofline,
        "pack": pack,
        "per_layer": per_layer,
        "configs": configs,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_sweep(args):
    """Engine comparison on the GEMM sweep and the single-layer workloads (not the headline line).

    Prints one JSON object per (shape, output kind, engine): time (median of --steps launches after
    --warmup), TOPS and, for the int32 output, the output write rate."""
    import torch
    from paper_2010_00704_b200 import build, binding
    build.build()
    binding.load()
    torch.cuda.set_device(0)
    engines = args.engines.split(",")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

    def timeit(fn):
        for _ in range(args.warmup):
            fn()
        ts = []
        for _ in range(args.steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return float(np.median(ts)), float(min(ts))

    rows = []
    rng = np.random.default_rng(1)
    shapes = []
    if args.sweep_set in ("gemm", "all"):
        for mn in wl.GEMM_SWEEP_MN:
            for k in wl.GEMM_SWEEP_K:
                shapes.append(("gemm", mn, mn, k, None, 1))
    if args.sweep_set in ("conv", "all"):
        shapes.append(("conv", None, None, None, wl.SINGLE_3X3, wl.SINGLE_3X3_BATCH))
        for l in wl.STEM_DOWN:
            shapes.append(("conv", None, None, None, l, wl.STEM_DOWN_BATCH))
        for l in wl.BLOCK_STACK:
            shapes.append(("conv", None, None, None, l, wl.BLOCK_STACK_BATCH))
        for l in wl.BACKBONE18:
            shapes.append(("conv", None, None, None, l, wl.BACKBONE18_BATCH))
    if args.sweep_set == "paper":
        for l, _count in wl.paper_binary_1x1_convs(1):
            shapes.append(("conv", None, None, None, l, wl.BACKBONE18_BATCH))
    for kind, M, N, K, l, B in shapes:
        label = f"gemm M=N={M} K={K}" if kind == "gemm" else f"conv {l.name} "
        if args.only and args.only not in label:
            continue
        if kind == "gemm":
            A = torch.from_numpy(synth.random_bits(rng, (M, K // 8))).cuda()
            Wb = torch.from_numpy(synth.random_bits(rng, (N, K // 8))).cuda()
            thr = torch.from_numpy(synth.thresholds(rng, K, N)).cuda()
            out32 = torch.empty(M * N, dtype=torch.int32, device="cuda")
            outb = torch.empty(M * N // 8, dtype=torch.uint8, device="cuda")
            ops = wl.gemm_ops(M, N, K)
            name = f"gemm M=N={M} K={K}"
            prep = torch.empty(binding.bcnn_prepared_weights_bytes(N, K), dtype=torch.uint8, device="cuda")
            binding.bcnn_prepare_weights(Wb, prep, N, K)
            calls = {
                "int32": lambda e: binding.bcnn_gemm_b1_prepared(A, prep, None, out32, M, N, K) if e == "tc_pre"
                else binding.bcnn_gemm_b1(A, Wb, out32, M, N, K, engine=e),
                "fused": lambda e: binding.bcnn_gemm_b1_prepared(A, prep, thr, outb, M, N, K) if e == "tc_pre"
                else binding.bcnn_gemm_b1_fused(A, Wb, thr, outb, M, N, K, engine=e),
            }
            out_bytes = {"int32": 4 * M * N, "fused": M * N // 8}
        else:
            x = torch.from_numpy(synth.random_bits(rng, (l.in_bytes(B),))).cuda()
            Wb = torch.from_numpy(synth.random_bits(rng, (l.w_bytes(),))).cuda()
            thr = torch.from_numpy(synth.thresholds(rng, l.K, l.C_out)).cuda()
            outb = torch.empty(l.out_bits_bytes(B), dtype=torch.uint8, device="cuda")
            ops = l.ops(B)
            name = f"conv {l.name} B={B} M={l.M(B)} N={l.C_out} K={l.K}"
            prep = torch.empty(binding.bcnn_prepared_weights_bytes(l.C_out, l.K), dtype=torch.uint8, device="cuda")
            binding.bcnn_prepare_weights(Wb, prep, l.C_out, l.K)
            calls = {
                "fused": lambda e: binding.bcnn_conv2d_b1_prepared(x, prep, thr, outb, B, l.H, l.W, l.C_in, l.C_out, l.k, l.k,
                                                                    l.stride, l.pad) if e == "tc_pre"
                else binding.bcnn_conv2d_b1_fused(x, Wb, thr, outb, B, l.H, l.W, l.C_in, l.C_out,
                                                  l.k, l.k, l.stride, l.pad, engine=e),
            }
            out_bytes = {"fused": l.out_bits_bytes(B)}
        for okind, call in calls.items():
            if okind not in args.outs.split(","):
                continue
            for en in engines:
                e = "tc_pre" if en == "tc_pre" else binding.ENGINES[en]      # tc_pre: the *_prepared calls (weights expanded once)
                try:
                    med, mn_ = timeit(lambda: call(e))
                except binding.BcnnError as ex:
                    rows.append({"shape": name, "out": okind, "engine": en, "error": str(ex)})
                    continue
                rows.append({"shape": name, "out": okind, "engine": en, "ms": med, "ms_min": mn_,
                             "tops": ops / (med / 1e3) / 1e12, "out_gbs": out_bytes[okind] / (med / 1e3) / 1e9})
                print(json.dumps(rows[-1]), flush=True)
    err = binding.bcnn_device_error()
    print(json.dumps({"device_error": err}))
    return 0 if err == 0 else 1


def run_paper1x1(args):
    """The paper's own binary workload (not the headline line): the 32 binary 1x1 convolutions of the
    network of Table 1 (2.41e9 binary MACs per image; 64 convolutions for P = 2 parallel branches), each
    with the fused threshold epilogue, on independent seeded inputs (the real-valued depth-wise / batch
    norm / PReLU steps between them are outside the binary hot path).  One step = all convolutions for
    one batch, replayed from a CUDA graph.  Prints one JSON line."""
    import torch
    from paper_2010_00704_b200 import build, binding
    build.build()
    binding.load()
    torch.cuda.set_device(0)
    B, P = args.batch, args.branches
    module = args.epilogue == "module"
    peaks = load_peaks()
    # with the module epilogue the P branches of a module are ONE call (bcnn_conv2d_b1_branches: P binarizations side
    # by side in the packed input, P weight sets, P batch norms, summed before the identity); with the threshold
    # epilogue they are P independent convolutions
    branch_call = module and P > 1
    convs = wl.paper_binary_1x1_convs(1 if branch_call else P)
    PB = P if branch_call else 1
    jobs = []
    for li, (l, count) in enumerate(convs):
        rng = synth.rng_for(6, li)
        x = torch.from_numpy(synth.random_bits(rng, (PB * l.in_bytes(B),))).cuda()
        ident = yreal = None
        if module:
            # the module's real input (fp16 NHWC, standard normal) and its real output, shared by the repeats
            ident = torch.randn(l.M(B) * l.C_out, dtype=torch.float16, device="cuda",
                                generator=torch.Generator(device="cuda").manual_seed(synth.seed_for(6, li)))
            yreal = torch.empty(l.M(B) * l.C_out, dtype=torch.float16, device="cuda")
        for c in range(count):
            Wb = torch.from_numpy(synth.random_bits(rng, (PB * l.w_bytes(),))).cuda()
            thr = torch.from_numpy(synth.thresholds(rng, l.K, l.C_out)).cuda()
            out = torch.empty(l.out_bits_bytes(B), dtype=torch.uint8, device="cuda")
            extra = None
            if module:
                sc = torch.from_numpy((rng.standard_normal(PB * l.C_out) / np.sqrt(l.K)).astype(np.float32)).cuda()
                sh = torch.from_numpy(synth.real_input(rng, (PB * l.C_out,))).cuda()
                nb = torch.from_numpy(synth.real_input(rng, (l.C_out,))).cuda()
                sl = torch.from_numpy(rng.uniform(0.0, 0.5, l.C_out).astype(np.float32)).cuda()
                extra = (sc, sh, ident, sl, nb, yreal)
            elif binding.bcnn_prepared_preferred(B, l.H, l.W, l.C_in, l.C_out, 1, 1, 1, 0):
                # as FusedChain does: a layer's weights are expanded once, at set-up, where the library prefers that
                prep = torch.empty(binding.bcnn_prepared_weights_bytes(l.C_out, l.K), dtype=torch.uint8, device="cuda")
                binding.bcnn_prepare_weights(Wb, prep, l.C_out, l.K)
                extra = prep
            jobs.append((l, x, Wb, thr, out, extra))

    def launch(j):
        l, x, Wb, thr, out, extra = j
        if module:
            sc, sh, idn, sl, nb, yr = extra
            if branch_call:
                binding.bcnn_conv2d_b1_branches(x, Wb, sc, sh, None, idn, sl, nb, yr, out, B, l.H, l.W, l.C_in, l.C_out, P)
            else:
                binding.bcnn_conv2d_b1_module(x, Wb, sc, sh, idn, sl, nb, yr, out, B, l.H, l.W, l.C_in, l.C_out, 1, 1, 1, 0)
        elif extra is not None:
            binding.bcnn_conv2d_b1_prepared(x, extra, thr, out, B, l.H, l.W, l.C_in, l.C_out, 1, 1, 1, 0)
        else:
            binding.bcnn_conv2d_b1_fused(x, Wb, thr, out, B, l.H, l.W, l.C_in, l.C_out, 1, 1, 1, 0)

    def step():
        for j in jobs:
            launch(j)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    for _ in range(max(args.warmup, 3)):
        g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    ms_step = e0.elapsed_time(e1) / args.steps
    # per shape: CUDA events around each launch, averaged
    per = {}
    for _ in range(args.steps):
        for j in jobs:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            launch(j)
            b.record()
            per.setdefault(j[0].name, []).append((a, b))
    torch.cuda.synchronize()
    shapes = []
    for l, count in convs:
        ms = float(np.mean([a.elapsed_time(b) for a, b in per[l.name]]))
        shapes.append({"layer": l.name, "count": count, "M": l.M(B), "N": l.C_out, "K": l.K,
                       "engine": ("branches (CUDA cores)" if branch_call else "tc_ws") if module
                       else ("tc_pre" if binding.bcnn_prepared_preferred(B, l.H, l.W, l.C_in, l.C_out, 1, 1, 1, 0)
                             else binding.bcnn_auto_engine(B, l.H, l.W, l.C_in, l.C_out, 1, 1, 1, 0)),
                       "ms_per_launch": ms, "tops": PB * l.ops(B) / (ms / 1e3) / 1e12})
        # algorithmic bytes: packed input + packed output (+ fp16 identity read and fp16 map written by the module)
        nbytes = PB * l.in_bytes(B) + l.out_bits_bytes(B) + (4 * l.M(B) * l.C_out if module else 0)
        shapes[-1].update({"gbs": nbytes / (ms / 1e3) / 1e9, "hbm_frac": nbytes / (ms / 1e3) / 1e9 / peaks["hbm_gbs"]})
    err = binding.bcnn_device_error()
    ops = 2 * PB * sum(n * l.macs(B) for l, n in convs)
    print(json.dumps({
        "mode": "paper1x1", "epilogue": args.epilogue, "metric": "binary conv throughput (2*M*N*K bit-ops/s), the paper's 1x1 convolutions (Table 1)",
        "value": ops / (ms_step / 1e3) / 1e12, "unit": UNIT, "ms_per_step": ms_step, "images_per_s": B / (ms_step / 1e3),
        "binary_macs_per_image": ops // (2 * B), "n_gpus": 1, "steps": args.steps, "data": "synthetic",
        "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"],
        "config": {"workload": f"Table 1 network, binary 1x1 convolutions only, P = {P}, batch {B}, epilogue {args.epilogue}",
                   "launches": len(jobs),
                   "launch": "CUDA graph replay"},
        "per_shape": shapes, "device_error": err}))
    return 0 if err == 0 else 1


def run_block(args):
    """The real-valued vector operations of the paper's building block and head at the shapes of Table 1 (not the
    headline line): depth-wise 3x3 module at stride 1 and 2 (with the next module's sign bits), S x S average pooling
    with replication on the identity path, global pooling + fully connected layer; median of --steps launches with L2
    flushed in between; achieved GB/s on algorithmic bytes against the measured copy bandwidth.  One JSON line."""
    import torch
    from paper_2010_00704_b200 import build, binding
    build.build()
    binding.load()
    torch.cuda.set_device(0)
    B = args.batch
    peaks = load_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    gen = torch.Generator(device="cuda").manual_seed(synth.seed_for(7))
    rows = []

    def add(name, fn, nbytes):
        ts = timed_launches(fn, args.steps, args.warmup, flush)
        med = float(np.median(ts))
        rows.append({"op": name, "ms_median": med, "ms_min": float(min(ts)), "algorithmic_bytes": int(nbytes),
                     "gbs": nbytes / (med / 1e3) / 1e9, "hbm_frac": nbytes / (med / 1e3) / 1e9 / peaks["hbm_gbs"]})

    def f32(n):
        return torch.randn(n, dtype=torch.float32, device="cuda", generator=gen)

    # (level, resolution of the block's input, channels before replication, R, S) of the down-sampling blocks and of
    # one normal block per level (Table 1)
    for name, H, C_in, R, S in (("level1 down", 224, 32, 2, 2), ("level2 down", 112, 64, 2, 2), ("level3 down", 56, 128, 2, 2),
                                ("level3 normal", 28, 256, 1, 1), ("level4 down", 28, 256, 2, 2), ("level4 normal", 14, 512, 1, 1),
                                ("level5 down", 14, 512, 2, 2), ("level5 normal", 7, 1024, 1, 1)):
        C = C_in * R
        OH = (H - 1) // S + 1
        x = torch.randn(B * H * H * C_in, dtype=torch.float16, device="cuda", generator=gen)
        y = torch.empty(B * OH * OH * C, dtype=torch.float16, device="cuda")
        bits = torch.empty(B * OH * OH * C // 8, dtype=torch.uint8, device="cuda")
        w, sc, sh, sl, nb = f32(C * 9), f32(C), f32(C), f32(C), f32(C)
        add(f"{name}: depth-wise 3x3 / {S} module {H}x{H}x{C_in} -> {OH}x{OH}x{C} (+ next signs)",
            lambda: binding.bcnn_dwconv3x3_module(x, w, sc, sh, sl, nb, y, bits, B, H, H, C_in, R, S),
            2 * x.numel() + 2 * y.numel() + bits.numel())
        if S > 1:
            add(f"{name}: {S}x{S}/{S} average pooling, replication {R}, {H}x{H}x{C_in} -> {OH}x{OH}x{C}",
                lambda: binding.bcnn_avgpool(x, y, B, H, H, C_in, R, S), 2 * x.numel() + 2 * y.numel())
        del x, y, bits
    x = torch.randn(B * 49 * 1024, dtype=torch.float16, device="cuda", generator=gen)
    pooled = torch.empty(B * 1024, dtype=torch.float32, device="cuda")
    logits = torch.empty(B * 1000, dtype=torch.float32, device="cuda")
    wfc, bfc = f32(1000 * 1024), f32(1000)
    add("head: global average pooling 7x7x1024", lambda: binding.bcnn_gap(x, pooled, B, 7, 7, 1024), 2 * x.numel() + 4 * pooled.numel())
    add("head: fully connected 1024 -> 1000", lambda: binding.bcnn_fc(pooled, wfc, bfc, logits, B, 1024, 1000),
        4 * (pooled.numel() + wfc.numel() + logits.numel()))
    print(json.dumps({"mode": "block", "batch": B, "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"], "ops": rows,
                      "device_error": binding.bcnn_device_error()}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--mode", default="bench", choices=["bench", "sweep", "paper1x1", "block"])
    ap.add_argument("--engines", default="auto,lop3,mma_b1,tc_i8,mma_s8,tc_ws,tc_pw,tc_c3,tc_pn,tc_pre")
    ap.add_argument("--sweep-set", default="all", choices=["gemm", "conv", "all", "paper"])
    ap.add_argument("--only", default="", help="sweep mode: run only shapes whose label contains this text")
    ap.add_argument("--outs", default="int32,fused", help="sweep mode: output kinds to run")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the other workloads (single layer, GEMM sweep, stem / down, block stack)")
    ap.add_argument("--sustain-seconds", type=float, default=2.0, help="length of the sustained leg")
    ap.add_argument("--batch", type=int, default=256, help="paper1x1 mode: images per step")
    ap.add_argument("--epilogue", default="threshold", choices=["threshold", "module"],
                    help="paper1x1 mode: integer threshold, or the full convolution module (batch norm, fp16 identity, PReLU, next sign)")
    ap.add_argument("--branches", type=int, default=1, choices=[1, 2], help="paper1x1 mode: parallel binary branches P")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.mode == "sweep":
        return run_sweep(args)
    if args.mode == "paper1x1":
        return run_paper1x1(args)
    if args.mode == "block":
        return run_block(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
