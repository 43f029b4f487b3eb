#!/usr/bin/env python
"""Benchmark of the fixed-point 8-bit inference path: one step = one forward pass of the
ResNet-50-shaped fixed-point network on a batch of 256 synthetic 224x224x3 int8 images.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--layers] [--no-workloads]

Prints one JSON line (rank 0).  `value` is images/s with inputs resident in HBM; `e2e` is the same
metric through the library's host-buffer call (f8_net_forward_host): the image batch is copied from
pinned host memory and the logits are copied back every step.  `workloads` holds the other
configurations (layer sweep at batch 32, MobileNetV2 / V1 and ResNet-18 shaped networks at several
batches) with their layer-wise bound and a short timing of the CPU oracle.
With --impl reference the CPU oracle is timed instead (a deliberately plain program: context only).
With --gpus N and no launcher (WORLD_SIZE unset) the script starts N local ranks itself; under
torchrun it joins the ranks it is given.  Every rank runs the same batch on its own GPU (replicas,
no collective on the data path); the elapsed time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import socket
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2202_05239_b200 import synth  # noqa: E402

METRIC = "fixed-point inference images/sec"
UNIT = "images/s"
WORKLOAD = "resnet50_fixed_point_b256"
NET, BATCH, SEED = "resnet50", 256, 0
INT8_NOMINAL_TOPS = 4500.0


# ----------------------------------------------------------------------------- distributed plumbing

def dist_env():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def dist_init(backend: str):
    import torch.distributed as dist
    rank, _, world = dist_env()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, world


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """Maximum of a per-rank scalar (the job is as slow as its slowest rank)."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_per_step: int, steps: int, world: int, elapsed_ms_max: float) -> float:
    return units_per_rank_per_step * steps * world / (elapsed_ms_max * 1e-3)


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_local_ranks(n: int, argv) -> int:
    """`--gpus N` without a launcher: start N ranks of this script on this node (rank i on GPU i) and wait for them."""
    port = str(free_port())
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=port)
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=env))
    rc = 0
    for p in procs:
        rc = max(rc, p.wait())
    return rc


def dist_selftest(args):
    """The multi-rank plumbing alone, on CPU (gloo): rendezvous, barrier, max over ranks; rank 0 prints the world size."""
    rank, world = dist_init("gloo")
    barrier(world)
    slowest = max_over_ranks(float(rank + 1), world)
    assert slowest == float(world), (slowest, world)
    barrier(world)
    if rank == 0:
        print(json.dumps({"selftest": "dist", "n_gpus": world, "requested": args.gpus,
                          "value": whole_job_rate(BATCH, 1, world, 1000.0)}), flush=True)


# ----------------------------------------------------------------------------- clocks

CLOCK_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
               "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
               "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")


class ClockSampler:
    def __init__(self, gpu_index: int):
        self.proc = None
        self.path = os.path.join("/tmp", f"f8_clocks_{os.getpid()}.csv")
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={CLOCK_QUERY}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu_index), "-lms", "50"], stdout=self.f,
                                         stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.f.close()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1]))
                    smax.append(float(parts[2]))
                except ValueError:
                    continue
                for name, flag in zip(names, parts[5:9]):
                    if flag.lower().startswith("active"):
                        reasons.add(name)
            os.remove(self.path)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ----------------------------------------------------------------------------- reference arm / CPU baseline

def time_oracle(layers, images: int, seed: int):
    """Times the CPU oracle, as it stands, on `images` images of the workload; returns (images/s, seconds, threads)."""
    from oracle import f8ref
    f8ref.lib()
    first = layers[0]
    x = synth.draw_image(images, seed + 1, first.h, first.w, first.c)
    t0 = time.perf_counter()
    f8ref.net_forward(layers, x, keep_all=False)
    dt = time.perf_counter() - t0
    return images / dt, dt, f8ref.threads()


def cpu_baseline(layers, batch: int, workload: str, target_seconds: float = 15.0):
    ips1, dt1, threads = time_oracle(layers, min(4, batch), SEED)      # sizing probe (rows of an image run in parallel)
    n = int(max(1, min(batch, round(target_seconds * ips1))))
    if n <= 4:
        ips, dt = ips1, dt1
        n = min(4, batch)
    else:
        ips, dt, threads = time_oracle(layers, n, SEED)
    return {"value": ips, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"{n} of the {batch} images of {workload} ({dt:.1f} s); images are independent, so the rate is per image"}


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    layers = synth.make_net(NET, SEED)
    sample = 4
    for _ in range(max(0, min(args.warmup, 1))):
        time_oracle(layers, 1, SEED)
    t0 = time.perf_counter()
    threads = 0
    for _ in range(args.steps):
        _, _, threads = time_oracle(layers, sample, SEED)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": WORKLOAD, "net": NET, "global_batch": BATCH,
                       "note": f"each step is a {sample}-image sample of the batch run through the CPU oracle"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"{sample} images per step x {args.steps} steps"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- roofline helpers

def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured"
    except (OSError, KeyError, ValueError):
        return 6650.0, "fallback"


def shape_key(l) -> str:
    return f"{l.h}x{l.w}x{l.c}->{l.c_out} k{l.kh} s{l.stride} res{1 if l.res >= 0 else 0}"


def measured_traffic(layers, tc_flags, batch):
    """DRAM bytes per step of the tensor-core conv kernel: per-launch counters of every distinct layer shape, captured
    one single-layer launch at a time (profiles/dram_traffic_conv_gemm_tc_shapes.md; scaled by batch / capture batch
    when the two differ) and summed over the layers.  None when the kernel source has changed since, or a shape is
    missing."""
    try:
        text = open(os.path.join(ROOT, "profiles", "dram_traffic_conv_gemm_tc_shapes.md")).read()
        sha = re.search(r"kernel_source_sha256:\s*([0-9a-f]{64})", text).group(1)
        cap_batch = int(re.search(r"capture_batch:\s*(\d+)", text).group(1))
        src = open(os.path.join(ROOT, "paper_2202_05239_b200", "csrc", "f8_gemm_tc.cu"), "rb").read()
        if hashlib.sha256(src).hexdigest() != sha:
            return None
        table = {}
        for m in re.finditer(r"^\|\s*([^|]+?)\s*\|\s*([\d.]+)\s*\|\s*([\d.]+)\s*\|", text, flags=re.M):
            table[m.group(1)] = (float(m.group(2)) + float(m.group(3))) * 1e6
        total = 0.0
        for l, tc in zip(layers, tc_flags):
            if not tc or l.kind != synth.CONV:
                continue
            if shape_key(l) not in table:
                return None
            total += table[shape_key(l)] * batch / cap_batch
        return int(total)
    except (OSError, AttributeError, ValueError):
        return None


def layerwise_bound_ms(layers, batch, peak_gbs, peak_tops):
    """Sum over layers of max(bytes / HBM peak, ops / INT8 peak): the best a layer-by-layer execution can do."""
    hbm = tensor = both = 0.0
    for l in layers:
        b = batch * l.bytes_per_image() + l.param_bytes()
        o = 2.0 * batch * l.macs_per_image
        t_h = b / (peak_gbs * 1e9) * 1e3
        t_t = o / (peak_tops * 1e12) * 1e3 if l.kind in (synth.CONV, synth.LINEAR) else 0.0
        hbm += t_h
        tensor += t_t
        both += max(t_h, t_t)
    return both, hbm, tensor


# ----------------------------------------------------------------------------- the other configurations

def time_net(api, torch, layers, batch, steps, flush):
    """ms per forward pass of a whole network (CUDA events), launches per pass, micro-batching.  flush: write a buffer larger
    than L2 between passes and time each pass on its own (for configurations whose tensors would otherwise stay in L2)."""
    net = api.Net(layers, batch)
    first = layers[0]
    x = api.to_device(synth.draw_image(batch, SEED + 1, first.h, first.w, first.c))
    out = torch.empty((batch,) + net.out_shape, dtype=net.out_dtype, device="cuda")
    ws = torch.empty(net.workspace_bytes(batch), dtype=torch.uint8, device="cuda")
    for _ in range(3):
        net.forward(x, out=out, workspace=ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if flush is None:
        e0.record()
        for _ in range(steps):
            net.forward(x, out=out, workspace=ws)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
    else:
        total = 0.0
        for _ in range(steps):
            flush.fill_(1)
            e0.record()
            net.forward(x, out=out, workspace=ws)
            e1.record()
            torch.cuda.synchronize()
            total += e0.elapsed_time(e1)
        ms = total / steps
    api.f8_device_status()
    launches, micro = net.last_launch_count, net.micro_batching()
    net.close()
    return ms, launches, micro


def run_workloads(api, torch, peak_gbs, probe_tops, steps):
    """Configurations other than the headline one: throughput, the layer-wise bound, which roofline binds, the oracle."""
    from paper_2202_05239_b200 import layer_bench
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    flush = torch.empty(2 * l2, dtype=torch.uint8, device="cuda")
    out = []
    # the layer-shape sweep at batch 32: single-layer calls over rotating buffer sets larger than L2
    from oracle import f8ref
    f8ref.lib()
    for i in range(len(synth.SWEEP_SHAPES)):
        layer, x = synth.sweep_case(i, batch=32, seed=0)
        r = layer_bench.bench_layer(layer, 32, False, max(10, steps), 3)
        t_h = r["bytes"] / (peak_gbs * 1e9) * 1e3
        t_t = 2.0 * r["macs"] / (probe_tops * 1e12) * 1e3
        t0 = time.perf_counter()
        f8ref.run_layer(layer, x)
        dt = time.perf_counter() - t0
        out.append({"workload": f"layer_sweep_b32/{layer.name}", "unit": "layers/s", "value": 1e3 / r["ms"], "ms": r["ms"],
                    "tops": r["tops"], "gbs": r["gbs"], "bound": "tensor" if t_t > t_h else "hbm",
                    "bound_ms": max(t_h, t_t), "roofline_frac": max(t_h, t_t) / r["ms"],
                    "l2": f"{r['buffer_sets']} rotating buffer sets (together larger than L2)",
                    "cpu_baseline": {"value": 1.0 / dt, "unit": "layers/s", "cores": f8ref.threads(), "kind": "oracle",
                                     "sample": "the whole layer at batch 32"}})
    for name, batch in (("mobilenetv2", 1), ("mobilenetv2", 64), ("resnet18", 1), ("resnet18", 64), ("resnet18", 256),
                        ("mobilenetv1", 64), ("mobilenetv1", 256), ("resnet50", 1)):
        layers = synth.make_net(name, SEED)
        step_bytes = synth.net_bytes(layers, batch)
        small = step_bytes < 2 * l2
        ms, launches, micro = time_net(api, torch, layers, batch, steps if not small else min(steps, 20), flush if small else None)
        bound, hbm, tensor = layerwise_bound_ms(layers, batch, peak_gbs, probe_tops)
        ips1, dt1, threads = time_oracle(layers, min(2, batch), SEED)
        out.append({"workload": f"{name}_fixed_point_b{batch}", "unit": UNIT, "value": batch / (ms * 1e-3), "ms": ms,
                    "launches": launches, "micro_batched_runs": micro[0], "micro_batch": micro[1],
                    "tops": 2.0 * batch * synth.net_macs_per_image(layers) / (ms * 1e-3) / 1e12,
                    "gbs": step_bytes / (ms * 1e-3) / 1e9,
                    "bound": "tensor" if tensor > hbm else "hbm", "bound_ms": bound, "roofline_frac": bound / ms,
                    "l2": "flushed between passes (each pass timed on its own)" if small else "no flush: a pass moves more than twice the L2",
                    "cpu_baseline": {"value": ips1, "unit": UNIT, "cores": threads, "kind": "oracle",
                                     "sample": f"{min(2, batch)} images ({dt1:.1f} s)"}})
    return out


# ----------------------------------------------------------------------------- our arm

def run_ours(args):
    import torch
    from paper_2202_05239_b200 import api

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the fixed-point path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist_init("nccl")

    layers = synth.make_net(NET, SEED)
    net = api.Net(layers, BATCH)
    x_host = torch.from_numpy(synth.draw_image(BATCH, SEED + 1 + rank)).pin_memory()
    x_dev = x_host.to(dev)
    out = torch.empty((BATCH, 1000), dtype=torch.int32, device=dev)
    out_host = torch.empty((BATCH, 1000), dtype=torch.int32).pin_memory()
    ws = torch.empty(net.workspace_bytes(BATCH), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        net.forward(x_dev, out=out, workspace=ws)

    # ---- device-resident throughput
    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    api.f8_device_status()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_steps():
        """K steps between a barrier + synchronize on both sides; clocks sampled while the GPU runs them."""
        sampler = ClockSampler(local_rank)
        if rank == 0:
            sampler.start()
            # the sampler's first line takes nvidia-smi a moment: keep the GPU under the same load meanwhile
            for _ in range(max(3, min(args.steps, 100))):
                step()
        barrier(world)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(args.steps):
            step()
        e1.record(stream)
        torch.cuda.synchronize()
        barrier(world)
        ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
        return ms, (sampler.stop() if rank == 0 else None)

    incidents = []

    def device_ok(where: str) -> bool:
        """Reads the device status word; a kernel that gave up a bounded wait is recorded, not fatal the first time."""
        try:
            api.f8_device_status()
            return True
        except api.F8Error as exc:
            incidents.append(f"{where}: {exc}")
            if len(incidents) > 2:
                raise
            return False

    def on_any_rank(flag: bool) -> bool:
        """The ranks repeat a measurement together or not at all (it contains barriers)."""
        return max_over_ranks(1.0 if flag else 0.0, world, dev) > 0.0

    elapsed_ms, clocks = timed_steps()
    if on_any_rank(not device_ok("timed steps")):
        elapsed_ms, clocks = timed_steps()      # that measurement contained a 2 s time-out: take it again
        if on_any_rank(not device_ok("timed steps, second run")):
            raise SystemExit("bench.py: bounded waits timed out twice: " + "; ".join(incidents))
    if rank == 0:
        throttled = bool(set(clocks["reasons"]) & {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"})
        stuck = (clocks["sm_mhz"] is not None and not clocks["reasons"] and clocks["sm_mhz"] < 0.8 * clocks["sm_max_mhz"])
        again = torch.tensor([1 if (throttled or stuck) else 0], device=dev)
    else:
        again = torch.tensor([0], device=dev)
    if world > 1:
        import torch.distributed as dist
        dist.broadcast(again, 0)
    if int(again.item()):
        first = clocks
        elapsed_ms, clocks = timed_steps()      # rejected once: measure again
        if rank == 0:
            clocks["rejected_first"] = {"sm_mhz": first["sm_mhz"], "reasons": first["reasons"]}
    launches_per_step = net.last_launch_count
    launches = launches_per_step * args.steps
    value = whole_job_rate(BATCH, args.steps, world, elapsed_ms)
    micro = net.micro_batching()

    # ---- end to end through the library's host-buffer call (f8_net_forward_host behind api.HostPipeline): uploads,
    # forward passes and downloads of consecutive steps overlap; every step still moves its own input and result.
    pipe = api.HostPipeline(layers, BATCH, depth=2, device=dev)
    x_hosts = [x_host, x_host.clone().pin_memory()]
    out_hosts = [out_host, torch.empty_like(out_host).pin_memory()]
    for i in range(4):
        pipe.submit(x_hosts[i & 1], out_hosts[i & 1])
    pipe.wait()
    torch.cuda.synchronize()
    device_ok("end-to-end warm-up")
    t_e0, t_e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_e2e():
        barrier(world)
        t_e0.record(pipe.up_stream)                  # before the first upload ...
        for i in range(args.steps):
            pipe.submit(x_hosts[i & 1], out_hosts[i & 1])
        t_e1.record(pipe.down_stream)                # ... to after the last download
        pipe.wait()
        torch.cuda.synchronize()
        barrier(world)
        return max_over_ranks(t_e0.elapsed_time(t_e1), world, dev)

    e2e_ms = timed_e2e()
    if on_any_rank(not device_ok("end-to-end steps")):
        e2e_ms = timed_e2e()
        if on_any_rank(not device_ok("end-to-end steps, second run")):
            raise SystemExit("bench.py: bounded waits timed out twice: " + "; ".join(incidents))
    e2e_value = whole_job_rate(BATCH, args.steps, world, e2e_ms)
    e2e_ok = bool(torch.equal(out_hosts[0], out.cpu()))      # same images as the device-resident run: same logits
    pipe.close()
    del pipe

    # ---- per-layer device times of the timed configuration (events between the launches)
    net.set_profiling(True)
    reps = max(3, min(10, args.steps))
    acc_ms = np.zeros(len(layers))
    tc_flags = None
    for _ in range(reps):
        step()
        ms, tc_flags = net.layer_ms()
        acc_ms += np.array(ms)
    net.set_profiling(False)
    layer_ms = acc_ms / reps

    # ---- attainable INT8 rate of this device (MMA-only probe), same run
    iters = 4096
    api.f8_mma_i8_probe(iters)      # warm-up
    torch.cuda.synchronize()
    e0.record(stream)
    ops = api.f8_mma_i8_probe(iters)
    e1.record(stream)
    torch.cuda.synchronize()
    probe_tops = ops / (e0.elapsed_time(e1) * 1e-3) / 1e12
    device_ok("per-layer timing and probe")

    if rank != 0:
        return
    peak_gbs, peak_kind = measured_peaks()
    ms_per_step = elapsed_ms / args.steps
    # The events between the launches switch the overlap of consecutive layers off, so the per-layer times add up to
    # more than a step takes.  A kernel cannot take longer than the step that contains it: the per-layer times are
    # scaled by (timed step / sum of event times) so that they add up to the step.
    event_sum = float(layer_ms.sum())
    scale = min(1.0, ms_per_step / event_sum) if event_sum > 0 else 1.0
    tc_bytes = tc_ops = tc_ms = 0.0
    other_bytes = other_ms = 0.0
    per_layer = []
    fused_into_next = [False] * len(layers)      # a first layer whose kernel also computes the max pool behind it
    for i in range(len(layers) - 1):
        if layers[i].kind == synth.CONV and layers[i + 1].kind == synth.MAXPOOL and layer_ms[i] == 0.0 and layer_ms[i + 1] > 0.0:
            fused_into_next[i] = True
    # a 64 -> 64 convolution that runs in one launch with the pointwise layer behind it (f8_conv_pw_fused_tc_kernel): the
    # time is recorded with the second layer, the tensor between the two never reaches memory
    pair_first = [False] * len(layers)
    for i in range(len(layers) - 1):
        if (layers[i].kind == synth.CONV and layers[i + 1].kind == synth.CONV and layers[i + 1].src == i + 1 and layer_ms[i] == 0.0 and
                layer_ms[i + 1] > 0.0 and tc_flags[i] and tc_flags[i + 1]):
            pair_first[i] = True
    pair_bytes = pair_ops = pair_ms = 0.0
    for i, (l, ms_raw, tc) in enumerate(zip(layers, layer_ms, tc_flags)):
        ms = float(ms_raw) * scale
        if pair_first[i]:
            continue                              # counted with the pointwise layer below
        if i > 0 and pair_first[i - 1]:
            first = layers[i - 1]
            b = (BATCH * (first.h * first.w * first.c + l.ho * l.wo * l.c_out * (2 if l.res >= 0 else 1)) + first.param_bytes() +
                 l.param_bytes())
            o = 2.0 * BATCH * (first.macs_per_image + l.macs_per_image)
            pair_bytes += b
            pair_ops += o
            pair_ms += ms
            per_layer.append({"name": first.name + "+" + l.name, "ms": round(ms, 5), "ms_events": round(float(ms_raw), 5), "tc": True,
                              "gbs": round(b / (ms * 1e-3) / 1e9, 1) if ms > 0 else None,
                              "tops": round(o / (ms * 1e-3) / 1e12, 1) if ms > 0 else None})
            continue
        b = BATCH * l.bytes_per_image() + l.param_bytes()
        o = 2.0 * BATCH * l.macs_per_image
        if fused_into_next[i]:
            continue                              # counted with the pooling layer below
        first_kernel = i > 0 and fused_into_next[i - 1]
        if first_kernel:
            # one kernel: reads the image and the first layer's parameters, writes the pooled tensor; the
            # intermediate tensor never reaches memory, so it is not counted as traffic
            first = layers[i - 1]
            b = BATCH * (first.h * first.w * first.c + l.ho * l.wo * l.c_out) + first.param_bytes()
            o = 2.0 * BATCH * first.macs_per_image
        if tc and not first_kernel:
            tc_bytes += b
            tc_ops += o
            tc_ms += ms
        else:
            other_bytes += b
            other_ms += ms
        per_layer.append({"name": (layers[i - 1].name + "+" + l.name) if first_kernel else l.name,
                          "ms": round(ms, 5), "ms_events": round(float(ms_raw), 5), "tc": bool(tc),
                          "gbs": round(b / (ms * 1e-3) / 1e9, 1) if ms > 0 else None,
                          "tops": round(o / (ms * 1e-3) / 1e12, 1) if ms > 0 else None})
    assert tc_ms + pair_ms + other_ms <= ms_per_step * (1 + 1e-6), "per-kernel times exceed the step they are part of"
    achieved = tc_bytes / (tc_ms * 1e-3) / 1e9 if tc_ms > 0 else 0.0
    total_ops = 2.0 * BATCH * synth.net_macs_per_image(layers)
    n_pairs = int(sum(pair_first))
    n_tc = int(sum(1 for l, tc in zip(layers, tc_flags) if tc and l.kind in (synth.CONV, synth.LINEAR))) - 2 * n_pairs
    bound_ms, hbm_ms, tensor_ms = layerwise_bound_ms(layers, BATCH, peak_gbs, probe_tops)
    roofline = {
        "kernel": "f8_conv_gemm_tc_kernel",
        "bound": "hbm", "achieved": achieved, "peak": peak_gbs, "unit": "GB/s", "frac": achieved / peak_gbs,
        "peak_source": f"{peak_kind} HBM copy bandwidth",
        "traffic": measured_traffic(layers, [bool(tc) and not pair_first[i] and not (i > 0 and pair_first[i - 1])
                                             for i, tc in enumerate(tc_flags)], BATCH),
        "traffic_note": "DRAM bytes of this kernel's launches in one step: ncu counters of one cold single-layer launch per distinct layer "
                        "shape at the bench batch (profiles/dram_traffic_conv_gemm_tc_shapes.md), summed over the layers; tensors that "
                        "stay in L2 between two layers of a real step, and lines still dirty in L2 when a launch ends, are not "
                        "captured this way",
        "launches_per_step": n_tc, "kernel_ms_per_step": tc_ms, "kernel_ms_per_step_events": tc_ms / scale if scale > 0 else None,
        "event_sum_ms": event_sum, "event_to_step_scale": scale,
        "algorithmic_bytes_per_step": tc_bytes,
        "tensor": {"achieved_tops": tc_ops / (tc_ms * 1e-3) / 1e12 if tc_ms > 0 else 0.0,
                   "probe_peak_tops": probe_tops, "nominal_peak_tops": INT8_NOMINAL_TOPS,
                   "frac_of_probe": (tc_ops / (tc_ms * 1e-3) / 1e12) / probe_tops if tc_ms > 0 and probe_tops > 0 else None},
        "two_layer_kernel": {"kernel": "f8_conv_pw_fused_tc_kernel", "launches_per_step": n_pairs, "ms_per_step": pair_ms,
                             "algorithmic_bytes_per_step": pair_bytes,
                             "gbs": pair_bytes / (pair_ms * 1e-3) / 1e9 if pair_ms > 0 else None,
                             "frac_of_hbm_peak": pair_bytes / (pair_ms * 1e-3) / 1e9 / peak_gbs if pair_ms > 0 else None,
                             "tops": pair_ops / (pair_ms * 1e-3) / 1e12 if pair_ms > 0 else None},
        "both_tensor_core_kernels": {"ms_per_step": tc_ms + pair_ms, "algorithmic_bytes_per_step": tc_bytes + pair_bytes,
                                     "gbs": (tc_bytes + pair_bytes) / ((tc_ms + pair_ms) * 1e-3) / 1e9 if tc_ms + pair_ms > 0 else None,
                                     "frac_of_hbm_peak": (tc_bytes + pair_bytes) / ((tc_ms + pair_ms) * 1e-3) / 1e9 / peak_gbs
                                     if tc_ms + pair_ms > 0 else None},
        "other_kernels": {"ms_per_step": other_ms, "gbs": other_bytes / (other_ms * 1e-3) / 1e9 if other_ms > 0 else None},
        "whole_step": {"tops": total_ops / (ms_per_step * 1e-3) / 1e12,
                       "gbs": (tc_bytes + pair_bytes + other_bytes) / (ms_per_step * 1e-3) / 1e9,
                       "layerwise_bound_ms": bound_ms, "frac_of_layerwise_bound": bound_ms / ms_per_step,
                       "sum_hbm_ms": hbm_ms, "sum_tensor_ms": tensor_ms},
    }
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "int8", "data": "synthetic",
            "config": {"workload": WORKLOAD, "net": NET, "global_batch": BATCH * world, "batch_per_gpu": BATCH,
                       "image": "224x224x3 int8 FL=6", "parallelism": f"replicas x{world}",
                       "micro_batched_runs": micro[0], "micro_batch": micro[1],
                       "l2": "no flush: one step moves %.1f GB of activations, far beyond the 126 MB L2" %
                             ((tc_bytes + other_bytes) / 1e9)},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(x_host.numel()),
                    "d2h_bytes_per_step": int(out_host.numel() * 4), "ms_per_step": e2e_ms / args.steps,
                    "call": "f8_net_forward_host (C ABI; depth 2: copies of neighbouring steps overlap the forward pass)",
                    "logits_match_device_run": e2e_ok},
            "gpu_launches": int(launches),
            "roofline": roofline}
    if incidents:
        line["incidents"] = incidents       # bounded waits that gave up (each costs 2 s); the affected measurement was repeated
    if world == 1:
        line["cpu_baseline"] = cpu_baseline(layers, BATCH, WORKLOAD)
        if not args.no_workloads:
            del net, ws, x_dev
            torch.cuda.empty_cache()
            line["workloads"] = run_workloads(api, torch, peak_gbs, probe_tops, max(10, min(args.steps, 50)))
    if args.layers:
        line["layers"] = per_layer
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", action="store_true", help="add per-layer times to the JSON line")
    ap.add_argument("--no-workloads", action="store_true", help="skip the other configurations (headline fields only)")
    ap.add_argument("--dist-selftest", action="store_true", help="run only the multi-rank plumbing, on CPU (gloo)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher: this process becomes the launcher of args.gpus local ranks
        raise SystemExit(spawn_local_ranks(args.gpus, sys.argv[1:]))
    if args.dist_selftest:
        dist_selftest(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)
    try:
        import torch.distributed as dist
        if dist.is_available() and dist.is_initialized():
            dist.destroy_process_group()
    except Exception:
        pass


if __name__ == "__main__":
    main()
