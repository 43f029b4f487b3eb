"""Single-layer micro-benchmark: times one fixed-point conv layer through the C ABI.

    python -m paper_2202_05239_b200.layer_bench --sweep            # the six CNN layer shapes at batch 32
    python -m paper_2202_05239_b200.layer_bench --h 56 --w 56 --c 64 --c-out 256 --k 1 --batch 32 --res
    python -m paper_2202_05239_b200.layer_bench --net mobilenetv2 --batch 64     # per-layer times of a whole net

Each layer is run over several copies of its tensors, rotated so that consecutive launches do not find
their operands in L2 (the copies together exceed twice the L2 size).  Prints one JSON line per layer:
device time per launch (CUDA events), int8 TOPS and algorithmic GB/s.
"""
from __future__ import annotations

import argparse
import json
import math

import numpy as np
import torch

from . import api, synth


def bench_layer(layer: synth.Layer, batch: int, with_res: bool, iters: int, warmup: int, cold: bool = True):
    rng = np.random.default_rng(0)
    x_bytes = batch * layer.h * layer.w * layer.c
    y_elems = batch * layer.ho * layer.wo * layer.c_out
    per_set = x_bytes + y_elems * (2 if with_res else 1)
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    sets = max(2, math.ceil(2.2 * l2 / per_set)) if cold else 1
    sets = min(sets, 64)
    w = api.to_device(layer.weight)
    b = api.to_device(layer.bias)
    xs, rs, ys = [], [], []
    for _ in range(sets):
        if layer.x_dtype == synth.S8:
            x = rng.integers(-128, 128, size=(batch, layer.h, layer.w, layer.c), dtype=np.int64).astype(np.int8)
        else:
            x = rng.integers(0, 256, size=(batch, layer.h, layer.w, layer.c), dtype=np.int64).astype(np.uint8)
        xs.append(api.to_device(x))
        rs.append(torch.randint(0, 255, (batch, layer.ho, layer.wo, layer.c_out), dtype=torch.uint8, device="cuda")
                  if with_res else None)
        ys.append(torch.empty((batch, layer.ho, layer.wo, layer.c_out), dtype=api.torch_dtype(layer.y_dtype),
                              device="cuda"))
    desc = api.conv_desc(layer, batch)
    fn = api.f8_dwconv_fixed if layer.kind == synth.DWCONV else api.f8_conv2d_fixed
    for i in range(warmup):
        fn(desc, xs[i % sets], w, b, rs[i % sets], ys[i % sets])
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        fn(desc, xs[i % sets], w, b, rs[i % sets], ys[i % sets])
    e1.record()
    torch.cuda.synchronize()
    api.f8_device_status()
    ms = e0.elapsed_time(e1) / iters
    macs = batch * layer.macs_per_image
    ysz = 4 if layer.y_dtype == synth.S32 else 1
    byts = x_bytes + y_elems * ysz + (y_elems if with_res else 0) + layer.param_bytes()
    return {"layer": layer.name, "batch": batch, "ms": ms, "tops": 2 * macs / (ms * 1e-3) / 1e12,
            "gbs": byts / (ms * 1e-3) / 1e9, "macs": macs, "bytes": byts, "buffer_sets": sets}


def custom_layer(args) -> synth.Layer:
    rng = np.random.default_rng(1)
    depthwise = args.depthwise
    fan_in = args.k * args.k * (1 if depthwise else args.c)
    shape = (args.c, args.k, args.k) if depthwise else (args.c_out, args.k, args.k, args.c)
    wgt, flw = synth.draw_weight(rng, shape, math.sqrt(2.0 / fan_in))
    bias = synth.draw_bias(rng, args.c_out, 5 + flw)
    return synth.Layer(synth.DWCONV if depthwise else synth.CONV, f"c{args.k}x{args.k}_{args.h}_{args.c}_{args.c_out}", 0,
                       1 if args.res else -1, args.h, args.w or args.h, args.c, args.c_out, args.k, args.k, args.stride,
                       args.k // 2, synth.U8, synth.U8, synth.U8, 5, flw, 5, 5, wgt, bias)


def bench_net(name: str, batch: int, iters: int, warmup: int):
    """Per-layer device times of a whole synthetic network (CUDA events recorded by f8_net_forward)."""
    layers = synth.make_net(name, 0)
    net = api.Net(layers, batch)
    x = api.to_device(synth.draw_image(batch, 1))
    for _ in range(warmup):
        net.forward(x)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        net.forward(x)
    e1.record()
    torch.cuda.synchronize()
    total_ms = e0.elapsed_time(e1) / iters
    net.set_profiling(True)
    acc = np.zeros(len(layers))
    for _ in range(iters):
        net.forward(x)
        ms, tc = net.layer_ms()
        acc += np.array(ms)
    api.f8_device_status()
    acc /= iters
    for l, ms, on_tc in zip(layers, acc, tc):
        byts = batch * l.bytes_per_image() + l.param_bytes()
        print(json.dumps({"layer": l.name, "kind": synth.KIND_NAMES[l.kind], "shape": [l.h, l.w, l.c, l.c_out, l.kh, l.stride],
                          "tensor_cores": bool(on_tc), "ms": round(float(ms), 5),
                          "gbs": round(byts / (ms * 1e-3) / 1e9, 1) if ms > 0 else None,
                          "tops": round(2 * batch * l.macs_per_image / (ms * 1e-3) / 1e12, 1) if ms > 0 else None}))
    print(json.dumps({"net": name, "batch": batch, "ms_per_forward": total_ms, "images_per_s": batch / (total_ms * 1e-3),
                      "launches": net.last_launch_count}), flush=True)


def shape_key(l: synth.Layer) -> str:
    return f"{l.h}x{l.w}x{l.c}->{l.c_out} k{l.kh} s{l.stride} res{1 if l.res >= 0 else 0}"


def run_distinct_shapes(name: str, batch: int):
    """Every distinct dense-layer shape of a synthetic network once, as single-layer calls on fresh buffers, in the order
    printed: the launch list of a profiler run of this command maps one to one onto the printed shapes (layers that do
    not take the tensor-core kernel are listed with "tensor_cores": false and launch another kernel)."""
    rng = np.random.default_rng(0)
    seen = set()
    for l in synth.make_net(name, 0):
        if l.kind != synth.CONV or shape_key(l) in seen:
            continue
        seen.add(shape_key(l))
        if l.x_dtype == synth.S8:
            x = rng.integers(-128, 128, size=(batch, l.h, l.w, l.c), dtype=np.int64).astype(np.int8)
        else:
            x = rng.integers(0, 256, size=(batch, l.h, l.w, l.c), dtype=np.int64).astype(np.uint8)
        res = None
        if l.res >= 0:
            res = torch.randint(0, 255, (batch, l.ho, l.wo, l.c_out), dtype=torch.uint8, device="cuda")
            if l.r_dtype == synth.S8:
                res = res.view(torch.int8)
        before = api.f8_tc_launch_count()
        api.run_layer(l, api.to_device(x), res)
        torch.cuda.synchronize()
        print(json.dumps({"shape": shape_key(l), "layer": l.name, "batch": batch,
                          "tensor_cores": api.f8_tc_launch_count() - before == 1,
                          "algorithmic_bytes": batch * l.bytes_per_image() + l.param_bytes()}), flush=True)
    api.f8_device_status()


def bench_fold(c_out: int, k: int, iters: int, warmup: int):
    """Device time of the weight compile step (f8_fold_quantize_fixed) on one [c_out, k] fp32 tensor.  Algorithmic
    bytes: 4 read + 1 written per weight (the fp32 tensor has to be read twice -- statistics, then quantisation --
    unless it stays in L2, so DRAM traffic can be up to 9 bytes per weight)."""
    rng = np.random.default_rng(2)
    d = api.FoldDesc(c_out, k, 5, 0, 24, 0.11, 0.07)
    w = torch.from_numpy(rng.normal(0, 0.05, (c_out, k)).astype(np.float32)).cuda()
    vec = [torch.from_numpy(rng.uniform(0.5, 1.5, c_out).astype(np.float32)).cuda() for _ in range(4)]
    w_q = torch.empty((c_out, k), dtype=torch.int8, device="cuda")
    b_q = torch.empty(c_out, dtype=torch.int32, device="cuda")
    fl = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(api.f8_fold_workspace_bytes(d), dtype=torch.uint8, device="cuda")
    for _ in range(warmup):
        api.f8_fold_quantize_fixed(d, w, *vec, w_q, b_q, fl, ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        api.f8_fold_quantize_fixed(d, w, *vec, w_q, b_q, fl, ws)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    n = c_out * k
    print(json.dumps({"op": "fold_quantize", "c_out": c_out, "k": k, "ms": ms, "fl_w": int(fl.item()),
                      "algorithmic_gbs": 5.0 * n / (ms * 1e-3) / 1e9, "weights_per_s": n / (ms * 1e-3)}), flush=True)


def bench_requant(n: int, iters: int, warmup: int):
    """Device time of f8_requantize_dual_fixed on n int32 values (4 bytes read, 2 written per element)."""
    acc = torch.randint(-(1 << 18), 1 << 18, (n,), dtype=torch.int32, device="cuda")
    y1 = torch.empty(n, dtype=torch.uint8, device="cuda")
    y2 = torch.empty(n, dtype=torch.int8, device="cuda")
    for _ in range(warmup):
        api.f8_requantize_dual_fixed(acc, 12, y1, synth.U8, 4, y2, synth.S8, 5)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        api.f8_requantize_dual_fixed(acc, 12, y1, synth.U8, 4, y2, synth.S8, 5)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    print(json.dumps({"op": "requantize_dual", "n": n, "ms": ms, "algorithmic_gbs": 6.0 * n / (ms * 1e-3) / 1e9}), flush=True)


def bench_fused(h: int, batch: int, with_res: bool, iters: int, warmup: int):
    """Device time of the two-layer kernel (f8_conv_pointwise_fixed): 3x3 64 -> 64 and 1x1 64 -> 256 (+ shortcut) at h x h,
    over rotating buffer sets larger than twice the L2 cache.  Algorithmic bytes: the first layer's input, the shortcut,
    the second layer's output, both layers' parameters (the tensor between the layers does not travel)."""
    rng = np.random.default_rng(3)
    w1, fl1 = synth.draw_weight(rng, (64, 3, 3, 64), math.sqrt(2.0 / 576))
    w2, fl2 = synth.draw_weight(rng, (256, 1, 1, 64), math.sqrt(2.0 / 64))
    first = synth.Layer(synth.CONV, "conv3x3", 0, -1, h, h, 64, 64, 3, 3, 1, 1, synth.U8, synth.U8, synth.U8, 5, fl1, 5, 5, w1,
                        synth.draw_bias(rng, 64, 5 + fl1))
    second = synth.Layer(synth.CONV, "conv1x1", 1, 0 if with_res else -1, h, h, 64, 256, 1, 1, 1, 0, synth.U8, synth.U8, synth.U8, 5, fl2,
                         5, 5, w2, synth.draw_bias(rng, 256, 5 + fl2))
    x_bytes, y_bytes = batch * h * h * 64, batch * h * h * 256
    per_set = x_bytes + y_bytes * (2 if with_res else 1)
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    sets = min(16, max(2, math.ceil(2.2 * l2 / per_set)))
    xs = [torch.randint(0, 255, (batch, h, h, 64), dtype=torch.uint8, device="cuda") for _ in range(sets)]
    rs = [torch.randint(0, 255, (batch, h, h, 256), dtype=torch.uint8, device="cuda") if with_res else None for _ in range(sets)]
    ys = [torch.empty((batch, h, h, 256), dtype=torch.uint8, device="cuda") for _ in range(sets)]
    p1 = (api.to_device(first.weight), api.to_device(first.bias))
    p2 = (api.to_device(second.weight), api.to_device(second.bias))
    d1, d2 = api.conv_desc(first, batch), api.conv_desc(second, batch)

    def run(i):
        api.f8_conv_pointwise_fixed(d1, d2, xs[i % sets], p1[0], p1[1], p2[0], p2[1], rs[i % sets], None, ys[i % sets])

    for i in range(warmup):
        run(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        run(i)
    e1.record()
    torch.cuda.synchronize()
    api.f8_device_status()
    ms = e0.elapsed_time(e1) / iters
    byts = per_set + first.param_bytes() + second.param_bytes()
    macs = batch * (first.macs_per_image + second.macs_per_image)
    print(json.dumps({"op": "conv3x3_64_64 + conv1x1_64_256" + (" + shortcut" if with_res else ""), "h": h, "batch": batch, "ms": ms,
                      "gbs": byts / (ms * 1e-3) / 1e9, "tops": 2 * macs / (ms * 1e-3) / 1e12, "bytes": byts, "buffer_sets": sets}),
          flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--requant", type=int, default=0, help="time the dual requantisation on this many int32 values")
    ap.add_argument("--fold", action="store_true", help="time the weight compile step on a [c-out, k * k * c] tensor")
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--fused", action="store_true", help="time the two-layer kernel: 3x3 64 -> 64 + 1x1 64 -> 256 at --h, --batch, --res")
    ap.add_argument("--net", default="", help="time every layer of a synthetic network: resnet18, resnet50, mobilenetv2")
    ap.add_argument("--distinct-shapes", default="", help="run every distinct dense-layer shape of this network once (for a profiler)")
    ap.add_argument("--h", type=int, default=56)
    ap.add_argument("--w", type=int, default=0)
    ap.add_argument("--c", type=int, default=64)
    ap.add_argument("--c-out", type=int, default=64)
    ap.add_argument("--k", type=int, default=3)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--batch", type=int, default=32)
    ap.add_argument("--res", action="store_true")
    ap.add_argument("--depthwise", action="store_true")
    ap.add_argument("--iters", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--warm-l2", action="store_true", help="reuse one buffer set (operands stay in L2)")
    args = ap.parse_args()
    if args.requant:
        bench_requant(args.requant, args.iters, args.warmup)
        return
    if args.fold:
        bench_fold(args.c_out, args.k * args.k * args.c, args.iters, args.warmup)
        return
    if args.fused:
        bench_fused(args.h, args.batch, args.res, args.iters, args.warmup)
        return
    if args.distinct_shapes:
        run_distinct_shapes(args.distinct_shapes, args.batch)
    elif args.net:
        bench_net(args.net, args.batch, args.iters, args.warmup)
    elif args.sweep:
        for i in range(len(synth.SWEEP_SHAPES)):
            layer, _ = synth.sweep_case(i, batch=1)
            print(json.dumps(bench_layer(layer, args.batch, False, args.iters, args.warmup, not args.warm_l2)), flush=True)
    else:
        if args.depthwise:
            args.c_out = args.c
        print(json.dumps(bench_layer(custom_layer(args), args.batch, args.res, args.iters, args.warmup, not args.warm_l2)),
              flush=True)


if __name__ == "__main__":
    main()
