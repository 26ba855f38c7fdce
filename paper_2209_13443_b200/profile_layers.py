"""Runs single layers of a benchmark model alone, at a chosen batch, for profilers and quick timings.

  python -m paper_2209_13443_b200.profile_layers --workload resnet50 --max-batch 64 --layers 2:5:30,3:4:27 [--variant V] [--reps N]

``--layers`` is a comma-separated list of stage:layer:batch.  Every layer runs through ee_layer_run in the kernel and
launch configuration ee_stage_run would use for it (the model's per-(layer, batch) table applies unless ``--variant``
forces one), on random inputs of the right shape.  Nothing beyond the chosen layers' tensors is allocated (a few
hundred MB at most), so that a profiler capture of a handful of launches ends in seconds.  Prints one line per
layer with the CUDA-event time of a launch (the launches of a layer run back to back).
"""
from __future__ import annotations

import argparse

import torch

from . import binding as eb
from . import workloads as wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="resnet50")
    ap.add_argument("--max-batch", type=int, default=64)
    ap.add_argument("--layers", required=True)
    ap.add_argument("--variant", type=int, default=None)
    ap.add_argument("--reps", type=int, default=3)
    args = ap.parse_args()
    spec, _ = wl.benchmark_model(args.workload, args.max_batch)
    m = eb.EEModel(spec)
    shapes = wl.stage_shapes(spec)
    ws = m.workspace()
    for item in args.layers.split(","):
        s, i, B = (int(v) for v in item.split(":"))
        l = spec.stages[s].layers[i]
        sh = shapes[s]
        src = l.input_from
        ishape = sh["in"] if (src == wl.FROM_STAGE_INPUT or (src == wl.FROM_PREV and i == 0)) else sh["layers"][i - 1 if src == wl.FROM_PREV else src]
        oshape = sh["layers"][i]
        if args.variant is not None:
            m.set_layer_variant(s, i, 1, spec.max_batch, args.variant)
        x = torch.randn((B,) + tuple(ishape), device="cuda").to(torch.bfloat16)
        res = torch.randn((B,) + tuple(oshape), device="cuda").to(torch.bfloat16) if l.residual_from != wl.NO_RESIDUAL else None
        out = torch.empty((B,) + tuple(oshape), dtype=torch.bfloat16, device="cuda")
        m.layer_run(s, i, x, res, B, out, ws)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.reps):
            m.layer_run(s, i, x, res, B, out, ws)
        b.record()
        b.synchronize()
        m.check()
        cfg = m.layer_config(s, i, B)
        flops = 2.0 * B * oshape[0] * oshape[1] * l.cout * l.kh * l.kw * l.cin
        us = a.elapsed_time(b) * 1e3 / args.reps
        print(f"stage {s} layer {i} {l.kh}x{l.kw} {l.cin}->{l.cout} s{l.stride} B={B} M={B * oshape[0] * oshape[1]} variant {cfg['variant']} "
              f"splits {cfg['splits']}: {us:.1f} us per launch (host-paced), {flops / 1e9:.2f} GFLOP")


if __name__ == "__main__":
    main()
