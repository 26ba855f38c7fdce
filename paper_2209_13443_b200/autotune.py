"""Fills the per-(layer, batch) kernel table of a model by measurement.

The paper's design-space exploration picks, offline, the configuration that maximises a throughput objective
summed over the batch sizes the device will see (Section III-D, Eq. 2) and stores the per-(layer, batch) choice in a
look-up table the hardware addresses at run time (Section III-C).  This script is the counterpart for the kernels
of this library: for every tensor-core layer it times every kernel variant (one-CTA tiles, CTA pairs with 256- or
128-wide tiles) for every candidate number of K ranges and every batch size on the GPU at hand, picks the number
of K ranges per layer that minimises sum_b w_b T(b) with every batch taking its fastest variant (the K ranges must not
depend on the batch: they fix the grouping of the sums), then the variant per (layer, batch), and writes the table as JSON:

  python -m paper_2209_13443_b200.autotune --workload resnet50 --max-batch 64 [--out FILE] [--raw FILE]

``EEModel`` applies a table written for (workload, max_batch) at creation (see ``binding.apply_table``).
"""
from __future__ import annotations

import argparse
import json
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
SPLITS = (1, 2, 3, 4, 6, 8)
VARIANTS = (0, 1, 2)


def table_path(name: str, max_batch: int) -> str:
    return os.path.join(HERE, "tables", f"{name}_b{max_batch}.json")


def layer_shapes(spec):
    from . import workloads as wl

    return wl.stage_shapes(spec)


def time_layer(m, s, i, x, res, out, B, ws, reps=20, rounds=3):
    """Device time (us) of one launch of a layer: `reps` back-to-back launches replayed as one CUDA graph (so that the
    host's launch cost does not bound the measurement), best of `rounds` replays."""
    st = torch.cuda.current_stream()
    m.layer_run(s, i, x, res, B, out, ws)           # tensor maps cached, lazy module loading done before the capture
    st.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        for _ in range(reps):
            m.layer_run(s, i, x, res, B, out, ws)
    best = float("inf")
    for _ in range(rounds + 1):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        b.synchronize()
        best = min(best, a.elapsed_time(b) * 1e3 / reps)
    return best


def measure(spec, batches, verbose=True):
    from . import binding as eb
    from . import workloads as wl

    m = eb.EEModel(spec, apply_tables=False)
    m.set_wait_limit(200_000_000)       # a wait that runs out should cost 0.1 s, not seconds, per launch of a sweep
    shapes = layer_shapes(spec)
    rows = []
    ws = m.workspace()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for s, st in enumerate(spec.stages):
            sh = shapes[s]
            for i, l in enumerate(st.layers):
                cfg = m.layer_config(s, i, 1)
                if cfg["tensor_core"] < 0:
                    continue
                src = l.input_from
                ishape = sh["in"] if (src == wl.FROM_STAGE_INPUT or (src == wl.FROM_PREV and i == 0)) else sh["layers"][i - 1 if src == wl.FROM_PREV else src]
                oshape = sh["layers"][i]
                default_splits = cfg["splits"]
                for sp in SPLITS:
                    try:
                        m.set_layer_splits(s, i, sp)
                    except eb.EEError:
                        continue
                    need = m.query(s)["workspace_bytes"]
                    if ws.numel() < need + 256:
                        ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
                    for B in batches:
                        x = torch.randn((B,) + tuple(ishape), device="cuda").to(torch.bfloat16)
                        res = torch.randn((B,) + tuple(oshape), device="cuda").to(torch.bfloat16) if l.residual_from != wl.NO_RESIDUAL else None
                        out = torch.empty((B,) + tuple(oshape), dtype=torch.bfloat16, device="cuda")
                        for v in VARIANTS:
                            if v > 0 and not (cfg["tensor_core"] >> (v - 1)) & 1:
                                continue
                            if v == 0 and sp > 4:
                                continue       # cluster split-K of the one-CTA kernel: up to four ranges
                            m.set_layer_variant(s, i, 1, spec.max_batch, v)
                            us = time_layer(m, s, i, x, res, out, B, ws)
                            m.check()          # a device-side fault stops the sweep here, not minutes later
                            rows.append({"stage": s, "layer": i, "splits": sp, "batch": B, "variant": v, "us": us,
                                         "default_splits": default_splits,
                                         "geom": [l.kh, l.cin, l.cout, l.stride, oshape[0], oshape[1]]})
                    m.check()
                    if verbose:
                        last = [r for r in rows if r["stage"] == s and r["layer"] == i and r["splits"] == sp]
                        print(f"stage {s} layer {i} {l.kh}x{l.kw} {l.cin}->{l.cout} splits {sp}: " +
                              " ".join(f"B{r['batch']}v{r['variant']}={r['us']:.1f}" for r in last), flush=True)
                m.set_layer_splits(s, i, default_splits)
                m.set_layer_variant(s, i, 1, spec.max_batch, 0)
    return rows


def choose(rows, max_batch, weights=None):
    """Per layer: the number of K ranges minimising sum_b w_b min_v T(b, splits, v); then the variant per batch
    (measured batches are extended to the batches between them: batch b takes the choice of the nearest measured
    batch at or above it)."""
    layers = {}
    for r in rows:
        layers.setdefault((r["stage"], r["layer"]), []).append(r)
    table = []
    for (s, i), rs in sorted(layers.items()):
        batches = sorted({r["batch"] for r in rs})
        best_sp, best_cost = None, float("inf")
        for sp in sorted({r["splits"] for r in rs}):
            cost = 0.0
            for b in batches:
                ts = [r["us"] for r in rs if r["splits"] == sp and r["batch"] == b]
                if not ts:
                    cost = float("inf")
                    break
                cost += (weights or {}).get(b, 1.0) * min(ts)
            if cost < best_cost:
                best_sp, best_cost = sp, cost
        per_b = {}
        for b in batches:
            cand = [(r["us"], r["variant"]) for r in rs if r["splits"] == best_sp and r["batch"] == b]
            per_b[b] = min(cand)[1]
        variants = []
        for b in range(1, max_batch + 1):
            nb = min([x for x in batches if x >= b] or [batches[-1]])
            variants.append(per_b[nb])
        table.append({"stage": s, "layer": i, "splits": best_sp, "variants": variants, "geom": rs[0]["geom"]})
    return table


def main():
    from . import workloads as wl

    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="resnet50")
    ap.add_argument("--max-batch", type=int, default=64)
    ap.add_argument("--batches", default="")
    ap.add_argument("--out", default=None)
    ap.add_argument("--raw", default=None)
    args = ap.parse_args()
    spec, _ = wl.benchmark_model(args.workload, args.max_batch)
    if args.batches:
        batches = [int(b) for b in args.batches.split(",")]
    else:
        batches = sorted({b for b in (1, 2, 3, 4, 6, 8, 12, 16, 24, 32, 48, 64, 96, 128) if b < args.max_batch} | {args.max_batch})
    rows = measure(spec, batches)
    if args.raw:
        with open(args.raw, "w") as f:
            json.dump(rows, f)
    table = {"workload": spec.name, "max_batch": args.max_batch, "input": [spec.in_h, spec.in_w, spec.in_c], "gpu": torch.cuda.get_device_name(0), "batches_measured": batches,
             "layers": choose(rows, args.max_batch)}
    out = args.out or table_path(spec.name, args.max_batch)
    os.makedirs(os.path.dirname(out), exist_ok=True)
    with open(out, "w") as f:
        json.dump(table, f, indent=1)
    print("wrote", out)


if __name__ == "__main__":
    main()
