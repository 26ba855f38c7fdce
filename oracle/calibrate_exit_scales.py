"""Chooses the FC scale factor of every early exit so that a target fraction of the samples that
REACH the exit leave there, and stores the factors in the package's ``exit_calibration.json``.

Runs the CPU oracle only (never the CUDA library): the factors are workload parameters that both
sides then read.  The paper's own exit rates come from ImageNet-trained heads (Section IV,
Benchmarks) and cannot be reproduced offline, so the targets are the benchmark configuration's
(30 % / 25 % / 20 % for the ResNet-50-shaped model, 25 % for the MobileNetV2-shaped one) and the
result has no pin from the paper: parity unpinned beyond "measured rate within a few points of
the target on the calibration set".

usage: python -m oracle.calibrate_exit_scales [resnet50_ee] [mobilenetv2_ee] [--n 256]
"""
from __future__ import annotations

import json
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import ee_oracle as eo                      # noqa: E402
from paper_2209_13443_b200 import workloads as wl       # noqa: E402  (data generators only)

OUT = os.path.join(ROOT, "paper_2209_13443_b200", "exit_calibration.json")
TARGETS = {"resnet50_ee": (0.30, 0.25, 0.20), "mobilenetv2_ee": (0.25, 0.25, 0.25)}
STREAM0 = {"resnet50_ee": 200, "mobilenetv2_ee": 300}   # head random streams used by the generators
CAL_SEED = 1000   # calibration images are disjoint from every benchmark / test seed


def _rate(gap32, name, spec, e, alpha, thr):
    c = gap32.shape[-1]
    w, b = wl.head_weights(spec.meta["seed"], STREAM0[name] + e, c, spec.stages[e].n_classes, alpha, spec.dtype == "bf16")
    r = eo.exit_head(gap32, w, b, thr)
    return float(r["exit"].mean()), r


def calibrate(name: str, n: int):
    make = {"resnet50_ee": wl.resnet50_ee, "mobilenetv2_ee": wl.mobilenetv2_ee}[name]
    spec = make(alphas=[1.0, 1.0, 1.0, 1.0])
    x = wl.make_input(spec, n, seed=CAL_SEED)
    alphas, rates, bands = [], [], []
    for e, target in enumerate(TARGETS[name]):
        t0 = time.time()
        feats = np.concatenate([eo.run_layers(spec, e, x[i:i + 16]) for i in range(0, len(x), 16)])
        st = spec.stages[e]
        # the pooled vector of an [n][1][1][C] map is the map itself: pool once, bisect on the cheap part
        gap = eo.exit_head(feats, st.fc_weight, st.fc_bias, 2.0)["gap"].astype(np.float32)[:, None, None, :]
        lo, hi = 0.05, 200.0
        for _ in range(40):                              # the exit rate grows with the scale: bisect
            mid = float(np.sqrt(lo * hi))
            r, _ = _rate(gap, name, spec, e, mid, st.threshold)
            lo, hi = (mid, hi) if r < target else (lo, mid)
        alpha = float(np.sqrt(lo * hi))
        r, res = _rate(gap, name, spec, e, alpha, st.threshold)
        band = int(np.sum(np.abs(res["conf"] - st.threshold) < 1e-3))
        alphas.append(alpha); rates.append(r); bands.append(band)
        print(f"{name} exit {e}: reached {len(x)}, alpha {alpha:.4f}, rate {r:.3f} (target {target}), "
              f"within 1e-3 of the threshold: {band}, conf p10/p50/p90 "
              f"{np.percentile(res['conf'], 10):.3f}/{np.percentile(res['conf'], 50):.3f}/{np.percentile(res['conf'], 90):.3f}, "
              f"{time.time() - t0:.0f}s", flush=True)
        x = feats[res["exit"] == 0]
    alphas.append(alphas[-1])                            # the final head is always taken; reuse the last scale
    return {"alphas": alphas, "calibration_rates": rates, "near_threshold": bands, "n": n, "seed": CAL_SEED,
            "targets": list(TARGETS[name])}


def main(argv):
    n = int(argv[argv.index("--n") + 1]) if "--n" in argv else 256
    names = [a for a in argv if a in TARGETS] or list(TARGETS)
    data = json.load(open(OUT)) if os.path.exists(OUT) else {}
    for name in names:
        data[name] = calibrate(name, n)
        with open(OUT, "w") as f:
            json.dump(data, f, indent=1)
    print("wrote", OUT)


if __name__ == "__main__":
    main(sys.argv[1:])
