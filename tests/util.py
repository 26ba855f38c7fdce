"""Helpers shared by the GPU parity tests: run the CUDA library through its C ABI and compare
with the CPU oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import ee_oracle as eo
from paper_2209_13443_b200 import binding as eb
from paper_2209_13443_b200 import workloads as wl

# Parity bars (max relative error of features and logits against the fp64 oracle):
#   fp32 path 1e-5, bf16 activations with fp32 accumulation 1e-2.
# "Relative" is taken element-wise against max(|oracle|, FLOOR * max|oracle|).  Post-ReLU maps contain
# exact zeros and values far below the tensor's scale, where a pure element-wise ratio is undefined, and
# the rounding error of a length-K fp32 dot product scales with sum|x_i w_i| (the tensor's scale), not with
# the element's own value: an element at 1e-3 of the scale legitimately carries ~K*2^-24/1e-3 relative
# error in ANY fp32 summation order.  FLOOR = 0.05 keeps the bar meaningful for every element that
# matters and still bounds the small ones in absolute terms (tol * 0.05 * scale).
TOL = {"f32": 1e-5, "bf16": 1e-2}
# Whole stages of a bf16 model (10-19 layers, each output rounded to bf16 on both sides) are held to two bf16 ulps in
# the max-norm, 2^-6: a legitimate last-bit difference early in the chain moves later pre-rounding values across
# rounding boundaries, so the largest elements of a 10^7-element map end up one to two ulps (2^-7 each at the bottom
# of a binade) apart in ANY correct implementation.  The 1e-2 bar itself is enforced layer by layer
# (test_every_layer_of_the_full_size_models), where both sides round the same pre-activation once.
STAGE_TOL = {"f32": 1e-5, "bf16": 2.0 ** -6}
FLOOR = 0.05
BAND = 1e-3   # samples whose oracle confidence is within BAND of the threshold may flip; they are listed and counted


def rel_err(a: np.ndarray, o: np.ndarray) -> float:
    a = np.asarray(a, dtype=np.float64)
    o = np.asarray(o, dtype=np.float64)
    if o.size == 0:
        return 0.0
    scale = float(np.max(np.abs(o)))
    if scale == 0.0:
        return float(np.max(np.abs(a)))
    return float(np.max(np.abs(a - o) / np.maximum(np.abs(o), FLOOR * scale)))


def norm_err(a, o) -> float:
    a = np.asarray(a, dtype=np.float64)
    o = np.asarray(o, dtype=np.float64)
    if o.size == 0:
        return 0.0
    return float(np.max(np.abs(a - o)) / max(float(np.max(np.abs(o))), 1e-30))


class GpuRunner:
    """One model on the GPU with the buffers a caller allocates once (sized for max_batch)."""

    def __init__(self, spec):
        self.spec = spec
        self.m = eb.EEModel(spec)
        self.bufs = [eb.StageBuffers(self.m, s) for s in range(self.m.n_stages)]
        self.ws = self.m.workspace()

    def stage(self, s, x_np, ids=None, shift=None, shift_cls=None):
        """Runs stage ``s`` on host features ``x_np``; returns host copies of every output."""
        B = x_np.shape[0]
        x = eb.to_device(self.spec.dtype, x_np) if B else None
        ids_d = None if ids is None else torch.as_tensor(np.asarray(ids, dtype=np.int32), device="cuda")
        sh = None if shift is None else torch.as_tensor(np.asarray(shift, dtype=np.float32), device="cuda")
        sc = None if shift_cls is None else torch.as_tensor(np.asarray(shift_cls, dtype=np.int32), device="cuda")
        out = self.bufs[s]
        out.n_surv_host.fill_(-7)
        self.m.stage_run(s, x, B, out, self.ws, ids_d, sh, sc)
        torch.cuda.synchronize()
        self.m.check()
        n = int(out.n_surv_host[0])
        assert n == int(out.n_surv_dev.cpu()[0])
        return {
            "n_surv": n,
            "features_out": out.features_out[:n].float().cpu().numpy(),
            "conf": out.conf[:B].cpu().numpy(),
            "pred": out.pred[:B].cpu().numpy(),
            "z": out.logits[:B].cpu().numpy(),
            "exit": out.exit_mask[:B].cpu().numpy(),
            "surv_idx": out.survivor_idx[:n].cpu().numpy(),
            "ids_out": None if ids is None else out.ids_out[:n].cpu().numpy(),
        }


def check_stage(spec, g: dict, o: dict, where="", tol=None, elementwise=False):
    """GPU stage result ``g`` against oracle result ``o`` (both from the same stage input).

    Features are held to ``tol`` in the max-norm relative to the tensor's scale.  With
    ``elementwise`` (single-layer cases, where both sides round the same pre-activation once) the
    floored element-wise ratio is held to ``tol`` as well.  Across a chain of bf16 layers the
    element-wise ratio is not a property of an implementation: one legitimate last-bit difference
    perturbs every downstream pre-rounding value, and each perturbed value that straddles a bf16
    rounding boundary moves by a full ulp (2^-8 relative), so individual elements drift by a few
    percent in any summation order while the max-norm error stays near one ulp."""
    if tol is None:
        tol = TOL[spec.dtype] if elementwise else STAGE_TOL[spec.dtype]
    ferr = rel_err if elementwise else norm_err
    B = len(o["conf"])
    st_thr = o.get("threshold")
    e_z = ferr(g["z"], o["z"])
    assert e_z <= TOL[spec.dtype], f"{where}: logits rel err {e_z:.3e} > {TOL[spec.dtype]}"
    # softmax top-1 is 1/2-Lipschitz in the max-norm of the logits (d conf = conf (1 - conf) d(z_top - z_k)):
    # the confidence may move by at most half the largest logit difference, plus fp32 rounding of the exp-sum
    dz = np.max(np.abs(g["z"] - o["z"]), axis=1) if B else np.zeros(0)
    assert np.all(np.abs(g["conf"] - o["conf"]) <= 0.5 * dz + 2e-6), f"{where}: conf"
    # argmax may differ only where the two top logits are within tolerance of each other
    for b in np.nonzero(g["pred"] != o["pred"])[0]:
        zz = o["z"][b]
        assert abs(zz[g["pred"][b]] - zz[o["pred"][b]]) <= tol * max(1.0, np.max(np.abs(zz))), f"{where}: pred[{b}]"
    band = np.zeros(B, dtype=bool) if st_thr is None else (np.abs(o["conf"] - st_thr) < BAND)
    outside = ~band
    assert np.array_equal(g["exit"][outside], o["exit"][outside]), f"{where}: exit mask outside the near-threshold band"
    # the GPU's own compaction must be the stable compaction of its own mask
    want_idx = np.nonzero(g["exit"] == 0)[0]
    assert g["n_surv"] == len(want_idx) == B - int(g["exit"].sum()), f"{where}: n_surv"
    assert np.array_equal(g["surv_idx"], want_idx), f"{where}: surv_idx"
    flips = int(np.sum(g["exit"] != o["exit"]))
    if flips == 0:
        assert g["n_surv"] == o["n_surv"] and np.array_equal(g["surv_idx"], o["surv_idx"]), f"{where}: compaction"
        if o.get("ids_out") is not None:
            assert np.array_equal(g["ids_out"], o["ids_out"]), f"{where}: ids"
        e_f = ferr(g["features_out"], o["features_out"])
        assert e_f <= tol, f"{where}: features rel err {e_f:.3e} > {tol}"
    else:
        so = o["stage_out"][g["surv_idx"]]
        e_f = ferr(g["features_out"], so)
        assert e_f <= tol, f"{where}: features rel err {e_f:.3e} > {tol}"
    return {"z_err": e_z, "feat_err": e_f, "band": int(band.sum()), "flips": flips}


def oracle_stage(spec, s, x_np, ids=None, shift=None, shift_cls=None):
    o = eo.run_stage(spec, s, x_np, None if ids is None else np.asarray(ids, dtype=np.int32), shift, shift_cls)
    o["threshold"] = None if spec.stages[s].always_exit else spec.stages[s].threshold
    return o


def single_layer_model(dtype, H, W, cin, cout, k, stride, pad, act, residual, seed, n_classes=7, max_batch=4, op=wl.OP_CONV):
    """One backbone layer (optionally preceded by a 1x1 conv that supplies the residual operand)
    followed by an exit head nobody passes (threshold 2), so the whole layer output is returned."""
    rng = wl._rng(seed, 900)
    bf16 = dtype == "bf16"
    layers = []
    if residual:
        ho, wo = (H + 2 * pad - k) // stride + 1, (W + 2 * pad - k) // stride + 1
        # residual operand: a strided 1x1 conv of the stage input with the same output shape
        assert (H - 1) // stride + 1 == ho and (W - 1) // stride + 1 == wo
        layers.append(wl._conv(rng, wl.OP_CONV, cin, cout, 1, stride, 0, wl.ACT_NONE, bf16=bf16, input_from=wl.FROM_STAGE_INPUT))
        layers.append(wl._conv(rng, op, cin, cout, k, stride, pad, act, bf16=bf16, input_from=wl.FROM_STAGE_INPUT, residual_from=0))
    else:
        layers.append(wl._conv(rng, op, cin, cout, k, stride, pad, act, bf16=bf16))
    fw, fb = wl._head(rng, cout, n_classes, 1.0, bf16)
    st = wl.Stage(layers, n_classes, fw, fb, 2.0, False)
    return wl.Model("single", dtype, H, W, cin, [st], max_batch)
