"""ctypes front end of the CPU oracle (``eo.c``) plus the stage/sample drivers built on it.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this module; it is used
by ``tests/``, by the smoke check and by the CPU-baseline legs of ``bench.py``.  It imports
nothing from the CUDA package: model descriptions are read by attribute (duck typing) from
whatever object the caller passes (``layers``, ``fc_weight``, ``threshold`` ...).

Driver functions and the passages they follow:
  run_stage            one subnet up to its exit, then the exit head, then the write-back of
                       the B_rem = B_act - B_exit remaining samples (Section III overview,
                       steps 2-4; Section III-B Preemption Mechanism)
  refill               merge of the halted batch with newly issued samples
                       (Section III-B; Algorithm 1: B_incr, B_merged)
  run_sample_serial    a single sample run alone until its first exit: the reference every
                       batched or refilled schedule has to reproduce per sample id, because
                       samples finish out of order and are re-associated by id (Section III-B,
                       Overhead)
  serve_trace          Algorithm 1 on a virtual clock, with the SLO-aware preemption criterion (Eq. 3-4;
                       T_SLO = infinity by default)
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from collections import deque

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libeeoracle.so")
_SRC = os.path.join(_HERE, "eo.c")


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"])
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        fp, ip, up, dp = C.POINTER(C.c_float), C.POINTER(C.c_int32), C.POINTER(C.c_uint8), C.POINTER(C.c_double)
        L.eo_round_bf16.restype = C.c_double
        L.eo_round_bf16.argtypes = [C.c_double]
        L.eo_conv2d.argtypes = [fp, C.c_int, C.c_int, C.c_int, C.c_int, fp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                C.c_int, fp, fp, fp, C.c_int, C.c_int, fp]
        L.eo_conv2d_hw.argtypes = [fp, C.c_int, C.c_int, C.c_int, C.c_int, fp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                   C.c_int, fp, fp, fp, C.c_int, C.c_int, fp]
        L.eo_maxpool.argtypes = [fp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, fp]
        L.eo_exit_head.argtypes = [fp, C.c_int, C.c_int, C.c_int, fp, fp, C.c_int, fp, ip, C.c_float, C.c_int,
                                   dp, dp, dp, ip, up]
        L.eo_compact.argtypes = [up, C.c_int, fp, C.c_size_t, ip, ip, fp, ip]
        L.eo_refill.argtypes = [fp, ip, C.c_int, C.c_size_t, fp, ip, C.c_int, C.c_int]
        _lib = L
    return _lib


def n_threads() -> int:
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v else (os.cpu_count() or 1)


def _f(a):
    return None if a is None else a.ctypes.data_as(C.POINTER(C.c_float))


def _i(a):
    return None if a is None else a.ctypes.data_as(C.POINTER(C.c_int32))


def _c32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def round_bf16(v: float) -> float:
    return lib().eo_round_bf16(float(v))


OP_CONV, OP_DWCONV, OP_MAXPOOL = 0, 1, 2


def conv2d(x, w, stride=1, pad=0, groups=1, scale=None, bias=None, residual=None, act=0, bf16=False, pad_w=None):
    """``pad`` pads the rows and, unless ``pad_w`` is given, the columns too."""
    x = _c32(x); w = _c32(w); scale = _c32(scale); bias = _c32(bias); residual = _c32(residual)
    B, H, W, Cin = x.shape
    Cout, kh, kw, cpg = w.shape
    assert cpg * groups == Cin
    pad_w = pad if pad_w is None or pad_w < 0 else pad_w
    Ho, Wo = (H + 2 * pad - kh) // stride + 1, (W + 2 * pad_w - kw) // stride + 1
    y = np.empty((B, Ho, Wo, Cout), dtype=np.float32)
    if B == 0:
        return y
    rc = lib().eo_conv2d_hw(_f(x), B, H, W, Cin, _f(w), Cout, kh, kw, stride, pad, pad_w, groups, _f(scale), _f(bias),
                            _f(residual), act, 1 if bf16 else 0, _f(y))
    assert rc == 0
    return y


def maxpool(x, k=3, stride=2, pad=1):
    x = _c32(x)
    B, H, W, Cc = x.shape
    Ho, Wo = (H + 2 * pad - k) // stride + 1, (W + 2 * pad - k) // stride + 1
    y = np.empty((B, Ho, Wo, Cc), dtype=np.float32)
    if B:
        assert lib().eo_maxpool(_f(x), B, H, W, Cc, k, stride, pad, _f(y)) == 0
    return y


def exit_head(x, wfc, bfc, threshold, always_exit=False, shift=None, shift_cls=None):
    """Returns dict(gap f64 [B][C], z f64 [B][K], conf f64 [B], pred i32 [B], exit u8 [B])."""
    x = _c32(x); wfc = _c32(wfc); bfc = _c32(bfc); shift = _c32(shift)
    shift_cls = None if shift_cls is None else np.ascontiguousarray(shift_cls, dtype=np.int32)
    B = x.shape[0]
    Cc = x.shape[-1]
    HW = int(np.prod(x.shape[1:-1]))
    K = wfc.shape[0]
    gap = np.zeros((B, Cc)); z = np.zeros((B, K)); conf = np.zeros(B)
    pred = np.zeros(B, dtype=np.int32); ex = np.zeros(B, dtype=np.uint8)
    if B:
        dp = C.POINTER(C.c_double)
        lib().eo_exit_head(_f(x), B, HW, Cc, _f(wfc), _f(bfc), K, _f(shift), _i(shift_cls), C.c_float(threshold),
                           int(bool(always_exit)), gap.ctypes.data_as(dp), z.ctypes.data_as(dp), conf.ctypes.data_as(dp),
                           _i(pred), ex.ctypes.data_as(C.POINTER(C.c_uint8)))
    return {"gap": gap, "z": z, "conf": conf, "pred": pred, "exit": ex}


def compact(exit_mask, feat, ids=None):
    """Returns (surv_idx i32 [n], feat_out [n][...], ids_out i32 [n] or None)."""
    exit_mask = np.ascontiguousarray(exit_mask, dtype=np.uint8)
    feat = _c32(feat)
    B = exit_mask.shape[0]
    eps = int(np.prod(feat.shape[1:]))
    idx = np.zeros(B, dtype=np.int32)
    out = np.zeros_like(feat)
    ids_c = None if ids is None else np.ascontiguousarray(ids, dtype=np.int32)
    ids_out = None if ids is None else np.zeros(B, dtype=np.int32)
    n = lib().eo_compact(exit_mask.ctypes.data_as(C.POINTER(C.c_uint8)), B, _f(feat), eps, _i(ids_c), _i(idx), _f(out), _i(ids_out))
    return idx[:n].copy(), out[:n].copy(), (None if ids is None else ids_out[:n].copy())


def refill(surv_feat, surv_ids, arr_feat, arr_ids, max_batch):
    """survivors ++ first n_acc arrivals.  Returns (feat [n_merged][...], ids, n_acc)."""
    surv_feat = _c32(surv_feat); arr_feat = _c32(arr_feat)
    n_surv, n_arr = surv_feat.shape[0], arr_feat.shape[0]
    eps = int(np.prod(arr_feat.shape[1:])) if n_arr else int(np.prod(surv_feat.shape[1:]))
    buf = np.zeros((max_batch,) + tuple(surv_feat.shape[1:] if n_surv else arr_feat.shape[1:]), dtype=np.float32)
    ids = np.zeros(max_batch, dtype=np.int32)
    buf[:n_surv] = surv_feat
    ids[:n_surv] = surv_ids
    arr_ids = np.ascontiguousarray(arr_ids, dtype=np.int32)
    n_acc = lib().eo_refill(_f(buf), _i(ids), n_surv, eps, _f(arr_feat), _i(arr_ids), n_arr, max_batch)
    assert n_acc >= 0
    return buf[:n_surv + n_acc].copy(), ids[:n_surv + n_acc].copy(), n_acc


# ----------------------------------------------------------------------------- drivers

def run_layers(model, stage: int, x, keep_all: bool = False):
    """Output of the stage's backbone layers for input ``x`` ([B][H][W][C])."""
    st = model.stages[stage]
    bf16 = model.dtype == "bf16"
    outs = []
    x = _c32(x)
    for i, l in enumerate(st.layers):
        if l.input_from == -2 or (l.input_from == -1 and i == 0):
            src = x
        elif l.input_from == -1:
            src = outs[i - 1]
        else:
            src = outs[l.input_from]
        if l.op == OP_MAXPOOL:
            outs.append(maxpool(src, l.kh, l.stride, l.pad))
            continue
        res = None
        if l.residual_from == -2:
            res = x
        elif l.residual_from >= 0:
            res = outs[l.residual_from]
        groups = l.cin if l.op == OP_DWCONV else 1
        outs.append(conv2d(src, l.weight, l.stride, l.pad, groups, l.scale, l.bias, res, l.act, bf16, getattr(l, "pad_w", None)))
    return outs if keep_all else outs[st.out_layer]


def run_stage(model, stage: int, x, ids=None, shift=None, shift_cls=None):
    """Subnet -> exit head -> compaction.  Returns a dict with every intermediate a parity
    test may want: stage_out, gap, z, conf, pred, exit, surv_idx, features_out, ids_out, n_surv."""
    st = model.stages[stage]
    so = run_layers(model, stage, x)
    h = exit_head(so, st.fc_weight, st.fc_bias, st.threshold, st.always_exit, shift, shift_cls)
    idx, fo, io = compact(h["exit"], so, ids)
    h.update(stage_out=so, surv_idx=idx, features_out=fo, ids_out=io, n_surv=len(idx))
    return h


def run_sample_serial(model, x1, shifts=None, shift_cls=None):
    """One sample alone (B = 1) until its first exit.  ``shifts`` is an optional per-exit
    logit shift.  Returns (exit_index, pred, conf list per visited exit)."""
    feat = _c32(x1)[None] if x1.ndim == 3 else _c32(x1)
    confs = []
    for s in range(len(model.stages)):
        sh = None if shifts is None else np.array([shifts[s]], dtype=np.float32)
        sc = None if shift_cls is None else np.array([shift_cls], dtype=np.int32)
        r = run_stage(model, s, feat, None, sh, sc)
        confs.append(float(r["conf"][0]))
        if r["exit"][0]:
            return s, int(r["pred"][0]), confs
        feat = r["features_out"]
    raise AssertionError("final exit must always be taken")


def serve_trace(n_stages, max_batch, arrivals, exit_of, stage_time, slo=float("inf")):
    """Algorithm 1 on a virtual clock: exit-aware preemptive scheduling with the SLO-aware
    preemption criterion (Eq. 3-4); backfilling per exit, non-recursive.

    ``arrivals``  sorted arrival times; request r has id r.
    ``exit_of``   exit index at which request r leaves (from ``run_sample_serial``).
    ``stage_time(stage, batch)`` service time of one subnet at a batch size; it is also the
                  exit-level latency table the criterion looks up (Section III-B, Exit-Level
                  Latency Prediction), so on this clock the prediction is exact.
    ``slo``       T_SLO in the unit of ``arrivals``.  At the preemption point behind exit i, with
                  B_rem samples left, B_incr = min(N_Q, B_max - B_rem) > 0 candidates queued:
                    T_slack    = T_SLO - (now - arrival of the oldest sample of the active batch)   (Eq. 3)
                    T_overhead = T_{0:i}(B_incr) + T_{i+1:L-1}(B_rem + B_incr)                     (Eq. 4)
                  and the batch is preempted iff T_overhead < T_slack.  An active batch that has
                  lost all its samples constrains nothing (its slack is infinite).  With
                  slo = inf every backfill that fits is taken.
    Returns (finish_time per request, list of (stage, ids tuple) launches in order)."""
    n = len(arrivals)
    finish = np.zeros(n)
    launches = []
    q = deque()
    nxt = 0
    t = 0.0

    def admit(now):
        nonlocal nxt
        while nxt < n and arrivals[nxt] <= now:
            q.append(nxt)
            nxt += 1

    def proc(stage, ids, now):
        launches.append((stage, tuple(ids)))
        now += stage_time(stage, len(ids))
        rem = []
        for r in ids:
            if exit_of[r] == stage:
                finish[r] = now
            else:
                rem.append(r)
        return rem, now

    def span(first, last, batch):
        """T_{first:last}^{batch}: subnets first..last (inclusive) at one batch size."""
        total = 0.0
        for j in range(first, last + 1):
            total += stage_time(j, batch)
        return total

    while nxt < n or q:
        admit(t)
        if not q:
            t = arrivals[nxt]
            admit(t)
        act = [q.popleft() for _ in range(min(len(q), max_batch))]
        i = 0
        while i < n_stages - 1:
            act, t = proc(i, act, t)
            while len(act) < max_batch:
                admit(t)
                incr = min(len(q), max_batch - len(act))
                if incr == 0:
                    break
                if act:
                    oldest = min(arrivals[r] for r in act)
                    t_slack = slo - (t - oldest)
                    t_overhead = span(0, i, incr) + span(i + 1, n_stages - 1, len(act) + incr)
                    if not t_overhead < t_slack:
                        break
                new = [q.popleft() for _ in range(incr)]
                for j in range(i + 1):          # the new batch catches up to exit i
                    new, t = proc(j, new, t)
                    if not new:
                        break
                act = act + new                 # B_merged = B_rem + B_incr - B_exit
            if not act:
                break
            i += 1
        if act:
            act, t = proc(n_stages - 1, act, t)
            assert not act
    return finish, launches
