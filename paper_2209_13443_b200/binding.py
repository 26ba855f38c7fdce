"""ctypes binding of ``libeecnn.so`` (declared in ``include/ee.h``).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch supplies device memory and streams.  There is no CPU fallback: if the shared
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libeecnn.so")

EE_OK = 0
STATUS_NAMES = ["EE_OK", "EE_ERR_INVALID_ARG", "EE_ERR_SHAPE", "EE_ERR_CAPACITY", "EE_ERR_STAGE", "EE_ERR_UNSUPPORTED",
                "EE_ERR_CUDA", "EE_ERR_TIMEOUT", "EE_ERR_INTERNAL"]
EXPORTS = ["ee_model_create", "ee_model_destroy", "ee_model_query", "ee_stage_run", "ee_layer_run", "ee_batch_refill", "ee_exit_head",
           "ee_exit_head_scratch_bytes", "ee_exit_head_static", "ee_gather_survivors", "ee_model_set_graphs", "ee_model_set_branches", "ee_model_set_fused_head", "ee_model_set_proj_fusion", "ee_model_set_gap_fusion", "ee_model_gap_partials", "ee_model_head_launches", "ee_model_set_stage_kernel", "ee_model_set_chain", "ee_model_set_timing", "ee_model_get_timing",
           "ee_model_plan", "ee_model_check", "ee_model_set_layer_variant", "ee_model_set_layer_splits", "ee_model_get_layer_config",
           "ee_model_set_wait_limit", "ee_model_selftest_wait", "ee_wait_count", "ee_run_until_exit", "ee_status_string", "ee_last_cuda_error"]


class EEError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: {name}" + (f" ({detail})" if detail else ""))


class LayerDesc(C.Structure):
    _fields_ = [("op", C.c_int), ("cin", C.c_int), ("cout", C.c_int), ("kh", C.c_int), ("kw", C.c_int), ("stride", C.c_int),
                ("pad", C.c_int), ("act", C.c_int), ("input_from", C.c_int), ("residual_from", C.c_int),
                ("weight", C.c_void_p), ("scale", C.c_void_p), ("bias", C.c_void_p), ("pad_w", C.c_int)]


class StageDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("layers", C.POINTER(LayerDesc)), ("out_layer", C.c_int), ("n_classes", C.c_int),
                ("fc_weight", C.c_void_p), ("fc_bias", C.c_void_p), ("threshold", C.c_float), ("always_exit", C.c_int)]


class ModelDesc(C.Structure):
    _fields_ = [("dtype", C.c_int), ("in_h", C.c_int), ("in_w", C.c_int), ("in_c", C.c_int), ("n_stages", C.c_int),
                ("stages", C.POINTER(StageDesc)), ("max_batch", C.c_int), ("weights_on_device", C.c_int)]


class StageInfo(C.Structure):
    _fields_ = [("in_h", C.c_int), ("in_w", C.c_int), ("in_c", C.c_int), ("out_h", C.c_int), ("out_w", C.c_int),
                ("out_c", C.c_int), ("in_bytes_per_sample", C.c_size_t), ("out_bytes_per_sample", C.c_size_t),
                ("workspace_bytes", C.c_size_t), ("n_layers", C.c_int), ("flops_per_sample", C.c_double)]


class StageIn(C.Structure):
    _fields_ = [("features", C.c_void_p), ("ids", C.c_void_p), ("batch", C.c_int), ("logit_shift", C.c_void_p),
                ("shift_class", C.c_void_p)]


class StageOut(C.Structure):
    _fields_ = [("features_out", C.c_void_p), ("conf", C.c_void_p), ("pred", C.c_void_p), ("logits", C.c_void_p),
                ("exit_mask", C.c_void_p), ("survivor_idx", C.c_void_p), ("ids_out", C.c_void_p), ("n_surv_dev", C.c_void_p),
                ("n_surv_host", C.c_void_p)]


class LayerPlan(C.Structure):
    _fields_ = [("kernel", C.c_char_p), ("m", C.c_int), ("n", C.c_int), ("k", C.c_int), ("flops", C.c_double),
                ("bytes", C.c_double), ("launches", C.c_int)]


_lib = None


def load_library() -> C.CDLL:
    """Loads the in-tree shared library and declares the prototypes.  Raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_SO):
        raise FileNotFoundError(f"{_SO} not built: run `python -m paper_2209_13443_b200.build` (or __graft_entry__.build())")
    L = C.CDLL(_SO)
    vp, i = C.c_void_p, C.c_int
    L.ee_model_create.argtypes = [C.POINTER(ModelDesc), vp, C.POINTER(vp)]
    L.ee_model_destroy.argtypes = [vp]
    L.ee_model_query.argtypes = [vp, i, C.POINTER(StageInfo)]
    L.ee_stage_run.argtypes = [vp, i, C.POINTER(StageIn), vp, C.c_size_t, C.POINTER(StageOut), vp]
    L.ee_layer_run.argtypes = [vp, i, i, vp, vp, i, vp, vp, C.c_size_t, vp]
    L.ee_batch_refill.argtypes = [vp, i, vp, vp, i, vp, vp, i, C.POINTER(i), C.POINTER(i), vp]
    L.ee_exit_head.argtypes = [vp, i, vp, i, i, vp, vp, vp, C.c_size_t, C.POINTER(StageOut), vp]
    L.ee_exit_head_static.argtypes = [vp, i, vp, i, i, vp, vp, C.POINTER(StageOut), vp]
    L.ee_exit_head_scratch_bytes.argtypes = [vp, i]
    L.ee_exit_head_scratch_bytes.restype = C.c_size_t
    L.ee_gather_survivors.argtypes = [vp, C.c_size_t, vp, vp, i, vp, vp]
    L.ee_model_set_graphs.argtypes = [vp, i]
    L.ee_model_set_timing.argtypes = [vp, i]
    L.ee_model_set_branches.argtypes = [vp, i]
    L.ee_model_set_fused_head.argtypes = [vp, i]
    L.ee_model_set_proj_fusion.argtypes = [vp, i]
    L.ee_model_set_gap_fusion.argtypes = [vp, i]
    L.ee_model_gap_partials.argtypes = [vp, i, i]
    L.ee_model_gap_partials.restype = i
    L.ee_model_head_launches.argtypes = [vp, i]
    L.ee_model_head_launches.restype = i
    L.ee_model_set_stage_kernel.argtypes = [vp, i, i]
    L.ee_model_set_chain.argtypes = [vp, i]
    L.ee_model_get_timing.argtypes = [vp, i, i, C.POINTER(C.c_float), C.POINTER(C.c_char_p), C.POINTER(i)]
    L.ee_model_plan.argtypes = [vp, i, i, i, C.POINTER(LayerPlan), C.POINTER(i)]
    L.ee_run_until_exit.argtypes = [vp, i, C.POINTER(StageIn), vp, C.c_size_t, C.POINTER(StageOut), C.POINTER(C.c_int32), C.c_double, vp]
    L.ee_wait_count.argtypes = [vp, C.c_int32, C.c_double, C.POINTER(C.c_int32)]
    L.ee_model_check.argtypes = [vp, vp]
    L.ee_model_set_layer_variant.argtypes = [vp, i, i, i, i, i]
    L.ee_model_set_layer_splits.argtypes = [vp, i, i, i]
    L.ee_model_get_layer_config.argtypes = [vp, i, i, i, C.POINTER(i), C.POINTER(i), C.POINTER(i)]
    L.ee_model_set_wait_limit.argtypes = [vp, C.c_longlong]
    L.ee_model_selftest_wait.argtypes = [vp, C.c_longlong, vp]
    L.ee_status_string.argtypes = [i]
    L.ee_status_string.restype = C.c_char_p
    L.ee_last_cuda_error.restype = C.c_char_p
    _lib = L
    return L


def _check(rc: int, where: str):
    if rc != EE_OK:
        raise EEError(rc, where, load_library().ee_last_cuda_error().decode())


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return int(t)


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def torch_dtype(model_dtype: str):
    return torch.bfloat16 if model_dtype == "bf16" else torch.float32


class StageBuffers:
    """Caller-owned device buffers of one ee_stage_run call, sized for max_batch (allocated once)."""

    def __init__(self, model: "EEModel", stage: int, with_logits: bool = True, pinned_count: bool = True):
        info = model.query(stage)
        dev, B = model.device, model.max_batch
        td = torch_dtype(model.dtype)
        self.info = info
        self.features_out = torch.empty((B, info["out_h"], info["out_w"], info["out_c"]), dtype=td, device=dev)
        self.conf = torch.empty(B, dtype=torch.float32, device=dev)
        self.pred = torch.empty(B, dtype=torch.int32, device=dev)
        self.logits = torch.empty((B, model.n_classes[stage]), dtype=torch.float32, device=dev) if with_logits else None
        self.exit_mask = torch.empty(B, dtype=torch.uint8, device=dev)
        self.survivor_idx = torch.empty(B, dtype=torch.int32, device=dev)
        self.ids_out = torch.empty(B, dtype=torch.int32, device=dev)
        self.n_surv_dev = torch.zeros(1, dtype=torch.int32, device=dev)
        self.n_surv_host = torch.zeros(1, dtype=torch.int32).pin_memory() if pinned_count else None
        self._count_word = C.c_int32.from_address(self.n_surv_host.data_ptr()) if pinned_count else None
        self._struct = None

    def arm_count(self):
        """Stores the sentinel -1 in the pinned count word; call before ee_stage_run, then wait_count()."""
        self._count_word.value = -1

    def wait_count(self, timeout_s: float = 10.0) -> int:
        """B_rem of the stage launched after arm_count(), as soon as the exit decisions are taken (ee_wait_count):
        the stream is not synchronised and the gather of the survivors' features may still be running."""
        v = C.c_int32(-1)
        _check(load_library().ee_wait_count(self.n_surv_host.data_ptr(), -1, float(timeout_s), C.byref(v)), "ee_wait_count")
        return int(v.value)

    def as_struct(self) -> StageOut:
        """The ee_stage_out_t of these buffers (built once: the buffers never move)."""
        if self._struct is None:
            self._struct = StageOut(_ptr(self.features_out), _ptr(self.conf), _ptr(self.pred), _ptr(self.logits), _ptr(self.exit_mask),
                                    _ptr(self.survivor_idx), _ptr(self.ids_out), _ptr(self.n_surv_dev), _ptr(self.n_surv_host))
        return self._struct


class EEModel:
    """Handle of one early-exit model on the current CUDA device (wraps ee_model_t)."""

    def __init__(self, spec, device: str = "cuda", stream=None, apply_tables: bool = True):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this library has no CPU path")
        self._L = load_library()
        self.device = torch.device(device)
        self.dtype = spec.dtype
        self.max_batch = spec.max_batch
        self.n_stages = len(spec.stages)
        self.n_classes = [s.n_classes for s in spec.stages]
        self._keep = []   # host arrays referenced by the descriptor until create returns

        def host(a, narrow: bool):
            if a is None:
                return None
            t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
            if narrow and self.dtype == "bf16":
                t = t.to(torch.bfloat16)
            self._keep.append(t)
            return t.data_ptr()

        stage_structs = (StageDesc * self.n_stages)()
        for si, st in enumerate(spec.stages):
            layers = (LayerDesc * len(st.layers))()
            self._keep.append(layers)
            for li, l in enumerate(st.layers):
                layers[li] = LayerDesc(l.op, l.cin, l.cout, l.kh, l.kw, l.stride, l.pad, l.act, l.input_from, l.residual_from,
                                       host(l.weight, True), host(l.scale, False), host(l.bias, False), int(getattr(l, "pad_w", -1)))
            stage_structs[si] = StageDesc(len(st.layers), layers, st.out_layer, st.n_classes, host(st.fc_weight, True),
                                          host(st.fc_bias, False), float(st.threshold), int(bool(st.always_exit)))
        desc = ModelDesc(1 if self.dtype == "bf16" else 0, spec.in_h, spec.in_w, spec.in_c, self.n_stages, stage_structs,
                         spec.max_batch, 0)
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(self._L.ee_model_create(C.byref(desc), _stream(stream), C.byref(h)), "ee_model_create")
        self._h = h
        self._keep = []
        self._outs_key, self._outs_arr = None, None
        self.table = None
        if apply_tables:
            self.table = apply_table(self, spec)

    def close(self):
        if getattr(self, "_h", None):
            torch.cuda.synchronize()
            self._L.ee_model_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def query(self, stage: int) -> dict:
        info = StageInfo()
        _check(self._L.ee_model_query(self._h, stage, C.byref(info)), "ee_model_query")
        return {k: getattr(info, k) for k, _ in StageInfo._fields_}

    def workspace(self, stage: Optional[int] = None) -> torch.Tensor:
        stages = range(self.n_stages) if stage is None else [stage]
        nbytes = max(self.query(s)["workspace_bytes"] for s in stages)
        return torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)

    def stage_run(self, stage: int, features, batch: int, out: StageBuffers, workspace: torch.Tensor, ids=None,
                  logit_shift=None, shift_class=None, stream=None):
        base = workspace.data_ptr()
        aligned = (base + 255) // 256 * 256
        sin = StageIn(_ptr(features), _ptr(ids), int(batch), _ptr(logit_shift), _ptr(shift_class))
        so = out.as_struct() if isinstance(out, StageBuffers) else out
        _check(self._L.ee_stage_run(self._h, stage, C.byref(sin), aligned, workspace.numel() - (aligned - base), C.byref(so),
                                    _stream(stream)), "ee_stage_run")

    def run_until_exit(self, first_stage: int, features, batch: int, outs: Sequence[StageBuffers], workspace: torch.Tensor, ids=None,
                       logit_shift=None, shift_class=None, timeout_s: float = 10.0, stream=None):
        """ee_run_until_exit: every stage from ``first_stage`` on, each on the survivors of the one before, until the
        batch is empty or the last stage has been launched.  ``outs`` holds one StageBuffers per stage of the model.
        Returns the batch each stage ran on (0 for stages not reached)."""
        key = tuple(id(o) for o in outs)
        if self._outs_key != key:       # the array of ee_stage_out_t is built once per set of buffers
            arr = (StageOut * self.n_stages)()
            for s, o in enumerate(outs):
                arr[s] = o.as_struct()
            self._outs_key, self._outs_arr = key, arr
        base = workspace.data_ptr()
        aligned = (base + 255) // 256 * 256
        sin = StageIn(_ptr(features), _ptr(ids), int(batch), _ptr(logit_shift), _ptr(shift_class))
        sizes = (C.c_int32 * self.n_stages)()
        _check(self._L.ee_run_until_exit(self._h, first_stage, C.byref(sin), aligned, workspace.numel() - (aligned - base),
                                         self._outs_arr, sizes, float(timeout_s), _stream(stream)), "ee_run_until_exit")
        return list(sizes)

    def layer_run(self, stage: int, layer: int, x, residual, batch: int, out, workspace: torch.Tensor, stream=None):
        base = workspace.data_ptr()
        aligned = (base + 255) // 256 * 256
        _check(self._L.ee_layer_run(self._h, stage, layer, _ptr(x), _ptr(residual), int(batch), _ptr(out), aligned,
                                    workspace.numel() - (aligned - base), _stream(stream)), "ee_layer_run")

    def batch_refill(self, boundary: int, batch_feat, batch_ids, n_surv: int, arr_feat, arr_ids, n_arr: int, stream=None):
        n_acc, n_mer = C.c_int(-1), C.c_int(-1)
        _check(self._L.ee_batch_refill(self._h, boundary, _ptr(batch_feat), _ptr(batch_ids), int(n_surv), _ptr(arr_feat),
                                       _ptr(arr_ids), int(n_arr), C.byref(n_acc), C.byref(n_mer), _stream(stream)),
               "ee_batch_refill")
        return n_acc.value, n_mer.value

    def exit_head_scratch_bytes(self, stage: int) -> int:
        return int(self._L.ee_exit_head_scratch_bytes(self._h, stage))

    def exit_head(self, stage: int, x, batch: int, hw: int, out: StageBuffers, scratch: torch.Tensor, logit_shift=None,
                  shift_class=None, stream=None):
        base = scratch.data_ptr()
        aligned = (base + 255) // 256 * 256
        so = out.as_struct() if isinstance(out, StageBuffers) else out
        _check(self._L.ee_exit_head(self._h, stage, _ptr(x), int(batch), int(hw), _ptr(logit_shift), _ptr(shift_class), aligned,
                                    scratch.numel() - (aligned - base), C.byref(so), _stream(stream)), "ee_exit_head")

    def exit_head_static(self, stage: int, x, batch: int, hw: int, out: StageBuffers, logit_shift=None, shift_class=None,
                         stream=None):
        """ee_exit_head on the library's built-in scratch array: nothing is allocated, here or in the library.
        For callers that must not allocate device memory at decision time; calls that overlap on the GPU race."""
        so = out.as_struct() if isinstance(out, StageBuffers) else out
        _check(self._L.ee_exit_head_static(self._h, stage, _ptr(x), int(batch), int(hw), _ptr(logit_shift), _ptr(shift_class),
                                           C.byref(so), _stream(stream)), "ee_exit_head_static")

    def set_graphs(self, enabled: bool):
        _check(self._L.ee_model_set_graphs(self._h, int(enabled)), "ee_model_set_graphs")

    def set_branches(self, enabled: bool):
        _check(self._L.ee_model_set_branches(self._h, int(enabled)), "ee_model_set_branches")

    def set_proj_fusion(self, enabled: bool):
        """Projection shortcuts computed inside the layer that adds them (bit-identical either way)."""
        _check(self._L.ee_model_set_proj_fusion(self._h, int(enabled)), "ee_model_set_proj_fusion")

    def set_gap_fusion(self, enabled: bool):
        """Pooling partials written by the last layer's epilogue (bit-identical either way)."""
        _check(self._L.ee_model_set_gap_fusion(self._h, int(enabled)), "ee_model_set_gap_fusion")

    def gap_partials(self, stage: int, batch: int) -> int:
        return int(self._L.ee_model_gap_partials(self._h, stage, batch))

    def set_fused_head(self, enabled: bool):
        """One-launch exit head (cluster kernel) on / off; off = pooling kernel + FC/decision kernel."""
        _check(self._L.ee_model_set_fused_head(self._h, int(enabled)), "ee_model_set_fused_head")

    def head_launches(self, stage: int) -> int:
        return int(self._L.ee_model_head_launches(self._h, stage))

    def set_stage_kernel(self, enabled: bool, max_batch: int = 0):
        _check(self._L.ee_model_set_stage_kernel(self._h, int(enabled), int(max_batch)), "ee_model_set_stage_kernel")

    def set_chain(self, max_batch: int):
        _check(self._L.ee_model_set_chain(self._h, int(max_batch)), "ee_model_set_chain")

    def set_timing(self, enabled: bool):
        _check(self._L.ee_model_set_timing(self._h, int(enabled)), "ee_model_set_timing")

    def get_timing(self, stage: int, cap: int = 256):
        ms = (C.c_float * cap)()
        names = (C.c_char_p * cap)()
        n = C.c_int(0)
        _check(self._L.ee_model_get_timing(self._h, stage, cap, ms, names, C.byref(n)), "ee_model_get_timing")
        return [(names[i].decode(), float(ms[i])) for i in range(n.value)]

    def plan(self, stage: int, batch: int, cap: int = 256):
        arr = (LayerPlan * cap)()
        n = C.c_int(0)
        _check(self._L.ee_model_plan(self._h, stage, int(batch), cap, arr, C.byref(n)), "ee_model_plan")
        return [dict(kernel=arr[i].kernel.decode(), m=arr[i].m, n=arr[i].n, k=arr[i].k, flops=arr[i].flops, bytes=arr[i].bytes,
                     launches=arr[i].launches)
                for i in range(n.value)]

    def set_layer_variant(self, stage: int, layer: int, batch_lo: int, batch_hi: int, variant: int):
        _check(self._L.ee_model_set_layer_variant(self._h, stage, layer, batch_lo, batch_hi, variant), "ee_model_set_layer_variant")

    def set_layer_splits(self, stage: int, layer: int, splits: int):
        _check(self._L.ee_model_set_layer_splits(self._h, stage, layer, splits), "ee_model_set_layer_splits")

    def layer_config(self, stage: int, layer: int, batch: int) -> dict:
        v, s, t = C.c_int(0), C.c_int(0), C.c_int(0)
        _check(self._L.ee_model_get_layer_config(self._h, stage, layer, batch, C.byref(v), C.byref(s), C.byref(t)), "ee_model_get_layer_config")
        return {"variant": v.value, "splits": s.value, "tensor_core": t.value}

    def set_wait_limit(self, cycles: int):
        _check(self._L.ee_model_set_wait_limit(self._h, int(cycles)), "ee_model_set_wait_limit")

    def selftest_wait(self, limit_cycles: int, stream=None):
        _check(self._L.ee_model_selftest_wait(self._h, int(limit_cycles), _stream(stream)), "ee_model_selftest_wait")

    def check(self, stream=None):
        _check(self._L.ee_model_check(self._h, _stream(stream)), "ee_model_check")


def apply_table(model: EEModel, spec, path: Optional[str] = None):
    """Loads the measured per-(layer, batch) kernel table written by ``autotune.py`` for this (model name, max_batch),
    checks that it describes this model's layers, and installs it (ee_model_set_layer_splits / _variant).
    Returns the table's path, or None when there is none (the library's built-in choices stay in force)."""
    import json

    if path is None:
        path = os.path.join(_HERE, "tables", f"{spec.name}_b{spec.max_batch}.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        t = json.load(f)
    if t.get("max_batch") != spec.max_batch or t.get("input") != [spec.in_h, spec.in_w, spec.in_c]:
        return None
    for e in t["layers"]:
        s, i = e["stage"], e["layer"]
        if s >= len(spec.stages) or i >= len(spec.stages[s].layers):
            return None
        l = spec.stages[s].layers[i]
        if [l.kh, l.cin, l.cout, l.stride] != e["geom"][:4] or len(e["variants"]) != spec.max_batch:
            return None
    for e in t["layers"]:
        s, i = e["stage"], e["layer"]
        model.set_layer_splits(s, i, e["splits"])
        v = e["variants"]
        lo = 1
        for b in range(2, spec.max_batch + 2):     # runs of equal entries
            if b == spec.max_batch + 1 or v[b - 1] != v[lo - 1]:
                model.set_layer_variant(s, i, lo, b - 1, v[lo - 1])
                lo = b
    return path


def gather_survivors(feat, bytes_per_sample: int, survivor_idx, n_surv_dev, max_rows: int, feat_out, stream=None):
    _check(load_library().ee_gather_survivors(_ptr(feat), int(bytes_per_sample), _ptr(survivor_idx), _ptr(n_surv_dev),
                                              int(max_rows), _ptr(feat_out), _stream(stream)), "ee_gather_survivors")


def to_device(model_dtype: str, a: np.ndarray, device="cuda") -> torch.Tensor:
    """Host float32 array (already on the model's grid) -> device tensor of the model dtype."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device=device, dtype=torch_dtype(model_dtype))
