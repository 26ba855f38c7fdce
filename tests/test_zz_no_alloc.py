"""ee_exit_head_static: the exit head on the library's built-in scratch array.

Some users of this library cannot allocate device memory at the moment they need an exit decision (a host
application that owns all device memory and forbids later cudaMalloc calls, or a latency-bound serving thread).
For them the library carries its own fixed scratch array.  This test drives the entry point through the C ABI and
holds it to the existing ee_exit_head on the same inputs, twice in a row with different batches, so that whatever
the first call left behind in the shared array must not leak into the second; it also holds it to the CPU oracle,
checks that a call leaves the amount of free device memory untouched, runs a second model with another head
layout on the same dirty array, and the empty batch.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import ee_oracle as eo
from paper_2209_13443_b200 import binding as eb
from paper_2209_13443_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def _head_model(dtype, HW, C, K, max_batch):
    rng = wl._rng(C + K, 903)
    bf16 = dtype == "bf16"
    fw, fb = wl._head(rng, C, K, 0.5, bf16)          # flat logits: only the shifted samples reach the threshold
    layers = [wl._conv(rng, wl.OP_CONV, C, C, 1, 1, 0, wl.ACT_NONE, bf16=bf16)]
    return wl.Model("head", dtype, 1, HW, C, [wl.Stage(layers, K, fw, fb, 0.5, False)], max_batch)


def _run(m, out, fn, x, B, HW, shift, cls):
    out.logits.fill_(float("nan"))
    out.n_surv_dev.fill_(-1)
    fn(0, x, B, HW, out, logit_shift=shift, shift_class=cls)
    torch.cuda.synchronize()
    n = int(out.n_surv_dev.cpu()[0])
    return {"z": out.logits[:B].cpu().numpy(), "conf": out.conf[:B].cpu().numpy(), "pred": out.pred[:B].cpu().numpy(),
            "exit": out.exit_mask[:B].cpu().numpy(), "idx": out.survivor_idx[:n].cpu().numpy(), "n": n}


@pytest.mark.parametrize("dtype,HW,C,K", [("bf16", 196, 256, 1000), ("f32", 50, 40, 17)])
def test_static_scratch_head_matches_caller_scratch_head_twice(dtype, HW, C, K):
    spec = _head_model(dtype, HW, C, K, max_batch=48)
    m = eb.EEModel(spec)
    out_ref, out_new = eb.StageBuffers(m, 0), eb.StageBuffers(m, 0)
    scratch = torch.empty(m.exit_head_scratch_bytes(0) + 256, dtype=torch.uint8, device="cuda")
    tol = util.TOL[dtype]
    for call, B in enumerate((48, 19)):                                  # second call: smaller batch on a dirty array
        x = eb.to_device(dtype, wl.random_features((B, HW, C), seed=60 + call, bf16=dtype == "bf16"))
        shift = torch.as_tensor((np.arange(B) % 4 == 0).astype(np.float32) * 9.0, device="cuda")
        cls = torch.as_tensor((np.arange(B) * 3 % K).astype(np.int32), device="cuda")
        ref = _run(m, out_ref, lambda *a, **k: m.exit_head(*a[:5], scratch, **k), x, B, HW, shift, cls)
        new = _run(m, out_new, m.exit_head_static, x, B, HW, shift, cls)
        assert util.norm_err(new["z"], ref["z"]) <= tol and util.rel_err(new["z"], ref["z"], dtype, floor=util.LOGIT_FLOOR[dtype]) <= tol
        assert np.max(np.abs(new["conf"] - ref["conf"])) <= tol
        assert np.array_equal(new["pred"], ref["pred"]) and np.array_equal(new["exit"], ref["exit"])
        assert new["n"] == ref["n"] and np.array_equal(new["idx"], ref["idx"])
        assert new["n"] == B - len(range(0, B, 4))                       # every fourth sample was pushed over the threshold
        # against the CPU oracle's exit head on the same inputs
        st = spec.stages[0]
        o = eo.exit_head(x.float().cpu().numpy(), st.fc_weight, st.fc_bias, st.threshold, False, shift.cpu().numpy(), cls.cpu().numpy())
        assert util.norm_err(new["z"], o["z"]) <= (2e-3 if dtype == "bf16" else 1e-5)
        band = np.abs(o["conf"] - st.threshold) < util.BAND
        assert np.array_equal(new["exit"][~band], o["exit"][~band])
        if not band.any():
            assert np.array_equal(new["idx"], np.nonzero(o["exit"] == 0)[0])
        # the property the entry point exists for: a call allocates no device memory
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        m.exit_head_static(0, x, B, HW, out_new, logit_shift=shift, shift_class=cls)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before
    # the empty batch: only the count is written
    out_new.n_surv_dev.fill_(77)
    m.exit_head_static(0, None, 0, HW, out_new)
    torch.cuda.synchronize()
    assert int(out_new.n_surv_dev.cpu()[0]) == 0
    # another model with another head layout (C, K, max_batch) on the same, now dirty, array
    spec2 = _head_model(dtype, 9, 72, 33, max_batch=7)
    m2 = eb.EEModel(spec2)
    o_ref, o_new = eb.StageBuffers(m2, 0), eb.StageBuffers(m2, 0)
    scratch2 = torch.empty(m2.exit_head_scratch_bytes(0) + 256, dtype=torch.uint8, device="cuda")
    x2 = eb.to_device(dtype, wl.random_features((7, 9, 72), seed=77, bf16=dtype == "bf16"))
    ref = _run(m2, o_ref, lambda *a, **k: m2.exit_head(*a[:5], scratch2, **k), x2, 7, 9, None, None)
    new = _run(m2, o_new, m2.exit_head_static, x2, 7, 9, None, None)
    assert np.array_equal(new["z"], ref["z"]) and np.array_equal(new["exit"], ref["exit"]) and new["n"] == ref["n"]


def test_static_scratch_head_refuses_what_does_not_fit():
    # 8 MiB array: the pooled vectors of 1100 samples x 2048 channels in fp32 alone need 9 MB
    spec = _head_model("bf16", 4, 2048, 10, max_batch=1100)
    m = eb.EEModel(spec)
    out = eb.StageBuffers(m, 0)
    x = torch.zeros((1, 4, 2048), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(eb.EEError) as e:
        m.exit_head_static(0, x, 1, 4, out)
    assert e.value.status == 3 and "scratch bytes" in str(e.value)
