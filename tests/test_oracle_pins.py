"""Pins of the CPU oracle against things other than itself.

Each check is chosen so that a plausible mistake in the oracle (dropped tap, wrong sign of
the padding offset, transposed weight index, stride applied to the wrong axis, missing
max-subtraction, unstable compaction ...) fails at least one of them:
closed forms, brute force of a different structure, torch CPU library routines in fp64,
the paper's scheduling-timeline example and Algorithm 1's identities.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import ee_oracle as eo
from paper_2209_13443_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- rounding

def test_bf16_rne_hand_values():
    # bf16 keeps 8 significant bits: ulp at 1.0 is 2^-7.
    assert eo.round_bf16(1.0 + 2.0 ** -8) == 1.0                       # tie -> even (down)
    assert eo.round_bf16(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6       # tie -> even (up)
    assert eo.round_bf16(1.0 + 2.0 ** -8 + 2.0 ** -16) == 1.0 + 2.0 ** -7
    assert eo.round_bf16(-(1.0 + 3 * 2.0 ** -8)) == -(1.0 + 2.0 ** -6)
    assert eo.round_bf16(0.0) == 0.0
    assert eo.round_bf16(255.5) == 256.0 and eo.round_bf16(254.5) == 254.0   # ties across a binade
    assert eo.round_bf16(2.0 ** -133) == 2.0 ** -133                   # smallest subnormal
    assert eo.round_bf16(0.49 * 2.0 ** -133) == 0.0
    assert math.isinf(eo.round_bf16(3.4e38))


def test_bf16_rne_matches_library_conversion():
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-6, 6, 20000),
                        rng.standard_normal(2000) * 1e-39]).astype(np.float32)
    ref = torch.from_numpy(v).to(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([eo.round_bf16(float(x)) for x in v])
    assert np.array_equal(got, ref)


# ----------------------------------------------------------------------------- convolution

def _im2col_conv(x, w, stride, pad):
    """Different structure on purpose: materialise the Toeplitz matrix R x P, then one dot
    per output (the paper's GEMM view of a convolution, Section II-C)."""
    B, H, W, Cin = x.shape
    Cout, kh, kw, _ = w.shape
    xp = np.zeros((B, H + 2 * pad, W + 2 * pad, Cin))
    xp[:, pad:pad + H, pad:pad + W] = x
    Ho, Wo = (H + 2 * pad - kh) // stride + 1, (W + 2 * pad - kw) // stride + 1
    rows = []
    for b in range(B):
        for i in range(Ho):
            for j in range(Wo):
                rows.append(xp[b, i * stride:i * stride + kh, j * stride:j * stride + kw, :].reshape(-1))
    A = np.array(rows, dtype=np.float64)                 # R x P
    Wm = w.reshape(Cout, -1).astype(np.float64).T        # P x C
    return (A @ Wm).reshape(B, Ho, Wo, Cout)


@pytest.mark.parametrize("H,W,Cin,Cout,k,stride,pad", [
    (5, 7, 3, 4, 3, 1, 1), (6, 5, 3, 2, 3, 2, 1), (9, 9, 3, 5, 7, 2, 3), (7, 6, 4, 3, 1, 1, 0),
    (7, 7, 4, 3, 1, 2, 0), (4, 4, 2, 2, 3, 1, 0), (8, 5, 5, 6, 3, 2, 1)])
def test_conv_matches_toeplitz_product(H, W, Cin, Cout, k, stride, pad):
    rng = np.random.default_rng(H * 100 + W)
    x = rng.standard_normal((2, H, W, Cin)).astype(np.float32)
    w = rng.standard_normal((Cout, k, k, Cin)).astype(np.float32)
    got = eo.conv2d(x, w, stride, pad)
    ref = _im2col_conv(x, w, stride, pad)
    assert got.shape == ref.shape
    np.testing.assert_allclose(got, ref, rtol=2e-7, atol=1e-6)


def test_conv_all_ones_closed_form():
    Cin = 5
    x = np.ones((1, 6, 8, Cin), np.float32)
    w = np.ones((2, 3, 3, Cin), np.float32)
    y = eo.conv2d(x, w, 1, 1)
    assert y[0, 2, 3, 0] == 9 * Cin          # interior
    assert y[0, 0, 3, 1] == 6 * Cin          # edge
    assert y[0, 5, 0, 0] == 4 * Cin          # corner
    assert y[0, 3, 7, 1] == 6 * Cin


def test_conv_centre_delta_is_identity_and_offsets_have_the_right_sign():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((2, 5, 6, 3)).astype(np.float32)
    w = np.zeros((3, 3, 3, 3), np.float32)
    for c in range(3):
        w[c, 1, 1, c] = 1
    np.testing.assert_array_equal(eo.conv2d(x, w, 1, 1), x)
    # tap (r=0, s=1) reads the pixel one row ABOVE: y[h, w] = x[h-1, w]
    w2 = np.zeros((3, 3, 3, 3), np.float32)
    for c in range(3):
        w2[c, 0, 1, c] = 1
    y = eo.conv2d(x, w2, 1, 1)
    np.testing.assert_array_equal(y[:, 1:], x[:, :-1])
    assert np.all(y[:, 0] == 0)
    # tap (r=1, s=2) reads the pixel to the RIGHT: y[h, w] = x[h, w+1]
    w3 = np.zeros((3, 3, 3, 3), np.float32)
    for c in range(3):
        w3[c, 1, 2, c] = 1
    y = eo.conv2d(x, w3, 1, 1)
    np.testing.assert_array_equal(y[:, :, :-1], x[:, :, 1:])
    assert np.all(y[:, :, -1] == 0)


def test_conv_1x1_is_per_pixel_matvec_and_stride2_subsamples():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((2, 6, 6, 7)).astype(np.float32)
    w = rng.standard_normal((4, 1, 1, 7)).astype(np.float32)
    y = eo.conv2d(x, w)
    ref = x.astype(np.float64) @ w.reshape(4, 7).astype(np.float64).T
    np.testing.assert_allclose(y, ref, rtol=2e-7, atol=1e-6)
    w3 = rng.standard_normal((4, 3, 3, 7)).astype(np.float32)
    np.testing.assert_array_equal(eo.conv2d(x, w3, 2, 1), eo.conv2d(x, w3, 1, 1)[:, ::2, ::2])
    np.testing.assert_array_equal(eo.conv2d(x, w, 2, 0), y[:, ::2, ::2])


@pytest.mark.parametrize("groups", [1, 6])
@pytest.mark.parametrize("stride,pad,k", [(1, 1, 3), (2, 1, 3), (2, 3, 7), (1, 0, 1)])
def test_conv_matches_torch_fp64(groups, stride, pad, k):
    rng = np.random.default_rng(3)
    Cin, Cout = 6, 6 if groups == 6 else 5
    x = rng.standard_normal((2, 11, 9, Cin)).astype(np.float32)
    w = rng.standard_normal((Cout, k, k, Cin // groups)).astype(np.float32)
    scale = rng.uniform(0.5, 1.5, Cout).astype(np.float32)
    bias = rng.standard_normal(Cout).astype(np.float32)
    ref = F.conv2d(torch.from_numpy(x).double().permute(0, 3, 1, 2), torch.from_numpy(w).double().permute(0, 3, 1, 2),
                   stride=stride, padding=pad, groups=groups).permute(0, 2, 3, 1)
    res = rng.standard_normal(tuple(ref.shape)).astype(np.float32)
    ref = ref * torch.from_numpy(scale).double() + torch.from_numpy(bias).double() + torch.from_numpy(res).double()
    for act, fn in [(0, lambda t: t), (1, torch.relu), (2, lambda t: t.clamp(0, 6))]:
        got = eo.conv2d(x, w, stride, pad, groups, scale, bias, res, act)
        np.testing.assert_allclose(got, fn(ref).numpy(), rtol=2e-7, atol=1e-6)


@pytest.mark.parametrize("kh,kw,ph,pw,stride", [(1, 7, 0, 3, 1), (7, 1, 3, 0, 1), (3, 5, 1, 2, 2), (1, 3, 0, 0, 1), (5, 1, 0, 0, 2)])
def test_conv_with_per_axis_padding_matches_torch_fp64_and_closed_forms(kh, kw, ph, pw, stride):
    """Filters that are not square and pad only along their own axis (the factorised 1 x 7 / 7 x 1 convolutions of
    Inception-v3, Section IV Benchmarks): torch fp64 with padding=(ph, pw), and an all-ones closed form that tells the
    axes apart (a transposed pad or filter changes the count of in-range taps at the borders)."""
    rng = np.random.default_rng(kh * 10 + kw)
    x = rng.standard_normal((2, 9, 11, 4)).astype(np.float32)
    w = rng.standard_normal((3, kh, kw, 4)).astype(np.float32)
    got = eo.conv2d(x, w, stride, ph, pad_w=pw)
    ref = F.conv2d(torch.from_numpy(x).double().permute(0, 3, 1, 2), torch.from_numpy(w).double().permute(0, 3, 1, 2),
                   stride=stride, padding=(ph, pw)).permute(0, 2, 3, 1).numpy()
    assert got.shape == ref.shape
    np.testing.assert_allclose(got, ref, rtol=2e-7, atol=1e-6)
    ones = eo.conv2d(np.ones((1, 9, 11, 2), np.float32), np.ones((1, kh, kw, 2), np.float32), 1, ph, pad_w=pw)
    rows_in = lambda c, n, k, p: sum(0 <= c - p + t < n for t in range(k))     # noqa: E731
    for (ho, wo) in [(0, 0), (0, ones.shape[2] - 1), (ones.shape[1] - 1, 0), (ones.shape[1] // 2, ones.shape[2] // 2)]:
        assert ones[0, ho, wo, 0] == 2 * rows_in(ho, 9, kh, ph) * rows_in(wo, 11, kw, pw)
    # pad_w left out or negative: the same padding on both axes, i.e. the square-padding routine
    if kh == kw:
        np.testing.assert_array_equal(eo.conv2d(x, w, stride, ph), eo.conv2d(x, w, stride, ph, pad_w=ph))


def test_epilogue_order_and_bf16_store():
    # residual is added BEFORE the activation; ReLU6 clamps at 6; the store rounds once to bf16
    x = np.array([[[[1.0]]]], np.float32)
    w = np.array([[[[2.0]]]], np.float32)
    res = np.array([[[[-5.0]]]], np.float32)
    assert eo.conv2d(x, w, residual=res, act=1)[0, 0, 0, 0] == 0.0           # relu(2-5) not relu(2)-5
    assert eo.conv2d(x, w, scale=[4.0], bias=[1.0], act=2)[0, 0, 0, 0] == 6.0
    assert eo.conv2d(x, w, scale=[4.0], bias=[1.0], act=0)[0, 0, 0, 0] == 9.0
    w2 = np.array([[[[1.0 + 3 * 2.0 ** -8]]]], np.float32)
    assert eo.conv2d(x, w2, bf16=True)[0, 0, 0, 0] == np.float32(1.0 + 2.0 ** -6)
    assert eo.conv2d(x, w2, bf16=False)[0, 0, 0, 0] == np.float32(1.0 + 3 * 2.0 ** -8)


def test_conv_linearity():
    rng = np.random.default_rng(4)
    x1 = rng.standard_normal((1, 6, 6, 3)).astype(np.float32)
    x2 = rng.standard_normal((1, 6, 6, 3)).astype(np.float32)
    w = rng.standard_normal((4, 3, 3, 3)).astype(np.float32)
    a = eo.conv2d(x1, w, 2, 1).astype(np.float64) + 2 * eo.conv2d(x2, w, 2, 1)
    b = eo.conv2d((x1.astype(np.float64) + 2 * x2).astype(np.float32), w, 2, 1)
    np.testing.assert_allclose(a, b, rtol=1e-5, atol=1e-5)


def test_maxpool_matches_torch_and_ignores_padding():
    rng = np.random.default_rng(5)
    x = -np.abs(rng.standard_normal((2, 9, 8, 3))).astype(np.float32) - 1.0   # all negative: zero padding would win
    ref = F.max_pool2d(torch.from_numpy(x).permute(0, 3, 1, 2), 3, 2, 1).permute(0, 2, 3, 1).numpy()
    np.testing.assert_array_equal(eo.maxpool(x, 3, 2, 1), ref)


# ----------------------------------------------------------------------------- exit head

def test_softmax_top1_closed_forms():
    g = json.load(open(os.path.join(GOLD, "softmax_top1_closed_form.json")))
    for row in g["critical_margin"]:
        K, tau, d = row["K"], row["tau"], row["d"]
        assert abs(d - math.log(tau * (K - 1) / (1 - tau))) < 1e-12
        # identity FC on a 1x1 map: logits == features
        eye = np.eye(K, dtype=np.float32)
        for delta, want in [(+0.01, 1), (-0.01, 0)]:
            x = np.zeros((1, 1, 1, K), np.float32)
            x[0, 0, 0, 3] = d + delta
            r = eo.exit_head(x, eye, None, tau)
            assert r["exit"][0] == want and r["pred"][0] == 3
            assert abs(r["conf"][0] - 1 / (1 + (K - 1) * math.exp(-(d + delta)))) < 1e-6
    for K in (10, 1000):
        r = eo.exit_head(np.full((1, 2, 2, 4), 0.3, np.float32), np.ones((K, 4), np.float32), None, 0.5)
        assert abs(r["conf"][0] - 1.0 / K) < 1e-12 and r["pred"][0] == 0     # uniform logits, lowest index on ties


def test_head_worked_example():
    ex = json.load(open(os.path.join(GOLD, "softmax_top1_closed_form.json")))["worked_example"]
    x = np.array(ex["logits"], np.float32).reshape(4, 1, 1, 3)
    r = eo.exit_head(x, np.eye(3, dtype=np.float32), None, ex["tau"])
    np.testing.assert_allclose(r["conf"], ex["conf"], rtol=1e-12)
    assert r["exit"].tolist() == ex["exit_mask"] and r["pred"].tolist() == ex["pred"]
    idx, _, _ = eo.compact(r["exit"], x)
    assert idx.tolist() == ex["surv_idx"] and len(idx) == ex["n_surv"]


def test_head_gap_fc_match_torch_and_large_logits_are_stable():
    rng = np.random.default_rng(6)
    x = rng.standard_normal((3, 5, 4, 8)).astype(np.float32)
    wfc = rng.standard_normal((7, 8)).astype(np.float32)
    bfc = rng.standard_normal(7).astype(np.float32)
    r = eo.exit_head(x, wfc, bfc, 0.5)
    gap = F.adaptive_avg_pool2d(torch.from_numpy(x).double().permute(0, 3, 1, 2), 1).flatten(1)
    z = gap @ torch.from_numpy(wfc).double().T + torch.from_numpy(bfc).double()
    p = torch.softmax(z, 1)
    np.testing.assert_allclose(r["gap"], gap.numpy(), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(r["z"], z.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(r["conf"], p.max(1).values.numpy(), rtol=1e-12)
    assert r["pred"].tolist() == p.argmax(1).tolist()
    big = np.zeros((1, 1, 1, 3), np.float32)
    big[0, 0, 0] = [1000.0, 999.0, 0.0]                                # naive exp overflows
    rb = eo.exit_head(big, np.eye(3, dtype=np.float32), None, 0.5)
    assert abs(rb["conf"][0] - 1 / (1 + math.exp(-1.0))) < 1e-12
    # logit shift lands on the named class only; always_exit overrides the threshold
    rs = eo.exit_head(x, wfc, bfc, 0.999, shift=np.array([16, 0, 16], np.float32), shift_cls=np.array([2, 2, 5], np.int32))
    assert rs["pred"].tolist()[0] == 2 and rs["pred"].tolist()[2] == 5 and rs["exit"].tolist() == [1, 0, 1]
    np.testing.assert_allclose(rs["z"][1], r["z"][1])
    assert eo.exit_head(x, wfc, bfc, 2.0, always_exit=True)["exit"].tolist() == [1, 1, 1]


def test_paper_exit_rates_partition_the_samples():
    g = json.load(open(os.path.join(GOLD, "softmax_top1_closed_form.json")))["paper_exit_rates_percent"]
    for k in ("resnet50", "inception_v3"):
        assert abs(sum(g[k]) - 100.0) < 0.06          # every sample leaves at exactly one exit


# ----------------------------------------------------------------------------- compaction / refill

def test_compaction_brute_force_all_masks():
    for B in range(0, 11):
        feat = np.arange(B * 3, dtype=np.float32).reshape(B, 3)
        ids = np.arange(100, 100 + B, dtype=np.int32)
        for bits in itertools.product([0, 1], repeat=B) if B <= 8 else list(itertools.product([0, 1], repeat=B))[::7]:
            m = np.array(bits, np.uint8)
            idx, fo, io = eo.compact(m, feat, ids)
            want = [b for b in range(B) if not bits[b]]
            assert idx.tolist() == want                               # ascending, stable
            assert len(idx) + int(m.sum()) == B                       # exited + surviving = input
            assert len(idx) == int((m == 0).sum())                    # popcount of the not-exit mask
            assert np.array_equal(fo, feat[want]) and io.tolist() == ids[want].tolist()


def test_refill_algorithm1_identities_and_clamp():
    # B_slack = B_max - B_rem, B_incr = min(N_Q, B_slack), B_merged = B_rem + B_incr
    for b_max, b_rem, n_q in [(8, 1, 4), (8, 6, 5), (8, 8, 3), (4, 0, 9), (8, 3, 0)]:
        surv = np.arange(b_rem * 2, dtype=np.float32).reshape(b_rem, 2)
        arr = 100 + np.arange(n_q * 2, dtype=np.float32).reshape(n_q, 2)
        f, ids, n_acc = eo.refill(surv, np.arange(b_rem), arr, 50 + np.arange(n_q), b_max)
        assert n_acc == min(n_q, b_max - b_rem)
        assert len(ids) == b_rem + n_acc <= b_max
        assert ids.tolist() == list(range(b_rem)) + list(range(50, 50 + n_acc))
        assert np.array_equal(f[:b_rem], surv) and np.array_equal(f[b_rem:], arr[:n_acc])


def test_paper_scheduling_timeline_example():
    g = json.load(open(os.path.join(GOLD, "sched_timeline_example.json")))
    ids = np.array(g["active_ids"], np.int32)
    feat = ids.astype(np.float32).reshape(-1, 1)
    _, f_rem, id_rem = eo.compact(np.array(g["active_exit_mask_at_e1"], np.uint8), feat, ids)
    assert len(id_rem) == g["b_rem"]
    new = np.array(g["issued_ids"], np.int32)
    _, f_new, id_new = eo.compact(np.array(g["issued_exit_mask_at_e1"], np.uint8), new.astype(np.float32).reshape(-1, 1), new)
    f, merged, n_acc = eo.refill(f_rem, id_rem, f_new, id_new, g["b_max"])
    assert merged.tolist() == g["merged_ids"] and len(merged) == g["b_merged"]
    assert f.reshape(-1).tolist() == [float(i) for i in g["merged_ids"]]      # features travel with their ids


# ----------------------------------------------------------------------------- whole path

def test_every_sample_exits_once_and_schedules_are_batch_invariant():
    m = wl.tiny_ee_cnn(seed=0)
    x = wl.make_input(m, 8, seed=0)
    serial = [eo.run_sample_serial(m, x[i]) for i in range(8)]
    assert all(0 <= s[0] <= 2 for s in serial)
    assert len({s[0] for s in serial}) > 1, "workload should exercise more than one exit"
    # batched run with a refill at the first boundary: ids 0-4 start, 5-7 catch up and merge
    done = {}
    r0 = eo.run_stage(m, 0, x[:5], np.arange(5, dtype=np.int32))
    for b in np.nonzero(r0["exit"])[0]:
        done[int(b)] = (0, int(r0["pred"][b]))
    c0 = eo.run_stage(m, 0, x[5:], np.arange(5, 8, dtype=np.int32))
    for j in np.nonzero(c0["exit"])[0]:
        done[5 + int(j)] = (0, int(c0["pred"][j]))
    feat, ids, _ = eo.refill(r0["features_out"], r0["ids_out"], c0["features_out"], c0["ids_out"], m.max_batch)
    for s in (1, 2):
        r = eo.run_stage(m, s, feat, ids)
        for j in np.nonzero(r["exit"])[0]:
            assert int(ids[j]) not in done
            done[int(ids[j])] = (s, int(r["pred"][j]))
        feat, ids = r["features_out"], r["ids_out"]
    assert len(ids) == 0 and sorted(done) == list(range(8))
    for i in range(8):
        assert done[i] == serial[i][:2]


def test_activation_scale_stays_order_one():
    m = wl.resnet50_ee(in_hw=64, width0=16, n_classes=20, max_batch=2)
    x = wl.make_input(m, 2, seed=1)
    for s in range(4):
        r = eo.run_stage(m, s, x)
        rms = float(np.sqrt(np.mean(r["stage_out"].astype(np.float64) ** 2)))
        assert 0.1 < rms < 10.0, (s, rms)
        x = r["stage_out"]
    m = wl.mobilenetv2_ee(in_hw=64, n_classes=20, max_batch=2)
    x = wl.make_input(m, 2, seed=2)
    for s in range(4):
        r = eo.run_stage(m, s, x)
        rms = float(np.sqrt(np.mean(r["stage_out"].astype(np.float64) ** 2)))
        assert 0.05 < rms < 10.0, (s, rms)
        x = r["stage_out"]


def _torch_conv(x, l, residual=None):
    """One layer from torch CPU fp64 primitives: conv2d (groups for depthwise), folded-BN scale and bias,
    the residual operand before the activation.  x and the result are NCHW float64 tensors."""
    w = torch.from_numpy(l.weight.astype(np.float64)).permute(0, 3, 1, 2)
    y = F.conv2d(x, w, stride=l.stride, padding=l.pad, groups=l.groups)
    y = y * torch.from_numpy(l.scale.astype(np.float64)).view(1, -1, 1, 1) + torch.from_numpy(l.bias.astype(np.float64)).view(1, -1, 1, 1)
    if residual is not None:
        y = y + residual
    if l.act == wl.ACT_RELU:
        y = torch.relu(y)
    elif l.act == wl.ACT_RELU6:
        y = torch.clamp(y, 0.0, 6.0)
    return y


def _nhwc(t):
    return t.permute(0, 2, 3, 1).numpy()


def test_run_layers_wires_bottlenecks_and_inverted_residuals_like_the_block_definitions():
    """The driver that chains layers (input_from / residual_from / depthwise groups) against the block
    definitions written out by hand with torch fp64 calls: a ResNet bottleneck with a projection shortcut
    (1x1 -> 3x3 stride s -> 1x1, shortcut = strided 1x1 of the BLOCK input), one with an identity shortcut
    (the block input itself), and inverted-residual blocks with (stride 1, Cin == Cout) and without a
    residual connection.  A wrong source for an input or a residual operand changes the result by O(1)."""
    # ---- two chained bottlenecks: projection (stride 2), then identity
    rng = wl._rng(7, 950)
    layers = []
    last = wl._bottleneck(rng, layers, 16, 8, 2, True, False, wl.FROM_STAGE_INPUT)
    last = wl._bottleneck(rng, layers, 32, 8, 1, False, False, last)
    assert len(layers) == 7 and last == 6
    fw, fb = wl._head(rng, 32, 5, 1.0, False)
    m = wl.Model("blocks", "f32", 9, 9, 16, [wl.Stage(layers, 5, fw, fb, 2.0, False)], 2)
    x_np = wl.random_features((2, 9, 9, 16), seed=5, bf16=False, relu=False)
    outs = eo.run_layers(m, 0, x_np, keep_all=True)
    x = torch.from_numpy(x_np.astype(np.float64)).permute(0, 3, 1, 2)
    a1 = _torch_conv(x, layers[0])                      # 1x1 reduce of the block input
    a2 = _torch_conv(a1, layers[1])                     # 3x3, stride 2
    sc = _torch_conv(x, layers[2])                      # projection shortcut: strided 1x1 of the block input
    a3 = _torch_conv(a2, layers[3], residual=sc)        # 1x1 expand + shortcut, then ReLU
    b1 = _torch_conv(a3, layers[4])
    b2 = _torch_conv(b1, layers[5])
    b3 = _torch_conv(b2, layers[6], residual=a3)        # identity shortcut: the block input itself
    for got, want in zip(outs, (a1, a2, sc, a3, b1, b2, b3)):
        want = _nhwc(want)
        assert got.shape == want.shape
        assert np.max(np.abs(got - want)) <= 2e-6 * max(1.0, float(np.max(np.abs(want))))
    # the check has teeth: the same block with its shortcut taken from the wrong tensor is far away
    assert float(np.max(np.abs(_nhwc(b3) - _nhwc(_torch_conv(b2, layers[6], residual=sc))))) > 0.1
    # ---- inverted-residual blocks as the MobileNetV2-shaped builder lays them out: stem, t=1 block (no expand,
    # no residual: 32 -> 16), t=6 stride-2 block (no residual), t=6 stride-1 block with Cin == Cout (residual)
    mv = wl.mobilenetv2_ee(seed=2, in_hw=32, n_classes=10, max_batch=2, dtype="f32")
    st = mv.stages[0]
    L = st.layers
    assert [l.op for l in L[:9]] == [wl.OP_CONV, wl.OP_DWCONV, wl.OP_CONV, wl.OP_CONV, wl.OP_DWCONV, wl.OP_CONV,
                                     wl.OP_CONV, wl.OP_DWCONV, wl.OP_CONV]
    x_np = wl.make_input(mv, 2, seed=6)
    outs = eo.run_layers(mv, 0, x_np, keep_all=True)
    x = torch.from_numpy(x_np.astype(np.float64)).permute(0, 3, 1, 2)
    s0 = _torch_conv(x, L[0])                           # stem 3x3 s2
    d1 = _torch_conv(s0, L[1])                          # block 1 (t = 1): depthwise straight on the block input
    p1 = _torch_conv(d1, L[2])                          # linear projection 32 -> 16, no residual (Cin != Cout)
    e2 = _torch_conv(p1, L[3])                          # block 2: expand
    d2 = _torch_conv(e2, L[4])                          # depthwise stride 2
    p2 = _torch_conv(d2, L[5])                          # projection, no residual (stride 2)
    e3 = _torch_conv(p2, L[6])                          # block 3: expand
    d3 = _torch_conv(e3, L[7])                          # depthwise stride 1
    p3 = _torch_conv(d3, L[8], residual=p2)             # projection + the block input (stride 1, 24 -> 24)
    assert L[8].residual_from != wl.NO_RESIDUAL and L[5].residual_from == wl.NO_RESIDUAL and L[2].residual_from == wl.NO_RESIDUAL
    for got, want in zip(outs[:9], (s0, d1, p1, e2, d2, p2, e3, d3, p3)):
        want = _nhwc(want)
        assert got.shape == want.shape
        assert np.max(np.abs(got - want)) <= 2e-6 * max(1.0, float(np.max(np.abs(want))))
    # the stage output is the last layer's; run_layers without keep_all returns exactly it
    assert np.array_equal(eo.run_layers(mv, 0, x_np), outs[st.out_layer])


def _run_layers_fp32_accumulator(model, stage, x):
    """The stage's layers with the SAME arithmetic as the oracle except that every accumulator is rounded to fp32
    once before an fp32 epilogue (what any fp32-accumulating implementation does at best): a second correct
    implementation, built from the oracle's raw convolution sums and numpy."""
    st = model.stages[stage]
    outs = []
    x = np.ascontiguousarray(x, dtype=np.float32)
    for i, l in enumerate(st.layers):
        src = x if (l.input_from == wl.FROM_STAGE_INPUT or (l.input_from == wl.FROM_PREV and i == 0)) else \
            (outs[i - 1] if l.input_from == wl.FROM_PREV else outs[l.input_from])
        if l.op == wl.OP_MAXPOOL:
            outs.append(eo.maxpool(src, l.kh, l.stride, l.pad))
            continue
        res = x if l.residual_from == wl.FROM_STAGE_INPUT else (outs[l.residual_from] if l.residual_from >= 0 else None)
        y = eo.conv2d(src, l.weight, l.stride, l.pad, l.groups) * l.scale.astype(np.float32) + l.bias.astype(np.float32)
        if res is not None:
            y = y + res
        y = np.maximum(y, 0) if l.act == wl.ACT_RELU else (np.clip(y, 0, 6) if l.act == wl.ACT_RELU6 else y)
        outs.append(wl.to_bf16_grid(y.astype(np.float32)))
    return outs[st.out_layer]


@pytest.mark.parametrize("name", ["resnet50", "mobilenetv2"])
def test_bf16_chain_drift_between_two_correct_cpu_implementations(name):
    """Why whole bf16 stages are not held element-wise to 1e-2: two CPU implementations of the benchmark's stages
    that differ only by one fp32 rounding of each accumulator agree on most elements bit for bit, yet a measurable
    share of the elements ends up more than 1e-2 apart (each flipped bf16 rounding perturbs everything downstream),
    while the max-norm stays within two bf16 ulps and the L2 error between 1e-3 and 6e-3.  The stage bars of the GPU parity tests
    (tests/util.py: STAGE_TOL, STAGE_L2, STAGE_EXCEED) must admit this pair, and the drift must be real (otherwise the
    element-wise bar could be asked of whole stages)."""
    from tests import util

    spec = wl.resnet50_ee(seed=1, max_batch=2) if name == "resnet50" else wl.mobilenetv2_ee(seed=2, max_batch=2)
    x = wl.make_input(spec, 2, seed=1)
    worst_share = 0.0
    for s in range(4):
        a = eo.run_layers(spec, s, x)
        b = _run_layers_fp32_accumulator(spec, s, x)
        share = util.exceed_share(b, a, util.TOL["bf16"], util.STAGE_FLOOR)
        worst_share = max(worst_share, share)
        assert util.norm_err(b, a) <= util.STAGE_TOL["bf16"]
        assert util.l2_err(b, a) <= util.STAGE_L2["bf16"]
        assert share <= util.STAGE_EXCEED
        assert float(np.mean(a != b)) > 1e-3                 # the two do part ways
        x = a
    assert worst_share > 1e-2                                # ... by more than the element-wise bar, for whole percents of a stage


def test_serve_trace_bookkeeping():
    n, bmax = 200, 8
    arr = wl.poisson_arrivals(3, n, 1000.0)
    rng = np.random.default_rng(0)
    exit_of = rng.integers(0, 4, n)
    fin, launches = eo.serve_trace(4, bmax, arr, exit_of, lambda s, b: 1e-3 + 1e-4 * b)
    assert np.all(fin > arr)                                         # nobody finishes before arriving
    seen = {}
    for stage, ids in launches:
        assert 1 <= len(ids) <= bmax
        for r in ids:
            assert seen.get(r, -1) == stage - 1                      # stages visited in order, once
            seen[r] = stage
    assert all(seen[r] == exit_of[r] for r in range(n))              # every request leaves at its exit


# ----------------------------------------------------------------------------- SLO-aware preemption criterion (Eq. 3-4)

def test_slo_criterion_worked_example():
    """Hand-computed from Eq. 3-4.  Three subnets of 1 time unit each at any batch, B_max = 4; request 0 arrives at
    t = 0, request 1 at t = 0.5, both leave at the last exit.  At the first preemption point (t = 1) one request is
    queued: T_slack = T_SLO - 1, T_overhead = T_{0:0}(1) + T_{1:2}(2) = 3, so the batch is preempted iff T_SLO > 4.
    T_SLO = 4.5: request 1 catches up (t = 2), the merged pair finishes at t = 4.
    T_SLO = 4 (3 < 3 is false: strict inequality): request 0 runs on; at the second point (t = 2) T_slack = 2,
    T_overhead = T_{0:1}(1) + T_{2:2}(2) = 3: declined again; request 0 finishes at 3, request 1 runs alone, done at 6."""
    arr = np.array([0.0, 0.5])
    exit_of = np.array([2, 2])
    unit = lambda s, b: 1.0   # noqa: E731
    fin, launches = eo.serve_trace(3, 4, arr, exit_of, unit, slo=4.5)
    assert launches == [(0, (0,)), (0, (1,)), (1, (0, 1)), (2, (0, 1))] and fin.tolist() == [4.0, 4.0]
    fin, launches = eo.serve_trace(3, 4, arr, exit_of, unit, slo=4.0)
    assert launches == [(0, (0,)), (1, (0,)), (2, (0,)), (0, (1,)), (1, (1,)), (2, (1,))] and fin.tolist() == [3.0, 6.0]
    # a subnet that takes `batch` time units tells the two batch sizes of Eq. 4 apart: at t = 1,
    # T_overhead = T_{0:0}(B_incr = 1) + T_{1:2}(B_merged = 2) = 1 + 4 = 5 and T_slack = T_SLO - 1: preempt iff T_SLO > 6
    by_batch = lambda s, b: float(b)   # noqa: E731
    fin, launches = eo.serve_trace(3, 4, arr, exit_of, by_batch, slo=6.5)
    assert launches == [(0, (0,)), (0, (1,)), (1, (0, 1)), (2, (0, 1))] and fin.tolist() == [6.0, 6.0]
    fin, launches = eo.serve_trace(3, 4, arr, exit_of, by_batch, slo=5.0)   # second point: slack 3 against 2 + 2: declined
    assert launches == [(0, (0,)), (1, (0,)), (2, (0,)), (0, (1,)), (1, (1,)), (2, (1,))] and fin.tolist() == [3.0, 6.0]


def _random_trace(seed, n=300, rate=1500.0, n_stages=4):
    arr = wl.poisson_arrivals(seed, n, rate)
    exit_of = np.random.default_rng(seed).integers(0, n_stages, n)
    return arr, exit_of


def test_slo_infinite_is_plain_backfilling_and_zero_never_preempts():
    st = lambda s, b: 2e-4 * (s + 1) + 3e-5 * b   # noqa: E731
    arr, exit_of = _random_trace(11)
    ref = eo.serve_trace(4, 8, arr, exit_of, st)
    big = eo.serve_trace(4, 8, arr, exit_of, st, slo=1e9)
    assert ref[1] == big[1] and np.array_equal(ref[0], big[0])
    # T_SLO = 0: the slack of a non-empty active batch is never positive, so a batch with survivors is never preempted:
    # between two consecutive subnets of a surviving batch nothing else is launched
    _, launches = eo.serve_trace(4, 8, arr, exit_of, st, slo=0.0)
    for (s0, ids0), (s1, ids1) in zip(launches, launches[1:]):
        rem = [r for r in ids0 if exit_of[r] != s0]
        if rem:
            assert s1 == s0 + 1 and list(ids1) == rem


@pytest.mark.parametrize("slo", [4e-3, 8e-3, 16e-3])
def test_slo_criterion_never_pushes_a_preempted_sample_past_its_slo(slo):
    """The overhead estimate is an upper bound when a subnet is not slower at a smaller batch (Section III-B): a sample
    whose batch was preempted (something ran between two of its consecutive subnets) still meets the SLO."""
    st = lambda s, b: 2e-4 * (s + 1) + 3e-5 * b   # noqa: E731
    checked = 0
    for seed in (1, 2, 3):
        arr, exit_of = _random_trace(seed)
        fin, launches = eo.serve_trace(4, 8, arr, exit_of, st, slo=slo)
        last = {}                                   # request -> index of its latest launch
        preempted = set()
        for k, (s, ids) in enumerate(launches):
            for r in ids:
                if s > 0 and last[r] != k - 1:
                    preempted.add(r)
                last[r] = k
        assert all(exit_of[r] == launches[last[r]][0] for r in range(len(arr)))
        for r in preempted:
            assert fin[r] - arr[r] <= slo + 1e-12, (seed, r, fin[r] - arr[r])
        checked += len(preempted)
    assert checked > 20                              # the traces do exercise preemptions at these SLOs
