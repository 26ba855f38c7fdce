"""Parity of the CUDA library (through its C ABI) against the CPU oracle, element by element,
on seeded inputs small enough for the oracle to finish in seconds yet spanning several tiles
and ragged tails.  Every stage is fed the ORACLE's stage input (stage-local parity)."""
import itertools

import numpy as np
import pytest
import torch

from oracle import ee_oracle as eo
from paper_2209_13443_b200 import binding as eb
from paper_2209_13443_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


# ----------------------------------------------------------------------------- config 1

@pytest.mark.parametrize("B", [1, 2, 3, 5, 7, 8])
def test_tiny_fp32_stagewise(B):
    spec = wl.tiny_ee_cnn(seed=0)
    run = util.GpuRunner(spec)
    x = wl.make_input(spec, B, seed=0)
    ids = 100 + np.arange(B, dtype=np.int32)
    exited = 0
    for s in range(3):
        o = util.oracle_stage(spec, s, x, ids)
        g = run.stage(s, x, ids)
        util.check_stage(spec, g, o, f"tiny B={B} stage {s}")
        exited += int(o["exit"].sum())
        x, ids = o["features_out"], o["ids_out"]
        if len(ids) == 0:
            break
    assert exited == B                                              # every sample leaves exactly once


def test_tiny_end_to_end_schedule_reproduces_serial_reference():
    """GPU-only chain with a refill at the first boundary; per id the exit and prediction must be
    those of the sample run alone through the oracle (samples finish out of order, matched by id)."""
    spec = wl.tiny_ee_cnn(seed=0)
    run = util.GpuRunner(spec)
    m = run.m
    x = wl.make_input(spec, 8, seed=0)
    serial = [eo.run_sample_serial(spec, x[i]) for i in range(8)]
    near = [i for i in range(8) if any(abs(c - 0.6) < util.BAND for c in serial[i][2][:2])]
    done = {}

    def harvest(s, ids_np, B):
        out = run.bufs[s]
        mask = out.exit_mask[:B].cpu().numpy()
        pred = out.pred[:B].cpu().numpy()
        for j in np.nonzero(mask)[0]:
            assert int(ids_np[j]) not in done
            done[int(ids_np[j])] = (s, int(pred[j]))

    xd = eb.to_device("f32", x)
    ids_a = torch.arange(0, 5, dtype=torch.int32, device="cuda")
    ids_b = torch.arange(5, 8, dtype=torch.int32, device="cuda")
    # active batch {0..4} to exit 0, parked in `park`
    m.stage_run(0, xd[:5], 5, run.bufs[0], run.ws, ids_a)
    torch.cuda.synchronize()
    harvest(0, ids_a.cpu().numpy(), 5)
    n_rem = int(run.bufs[0].n_surv_host[0])
    park = run.bufs[0].features_out.clone()
    park_ids = run.bufs[0].ids_out.clone()
    # catch-up batch {5,6,7} to exit 0, then merged behind the parked survivors
    m.stage_run(0, xd[5:], 3, run.bufs[0], run.ws, ids_b)
    torch.cuda.synchronize()
    harvest(0, ids_b.cpu().numpy(), 3)
    n_new = int(run.bufs[0].n_surv_host[0])
    n_acc, n_mer = m.batch_refill(1, park, park_ids, n_rem, run.bufs[0].features_out, run.bufs[0].ids_out, n_new)
    assert n_acc == min(n_new, spec.max_batch - n_rem) and n_mer == n_rem + n_acc
    feat, ids, n = park, park_ids, n_mer
    for s in (1, 2):
        if n == 0:
            break
        m.stage_run(s, feat, n, run.bufs[s], run.ws, ids)
        torch.cuda.synchronize()
        harvest(s, ids[:n].cpu().numpy(), n)
        feat, ids, n = run.bufs[s].features_out, run.bufs[s].ids_out, int(run.bufs[s].n_surv_host[0])
    assert n == 0 and sorted(done) == list(range(8))
    for i in range(8):
        if i not in near:
            assert done[i] == serial[i][:2], (i, done[i], serial[i])


# ----------------------------------------------------------------------------- single layers

GEOMS = [
    # H, W, cin, cout, k, stride, pad, act, residual
    (9, 7, 3, 5, 3, 1, 1, wl.ACT_RELU, False),          # odd sizes, ragged M and N
    (13, 11, 3, 64, 7, 2, 3, wl.ACT_RELU, False),       # stem-like
    (8, 8, 16, 24, 1, 1, 0, wl.ACT_NONE, True),         # pointwise + residual, linear
    (10, 6, 24, 32, 3, 2, 1, wl.ACT_RELU6, False),
    (7, 7, 64, 64, 3, 1, 1, wl.ACT_RELU, True),
    (14, 14, 64, 256, 1, 1, 0, wl.ACT_RELU, True),
    (15, 9, 64, 128, 1, 2, 0, wl.ACT_NONE, False),      # strided projection, odd input
    (12, 12, 128, 128, 3, 2, 1, wl.ACT_RELU, False),
    (6, 6, 320, 96, 1, 1, 0, wl.ACT_NONE, False),
    (5, 5, 136, 72, 3, 1, 1, wl.ACT_RELU, False),       # K and N not multiples of 64
    (11, 9, 3, 32, 3, 2, 1, wl.ACT_RELU6, False),       # 3x3 stem on 3 channels, stride 2, odd image
    (8, 8, 3, 16, 3, 1, 1, wl.ACT_NONE, False),         # the same, stride 1
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("geom", GEOMS)
def test_conv_layer(dtype, geom):
    H, W, cin, cout, k, stride, pad, act, residual = geom
    spec = util.single_layer_model(dtype, H, W, cin, cout, k, stride, pad, act, residual, seed=hash(geom) % 1000, max_batch=5)
    run = util.GpuRunner(spec)
    for B in (1, 5):
        x = wl.random_features((B, H, W, cin), seed=B, bf16=dtype == "bf16", relu=False)
        o = util.oracle_stage(spec, 0, x)
        g = run.stage(0, x)
        r = util.check_stage(spec, g, o, f"{dtype} {geom} B={B}", elementwise=True)
        assert g["n_surv"] == B


# 3x3 / 64-channel bf16 layers, which the halo-block kernel takes: one tile per image, several tiles per image with a
# ragged last one, a tile of one image row, the benchmark's 56x56 map, fewer than 64 filters, a one-pixel-wide image
HALO_GEOMS = [
    (7, 7, 64, 64, wl.ACT_RELU),
    (23, 19, 64, 64, wl.ACT_RELU),
    (5, 61, 64, 40, wl.ACT_NONE),
    (56, 56, 64, 64, wl.ACT_RELU),
    (3, 1, 64, 8, wl.ACT_RELU6),
]


# narrow 1x1 layers, which run with g pixels per row (g * Cin <= 64, g divides H * W): g = 4 and 2 with full 64-column
# rows, g = 3 (48 columns: ragged K block), g = 1 because nothing divides, 8 channels (g = 7 of 49 pixels), with and
# without a residual operand
GROUP_GEOMS = [
    (8, 8, 16, 96, wl.ACT_RELU6, False),
    (6, 10, 32, 16, wl.ACT_NONE, True),
    (5, 3, 16, 24, wl.ACT_RELU, True),
    (7, 7, 24, 144, wl.ACT_RELU6, False),
    (7, 7, 8, 40, wl.ACT_RELU, False),
]


@pytest.mark.parametrize("geom", GROUP_GEOMS)
def test_narrow_pointwise_layer(geom):
    H, W, cin, cout, act, residual = geom
    spec = util.single_layer_model("bf16", H, W, cin, cout, 1, 1, 0, act, residual, seed=hash(geom) % 1000, max_batch=5)
    run = util.GpuRunner(spec)
    for B in (1, 5):
        x = wl.random_features((B, H, W, cin), seed=B, bf16=True, relu=False)
        o = util.oracle_stage(spec, 0, x)
        g = run.stage(0, x)
        util.check_stage(spec, g, o, f"narrow 1x1 {geom} B={B}", elementwise=True)
        assert g["n_surv"] == B


# layers forced onto the CTA-pair kernel (variant 1: 256 x 256 tiles, 2: 256 x 128 tiles) with a forced number of K ranges:
# 1x1 and 3x3, stride 1 and 2, with and without residual, M tails (a pair whose second CTA has no valid row: 7x7 maps at
# B = 1), N tails (200 and 136 columns), a K tail (136 channels), split-K through global memory with 2, 3 and 5 ranges
PAIR_GEOMS = [
    # H, W, cin, cout, k, stride, pad, act, residual, variant, splits
    (14, 14, 256, 256, 1, 1, 0, wl.ACT_RELU, False, 1, 1),
    (14, 14, 1024, 256, 1, 1, 0, wl.ACT_RELU, False, 1, 3),
    (14, 14, 256, 1024, 1, 1, 0, wl.ACT_RELU, True, 1, 1),
    (14, 14, 256, 256, 3, 1, 1, wl.ACT_RELU, False, 1, 3),
    (28, 28, 128, 128, 3, 2, 1, wl.ACT_RELU, False, 2, 2),
    (7, 7, 512, 2048, 1, 1, 0, wl.ACT_RELU, True, 1, 2),
    (7, 7, 2048, 512, 1, 1, 0, wl.ACT_RELU, False, 1, 5),
    (14, 14, 512, 512, 3, 2, 1, wl.ACT_NONE, False, 1, 3),
    (9, 7, 136, 200, 3, 1, 1, wl.ACT_RELU6, False, 1, 2),
    (9, 7, 136, 200, 1, 1, 0, wl.ACT_RELU6, True, 2, 1),
    (13, 11, 64, 136, 3, 1, 1, wl.ACT_RELU, False, 2, 3),
    (15, 9, 64, 256, 1, 2, 0, wl.ACT_NONE, False, 1, 1),
]


@pytest.mark.parametrize("geom", PAIR_GEOMS)
def test_pair_kernel_layer(geom):
    H, W, cin, cout, k, stride, pad, act, residual, variant, splits = geom
    max_batch = 11
    spec = util.single_layer_model("bf16", H, W, cin, cout, k, stride, pad, act, residual, seed=hash(geom) % 1000, max_batch=max_batch)
    layer = 1 if residual else 0

    def configure(m):
        m.set_layer_splits(0, layer, splits)
        m.set_layer_variant(0, layer, 1, max_batch, variant)
        assert m.layer_config(0, layer, 3) == {"variant": variant, "splits": splits, "tensor_core": 3 if cout > 128 else 2}

    m = eb.EEModel(spec)
    configure(m)
    ws, ws_guard = util.guarded((m.query(0)["workspace_bytes"],), torch.uint8)
    for B in (1, 5, 11):
        x = wl.random_features((B, H, W, cin), seed=B, bf16=True, relu=False)
        outs = eo.run_layers(spec, 0, x, keep_all=True)        # the layer runs alone on the oracle's input and residual operand
        res = eb.to_device("bf16", outs[0]) if residual else None
        for rep in range(2):                                   # twice: the split-K counters must be back at zero
            out, guard = util.guarded(outs[layer].shape, torch.bfloat16)
            m.layer_run(0, layer, eb.to_device("bf16", x), res, B, out, ws)
            torch.cuda.synchronize()
            m.check()
            assert bool(torch.all(guard == util.CANARY)) and bool(torch.all(ws_guard == util.CANARY))
            e = util.rel_err(out.float().cpu().numpy(), outs[layer], "bf16")
            assert e <= util.TOL["bf16"], f"pair {geom} B={B} run {rep}: {e:.3e}"


RANGE_GEOMS = [
    # H, W, cin, cout, k, stride, pad, act, residual, K ranges
    (14, 14, 256, 256, 3, 1, 1, wl.ACT_RELU, False, 4),
    (14, 14, 256, 256, 3, 1, 1, wl.ACT_RELU, False, 3),
    (14, 14, 1024, 256, 1, 1, 0, wl.ACT_RELU, False, 4),
    (14, 14, 512, 512, 3, 2, 1, wl.ACT_RELU, False, 2),
    (7, 7, 512, 2048, 1, 1, 0, wl.ACT_RELU, True, 2),
    (7, 7, 2048, 512, 1, 1, 0, wl.ACT_NONE, False, 4),
    (28, 28, 256, 64, 3, 1, 1, wl.ACT_RELU6, False, 8),     # 64-wide tiles: eight accumulators of 64 columns
    (14, 14, 136, 72, 3, 1, 1, wl.ACT_RELU, False, 3),      # ragged channels and filters
]


@pytest.mark.parametrize("geom", RANGE_GEOMS)
def test_k_ranges_in_one_cta_give_the_bits_of_the_cluster_of_ctas(geom):
    """A layer's K ranges run as a cluster of CTAs per tile or, one accumulator per range, inside ONE CTA per tile: the
    choice may change with the batch (table variants 3 and 4; by default the cluster while the grid fits one wave), the
    bits may not.  Both against the oracle, and against each other bit for bit, at batches on both sides of the default
    switch-over."""
    H, W, cin, cout, k, stride, pad, act, residual, ranges = geom
    max_batch = 40
    spec = util.single_layer_model("bf16", H, W, cin, cout, k, stride, pad, act, residual, seed=hash(geom) % 1000, max_batch=max_batch)
    layer = 1 if residual else 0
    m = eb.EEModel(spec)
    m.set_layer_splits(0, layer, ranges)
    ws, ws_guard = util.guarded((m.query(0)["workspace_bytes"],), torch.uint8)
    for B in (1, 6, 40):
        x = wl.random_features((B, H, W, cin), seed=B, bf16=True, relu=False)
        outs = eo.run_layers(spec, 0, x, keep_all=True)
        res = eb.to_device("bf16", outs[0]) if residual else None
        got = {}
        for variant in (3, 4, 0, 4):
            m.set_layer_variant(0, layer, 1, max_batch, variant)
            out, guard = util.guarded(outs[layer].shape, torch.bfloat16)
            m.layer_run(0, layer, eb.to_device("bf16", x), res, B, out, ws)
            torch.cuda.synchronize()
            m.check()
            assert bool(torch.all(guard == util.CANARY)) and bool(torch.all(ws_guard == util.CANARY))
            if variant in got:
                assert torch.equal(out, got[variant])
            got[variant] = out.clone()
        assert torch.equal(got[3], got[4]) and torch.equal(got[0], got[3]), f"{geom} B={B}"
        e = util.rel_err(got[4].float().cpu().numpy(), outs[layer], "bf16")
        assert e <= util.TOL["bf16"], f"{geom} B={B}: {e:.3e}"


@pytest.mark.parametrize("geom", HALO_GEOMS)
def test_conv3x3_halo_layer(geom):
    H, W, cin, cout, act = geom
    spec = util.single_layer_model("bf16", H, W, cin, cout, 3, 1, 1, act, False, seed=hash(geom) % 1000, max_batch=5)
    run = util.GpuRunner(spec)
    for B in (1, 5):
        x = wl.random_features((B, H, W, cin), seed=B, bf16=True, relu=False)
        o = util.oracle_stage(spec, 0, x)
        g = run.stage(0, x)
        util.check_stage(spec, g, o, f"halo {geom} B={B}", elementwise=True)
        assert g["n_surv"] == B


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("C,stride,H,W", [(32, 1, 9, 9), (96, 2, 10, 7), (144, 1, 6, 6), (12, 2, 8, 8)])
def test_depthwise_layer(dtype, C, stride, H, W):
    spec = util.single_layer_model(dtype, H, W, C, C, 3, stride, 1, wl.ACT_RELU6, False, seed=C, op=wl.OP_DWCONV)
    run = util.GpuRunner(spec)
    x = wl.random_features((3, H, W, C), seed=3, bf16=dtype == "bf16", relu=False)
    util.check_stage(spec, run.stage(0, x), util.oracle_stage(spec, 0, x), f"dw {dtype} C={C}", elementwise=True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_maxpool_layer(dtype):
    rng = wl._rng(5, 901)
    bf16 = dtype == "bf16"
    layers = [wl.Layer(wl.OP_MAXPOOL, 16, 16, 3, 3, 2, 1)]
    fw, fb = wl._head(rng, 16, 5, 1.0, bf16)
    spec = wl.Model("pool", dtype, 11, 9, 16, [wl.Stage(layers, 5, fw, fb, 2.0, False)], 3)
    run = util.GpuRunner(spec)
    x = -np.abs(wl.random_features((3, 11, 9, 16), seed=4, bf16=bf16)) - 1.0    # zero padding would win if it took part
    x = wl.to_bf16_grid(x) if bf16 else x
    o = util.oracle_stage(spec, 0, x)
    g = run.stage(0, x)
    assert np.array_equal(g["features_out"], o["features_out"])


# filters that are not square, padded along their own axis (the factorised convolutions of Inception-style towers)
ASYM_GEOMS = [
    # H, W, cin, cout, kh, kw, stride, pad_h, pad_w, act, variant
    (17, 17, 96, 96, 1, 7, 1, 0, 3, wl.ACT_RELU, 0),
    (17, 17, 96, 96, 7, 1, 1, 3, 0, wl.ACT_RELU, 0),
    (13, 9, 24, 40, 3, 5, 2, 1, 2, wl.ACT_RELU6, 0),
    (9, 12, 16, 32, 1, 3, 1, 0, 0, wl.ACT_NONE, 0),          # no padding: the map shrinks along one axis only
    (17, 17, 192, 192, 1, 7, 1, 0, 3, wl.ACT_RELU, 1),        # the same on the CTA-pair kernel
    (17, 17, 192, 192, 7, 1, 1, 3, 0, wl.ACT_RELU, 2),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("geom", ASYM_GEOMS)
def test_conv_layer_with_a_filter_that_is_not_square(dtype, geom):
    H, W, cin, cout, kh, kw, stride, ph, pw, act, variant = geom
    if dtype == "f32" and variant:
        pytest.skip("the CTA-pair kernel is a bf16 kernel")
    bf16 = dtype == "bf16"
    rng = wl._rng(hash(geom) % 1000, 904)
    layer = wl._conv_hw(rng, cin, cout, kh, kw, stride, ph, pw, act, bf16=bf16)
    fw, fb = wl._head(rng, cout, 7, 1.0, bf16)
    spec = wl.Model("asym", dtype, H, W, cin, [wl.Stage([layer], 7, fw, fb, 2.0, False)], 5)

    def configure(m):
        if variant:
            m.set_layer_splits(0, 0, 2)
            m.set_layer_variant(0, 0, 1, 5, variant)

    run = util.GpuRunner(spec, configure)
    for B in (1, 5):
        x = wl.random_features((B, H, W, cin), seed=B, bf16=bf16, relu=False)
        o = util.oracle_stage(spec, 0, x)
        g = run.stage(0, x)
        assert g["features_out"].shape == o["features_out"].shape
        util.check_stage(spec, g, o, f"{dtype} {geom} B={B}", elementwise=True)


@pytest.mark.parametrize("B", [1, 4])
def test_factorised_tower_shaped_small(B):
    spec = wl.factorised_tower_ee(seed=5, in_hw=36, width=64, n_classes=50, max_batch=4)
    _stagewise(spec, B, seed=5)


# ----------------------------------------------------------------------------- configs 2-3 at reduced size

def _stagewise(spec, B, seed, tol=None):
    run = util.GpuRunner(spec)
    x = wl.make_input(spec, B, seed=seed)
    ids = np.arange(B, dtype=np.int32)
    stats = []
    for s in range(len(spec.stages)):
        o = util.oracle_stage(spec, s, x, ids)
        g = run.stage(s, x, ids)
        stats.append(util.check_stage(spec, g, o, f"{spec.name} B={B} stage {s}", tol))
        # next stage is fed ALL samples' oracle output (not only survivors) to keep every stage busy
        x = o["stage_out"]
    return stats


@pytest.mark.parametrize("B", [1, 6])
def test_resnet50_shaped_small(B):
    spec = wl.resnet50_ee(seed=1, in_hw=64, n_classes=100, max_batch=6)
    _stagewise(spec, B, seed=1)


@pytest.mark.parametrize("B", [1, 5])
def test_mobilenetv2_shaped_small(B):
    spec = wl.mobilenetv2_ee(seed=2, in_hw=64, n_classes=100, max_batch=5)
    _stagewise(spec, B, seed=2)


# ----------------------------------------------------------------------------- head, compaction, refill

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,HW,C,K", [(1, 1, 8, 3), (5, 49, 64, 10), (64, 196, 256, 1000), (33, 50, 40, 17), (7, 3136, 32, 100),
                                     (3, 7, 2048, 1000), (4, 9, 6, 5)])
def test_exit_head_alone(dtype, B, HW, C, K):
    bf16 = dtype == "bf16"
    rng = wl._rng(B * 1000 + C, 902)
    fw, fb = wl._head(rng, C, K, 8.0, bf16)
    layers = [wl._conv(rng, wl.OP_CONV, C, C, 1, 1, 0, wl.ACT_NONE, bf16=bf16)]
    spec = wl.Model("head", dtype, 1, HW, C, [wl.Stage(layers, K, fw, fb, 0.5, False)], max(B, 1))
    m = eb.EEModel(spec)
    out = eb.StageBuffers(m, 0)
    scratch = torch.empty(m.exit_head_scratch_bytes(0) + 256, dtype=torch.uint8, device="cuda")
    x = wl.random_features((B, HW, C), seed=HW, bf16=bf16)
    shift = (np.arange(B) % 3 == 0).astype(np.float32) * 9.0
    cls = (np.arange(B) * 5 % K).astype(np.int32)
    m.exit_head(0, eb.to_device(dtype, x), B, HW, out, scratch, torch.as_tensor(shift, device="cuda"), torch.as_tensor(cls, device="cuda"))
    torch.cuda.synchronize()
    o = eo.exit_head(x, fw, fb, 0.5, False, shift, cls)
    g = {"z": out.logits[:B].cpu().numpy(), "conf": out.conf[:B].cpu().numpy(), "pred": out.pred[:B].cpu().numpy(),
         "exit": out.exit_mask[:B].cpu().numpy()}
    n = int(out.n_surv_dev.cpu()[0])
    assert util.rel_err(g["z"], o["z"], dtype, floor=util.LOGIT_FLOOR[dtype]) <= (2e-3 if bf16 else 1e-5)
    band = np.abs(o["conf"] - 0.5) < util.BAND
    assert np.array_equal(g["exit"][~band], o["exit"][~band])
    assert np.array_equal(out.survivor_idx[:n].cpu().numpy(), np.nonzero(g["exit"] == 0)[0])
    # a second call on the same scratch must give bit-identical results (scratch is re-initialised by the call)
    z1 = out.logits[:B].clone()
    m.exit_head(0, eb.to_device(dtype, x), B, HW, out, scratch, torch.as_tensor(shift, device="cuda"), torch.as_tensor(cls, device="cuda"))
    torch.cuda.synchronize()
    assert torch.equal(z1, out.logits[:B])


@pytest.mark.parametrize("B,HW,C,K", [(27, 49, 2048, 1000), (5, 3136, 256, 1000), (37, 196, 1024, 1000), (7, 9, 72, 33), (1, 4, 8, 3),
                                     (19, 16, 1280, 1000), (40, 25, 320, 10), (64, 49, 512, 1024), (18, 1, 264, 129)])
def test_one_launch_head_against_the_two_kernel_head_and_the_oracle(B, HW, C, K):
    """The cluster kernel (pool + FC + decision + scan in one launch; an option) and the pooling + FC kernels on the same inputs:
    logits within fp32 rounding of each other and within the bf16 bar of the oracle, the same predictions and exit
    decisions away from the threshold, a survivor list consistent with the decisions; each sample alone in a batch of
    one gives the same bits as inside the batch (tile heights 1, 2 and 4 are all crossed by the batch sizes)."""
    rng = wl._rng(B * 1000 + C, 905)
    fw, fb = wl._head(rng, C, K, 8.0, True)
    layers = [wl._conv(rng, wl.OP_CONV, C, C, 1, 1, 0, wl.ACT_NONE, bf16=True)]
    spec = wl.Model("head", "bf16", 1, HW, C, [wl.Stage(layers, K, fw, fb, 0.5, False)], B)
    m = eb.EEModel(spec)
    out = eb.StageBuffers(m, 0)
    scratch = torch.empty(m.exit_head_scratch_bytes(0) + 256, dtype=torch.uint8, device="cuda")
    x = wl.random_features((B, HW, C), seed=HW + 1, bf16=True)
    shift = (np.arange(B) % 3 == 0).astype(np.float32) * 9.0
    cls = (np.arange(B) * 5 % K).astype(np.int32)
    xd, sd, cd = eb.to_device("bf16", x), torch.as_tensor(shift, device="cuda"), torch.as_tensor(cls, device="cuda")
    got = {}
    for fused in (True, False, True):            # the last run: the arrival counter of the first must be back at zero
        m.set_fused_head(fused)
        assert m.head_launches(0) == (1 if fused else 2)
        out.logits.fill_(float("nan"))
        out.n_surv_dev.fill_(-1)
        m.exit_head(0, xd, B, HW, out, scratch, sd, cd)
        torch.cuda.synchronize()
        n = int(out.n_surv_dev.cpu()[0])
        got[fused] = {"z": out.logits[:B].cpu().numpy(), "conf": out.conf[:B].cpu().numpy(), "pred": out.pred[:B].cpu().numpy(),
                      "exit": out.exit_mask[:B].cpu().numpy(), "idx": out.survivor_idx[:n].cpu().numpy(), "n": n}
    one, two = got[True], got[False]
    o = eo.exit_head(x, fw, fb, 0.5, False, shift, cls)
    assert util.rel_err(one["z"], two["z"], "bf16", floor=util.LOGIT_FLOOR["bf16"]) <= 1e-3   # fp32 sums over up to 2048 terms, grouped differently
    assert util.rel_err(one["z"], o["z"], "bf16", floor=util.LOGIT_FLOOR["bf16"]) <= 2e-3
    assert np.max(np.abs(one["conf"] - o["conf"])) <= 1e-2
    band = np.abs(o["conf"] - 0.5) < util.BAND
    assert np.array_equal(one["exit"][~band], o["exit"][~band]) and np.array_equal(one["exit"][~band], two["exit"][~band])
    top2 = np.sort(o["z"], axis=1)[:, -2:]
    clear = (top2[:, 1] - top2[:, 0]) > 1e-2 * np.abs(top2[:, 1])
    assert np.array_equal(one["pred"][clear], o["pred"][clear])
    assert np.array_equal(one["idx"], np.nonzero(one["exit"] == 0)[0]) and one["n"] == len(one["idx"])
    # batch invariance: every fourth sample alone
    for b in range(0, B, 4):
        m.exit_head(0, xd[b:b + 1].contiguous(), 1, HW, out, scratch, sd[b:b + 1].contiguous(), cd[b:b + 1].contiguous())
        torch.cuda.synchronize()
        assert np.array_equal(out.logits[:1].cpu().numpy()[0], one["z"][b]) and float(out.conf[0]) == float(one["conf"][b])


def test_compaction_masks_and_gather_bit_exact():
    """Force every mask pattern of a small batch through the head (identity-like FC on 1x1 maps with a
    decisive logit) and check indices, ids, count and the gathered rows bit for bit."""
    K = 4
    spec = wl.Model("mask", "f32", 1, 1, K, [wl.Stage([wl.Layer(wl.OP_CONV, K, K, 1, 1, 1, 0, wl.ACT_NONE, weight=np.eye(K, dtype=np.float32).reshape(K, 1, 1, K),
                                                              scale=np.ones(K, np.float32), bias=np.zeros(K, np.float32))],
                                                    K, np.eye(K, dtype=np.float32), np.zeros(K, np.float32), 0.9, False)], 8)
    run = util.GpuRunner(spec)
    for B in (1, 2, 5, 8):
        for bits in itertools.product([0, 1], repeat=B):
            x = np.zeros((B, 1, 1, K), np.float32)
            x[:, 0, 0, 1] = np.array(bits, np.float32) * 12.0          # exits iff the decisive logit is present
            x[:, 0, 0, 2] = np.arange(B) * 0.01                        # make rows distinguishable
            ids = 50 + np.arange(B, dtype=np.int32)
            g = run.stage(0, x, ids)
            want = [b for b in range(B) if not bits[b]]
            assert g["exit"].tolist() == list(bits)
            assert g["surv_idx"].tolist() == want and g["n_surv"] == len(want) == B - sum(bits)
            assert g["ids_out"].tolist() == [50 + b for b in want]
            assert np.array_equal(g["features_out"], x[want])


@pytest.mark.parametrize("dtype,row_elems", [("bf16", 56 * 56 * 256), ("f32", 1000), ("bf16", 8)])
def test_gather_survivors_large_rows(dtype, row_elems):
    td = eb.torch_dtype(dtype)
    B = 19
    g = torch.Generator(device="cpu").manual_seed(1)
    feat = torch.randn((B, row_elems), generator=g).to(td).cuda()
    mask = (torch.arange(B) % 3 == 1)
    idx = torch.nonzero(~mask).flatten().to(torch.int32).cuda()
    n = torch.tensor([idx.numel()], dtype=torch.int32, device="cuda")
    idx_full = torch.zeros(B, dtype=torch.int32, device="cuda")
    idx_full[: idx.numel()] = idx
    out = torch.full((B, row_elems), -1.0, dtype=td, device="cuda")
    eb.gather_survivors(feat, row_elems * feat.element_size(), idx_full, n, B, out)
    torch.cuda.synchronize()
    assert torch.equal(out[: idx.numel()], feat[idx.long()])
    assert torch.all(out[idx.numel():] == -1.0)                        # rows past n_surv are untouched


def test_refill_matches_oracle_and_clamps():
    spec = wl.tiny_ee_cnn(seed=0)
    m = eb.EEModel(spec)
    info = m.query(1)
    shape = (info["in_h"], info["in_w"], info["in_c"])
    for n_surv, n_arr in [(0, 3), (2, 4), (6, 5), (8, 2), (3, 0)]:
        surv = wl.random_features((n_surv,) + shape, seed=n_surv + 10, bf16=False)
        arr = wl.random_features((n_arr,) + shape, seed=n_arr + 20, bf16=False)
        sid, aid = np.arange(n_surv, dtype=np.int32), 40 + np.arange(n_arr, dtype=np.int32)
        f_o, id_o, acc_o = eo.refill(surv, sid, arr, aid, spec.max_batch)
        buf = torch.zeros((spec.max_batch,) + shape, device="cuda")
        ids = torch.zeros(spec.max_batch, dtype=torch.int32, device="cuda")
        buf[:n_surv] = torch.from_numpy(surv).cuda()
        ids[:n_surv] = torch.from_numpy(sid).cuda()
        n_acc, n_mer = m.batch_refill(1, buf, ids, n_surv, torch.from_numpy(arr).cuda(), torch.from_numpy(aid).cuda(), n_arr)
        torch.cuda.synchronize()
        assert (n_acc, n_mer) == (acc_o, n_surv + acc_o)
        assert np.array_equal(buf[:n_mer].cpu().numpy(), f_o) and np.array_equal(ids[:n_mer].cpu().numpy(), id_o)


# ----------------------------------------------------------------------------- API errors and degenerate cases

def test_error_codes_and_empty_batch():
    spec = wl.tiny_ee_cnn(seed=0)
    run = util.GpuRunner(spec)
    m = run.m
    x = eb.to_device("f32", wl.make_input(spec, 8, seed=0))
    with pytest.raises(eb.EEError) as e:
        m.stage_run(5, x, 8, run.bufs[0], run.ws)
    assert e.value.status == 4
    with pytest.raises(eb.EEError) as e:
        m.stage_run(0, x, 9, run.bufs[0], run.ws)
    assert e.value.status == 3
    with pytest.raises(eb.EEError) as e:
        m.stage_run(0, x, 8, run.bufs[0], run.ws[:1024])
    assert e.value.status == 3
    with pytest.raises(eb.EEError) as e:
        m.stage_run(0, None, 8, run.bufs[0], run.ws)
    assert e.value.status == 1
    with pytest.raises(eb.EEError) as e:
        m.batch_refill(7, x, None, 0, x, None, 1)
    assert e.value.status == 4
    run.bufs[0].n_surv_dev.fill_(99)
    m.stage_run(0, None, 0, run.bufs[0], run.ws)                       # empty batch: only the count is written
    torch.cuda.synchronize()
    assert int(run.bufs[0].n_surv_dev.cpu()[0]) == 0 and int(run.bufs[0].n_surv_host[0]) == 0
    # ee_run_until_exit: an empty batch runs nothing past the first stage; a stage that is not the last needs its pinned
    # count word; stage and capacity errors are those of ee_stage_run
    bufs = [eb.StageBuffers(m, s) for s in range(m.n_stages)]
    assert m.run_until_exit(0, x, 0, bufs, run.ws) == [0] * m.n_stages
    assert m.run_until_exit(m.n_stages - 1, bufs[m.n_stages - 2].features_out, 0, bufs, run.ws) == [0] * m.n_stages
    no_word = [eb.StageBuffers(m, s, pinned_count=False) for s in range(m.n_stages)]
    with pytest.raises(eb.EEError) as e:
        m.run_until_exit(0, x, 1, no_word, run.ws)
    assert e.value.status == 1
    with pytest.raises(eb.EEError) as e:
        m.run_until_exit(m.n_stages, x, 1, bufs, run.ws)
    assert e.value.status == 4
    with pytest.raises(eb.EEError) as e:
        m.run_until_exit(0, x, spec.max_batch + 1, bufs, run.ws)
    assert e.value.status == 3
    bad = wl.tiny_ee_cnn(seed=0)
    bad.stages[1].layers[0].cin = 5                                    # does not chain
    with pytest.raises(eb.EEError) as e:
        eb.EEModel(bad)
    assert e.value.status == 2


def test_device_side_timeout_is_reported_and_the_model_keeps_working():
    """The bounded waits of the kernels: a wait that nothing will ever satisfy runs out after its limit, the kernel returns,
    ee_model_check reports EE_ERR_TIMEOUT exactly once, and a normal stage then runs and matches the oracle."""
    spec = wl.tiny_ee_cnn(seed=0)
    run = util.GpuRunner(spec)
    m = run.m
    m.check()
    m.selftest_wait(2_000_000)                                         # about 1 ms of SM clocks
    with pytest.raises(eb.EEError) as e:
        m.check()
    assert e.value.status == 7                                         # EE_ERR_TIMEOUT
    m.check()                                                          # the flag was cleared by the failing check
    with pytest.raises(eb.EEError) as e:
        m.selftest_wait(0)
    assert e.value.status == 1
    x = wl.make_input(spec, 8, seed=0)
    util.check_stage(spec, run.stage(0, x), util.oracle_stage(spec, 0, x), "after the time-out self-test")


# ----------------------------------------------------------------------------- full benchmark sizes

def _full_size(spec, B, seed):
    """Benchmark-size model and batch, the launch configuration bench.py times; every stage is fed the
    oracle's stage input and compared element by element (the oracle needs well under a minute)."""
    run = util.GpuRunner(spec)
    x = wl.make_input(spec, B, seed=seed)
    ids = np.arange(B, dtype=np.int32)
    near, exited = 0, 0
    for s in range(len(spec.stages)):
        o = util.oracle_stage(spec, s, x, ids)
        g = run.stage(s, x, ids)
        r = util.check_stage(spec, g, o, f"{spec.name} full size B={B} stage {s}")
        print(f"{spec.name} full size B={B} stage {s}: batch {len(ids)}, features max-norm err {r['feat_norm_err']:.3e}, L2 err {r['feat_l2_err']:.3e}, "
              f"1e-3-floor element-wise err {r['feat_err_floor3']:.3e}, share of elements off by > 1e-2: "
              f"{r['exceed_share']:.2e} (floor 0.05) / {r['exceed_share_floor3']:.2e} (floor 1e-3), logits err {r['z_err']:.2e}, "
              f"near-threshold samples {r['band']}, flips {r['flips']}")
        near += r["band"]
        exited += int(o["exit"].sum())
        x, ids = o["features_out"], o["ids_out"]
        if len(ids) == 0:
            break
    assert exited == B
    assert near <= max(2, B // 16), f"{near} samples within 1e-3 of a threshold"
    return near


def test_resnet50_full_size_batch64():
    _full_size(wl.resnet50_ee(seed=1, max_batch=64), 64, seed=1)


@pytest.mark.parametrize("B", [1, 4, 16])
def test_resnet50_full_size_small_batches(B):
    _full_size(wl.resnet50_ee(seed=1, max_batch=64), B, seed=1)


def test_mobilenetv2_full_size_batch32():
    _full_size(wl.mobilenetv2_ee(seed=2, max_batch=32), 32, seed=2)


# ----------------------------------------------------------------------------- config 4: forced exit rates

@pytest.mark.parametrize("p", [0.0, 0.1, 0.3, 0.5, 0.8])
def test_forced_exit_rate_sweep(p):
    """Seeded Bernoulli logit shifts decide the exits: with flat unshifted logits the masks must equal the draws
    exactly, stage after stage, and the surviving batch shrinks as (1-p)^k."""
    B, K = 24, 100
    spec = wl.resnet50_ee(seed=1, in_hw=64, n_classes=K, max_batch=B, alphas=[0.01] * 4)
    run = util.GpuRunner(spec)
    draws, shifts, cls = wl.bernoulli_exit_shifts(seed=4, n_ids=B, n_exits=3, p=p, n_classes=K)
    x = wl.make_input(spec, B, seed=1)
    ids = np.arange(B, dtype=np.int32)
    for s in range(4):
        sh = shifts[s][ids] if s < 3 else None
        sc = cls[ids] if s < 3 else None
        o = util.oracle_stage(spec, s, x, ids, sh, sc)
        g = run.stage(s, x, ids, sh, sc)
        r = util.check_stage(spec, g, o, f"forced p={p} stage {s}")
        assert r["band"] == 0 and r["flips"] == 0
        if s < 3:
            assert np.array_equal(g["exit"], draws[s][ids])             # the masks ARE the Bernoulli draws
            assert np.array_equal(g["pred"][g["exit"] == 1], cls[ids][g["exit"] == 1])
        x, ids = o["features_out"], o["ids_out"]
        if len(ids) == 0:
            break


@pytest.mark.parametrize("name,max_batch,batches", [
    ("resnet50", 9, (9, 9, 9, 9)),
    ("mobilenetv2", 5, (5, 5, 5, 5)),
    ("resnet50", 64, (64, 48, 30, 27)),        # the benchmark's model and its calibrated batch per stage
    ("resnet50", 64, (64, 64, 64, 64)),        # nobody exits (forced exit rate 0)
    ("resnet50", 64, (16, 10, 8, 8)),          # a small batch on the same model (same split-K plan, other grids)
    ("mobilenetv2", 32, (32, 21, 12, 10)),
])
def test_every_layer_of_the_full_size_models(name, max_batch, batches):
    """Layer-local parity at benchmark shapes: every layer of every stage runs alone on the ORACLE's input (and
    residual) for that layer, in the kernel and launch configuration ee_stage_run uses for this (max_batch, batch) --
    split-K plan, ring depth, persistent or one-tile grid, walk direction -- and must match the oracle's output of
    that layer element-wise within the 1e-2 bar (both sides round the same pre-activation once)."""
    spec = wl.resnet50_ee(seed=1, max_batch=max_batch) if name == "resnet50" else wl.mobilenetv2_ee(seed=2, max_batch=max_batch)
    m = eb.EEModel(spec)
    ws = m.workspace()
    x = wl.make_input(spec, batches[0], seed=3)
    worst, worst3 = 0.0, 0.0
    for s, st in enumerate(spec.stages):
        B = batches[s]
        x = x[:B]
        outs = eo.run_layers(spec, s, x, keep_all=True)
        for i, l in enumerate(st.layers):
            src = x if (l.input_from == wl.FROM_STAGE_INPUT or (l.input_from == wl.FROM_PREV and i == 0)) else \
                outs[i - 1 if l.input_from == wl.FROM_PREV else l.input_from]
            res = None if l.residual_from == wl.NO_RESIDUAL else (x if l.residual_from == wl.FROM_STAGE_INPUT else outs[l.residual_from])
            out, guard = util.guarded(outs[i].shape, torch.bfloat16)
            m.layer_run(s, i, eb.to_device("bf16", src), None if res is None else eb.to_device("bf16", res), B, out, ws)
            torch.cuda.synchronize()
            assert bool(torch.all(guard == util.CANARY)), f"{name} stage {s} layer {i}: wrote past the output"
            got = out.float().cpu().numpy()
            e = util.rel_err(got, outs[i], "bf16")
            worst = max(worst, e)
            assert e <= util.TOL["bf16"], f"{name} stage {s} layer {i} ({l.kh}x{l.kw} {l.cin}->{l.cout} s{l.stride}) B={B}: {e:.3e}"
        x = outs[st.out_layer]
    m.check()
    print(f"layer-local parity {name} max_batch={max_batch} batches={batches}: worst floored(1e-3) element-wise error {worst:.3e}")


def _bits(t):
    return t.contiguous().view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32)


@pytest.mark.parametrize("name", ["resnet50", "mobilenetv2"])
def test_bf16_results_do_not_depend_on_the_batch_a_sample_rides_in(name):
    """Samples finish out of order and are re-associated by id, so a sample's result must not depend on its batch:
    on the benchmark model (max_batch as benchmarked) sample k's logits and stage output, run alone (B = 1), are
    compared BIT FOR BIT with its rows inside the full batch, inside a mid-size batch at another position, and
    inside a batch merged by ee_batch_refill at every stage boundary.  Flat heads keep every sample in flight through
    all four stages, so every layer, every grid-dependent kernel variant (one-tile, persistent, split-K, deep or
    shallow ring, walk direction) and every head is covered."""
    B = 64 if name == "resnet50" else 32
    spec = wl.resnet50_ee(seed=1, max_batch=B, alphas=[0.01] * 4) if name == "resnet50" else \
        wl.mobilenetv2_ee(seed=2, max_batch=B, alphas=[0.01] * 4)
    run = util.GpuRunner(spec)
    m, ws = run.m, run.ws
    x = eb.to_device("bf16", wl.make_input(spec, B, seed=11))
    picks = [0, B // 3, B - 1]

    def chain(feat, n):
        """All stages on the first n rows of ``feat``; returns per stage (logits, stage output) clones."""
        res = []
        for s in range(m.n_stages):
            m.stage_run(s, feat, n, run.bufs[s], ws)
            torch.cuda.synchronize()
            assert int(run.bufs[s].n_surv_host[0]) == (0 if s == m.n_stages - 1 else n)      # flat heads: nobody leaves early
            res.append((run.bufs[s].logits[:n].clone(), run.bufs[s].features_out[:n].clone() if s < m.n_stages - 1 else None))
            feat = run.bufs[s].features_out.clone()
        run.check_guards()
        return res

    full = chain(x, B)
    # alone
    for k in picks:
        one = chain(x[k:k + 1].clone(), 1)
        for s in range(m.n_stages):
            assert torch.equal(_bits(one[s][0][0]), _bits(full[s][0][k])), f"{name}: logits of sample {k} alone differ at stage {s}"
            if one[s][1] is not None:
                assert torch.equal(_bits(one[s][1][0]), _bits(full[s][1][k])), f"{name}: features of sample {k} alone differ at stage {s}"
    # a mid-size batch in another order
    perm = [B - 1, 5, B // 3, 0, 9, 2, 7]
    mid = chain(x[perm].clone(), len(perm))
    for j, k in enumerate(perm):
        for s in range(m.n_stages):
            assert torch.equal(_bits(mid[s][0][j]), _bits(full[s][0][k])), f"{name}: logits of sample {k} differ in a batch of {len(perm)} at stage {s}"
    # a schedule with a refill at every boundary: {0..a-1} runs a stage, {a..B-1} catches up, the two are merged
    a = B // 2 + 3
    feat_a, feat_b = x[:a].clone(), x[a:].clone()
    for s in range(m.n_stages):
        m.stage_run(s, feat_a, a, run.bufs[s], ws)
        torch.cuda.synchronize()
        za = run.bufs[s].logits[:a].clone()
        fa = run.bufs[s].features_out.clone()
        m.stage_run(s, feat_b, B - a, run.bufs[s], ws)
        torch.cuda.synchronize()
        zb = run.bufs[s].logits[:B - a].clone()
        assert torch.equal(_bits(torch.cat([za, zb])), _bits(full[s][0])), f"{name}: split schedule differs at stage {s}"
        if s < m.n_stages - 1:
            n_acc, n_mer = m.batch_refill(s + 1, fa, None, a, run.bufs[s].features_out, None, B - a)
            assert (n_acc, n_mer) == (B - a, B)
            torch.cuda.synchronize()
            assert torch.equal(_bits(fa), _bits(full[s][1])), f"{name}: merged batch differs at boundary {s + 1}"
            # next round: other split point, so the merged rows ride at new positions
            feat_a, feat_b = fa[:a].clone(), fa[a:].clone()
    m.check()


# ----------------------------------------------------------------------------- config 5: streaming trace

def test_streaming_trace_matches_oracle_schedule():
    """Algorithm 1 (T_SLO = infinity) on a virtual clock: the GPU-driven loop must launch exactly the batches the
    oracle-side replay launches, and every request must leave at the exit and with the class of its serial run."""
    from paper_2209_13443_b200.serving import FluidServer

    spec = wl.tiny_ee_cnn(seed=0)
    pool_np = wl.make_input(spec, 48, seed=9)
    serial = [eo.run_sample_serial(spec, pool_np[i]) for i in range(len(pool_np))]
    keep = [i for i, sref in enumerate(serial) if all(abs(c - 0.6) > 10 * util.BAND for c in sref[2][:2])][:32]
    assert len(keep) == 32
    pool_np, serial = pool_np[keep], [serial[i] for i in keep]
    n = 300
    arrivals = wl.poisson_arrivals(3, n, 2000.0)
    image_of = [r % 32 for r in range(n)]
    stage_time = lambda s, b: 2e-4 * (s + 1) + 3e-5 * b      # noqa: E731
    srv = FluidServer(spec)
    got = srv.serve(arrivals, image_of, eb.to_device("f32", pool_np), stage_time)
    exit_of = np.array([serial[image_of[r]][0] for r in range(n)])
    fin, launches = eo.serve_trace(3, spec.max_batch, arrivals, exit_of, stage_time)
    assert got["launches"] == launches
    assert np.array_equal(got["exit_stage"], exit_of)
    assert got["pred"].tolist() == [serial[image_of[r]][1] for r in range(n)]
    np.testing.assert_allclose(got["finish"], fin, rtol=0, atol=1e-9)
    assert len({len(ids) for _, ids in launches}) > 3                          # the trace exercises varying batch sizes
    # the same trace under the SLO-aware preemption criterion (Eq. 3-4): some backfills are declined, and the server
    # takes exactly the decisions of the oracle-side replay
    for slo in (1.2e-3, 2.5e-3):
        got = srv.serve(arrivals, image_of, eb.to_device("f32", pool_np), stage_time, slo=slo)
        fin, launches_slo = eo.serve_trace(3, spec.max_batch, arrivals, exit_of, stage_time, slo=slo)
        assert got["launches"] == launches_slo and got["declined"] > 0
        assert np.array_equal(got["exit_stage"], exit_of)
        np.testing.assert_allclose(got["finish"], fin, rtol=0, atol=1e-9)
    assert launches_slo != launches


def test_comparison_policies_serve_every_request_like_its_serial_run():
    """SERIAL and adaptive batching <B_max, T_timeout> on the same calls: whatever the batches, every request leaves
    at the exit and with the class of its own serial run through the oracle; SERIAL launches single samples in
    arrival order; adaptive batching with a long time-out issues full batches and never refills one."""
    from paper_2209_13443_b200.serving import FluidServer

    spec = wl.tiny_ee_cnn(seed=0)
    pool_np = wl.make_input(spec, 40, seed=9)
    serial = [eo.run_sample_serial(spec, pool_np[i]) for i in range(len(pool_np))]
    keep = [i for i, sref in enumerate(serial) if all(abs(c - 0.6) > 10 * util.BAND for c in sref[2][:2])][:24]
    pool_np, serial = pool_np[keep], [serial[i] for i in keep]
    n = 120
    arrivals = wl.poisson_arrivals(3, n, 2000.0)
    image_of = [r % len(keep) for r in range(n)]
    stage_time = lambda s, b: 2e-4 * (s + 1) + 3e-5 * b      # noqa: E731
    srv = FluidServer(spec)
    pool = eb.to_device("f32", pool_np)
    want_exit = np.array([serial[image_of[r]][0] for r in range(n)])
    want_pred = [serial[image_of[r]][1] for r in range(n)]
    got = srv.serve_serial(arrivals, image_of, pool, stage_time)
    assert np.array_equal(got["exit_stage"], want_exit) and got["pred"].tolist() == want_pred
    assert all(len(ids) == 1 for _, ids in got["launches"])
    assert [ids[0] for s, ids in got["launches"] if s == 0] == list(range(n))          # arrival order
    assert np.all(np.diff(got["finish"]) > 0) and np.all(got["finish"] > arrivals)
    # service time of a request alone: the subnets up to its exit at batch 1
    alone = np.array([sum(stage_time(s, 1) for s in range(e + 1)) for e in want_exit])
    assert np.all(got["finish"] - arrivals >= alone - 1e-12)
    got = srv.serve_adaptive_batching(arrivals, image_of, pool, max_batch=4, timeout=1.0, stage_time=stage_time)
    assert np.array_equal(got["exit_stage"], want_exit) and got["pred"].tolist() == want_pred
    first = [ids for s, ids in got["launches"] if s == 0]
    assert all(len(ids) == 4 for ids in first[:-1]) and sum(len(ids) for ids in first) == n
    for (s0, a), (s1, b) in zip(got["launches"], got["launches"][1:]):                  # a batch only ever shrinks
        if s1 == s0 + 1:
            assert set(b) <= set(a)
    got0 = srv.serve_adaptive_batching(arrivals, image_of, pool, max_batch=8, timeout=0.0, stage_time=stage_time)
    assert np.array_equal(got0["exit_stage"], want_exit)
    assert np.mean(got0["finish"] - arrivals) < np.mean(got["finish"] - arrivals)       # waiting a second for full batches costs latency


def test_stage_replay_as_graph_is_bit_identical():
    """On a side stream a stage is captured into a CUDA graph at its first call and replayed afterwards; the replay,
    and a replay on new input values in the same buffers, must equal plain launches bit for bit."""
    spec = wl.resnet50_ee(seed=1, in_hw=64, n_classes=100, max_batch=6)
    run = util.GpuRunner(spec)
    m, out, ws = run.m, run.bufs[0], run.ws
    B = 5
    xa = eb.to_device("bf16", wl.make_input(spec, B, seed=1))
    xb = eb.to_device("bf16", wl.make_input(spec, B, seed=2))
    ids = torch.arange(B, dtype=torch.int32, device="cuda")

    def snapshot():
        torch.cuda.synchronize()
        n = int(out.n_surv_host[0])
        return (n, out.features_out[:n].clone(), out.logits[:B].clone(), out.exit_mask[:B].clone(), out.survivor_idx[:n].clone())

    m.set_graphs(False)
    m.stage_run(0, xa, B, out, ws, ids)
    ref_a = snapshot()
    buf = xa.clone()
    m.set_graphs(True)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for expect_from in (xa, xa, xb):                     # capture, replay, replay on new values
            buf.copy_(expect_from)
            m.stage_run(0, buf, B, out, ws, ids)
            got = snapshot()
            if expect_from is xa:
                assert got[0] == ref_a[0] and all(torch.equal(g, r) for g, r in zip(got[1:], ref_a[1:]))
        got_b = got
    m.set_graphs(False)
    m.stage_run(0, xb, B, out, ws, ids)
    ref_b = snapshot()
    assert got_b[0] == ref_b[0] and all(torch.equal(g, r) for g, r in zip(got_b[1:], ref_b[1:]))
    m.check()


def test_branch_execution_of_shortcut_layers_is_bit_identical():
    """The projection shortcut of a block runs on the model's branch stream beside the block's main chain (plain
    launches and captured stages); switching that off must not change a bit of the stage's results."""
    spec = wl.resnet50_ee(seed=1, in_hw=96, n_classes=100, max_batch=7)
    run = util.GpuRunner(spec)
    m, ws = run.m, run.ws
    B = 7
    x = wl.make_input(spec, B, seed=4)
    side = torch.cuda.Stream()
    for s in range(m.n_stages):
        o = util.oracle_stage(spec, s, x)
        xd = eb.to_device("bf16", x)
        snaps = []
        for branches, stream in ((False, None), (True, None), (True, side), (True, side)):
            m.set_branches(branches)
            run.bufs[s].logits.fill_(0)
            run.bufs[s].features_out.fill_(0)
            with torch.cuda.stream(stream or torch.cuda.current_stream()):
                m.stage_run(s, xd, B, run.bufs[s], ws)
            torch.cuda.synchronize()
            n = int(run.bufs[s].n_surv_host[0])
            snaps.append((n, run.bufs[s].logits[:B].clone(), run.bufs[s].features_out[:n].clone()))
        for n, z, f in snaps[1:]:
            assert n == snaps[0][0] and torch.equal(z, snaps[0][1]) and torch.equal(f, snaps[0][2]), f"stage {s}"
        x = o["stage_out"]
    run.check_guards()
    m.check()


STEM_POOL_CASES = [  # (H, W, cout, act, B): even and odd output heights and widths, rows past the tile, row ranges across images
    (224, 224, 64, wl.ACT_RELU, 3), (222, 216, 64, wl.ACT_NONE, 2), (64, 64, 64, wl.ACT_RELU, 7), (30, 40, 32, wl.ACT_RELU6, 5),
    (18, 8, 64, wl.ACT_NONE, 1), (226, 224, 48, wl.ACT_RELU, 4)]


@pytest.mark.parametrize("case", STEM_POOL_CASES)
def test_stem_with_the_pool_in_its_epilogue_equals_the_two_layers_run_apart(case):
    """ee_stage_run lets the 7x7/2 stem kernel pool (3x3, stride 2, pad 1) in its epilogue; ee_layer_run runs the
    convolution and the pooling as two kernels.  The maximum of bf16 values is exact, so the stage's features must
    equal the two-kernel result bit for bit (and the oracle within the bf16 bar); the plan reports one launch."""
    H, W, cout, act, B = case
    rng = wl._rng(11, H, W, cout)
    layers = [wl._conv(rng, wl.OP_CONV, 3, cout, 7, 2, 3, act, bf16=True), wl.Layer(wl.OP_MAXPOOL, cout, cout, 3, 3, 2, 1)]
    fw, fb = wl._head(rng, cout, 5, 1.0, True)
    spec = wl.Model("stem_pool", "bf16", H, W, 3, [wl.Stage(layers, 5, fw, fb, 2.0, False)], 7)
    run = util.GpuRunner(spec)
    m, ws, out = run.m, run.ws, run.bufs[0]
    plan = m.plan(0, B)
    assert [pl["launches"] for pl in plan] == [1, 0]
    x = wl.make_input(spec, B, seed=5)
    xd = eb.to_device("bf16", x)
    ho, wo = (H - 1) // 2 + 1, (W - 1) // 2 + 1
    hp, wp = (ho - 1) // 2 + 1, (wo - 1) // 2 + 1
    conv = torch.empty((B, ho, wo, cout), dtype=torch.bfloat16, device="cuda")
    apart = torch.empty((B, hp, wp, cout), dtype=torch.bfloat16, device="cuda")
    m.layer_run(0, 0, xd, None, B, conv, ws)
    m.layer_run(0, 1, conv, None, B, apart, ws)
    for graphs in (False, True, True):
        m.set_graphs(graphs)
        out.features_out.fill_(0)
        m.stage_run(0, xd, B, out, ws)
        torch.cuda.synchronize()
        m.check()
        assert int(out.n_surv_host[0]) == B
        assert torch.equal(out.features_out[:B], apart)
    run.check_guards()
    want = eo.run_layers(spec, 0, x)
    assert util.rel_err(apart.float().cpu().numpy(), want, "bf16") <= util.TOL["bf16"]


PROJ_BLOCKS = [  # H, W, cin, mid, cout, stride, act of the projection: 64-wide tiles, ragged channels, stride 2, an activation on the shortcut
    (16, 16, 40, 48, 64, 1, wl.ACT_NONE), (16, 16, 64, 64, 136, 2, wl.ACT_NONE), (12, 20, 72, 40, 256, 2, wl.ACT_RELU),
    (9, 9, 264, 64, 72, 1, wl.ACT_RELU6)]


@pytest.mark.parametrize("blk", PROJ_BLOCKS)
def test_projection_block_shapes_against_the_oracle_and_their_own_launches(blk):
    """One block `1x1 -> 3x3 (stride) -> [1x1 projection of the input] -> 1x1 + projection` per case: the launch that
    absorbs the projection against the oracle, and bit for bit against the layers launched one by one."""
    H, W, cin, mid, cout, stride, pact = blk
    rng = wl._rng(17, H, cin, cout)
    layers = [wl._conv(rng, wl.OP_CONV, cin, mid, 1, 1, 0, wl.ACT_RELU, bf16=True, input_from=wl.FROM_STAGE_INPUT),
              wl._conv(rng, wl.OP_CONV, mid, mid, 3, stride, 1, wl.ACT_RELU, bf16=True),
              wl._conv(rng, wl.OP_CONV, cin, cout, 1, stride, 0, pact, gamma=0.7, bf16=True, input_from=wl.FROM_STAGE_INPUT),
              wl._conv(rng, wl.OP_CONV, mid, cout, 1, 1, 0, wl.ACT_RELU, gamma=0.3, bf16=True, input_from=1, residual_from=2)]
    fw, fb = wl._head(rng, cout, 5, 1.0, True)
    spec = wl.Model("proj_block", "bf16", H, W, cin, [wl.Stage(layers, 5, fw, fb, 2.0, False)], 9)
    run = util.GpuRunner(spec)
    m, ws, out = run.m, run.ws, run.bufs[0]
    for B in (1, 9):
        assert [pl["launches"] for pl in m.plan(0, B)] == [1, 1, 0, 1]
        x = wl.make_input(spec, B, seed=B)
        xd = eb.to_device("bf16", x)
        snaps = []
        for fused in (True, False, True):
            m.set_proj_fusion(fused)
            out.features_out.fill_(0)
            m.stage_run(0, xd, B, out, ws)
            torch.cuda.synchronize()
            m.check()
            assert int(out.n_surv_host[0]) == B
            snaps.append(out.features_out[:B].clone())
        assert torch.equal(snaps[0], snaps[1]) and torch.equal(snaps[0], snaps[2])
        # the absorbing layer is also the stage's last one: its epilogue pools in row blocks where Ho * Wo has blocks of 32 rows
        ho, wo = (H - 1) // stride + 1, (W - 1) // stride + 1
        assert m.gap_partials(0, B) == (32 if (ho * wo) % 32 == 0 else 0)
        z_on = out.logits[:B].clone()
        m.set_gap_fusion(False)
        m.stage_run(0, xd, B, out, ws)
        torch.cuda.synchronize()
        assert m.gap_partials(0, B) == 0 and torch.equal(out.logits[:B], z_on)
        m.set_gap_fusion(True)
        want = eo.run_layers(spec, 0, x)
        got = snaps[0].float().cpu().numpy()
        # a chain of four bf16 layers: max-norm and L2 bars, and a bounded share of elements beyond 1e-2 (tests/util.py)
        assert util.norm_err(got, want) <= util.STAGE_TOL["bf16"] and util.l2_err(got, want) <= util.STAGE_L2["bf16"], f"{blk} B={B}"
        assert util.exceed_share(got, want, util.TOL["bf16"], util.STAGE_FLOOR) <= util.STAGE_EXCEED, f"{blk} B={B}"
    run.check_guards()


@pytest.mark.parametrize("B", [26, 9])
def test_projection_inside_the_adding_layer_is_bit_identical_to_its_own_launch(B):
    """The projection shortcut of a stage's first block computed inside the launch of the layer that adds it (the
    default) against the two launches: logits and survivors' features
    agree bit for bit, on plain launches and replayed graphs; the plan shows one launch less per stage."""
    spec = wl.resnet50_ee(seed=1, in_hw=224, n_classes=100, max_batch=26, alphas=[0.01] * 4)
    run = util.GpuRunner(spec)
    m, ws = run.m, run.ws
    x = wl.make_input(spec, B, seed=4)
    xd = eb.to_device("bf16", x)
    absorbed = []
    for s in range(m.n_stages):
        m.set_proj_fusion(True)
        on = [pl["launches"] for pl in m.plan(s, B)]
        m.set_proj_fusion(False)
        off = [pl["launches"] for pl in m.plan(s, B)]
        absorbed.append(sum(off) - sum(on))
        snaps = []
        for fused, graphs in ((False, False), (True, False), (True, True), (True, True), (False, True)):
            m.set_proj_fusion(fused)
            m.set_graphs(graphs)
            run.bufs[s].logits.fill_(0)
            run.bufs[s].features_out.fill_(0)
            m.stage_run(s, xd, B, run.bufs[s], ws)
            torch.cuda.synchronize()
            m.check()
            n = int(run.bufs[s].n_surv_host[0])
            snaps.append((n, run.bufs[s].logits[:B].clone(), run.bufs[s].features_out[:n].clone()))
        assert snaps[0][0] == (B if s + 1 < m.n_stages else 0)     # flat logits: nobody leaves before the last exit
        for n, z, f in snaps[1:]:
            assert n == snaps[0][0] and torch.equal(z, snaps[0][1]) and torch.equal(f, snaps[0][2]), f"stage {s}"
        xd = run.bufs[s].features_out[:B].clone()
    run.check_guards()
    assert absorbed == [1, 1, 1, 1]


@pytest.mark.parametrize("B", [26, 9, 1])
def test_pooling_partials_from_the_epilogue_give_the_bits_of_pooling_the_stored_map(B):
    """Where the last layer of a stage runs on the persistent kernel its epilogue writes block sums of the rows it holds
    and the head pools those; elsewhere, and in ee_exit_head, the pooling kernel forms the same blocks from the stored
    map.  Logits must agree bit for bit between the two routes, with ee_exit_head on the stage's own output, and - batch
    invariance across the routes - with the sample alone in a batch of one (which never takes the epilogue route)."""
    spec = wl.resnet50_ee(seed=1, in_hw=224, n_classes=100, max_batch=26, alphas=[0.01] * 4)
    run = util.GpuRunner(spec)
    m, ws = run.m, run.ws
    x = wl.make_input(spec, B, seed=6)
    xd = eb.to_device("bf16", x)
    routes = []
    for s in range(m.n_stages):
        routes.append(m.gap_partials(s, B))
        snaps = []
        for fused, graphs in ((False, False), (True, False), (True, True), (True, True)):
            m.set_gap_fusion(fused)
            m.set_graphs(graphs)
            assert m.gap_partials(s, B) == (routes[s] if fused else 0)
            run.bufs[s].logits.fill_(0)
            m.stage_run(s, xd, B, run.bufs[s], ws)
            torch.cuda.synchronize()
            m.check()
            snaps.append((run.bufs[s].logits[:B].clone(), run.bufs[s].conf[:B].clone()))
        for z, c in snaps[1:]:
            assert torch.equal(z, snaps[0][0]) and torch.equal(c, snaps[0][1]), f"stage {s}"
        n = int(run.bufs[s].n_surv_host[0])
        if s + 1 < m.n_stages:
            assert n == B
            feat = run.bufs[s].features_out[:B].clone()
            info = m.query(s)
            hw = info["out_h"] * info["out_w"]
            out2 = eb.StageBuffers(m, s)
            scratch = torch.empty(m.exit_head_scratch_bytes(s) + 256, dtype=torch.uint8, device="cuda")
            m.exit_head(s, feat, B, hw, out2, scratch)
            torch.cuda.synchronize()
            assert torch.equal(out2.logits[:B], snaps[0][0]), f"stage {s}: ee_exit_head on the stored map"
            b = B - 1                                   # the last sample alone: stage on its input row
            m.stage_run(s, xd[b:b + 1].contiguous(), 1, out2, ws)
            torch.cuda.synchronize()
            assert torch.equal(out2.logits[0], snaps[0][0][b]), f"stage {s}: batch of one"
            xd = feat
    run.check_guards()
    assert routes == {26: [32, 16, 0, 0], 9: [32, 0, 0, 0], 1: [0, 0, 0, 0]}[B]


@pytest.mark.parametrize("B", [1, 3, 7])
def test_multi_layer_launch_is_bit_identical_to_layer_by_layer(B):
    """Runs of layers executed as one persistent kernel with grid barriers between layers (an option) against the
    same stages launched layer by layer: logits and survivors' features must agree bit for bit, on plain launches and
    on replayed graphs, twice in a row (the barrier counters must return to zero)."""
    spec = wl.resnet50_ee(seed=1, in_hw=96, n_classes=100, max_batch=7, alphas=[0.01] * 4)
    run = util.GpuRunner(spec)
    m, ws = run.m, run.ws
    x = wl.make_input(spec, B, seed=4)
    side = torch.cuda.Stream()
    xd = eb.to_device("bf16", x)
    for s in range(m.n_stages):
        snaps = []
        for mega, stream in ((False, None), (True, None), (True, side), (True, side), (True, None)):
            m.set_stage_kernel(mega)
            run.bufs[s].logits.fill_(0)
            run.bufs[s].features_out.fill_(0)
            with torch.cuda.stream(stream or torch.cuda.current_stream()):
                m.stage_run(s, xd, B, run.bufs[s], ws)
            torch.cuda.synchronize()
            m.check()
            n = int(run.bufs[s].n_surv_host[0])
            snaps.append((n, run.bufs[s].logits[:B].clone(), run.bufs[s].features_out[:n].clone()))
        for n, z, f in snaps[1:]:
            assert n == snaps[0][0] and torch.equal(z, snaps[0][1]) and torch.equal(f, snaps[0][2]), f"stage {s}"
        xd = run.bufs[s].features_out[:B].clone() if s + 1 < m.n_stages else xd
    run.check_guards()
    m.set_stage_kernel(True)
    launches_on = sum(pl["launches"] for s in range(m.n_stages) for pl in m.plan(s, B))
    m.set_stage_kernel(False)
    launches_off = sum(pl["launches"] for s in range(m.n_stages) for pl in m.plan(s, B))
    assert launches_on < launches_off


def test_count_reaches_the_host_without_a_stream_sync():
    """B_exit is copied to the pinned word beside the gather (plain launches and graph replay): ee_wait_count returns it
    without synchronising the stream, and it equals the count of the synchronised run."""
    spec = wl.resnet50_ee(seed=1, in_hw=64, n_classes=100, max_batch=6)
    run = util.GpuRunner(spec)
    m, out, ws = run.m, run.bufs[0], run.ws
    B = 6
    x = eb.to_device("bf16", wl.make_input(spec, B, seed=3))
    ids = torch.arange(B, dtype=torch.int32, device="cuda")
    m.set_graphs(False)
    m.stage_run(0, x, B, out, ws, ids)
    torch.cuda.synchronize()
    want = int(out.n_surv_host[0])
    assert want == B - int(out.exit_mask[:B].sum().item())
    m.set_graphs(True)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(3):                                   # plain capture call, then replays
            out.arm_count()
            m.stage_run(0, x, B, out, ws, ids)
            assert out.wait_count(5.0) == want
        torch.cuda.synchronize()
    m.check()


@pytest.mark.parametrize("which", ["tiny", "resnet"])
def test_device_sized_chain_matches_the_host_sized_chain(which):
    """ee_run_until_exit as one graph whose switch nodes pick every next stage's batch on the device, against the
    same call with the host sizing every stage: same batch per stage, and every output of every stage bit for bit.
    tiny: samples leave at every exit (varying counts, including runs that end early); resnet: nobody leaves early."""
    spec = wl.tiny_ee_cnn(seed=0) if which == "tiny" else wl.resnet50_ee(seed=1, in_hw=64, n_classes=100, max_batch=8, alphas=[0.01] * 4)
    run = util.GpuRunner(spec)
    m, ws = run.m, run.ws
    bufs_h = [eb.StageBuffers(m, s) for s in range(m.n_stages)]
    bufs_d = [eb.StageBuffers(m, s) for s in range(m.n_stages)]
    side = torch.cuda.Stream()
    seen = set()
    with torch.cuda.stream(side):
        for B, seed in ((8, 5), (8, 6), (3, 7), (1, 8), (8, 5)):
            x = eb.to_device(spec.dtype, wl.make_input(spec, 8, seed=seed))
            ids = torch.arange(100, 108, dtype=torch.int32, device="cuda")
            m.set_chain(0)
            sizes_h = m.run_until_exit(0, x, B, bufs_h, ws, ids)
            torch.cuda.synchronize()
            m.set_chain(spec.max_batch)
            for b in bufs_d:
                b.exit_mask.fill_(9)
            sizes_d = m.run_until_exit(0, x, B, bufs_d, ws, ids)
            torch.cuda.synchronize()
            m.check()
            assert sizes_d == sizes_h, (B, seed, sizes_d, sizes_h)
            seen.add(tuple(sizes_h))
            for s, n in enumerate(sizes_h):
                if n == 0:
                    break
                h, d = bufs_h[s], bufs_d[s]
                ns = int(h.n_surv_host[0])
                assert int(d.n_surv_host[0]) == ns == int(d.n_surv_dev.cpu()[0])
                assert torch.equal(d.exit_mask[:n], h.exit_mask[:n]) and torch.equal(d.pred[:n], h.pred[:n]) and torch.equal(d.conf[:n], h.conf[:n])
                assert torch.equal(d.logits[:n], h.logits[:n]) and torch.equal(d.survivor_idx[:ns], h.survivor_idx[:ns])
                assert torch.equal(d.ids_out[:ns], h.ids_out[:ns]) and torch.equal(d.features_out[:ns], h.features_out[:ns])
    assert len(seen) >= (3 if which == "tiny" else 2)
    run.check_guards()


@pytest.mark.parametrize("which", ["tiny", "resnet"])
def test_run_until_exit_matches_the_stage_by_stage_loop(which):
    """ee_run_until_exit chains the stages inside the library; it must leave exactly what a caller's own loop of
    ee_stage_run + count read-back leaves: same batch per stage, same masks, predictions, ids and survivors.
    tiny: exits at every stage; resnet: flat heads, the whole batch reaches the last stage."""
    spec = wl.tiny_ee_cnn(seed=0) if which == "tiny" else wl.resnet50_ee(seed=1, in_hw=64, n_classes=100, max_batch=8, alphas=[0.01] * 4)
    run = util.GpuRunner(spec)
    m, ws = run.m, run.ws
    B = 8
    x = eb.to_device(spec.dtype, wl.make_input(spec, B, seed=5))
    ids = torch.arange(100, 100 + B, dtype=torch.int32, device="cuda")
    ref = []
    feat, idv, n = x, ids, B
    for s in range(m.n_stages):
        m.stage_run(s, feat, n, run.bufs[s], ws, idv)
        torch.cuda.synchronize()
        b = run.bufs[s]
        ns = int(b.n_surv_host[0])
        ref.append((n, b.exit_mask[:n].clone(), b.pred[:n].clone(), b.conf[:n].clone(), b.ids_out[:ns].clone(), b.features_out[:ns].clone()))
        feat, idv, n = b.features_out.clone(), b.ids_out.clone(), ns
        if n == 0:
            break
    assert len(ref) >= 2                                   # the batch does reach a later stage
    bufs2 = [eb.StageBuffers(m, s) for s in range(m.n_stages)]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(2):                                 # plain launches / capture, then graph replay
            sizes = m.run_until_exit(0, x, B, bufs2, ws, ids)
            torch.cuda.synchronize()
            assert sizes[:len(ref)] == [r[0] for r in ref] and all(v == 0 for v in sizes[len(ref):])
            for s, (n, mask, pred, conf, ids_out, feats) in enumerate(ref):
                b = bufs2[s]
                assert torch.equal(b.exit_mask[:n], mask) and torch.equal(b.pred[:n], pred) and torch.equal(b.conf[:n], conf)
                assert torch.equal(b.ids_out[:len(ids_out)], ids_out) and torch.equal(b.features_out[:len(feats)], feats)
    m.check()
