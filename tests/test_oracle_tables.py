"""Pins of the oracle's integer bookkeeping (partitions, live sets, micro-batches, schedule)."""
import os

import numpy as np
import pytest

import workloads as wl
from oracle import reference as ora


def _facts():
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = [t.strip() for t in line.split("=")]
                out[k] = v
    return out


def test_depth_and_counts_of_resnet1001():
    ops = wl.resnet_v2_cifar(111)
    n = 111
    weight_layers = sum(1 for o in ops if o.kind == wl.CONV and not (o.ksize == 1 and o.src0 >= 0 and ops[o.src0].kind != wl.BNRELU)) + 1
    assert weight_layers == int(_facts()["resnet1001_depth"])     # stem + 9n block convs + FC, projections not counted
    assert len(ops) == 21 * n + 6
    # closed-form parameter count, independent of the op loop
    def stage(c_t, w, first):
        convs = c_t * w + 9 * w * w + 4 * w * w + (c_t * 4 * w if first else 0)
        return convs + 2 * (c_t + w + w)
    G = 3 * 9 * 16
    c_t = 16
    for w in (16, 32, 64):
        G += stage(c_t, w, True) + (n - 1) * stage(4 * w, w, False)
        c_t = 4 * w
    G += 2 * 256 + 256 * 10 + 10
    assert ora.param_layout(ops)[4] == G == 10327706


def test_keras_width_variant_has_the_parameter_count_the_paper_quotes():
    """With the Keras example's chaining rule (a stage's bottleneck width = the previous stage's output channels:
    16/64/128 -> 64/128/256) the 1001-layer net has the ~30 M parameters the paper states; closed form, independent
    of the op loop."""
    n = 111
    ops = wl.config("r1001k")["ops"]
    def block(c_t, w, co, first):
        return c_t * w + 9 * w * w + w * co + (c_t * co if first else 0) + 2 * (c_t + w + w)
    G = 3 * 9 * 16
    c_t = 16
    for w, co in ((16, 64), (64, 128), (128, 256)):
        G += block(c_t, w, co, True) + (n - 1) * block(co, w, co, False)
        c_t = co
    G += 2 * 256 + 256 * 10 + 10
    assert ora.param_layout(ops)[4] == G == 30251290
    assert round(G / 1e6) == int(_facts()["resnet1001_params_millions"])
    assert len(ops) == 21 * n + 6


def test_depth_and_counts_of_resnet110_v1():
    """The paper's ResNet-110 is the post-activation basic-block net: depth 6n+2 with n = 18 (Section 6.1 names the
    model); closed-form parameter count, independent of the op loop."""
    n = 18
    ops = wl.resnet_v1_cifar(n)
    weight_layers = sum(1 for o in ops if o.kind == wl.CONV and o.ksize == 3) + 1      # 3x3 convolutions + FC
    assert weight_layers == 6 * n + 2 == 110
    G = 3 * 9 * 16 + 2 * 16
    c_t = 16
    for w in (16, 32, 64):
        first = 9 * c_t * w + 2 * w + 9 * w * w + 2 * w + (c_t * w if c_t != w else 0)
        G += first + (n - 1) * (2 * (9 * w * w + 2 * w))
        c_t = w
    G += 64 * 10 + 10
    assert ora.param_layout(ops)[4] == G == wl.param_offsets(ops)[1]


def test_param_layout_is_dense_and_ordered():
    ops = wl.resnet_v2_imagenet(blocks=(1, 1), widths=(4, 8), n_classes=7)
    w_off, w_cnt, b_off, b_cnt, G = ora.param_layout(ops)
    at = 0
    for i, o in enumerate(ops):
        assert w_off[i] == at; at += w_cnt[i]
        assert b_off[i] == at; at += b_cnt[i]
        if o.kind == wl.CONV:
            assert (w_cnt[i], b_cnt[i]) == (o.c_out * o.ksize ** 2 * o.c_in, 0)
        if o.kind in (wl.ADD, wl.MAXPOOL):
            assert (w_cnt[i], b_cnt[i]) == (0, 0)
    assert at == G


def test_shapes_match_generator_and_downsample():
    c = wl.config("r11")
    assert ora.shapes(c["ops"], c["in_hwc"]) == wl.tensor_shapes(c["ops"], c["in_hwc"])
    shp = ora.shapes(wl.resnet_v2_imagenet(), (224, 224, 3))
    assert shp[0] == (112, 112, 64) and shp[1] == (56, 56, 64) and shp[-2] == (7, 7, 2048) and shp[-1] == (1, 1, 1000)


def test_partition_of_ops_and_cut_validation():
    assert ora.partition_of_ops(6, [2, 3]) == [0, 0, 1, 2, 2, 2]
    assert ora.partition_of_ops(4, []) == [0, 0, 0, 0]
    assert ora.partition_of_ops(4, [1, 2, 3]) == [0, 1, 2, 3]          # one op per partition is the limit
    for bad in ([0], [4], [2, 2], [3, 2], [1, 2, 3, 3]):
        with pytest.raises(ValueError):
            ora.partition_of_ops(4, bad)


def test_live_sets_of_the_benchmark_cuts():
    """Every default cut of ResNet-1001 falls inside a residual block or at its edge:
    at most the trunk and the shortcut cross it."""
    c = wl.config("r1001")
    ops = c["ops"]
    for cut in c["cuts"]:
        live = ora.live_set(ops, cut)
        brute = sorted({t for i in range(cut, len(ops)) for t in ((ops[i].src0, ops[i].src1) if ops[i].kind == wl.ADD else (ops[i].src0,)) if 0 <= t < cut})
        assert live == brute
        assert 1 <= len(live) <= 2
    # block-aligned cut: just the trunk
    r11 = wl.config("r11")["ops"]
    assert ora.live_set(r11, 9) == [8]
    assert ora.live_set(r11, 4) == [0, 3]      # mid-block: stem output (shortcut) + c1 path


def test_microbatch_ranges_cover_the_batch():
    for B, M in ((8, 2), (128, 8), (64, 4), (5, 5), (7, 1)):
        spans = [ora.microbatch_range(B, M, m) for m in range(M)]
        assert spans[0][0] == 0 and spans[-1][1] == B
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        assert len({e - s for s, e in spans}) == 1
    for B, M in ((8, 3), (4, 8), (8, 0)):
        with pytest.raises(ValueError):
            ora.microbatch_range(B, M, 0)


def test_schedule_is_a_valid_fill_drain_pipeline():
    for P, M in ((2, 2), (4, 4), (8, 8), (3, 5)):
        f = {(p, m): ora.schedule_tick(P, M, p, m) for p in range(P) for m in range(M)}
        for (p, m), (ft, bt) in f.items():
            if p > 0:
                assert ft > f[(p - 1, m)][0]      # needs the previous partition's activation
            if p < P - 1:
                assert bt > f[(p + 1, m)][1]      # needs the next partition's partial error
            if m > 0:
                assert ft > f[(p, m - 1)][0] and bt > f[(p, m - 1)][1]   # one micro-batch at a time per partition
        assert max(v[0] for v in f.values()) == P + M - 2 == max(v[1] for v in f.values())
        # a partition is never asked to do two things in one tick
        assert len({(p, v[0]) for (p, m), v in f.items()}) == P * M
