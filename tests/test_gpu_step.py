"""Parity of the CUDA step against the fp64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import paper_1911_05146_b200 as hpf
import workloads as wl
from oracle import reference as ora
from hpf_testlib import (Bound, rel_l2, seeded, matched_oracle, compare_microbatch, log_parity, TOL_TENSOR, TOL_LOSS, TAU, TAU_ONE_PASS,
                         MAX_DECISION_FRACTION, MAX_DECISION_FRACTION_ONE_PASS)

pytestmark = pytest.mark.gpu


def check_step(ops, in_hwc, B, M, cuts, options=None, seed=0, bn_jitter=0.0, microbatches=None, tensors=True, name=None, edit_theta=None,
               skip=()):
    x, labels, theta = seeded(ops, in_hwc, B, seed, bn_jitter)
    if edit_theta is not None:
        theta = edit_theta(theta)
    bd = Bound(ops, in_hwc, B, M, cuts, theta, options)
    bd.upload(x, labels)
    loss = bd.step()
    ref = ora.step(ops, in_hwc, theta, x, labels, M, cuts=list(cuts))
    assert abs(loss - ref["loss"]) <= TOL_LOSS * abs(ref["loss"]), (loss, ref["loss"])
    assert np.allclose(bd.loss_slots(), ref["losses"], rtol=TOL_LOSS, atol=0)
    slots = bd.slots.cpu().numpy()
    avg = bd.avg.cpu().numpy()
    assert np.isfinite(slots).all() and np.isfinite(avg).all()     # every parameter got a gradient
    # the average is exactly the fixed-order fp32 sum of the slots over M
    acc = slots[0].copy()
    for m in range(1, M):
        acc += slots[m]
    assert np.array_equal(avg, acc * np.float32(1.0 / M))
    offs, G = wl.param_offsets(ops)
    one_pass = (options or {}).get(hpf.OPT_CONV_PATH) == 2
    tau = TAU_ONE_PASS if one_pass else TAU
    frac = MAX_DECISION_FRACTION_ONE_PASS if one_pass else MAX_DECISION_FRACTION
    losses = bd.loss_slots()
    want_m = set(range(M) if microbatches is None else microbatches)
    # every micro-batch: the plain oracle first, the oracle under the GPU's in-window decisions as a diagnostic
    res = [compare_microbatch(bd, m, theta, x, labels, slots, offs, float(losses[m]), cuts=list(cuts), tau=tau, max_fraction=frac,
                              tensors=tensors and m in want_m, skip=skip) for m in range(M)]
    # the averaged gradient against the plain oracle's step; where slots needed the GPU's decisions, against their average
    need_matched = any(r["over"] for r in res)
    g_avg_ref = ref["g_avg"] if not need_matched else ora.grad_average(np.stack([r["matched_result"]["g"] for r in res]))
    for i, (w_off, w_cnt, b_off, b_cnt) in enumerate(offs):
        for which, off, cnt in (("w", w_off, w_cnt), ("b", b_off, b_cnt)):
            if cnt and ("g", i, which) not in skip:
                e = rel_l2(avg[off:off + cnt], g_avg_ref[off:off + cnt])
                assert e <= TOL_TENSOR, ("avg op", i, e)
    import inspect
    log_parity(name or inspect.stack()[1].function, res)
    worst = max(max(r["plain"].values()) for r in res)
    return bd, ref, worst


@pytest.mark.parametrize("conv_path", [0, 1, 2])
@pytest.mark.parametrize("graph", [1, 0])
def test_config1_resnet11(conv_path, graph):
    c = wl.config("r11")
    check_step(c["ops"], c["in_hwc"], c["B"], c["M"], c["cuts"],
               {hpf.OPT_CONV_PATH: conv_path, hpf.OPT_GRAPH: graph})


@pytest.mark.parametrize("fuse_bn,pdl,wgrad_passes", [(0, 1, 1), (1, 0, 3), (3, 0, 3)])
def test_config1_without_the_fusions(fuse_bn, pdl, wgrad_passes):
    """The BN reductions in their own kernels or both folded into the convolutions, plain stream-ordered
    launches, three-pass weight gradient."""
    c = wl.config("r11")
    check_step(c["ops"], c["in_hwc"], c["B"], c["M"], c["cuts"],
               {hpf.OPT_FUSE_BN: fuse_bn, hpf.OPT_PDL: pdl, hpf.OPT_WGRAD_PASSES: wgrad_passes})


@pytest.mark.parametrize("cuts", [[], [4], [3, 7, 8], [1, 5, 12, 25]])
@pytest.mark.parametrize("fuse_add", [1, 0])
def test_mid_block_cuts_and_jittered_bn(cuts, fuse_add):
    ops = wl.resnet_v2_cifar(1)
    bd, _, _ = check_step(ops, (32, 32, 3), 4, 2, cuts, {hpf.OPT_FUSE_ADD: fuse_add}, seed=3, bn_jitter=0.3)
    stored = [bd.tensor_or_none(i, 0) is not None for i in range(len(ops))]
    if fuse_add == 0:
        assert all(stored)
    else:
        # every cut list leaves at least one (projection, ADD) pair inside one partition
        assert not all(stored)


@pytest.mark.parametrize("B,M,cuts", [(4, 1, []), (4, 4, [9]), (3, 3, "every op"), (6, 2, "every op")],
                         ids=["one_partition_one_microbatch", "microbatches_of_one_sample", "one_op_per_partition_b1", "one_op_per_partition"])
def test_degenerate_partitionings(B, M, cuts):
    """The ends of the ranges the method allows (Section 5.3: 1..batch size micro-batches; Section 7: at most one layer
    per partition): no pipelining at all, micro-batches of a single sample, and every op its own partition."""
    ops = wl.resnet_v2_cifar(1)
    if cuts == "every op":
        cuts = list(range(1, len(ops)))
    bd, _, _ = check_step(ops, (32, 32, 3), B, M, cuts, seed=4, bn_jitter=0.2)
    assert bd.model.num_partitions() == len(cuts) + 1


@pytest.mark.parametrize("cuts", [[11], [4, 9, 16]])
def test_post_activation_basic_blocks(cuts):
    """ResNet v1 blocks (CONV BNRELU CONV BN, ADD with the shortcut, RELU), with a strided 3x3 convolution and a
    projection shortcut: the paper's ResNet-110 family at depth 8."""
    c = wl.config("r8v1")
    bd, _, _ = check_step(c["ops"], c["in_hwc"], c["B"], c["M"], cuts, seed=6, bn_jitter=0.2)
    assert bd.model.num_partitions() == len(cuts) + 1


def test_vgg_style_net_without_batch_norm():
    """Convolution + ReLU groups, 2x2 max-pools down to one pixel, hidden fully connected layers as 1x1 convolutions:
    the paper's VGG-16 layout at reduced width."""
    c = wl.config("vgg16s")
    check_step(c["ops"], c["in_hwc"], c["B"], c["M"], c["cuts"], seed=8)


def test_large_microbatch_uses_the_multi_tile_convolutions_with_the_bn_fusions():
    """A micro-batch of 80 images at 32x32 is 640 pixel tiles per convolution: the launches give each CTA several tiles,
    with the BN statistics and the BN+ReLU-on-the-way-in riding in the same kernels."""
    c = wl.config("r11")
    check_step(c["ops"], c["in_hwc"], 80, 1, c["cuts"], seed=9, bn_jitter=0.1, microbatches=[0])


@pytest.mark.parametrize("fuse_bn", [0, 1, 3])
def test_bn_statistics_of_channels_whose_mean_dwarfs_their_spread(fuse_bn):
    """BN shifts of ten and scales of a tenth: the activations a convolution reads are then ten +- 0.1, and its output,
    the next BN's input, has per-channel means of a hundred and more standard deviations.  The statistics must come out
    right whether the BN runs its own kernels (0), takes its moments from the producing convolution's write-out (1) or is
    applied by the reading convolution (3)."""
    ops = wl.resnet_v2_cifar(1)
    offs, G = wl.param_offsets(ops)

    def shifted(theta):
        theta = theta.copy()
        for i, o in enumerate(ops):
            if o.kind == wl.BNRELU:
                w_off, w_cnt, b_off, b_cnt = offs[i]
                theta[w_off:w_off + w_cnt] *= np.float32(0.1)
                theta[b_off:b_off + b_cnt] += np.float32(10.0)
        return theta

    # With shifts this large no activation is ever clipped, so a BN's shift only adds a constant per channel to the
    # convolution that follows (but for the padding ring of a 3x3 window), which the next BN removes again: its gradient
    # is zero analytically, or a sum that cancels to almost nothing (both sides compute rounding noise there), and a
    # relative error of it means nothing.
    zero_grad = {("g", i, "b") for i, o in enumerate(ops) if o.kind == wl.BNRELU and ops[i + 1].kind == wl.CONV}
    # (three-pass weight gradients: with activations of ten +- 0.1 a single TF32 pass keeps too little of the +- 0.1, which
    # is all that survives the sum against a gradient whose channel sums vanish)
    # The weight gradient of a convolution that reads such a BN's output sums dy * (10 +- 0.1) over the pixels against a dy
    # whose channel sums all but vanish: two digits cancel in any fp32 evaluation (the two weight-gradient kernels, fed the
    # same bits, differ from each other by as much as either differs from the oracle).  Those tensors are held to 5e-2 here;
    # everything else, the BN statistics and activations above all, to the usual tolerance.
    shifted_input = {("g", i, "w") for i, o in enumerate(ops) if o.kind == wl.CONV and o.src0 >= 0 and ops[o.src0].kind == wl.BNRELU}
    bd, ref, _ = check_step(ops, (32, 32, 3), 8, 2, [9], {hpf.OPT_FUSE_BN: fuse_bn, hpf.OPT_WGRAD_PASSES: 3}, seed=21, bn_jitter=0.2, edit_theta=shifted,
                            name="mean >> sigma, fuse_bn=%d" % fuse_bn, skip=zero_grad | shifted_input)
    avg = bd.avg.cpu().numpy()
    for _, i, _ in sorted(shifted_input):
        w_off, w_cnt, _, _ = offs[i]
        assert rel_l2(avg[w_off:w_off + w_cnt], ref["g_avg"][w_off:w_off + w_cnt]) <= 5e-2, i
    # the premise: some BN input really is that badly centred
    ratios = []
    for i, o in enumerate(ops):
        if o.kind == wl.BNRELU and ops[o.src0].kind == wl.CONV and ops[o.src0].src0 >= 0:
            t = bd.tensor_or_none(o.src0, 0)
            if t is not None:
                t = t.reshape(-1, t.shape[-1]).astype(np.float64)
                ratios.append(float(np.max(np.abs(t.mean(0)) / t.std(0))))
    assert max(ratios) > 50, ratios


@pytest.mark.parametrize("ctas", [3, 16, 40])
def test_persistent_forward_cells_give_the_same_bits_as_one_launch_per_convolution(ctas):
    """Section 5.3's stage as one resident grid: the forward convolutions of a cell run inside ONE persistent kernel that
    walks the list with grid-wide barriers.  Fewer CTAs than tiles (several rounds and several tiles per CTA), about as many,
    and more than any launch has; against the oracle, and bit for bit against the step made of single launches."""
    ops = wl.resnet_v2_cifar(2)
    cuts = wl.default_cuts(len(ops), 3)
    bd, _, _ = check_step(ops, (32, 32, 3), 8, 2, cuts, {hpf.OPT_CELL_CTAS: ctas}, seed=12, bn_jitter=0.2, name="persistent cells, %d CTAs" % ctas)
    x, labels, theta = seeded(ops, (32, 32, 3), 8, 12, 0.2)
    ref = Bound(ops, (32, 32, 3), 8, 2, cuts, theta, {hpf.OPT_CELL_CTAS: 0})
    ref.upload(x, labels)
    loss = ref.step()
    assert bd.model.launch_count() < ref.model.launch_count()          # the cells replaced launches
    assert loss == bd.model.loss()
    assert torch.equal(ref.slots, bd.slots) and torch.equal(ref.avg, bd.avg)
    for i in range(len(ops)):
        a, b2 = ref.tensor_or_none(i, 1), bd.tensor_or_none(i, 1)
        assert (a is None) == (b2 is None)
        if a is not None:
            assert np.array_equal(a, b2), i


def test_persistent_forward_cells_on_wide_channels_and_repeated_steps():
    """ImageNet-layout block with 256..1024 channels (stages too large for two CTAs per SM, channel slices) inside cells; the
    second step must find the grid barrier as the first one left it."""
    ops = wl.resnet_v2_imagenet(blocks=(2, 1), widths=(128, 256), n_classes=9)
    bd, _, _ = check_step(ops, (32, 32, 3), 4, 2, [9, 20], {hpf.OPT_CELL_CTAS: 12}, seed=3, bn_jitter=0.2, name="persistent cells, wide channels")
    s1 = bd.slots.clone()
    l1 = bd.model.loss()
    assert bd.step() == l1 and torch.equal(s1, bd.slots)


def test_odd_widths_run_on_cuda_cores():
    ops = wl.resnet_v2_cifar(1, widths=(4, 8, 12), n_classes=5)
    bd, _, _ = check_step(ops, (8, 8, 3), 6, 3, [9], seed=1, bn_jitter=0.2)
    n_tc, n_cc = bd.model.conv_path_counts()
    assert n_cc > 0          # 4-, 8-, 12-channel convolutions have no tensor-core kernel


def test_imagenet_layout_small_with_maxpool():
    ops = wl.resnet_v2_imagenet(blocks=(1, 1), widths=(16, 32), n_classes=7)
    check_step(ops, (32, 32, 3), 4, 2, [2, 11], seed=2, bn_jitter=0.2)


def test_imagenet_layout_wide_channels():
    """Channel counts beyond 256 (512 and 1024 block outputs, 3x3 at 128 and 256): convolutions, BN and the fusions that
    apply only up to 256 channels side by side."""
    ops = wl.resnet_v2_imagenet(blocks=(2, 1), widths=(128, 256), n_classes=9)
    check_step(ops, (32, 32, 3), 4, 2, [9, 20], seed=3, bn_jitter=0.2)


def test_long_k_loops_split_over_ctas():
    """A 3x3 convolution on 512 channels over a 4x4 map: one pixel tile, 576 K steps, no BN fusion beyond 256 channels, so
    the forward and the data gradient split their K loop over several CTAs (partial tiles, ticket, ordered sum)."""
    ops = wl.resnet_v2_imagenet(blocks=(1, 1), widths=(64, 512), n_classes=9)
    check_step(ops, (32, 32, 3), 4, 2, [11], seed=13, bn_jitter=0.2)


def test_many_class_head_on_ragged_sizes():
    """The head kernels for many classes (one warp per class, 64-channel x 8-sample blocks in the backward): 350 classes on
    96 channels with micro-batches of 3 samples, so that no block or warp loop is full."""
    ops = wl.resnet_v2_imagenet(blocks=(1, 1), widths=(16, 24), n_classes=350)
    check_step(ops, (32, 32, 3), 6, 2, [7], seed=11, bn_jitter=0.2)


def test_second_step_and_new_inputs_reuse_the_model():
    c = wl.config("r11")
    ops = c["ops"]
    x, labels, theta = seeded(ops, c["in_hwc"], c["B"])
    bd = Bound(ops, c["in_hwc"], c["B"], c["M"], c["cuts"], theta)
    bd.upload(x, labels)
    l1 = bd.step(); s1 = bd.slots.clone()
    l2 = bd.step()
    assert l1 == l2 and torch.equal(s1, bd.slots)          # same inputs -> bit-identical, nothing left over
    x2, labels2, _ = seeded(ops, c["in_hwc"], c["B"], seed=5)
    bd.upload(x2, labels2)                                   # new device buffers -> the phases are re-captured
    l3 = bd.step()
    ref = ora.step(ops, c["in_hwc"], theta, x2, labels2, c["M"], cuts=c["cuts"])
    assert abs(l3 - ref["loss"]) <= TOL_LOSS * abs(ref["loss"])
    assert rel_l2(bd.avg.cpu().numpy(), ref["g_avg"]) <= TOL_TENSOR
    # the host-buffer entry point gives the same numbers
    hx = torch.from_numpy(x2).pin_memory(); hl = torch.from_numpy(labels2).pin_memory()
    l4 = bd.model.step_host(hx, hl)
    bd.model.synchronize(60000)
    assert l4 == l3
    assert rel_l2(bd.avg.cpu().numpy(), ref["g_avg"]) <= TOL_TENSOR


def test_single_stream_equals_multi_stream_bitwise():
    """Stream-hazard check: a missing event would show up as a difference."""
    ops = wl.resnet_v2_cifar(2)
    x, labels, theta = seeded(ops, (32, 32, 3), 8, seed=4)
    cuts = wl.default_cuts(len(ops), 4)
    outs = []
    for single, side in ((0, True), (1, True), (0, False)):
        bd = Bound(ops, (32, 32, 3), 8, 4, cuts, theta, {hpf.OPT_SINGLE_STREAM: single}, side_streams=side)
        bd.upload(x, labels)
        loss = bd.step()
        outs.append((loss, bd.slots.clone(), bd.avg.clone()))
    for o in outs[1:]:
        assert outs[0][0] == o[0]
        assert torch.equal(outs[0][1], o[1]) and torch.equal(outs[0][2], o[2])


@pytest.mark.parametrize("streams", ["3P", "2P", "P"])
def test_forward_and_backward_as_one_graph_give_the_same_bits(streams):
    """hpf_forward_backward: the backward pipeline fills while the forward pipeline drains (a cell starts as soon as the
    cell that feeds it is done).  Same kernels on the same data, so every bit must equal the two-phase step - also when
    the caller gave no streams for the backward cells (then the call is the two phases in one graph)."""
    ops = wl.resnet_v2_cifar(2)
    x, labels, theta = seeded(ops, (32, 32, 3), 8, seed=4, bn_jitter=0.1)
    cuts = wl.default_cuts(len(ops), 4)
    ref = Bound(ops, (32, 32, 3), 8, 4, cuts, theta)
    ref.upload(x, labels)
    l_ref = ref.step()
    bd = Bound(ops, (32, 32, 3), 8, 4, cuts, theta, {hpf.OPT_CELL_TIMES: 1}, side_streams=streams != "P", backward_streams=streams == "3P")
    bd.upload(x, labels)
    for _ in range(2):                           # the second replay must find every ticket and barrier as the first left it
        assert bd.step(one_graph=True) == l_ref
        assert torch.equal(ref.slots, bd.slots) and torch.equal(ref.avg, bd.avg)
    for i in range(len(ops)):
        assert np.array_equal(ref.tensor(i, 3, grad=True), bd.tensor(i, 3, grad=True)), i
    if streams == "3P":
        # the point of it: some backward cell starts before the last forward cell has ended
        fwd, bwd = bd.model.cell_times(0), bd.model.cell_times(1)
        assert min(s for row in bwd for s, _ in row) < max(e for row in fwd for _, e in row)
        P, M = 4, 4
        for m in range(M):
            assert bwd[P - 1][m][0] >= fwd[P - 1][m][1]          # the last partition turns around only after its forward cell
            for p in range(P - 1):
                assert bwd[p][m][0] >= bwd[p + 1][m][1]          # partial errors arrive from the partition above
    with pytest.raises(hpf.HpfError):
        bd.model.backward()                      # the step is complete: a second backward needs a fresh forward


@pytest.mark.parametrize("lanes,one_graph", [(2, True), (3, True), (4, True), (8, True), (2, False)])
def test_stage_lanes_give_the_same_bits_and_fill_the_bubble(lanes, one_graph):
    """HPF_OPT_STAGE_LANES: a stage keeps several of its micro-batches under way at once, each lane on its own streams and
    scratch.  Every cell runs the same kernels on the same data, so every bit must equal the one-lane schedule; the hand-offs
    between stages still order the cells of one micro-batch; and cells of one stage really do overlap."""
    ops = wl.resnet_v2_cifar(2)
    x, labels, theta = seeded(ops, (32, 32, 3), 8, seed=6, bn_jitter=0.1)
    P, M = 3, 4
    cuts = wl.default_cuts(len(ops), P)
    ref = Bound(ops, (32, 32, 3), 8, M, cuts, theta)
    ref.upload(x, labels)
    l_ref = ref.step()
    bd = Bound(ops, (32, 32, 3), 8, M, cuts, theta, {hpf.OPT_STAGE_LANES: lanes, hpf.OPT_CELL_TIMES: 1}, backward_streams=one_graph)
    assert bd.model.num_stream_slots() == P * min(lanes, M)
    bd.upload(x, labels)
    for _ in range(2):
        assert bd.step(one_graph=one_graph) == l_ref
        assert torch.equal(ref.slots, bd.slots) and torch.equal(ref.avg, bd.avg)
    for i in range(len(ops)):
        assert np.array_equal(ref.tensor(i, M - 1, grad=True), bd.tensor(i, M - 1, grad=True)), i
    fwd, bwd = bd.model.cell_times(0), bd.model.cell_times(1)
    for m in range(M):
        for p in range(1, P):
            assert fwd[p][m][0] >= fwd[p - 1][m][1]              # activations arrive from the partition below
        for p in range(P - 1):
            assert bwd[p][m][0] >= bwd[p + 1][m][1]              # partial errors arrive from the partition above
        assert bwd[P - 1][m][0] >= fwd[P - 1][m][1]
    L = min(lanes, M)
    for p in range(P):
        for m in range(L, M):
            assert fwd[p][m][0] >= fwd[p][m - L][1]              # a lane works through its micro-batches in order
    # the point of it: micro-batches 0 and 1 of the first stage run side by side
    assert fwd[0][1][0] < fwd[0][0][1]


def test_too_few_streams_for_the_lanes_are_refused():
    ops = wl.resnet_v2_cifar(1)
    model = hpf.Model(ops, (4, 32, 32, 3), wl.default_cuts(len(ops), 2), 2)
    model.set_option(hpf.OPT_STAGE_LANES, 2)
    assert model.num_stream_slots() == 4
    G = model.num_params()
    params = torch.zeros(G, device="cuda"); slots = torch.zeros((2, G), device="cuda"); avg = torch.zeros(G, device="cuda")
    ws = torch.empty(model.workspace_bytes(), dtype=torch.uint8, device="cuda")
    with pytest.raises(hpf.HpfError):
        model.bind(params, slots, avg, ws, [torch.cuda.Stream() for _ in range(2)])


@pytest.mark.parametrize("P,R,cuts", [(2, 1, [12]), (3, 1, [9, 30]), (2, 2, [25])], ids=["two_stages_mid_block_cut", "three_stages", "two_stages_two_replicas"])
def test_stage_per_gpu_hand_offs_emulated_on_one_gpu(P, R, cuts):
    """Hybrid parallelism (Section 5.3): every rank binds the same model and runs only its partition's cells; what crosses
    a cut is copied between the ranks' workspaces.  All ranks are emulated in one process on this GPU (cell by cell, device
    copies for the hand-offs, a mean over the replicas for the per-partition allreduce): the averaged gradient must equal,
    bit for bit, what ordinary single-model steps give, and match the oracle."""
    from paper_1911_05146_b200.hybrid import HybridLayout, Stage, emulate_step
    ops = wl.resnet_v2_cifar(2)
    B, M, hwc = 4, 2, (32, 32, 3)
    theta = wl.draw_params(ops, seed=wl.inputs.SEED_PARAMS + 17, bn_jitter=0.2)
    layout = HybridLayout(P * R, P)
    data = [wl.draw_inputs(B, hwc, 10, seed_x=wl.inputs.SEED_X + 30 + r, seed_labels=wl.inputs.SEED_LABELS + 30 + r) for r in range(R)]
    dev = torch.device("cuda:0")
    batches = [(torch.from_numpy(x).to(dev), torch.from_numpy(l).to(dev)) for x, l in data]
    stages = [Stage(ops, (B,) + hwc, cuts, M, torch.from_numpy(theta), layout.coords(rank)[1], dev) for rank in range(layout.world)]
    slices = emulate_step(stages, layout, batches)
    # the same batches through ordinary single-model steps, averaged over the replicas the same way
    singles, losses = [], []
    for x, l in data:
        bd = Bound(ops, hwc, B, M, cuts, theta, {hpf.OPT_GRAPH: 0})
        bd.upload(x, l)
        losses.append(bd.step())
        singles.append(bd.avg.clone())
    mean = singles[0].clone()
    for g in singles[1:]:
        mean += g
    mean /= R
    for rank, st in enumerate(stages):
        a, n = st.plan.param_first, st.plan.param_count
        assert torch.equal(slices[rank], mean[a:a + n]), (rank, float((slices[rank] - mean[a:a + n]).abs().max()))
    covered = sorted((st.plan.param_first, st.plan.param_count) for st in stages[:P])
    assert covered[0][0] == 0 and all(covered[k][0] + covered[k][1] == covered[k + 1][0] for k in range(P - 1))
    assert covered[-1][0] + covered[-1][1] == theta.size
    # the last partition of every replica holds that replica's losses
    for r in range(R):
        got = stages[layout.rank_of(r, P - 1)].losses().cpu().numpy()
        assert abs(float(got.astype(np.float32).sum() / np.float32(M)) - losses[r]) <= 1e-6 * abs(losses[r])
    # and against the oracle: the mean over replicas of the oracle's averaged gradients
    g_ref = np.mean([ora.step(ops, hwc, theta, x, l, M)["g_avg"] for x, l in data], axis=0)
    full = torch.cat([slices[layout.rank_of(0, p)] for p in range(P)]).cpu().numpy()
    offs, G = wl.param_offsets(ops)
    for i, (w_off, w_cnt, b_off, b_cnt) in enumerate(offs):
        for off, cnt in ((w_off, w_cnt), (b_off, b_cnt)):
            if cnt:
                assert rel_l2(full[off:off + cnt], g_ref[off:off + cnt]) <= TOL_TENSOR, ("op", i)


def test_one_rank_of_the_hybrid_step_is_the_ordinary_step():
    """hybrid.run_step on a world of one rank (one replica, one partition): the same cells, the library's average, no
    neighbour and no allreduce; bit for bit the ordinary step without a CUDA graph."""
    from paper_1911_05146_b200.hybrid import HybridLayout, Stage, SingleRankComm, run_step
    c = wl.config("r11")
    ops, hwc, B, M = c["ops"], c["in_hwc"], c["B"], c["M"]
    x, labels, theta = seeded(ops, hwc, B, seed=2)
    dev = torch.device("cuda:0")
    stage = Stage(ops, (B,) + tuple(hwc), [], M, torch.from_numpy(theta), 0, dev)
    g = run_step(stage, HybridLayout(1, 1), 0, SingleRankComm(), torch.from_numpy(x).to(dev), torch.from_numpy(labels).to(dev))
    bd = Bound(ops, hwc, B, M, [], theta, {hpf.OPT_GRAPH: 0})
    bd.upload(x, labels)
    bd.step()
    assert g.numel() == theta.size and torch.equal(g, bd.avg)


def test_messages_across_cuts_match_the_oracle():
    """Activations sent forward and partial errors sent back (Eq. 7) per cut and micro-batch."""
    ops = wl.resnet_v2_cifar(1)
    cuts = [4, 8, 12]          # mid-block, block edge, mid-block
    B, M = 4, 2
    x, labels, theta = seeded(ops, (32, 32, 3), B, seed=6, bn_jitter=0.2)
    bd = Bound(ops, (32, 32, 3), B, M, cuts, theta, {hpf.OPT_KEEP_MESSAGES: 1})
    bd.upload(x, labels)
    bd.step()
    b = B // M
    for m in range(M):
        r = ora.microbatch(ops, (32, 32, 3), theta, x[m * b:(m + 1) * b], labels[m * b:(m + 1) * b], cuts=cuts)     # the plain oracle
        for (j, k), msg in r["fwd_msg"].items():
            assert rel_l2(bd.message(j, k, m), msg) <= TOL_TENSOR, ("fwd", j, k, m)
        over = [(j, k) for (j, k), msg in r["bwd_msg"].items() if not rel_l2(bd.message(j, k, m, grad=True), msg) <= TOL_TENSOR]
        if over:      # a flipped ReLU decision upstream: those messages are judged under the GPU's in-window decisions
            rm = matched_oracle(bd, m, theta, x, labels, cuts=cuts)
            assert rm["decisions_used"] <= 8, rm["decisions_used"]
            for (j, k) in over:
                assert rel_l2(bd.message(j, k, m, grad=True), rm["bwd_msg"][(j, k)]) <= TOL_TENSOR, ("bwd", j, k, m)
        print("micro-batch %d: partial-error messages beyond the tolerance against the plain oracle: %s" % (m, over))


def test_state_machine_on_a_bound_model():
    c = wl.config("r11")
    x, labels, theta = seeded(c["ops"], c["in_hwc"], c["B"])
    bd = Bound(c["ops"], c["in_hwc"], c["B"], c["M"], c["cuts"], theta)
    bd.upload(x, labels)
    for call in (bd.model.backward, bd.model.grad_average):
        with pytest.raises(hpf.HpfError) as e:
            call()
        assert e.value.status == -3
    bd.model.forward(bd.x, bd.labels)
    with pytest.raises(hpf.HpfError):
        bd.model.grad_average()
    bd.model.backward()
    with pytest.raises(hpf.HpfError):
        bd.model.backward()
    bd.model.grad_average()
    bd.model.synchronize(60000)
    with pytest.raises(hpf.HpfError) as e:
        bd.model.set_option(hpf.OPT_GRAPH, 0)
    assert e.value.status == -3
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    m2 = hpf.Model(c["ops"], (c["B"],) + c["in_hwc"], c["cuts"], c["M"])
    with pytest.raises(hpf.HpfError) as e:
        m2.bind(bd.params, bd.slots, bd.avg, small, bd.streams)
    assert e.value.status == -4
    assert bd.model.launch_count() > 0


def test_training_steps_follow_the_oracle_and_lower_the_loss():
    """Forward + backward + (average and SGD-momentum update), several steps on one batch: the parameters follow the
    oracle's trajectory and the loss falls (the step of Section 5.3 closed by apply_gradients)."""
    c = wl.config("r11")
    ops, hwc, B, M, cuts = c["ops"], c["in_hwc"], c["B"], c["M"], c["cuts"]
    x, labels = wl.draw_inputs(B, hwc, 10)
    theta = wl.draw_params(ops, bn_jitter=0.1)
    bd = Bound(ops, hwc, B, M, cuts, theta)
    bd.upload(x, labels)
    vel = torch.zeros(bd.G, device=bd.dev)
    lr, mu, wd = 0.05, 0.9, 1e-4
    th_ref, v_ref = theta.astype(np.float64), np.zeros(theta.size)
    losses = []
    with pytest.raises(hpf.HpfError):
        bd.model.sgd_momentum_step(vel, lr, mu, wd)          # no backward yet
    for step in range(4):
        bd.model.forward(bd.x, bd.labels)
        bd.model.backward()
        bd.model.sgd_momentum_step(vel, lr, mu, wd)
        losses.append(bd.model.loss())
        bd.model.synchronize(60000)
        r = ora.step(ops, hwc, th_ref, x, labels, M)
        assert abs(losses[-1] - r["loss"]) <= 5e-3 * abs(r["loss"]), (step, losses[-1], r["loss"])
        th_ref, v_ref = ora.sgd_momentum(th_ref, v_ref, r["g_avg"], lr, mu, wd)
        # trajectories drift apart through the ReLU decisions both sides take on their own, so the bound is loose
        assert rel_l2(bd.params.cpu().numpy(), th_ref) <= 2e-3, (step, rel_l2(bd.params.cpu().numpy(), th_ref))
    assert losses[-1] < losses[0], losses
    with pytest.raises(hpf.HpfError):
        bd.model.sgd_momentum_step(vel, -1.0, mu, wd)


def test_pipeline_cells_follow_the_schedule_and_overlap():
    """Section 5.3's pipelining, as it really ran (device timestamps at the start and end of every cell): a cell starts
    only after the cell that feeds it and after the same stage's previous cell, in both directions, and in the steady
    state stage p works on micro-batch m while stage p+1 works on micro-batch m-1."""
    c = wl.config("r110")
    ops, hwc, B, M, cuts = c["ops"], c["in_hwc"], c["B"], c["M"], c["cuts"]
    x, labels, theta = seeded(ops, hwc, B)
    bd = Bound(ops, hwc, B, M, cuts, theta, {hpf.OPT_CELL_TIMES: 1})
    bd.upload(x, labels)
    bd.step(); bd.step()
    P = bd.model.num_partitions()
    fwd, bwd = bd.model.cell_times(0), bd.model.cell_times(1)
    for cells, feeder in ((fwd, -1), (bwd, +1)):
        overlapped, pairs = 0, 0
        for p in range(P):
            for m in range(M):
                s, e = cells[p][m]
                assert e > s
                if 0 <= p + feeder < P:
                    assert s >= cells[p + feeder][m][1], ("a cell started before the cell that feeds it ended", p, m)
                if m > 0:
                    assert s >= cells[p][m - 1][1], ("two cells of one stage overlapped", p, m)
                q = p - feeder                      # the stage this one feeds
                if 0 <= q < P and m > 0:
                    s2, e2 = cells[q][m - 1]
                    pairs += 1
                    overlapped += int(s < e2 and s2 < e)
        assert pairs == (P - 1) * (M - 1)
        assert overlapped >= 0.75 * pairs, (overlapped, pairs)      # the stages do run side by side
    # the forward phase is over before the backward phase starts (fill / drain schedule)
    assert min(s for row in bwd for s, _ in row) >= max(e for row in fwd for _, e in row)
    span = max(e for row in fwd for _, e in row) - min(s for row in fwd for s, _ in row)
    busy = sum(e - s for row in fwd for s, e in row)
    print("forward: %d cells, span %.2f ms, summed cell time %.2f ms (concurrency %.2f)" % (P * M, span / 1e6, busy / 1e6, busy / span))
    assert busy > 1.5 * span                        # more than one stage busy on average


def test_cuts_from_measured_cell_times_run_and_match_the_oracle():
    """The load balancer fed with what the pipeline measures (Section 5.4): the cuts it returns are valid, the step on
    them matches the oracle, and the search reports the timing of every cut list it tried, equal op counts first."""
    from paper_1911_05146_b200.tuner import balance_by_measurement
    ops = wl.resnet_v2_cifar(3)
    B, M, P = 16, 4, 4
    start = wl.default_cuts(len(ops), P)
    theta = torch.from_numpy(wl.draw_params(ops))
    cuts, history = balance_by_measurement(ops, (B, 32, 32, 3), P, M, theta, start, rounds=2, steps=2)
    assert history[0]["cuts"] == start and len(history) >= 1
    assert len(cuts) == P - 1 and all(a < b2 for a, b2 in zip([0] + cuts, cuts + [len(ops)]))
    assert all(len(h["partition_us"]) == P and h["ms"] > 0 for h in history)
    assert min(h["ms"] for h in history) == [h["ms"] for h in history if h["cuts"] == cuts][0]
    check_step(ops, (32, 32, 3), B, M, cuts, seed=14, bn_jitter=0.1, name="cuts from measured cell times %s" % cuts)


def test_microbatch_tuner_returns_the_fastest_candidate():
    from paper_1911_05146_b200.tuner import tune_microbatches, halving_candidates
    c = wl.config("r11")
    theta = torch.from_numpy(wl.draw_params(c["ops"]))
    best, tried = tune_microbatches(c["ops"], (c["B"],) + tuple(c["in_hwc"]), c["cuts"], theta, patience=8, steps=2)
    assert set(tried) == set(halving_candidates(c["B"]))
    assert best in tried and tried[best] == min(tried.values())
    assert all(ms > 0 for ms in tried.values())
