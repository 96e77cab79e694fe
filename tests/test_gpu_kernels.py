"""Single kernels through the C ABI against the oracle: the convolution sweep shapes (forward, data
gradient, weight gradient; tensor-core and CUDA-core paths), BN+ReLU forward/backward on ragged
sizes, the gradient average."""
import numpy as np
import pytest
import torch

import paper_1911_05146_b200 as hpf
import workloads as wl
from oracle import reference as ora
from hpf_testlib import rel_l2, TOL_TENSOR

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(DEV)


def _conv_case(ks, st, ci, co, H, N, path, seed=0):
    pad = 1 if ks == 3 else (3 if ks == 7 else 0)
    rng = np.random.Generator(np.random.PCG64(1000 + seed))
    x = rng.standard_normal((N, H, H, ci)).astype(np.float32)
    w = (rng.standard_normal((co, ks, ks, ci)) * np.sqrt(2.0 / (ci * ks * ks))).astype(np.float32)
    P = (H + 2 * pad - ks) // st + 1
    dy = rng.standard_normal((N, P, P, co)).astype(np.float32)
    dx_, dw_, dy_ = _dev(x), _dev(w), _dev(dy)
    scratch = torch.zeros(hpf.conv_scratch_bytes(N, H, H, ci, co, ks, st, pad), dtype=torch.uint8, device=DEV)
    y = torch.full((N, P, P, co), float("nan"), device=DEV)
    gx = torch.full((N, H, H, ci), float("nan"), device=DEV)
    gw = torch.full((co, ks, ks, ci), float("nan"), device=DEV)
    wprep = torch.empty(4 * dw_.numel(), device=DEV)
    args = (N, H, H, ci, co, ks, st, pad, path)
    hpf.conv_prepare_weights(dw_, wprep, ci, co, ks)
    hpf.conv_fwd(dx_, dw_, wprep, y, *args, scratch)
    hpf.conv_dgrad(dy_, dw_, wprep, gx, *args, scratch)
    hpf.conv_wgrad(dx_, dy_, gw, *args, scratch)
    torch.cuda.synchronize()
    status = scratch[-256:-248].view(torch.int32).cpu().tolist()
    assert status == [0, 0], status          # no bounded wait gave up
    e_f = rel_l2(y.cpu().numpy(), ora.conv_fwd(x, w, st, pad))
    e_d = rel_l2(gx.cpu().numpy(), ora.conv_dgrad(dy, w, x.shape, st, pad))
    e_w = rel_l2(gw.cpu().numpy(), ora.conv_wgrad(x, dy, ks, st, pad))
    return e_f, e_d, e_w


@pytest.mark.parametrize("shape", wl.conv_sweep_shapes(), ids=lambda s: "k%d_s%d_%dto%d_at%d" % s)
@pytest.mark.parametrize("path", [0, 2])
def test_conv_sweep_tensor_core_path(shape, path):
    """Sweep shapes at batch 6 (spans several tiles and a ragged tail of the pixel tiling).
    path 0: three-pass TF32, fp32-class accuracy; path 2: one TF32 pass, inside the parity tolerance."""
    ks, st, ci, co, H = shape
    try:
        e = _conv_case(ks, st, ci, co, H, N=6, path=path)
    except hpf.HpfError as err:
        assert err.status == -2
        pytest.fail("sweep shape not covered by the tensor-core kernels: %s" % (shape,))
    assert max(e) <= (2e-5 if path == 0 else TOL_TENSOR), e
    if path == 2:
        assert min(e) > 1e-5          # it really is the 11-bit path


def _wgrad_case(ks, st, ci, co, H, N, path, seed=0):
    pad = 1 if ks == 3 else 0
    rng = np.random.Generator(np.random.PCG64(2000 + seed))
    x = rng.standard_normal((N, H, H, ci)).astype(np.float32)
    P = (H + 2 * pad - ks) // st + 1
    dy = rng.standard_normal((N, P, P, co)).astype(np.float32)
    scratch = torch.zeros(hpf.conv_scratch_bytes(N, H, H, ci, co, ks, st, pad), dtype=torch.uint8, device=DEV)
    gw = torch.full((co, ks, ks, ci), float("nan"), device=DEV)
    hpf.conv_wgrad(_dev(x), _dev(dy), gw, N, H, H, ci, co, ks, st, pad, path, scratch)
    torch.cuda.synchronize()
    assert scratch[-256:-248].view(torch.int32).cpu().tolist() == [0, 0]
    return rel_l2(gw.cpu().numpy(), ora.conv_wgrad(x, dy, ks, st, pad)), gw


@pytest.mark.parametrize("shape", [(1, 1, 64, 16, 32), (3, 1, 16, 16, 32), (3, 1, 64, 64, 8), (1, 2, 64, 32, 32), (3, 1, 128, 128, 14), (1, 1, 48, 16, 8),
                                   (1, 1, 512, 2048, 7), (3, 1, 512, 512, 7), (1, 2, 256, 512, 56), (3, 1, 64, 64, 56), (1, 1, 16, 16, 4)],
                         ids=lambda s: "k%d_s%d_%dto%d_at%d" % s)
@pytest.mark.parametrize("passes", [3, 1])
def test_weight_gradient_kernels_agree(shape, passes):
    """The weight gradient has two tensor-core kernels: one hands the TMA tiles (pixels x channels) to the tensor core as
    MN-major operands as they land, the other transposes them in shared memory first (kept as a cross-check, and for
    channel counts like 48 that the first does not take).  Both against the oracle; with three passes they agree to
    fp32 rounding with each other."""
    ks, st, ci, co, H = shape
    N = 6 if H <= 32 else 2
    e_direct, g_direct = _wgrad_case(ks, st, ci, co, H, N, 0 if passes == 3 else 2)
    e_transp, g_transp = _wgrad_case(ks, st, ci, co, H, N, 3 if passes == 3 else 4)
    tol = 2e-5 if passes == 3 else TOL_TENSOR
    assert e_direct <= tol and e_transp <= tol, (e_direct, e_transp)
    if passes == 3:
        assert rel_l2(g_direct.cpu().numpy(), g_transp.cpu().numpy()) <= 1e-5
    else:
        assert e_direct > 1e-5 and e_transp > 1e-5          # both really are 11-bit paths


@pytest.mark.parametrize("shape", [(1, 1, 64, 16, 32), (3, 1, 16, 16, 32), (1, 1, 16, 64, 32), (1, 2, 64, 32, 32)],
                         ids=lambda s: "k%d_s%d_%dto%d_at%d" % s)
def test_conv_launches_of_several_waves_use_two_tiles_per_cta(shape):
    """Batch 80 at 32x32: 640 pixel tiles, more than two CTAs per SM can hold at once, so the forward and data-gradient
    launches give each CTA two tiles (the second tile's loads under the first tile's write-out)."""
    ks, st, ci, co, H = shape
    e = _conv_case(ks, st, ci, co, H, N=80, path=0)
    assert max(e) <= 2e-5, e


@pytest.mark.parametrize("shape", wl.conv_sweep_shapes(), ids=lambda s: "k%d_s%d_%dto%d_at%d" % s)
def test_conv_sweep_at_batch_128_sampled_against_the_oracle(shape):
    """Configuration 2 in the launch configuration the sweep benchmark times (batch 128, three-pass path: several tiles per
    CTA, K splits and channel slices as the planner chooses them at that size).  Forward and data gradient are independent
    per image, so the oracle recomputes three sampled images; the weight gradient sums over the batch, so the oracle
    recomputes it whole."""
    ks, st, ci, co, H = shape
    N, pad = 128, (1 if ks == 3 else 0)
    rng = np.random.Generator(np.random.PCG64(4242 + ks * 1000 + ci + 7 * co + H))
    x = rng.standard_normal((N, H, H, ci)).astype(np.float32)
    w = (rng.standard_normal((co, ks, ks, ci)) * np.sqrt(2.0 / (ci * ks * ks))).astype(np.float32)
    P = (H + 2 * pad - ks) // st + 1
    dy = rng.standard_normal((N, P, P, co)).astype(np.float32)
    dx_, dw_, dy_ = _dev(x), _dev(w), _dev(dy)
    scratch = torch.zeros(hpf.conv_scratch_bytes(N, H, H, ci, co, ks, st, pad), dtype=torch.uint8, device=DEV)
    y = torch.full((N, P, P, co), float("nan"), device=DEV)
    gx = torch.full((N, H, H, ci), float("nan"), device=DEV)
    gw = torch.full((co, ks, ks, ci), float("nan"), device=DEV)
    wprep = torch.empty(4 * dw_.numel(), device=DEV)
    args = (N, H, H, ci, co, ks, st, pad, 0)
    hpf.conv_prepare_weights(dw_, wprep, ci, co, ks)
    for _ in range(2):                      # twice: tickets of K-split launches must be left clean
        hpf.conv_fwd(dx_, dw_, wprep, y, *args, scratch)
        hpf.conv_dgrad(dy_, dw_, wprep, gx, *args, scratch)
        hpf.conv_wgrad(dx_, dy_, gw, *args, scratch)
    torch.cuda.synchronize()
    assert scratch[-256:-248].view(torch.int32).cpu().tolist() == [0, 0]
    yh, gxh = y.cpu().numpy(), gx.cpu().numpy()
    assert np.isfinite(yh).all() and np.isfinite(gxh).all()
    for n in (0, 77, 127):
        assert rel_l2(yh[n:n + 1], ora.conv_fwd(x[n:n + 1], w, st, pad)) <= 2e-5, ("fwd", n)
        assert rel_l2(gxh[n:n + 1], ora.conv_dgrad(dy[n:n + 1], w, (1, H, H, ci), st, pad)) <= 2e-5, ("dgrad", n)
    assert rel_l2(gw.cpu().numpy(), ora.conv_wgrad(x, dy, ks, st, pad)) <= 5e-5


@pytest.mark.parametrize("shape", [(3, 1, 64, 64, 56), (1, 1, 256, 64, 56), (1, 2, 256, 128, 56), (3, 1, 128, 128, 28),
                                   (1, 1, 128, 512, 28), (3, 1, 256, 256, 14), (1, 2, 1024, 512, 14), (3, 1, 512, 512, 7),
                                   (1, 1, 512, 2048, 7), (1, 1, 2048, 512, 7)],
                         ids=lambda s: "k%d_s%d_%dto%d_at%d" % s)
def test_conv_imagenet_layout_map_sizes_on_the_tensor_core_path(shape):
    """Feature maps 56, 28, 14 and 7 pixels wide (the 224x224 layout): pixel boxes that are not multiples of 32 pixels
    (weight gradient: zero-padded tile rows) and ragged box rows."""
    ks, st, ci, co, H = shape
    e = _conv_case(ks, st, ci, co, H, N=3, path=0)
    # fp32 accumulation over up to 9*512 products: the error grows with the length of the sum (3e-5 at K = 4608)
    assert max(e) <= 5e-5, e


@pytest.mark.parametrize("shape", [(1, 1, 16, 64, 32), (3, 1, 32, 32, 16), (1, 2, 128, 64, 16), (3, 1, 3, 16, 32),
                                   (7, 2, 3, 64, 32), (3, 2, 5, 7, 9), (1, 1, 12, 20, 5)],
                         ids=lambda s: "k%d_s%d_%dto%d_at%d" % s)
def test_conv_cuda_core_path(shape):
    ks, st, ci, co, H = shape
    e = _conv_case(ks, st, ci, co, H, N=3, path=1)
    assert max(e) <= 1e-5, e          # fp32 FMA: far inside the tolerance


def test_conv_bad_arguments():
    s = torch.zeros(1024, dtype=torch.uint8, device=DEV)
    with pytest.raises(hpf.HpfError) as e:
        hpf.conv_fwd(s, s, s, s, 1, 4, 4, 3, 8, 5, 1, 0, 1, s)      # window larger than the input
    assert e.value.status == -1
    with pytest.raises(hpf.HpfError) as e:
        hpf.conv_fwd(s, s, s, s, 1, 8, 8, 3, 8, 3, 1, 1, 0, s)      # 3 channels: no tensor-core kernel
    assert e.value.status == -2


@pytest.mark.parametrize("rows,C", [(1, 4), (7, 12), (5, 16), (1000, 16), (4096 + 37, 64), (16384, 16), (16384, 64), (4096, 32),
                                    (4096, 128), (1024, 64), (1024, 256), (50, 2048), (131072, 16), (8192, 256), (65536 + 11, 64),
                                    (3000, 2048), (40000, 96), (784, 2048), (200, 1024), (32768, 16), (999, 4),
                                    (131072, 64), (60000 + 3, 128), (262144 + 5, 32), (16384 + 1, 512)])
def test_bnrelu_fwd_bwd(rows, C):
    rng = np.random.Generator(np.random.PCG64(rows * 7 + C))
    x = (rng.standard_normal((rows, C)) * 2 + 3).astype(np.float32)       # mean >> 0: the cancellation case
    dy = rng.standard_normal((rows, C)).astype(np.float32)
    gamma = (1 + 0.3 * rng.standard_normal(C)).astype(np.float32)
    beta = (0.3 * rng.standard_normal(C)).astype(np.float32)
    addend = rng.standard_normal((rows, C)).astype(np.float32)
    eps = 1e-5
    scratch = torch.zeros(hpf.bnrelu_scratch_bytes(rows, C), dtype=torch.uint8, device=DEV)
    dx_, ddy, dg, db, dadd = _dev(x), _dev(dy), _dev(gamma), _dev(beta), _dev(addend)
    y = torch.empty_like(dx_); stats = torch.empty(2 * C, device=DEV)
    for _ in range(2):          # twice: the block ticket must be left clean
        hpf.bnrelu_fwd(dx_, dg, db, eps, y, stats, rows, C, scratch)
    torch.cuda.synchronize()
    mean, var = ora.bn_stats(x)
    if rows > 1:
        assert rel_l2(stats[:C].cpu().numpy(), mean) <= 1e-5
        assert rel_l2(stats[C:].cpu().numpy(), 1 / np.sqrt(var + eps)) <= 1e-4
    y_ref = ora.bnrelu_fwd(x, gamma, beta, eps)
    assert rel_l2(y.cpu().numpy(), y_ref) <= 1e-4
    gx = torch.full_like(dx_, float("nan")); ggam = torch.empty(C, device=DEV); gbet = torch.empty(C, device=DEV)
    hpf.bnrelu_bwd(dx_, ddy, dg, db, stats, gx, None, 0, ggam, gbet, rows, C, scratch)
    torch.cuda.synchronize()
    rx, rg, rb = ora.bnrelu_bwd(x, dy, gamma, beta, eps)
    if rows > 8:
        assert rel_l2(gx.cpu().numpy(), rx) <= 1e-3
        assert rel_l2(ggam.cpu().numpy(), rg) <= 1e-3 and rel_l2(gbet.cpu().numpy(), rb) <= 1e-3
    # accumulate + addend: dx_total = existing + dx + addend
    base = gx.clone()
    hpf.bnrelu_bwd(dx_, ddy, dg, db, stats, gx, dadd, 1, ggam, gbet, rows, C, scratch)
    torch.cuda.synchronize()
    assert torch.allclose(gx, base + base + dadd, rtol=1e-5, atol=1e-5)
    assert hpf.bnrelu_status(scratch) is False           # no bounded wait gave up; the scratch is fit for the next call


def test_bnrelu_rejects_odd_channels():
    s = torch.zeros(4096, dtype=torch.uint8, device=DEV)
    with pytest.raises(hpf.HpfError) as e:
        hpf.bnrelu_fwd(s, s, s, 1e-5, s, s, 10, 6, s)
    assert e.value.status == -2


@pytest.mark.parametrize("M,G", [(1, 5), (3, 1023), (8, 4096 * 33 + 2), (4, 1 << 20)])
def test_grad_average_flat(M, G):
    rng = np.random.Generator(np.random.PCG64(M * 100 + 1))
    slots = rng.standard_normal((M, G)).astype(np.float32)
    d = _dev(slots); out = torch.empty(G, device=DEV)
    hpf.grad_average_flat(d, out, M, G)
    torch.cuda.synchronize()
    acc = slots[0].copy()
    for m in range(1, M):
        acc += slots[m]
    assert np.array_equal(out.cpu().numpy(), acc * np.float32(1.0 / M))      # fixed ascending order, bit-exact
    assert rel_l2(out.cpu().numpy(), ora.grad_average(slots)) <= 1e-6


@pytest.mark.parametrize("M,G", [(1, 7), (8, 4096 * 33 + 2), (4, 1 << 20)])
@pytest.mark.parametrize("mu,wd", [(0.0, 0.0), (0.9, 1e-4)])
def test_sgd_momentum_flat(M, G, mu, wd):
    """Average + parameter update in one kernel (Section 5.3, apply_gradients) against the fp64 oracle, two steps."""
    rng = np.random.Generator(np.random.PCG64(M * 10 + G % 97))
    theta = rng.standard_normal(G).astype(np.float32)
    vel = np.zeros(G, dtype=np.float32)
    d_theta, d_vel, d_avg = _dev(theta), _dev(vel), torch.empty(G, device=DEV)
    th_ref, v_ref = theta.astype(np.float64), np.zeros(G)
    for step in range(2):
        slots = rng.standard_normal((M, G)).astype(np.float32)
        hpf.sgd_momentum_flat(_dev(slots), d_avg, d_theta, d_vel, M, G, 0.05, mu, wd)
        torch.cuda.synchronize()
        gbar = ora.grad_average(slots)
        th_ref, v_ref = ora.sgd_momentum(th_ref, v_ref, gbar, 0.05, mu, wd)
        assert rel_l2(d_avg.cpu().numpy(), gbar) <= 1e-6
        assert rel_l2(d_theta.cpu().numpy(), th_ref) <= 1e-6
        assert rel_l2(d_vel.cpu().numpy(), v_ref) <= 1e-5
    # gbar may be omitted
    before = d_theta.clone()
    hpf.sgd_momentum_flat(_dev(np.zeros((M, G), dtype=np.float32)), None, d_theta, torch.zeros(G, device=DEV), M, G, 0.05, 0.0, 0.0)
    torch.cuda.synchronize()
    assert torch.equal(before, d_theta)          # zero gradient, no decay, no velocity: nothing moves
