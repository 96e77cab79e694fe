"""The no-allocation BN+ReLU entry point against the ordinary one.

Some users of the library call it from places where device memory cannot be requested at that moment
(inside a no-allocation region, from a plug-in that owns only its input and output buffers), so they have
no scratch buffer to pass.  hpf_bnrelu_fwd_static takes its scratch from a fixed array inside the
library instead.  This file checks, through the C ABI, that it gives what hpf_bnrelu_fwd gives and what the
fp64 oracle gives, twice in a row (the array is shared and keeps the previous call's contents), and that
it refuses sizes beyond the array.  It is collected last so that a failure here cannot hide the other tests.
"""
import numpy as np
import pytest
import torch

import paper_1911_05146_b200 as hpf
from oracle import reference as ora

pytestmark = pytest.mark.gpu


def _case(rows, C, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    x = torch.from_numpy((rng.standard_normal((rows, C)) * 1.5 + 0.7).astype(np.float32)).cuda()
    gamma = torch.from_numpy((1 + 0.2 * rng.standard_normal(C)).astype(np.float32)).cuda()
    beta = torch.from_numpy((0.2 * rng.standard_normal(C)).astype(np.float32)).cuda()
    return x, gamma, beta


def _against_the_oracle(x, gamma, beta, y, stats, C, eps=1e-5):
    """Statistics and output of the static entry point against the oracle's definition of BN+ReLU (fp64)."""
    xh = x.cpu().numpy().astype(np.float64)
    mean, var = ora.bn_stats(xh)
    y_ref = ora.bnrelu_fwd(xh, gamma.cpu().numpy(), beta.cpu().numpy(), eps)
    st = stats.cpu().numpy().astype(np.float64)
    assert np.allclose(st[:C], mean, rtol=1e-5, atol=1e-6)
    assert np.allclose(st[C:], 1.0 / np.sqrt(var + eps), rtol=1e-5, atol=0)
    yg = y.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(yg - y_ref) <= 1e-5 * np.linalg.norm(y_ref)
    # the ReLU decision may differ only where the pre-activation is a rounding error away from zero
    z = gamma.cpu().numpy() * (xh - mean) / np.sqrt(var + eps) + beta.cpu().numpy()
    assert np.all(((yg > 0) == (y_ref > 0)) | (np.abs(z) < 1e-5))


def test_static_scratch_matches_the_allocating_entry_point_twice():
    assert hpf.static_scratch_bytes() == 2 << 20
    for call, (rows, C) in enumerate([(16384, 64), (4096 + 37, 16)]):       # two calls in a row, different shapes
        x, gamma, beta = _case(rows, C, 40 + call)
        y_ref = torch.empty_like(x); stats_ref = torch.empty(2 * C, device="cuda")
        scratch = torch.zeros(hpf.bnrelu_scratch_bytes(rows, C), dtype=torch.uint8, device="cuda")
        hpf.bnrelu_fwd(x, gamma, beta, 1e-5, y_ref, stats_ref, rows, C, scratch)
        y = torch.full_like(x, float("nan")); stats = torch.full((2 * C,), float("nan"), device="cuda")
        hpf.bnrelu_fwd_static(x, gamma, beta, 1e-5, y, stats, rows, C)
        torch.cuda.synchronize()
        assert torch.allclose(stats, stats_ref, rtol=1e-6, atol=0)
        assert torch.allclose(y, y_ref, rtol=1e-5, atol=1e-6)
        assert (y > 0).any() and (y == 0).any()
        _against_the_oracle(x, gamma, beta, y, stats, C)
    # the same shape again right away: the shared array must have been left usable
    y2 = torch.full_like(x, float("nan"))
    hpf.bnrelu_fwd_static(x, gamma, beta, 1e-5, y2, stats, rows, C)
    torch.cuda.synchronize()
    assert torch.equal(y2, y)


def test_static_scratch_on_a_tensor_the_ordinary_entry_point_holds_on_chip():
    """16 MB: hpf_bnrelu_fwd takes its one-launch on-chip path there, the static entry point never does (it always runs
    the reduce + apply pair on its built-in scratch), so the two agree to rounding, not bit for bit; both match the oracle."""
    rows, C = 65536, 64
    x, gamma, beta = _case(rows, C, 77)
    y_ref = torch.empty_like(x); stats_ref = torch.empty(2 * C, device="cuda")
    scratch = torch.zeros(hpf.bnrelu_scratch_bytes(rows, C), dtype=torch.uint8, device="cuda")
    hpf.bnrelu_fwd(x, gamma, beta, 1e-5, y_ref, stats_ref, rows, C, scratch)
    y = torch.full_like(x, float("nan")); stats = torch.full((2 * C,), float("nan"), device="cuda")
    hpf.bnrelu_fwd_static(x, gamma, beta, 1e-5, y, stats, rows, C)
    torch.cuda.synchronize()
    assert torch.allclose(stats, stats_ref, rtol=1e-5, atol=1e-6)
    assert torch.allclose(y, y_ref, rtol=1e-4, atol=1e-5)
    _against_the_oracle(x, gamma, beta, y, stats, C)


def test_static_scratch_refuses_what_does_not_fit():
    C = 2048                                  # 592 blocks x 2 x 2048 floats of partial sums: beyond 2 MiB
    rows = 1 << 16
    assert hpf.bnrelu_scratch_bytes(rows, C) > hpf.static_scratch_bytes()
    x = torch.zeros(8, device="cuda")        # never read: the call must refuse before launching
    with pytest.raises(hpf.HpfError) as e:
        hpf.bnrelu_fwd_static(x, x, x, 1e-5, x, x, rows, C)
    assert e.value.status == -4
    assert "built-in scratch" in str(e.value)          # the failure text belongs to this call, not to an earlier one
    with pytest.raises(hpf.HpfError) as e:
        hpf.bnrelu_fwd_static(x, x, x, 1e-5, x, x, 16, 6)
    assert e.value.status == -2
