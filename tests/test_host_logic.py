"""Host-side logic of the CUDA library, no GPU needed: the C-ABI exports, the integer bookkeeping
(bit-exact against the oracle's tables), and the error paths that must answer before any launch."""
import ctypes
import os
import re

import pytest

import paper_1911_05146_b200 as hpf
import workloads as wl
from oracle import reference as ora

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "hpf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = sorted(set(re.findall(r"\b(hpf_[a-z_0-9]+)\s*\(", text)))
    assert len(declared) >= 30
    L = hpf.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert set(declared) == set(hpf.binding.EXPORTS)


@pytest.mark.parametrize("name", ["r11", "r110", "r1001", "r152"])
def test_bookkeeping_matches_oracle_bit_exactly(name):
    c = wl.config(name)
    ops, cuts, M, B = c["ops"], c["cuts"], c["M"], c["B"]
    m = hpf.Model(ops, (B,) + c["in_hwc"], cuts, M)
    n = len(ops)
    w_off, w_cnt, b_off, b_cnt, G = ora.param_layout(ops)
    assert m.num_params() == G
    shapes = ora.shapes(ops, c["in_hwc"])
    parts = ora.partition_of_ops(n, cuts)
    step = 1 if n < 400 else 7
    for i in list(range(0, n, step)) + [n - 1]:
        assert m.param_layout(i) == (w_off[i], w_cnt[i], b_off[i], b_cnt[i])
        assert m.op_shape(i) == shapes[i]
        assert m.partition_of_op(i) == parts[i]
    P = m.num_partitions()
    assert P == c["P"]
    for p in range(P):
        lo, hi = m.partition_range(p)
        assert [i for i in range(n) if parts[i] == p] == list(range(lo, hi))
    for mm in range(M):
        assert m.microbatch_range(mm) == ora.microbatch_range(B, M, mm)
    for j, cut in enumerate(cuts):
        live = ora.live_set(ops, cut)
        assert m.boundary_count(j) == len(live)
        for k, t in enumerate(live):
            prod, shp = m.boundary_desc(j, k)
            assert prod == t and shp == (B // M,) + shapes[t]
    for p in range(P):
        for mm in range(M):
            assert m.schedule_tick(p, mm) == ora.schedule_tick(P, M, p, mm)


def test_mid_block_and_one_op_per_partition_cuts():
    ops = wl.resnet_v2_cifar(1)
    n = len(ops)
    for cuts in ([4], [3, 7, 8], list(range(1, n))):
        m = hpf.Model(ops, (4, 32, 32, 3), cuts, 2)
        for j, cut in enumerate(cuts):
            live = ora.live_set(ops, cut)
            assert [m.boundary_desc(j, k)[0] for k in range(m.boundary_count(j))] == live


def _expect(status, fn):
    with pytest.raises(hpf.HpfError) as e:
        fn()
    assert e.value.status == status, e.value


def test_error_paths_answer_on_the_host():
    ops = wl.resnet_v2_cifar(1)
    n = len(ops)
    INVALID, UNSUPPORTED, STATE = -1, -2, -3
    shape = (8, 32, 32, 3)
    _expect(INVALID, lambda: hpf.Model(ops, shape, [0], 2))              # cut out of range
    _expect(INVALID, lambda: hpf.Model(ops, shape, [n], 2))
    _expect(INVALID, lambda: hpf.Model(ops, shape, [5, 5], 2))           # not increasing
    _expect(INVALID, lambda: hpf.Model(ops, shape, [9, 4], 2))
    _expect(INVALID, lambda: hpf.Model(ops, shape, list(range(1, n)) + [n], 2))   # more partitions than ops
    _expect(INVALID, lambda: hpf.Model(ops, shape, [13], 3))             # B % M != 0
    _expect(INVALID, lambda: hpf.Model(ops, shape, [13], 0))
    _expect(INVALID, lambda: hpf.Model(ops, shape, [13], 16))            # M > B
    _expect(INVALID, lambda: hpf.Model(ops[:-1], shape, [13], 2))        # no head
    bad = list(ops); bad[3] = bad[3]._replace(src0=5)                    # not a forward DAG
    _expect(INVALID, lambda: hpf.Model(bad, shape, [13], 2))
    bad = list(ops); bad[8] = bad[8]._replace(src1=2)                    # ADD shape mismatch
    _expect(INVALID, lambda: hpf.Model(bad, shape, [13], 2))
    bad = list(ops); bad[2] = bad[2]._replace(c_in=17)                   # channel mismatch
    _expect(INVALID, lambda: hpf.Model(bad, shape, [13], 2))
    odd = wl.resnet_v2_cifar(1, widths=(6, 12, 24))                      # BN channels not a multiple of 4? 6 -> no
    _expect(UNSUPPORTED, lambda: hpf.Model(odd, shape, [13], 2))
    m = hpf.Model(ops, shape, [13], 2)
    _expect(STATE, lambda: m.forward(0x1000, 0x1000))                    # not bound
    _expect(STATE, lambda: m.backward())
    _expect(STATE, lambda: m.grad_average())
    _expect(STATE, lambda: m.tensor_ptr(0, 0))
    _expect(INVALID, lambda: m.param_layout(n))
    _expect(INVALID, lambda: m.schedule_tick(2, 0))
    _expect(INVALID, lambda: m.boundary_count(1))
    _expect(INVALID, lambda: m.set_option(99, 1))
    assert m.workspace_bytes() > 0
    assert hpf.lib().hpf_strerror(-4) == b"workspace too small or misaligned"


def test_bind_without_a_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    ops = wl.resnet_v2_cifar(1)
    m = hpf.Model(ops, (8, 32, 32, 3), [13], 2)
    h = ctypes.c_void_p * 2
    with pytest.raises(hpf.HpfError) as e:
        hpf.binding._check(hpf.lib().hpf_bind(m._h, 0x1000, 0x1000, 0x1000, 0x1000, m.workspace_bytes(), h(0, 0), 2))
    assert e.value.status == -5      # HPF_ERR_CUDA: there is no CPU fallback


def test_workspace_grows_with_message_buffers():
    ops = wl.resnet_v2_cifar(1)
    a = hpf.Model(ops, (8, 32, 32, 3), [4], 2)
    b = hpf.Model(ops, (8, 32, 32, 3), [4], 2)
    b.set_option(hpf.OPT_KEEP_MESSAGES, 1)
    assert b.workspace_bytes() > a.workspace_bytes()


def test_stage_lanes_multiply_the_stream_slots_and_the_scratch():
    """HPF_OPT_STAGE_LANES: S = P * min(L, M) stream slots, each with scratch of its own, so the workspace grows with L;
    values outside 1..64 are refused.  Host only."""
    c = wl.config("r11")
    B = c["B"]
    m = hpf.Model(c["ops"], (B,) + tuple(c["in_hwc"]), c["cuts"], c["M"])
    P, M = m.num_partitions(), c["M"]
    assert m.num_stream_slots() == P
    one_lane = m.workspace_bytes()
    m.set_option(hpf.OPT_STAGE_LANES, 2)
    assert m.num_stream_slots() == P * min(2, M)
    assert m.workspace_bytes() > one_lane
    m.set_option(hpf.OPT_STAGE_LANES, 64)
    assert m.num_stream_slots() == P * M                   # never more lanes than micro-batches
    for bad in (0, -1, 65):
        with pytest.raises(hpf.HpfError) as e:
            m.set_option(hpf.OPT_STAGE_LANES, bad)
        assert e.value.status == -1
    m.close()


def test_load_balancer_cuts():
    """Section 5.4's load balancer: contiguous partitions minimising the largest modelled partition cost."""
    import itertools
    import numpy as np
    rng = np.random.default_rng(0)
    for n, P in ((6, 2), (7, 3), (9, 4), (8, 8), (5, 1)):
        cost = rng.uniform(0.1, 5.0, n).tolist()
        cuts = hpf.balance_cuts(cost, P)
        assert len(cuts) == P - 1 and all(0 < c < n for c in cuts) and cuts == sorted(set(cuts))
        b = [0] + cuts + [n]
        got = max(sum(cost[b[i]:b[i + 1]]) for i in range(P))
        best = min(max(sum(cost[x:y]) for x, y in zip((0,) + c, c + (n,))) for c in itertools.combinations(range(1, n), P - 1)) if P > 1 else sum(cost)
        assert got <= best * (1 + 1e-9), (cost, cuts, got, best)          # brute force over every cut placement
    with pytest.raises(hpf.HpfError):
        hpf.balance_cuts([1.0, 2.0], 3)                                    # more partitions than ops
    with pytest.raises(hpf.HpfError):
        hpf.balance_cuts([1.0, -2.0, 1.0], 2)
    # the modelled costs of ResNet-1001: 8x8-stage blocks are the dearest, so their partitions get fewer ops
    c = wl.config("r1001")
    costs = hpf.estimate_op_costs(c["ops"], (16, 32, 32, 3))
    assert len(costs) == len(c["ops"]) and min(costs) >= 0
    cuts = hpf.balance_cuts(costs, 8)
    sizes = np.diff([0] + cuts + [len(c["ops"])])
    assert sizes[-1] < sizes[0]
    parts = [sum(costs[a:b]) for a, b in zip([0] + cuts, cuts + [len(c["ops"])])]
    eq = [sum(costs[a:b]) for a, b in zip([0] + c["cuts"], c["cuts"] + [len(c["ops"])])]
    assert max(parts) < max(eq) and max(parts) / min(parts) < 1.05
    m = hpf.Model(c["ops"], (c["B"],) + c["in_hwc"], cuts, c["M"])       # the cuts are accepted by the model
    assert m.num_partitions() == 8


def test_microbatch_tuner_search_order():
    """Section 5.3: pipeline stages range from 1 to the batch size; the search starts at the batch size and halves."""
    from paper_1911_05146_b200.tuner import halving_candidates
    assert halving_candidates(128) == [128, 64, 32, 16, 8, 4, 2, 1]
    assert halving_candidates(12) == [12, 6, 3, 1]
    assert halving_candidates(96, smallest=8) == [96, 48, 24, 12]
    assert halving_candidates(1) == [1]
    for b in (7, 30, 128):
        assert all(b % m == 0 for m in halving_candidates(b))
