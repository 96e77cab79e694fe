"""Hybrid parallelism (partitions on different ranks, replicas side by side): the bookkeeping on CPU.

Two gloo ranks run the real layout / message tables / send-recv order / per-partition allreduce groups of
paper_1911_05146_b200.hybrid with stand-in cells (tests/hybrid_worker.py).  The arithmetic of the hand-offs is checked
on a GPU by tests/test_gpu_step.py (one-process emulation); a run on several GPUs has not been possible yet.
"""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
from paper_1911_05146_b200.hybrid import HybridLayout  # noqa: E402
from hybrid_worker import code  # noqa: E402   (tests/ is on the path: pytest puts it there)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run(P):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(_free_port()), os.path.join(ROOT, "tests", "hybrid_worker.py"), str(P)]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=dict(os.environ, OMP_NUM_THREADS="1"), cwd=ROOT)
    assert out.returncode == 0, out.stderr[-3000:]
    return json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])


def test_layout_maps_ranks_to_replicas_and_partitions():
    lay = HybridLayout(6, 3)
    assert (lay.R, lay.P) == (2, 3)
    assert [lay.coords(r) for r in range(6)] == [(0, 0), (0, 1), (0, 2), (1, 0), (1, 1), (1, 2)]
    assert lay.partition_group(1) == [1, 4]                      # one communicator per partition, one member per replica
    assert [lay.below(r) for r in range(6)] == [None, 0, 1, None, 3, 4]
    assert [lay.above(r) for r in range(6)] == [1, 2, None, 4, 5, None]
    assert all(lay.rank_of(*lay.coords(r)) == r for r in range(6))
    with pytest.raises(ValueError):
        HybridLayout(5, 2)


def test_two_partitions_on_two_ranks_exchange_what_the_tables_say():
    d = _run(2)
    lo, hi = d["ranks"]
    assert lo["coords"] == [0, 0] and hi["coords"] == [0, 1]
    # the cut sits inside a residual block: the trunk and the shortcut cross it forward ...
    assert lo["fwd_send"] == hi["fwd_recv"] and len(hi["fwd_recv"]) == 2 and lo["fwd_recv"] == [] and hi["fwd_send"] == []
    # ... and the partial errors come back, in the same order on both sides
    assert hi["bwd_send"] == lo["bwd_recv"] and len(lo["bwd_recv"]) >= 2 and hi["bwd_recv"] == [] and lo["bwd_send"] == []
    M = 2
    fwd = [e for e in hi["log"] if e[0] == "fwd"]
    assert [e[1] for e in fwd] == list(range(M))
    for _, m, got, whole in fwd:                                 # what partition 1 saw when its forward cell ran
        assert got == [code(1, 0, m, j) for j in range(len(hi["fwd_recv"]))] and all(whole)
    bwd = [e for e in lo["log"] if e[0] == "bwd"]
    assert [e[1] for e in bwd] == list(range(M))
    for _, m, got, whole in bwd:
        assert got == [code(2, 1, m, j) for j in range(len(lo["bwd_recv"]))] and all(whole)
    # the parameter slices of the two partitions tile the flat vector; a lone replica's gradient is left as it is
    (a0, n0), (a1, n1) = lo["param_range"], hi["param_range"]
    assert a0 == 0 and a1 == n0 and a1 + n1 == d["G"]
    assert lo["g0"] == 1.0 and hi["g0"] == 2.0 and lo["count"] == n0 and hi["count"] == n1


def test_two_replicas_average_their_partition_over_its_own_group():
    d = _run(1)
    a, b = d["ranks"]
    assert a["coords"] == [0, 0] and b["coords"] == [1, 0] and a["group"] == [0, 1] == b["group"]
    assert a["g0"] == b["g0"] == 1.5 and a["g_all_equal"] and b["g_all_equal"]      # (1 + 2) / 2 on both replicas
    assert a["count"] == d["G"] and a["fwd_recv"] == a["fwd_send"] == a["bwd_recv"] == a["bwd_send"] == []
