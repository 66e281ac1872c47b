"""The grouped step inside a CUDA graph: captured once (internal streams included: they fork from
and join the capturing stream through events), replayed, and compared bit for bit with the same
steps enqueued directly.  Launch-bound workloads (many small matrices) replay a step as one graph
launch instead of some eighty kernel launches."""
import pytest
import torch

from paper_2605_16341_b200 import binding as od
from paper_2605_16341_b200 import workloads as wl

from parity_util import poisoned_workspace
from test_gpu_parity import make_problem

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


def _state(shapes):
    hs, Xs, Ms, Gs, Qs = [], [], [], [], []
    for i, (m, n, r) in enumerate(shapes):
        spec, X, M, G, Q = make_problem(m, n, r, BF16, BF16, seed=40 + i)
        hs.append(od.orthdion_create(m, n, r, 0.95, 0.01, 0.0, od.MODE_ORTH))
        Xs.append(X.cuda()); Ms.append(M.cuda()); Gs.append(G.cuda()); Qs.append(Q.cuda())
    return hs, Xs, Ms, Gs, Qs


def test_captured_grouped_step_replays_bit_identically():
    shapes = [(384, 512, 64), (512, 384, 64), (384, 512, 64), (256, 256, 32), (640, 384, 256)]
    # direct: three steps
    hs, Xs, Ms, Gs, Qs = _state(shapes)
    ws = poisoned_workspace(od.orthdion_workspace_bytes_grouped(hs))
    table = od.PointerTable(hs, Xs, Ms, Gs, Qs)
    for _ in range(3):
        od.orthdion_step_grouped(table, ws)
    torch.cuda.synchronize()
    assert od.orthdion_last_status(hs, ws) == [0] * len(hs)
    # captured: one direct step (kernel attributes and internal streams are set up outside the
    # capture), then the step captured once and replayed twice
    hs2, Xs2, Ms2, Gs2, Qs2 = _state(shapes)
    ws2 = poisoned_workspace(od.orthdion_workspace_bytes_grouped(hs2))
    table2 = od.PointerTable(hs2, Xs2, Ms2, Gs2, Qs2)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        od.orthdion_step_grouped(table2, ws2, side)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        od.orthdion_step_grouped(table2, ws2, torch.cuda.current_stream())
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert od.orthdion_last_status(hs2, ws2) == [0] * len(hs2)
    for a, b in zip(Xs + Ms + Qs, Xs2 + Ms2 + Qs2):
        assert torch.equal(a, b)
    for h in hs + hs2:
        od.orthdion_destroy(h)
