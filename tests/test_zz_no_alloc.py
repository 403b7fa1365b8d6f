"""gnnco_objective_static: the objective for callers that cannot allocate device memory.

A coordination loop that lives inside another program's callback or plug-in interface gets a
probability vector and a place for the per-subgraph loss, and nothing else: it has no
allocator of its own and must not grow the host program's pool.  This entry point serves it
from a fixed scratch array inside the library.  The test calls it through the C ABI twice
in a row, with different inputs, and checks each result against the existing entry point
(gnnco_train_step's loss for the same probabilities).  This file is collected last on
purpose, so a run that stops at the first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest

import synth_inputs as si
from gpu_common import F32_ATOL, F32_RTOL, load_graph, to_dev

pytestmark = pytest.mark.gpu


def _reference_losses(graph, w, Wd, Xd, pen, lam):
    """Existing entry point: forward-only gnnco_train_step gives (loss, p) for a model."""
    import paper_2511_09261_b200 as gnnco
    model = gnnco.Model(w.dims, Wd)
    loss, p = graph.train_step(model, Xd, w.alpha, w.beta, lam, pen, flags=gnnco.FORWARD_ONLY)
    return loss.clone(), p.clone()


def test_objective_static_matches_train_step_twice_in_a_row():
    import torch
    import paper_2511_09261_b200 as gnnco
    w = si.make_workload(3)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    perm = graph.arrays()["perm"].cpu().numpy()
    Xd = to_dev(w.features_f32()[perm])
    pen = to_dev(w.penalty()[perm])
    W_a = [to_dev(w.weights(l)) for l in range(w.L)]
    W_b = [to_dev(-0.5 * w.weights(l)) for l in range(w.L)]
    loss_a, p_a = _reference_losses(graph, w, W_a, Xd, None, 0.0)
    loss_b, p_b = _reference_losses(graph, w, W_b, Xd, pen, 0.7)
    assert not torch.equal(loss_a, loss_b)
    out = torch.full((w.S,), float("nan"), device=Xd.device)        # caller-provided output
    lib = gnnco.load_library()
    stream = torch.cuda.current_stream().cuda_stream
    for p, pen_t, lam, ref in ((p_a, None, 0.0, loss_a), (p_b, pen, 0.7, loss_b), (p_a, None, 0.0, loss_a)):
        obj = gnnco.Objective(w.alpha, w.beta, lam, None if pen_t is None else pen_t.data_ptr())
        before = torch.cuda.memory_allocated()
        st = lib.gnnco_objective_static(graph._handle, p.data_ptr(), ctypes.byref(obj), out.data_ptr(), stream)
        assert st == gnnco.OK, gnnco.status_string(st)
        assert torch.cuda.memory_allocated() == before
        torch.cuda.synchronize()
        got, want = out.cpu().numpy().astype(np.float64), ref.cpu().numpy().astype(np.float64)
        tol = F32_ATOL * max(1.0, float(np.abs(want).max())) + F32_RTOL * np.abs(want)
        assert np.all(np.abs(got - want) <= tol), float(np.abs(got - want).max())


def test_objective_static_rejects_graphs_beyond_its_fixed_scratch():
    import torch
    import paper_2511_09261_b200 as gnnco
    n = gnnco.load_library() and 70_000          # one subgraph per node: 70,000 work items > 65,536
    part = np.arange(n, dtype=np.int32)
    graph = load_graph(n, np.zeros(0, np.int32), np.zeros(0, np.int32), part, n)
    p = torch.full((n,), 0.5, device="cuda:0")
    loss = torch.zeros(n, device="cuda:0")
    with pytest.raises(gnnco.GnncoError) as e:
        graph.objective_static(p, 2.0, 1.0, loss=loss)
    assert e.value.status == gnnco.WORKSPACE_TOO_SMALL
    assert float(loss.abs().sum()) == 0.0          # nothing was written
