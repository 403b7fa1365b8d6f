"""gnnco_objective_static: the objective for callers that cannot allocate device memory.

A coordination loop that lives inside another program's callback or plug-in interface gets a
probability vector and a place for the per-subgraph loss, and nothing else: it has no
allocator of its own and must not grow the host program's pool.  This entry point serves it
from a fixed scratch array inside the library.  The test calls it through the C ABI twice
in a row, with different inputs, and checks each result against the existing entry point
(gnnco_train_step's loss for the same probabilities) and against the CPU oracle.  This file is collected last on
purpose, so a run that stops at the first failure has already run every other test.
"""
import ctypes

import numpy as np
import pytest

import oracle
import synth_inputs as si
from gpu_common import F32_ATOL, F32_RTOL, load_graph, to_dev

pytestmark = pytest.mark.gpu


def _reference_losses(graph, w, Wd, Xd, pen, lam):
    """Existing entry point: forward-only gnnco_train_step gives (loss, p) for a model."""
    import paper_2511_09261_b200 as gnnco
    model = gnnco.Model(w.dims, Wd)
    loss, p = graph.train_step(model, Xd, w.alpha, w.beta, lam, pen, flags=gnnco.FORWARD_ONLY)
    return loss.clone(), p.clone()


def _within_f32_bound(got, want):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    return np.all(np.abs(got - want) <= F32_ATOL + F32_RTOL * np.abs(want)), float(np.abs(got - want).max())


def test_objective_static_matches_train_step_twice_in_a_row():
    import torch
    import paper_2511_09261_b200 as gnnco
    w = si.make_workload(3)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    book = oracle.bookkeeping(w.n, w.eu, w.ev, w.part, w.S)
    perm = graph.arrays()["perm"].cpu().numpy()
    X = w.features_f32()[perm]
    Xd = to_dev(X)
    pen_np = w.penalty()[perm]
    pen = to_dev(pen_np)
    Wn_a = [w.weights(l) for l in range(w.L)]
    Wn_b = [-0.5 * x for x in Wn_a]
    W_a = [to_dev(x) for x in Wn_a]
    W_b = [to_dev(x) for x in Wn_b]
    loss_a, p_a = _reference_losses(graph, w, W_a, Xd, None, 0.0)
    loss_b, p_b = _reference_losses(graph, w, W_b, Xd, pen, 0.7)
    assert not torch.equal(loss_a, loss_b)
    # the oracle's loss for the same X, W and penalty list (its own forward pass, in double)
    ora_a = oracle.train_step(book, w.dims, X, Wn_a, w.alpha, w.beta, 0.0, None, want_dW=False, threads=4)["loss"]
    ora_b = oracle.train_step(book, w.dims, X, Wn_b, w.alpha, w.beta, 0.7, pen_np, want_dW=False, threads=4)["loss"]
    out = torch.full((w.S,), float("nan"), device=Xd.device)        # caller-provided output
    lib = gnnco.load_library()
    stream = torch.cuda.current_stream().cuda_stream
    for p, pen_t, lam, ref, ora in ((p_a, None, 0.0, loss_a, ora_a), (p_b, pen, 0.7, loss_b, ora_b),
                                    (p_a, None, 0.0, loss_a, ora_a)):
        obj = gnnco.Objective(w.alpha, w.beta, lam, None if pen_t is None else pen_t.data_ptr())
        before = torch.cuda.memory_allocated()
        st = lib.gnnco_objective_static(graph._handle, p.data_ptr(), ctypes.byref(obj), out.data_ptr(), stream)
        assert st == gnnco.OK, gnnco.status_string(st)
        assert torch.cuda.memory_allocated() == before
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        ok, worst = _within_f32_bound(got, ref.cpu().numpy())        # against the existing entry point
        assert ok, worst
        ok, worst = _within_f32_bound(got, ora)                      # and against the oracle
        assert ok, worst


def test_objective_static_with_a_hub_row():
    """A row of 4,499 neighbours: gnnco_train_step sums such a row through its pre-summed segments,
    this entry point lets the row's block sum it, so the two agree to float32 rounding, not bit for bit."""
    import torch
    n = 9000
    half = n // 2
    eu, ev = np.zeros(half - 1, np.int32), np.arange(1, half, dtype=np.int32)
    part = np.zeros(n, np.int32)
    graph = load_graph(n, eu, ev, part, 1)
    book = oracle.bookkeeping(n, eu, ev, part, 1)
    p_np = si.uniform01(31, 0, n).astype(np.float32)
    pen_np = (si.uniform01(32, 0, n) < 0.2).astype(np.float32)
    loss = torch.full((1,), float("nan"), device="cuda:0")
    for _ in range(2):
        graph.objective_static(to_dev(p_np), 2.0, 1.0, 0.3, to_dev(pen_np), loss=loss)
        torch.cuda.synchronize()
        # Eq. 5 with the penalty, written out on the oracle's bookkeeping in double
        pd = p_np.astype(np.float64)
        rows = np.repeat(np.arange(n), np.diff(book["rowptr"]))
        cols = book["colidx"]
        once = rows < cols
        want = 2.0 * float((pd[rows[once]] * pd[cols[once]]).sum()) - float(pd.sum()) + 0.3 * float((pen_np * pd).sum())
        ok, worst = _within_f32_bound(loss.cpu().numpy(), np.array([want]))
        assert ok, worst


def test_objective_static_accepts_exactly_its_maximum_and_rejects_one_more():
    import torch
    import paper_2511_09261_b200 as gnnco
    top = 65_536                                   # GNNCO_STATIC_OBJECTIVE_MAX_ITEMS
    for n, accepted in ((top, True), (top + 1, False), (70_000, False)):
        part = np.arange(n, dtype=np.int32)        # one subgraph per node: n objective work items
        graph = load_graph(n, np.zeros(0, np.int32), np.zeros(0, np.int32), part, n)
        p = torch.full((n,), 0.25, device="cuda:0")
        loss = torch.zeros(n, device="cuda:0")
        if accepted:
            graph.objective_static(p, 2.0, 1.0, loss=loss)
            torch.cuda.synchronize()
            assert torch.equal(loss, torch.full_like(loss, -0.25))      # no edges: loss_s = -beta * p
        else:
            with pytest.raises(gnnco.GnncoError) as e:
                graph.objective_static(p, 2.0, 1.0, loss=loss)
            assert e.value.status == gnnco.WORKSPACE_TOO_SMALL
            assert float(loss.abs().sum()) == 0.0                       # nothing was written
