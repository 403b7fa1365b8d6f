"""GPU parity on the five benchmark configurations (full sizes, the launch configuration
the benchmark times): bit-exact bookkeeping and decoding, teacher-forced training steps
against the oracle -- whole batch where the oracle finishes in seconds, sampled subgraphs
otherwise."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from gpu_common import (Report, StepCase, assert_close, check_bookkeeping, check_decode, check_stage3, load_graph, pick_parts,
                        sampled_step_check, to_dev)

pytestmark = pytest.mark.gpu


def _train_free(graph, w, Xd, Wd, steps, checkpoints, on_checkpoint):
    """Run ``steps`` optimiser steps on the GPU; before each step listed in ``checkpoints``
    hand the current (W, m, v, t) to ``on_checkpoint``."""
    import torch
    import paper_2511_09261_b200 as gnnco
    model = gnnco.Model(w.dims, Wd, gnnco.BF16 if w.dtype == "bf16" else gnnco.F32)
    opt = gnnco.Adam(model, lr=w.lr)
    first = last = None
    for t in range(steps):
        if t in checkpoints:
            torch.cuda.synchronize()
            on_checkpoint(t, opt)
        loss, _ = graph.train_step(model, Xd, w.alpha, w.beta, opt=opt)
        if t == 0:
            first = loss.clone()
        last = loss
    return first.cpu().numpy(), last.cpu().numpy(), opt


# tensors that meet the flat bound at every checkpoint of a whole-batch configuration (measured; a
# regression that pushes one of them into the group-scaled bound fails the test)
FLAT_ONLY = {1: ("loss", "p", "z", "dW0", "dW1", "dX", "adam m", "adam v", "adam W"),
             2: ("loss", "p", "z", "dW0", "dW1", "dX"),
             3: ("loss", "p", "z", "dW0", "dW1", "dW2", "dX", "adam m", "adam v", "adam W"),
             # sampled full-size configurations: the first layer's gradient of configuration 4 (hub subgraphs,
             # entries in the hundreds) and the wide gradients of the bfloat16 configuration need the
             # group-scaled bound for a few entries
             4: ("loss", "p", "z", "dW1", "dX"),
             5: ("loss", "p", "z", "dW2")}


@pytest.mark.parametrize("idx,checkpoints", [(1, (0, 1, 10, 50, 99)), (2, (0, 1, 10, 50, 499)), (3, (0, 1, 10, 50, 99))])
def test_config_whole_batch(idx, checkpoints):
    w = si.make_workload(idx)
    book = oracle.bookkeeping(w.n, w.eu, w.ev, w.part, w.S)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    check_bookkeeping(graph, book)
    X = w.features_f32()[book["perm"]]
    Xd = to_dev(X)
    Wd = [to_dev(w.weights(l)) for l in range(w.L)]
    case = StepCase(book, w.dims, w.dtype, w.S, w.alpha, w.beta)
    worst = {}

    def on_checkpoint(t, opt):
        Wn = [x.cpu().numpy().copy() for x in Wd]
        adam = dict(lr=w.lr, step=opt.step, m=[x.cpu().numpy().copy() for x in opt.m],
                    v=[x.cpu().numpy().copy() for x in opt.v])
        g, stats = case.run(graph, X, Wn, None, want_dx=True, adam=adam, threads=8, label="%s step %d" % (w.name, t))
        for k, v in stats.items():
            worst[k] = max(worst.get(k, 0), v)
        check_decode(graph, book, g["p"])

    first, last, opt = _train_free(graph, w, Xd, Wd, w.steps, set(checkpoints), on_checkpoint)
    assert np.all(last < first)                  # every subgraph's objective went down
    print("\n%s worst abs errors: %s" % (w.name, {k: float("%.3g" % v) for k, v in worst.items()}))
    print("%s: bound each tensor needed\n%s" % (w.name, case.report))
    # the criteria's flat float32 bound (rtol 1e-4, atol 1e-5) holds for every value tensor, and on
    # these configurations for every gradient and updated weight as well
    for name in FLAT_ONLY[idx]:
        assert case.report.needs_only_flat(name), name
    if idx == 1:
        # free-running trajectory of the small case: the oracle trains on its own for the
        # same number of steps; the drift of the final per-subgraph loss is reported and
        # held to the float32 tolerance
        Wo = [w.weights(l).astype(np.float64) for l in range(w.L)]
        mo = [np.zeros_like(x) for x in Wo]
        vo = [np.zeros_like(x) for x in Wo]
        f32 = lambda x: float(np.float32(x))
        for t in range(1, w.steps + 1):
            r = oracle.train_step(book, w.dims, X, Wo, w.alpha, w.beta, threads=8)
            if t == w.steps:
                break
            for l in range(w.L):
                oracle.adam(Wo[l], mo[l], vo[l], r["dW"][l], f32(w.lr), t, f32(0.9), f32(0.999), f32(1e-8))
        drift = assert_close(last, r["loss"], "f32", "free-running loss after %d steps" % w.steps)
        print("free-running final-loss drift %.3g" % drift)


def test_config2_sixteen_node_subinstances_on_gpu():
    """Three 16-node breadth-first balls of configuration 2, trained as one batch of three
    subgraphs; the decoded sets are scored with integer arithmetic against brute force."""
    import torch
    import paper_2511_09261_b200 as gnnco
    w = si.make_workload(2)
    k, balls = 16, []
    for s in range(w.S):
        if len(balls) == 3:
            break
        members = np.where(w.part == s)[0]
        inside = np.isin(w.eu, members) & np.isin(w.ev, members)
        nb = {}
        for a, c in zip(w.eu[inside].tolist(), w.ev[inside].tolist()):
            nb.setdefault(a, []).append(c)
            nb.setdefault(c, []).append(a)
        nodes, seen = [int(members[0])], {int(members[0])}
        for v in nodes:
            for c in sorted(nb.get(v, [])):
                if c not in seen and len(nodes) < k:
                    seen.add(c)
                    nodes.append(c)
        if len(nodes) == k:
            idx = {v: i for i, v in enumerate(nodes)}
            sel = np.isin(w.eu, nodes) & np.isin(w.ev, nodes)
            balls.append([(idx[a], idx[c]) for a, c in zip(w.eu[sel].tolist(), w.ev[sel].tolist())])
    eu = np.array([a + k * b for b, ball in enumerate(balls) for a, _ in ball], np.int32)
    ev = np.array([c + k * b for b, ball in enumerate(balls) for _, c in ball], np.int32)
    n, S = 3 * k, 3
    part = si.contiguous_partition(n, S)
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    check_bookkeeping(graph, book)
    dims = [16, 8, 1]
    X = si.normal_f32(991, 0, n * 16).reshape(n, 16)
    Wd = [to_dev(si.uniform_f32(992 + l, 0, S * dims[l] * dims[l + 1], -0.5, 0.5).reshape(S, dims[l], dims[l + 1]))
          for l in range(2)]
    model = gnnco.Model(dims, Wd)
    opt = gnnco.Adam(model, lr=1e-2)
    Xd = to_dev(X[book["perm"]])
    for _ in range(300):
        loss, p = graph.train_step(model, Xd, 2.0, 1.0, opt=opt)
    torch.cuda.synchronize()
    ref = check_decode(graph, book, p.cpu().numpy())
    x = ref["x"]
    for b, ball in enumerate(balls):
        nbm = [0] * k
        for a, c in ball:
            nbm[a] |= 1 << c
            nbm[c] |= 1 << a
        best = 0
        for mask in range(1 << k):
            if all(not (nbm[i] & mask) for i in range(k) if (mask >> i) & 1):
                best = max(best, bin(mask).count("1"))
        xs = x[b * k:(b + 1) * k]            # contiguous parts: new order == original order
        conf = sum(1 for a, c in ball if xs[a] and xs[c])
        # dropping one endpoint of every conflict leaves an independent set, which cannot beat the optimum
        keep = xs.copy()
        for a, c in ball:
            if keep[a] and keep[c]:
                keep[c] = 0
        assert not any(keep[a] and keep[c] for a, c in ball) and int(keep.sum()) <= best
        # and the trained, decoded assignment must come close to the optimum of the integer objective
        # alpha * conflicts - beta * |x| (whose minimum is -|MIS| for alpha > beta): within 2 of it
        achieved = 2 * conf - int(xs.sum())
        print("ball %d: objective %d, optimum %d (set %d, conflicts %d)" % (b, achieved, -best, int(xs.sum()), conf))
        assert achieved <= -(best - 2)
    assert ref["boundary_viol"] == 0 and ref["intra_viol"] == sum(
        1 for b, ball in enumerate(balls) for a, c in ball if x[b * k + a] and x[b * k + c])


def _full_size_sampled(idx, steps, n_parts, whole_batch_forward=False):
    import torch
    import paper_2511_09261_b200 as gnnco
    w = si.make_workload(idx)
    book = oracle.bookkeeping(w.n, w.eu, w.ev, w.part, w.S)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    check_bookkeeping(graph, book)
    quality, ref_quality = graph.partition_quality(), oracle.partition_quality(w.eu, w.ev, w.part, w.S)
    assert np.array_equal(quality["in_edges"].cpu().numpy(), ref_quality["in_edges"])
    assert np.array_equal(quality["tot"].cpu().numpy(), ref_quality["tot"])
    np.testing.assert_allclose(float(quality["Q"].item()), ref_quality["Q"], rtol=1e-12)
    arr = graph.arrays()
    bf16 = w.dtype == "bf16"
    if bf16:
        X_orig = torch.from_numpy(w.features_bf16_bits().view(np.int16)).to("cuda:0").view(torch.bfloat16)
    else:
        X_orig = to_dev(w.features_f32())
    Xd = graph.gather_rows(X_orig, arr["perm"])
    del X_orig
    Wd = [to_dev(w.weights(l)) for l in range(w.L)]
    parts = pick_parts(book, n_parts, seed=idx)
    report = Report()
    x_rows = lambda lo, hi: w.features_f32(book["perm"][lo:hi])
    pen = w.penalty()
    pen_new = pen[book["perm"]]
    pen_d = to_dev(pen_new)
    model_opt = gnnco.Adam(gnnco.Model(w.dims, Wd, gnnco.BF16 if bf16 else gnnco.F32), lr=w.lr)
    # step 0: every oracle input comes from the generators
    stats, loss, p = sampled_step_check(graph, book, w.dims, w.dtype, Xd, Wd, parts, x_rows,
                                        lambda l, s: w.weights(l, [s])[0], w.alpha, w.beta, w.lam, pen_d,
                                        lambda lo, hi: pen_new[lo:hi], model_opt, True, "%s step 0" % w.name, report)
    print("\n%s step 0, %d subgraphs, worst abs errors: %s" % (w.name, len(parts), {k: float("%.3g" % v) for k, v in stats.items()}))
    if whole_batch_forward:
        # every subgraph, forward only: loss, p and z of the whole batch against the oracle
        ref = oracle.train_step(book, w.dims, w.features_f32()[book["perm"]], [w.weights(l) for l in range(w.L)],
                                w.alpha, w.beta, w.lam, pen_new, want_dW=False, threads=16)
        assert_close(loss.cpu().numpy(), ref["loss"], w.dtype, "whole-batch loss", report=report, name="loss")
        assert_close(p.cpu().numpy(), ref["p"], w.dtype, "whole-batch p", report=report, name="p")
        del ref
    check_decode(graph, book, p.cpu().numpy())
    check_stage3(graph, book, p.cpu().numpy(), policy_seed=7)
    # free-run, then one teacher-forced step from the GPU's current weights
    model = gnnco.Model(w.dims, Wd, gnnco.BF16 if bf16 else gnnco.F32)
    for _ in range(steps - 2):
        graph.train_step(model, Xd, w.alpha, w.beta, w.lam, pen_d, model_opt)
    torch.cuda.synchronize()
    snap = {(l, s): Wd[l][s].cpu().numpy().copy() for l in range(w.L) for s in parts}
    stats, loss, p = sampled_step_check(graph, book, w.dims, w.dtype, Xd, Wd, parts, x_rows,
                                        lambda l, s: snap[(l, s)], w.alpha, w.beta, w.lam, pen_d,
                                        lambda lo, hi: pen_new[lo:hi], model_opt, True,
                                        "%s step %d" % (w.name, steps - 1), report)
    print("%s last step worst abs errors: %s" % (w.name, {k: float("%.3g" % v) for k, v in stats.items()}))
    print("%s: bound each tensor needed\n%s" % (w.name, report))
    for name in FLAT_ONLY[idx]:
        assert report.needs_only_flat(name), name
    d = check_decode(graph, book, p.cpu().numpy())
    assert d["set_size"] > 0
    conf, _, _ = check_stage3(graph, book, p.cpu().numpy(), policy_seed=8)
    print("%s conflicts after the last step: %d of %d boundary edges" % (w.name, conf.size, graph.E_b))


def test_config4_full_size_sampled_subgraphs():
    _full_size_sampled(4, steps=20, n_parts=64, whole_batch_forward=True)


def test_config5_full_size_sampled_subgraphs():
    _full_size_sampled(5, steps=5, n_parts=64)


def test_config5_full_size_one_kernel_layers_against_the_plain_step():
    """GNNCO_ONE_KERNEL_LAYERS at the full size of configuration 5 (every CTA pair walks hundreds of double
    tiles of dozens of subgraphs; the tiles around the hubs go through the separate kernels): two training steps
    with the flag against two plain steps, whose parity with the oracle the test above establishes.  Subgraphs
    without a row of more than 256 neighbours must agree bit for bit in loss and p; the others (the plain step
    sums such rows inline at this size, the flagged step by segments) within the bfloat16 bound."""
    import torch
    import paper_2511_09261_b200 as gnnco
    from gpu_common import BF16_RTOL, BF16_ATOL
    w = si.make_workload(5)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    arr = graph.arrays()
    X_orig = torch.from_numpy(w.features_bf16_bits().view(np.int16)).to("cuda:0").view(torch.bfloat16)
    Xd = graph.gather_rows(X_orig, arr["perm"])
    del X_orig
    runs = []
    for extra in (0, gnnco.ONE_KERNEL_LAYERS):
        Wd = [to_dev(w.weights(l)) for l in range(w.L)]
        model = gnnco.Model(w.dims, Wd, gnnco.BF16)
        opt = gnnco.Adam(model, lr=w.lr)
        for _ in range(2):
            loss, p = graph.train_step(model, Xd, w.alpha, w.beta, flags=extra, opt=opt)
        torch.cuda.synchronize()
        assert graph.async_status() == 0
        runs.append((loss.clone(), p.clone()))
        del Wd, model, opt
    (loss_a, p_a), (loss_b, p_b) = runs
    rowptr, part_ptr = arr["rowptr"].long(), arr["part_ptr"].long()
    deg = rowptr[1:] - rowptr[:-1]
    node_part = arr["node_part"].long()
    long_parts = torch.zeros(w.S, dtype=torch.bool, device=deg.device)
    long_parts[node_part[deg > 256]] = True
    assert 0 < int(long_parts.sum()) < w.S // 4
    short = ~long_parts
    assert torch.equal(loss_a[short], loss_b[short])
    assert torch.equal(p_a[short[node_part]], p_b[short[node_part]])
    assert torch.allclose(p_a, p_b, rtol=BF16_RTOL, atol=BF16_ATOL)
    assert torch.allclose(loss_a, loss_b, rtol=BF16_RTOL, atol=BF16_ATOL * float(loss_a.abs().max()))
