"""GPU parity of the Stage-3 glue (Section 3.3; Algorithm 1, Stage 3): conflict list,
base action, actions -> penalty list / active subgraphs (bit-exact against the oracle),
and the fine-tuning step that updates active subgraphs only."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import tiny_graph, rand_weights, rand_features
from gpu_common import check_stage3, load_graph, to_dev

pytestmark = pytest.mark.gpu


def _levels(n, seed, levels=(0.2, 0.6, 0.9)):
    """Probabilities on a few levels only: many conflicts join endpoints with equal p."""
    return np.array(levels, np.float32)[(si.u64(seed, 0, n) % np.uint64(len(levels))).astype(int)]


@pytest.mark.parametrize("name,n,prob,S", [("random_parts", 300, 0.05, 7), ("many_parts", 500, 0.03, 61),
                                           ("every_node_own_part", 80, 0.1, 80), ("one_part", 120, 0.08, 1),
                                           ("several_tiles", 6000, 0.004, 13)])
def test_stage3_glue_small(name, n, prob, S):
    eu, ev, part = tiny_graph(n, prob, S, seed=31)
    S = max(S, int(part.max()) + 1)
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    if name == "several_tiles":
        assert book["bnd_u"].size > 2 * 4096 + 17          # three compaction tiles with a ragged tail
    for seed, p in [(1, _levels(n, 41)), (2, si.uniform01(42, 0, n).astype(np.float32)),
                    (3, np.full(n, 0.5, np.float32)), (4, np.zeros(n, np.float32))]:
        check_stage3(graph, book, p, policy_seed=50 + seed)


def test_stage3_glue_without_boundary_edges():
    import torch
    eu, ev, part = tiny_graph(100, 0.08, 1, seed=5)
    book = oracle.bookkeeping(100, eu, ev, part, 1)
    graph = load_graph(100, eu, ev, part, 1)
    assert graph.E_b == 0
    d = graph.decode_boundary(to_dev(np.full(100, 0.9, np.float32)))
    ca = graph.conflict_actions(d["viol"], to_dev(np.full(100, 0.9, np.float32)))
    ap = graph.apply_actions(ca["conflict_idx"], ca["action"], ca["count"])
    torch.cuda.synchronize()
    assert int(ca["count"].item()) == 0 and int(ap["chosen"].item()) == 0
    assert not ap["pen"].any().item() and not ap["active"].any().item()


def test_unaligned_flag_pointer():
    """The flag array may start at any byte address."""
    import torch
    eu, ev, part = tiny_graph(4000, 0.005, 9, seed=33)
    book = oracle.bookkeeping(4000, eu, ev, part, 9)
    graph = load_graph(4000, eu, ev, part, 9)
    p = _levels(4000, 43)
    ref = oracle.decode(book, p)
    conf = oracle.conflict_list(book, ref["viol"])
    buf = torch.zeros(graph.E_b + 3, dtype=torch.uint8, device="cuda")
    view = buf[3:]
    view.copy_(to_dev(ref["viol"]))
    ca = graph.conflict_actions(view, to_dev(p))
    torch.cuda.synchronize()
    C = int(ca["count"].item())
    assert C == conf.size
    assert np.array_equal(ca["conflict_idx"].cpu().numpy()[:C], conf)
    assert np.array_equal(ca["action"].cpu().numpy()[:C], oracle.base_action(book, conf, p))


def test_fine_tune_updates_active_subgraphs_only():
    """One fine-tuning step with the penalty list and the active mask of the base action:
    active subgraphs match the oracle's Adam fed the same gradient, the others keep
    weights and moments bit for bit; the loss carries the penalty term."""
    import torch
    import paper_2511_09261_b200 as gnnco
    n, S, dims = 400, 9, [16, 8, 1]
    eu, ev, part = tiny_graph(n, 0.04, S, seed=35)
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    X = rand_features(n, dims[0], 3).astype(np.float32)
    W = [w.astype(np.float32) for w in rand_weights(dims, S, 4, scale=1.5)]
    Xn = X[book["perm"]]
    Xd, Wd = to_dev(Xn), [to_dev(w) for w in W]
    model = gnnco.Model(dims, Wd)
    loss0, p0 = graph.train_step(model, Xd, 2.0, 1.0, flags=gnnco.FORWARD_ONLY)
    p = p0.cpu().numpy()
    conf, act, ap = check_stage3(graph, book, p)
    active = ap["active"].cpu().numpy()
    if not (0 < active.sum() < S):                      # make sure both kinds of subgraph occur
        active = np.zeros(S, np.uint8); active[::2] = 1
        ap["active"].copy_(to_dev(active))
    opt = gnnco.Adam(model, lr=1e-2)
    opt.active = ap["active"]
    before = [w.clone() for w in Wd]
    dW = [torch.zeros_like(w) for w in Wd]
    lam = 3.0
    loss, _ = graph.train_step(model, Xd, 2.0, 1.0, lam, ap["pen"], opt, dW=dW)
    torch.cuda.synchronize()
    pen = ap["pen"].cpu().numpy()
    ref = oracle.train_step(book, dims, Xn, W, 2.0, 1.0, lam, pen)
    np.testing.assert_allclose(loss.cpu().numpy(), ref["loss"], rtol=1e-4, atol=1e-5)
    for l in range(len(dims) - 1):
        g = dW[l].cpu().numpy().astype(np.float64)
        for s in range(S):
            got = Wd[l][s].cpu().numpy()
            if not active[s]:
                assert np.array_equal(got, before[l][s].cpu().numpy())
                assert not opt.m[l][s].any().item() and not opt.v[l][s].any().item()
                continue
            w = W[l][s].astype(np.float64).copy()
            m = np.zeros_like(w); v = np.zeros_like(w)
            oracle.adam(w, m, v, np.ascontiguousarray(g[s]), float(np.float32(1e-2)), 1, float(np.float32(0.9)),
                        float(np.float32(0.999)), float(np.float32(1e-8)))
            np.testing.assert_allclose(got, w, rtol=1e-4, atol=5e-7 * max(1.0, np.abs(w).max()))
    # shared weights cannot be restricted to some subgraphs
    shared = gnnco.Model(dims, [to_dev(w[:1].copy()) for w in W])
    opt2 = gnnco.Adam(shared)
    opt2.active = ap["active"]
    with pytest.raises(gnnco.GnncoError) as e:
        graph.train_step(shared, Xd, 2.0, 1.0, opt=opt2)
    assert e.value.status == gnnco.INVALID_ARGUMENT


@pytest.mark.parametrize("dtype,dims,n,S,one_kernel", [("f32", [48, 24, 1], 900, 7, False),
                                                       ("f32", [128, 128, 64, 1], 3000, 9, False),
                                                       ("bf16", [256, 256, 256, 1], 6000, 11, False),
                                                       ("bf16", [256, 256, 256, 1], 6000, 11, True),
                                                       ("bf16", [64, 32, 1], 700, 5, False)])
def test_active_only_step_equals_the_full_step_on_active_subgraphs(dtype, dims, n, S, one_kernel):
    """A fine-tuning step restricted to the active subgraphs (gnnco_active_plan + GNNCO_ACTIVE_ONLY): loss, p, z,
    dW, dX and the updated weights and moments of every ACTIVE subgraph are bit-identical to those of a full
    step with the same Adam mask; everything that belongs to an inactive subgraph keeps the value it had
    before the step (checked with canaries); with every subgraph active the step equals the plain one."""
    import torch
    import paper_2511_09261_b200 as gnnco
    from helpers import tiny_graph, rand_weights, rand_features
    eu, ev, part = tiny_graph(n, 8.0 / n, S, seed=41)
    part[part == 2] = 3                                         # an empty subgraph
    graph = load_graph(n, eu, ev, part, S)
    pp = graph.arrays()["part_ptr"].cpu().numpy()
    bf16 = dtype == "bf16"
    tdt = torch.bfloat16 if bf16 else torch.float32
    X = rand_features(n, dims[0], 3).astype(np.float32)
    X = to_dev(si.round_to_bf16(X) if bf16 else X, tdt)
    pen = to_dev((si.uniform01(5, 0, n) < 0.2).astype(np.float32))
    L = len(dims) - 1
    for flags_np in (np.array([(s * 7 + 3) % 3 == 0 for s in range(S)], np.uint8), np.ones(S, np.uint8),
                     np.zeros(S, np.uint8)):
        active = to_dev(flags_np)
        outs = []
        for only in (False, True):
            W = [to_dev(w.astype(np.float32)) for w in rand_weights(dims, S, 13, scale=1.5)]
            model = gnnco.Model(dims, W, gnnco.BF16 if bf16 else gnnco.F32)
            opt = gnnco.Adam(model, lr=1e-2)
            opt.active = active
            # one full step first so that the Adam moments are not zero, then the step under test
            graph.train_step(model, X, 2.0, 1.0, 0.5, pen, opt)
            canary = 1024.0
            loss = torch.full((S,), canary, device=X.device)
            p = torch.full((n,), canary, device=X.device)
            z = torch.full((n,), canary, device=X.device)
            dW = [torch.full_like(w, canary) for w in W]
            dX = torch.full_like(X, canary)
            flags = gnnco.WANT_DX | (gnnco.ONE_KERNEL_LAYERS if one_kernel else 0)   # the plan has its own tables for it
            if only:
                assert graph.active_plan(active) == int(flags_np.sum())
                flags |= gnnco.ACTIVE_ONLY
            graph.train_step(model, X, 2.0, 1.0, 0.5, pen, opt, loss=loss, p=p, z=z, dW=dW, dX=dX, flags=flags)
            torch.cuda.synchronize()
            assert graph.async_status() == 0
            outs.append(dict(loss=loss, p=p, z=z, dW=dW, dX=dX, W=[w.clone() for w in W], m=[t.clone() for t in opt.m],
                             v=[t.clone() for t in opt.v]))
        full, act = outs
        for s in range(S):
            lo, hi = int(pp[s]), int(pp[s + 1])
            if flags_np[s] and hi > lo:
                assert torch.equal(full["loss"][s], act["loss"][s])
                for key in ("p", "z", "dX"):
                    assert torch.equal(full[key][lo:hi], act[key][lo:hi]), (key, s)
                for l in range(L):
                    assert torch.equal(full["dW"][l][s], act["dW"][l][s]), ("dW", l, s)
            elif not flags_np[s]:
                assert float(act["loss"][s]) == 1024.0
                for key in ("p", "z", "dX"):
                    assert bool((act[key][lo:hi].float() == 1024.0).all()), (key, s)
                for l in range(L):
                    assert bool((act["dW"][l][s] == 1024.0).all())
            for l in range(L):
                for key in ("W", "m", "v"):
                    assert torch.equal(full[key][l][s], act[key][l][s]), (key, l, s)


def test_active_only_needs_a_matching_plan():
    import torch
    import paper_2511_09261_b200 as gnnco
    from helpers import tiny_graph, rand_weights, rand_features
    n, S, dims = 300, 4, [16, 8, 1]
    eu, ev, part = tiny_graph(n, 0.03, S, seed=43)
    graph = load_graph(n, eu, ev, part, S)
    X = to_dev(rand_features(n, dims[0], 3).astype(np.float32))
    W = [to_dev(w.astype(np.float32)) for w in rand_weights(dims, S, 13)]
    model = gnnco.Model(dims, W)
    opt = gnnco.Adam(model, lr=1e-2)
    opt.active = to_dev(np.ones(S, np.uint8))
    with pytest.raises(gnnco.GnncoError) as e:                  # no plan yet
        graph.train_step(model, X, 2.0, 1.0, opt=opt, flags=gnnco.ACTIVE_ONLY)
    assert e.value.status == gnnco.INVALID_ARGUMENT
    graph.active_plan(opt.active)
    graph.train_step(model, X, 2.0, 1.0, opt=opt, flags=gnnco.ACTIVE_ONLY)
    opt.active = to_dev(np.ones(S, np.uint8))                   # other flags than the plan's
    with pytest.raises(gnnco.GnncoError) as e:
        graph.train_step(model, X, 2.0, 1.0, opt=opt, flags=gnnco.ACTIVE_ONLY)
    assert e.value.status == gnnco.INVALID_ARGUMENT
    with pytest.raises(gnnco.GnncoError):                       # no optimiser
        graph.train_step(model, X, 2.0, 1.0, flags=gnnco.ACTIVE_ONLY)
