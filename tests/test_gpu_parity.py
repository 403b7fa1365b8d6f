"""GPU parity: the CUDA library, called through its C ABI binding, against the CPU oracle
on the same seeded inputs -- bit-exact for integer outputs, within the stated tolerances
for floating point."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import tiny_graph, rand_weights, rand_features
from gpu_common import StepCase, check_bookkeeping, check_decode, load_graph, to_dev

pytestmark = pytest.mark.gpu


def _star_plus_isolated(n):
    """Node 0 joined to every node of the first half (a hub row of length n/2-1), second
    half isolated."""
    half = n // 2
    eu = np.zeros(half - 1, np.int32)
    ev = np.arange(1, half, dtype=np.int32)
    return eu, ev


GRAPHS = {
    "er_random_parts": lambda: tiny_graph(200, 0.06, 7, seed=3),
    "one_part": lambda: tiny_graph(150, 0.08, 1, seed=4),
    "every_node_own_part": lambda: tiny_graph(64, 0.1, 64, seed=5),
    "empty_parts": lambda: (lambda g: (g[0], g[1], np.where(g[2] == 3, 2, g[2]).astype(np.int32)))(
        tiny_graph(120, 0.08, 6, seed=6)),
    "hub_and_isolated": lambda: _star_plus_isolated(300) + (np.zeros(300, np.int32),),
    "big_hub": lambda: _star_plus_isolated(1100) + (np.zeros(1100, np.int32),),     # hub row of 549 entries
    "huge_hub": lambda: _star_plus_isolated(9000) + (np.zeros(9000, np.int32),),   # hub row of 4499 entries (block-summed)
    "no_edges": lambda: (np.zeros(0, np.int32), np.zeros(0, np.int32), si.contiguous_partition(50, 4)),
    "dense_small": lambda: tiny_graph(90, 0.5, 2, seed=8, contiguous=True),
    "dense_medium": lambda: tiny_graph(400, 0.5, 2, seed=9, contiguous=True),    # every row has about 100 neighbours
}


def _n_S(part):
    return part.size, int(part.max()) + 1


@pytest.mark.parametrize("name", sorted(GRAPHS))
def test_bookkeeping_and_decode_small(name):
    eu, ev, part = GRAPHS[name]()
    n, S = _n_S(part)
    if name == "empty_parts":
        S = 6
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    check_bookkeeping(graph, book)
    p = si.uniform01(17, 0, n).astype(np.float32)
    p[::5] = 0.5
    check_decode(graph, book, p)
    check_decode(graph, book, np.full(n, 0.5, np.float32))
    check_decode(graph, book, np.zeros(n, np.float32))


@pytest.mark.parametrize("name", sorted(GRAPHS))
def test_partition_quality_small(name):
    eu, ev, part = GRAPHS[name]()
    n, S = _n_S(part)
    if name == "empty_parts":
        S = 6
    graph = load_graph(n, eu, ev, part, S)
    ref = oracle.partition_quality(eu, ev, part, S)
    got = graph.partition_quality()
    assert np.array_equal(got["in_edges"].cpu().numpy(), ref["in_edges"])
    assert np.array_equal(got["tot"].cpu().numpy(), ref["tot"])
    np.testing.assert_allclose(float(got["Q"].item()), ref["Q"], rtol=1e-12, atol=1e-15)


def test_partition_load_rejects_bad_graphs():
    import paper_2511_09261_b200 as gnnco
    part = np.zeros(4, np.int32)
    cases = [
        (np.array([0, 1, 2], np.int32), np.array([1, 2, 2], np.int32), part, 1, gnnco.NOT_SIMPLE_GRAPH),
        (np.array([0, 1], np.int32), np.array([1, 0], np.int32), part, 1, gnnco.NOT_SIMPLE_GRAPH),
        (np.array([0], np.int32), np.array([7], np.int32), part, 1, gnnco.OUT_OF_RANGE),
        (np.array([0], np.int32), np.array([1], np.int32), np.array([0, 0, 3, 0], np.int32), 2, gnnco.OUT_OF_RANGE),
        (np.array([0, 2], np.int32), np.array([2, 0], np.int32), np.array([0, 0, 1, 1], np.int32), 2,
         gnnco.NOT_SIMPLE_GRAPH),
    ]
    for eu, ev, pt, S, code in cases:
        with pytest.raises(gnnco.GnncoError) as e:
            load_graph(pt.size, eu, ev, pt, S)
        assert e.value.status == code


STEP_CASES = [
    ("er_random_parts", [5, 1], None, 0.0),
    ("er_random_parts", [6, 4, 1], None, 0.7),
    ("er_random_parts", [7, 5, 3, 1], None, 0.0),
    ("er_random_parts", [64, 32, 1], None, 0.5),
    ("er_random_parts", [20, 12, 8, 1], 1, 0.5),
    ("one_part", [128, 64, 1], None, 0.0),
    ("one_part", [16, 8, 1], 1, 1.0),
    ("every_node_own_part", [8, 4, 1], None, 0.0),
    ("empty_parts", [12, 12, 1], None, 0.3),
    ("hub_and_isolated", [32, 16, 1], None, 0.0),
    ("hub_and_isolated", [256, 8, 1], None, 0.0),
    ("big_hub", [32, 16, 1], None, 0.0),
    ("big_hub", [128, 8, 1], None, 0.0),
    ("big_hub", [256, 12, 1], None, 0.4),
    ("huge_hub", [16, 8, 1], None, 0.3),
    ("no_edges", [4, 4, 1], None, 0.0),
    ("dense_small", [24, 40, 1], None, 0.2),
    ("dense_small", [130, 70, 1], None, 0.0),
]


@pytest.mark.parametrize("name,dims,sets,lam", STEP_CASES)
def test_train_step_small_f32(name, dims, sets, lam):
    eu, ev, part = GRAPHS[name]()
    n, S = _n_S(part)
    if name == "empty_parts":
        S = 6
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    X = rand_features(n, dims[0], 11).astype(np.float32)
    nsets = S if sets is None else sets
    W = [w.astype(np.float32) for w in rand_weights(dims, nsets, 13, scale=1.5)]
    pen = (si.uniform01(7, 0, n) < 0.3).astype(np.float32) if lam else None
    case = StepCase(book, dims, "f32", nsets, lam=lam)
    adam = dict(lr=1e-3, step=3, m=[0.01 * rand_weights(dims, nsets, 21)[l].astype(np.float32) for l in range(len(W))],
                v=[np.square(0.02 * rand_weights(dims, nsets, 22)[l]).astype(np.float32) for l in range(len(W))])
    g, stats = case.run(graph, X, W, pen, want_dx=True, adam=adam, label=name)
    check_decode(graph, book, g["p"])


@pytest.mark.parametrize("dims,sets", [([16, 8, 1], None), ([64, 32, 16, 1], None), ([256, 256, 1], None),
                                       ([32, 16, 1], 1), ([6, 1], None), ([128, 64, 1], None),
                                       ([64, 256, 128, 1], None), ([256, 256, 256, 1], None), ([128, 128, 1], 1),
                                       ([64, 64, 64, 1], None)])
def test_train_step_small_bf16(dims, sets):
    eu, ev, part = tiny_graph(260, 0.05, 5, seed=9)
    n, S = _n_S(part)
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    X = si.round_to_bf16(rand_features(n, dims[0], 11).astype(np.float32))
    nsets = S if sets is None else sets
    W = [si.round_to_bf16(w.astype(np.float32)) for w in rand_weights(dims, nsets, 13, scale=1.5)]
    case = StepCase(book, dims, "bf16", nsets, lam=0.4)
    pen = (si.uniform01(7, 0, n) < 0.3).astype(np.float32)
    adam = dict(lr=1e-3, step=1, m=[np.zeros_like(w) for w in W], v=[np.zeros_like(w) for w in W])
    case.run(graph, X, W, pen, want_dx=True, adam=adam, label="bf16")


@pytest.mark.parametrize("name,dims", [("big_hub", [64, 16, 1]), ("huge_hub", [128, 64, 1]), ("hub_and_isolated", [64, 64, 8, 1])])
def test_train_step_bf16_with_hub_rows(name, dims):
    """bfloat16 on graphs whose hub row goes through the block-per-segment aggregation (plain and
    rank-1 mode) and the pre-summed long rows of the width-1 kernels."""
    eu, ev, part = GRAPHS[name]()
    n, S = _n_S(part)
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    X = si.round_to_bf16(rand_features(n, dims[0], 11).astype(np.float32))
    W = [si.round_to_bf16(w.astype(np.float32)) for w in rand_weights(dims, S, 13, scale=1.5)]
    case = StepCase(book, dims, "bf16", S)
    case.run(graph, X, W, None, want_dx=True, label=name + "-bf16")


def test_forward_only_matches_full_step_and_skips_update():
    import torch
    import paper_2511_09261_b200 as gnnco
    eu, ev, part = tiny_graph(200, 0.06, 7, seed=3)
    n, S = _n_S(part)
    graph = load_graph(n, eu, ev, part, S)
    dims = [16, 8, 1]
    X = to_dev(rand_features(n, 16, 1).astype(np.float32))
    W = [to_dev(w.astype(np.float32)) for w in rand_weights(dims, S, 2)]
    W0 = [w.clone() for w in W]
    model = gnnco.Model(dims, W)
    opt = gnnco.Adam(model)
    l1, p1 = graph.train_step(model, X, 2.0, 1.0, opt=opt, flags=gnnco.FORWARD_ONLY)
    l1, p1 = l1.clone(), p1.clone()
    assert opt.step == 1 and all(torch.equal(a, b) for a, b in zip(W, W0))
    l2, p2 = graph.train_step(model, X, 2.0, 1.0, opt=None)
    assert torch.equal(l1, l2) and torch.equal(p1, p2)
    assert all(torch.equal(a, b) for a, b in zip(W, W0))          # opt=None: gradients only
    graph.train_step(model, X, 2.0, 1.0, opt=opt)
    assert opt.step == 2 and not torch.equal(W[0], W0[0])


def test_step_is_deterministic_run_to_run():
    import torch
    import paper_2511_09261_b200 as gnnco
    w = si.make_workload(3)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    perm = graph.arrays()["perm"].cpu().numpy()
    X = to_dev(w.features_f32()[perm])
    outs = []
    for _ in range(2):
        W = [to_dev(w.weights(l)) for l in range(w.L)]
        model = gnnco.Model(w.dims, W)
        dW = [torch.empty_like(t) for t in W]
        dX = torch.empty_like(X)
        loss, p = graph.train_step(model, X, 2.0, 1.0, dW=dW, dX=dX, flags=gnnco.WANT_DX)
        outs.append([loss.clone(), p.clone(), dX.clone()] + [d.clone() for d in dW])
    for a, b in zip(*outs):
        assert torch.equal(a, b)


@pytest.mark.parametrize("cfg", [1, 3])
def test_cached_first_aggregation_is_bit_identical(cfg):
    """Three Adam steps with the first layer's aggregated input stored on step 1 and
    reused afterwards equal three plain steps bit for bit; bad flag combinations are refused."""
    import torch
    import paper_2511_09261_b200 as gnnco
    w = si.make_workload(cfg)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    perm = graph.arrays()["perm"].cpu().numpy()
    X = to_dev(w.features_f32()[perm])
    runs = []
    for cached in (False, True):
        W = [to_dev(w.weights(l)) for l in range(w.L)]
        model = gnnco.Model(w.dims, W)
        opt = gnnco.Adam(model, lr=1e-2)
        cache = torch.empty_like(X) if cached else None
        trace = []
        for step in range(3):
            flags = gnnco.WANT_DX
            if cached:
                flags |= gnnco.AX_STORE if step == 0 else gnnco.AX_REUSE
            dX = torch.empty_like(X)
            loss, p = graph.train_step(model, X, 2.0, 1.0, opt=opt, dX=dX, flags=flags, ax_cache=cache)
            trace += [loss.clone(), p.clone(), dX]
        runs.append(trace + [t.clone() for t in W])
    for a, b in zip(*runs):
        assert torch.equal(a, b)
    W = [to_dev(w.weights(l)) for l in range(w.L)]
    model = gnnco.Model(w.dims, W)
    for flags, cache in ((gnnco.AX_STORE, None), (gnnco.AX_STORE | gnnco.AX_REUSE, torch.empty_like(X))):
        with pytest.raises(gnnco.GnncoError) as e:
            graph.train_step(model, X, 2.0, 1.0, flags=flags, ax_cache=cache)
        assert e.value.status == gnnco.INVALID_ARGUMENT


@pytest.mark.parametrize("dims,n,S", [([256, 256, 1], 3100, 5), ([256, 256, 256, 1], 3100, 5),
                                      ([256, 256, 256, 1], 70000, 24)])
def test_one_kernel_layers_equal_the_separate_kernels_bit_for_bit(dims, n, S):
    """GNNCO_ONE_KERNEL_LAYERS, width 256 in bfloat16: a hidden layer runs as ONE kernel (the aggregated rows
    are summed on chip into the MMA operand).  It adds a row's sources in the order of the stand-alone
    aggregation kernel, so where no row is long enough for that kernel to sum it by segments the step must
    give the bits of the plain step: loss, p, dX and the weights after two Adam steps.  The large case gives
    every CTA pair several double tiles and several subgraphs (ring wrap-around, weight reloads)."""
    import torch
    import paper_2511_09261_b200 as gnnco
    eu, ev, part = tiny_graph(n, float(S) / n, S, seed=131)     # about one neighbour inside the subgraph per row
    graph = load_graph(n, eu, ev, part, S)
    assert graph.max_row <= 256
    X = to_dev(rand_features(n, dims[0], 137).astype(np.float32)).to(torch.bfloat16)
    runs = []
    for extra in (gnnco.ONE_KERNEL_LAYERS, 0):
        W = [to_dev(si.round_to_bf16(w.astype(np.float32))) for w in rand_weights(dims, S, 139)]
        model = gnnco.Model(dims, W, feat_dtype=gnnco.BF16)
        opt = gnnco.Adam(model, lr=1e-2)
        trace = []
        before = graph.launch_count()
        for step in range(2):
            dX = torch.empty_like(X)
            loss, p = graph.train_step(model, X, 2.0, 1.0, opt=opt, dX=dX, flags=gnnco.WANT_DX | extra)
            trace += [loss.clone(), p.clone(), dX]
        runs.append(trace + [t.clone() for t in W] + [graph.launch_count() - before])
    assert runs[0][-1] < runs[1][-1]                 # the flag really replaced launches
    for a, b in zip(runs[0][:-1], runs[1][:-1]):
        assert torch.equal(a, b)


@pytest.mark.parametrize("graph_name,dims", [("big_hub", [256, 256, 1]), ("big_hub", [256, 256, 256, 1]),
                                             ("dense_small", [256, 256, 256, 1]), ("dense_medium", [256, 256, 1]), ("empty_parts", [256, 256, 1]),
                                             ("no_edges", [256, 256, 1])])
def test_one_kernel_layers_against_the_oracle(graph_name, dims):
    """The same flag on graphs with a hub row (its double tile goes through the separate kernels, the others
    through the one-kernel layer) and on a small dense-ish graph, against the oracle."""
    import paper_2511_09261_b200 as gnnco
    eu, ev, part = GRAPHS[graph_name]()
    n, S = _n_S(part)
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    X = si.round_to_bf16(rand_features(n, dims[0], 31).astype(np.float32))
    W = [si.round_to_bf16(w.astype(np.float32)) for w in rand_weights(dims, S, 37)]
    case = StepCase(book, dims, "bf16", S)
    case.extra_flags = gnnco.ONE_KERNEL_LAYERS
    case.run(graph, X, W, None, want_dx=True, label="one-kernel")


def test_weight_copies_left_by_adam_are_bit_identical_to_fresh_ones():
    """bfloat16 run: with GNNCO_WEIGHTS_UNTOUCHED the step reuses the bfloat16 weight copies that the
    previous step's Adam kernel wrote; four steps (the third with only some subgraphs active, then a
    forward-only step) equal the same steps without the flag bit for bit."""
    import torch
    import paper_2511_09261_b200 as gnnco
    eu, ev, part = tiny_graph(700, 0.02, 5, seed=29)
    n, S = _n_S(part)
    graph = load_graph(n, eu, ev, part, S)
    dims = [256, 256, 128, 1]
    X = to_dev(si.round_to_bf16(rand_features(n, dims[0], 11).astype(np.float32)), torch.bfloat16)
    active = to_dev(np.array([1, 0, 1, 1, 0], np.uint8))
    runs = []
    for reuse in (0, gnnco.WEIGHTS_UNTOUCHED):
        W = [to_dev(si.round_to_bf16(w.astype(np.float32))) for w in rand_weights(dims, S, 13, scale=1.5)]
        model = gnnco.Model(dims, W, gnnco.BF16)
        opt = gnnco.Adam(model, lr=1e-2)
        trace = []
        for step in range(4):
            opt.active = active if step == 2 else None
            dX = torch.empty_like(X)
            loss, p = graph.train_step(model, X, 2.0, 1.0, opt=opt, dX=dX, flags=gnnco.WANT_DX | reuse)
            trace += [loss.clone(), p.clone(), dX]
        loss, p = graph.train_step(model, X, 2.0, 1.0, flags=gnnco.FORWARD_ONLY | reuse)
        runs.append(trace + [loss.clone(), p.clone()] + [t.clone() for t in W] + [t.clone() for t in opt.m])
    torch.cuda.synchronize()
    assert graph.async_status() == 0
    for a, b in zip(*runs):
        assert torch.equal(a, b)


@pytest.mark.parametrize("cfg", [1, 3])
def test_steps_replayed_from_a_cuda_graph_equal_eager_steps(cfg):
    """With the Adam step counter on the device (gnnco_adam_state.step_dev) a step depends on no host value that
    changes between steps: ONE step plus its decode, recorded once by stream capture, replayed five times, gives
    the bits of five eager steps (loss, p, weights, moments, decode counts), and the counter reads 5.  The same
    five eager steps with the counter on the host give those bits too."""
    import torch
    import paper_2511_09261_b200 as gnnco
    w = si.make_workload(cfg)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    perm = graph.arrays()["perm"].cpu().numpy()
    X = to_dev(w.features_f32()[perm])
    pen = to_dev(w.penalty()[perm])
    loss, p = torch.empty(w.S, device=X.device), torch.empty(w.n, device=X.device)
    counts = torch.zeros(3, dtype=torch.int64, device=X.device)
    x = torch.empty(w.n, dtype=torch.uint8, device=X.device)
    viol = torch.empty(graph.E_b, dtype=torch.uint8, device=X.device)
    per_part = torch.empty(w.S, dtype=torch.int32, device=X.device)

    def fresh(device_step):
        W = [to_dev(w.weights(l)) for l in range(w.L)]
        model = gnnco.Model(w.dims, W)
        return W, model, gnnco.Adam(model, lr=w.lr, device_step=device_step)

    def one(model, opt, stream=None):
        graph.train_step(model, X, w.alpha, w.beta, w.lam, pen, opt, loss=loss, p=p, stream=stream)
        graph.decode_boundary(p, 0.5, x=x, viol=viol, per_part=per_part, counts=counts, stream=stream)

    results = []
    for mode in ("host counter", "device counter", "graph"):
        W, model, opt = fresh(mode != "host counter")
        if mode == "graph":
            side = torch.cuda.Stream()
            with torch.cuda.stream(side):
                W0, model0, opt0 = fresh(True)
                one(model0, opt0, side)                  # everything lazy happens outside the capture
                torch.cuda.synchronize()
                g = torch.cuda.CUDAGraph()
                g.capture_begin()
                one(model, opt, side)
                g.capture_end()
            torch.cuda.synchronize()
            for _ in range(5):
                g.replay()
        else:
            for _ in range(5):
                one(model, opt)
        torch.cuda.synchronize()
        assert graph.async_status() == 0
        if opt.step_dev is not None:
            assert int(opt.step_dev.item()) == 5
        results.append([loss.clone(), p.clone(), counts.clone()] + [t.clone() for t in W] + [t.clone() for t in opt.m] +
                       [t.clone() for t in opt.v])
    for other in results[1:]:
        for a, b in zip(results[0], other):
            assert torch.equal(a, b)


def test_host_variant_matches_device_variant():
    import torch
    import paper_2511_09261_b200 as gnnco
    w = si.make_workload(1)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    perm = graph.arrays()["perm"].cpu().numpy()
    Xh = torch.from_numpy(w.features_f32()[perm]).pin_memory()
    pen = torch.from_numpy(w.penalty()[perm]).pin_memory()
    res = []
    for host in (False, True):
        W = [to_dev(w.weights(l)) for l in range(w.L)]
        model = gnnco.Model(w.dims, W)
        opt = gnnco.Adam(model)
        if host:
            loss, p = graph.train_step_host(model, Xh, 2.0, 1.0, 1.0, pen, opt)
            res.append((loss.clone(), p.clone(), W[0].cpu()))
        else:
            loss, p = graph.train_step(model, Xh.cuda(), 2.0, 1.0, 1.0, pen.cuda(), opt)
            res.append((loss.cpu(), p.cpu(), W[0].cpu()))
    for a, b in zip(*res):
        assert torch.equal(a, b)


@pytest.mark.parametrize("dtype,dims,n,S,hub", [("bf16", [256, 256, 256, 1], 150000, 37, False),
                                                ("f32", [128, 128, 1], 140000, 3, True)])
def test_host_variant_with_inputs_arriving_in_ranges(dtype, dims, n, S, hub):
    """Inputs of 64 MB and more reach the device in ranges of subgraphs while the first hidden layer already
    runs on the ranges that are there; two steps give the bits of two device-buffer steps (loss, p, weights).
    The second case has a row too long for the row-per-warp kernel (summed by segments on a side stream)."""
    import torch
    import paper_2511_09261_b200 as gnnco
    eu, ev = si.random_regular(n, 3, 211)
    part = si.contiguous_partition(n, S)
    if hub:                                         # node 5 joined to 700 nodes of its own subgraph
        extra = np.arange(100, 800, dtype=eu.dtype)
        keep = ~(((eu == 5) & (ev >= 100) & (ev < 800)) | ((ev == 5) & (eu >= 100) & (eu < 800)))
        eu, ev = np.concatenate([eu[keep], np.full(700, 5, eu.dtype)]), np.concatenate([ev[keep], extra])
    graph = load_graph(n, eu, ev, part, S)
    assert (graph.max_row > 256) == hub
    bf16 = dtype == "bf16"
    perm = graph.arrays()["perm"].cpu().numpy()
    X = rand_features(n, dims[0], 223).astype(np.float32)[perm]
    Xh = torch.from_numpy(X)
    if bf16:
        Xh = Xh.to(torch.bfloat16)
    Xh = Xh.pin_memory()
    assert Xh.numel() * Xh.element_size() >= 64 << 20
    pen = torch.from_numpy((si.uniform01(227, 0, n) < 0.3).astype(np.float32)).pin_memory()
    res = []
    for host in (False, True):
        W = [to_dev(si.round_to_bf16(w.astype(np.float32))) for w in rand_weights(dims, S, 229)]
        model = gnnco.Model(dims, W, gnnco.BF16 if bf16 else gnnco.F32)
        opt = gnnco.Adam(model, lr=1e-2)
        out = []
        for step in range(2):
            if host:
                loss, p = graph.train_step_host(model, Xh, 2.0, 1.0, 0.5, pen, opt)
                out += [loss.clone(), p.clone()]
            else:
                loss, p = graph.train_step(model, Xh.cuda(), 2.0, 1.0, 0.5, pen.cuda(), opt)
                out += [loss.cpu(), p.cpu()]
        res.append(out + [t.cpu() for t in W])
    assert graph.async_status() == 0
    for a, b in zip(*res):
        assert torch.equal(a, b)


def test_gather_rows_roundtrip():
    import torch
    w = si.make_workload(1)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    arr = graph.arrays()
    X = to_dev(w.features_f32())
    Xn = graph.gather_rows(X, arr["perm"])
    assert torch.equal(Xn, X[arr["perm"].long()])
    back = graph.gather_rows(Xn, arr["inv_perm"])
    assert torch.equal(back, X)
    v = to_dev(np.arange(w.n, dtype=np.float32))
    assert torch.equal(graph.gather_rows(v, arr["perm"]), arr["perm"].float())


@pytest.mark.parametrize("dims,n,S", [([256, 256, 256, 1], 3200, 8), ([128, 128, 1], 1500, 2), ([256, 64, 1], 900, 4),
                                      ([128, 256, 1], 1300, 1)])
def test_train_step_bf16_long_subgraphs(dims, n, S):
    """Subgraphs of several hundred rows: many 128-row tiles per subgraph and a multi-stage
    reduction in the weight-gradient kernel, with ragged tails."""
    eu, ev, part = tiny_graph(n, 4.0 / n, S, seed=19)
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    X = si.round_to_bf16(rand_features(n, dims[0], 23).astype(np.float32))
    W = [si.round_to_bf16(w.astype(np.float32)) for w in rand_weights(dims, S, 29)]
    case = StepCase(book, dims, "bf16", S, lam=0.0)
    adam = dict(lr=1e-3, step=2, m=[np.zeros_like(w) for w in W], v=[np.zeros_like(w) for w in W])
    case.run(graph, X, W, None, want_dx=True, adam=adam, label="bf16-long")


@pytest.mark.parametrize("dims", [[256, 64, 1], [64, 64, 1], [512, 64, 1], [256, 256, 1]])
def test_train_step_bf16_hub_row(dims):
    """A hub row longer than the block-per-row threshold, bf16 features."""
    eu, ev, part = GRAPHS["big_hub"]()
    n, S = _n_S(part)
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    assert graph.max_row > 256
    X = si.round_to_bf16(rand_features(n, dims[0], 31).astype(np.float32))
    W = [si.round_to_bf16(w.astype(np.float32)) for w in rand_weights(dims, S, 37)]
    StepCase(book, dims, "bf16", S).run(graph, X, W, None, want_dx=True, label="bf16-hub")


@pytest.mark.parametrize("dims,n,S,sets", [([128, 128, 128, 1], 2300, 5, None), ([128, 64, 1], 1500, 2, None),
                                           ([64, 128, 64, 1], 900, 4, None), ([64, 64, 1], 700, 1, None),
                                           ([128, 128, 1], 1000, 3, 1)])
def test_train_step_f32_tensor_core_widths(dims, n, S, sets):
    """float32 features at widths the tensor-core path takes (operands split into bf16 limbs):
    the result must still meet the float32 tolerance."""
    eu, ev, part = tiny_graph(n, 5.0 / n, S, seed=41)
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    X = rand_features(n, dims[0], 43).astype(np.float32)
    nsets = S if sets is None else sets
    W = [w.astype(np.float32) for w in rand_weights(dims, nsets, 47, scale=1.5)]
    pen = (si.uniform01(5, 0, n) < 0.2).astype(np.float32)
    case = StepCase(book, dims, "f32", nsets, lam=0.3)
    adam = dict(lr=1e-3, step=4, m=[0.01 * rand_weights(dims, nsets, 51)[l].astype(np.float32) for l in range(len(W))],
                v=[np.square(0.02 * rand_weights(dims, nsets, 52)[l]).astype(np.float32) for l in range(len(W))])
    g, stats = case.run(graph, X, W, pen, want_dx=True, adam=adam, label="f32-tc")
    print({k: float("%.3g" % v) for k, v in stats.items()})


@pytest.mark.parametrize("dtype,dims,n,S", [("bf16", [256, 128, 1], 9000, 2), ("f32", [128, 64, 1], 7000, 1),
                                            ("bf16", [256, 256, 1], 7000, 3),
                                            ("bf16", [128, 128, 1], 6100, 3), ("f32", [64, 36, 1], 7000, 1),
                                            ("f32", [20, 24, 1], 5000, 2)])
def test_train_step_few_very_long_subgraphs(dtype, dims, n, S):
    """Few subgraphs of several thousand rows (the shape community detection gives): the
    weight gradient of such a subgraph is cut into row chunks whose partial results are summed
    in a fixed order."""
    eu, ev, part = tiny_graph(n, 4.0 / n, S, seed=61, contiguous=True)
    if S == 3:
        part = np.where(np.arange(n) < 5000, 0, np.where(np.arange(n) < 6000, 1, 2)).astype(np.int32)   # uneven
    book = oracle.bookkeeping(n, eu, ev, part, S)
    graph = load_graph(n, eu, ev, part, S)
    X = rand_features(n, dims[0], 63).astype(np.float32)
    W = [w.astype(np.float32) for w in rand_weights(dims, S, 67)]
    if dtype == "bf16":
        X, W = si.round_to_bf16(X), [si.round_to_bf16(w) for w in W]
    case = StepCase(book, dims, dtype, S)
    case.run(graph, X, W, None, want_dx=True, label="long-subgraphs")
    again = case.run(graph, X, W, None, want_dx=True, label="long-subgraphs")[0]
    first = case.run(graph, X, W, None, want_dx=True, label="long-subgraphs")[0]
    for a, b in zip(again["dW"], first["dW"]):
        assert np.array_equal(a, b)                      # deterministic combine
