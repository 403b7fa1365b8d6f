"""GPU parity of gnnco_louvain (Section 3.1): the community vector, the number of communities, the exact
modularity numerator and the level / sweep counts are integers that are uniquely defined, so they must be
bit-exact against the CPU oracle; the partition then goes through gnnco_partition_load and a training step."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from gpu_common import StepCase, check_bookkeeping, load_graph, to_dev
from helpers import rand_features, rand_weights

pytestmark = pytest.mark.gpu


def _planted(blocks, size, p_in, p_out, seed):
    n = blocks * size
    eu, ev = si.erdos_renyi(n, p_out, seed)
    keep = (eu // size) != (ev // size)
    iu, iv = si.erdos_renyi(n, p_in, seed + 1)
    inside = (iu // size) == (iv // size)
    return n, np.concatenate([eu[keep], iu[inside]]).astype(np.int32), np.concatenate([ev[keep], iv[inside]]).astype(np.int32)


def _star(n):
    return n, np.zeros(n - 1, np.int32), np.arange(1, n, dtype=np.int32)


GRAPHS = {
    "er_small": lambda: (60,) + si.erdos_renyi(60, 0.08, 1),
    "er_sweep_rejected": lambda: (8,) + si.erdos_renyi(8, 0.3, 5),
    "er_medium": lambda: (3000,) + si.erdos_renyi(3000, 0.002, 7),
    "planted": lambda: _planted(8, 60, 0.3, 0.004, 3),
    "no_edges": lambda: (40, np.zeros(0, np.int32), np.zeros(0, np.int32)),
    "one_edge": lambda: (2, np.array([1], np.int32), np.array([0], np.int32)),
    "star": lambda: _star(5000),
    "config1": lambda: (lambda w: (w.n, w.eu, w.ev))(si.make_workload(1)),
    "config3": lambda: (lambda w: (w.n, w.eu, w.ev))(si.make_workload(3)),
    "config2": lambda: (lambda w: (w.n, w.eu, w.ev))(si.make_workload(2)),
    "config4_scaled": lambda: (lambda w: (w.n, w.eu, w.ev))(si.make_workload(4, 0.05)),
}


@pytest.mark.parametrize("name", sorted(GRAPHS))
def test_louvain_is_bit_exact(name):
    import paper_2511_09261_b200 as gnnco
    n, eu, ev = GRAPHS[name]()
    ref = oracle.louvain(n, eu, ev)
    got = gnnco.gnnco_louvain(to_dev(eu.astype(np.int32)), to_dev(ev.astype(np.int32)), n)
    assert (got["S"], got["qnum"], got["two_m"], got["levels"], got["sweeps"]) == (
        ref["S"], ref["qnum"], ref["two_m"], ref["levels"], ref["sweeps"])
    assert np.array_equal(got["part"].cpu().numpy(), ref["part"])
    # limits are honoured the same way
    for levels, sweeps in ((1, 1), (2, 3)):
        r2 = oracle.louvain(n, eu, ev, max_levels=levels, max_sweeps=sweeps)
        g2 = gnnco.gnnco_louvain(to_dev(eu.astype(np.int32)), to_dev(ev.astype(np.int32)), n, levels, sweeps)
        assert np.array_equal(g2["part"].cpu().numpy(), r2["part"]) and g2["qnum"] == r2["qnum"]


def test_louvain_rejects_bad_graphs():
    import paper_2511_09261_b200 as gnnco
    with pytest.raises(gnnco.GnncoError) as e:
        gnnco.gnnco_louvain(to_dev(np.array([0, 2], np.int32)), to_dev(np.array([1, 2], np.int32)), 4)     # self loop
    assert e.value.status == gnnco.NOT_SIMPLE_GRAPH
    with pytest.raises(gnnco.GnncoError) as e:
        gnnco.gnnco_louvain(to_dev(np.array([0], np.int32)), to_dev(np.array([9], np.int32)), 4)
    assert e.value.status == gnnco.OUT_OF_RANGE


def test_louvain_partition_feeds_the_training_step():
    """Section 3.1 -> Section 3.2: the communities become the subgraphs of a block-diagonal batch (very uneven
    sizes) and one step on them matches the oracle."""
    import paper_2511_09261_b200 as gnnco
    w = si.make_workload(3)
    lv = gnnco.gnnco_louvain(to_dev(w.eu), to_dev(w.ev), w.n)
    part = lv["part"].cpu().numpy()
    S = lv["S"]
    q = oracle.partition_quality(w.eu, w.ev, part, S)
    np.testing.assert_allclose(q["Q"], lv["Q"], rtol=1e-12)
    book = oracle.bookkeeping(w.n, w.eu, w.ev, part, S)
    graph = load_graph(w.n, w.eu, w.ev, part, S)
    check_bookkeeping(graph, book)
    dims = [64, 32, 1]
    X = rand_features(w.n, dims[0], 5).astype(np.float32)
    W = [x.astype(np.float32) for x in rand_weights(dims, S, 7)]
    StepCase(book, dims, "f32", S).run(graph, X, W, None, want_dx=True, label="louvain-parts")
