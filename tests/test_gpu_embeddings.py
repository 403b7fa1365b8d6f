"""GPU parity of the input-embedding entry points (Section 3.2: random initial embeddings
"processed using the Gumbel-softmax trick"; trainable-embedding variant): the CUDA library
through its C ABI binding against the float64 oracle on the same seeded inputs."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import tiny_graph, rand_features
from gpu_common import load_graph, to_dev

pytestmark = pytest.mark.gpu

# float32: the two logarithms, the exponential and the division each carry a few ulp, and the
# logits are divided by tau >= 0.25, so 1e-4 relative is generous; bfloat16 output adds one
# rounding of 2^-9 relative.
TOL = {"f32": dict(rtol=1e-4, atol=1e-7), "bf16": dict(rtol=6e-3, atol=1e-7)}


def _graph(n=523, S=4):
    eu, ev, part = tiny_graph(n, 0.02, S, seed=77)
    return load_graph(n, eu, ev, part, int(part.max()) + 1), n


def _uniforms(n, F, seed):
    """float32 uniforms strictly inside (0, 1): what both sides receive."""
    u = si.uniform01(seed, 0, n * F).astype(np.float32).reshape(n, F)
    return np.clip(u, np.float32(2.0 ** -24), np.float32(1.0 - 2.0 ** -24))


@pytest.mark.parametrize("F", [1, 5, 32, 64, 200, 256, 300, 1000])
@pytest.mark.parametrize("tau", [0.25, 1.0, 3.0])
def test_gumbel_softmax_f32(F, tau):
    graph, n = _graph()
    E = rand_features(n, F, 3).astype(np.float32)
    U = _uniforms(n, F, 9)
    got = graph.gumbel_softmax(to_dev(E), to_dev(U), tau).cpu().numpy()
    ref = oracle.gumbel_softmax(E, U, tau)
    np.testing.assert_allclose(got, ref, **TOL["f32"])
    np.testing.assert_allclose(got.sum(axis=1), 1.0, rtol=1e-5)


@pytest.mark.parametrize("F", [8, 64, 256, 512])
def test_gumbel_softmax_bf16_in_place_and_without_noise(F):
    import torch
    graph, n = _graph()
    E = si.round_to_bf16(rand_features(n, F, 4).astype(np.float32))
    U = _uniforms(n, F, 10)
    Ed = to_dev(E).to(torch.bfloat16)
    got = graph.gumbel_softmax(Ed.clone(), to_dev(U), 0.5).float().cpu().numpy()
    np.testing.assert_allclose(got, oracle.gumbel_softmax(E, U, 0.5), **TOL["bf16"])
    buf = Ed.clone()
    graph.gumbel_softmax(buf, to_dev(U), 0.5, out=buf)                      # E and X the same buffer
    assert np.array_equal(buf.float().cpu().numpy(), got)
    plain = graph.gumbel_softmax(Ed, None, 2.0).float().cpu().numpy()
    np.testing.assert_allclose(plain, oracle.gumbel_softmax(E, None, 2.0), **TOL["bf16"])


def test_gumbel_softmax_rejects_bad_arguments():
    import paper_2511_09261_b200 as gnnco
    graph, n = _graph()
    E = to_dev(rand_features(n, 4, 1).astype(np.float32))
    for tau in (0.0, -1.0, float("nan")):
        with pytest.raises(gnnco.GnncoError) as e:
            graph.gumbel_softmax(E, None, tau)
        assert e.value.status == gnnco.INVALID_ARGUMENT


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_embedding_update_matches_oracle_adam(dtype):
    import torch
    graph, n = _graph()
    F = 48
    g = rand_features(n, F, 21).astype(np.float32) * 0.3
    g[::7] = 0.0                                                            # zero gradient: no move from zero moments
    if dtype == "bf16":
        g = si.round_to_bf16(g)
    Xm = rand_features(n, F, 22).astype(np.float32)
    m = 0.01 * rand_features(n, F, 23).astype(np.float32)
    v = np.square(0.02 * rand_features(n, F, 24)).astype(np.float32)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    Xm_d, m_d, v_d = to_dev(Xm), to_dev(m), to_dev(v)
    X_d = torch.empty(n, F, dtype=tdt, device=Xm_d.device)
    graph.embedding_update(to_dev(g).to(tdt), Xm_d, m_d, v_d, X_d, lr=1e-2, step=3)
    Xr, mr, vr = Xm.astype(np.float64), m.astype(np.float64), v.astype(np.float64)
    # the library receives its hyper-parameters as float32: the oracle gets the same rounded values
    f32 = lambda x: float(np.float32(x))
    oracle.adam(Xr, mr, vr, g.astype(np.float64), f32(1e-2), 3, f32(0.9), f32(0.999), f32(1e-8))
    # float32 moments: each is a sum of two rounded products, so the absolute error is a few
    # 2^-24 of the LARGER addend (|b1 m| + |(1-b1) g| <= 0.15, |b2 v| + |(1-b2) g^2| <= 2e-3), which
    # shows as a large relative error only where the two nearly cancel
    np.testing.assert_allclose(m_d.cpu().numpy(), mr, rtol=1e-5, atol=3e-8)
    np.testing.assert_allclose(v_d.cpu().numpy(), vr, rtol=1e-5, atol=4e-10)
    np.testing.assert_allclose(Xm_d.cpu().numpy(), Xr, rtol=1e-5, atol=1e-6)
    stored = X_d.float().cpu().numpy()
    if dtype == "bf16":
        assert np.array_equal(stored, si.round_to_bf16(Xm_d.cpu().numpy()))
    else:
        assert np.array_equal(stored, Xm_d.cpu().numpy())


def test_training_the_embeddings_lowers_the_objective():
    """Sanity, not parity: Gumbel-softmax inputs, then steps that update weights and embeddings."""
    import torch
    import paper_2511_09261_b200 as gnnco
    w = si.make_workload(1)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    perm = graph.arrays()["perm"].cpu().numpy()
    E = to_dev(w.features_f32()[perm])
    X = graph.gumbel_softmax(E, to_dev(_uniforms(w.n, w.dims[0], 5)), 1.0)
    Xm, m, v = X.clone(), torch.zeros_like(X), torch.zeros_like(X)
    W = [to_dev(w.weights(l)) for l in range(w.L)]
    model = gnnco.Model(w.dims, W)
    opt = gnnco.Adam(model, lr=1e-2)
    dX = torch.empty_like(X)
    totals = []
    for step in range(1, 41):
        loss, _ = graph.train_step(model, X, 2.0, 1.0, opt=opt, dX=dX, flags=gnnco.WANT_DX)
        totals.append(float(loss.sum()))
        graph.embedding_update(dX, Xm, m, v, X, lr=1e-2, step=step)
    assert totals[-1] < totals[0]
    assert graph.async_status() == gnnco.OK


@pytest.mark.parametrize("n,d,S", [(100, 10, 2), (500, 20, 4), (1000, 40, 8), (1000, 10, 1)])
def test_small_regular_workload_pipeline_matches_the_oracle(n, d, S):
    """The paper's small-graph experiment shape (Section 4: d-regular graphs of 100 to 1,000 nodes, degree 10 to
    40), through the whole variant in which embeddings are processed and trained: Gumbel-softmax of the random
    initial embeddings, one training step with the input gradient, Adam on the embeddings -- every stage
    against the oracle on the same seeded inputs."""
    import torch
    import paper_2511_09261_b200 as gnnco
    from gpu_common import StepCase, check_bookkeeping, check_decode
    w = si.small_regular_workload(n, d, S, [32, 16, 1], seed=100 + d)
    deg = np.bincount(np.concatenate([w.eu, w.ev]), minlength=n)
    assert deg.max() == d and (deg >= d - 2).mean() > 0.9          # configuration model: a few nodes lose an edge
    book = oracle.bookkeeping(w.n, w.eu, w.ev, w.part, w.S)
    graph = load_graph(w.n, w.eu, w.ev, w.part, w.S)
    check_bookkeeping(graph, book)
    E = w.features_f32()[book["perm"]]
    U = _uniforms(n, w.dims[0], 7)
    X_d = graph.gumbel_softmax(to_dev(E), to_dev(U), 0.7)
    X = X_d.cpu().numpy()
    np.testing.assert_allclose(X, oracle.gumbel_softmax(E, U, 0.7), **TOL["f32"])
    # the step is compared on the GPU's own float32 embeddings (teacher-forced at the stage boundary)
    W = [w.weights(l) for l in range(w.L)]
    case = StepCase(book, w.dims, "f32", w.S, w.alpha, w.beta)
    adam = dict(lr=1e-2, step=1, m=[np.zeros_like(x) for x in W], v=[np.zeros_like(x) for x in W])
    g, _ = case.run(graph, X, W, None, want_dx=True, adam=adam, label="regular-%d-%d" % (n, d))
    check_decode(graph, book, g["p"])
    for name in ("loss", "p", "z", "dW0", "dW1", "dX"):
        assert case.report.needs_only_flat(name), name
    # Adam on the embeddings with the GPU's own input gradient
    Xm, m, v = X_d.clone(), torch.zeros_like(X_d), torch.zeros_like(X_d)
    out = torch.empty_like(X_d)
    graph.embedding_update(to_dev(g["dX"].astype(np.float32)), Xm, m, v, out, lr=1e-2, step=1)
    Xr, mr, vr = X.astype(np.float64), np.zeros_like(X, np.float64), np.zeros_like(X, np.float64)
    f32 = lambda x: float(np.float32(x))
    oracle.adam(Xr, mr, vr, g["dX"].astype(np.float64), f32(1e-2), 1, f32(0.9), f32(0.999), f32(1e-8))
    np.testing.assert_allclose(Xm.cpu().numpy(), Xr, rtol=1e-5, atol=1e-6)
    assert torch.equal(out, Xm)
