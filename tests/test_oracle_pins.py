"""Pins for the CPU oracle: each test checks it against something other than itself --
a closed form, an invariant, a finite difference, exact rational arithmetic, a dense
linear-algebra restatement built from the ORIGINAL edge list, or brute force."""
import itertools
from fractions import Fraction
import decimal

import numpy as np
import pytest

import oracle
import synth_inputs as si
from helpers import tiny_graph, dense_intra_adjacency, rand_weights, rand_features

ALPHA, BETA = 2.0, 1.0


# ------------------------------------------------------------------ bookkeeping (a0)
def _brute_bookkeeping(n, eu, ev, part, S):
    order = sorted(range(n), key=lambda i: (int(part[i]), i))
    inv = {o: k for k, o in enumerate(order)}
    intra, bnd = set(), set()
    for a, b in zip(eu.tolist(), ev.tolist()):
        na, nb = inv[a], inv[b]
        (intra if part[a] == part[b] else bnd).add((min(na, nb), max(na, nb)))
    return order, inv, intra, bnd


@pytest.mark.parametrize("n,p,S,seed", [(12, 0.4, 3, 1), (40, 0.2, 5, 2), (64, 0.1, 64, 3), (30, 0.3, 1, 4),
                                        (25, 0.3, 9, 5)])
def test_bookkeeping_brute_force(n, p, S, seed):
    eu, ev, part = tiny_graph(n, p, S, seed)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    order, inv, intra, bnd = _brute_bookkeeping(n, eu, ev, part, S)
    assert b["perm"].tolist() == order
    assert [int(b["inv_perm"][i]) for i in range(n)] == [inv[i] for i in range(n)]
    assert b["E_in"] == len(intra) and b["E_b"] == len(bnd) and b["E_in"] + b["E_b"] == eu.size
    sizes = np.bincount(part, minlength=S)
    assert np.array_equal(np.diff(b["part_ptr"]), sizes) and b["part_ptr"][0] == 0
    rp, ci = b["rowptr"], b["colidx"]
    assert rp[0] == 0 and rp[n] == 2 * b["E_in"]
    got = set()
    for i in range(n):
        row = ci[rp[i]:rp[i + 1]].tolist()
        assert row == sorted(set(row)) and i not in row
        s = b["node_part"][i]
        assert all(b["part_ptr"][s] <= j < b["part_ptr"][s + 1] for j in row)
        for j in row:
            assert i in ci[rp[j]:rp[j + 1]].tolist()            # symmetric
            got.add((min(i, j), max(i, j)))
        assert b["inv_deg"][i] == np.float32(1.0) / np.float32(len(row) + 1)
    assert got == intra
    pairs = list(zip(b["bnd_u"].tolist(), b["bnd_v"].tolist()))
    assert pairs == sorted(bnd)
    isb = np.zeros(n, np.uint8)
    for a, c in bnd:
        isb[a] = isb[c] = 1
    assert np.array_equal(b["is_boundary"], isb)
    assert np.array_equal(b["node_part"], part[b["perm"]])


def test_bookkeeping_rejects_bad_input():
    eu = np.array([0, 1, 2], np.int32)
    ev = np.array([1, 2, 2], np.int32)
    part = np.zeros(4, np.int32)
    with pytest.raises(oracle.OracleError) as e:
        oracle.bookkeeping(4, eu, ev, part, 1)            # self loop 2-2
    assert e.value.code == oracle.NOT_SIMPLE
    with pytest.raises(oracle.OracleError) as e:
        oracle.bookkeeping(4, np.array([0, 1], np.int32), np.array([1, 0], np.int32), part, 1)   # repeated edge
    assert e.value.code == oracle.NOT_SIMPLE
    with pytest.raises(oracle.OracleError) as e:
        oracle.bookkeeping(4, np.array([0], np.int32), np.array([7], np.int32), part, 1)
    assert e.value.code == oracle.OUT_OF_RANGE
    with pytest.raises(oracle.OracleError) as e:
        oracle.bookkeeping(4, np.array([0], np.int32), np.array([1], np.int32), np.array([0, 0, 3, 0], np.int32), 2)
    assert e.value.code == oracle.OUT_OF_RANGE


@pytest.mark.parametrize("idx", [1, 2, 3])
def test_bookkeeping_invariants_on_configs(idx):
    w = si.make_workload(idx)
    b = oracle.bookkeeping(w.n, w.eu, w.ev, w.part, w.S)
    assert b["E_in"] + b["E_b"] == w.E and b["rowptr"][w.n] == 2 * b["E_in"]
    assert np.array_equal(np.sort(b["perm"]), np.arange(w.n))
    assert np.array_equal(b["inv_perm"][b["perm"]], np.arange(w.n))
    assert np.array_equal(np.diff(b["part_ptr"]), np.bincount(w.part, minlength=w.S))
    rows = np.repeat(np.arange(w.n), np.diff(b["rowptr"]))
    assert np.array_equal(b["node_part"][rows], b["node_part"][b["colidx"]])
    fwd = set(zip(rows.tolist(), b["colidx"].tolist()))
    assert len(fwd) == 2 * b["E_in"] and all((j, i) in fwd for i, j in itertools.islice(fwd, 5000))
    intra_direct = int((w.part[w.eu] == w.part[w.ev]).sum())
    assert b["E_in"] == intra_direct


# --------------------------------------------------- dense restatement (a1-a4), Eq. 3-5
def _dense_forward_loss(n, eu, ev, part, dims, X, W, pen, lam):
    """Dense linear algebra from the original edge list, original node order;
    W[l][part] applied row by row."""
    A = dense_intra_adjacency(n, eu, ev, part)
    Ahat = (A + np.eye(n)) / (A.sum(1) + 1.0)[:, None]
    H = X
    L = len(dims) - 1
    for l in range(L):
        M = Ahat @ H
        Z = np.stack([M[i] @ W[l][part[i] if W[l].shape[0] > 1 else 0] for i in range(n)])
        H = np.maximum(Z, 0.0) if l < L - 1 else Z
    z = H[:, 0]
    p = 1.0 / (1.0 + np.exp(-z))
    S = int(part.max()) + 1
    loss = np.zeros(S)
    for s in range(S):
        msk = part == s
        ps = p * msk
        loss[s] = ALPHA * 0.5 * ps @ A @ ps - BETA * ps.sum() + lam * (pen * ps).sum()
    return z, p, loss


@pytest.mark.parametrize("dims,sets_shared", [([5, 1], False), ([6, 4, 1], False), ([7, 5, 3, 1], True)])
def test_forward_and_loss_match_dense_definition(dims, sets_shared):
    n, S = 40, 4
    eu, ev, part = tiny_graph(n, 0.25, S, seed=11)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    X = rand_features(n, dims[0], 5)
    W = rand_weights(dims, 1 if sets_shared else S, 7, scale=2.0)
    pen = (si.uniform01(99, 0, n) < 0.3).astype(np.float64)
    z, p, loss = _dense_forward_loss(n, eu, ev, part, dims, X, W, pen, 0.7)
    r = oracle.train_step(b, dims, X[b["perm"]], W, ALPHA, BETA, 0.7, pen[b["perm"]])
    np.testing.assert_allclose(r["z"], z[b["perm"]], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(r["p"], p[b["perm"]], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(r["loss"], loss, rtol=1e-12, atol=1e-12)


def test_aggregation_preserves_constant_features_and_isolated_nodes():
    # identity weights expose M = A_hat X through the saved pre-activations
    n, S, F = 50, 5, 4
    eu, ev, part = tiny_graph(n, 0.15, S, seed=21)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    W = [np.tile(np.eye(F), (S, 1, 1)), np.zeros((S, F, 1))]
    X = np.tile(np.array([1.5, -2.0, 0.25, 3.0]), (n, 1))
    r = oracle.train_step(b, [F, F, 1], X, W, ALPHA, BETA, want_Z=True)
    assert np.array_equal(r["Z"][0], X)                       # rows of A_hat sum to one
    Xr = rand_features(n, F, 3)
    r = oracle.train_step(b, [F, F, 1], Xr, W, ALPHA, BETA, want_Z=True)
    deg = np.diff(b["rowptr"])
    iso = np.where(deg == 0)[0]
    assert iso.size > 0
    assert np.array_equal(r["Z"][0][iso], Xr[iso])            # no intra neighbour: M_i = H_i


def test_regular_partition_aggregation_is_doubly_stochastic():
    # one partition, 4-regular circulant graph: column sums of A_hat are one as well
    n, F = 31, 3
    eu = np.concatenate([np.arange(n), np.arange(n)]).astype(np.int32)
    ev = np.concatenate([(np.arange(n) + 1) % n, (np.arange(n) + 5) % n]).astype(np.int32)
    b = oracle.bookkeeping(n, eu, ev, np.zeros(n, np.int32), 1)
    assert np.all(np.diff(b["rowptr"]) == 4)
    X = rand_features(n, F, 8)
    r = oracle.train_step(b, [F, F, 1], X, [np.eye(F)[None], np.zeros((1, F, 1))], ALPHA, BETA, want_Z=True)
    np.testing.assert_allclose(r["Z"][0].sum(0), X.sum(0), rtol=1e-13)


def test_zero_weights_closed_forms():
    w = si.make_workload(1)
    b = oracle.bookkeeping(w.n, w.eu, w.ev, w.part, w.S)
    X = w.features_f32()[b["perm"]]
    W = [np.zeros((w.S, w.dims[l], w.dims[l + 1])) for l in range(w.L)]
    r = oracle.train_step(b, w.dims, X, W, ALPHA, BETA)
    assert np.all(r["z"] == 0.0) and np.all(r["p"] == 0.5)
    e_in_s = np.array([(b["rowptr"][b["part_ptr"][s + 1]] - b["rowptr"][b["part_ptr"][s]]) // 2 for s in range(w.S)])
    expect = ALPHA * e_in_s / 4.0 - BETA * np.diff(b["part_ptr"]) / 2.0
    assert np.array_equal(r["loss"], expect)
    d = oracle.decode(b, r["p"].astype(np.float32))
    assert d["set_size"] == w.n and d["boundary_viol"] == b["E_b"] and d["intra_viol"] == b["E_in"]
    assert np.all(d["x"] == 1) and np.all(d["viol"] == 1)
    assert d["per_part"].sum() == 2 * b["E_b"]


def test_single_node_subgraph_by_hand():
    # two isolated single-node subgraphs: p = sigmoid(relu(x W1) w2), own weights each
    X = np.array([[1.0, -2.0], [0.5, 3.0]])
    W1 = np.array([[[1.0, -1.0], [0.5, 2.0]], [[-1.0, 0.0], [1.0, 1.0]]])
    W2 = np.array([[[2.0], [-1.0]], [[0.5], [0.25]]])
    b = oracle.bookkeeping(2, np.zeros(0, np.int32), np.zeros(0, np.int32), np.array([0, 1], np.int32), 2)
    r = oracle.train_step(b, [2, 2, 1], X, [W1, W2], ALPHA, BETA)
    # node 0: x W1 = [1-1, -1-4] = [0, -5] -> relu [0, 0] -> z = 0
    # node 1: x W1 = [-0.5+3, 0+3] = [2.5, 3] -> z = 1.25 + 0.75 = 2
    assert r["z"].tolist() == [0.0, 2.0]
    np.testing.assert_allclose(r["p"], [0.5, 1.0 / (1.0 + np.exp(-2.0))], rtol=1e-15)
    np.testing.assert_allclose(r["loss"], [-0.5, -1.0 / (1.0 + np.exp(-2.0))], rtol=1e-15)


def test_complete_graph_identical_rows_give_equal_probabilities():
    k, F = 7, 5
    eu, ev = np.triu_indices(k, 1)
    b = oracle.bookkeeping(k, eu.astype(np.int32), ev.astype(np.int32), np.zeros(k, np.int32), 1)
    X = np.tile(rand_features(1, F, 4), (k, 1))
    r = oracle.train_step(b, [F, 4, 1], X, rand_weights([F, 4, 1], 1, 3), ALPHA, BETA)
    assert np.all(r["p"] == r["p"][0])


def test_relabelling_nodes_permutes_outputs():
    n, S, dims = 36, 3, [4, 3, 1]
    eu, ev, part = tiny_graph(n, 0.3, S, seed=31, contiguous=True)
    X, W = rand_features(n, 4, 6), rand_weights(dims, S, 9)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    r = oracle.train_step(b, dims, X[b["perm"]], W, ALPHA, BETA)
    # reverse the ids inside the graph (parts stay attached to their nodes)
    sigma = np.arange(n)[::-1].copy()                   # old id -> new id
    eu2, ev2 = sigma[eu].astype(np.int32), sigma[ev].astype(np.int32)
    part2 = np.empty(n, np.int32)
    part2[sigma] = part
    X2 = np.empty_like(X)
    X2[sigma] = X
    b2 = oracle.bookkeeping(n, eu2, ev2, part2, S)
    r2 = oracle.train_step(b2, dims, X2[b2["perm"]], W, ALPHA, BETA)
    p_orig = np.empty(n)
    p_orig[b["perm"]] = r["p"]
    p2_orig = np.empty(n)
    p2_orig[b2["perm"]] = r2["p"]
    np.testing.assert_allclose(p2_orig[sigma], p_orig, rtol=1e-12)
    np.testing.assert_allclose(r2["loss"], r["loss"], rtol=1e-12)


# ------------------------------------------------------------- loss at binary points
def _saturating_setup(n, eu, ev, t):
    """One subgraph, one layer, one-hot embeddings; weights solved so that z = +-800 with
    the sign pattern t, which makes p exactly 1 or 0 in double precision."""
    A = dense_intra_adjacency(n, eu, ev, np.zeros(n, np.int32))
    Ahat = (A + np.eye(n)) / (A.sum(1) + 1.0)[:, None]
    wvec = np.linalg.solve(Ahat, 800.0 * t)
    return A, wvec


def test_loss_on_binary_probabilities_is_the_qubo_value():
    n = 14
    eu, ev, _ = tiny_graph(n, 0.3, 1, seed=41)
    b = oracle.bookkeeping(n, eu, ev, np.zeros(n, np.int32), 1)
    for trial in range(6):
        t = np.where(si.uniform01(500 + trial, 0, n) < 0.5, 1.0, -1.0)
        A, wvec = _saturating_setup(n, eu, ev, t)
        r = oracle.train_step(b, [n, 1], np.eye(n)[b["perm"]], [wvec.reshape(1, n, 1)], ALPHA, BETA)
        x = (t > 0).astype(np.float64)[b["perm"]]
        assert np.array_equal(r["p"], x)
        xo = (t > 0).astype(np.float64)
        conflicts = int(round(0.5 * xo @ A @ xo))
        assert r["loss"][0] == ALPHA * conflicts - BETA * xo.sum()
        d = oracle.decode(b, r["p"].astype(np.float32))
        assert d["intra_viol"] == conflicts and d["set_size"] == int(xo.sum())


def _mis_brute(k, edges):
    nb = [0] * k
    for a, c in edges:
        nb[a] |= 1 << c
        nb[c] |= 1 << a
    best = 0
    for mask in range(1 << k):
        ok = True
        m = mask
        while m:
            i = (m & -m).bit_length() - 1
            if nb[i] & mask:
                ok = False
                break
            m &= m - 1
        if ok:
            best = max(best, bin(mask).count("1"))
    return best


def test_objective_minimum_equals_minus_beta_times_mis_on_small_instances():
    """For alpha > beta the minimum of the relaxed objective over binary assignments is
    -beta * MIS and is attained on an independent set (brute force, <= 12 nodes here;
    16-node instances are covered by the config-2 test below)."""
    k = 10
    for seed in range(51, 90):          # the saturation trick needs A + I to be invertible
        eu, ev, _ = tiny_graph(k, 0.35, 1, seed=seed)
        A0 = dense_intra_adjacency(k, eu, ev, np.zeros(k, np.int32))
        if np.linalg.cond(A0 + np.eye(k)) < 1e6:
            break
    b = oracle.bookkeeping(k, eu, ev, np.zeros(k, np.int32), 1)
    mis = _mis_brute(k, list(zip(eu.tolist(), ev.tolist())))
    best, best_x = None, None
    A = dense_intra_adjacency(k, eu, ev, np.zeros(k, np.int32))
    Ahat_inv = np.linalg.inv((A + np.eye(k)) / (A.sum(1) + 1.0)[:, None])
    for mask in range(1 << k):
        t = np.array([1.0 if (mask >> i) & 1 else -1.0 for i in range(k)])
        wvec = Ahat_inv @ (800.0 * t)
        r = oracle.train_step(b, [k, 1], np.eye(k)[b["perm"]], [wvec.reshape(1, k, 1)], ALPHA, BETA, want_dW=False)
        if best is None or r["loss"][0] < best:
            best, best_x = r["loss"][0], r["p"].copy()
    assert best == -BETA * mis
    d = oracle.decode(b, best_x.astype(np.float32))
    assert d["intra_viol"] == 0 and d["set_size"] == mis


def test_config2_sixteen_node_subinstances_qubo_vs_mis():
    """16-node induced sub-instances of configuration 2: the QUBO optimum (enumerated
    with integer arithmetic) equals -beta*MIS, and the oracle's loss reproduces the QUBO
    value of the optimal assignment and of random assignments."""
    w = si.make_workload(2)
    k, done = 16, 0
    for s in range(w.S):
        if done == 3:
            break
        members = np.where(w.part == s)[0]
        inside = np.isin(w.eu, members) & np.isin(w.ev, members)
        nb = {}
        for a, c in zip(w.eu[inside].tolist(), w.ev[inside].tolist()):
            nb.setdefault(a, []).append(c)
            nb.setdefault(c, []).append(a)
        nodes, seen = [int(members[0])], {int(members[0])}     # breadth-first ball of 16 nodes
        for v in nodes:
            for c in sorted(nb.get(v, [])):
                if c not in seen and len(nodes) < 16:
                    seen.add(c)
                    nodes.append(c)
        if len(nodes) < 16:
            continue
        nodes = np.array(nodes)
        idx = {int(v): i for i, v in enumerate(nodes)}
        sel = np.isin(w.eu, nodes) & np.isin(w.ev, nodes)
        edges = [(idx[a], idx[c]) for a, c in zip(w.eu[sel].tolist(), w.ev[sel].tolist())]
        A0 = np.zeros((k, k))
        for a, c in edges:
            A0[a, c] = A0[c, a] = 1.0
        if len(edges) < 8 or np.linalg.cond(A0 + np.eye(k)) > 1e6:
            continue                    # the saturation trick needs A + I to be invertible
        done += 1
        mis = _mis_brute(k, edges)
        nbm = [0] * k
        for a, c in edges:
            nbm[a] |= 1 << c
            nbm[c] |= 1 << a
        best, best_mask = None, None
        for mask in range(1 << k):
            conf = sum(bin(nbm[i] & mask).count("1") for i in range(k) if (mask >> i) & 1) // 2
            q = 2 * conf - bin(mask).count("1")
            if best is None or q < best:
                best, best_mask = q, mask
        assert best == -mis
        eu = np.array([e[0] for e in edges], np.int32)
        ev = np.array([e[1] for e in edges], np.int32)
        b = oracle.bookkeeping(k, eu, ev, np.zeros(k, np.int32), 1)
        for mask in [best_mask] + [int(m) for m in si.u64(s + 900, 0, 5) % np.uint64(1 << k)]:
            t = np.array([1.0 if (mask >> i) & 1 else -1.0 for i in range(k)])
            A, wvec = _saturating_setup(k, eu, ev, t)
            r = oracle.train_step(b, [k, 1], np.eye(k)[b["perm"]], [wvec.reshape(1, k, 1)], 2.0, 1.0, want_dW=False)
            conf = sum(bin(nbm[i] & mask).count("1") for i in range(k) if (mask >> i) & 1) // 2
            assert r["loss"][0] == 2.0 * conf - bin(mask).count("1")
            assert r["loss"][0] >= -mis
    assert done == 3


# ------------------------------------------------------------------ gradients (a5, a6)
def _total_loss(b, dims, X, W, pen, lam, which=None):
    r = oracle.train_step(b, dims, X, W, ALPHA, BETA, lam, pen, want_dW=False)
    return r["loss"].sum() if which is None else r["loss"][which]


@pytest.mark.parametrize("dims,shared", [([6, 1], False), ([5, 4, 1], False), ([6, 5, 4, 1], False), ([5, 4, 1], True)])
def test_gradients_match_central_finite_differences(dims, shared):
    n, S = 48, 3
    eu, ev, part = tiny_graph(n, 0.2, S, seed=61)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    X = rand_features(n, dims[0], 13)
    W = rand_weights(dims, 1 if shared else S, 17, scale=1.5)
    pen = (si.uniform01(77, 0, n) < 0.3).astype(np.float64)
    lam = 0.9
    r = oracle.train_step(b, dims, X, W, ALPHA, BETA, lam, pen, want_dX=True, want_Z=True)
    if r["Z"]:
        assert min(np.abs(z).min() for z in r["Z"]) > 1e-4          # away from ReLU kinks
    h = 1e-6
    worst = 0.0
    for l in range(len(W)):
        g = r["dW"][l]
        flat = W[l].reshape(-1)
        for q in range(flat.size):
            old = flat[q]
            flat[q] = old + h
            lp = _total_loss(b, dims, X, W, pen, lam)
            flat[q] = old - h
            lm = _total_loss(b, dims, X, W, pen, lam)
            flat[q] = old
            fd = (lp - lm) / (2 * h)
            worst = max(worst, abs(fd - g.reshape(-1)[q]) / (abs(fd) + 2e-2))   # 2e-8 floor: eps*|loss|/h
    assert worst < 1e-6, worst
    rows = (si.u64(5, 0, 12) % np.uint64(n)).astype(int)
    for i in rows:
        for f in range(dims[0]):
            old = X[i, f]
            X[i, f] = old + h
            lp = _total_loss(b, dims, X, W, pen, lam)
            X[i, f] = old - h
            lm = _total_loss(b, dims, X, W, pen, lam)
            X[i, f] = old
            fd = (lp - lm) / (2 * h)
            assert abs(fd - r["dX"][i, f]) <= 1e-6 * abs(fd) + 2e-8     # FD round-off floor: eps*|loss|/h


def test_subgraph_loss_depends_only_on_its_own_weights():
    n, S, dims = 40, 4, [5, 4, 1]
    eu, ev, part = tiny_graph(n, 0.25, S, seed=71)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    X, W = rand_features(n, 5, 2), rand_weights(dims, S, 3)
    base = oracle.train_step(b, dims, X, W, ALPHA, BETA, want_dW=False)["loss"]
    W2 = [w.copy() for w in W]
    W2[0][2] += 0.3
    W2[1][2] -= 0.2
    moved = oracle.train_step(b, dims, X, W2, ALPHA, BETA, want_dW=False)["loss"]
    assert moved[2] != base[2]
    assert np.array_equal(np.delete(moved, 2), np.delete(base, 2))


def test_sigmoid_chain_identity_for_one_layer():
    """L = 1: dW = X^T A_hat^T dz with dz_i = (alpha * sum_nbr p - beta) p (1-p): the
    column sums of that product, evaluated with dense algebra."""
    n = 30
    eu, ev, part = tiny_graph(n, 0.3, 2, seed=81)
    b = oracle.bookkeeping(n, eu, ev, part, 2)
    F = 4
    X = rand_features(n, F, 21)
    W = rand_weights([F, 1], 1, 5)
    r = oracle.train_step(b, [F, 1], X[b["perm"]], W, ALPHA, BETA)
    A = dense_intra_adjacency(n, eu, ev, part)
    Ahat = (A + np.eye(n)) / (A.sum(1) + 1.0)[:, None]
    p = 1.0 / (1.0 + np.exp(-(Ahat @ X @ W[0][0])[:, 0]))
    dz = (ALPHA * (A @ p) - BETA) * p * (1 - p)
    np.testing.assert_allclose(r["dW"][0][0][:, 0], X.T @ Ahat.T @ dz, rtol=1e-11, atol=1e-13)


# ------------------------------------------------------- Louvain partitioning (Section 3.1)
def _exact_modularity(n, edges, comm):
    """Q of Eq. 1's terms, sum_c [ Sigma_in(c)/2m - (Sigma_tot(c)/2m)^2 ] with Sigma_in counted from both ends,
    as an exact fraction, straight from the edge list."""
    two_m = 2 * len(edges)
    if two_m == 0:
        return Fraction(0)
    deg = [0] * n
    for a, b in edges:
        deg[a] += 1
        deg[b] += 1
    q = Fraction(0)
    for c in set(comm):
        inside = sum(2 for a, b in edges if comm[a] == c and comm[b] == c)
        tot = sum(deg[i] for i in range(n) if comm[i] == c)
        q += Fraction(inside, two_m) - Fraction(tot, two_m) ** 2
    return q


def _brute_force_sweep(n, edges, comm):
    """Every node's move by exhaustive evaluation: the change of the exact modularity when the node alone is
    re-assigned, over its own and its neighbours' communities."""
    nbrs = [set() for _ in range(n)]
    for a, b in edges:
        nbrs[a].add(b)
        nbrs[b].add(a)
    size = {c: comm.count(c) for c in set(comm)}
    nxt = list(comm)
    for i in range(n):
        own = comm[i]
        alone = list(comm)
        alone[i] = -1                                            # the node taken out of its community
        base = _exact_modularity(n, edges, alone)
        gain = {}
        for c in {comm[j] for j in nbrs[i]} | {own}:
            trial = list(comm)
            trial[i] = c
            gain[c] = _exact_modularity(n, edges, trial) - base
        best = own
        for c in sorted(gain):
            if c != own and (gain[c] > gain[best] or (gain[c] == gain[best] and best != own and c < best)):
                best = c
        if best != own and gain[best] > gain[own] and not (size[own] == 1 and size[best] == 1 and best > own):
            nxt[i] = best
    return nxt


@pytest.mark.parametrize("n,p,seed", [(9, 0.4, 1), (12, 0.3, 2), (11, 0.5, 3), (12, 0.2, 4), (10, 0.35, 5)])
def test_louvain_sweep_picks_the_brute_force_best_community(n, p, seed):
    eu, ev = si.erdos_renyi(n, p, seed)
    edges = list(zip(eu.tolist(), ev.tolist()))
    vectors = [list(range(n)),                                                    # every node alone
               (si.u64(seed + 50, 0, n) % np.uint64(3)).astype(int).tolist(),     # three random communities
               [i // 2 * 2 for i in range(n)]]                                    # pairs, ids with gaps
    for comm in vectors:
        got = oracle.louvain_sweep(n, eu, ev, np.array(comm, np.int32))
        want = _brute_force_sweep(n, edges, comm)
        assert got["next"].tolist() == want, (comm, got["next"].tolist(), want)
        assert got["moves"] == sum(1 for a, b in zip(comm, want) if a != b)


def test_eq2_gain_is_what_the_sweep_compares():
    # the integer score of the sweep is Eq. 2 times 2 m^2: both rank the candidate communities alike, and the
    # difference of two scores is the exact change of Q times 2 m^2 ... checked through single applied moves
    n = 12
    eu, ev = si.erdos_renyi(n, 0.35, 9)
    edges = list(zip(eu.tolist(), ev.tolist()))
    m = len(edges)
    comm = (si.u64(77, 0, n) % np.uint64(4)).astype(int).tolist()
    deg = np.bincount(np.concatenate([eu, ev]), minlength=n)
    nxt = oracle.louvain_sweep(n, eu, ev, np.array(comm, np.int32))["next"].tolist()
    moved = [i for i in range(n) if nxt[i] != comm[i]]
    assert moved
    for i in moved:
        one = list(comm)
        one[i] = nxt[i]
        dq = _exact_modularity(n, edges, one) - _exact_modularity(n, edges, comm)
        assert dq > 0                                           # a single applied move never lowers Q
        k_in_new = sum(1 for a, b in edges if (a == i and comm[b] == nxt[i]) or (b == i and comm[a] == nxt[i]))
        k_in_old = sum(1 for a, b in edges if (a == i and comm[b] == comm[i] and b != i) or (b == i and comm[a] == comm[i] and a != i))
        tot_new = sum(int(deg[j]) for j in range(n) if comm[j] == nxt[i])
        tot_old = sum(int(deg[j]) for j in range(n) if comm[j] == comm[i] and j != i)
        eq2 = lambda k_in, tot: Fraction(k_in, m) - Fraction(tot * int(deg[i]), 2 * m * m)
        assert dq == eq2(k_in_new, tot_new) - eq2(k_in_old, tot_old)


def test_louvain_recovers_planted_blocks_and_reports_their_exact_modularity():
    import networkx as nx
    blocks, size = 6, 30
    G = nx.planted_partition_graph(blocks, size, 0.5, 0.004, seed=5)
    e = np.array(G.edges(), dtype=np.int32)
    n = blocks * size
    r = oracle.louvain(n, e[:, 0].copy(), e[:, 1].copy())
    assert r["S"] == blocks
    truth = np.arange(n) // size
    # same partition up to the names of the parts; parts are numbered 0..S-1
    pairs = set(zip(truth.tolist(), r["part"].tolist()))
    assert len(pairs) == blocks and sorted(set(r["part"].tolist())) == list(range(blocks))
    comms = [set(np.where(r["part"] == s)[0].tolist()) for s in range(r["S"])]
    np.testing.assert_allclose(r["Q"], nx.community.modularity(G, comms), rtol=1e-12)
    assert Fraction(r["qnum"], r["two_m"] ** 2) == _exact_modularity(n, [tuple(x) for x in e.tolist()], r["part"].tolist())
    q = oracle.partition_quality(e[:, 0].copy(), e[:, 1].copy(), r["part"], r["S"])
    np.testing.assert_allclose(q["Q"], r["Q"], rtol=1e-12)


def test_louvain_small_cases_by_hand():
    # no edges: nobody moves
    r = oracle.louvain(5, np.zeros(0, np.int32), np.zeros(0, np.int32))
    assert r["S"] == 5 and r["part"].tolist() == [0, 1, 2, 3, 4] and r["levels"] == 0 and r["qnum"] == 0
    # one edge: the higher-numbered end joins the lower one (two single nodes never swap), Q goes from -1/2 to 0
    r = oracle.louvain(2, np.array([1], np.int32), np.array([0], np.int32))
    assert r["S"] == 1 and r["part"].tolist() == [0, 0] and r["qnum"] == 0
    # two triangles joined by one edge: the two triangles, Q = 2 * (6/14 - (7/14)^2) = 5/14
    eu = np.array([0, 1, 2, 3, 4, 5, 2], np.int32)
    ev = np.array([1, 2, 0, 4, 5, 3, 3], np.int32)
    r = oracle.louvain(6, eu, ev)
    assert r["part"].tolist() == [0, 0, 0, 1, 1, 1]
    assert Fraction(r["qnum"], r["two_m"] ** 2) == Fraction(5, 14)
    # a sweep that lowers Q is undone: the result is never worse than what it started from
    for seed in (1, 2, 3):
        eu, ev = si.erdos_renyi(60, 0.08, seed)
        r = oracle.louvain(60, eu, ev)
        edges = list(zip(eu.tolist(), ev.tolist()))
        assert Fraction(r["qnum"], r["two_m"] ** 2) == _exact_modularity(60, edges, r["part"].tolist())
        assert Fraction(r["qnum"], r["two_m"] ** 2) > _exact_modularity(60, edges, list(range(60)))
        bound = oracle.louvain(60, eu, ev, max_levels=1, max_sweeps=1)
        assert bound["qnum"] <= r["qnum"]


@pytest.mark.parametrize("n,p,seed", [(8, 0.2, 1), (8, 0.3, 5), (8, 0.4, 1), (12, 0.3, 7), (16, 0.2, 3)])
def test_louvain_level_keeps_a_sweep_only_if_exact_modularity_rises(n, p, seed):
    # first level replayed from outside: frozen-state sweeps, each kept only when the exact modularity of
    # the whole assignment rises strictly (synchronous moves can lower it; these graphs have such a sweep)
    eu, ev = si.erdos_renyi(n, p, seed)
    edges = list(zip(eu.tolist(), ev.tolist()))
    comm = list(range(n))
    q = _exact_modularity(n, edges, comm)
    rejected = False
    for _ in range(64):
        nxt = oracle.louvain_sweep(n, eu, ev, np.array(comm, np.int32))
        if nxt["moves"] == 0:
            break
        q2 = _exact_modularity(n, edges, nxt["next"].tolist())
        if q2 <= q:
            rejected = True
            break
        comm, q = nxt["next"].tolist(), q2
    r = oracle.louvain(n, eu, ev, max_levels=1)
    rank = {c: k for k, c in enumerate(sorted(set(comm)))}
    assert r["part"].tolist() == [rank[c] for c in comm]
    assert Fraction(r["qnum"], r["two_m"] ** 2) == q
    assert rejected or (n, p, seed) == (16, 0.2, 3)


# ------------------------------------------------- bfloat16-storage mode of the oracle
def _exact_bf16_of_float32(f):
    """Nearest bfloat16 (8 significant bits, float32's exponent range, ties to even, overflow
    to infinity) of a finite float32, in exact rational arithmetic."""
    x = Fraction(float(f))
    if x == 0:
        return float(f)                                         # keeps the sign of zero
    a = abs(x)
    e = 0
    while Fraction(2) ** (e + 1) <= a:
        e += 1
    while Fraction(2) ** e > a:
        e -= 1
    q = Fraction(2) ** (max(e, -126) - 7)                       # spacing of bfloat16 numbers around a
    k = a / q
    lo = k.numerator // k.denominator
    rem = k - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    r = lo * q
    if r >= Fraction(2) ** 128:
        return float("inf") if x > 0 else float("-inf")
    return float(r) if x > 0 else -float(r)


def test_round_bf16_is_exact_round_to_nearest_even():
    vals = []
    for base in (1.0, 2.0, 0.75, 3.0e-5, 1.0e20, 2.0 ** -126, 2.0 ** -130, 2.0 ** 127):
        ulp = 2.0 ** (int(np.floor(np.log2(base))) - 7)
        for k in range(0, 9):
            for tweak in (0.0, 2.0 ** -20, -(2.0 ** -20)):
                # k/4 of a bfloat16 spacing above a bfloat16 number: k = 2, 6 are exact ties with an even
                # and an odd neighbour below; the tweaks fall just off the ties on either side
                vals.append(base + ulp * (k / 4.0) * (1.0 + tweak))
    vals += [2.0 - 2.0 ** -9, 2.0 - 2.0 ** -8, 4.0 - 2.0 ** -8, 2.0 ** -133, 2.0 ** -134, 1.5 * 2.0 ** -133, 3.0 * 2.0 ** -134,
             3.3895313892515355e38, 3.3961775292304601e38, 3.4028234663852886e38, 0.0, -0.0]
    vals += si.normal_f32(4242, 0, 400).astype(np.float64).tolist()
    vals += (si.normal_f32(4243, 0, 200).astype(np.float64) * 1e-39).tolist()      # float32 subnormals
    for v in vals:
        for x in (v, -v):
            f = np.float32(x)                                     # IEEE round-to-nearest-even to float32
            want = _exact_bf16_of_float32(f)
            got = oracle.round_bf16(x)
            assert got == want and np.signbit(got) == np.signbit(want), (x, got, want)
    assert oracle.round_bf16(float("inf")) == float("inf") and oracle.round_bf16(float("-inf")) == float("-inf")
    assert np.isnan(oracle.round_bf16(float("nan")))
    # two roundings, not one: a double just above a bfloat16 tie first becomes the tie (as float32)
    assert oracle.round_bf16(1.0 + 2.0 ** -8 + 2.0 ** -40) == 1.0
    # every bfloat16 number is a fixed point
    for v in (1.0, 1.0078125, -3.5, 2.0 ** -133, 255.0, 0.00390625):
        assert oracle.round_bf16(v) == v


def _bf16_lib(a):
    """Library rounding float64 -> float32 -> bfloat16 (torch's conversion routines)."""
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64)).to(torch.float32).to(torch.bfloat16).to(
        torch.float64).numpy()


def _dense_forward_loss_bf16_storage(n, eu, ev, part, dims, X, W, pen, lam):
    """The dense restatement of Eqs. 3-5 with the two tensors that a bfloat16 run STORES per hidden
    layer -- the aggregated input M_l and the activation H_l -- rounded to bfloat16; the output
    layer's aggregate, z, p and the loss stay in double."""
    A = dense_intra_adjacency(n, eu, ev, part)
    Ahat = (A + np.eye(n)) / (A.sum(1) + 1.0)[:, None]
    H = X
    L = len(dims) - 1
    for l in range(L):
        M = Ahat @ H
        if l < L - 1:
            M = _bf16_lib(M)
        Z = np.stack([M[i] @ W[l][part[i] if W[l].shape[0] > 1 else 0] for i in range(n)])
        H = _bf16_lib(np.maximum(Z, 0.0)) if l < L - 1 else Z
    z = H[:, 0]
    p = 1.0 / (1.0 + np.exp(-z))
    S = int(part.max()) + 1
    loss = np.zeros(S)
    for s in range(S):
        ps = p * (part == s)
        loss[s] = ALPHA * 0.5 * ps @ A @ ps - BETA * ps.sum() + lam * (pen * ps).sum()
    return z, p, loss


@pytest.mark.parametrize("dims,sets_shared", [([6, 4, 1], False), ([7, 5, 3, 1], False), ([7, 5, 3, 1], True)])
def test_bf16_storage_forward_matches_dense_definition_with_rounding_written_out(dims, sets_shared):
    n, S = 40, 4
    eu, ev, part = tiny_graph(n, 0.25, S, seed=11)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    X = si.round_to_bf16(rand_features(n, dims[0], 5).astype(np.float32)).astype(np.float64)
    W = [si.round_to_bf16(w.astype(np.float32)).astype(np.float64)
         for w in rand_weights(dims, 1 if sets_shared else S, 7, scale=2.0)]
    pen = (si.uniform01(99, 0, n) < 0.3).astype(np.float64)
    z, p, loss = _dense_forward_loss_bf16_storage(n, eu, ev, part, dims, X, W, pen, 0.7)
    r = oracle.train_step(b, dims, X[b["perm"]], W, ALPHA, BETA, 0.7, pen[b["perm"]], store_bf16=True)
    # sums of a handful of double products in a different order: a few ulps of double, far below the
    # 2^-9 relative size of one bfloat16 rounding (a missing or an extra rounding shows at ~1e-3)
    np.testing.assert_allclose(r["z"], z[b["perm"]], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(r["p"], p[b["perm"]], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(r["loss"], loss, rtol=1e-11, atol=1e-11)
    # and the mode does change the result on such inputs (otherwise the check above says nothing)
    plain = oracle.train_step(b, dims, X[b["perm"]], W, ALPHA, BETA, 0.7, pen[b["perm"]], store_bf16=False)
    assert np.abs(plain["z"] - r["z"]).max() > 1e-5


def test_bf16_storage_hidden_preactivations_and_output_layer_keep_full_precision():
    # what is rounded is what is stored: Z_l (never stored) is the double product of the ROUNDED M_l,
    # and the last layer's aggregate is not rounded
    n, S, dims = 30, 3, [5, 4, 1]
    eu, ev, part = tiny_graph(n, 0.3, S, seed=17)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    perm = b["perm"]
    X = si.round_to_bf16(rand_features(n, dims[0], 8).astype(np.float32)).astype(np.float64)
    W = [si.round_to_bf16(w.astype(np.float32)).astype(np.float64) for w in rand_weights(dims, S, 9, scale=2.0)]
    r = oracle.train_step(b, dims, X[perm], W, ALPHA, BETA, want_Z=True, store_bf16=True)
    A = dense_intra_adjacency(n, eu, ev, part)
    Ahat = (A + np.eye(n)) / (A.sum(1) + 1.0)[:, None]
    M1 = _bf16_lib(Ahat @ X)
    Z1 = np.stack([M1[i] @ W[0][part[i]] for i in range(n)])
    np.testing.assert_allclose(r["Z"][0], Z1[perm], rtol=1e-12, atol=1e-13)
    H1 = _bf16_lib(np.maximum(Z1, 0.0))
    M2 = Ahat @ H1                                               # output layer: not rounded
    z = np.array([M2[i] @ W[1][part[i]][:, 0] for i in range(n)])
    np.testing.assert_allclose(r["z"], z[perm], rtol=1e-12, atol=1e-13)
    assert np.abs(_bf16_lib(M2) - M2).max() > 1e-4               # rounding M2 would have been visible


def test_bf16_storage_mode_is_a_no_op_when_every_stored_value_is_a_bf16_number():
    # degrees 0, 1 and 3 (means divide by 1, 2, 4), small integer features, weights in {-1, 0, 1} with a
    # signed permutation in the second layer: every M_l and H_l is a multiple of 1/16 below 2^4, i.e.
    # a bfloat16 number, so the two modes must agree bit for bit -- loss, p and every gradient
    n, S, dims = 24, 2, [4, 4, 4, 1]
    edges = [(0, 1), (2, 3), (4, 5), (4, 6), (4, 7), (5, 6), (5, 7), (6, 7),          # part 0: pairs and a K4
             (12, 13), (14, 15), (16, 17), (16, 18), (16, 19), (17, 18), (17, 19), (18, 19), (20, 21)]
    eu = np.array([a for a, _ in edges], np.int32)
    ev = np.array([c for _, c in edges], np.int32)
    part = (np.arange(n) >= 12).astype(np.int32)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    assert set(np.diff(b["rowptr"]).tolist()) == {0, 1, 3}
    X = (si.u64(5, 0, n * 4) % np.uint64(5)).astype(np.float64).reshape(n, 4) - 2.0
    W0 = (si.u64(6, 0, S * 16) % np.uint64(3)).astype(np.float64).reshape(S, 4, 4) - 1.0
    P = np.zeros((S, 4, 4))
    for s in range(S):
        for k, (j, sign) in enumerate(zip([2, 0, 3, 1], [1.0, -1.0, 1.0, 1.0])):
            P[s, k, (j + s) % 4] = sign
    W2 = (si.u64(7, 0, S * 4) % np.uint64(3)).astype(np.float64).reshape(S, 4, 1) - 1.0
    W = [W0, P, W2]
    a = oracle.train_step(b, dims, X, W, ALPHA, BETA, want_dX=True, want_Z=True, store_bf16=False)
    c = oracle.train_step(b, dims, X, W, ALPHA, BETA, want_dX=True, want_Z=True, store_bf16=True)
    assert np.abs(a["Z"][0]).max() > 0 and (a["Z"][1] > 0).any()
    for key in ("loss", "p", "z", "dX"):
        assert np.array_equal(a[key], c[key]), key
    for l in range(3):
        assert np.array_equal(a["dW"][l], c["dW"][l])
        if l < 2:
            assert np.array_equal(a["Z"][l], c["Z"][l])


def test_bf16_storage_gradients_are_those_of_the_rounded_forward_values():
    # The backward pass of the bfloat16 mode is the exact derivative taken AT the stored values
    # (straight-through: the rounding itself has no derivative).  With one hidden layer,
    #   dW_2 = (A_hat H_1)^T dz       with H_1 the rounded activation,
    #   dW_1 = M_1^T ((A_hat^T dz w_2^T) * [Z_1 > 0])   with M_1 the rounded aggregate.
    n, S, dims = 36, 3, [5, 4, 1]
    eu, ev, part = tiny_graph(n, 0.25, S, seed=23)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    perm = b["perm"]
    X = si.round_to_bf16(rand_features(n, dims[0], 2).astype(np.float32)).astype(np.float64)
    W = [si.round_to_bf16(w.astype(np.float32)).astype(np.float64) for w in rand_weights(dims, S, 3, scale=2.0)]
    r = oracle.train_step(b, dims, X[perm], W, ALPHA, BETA, store_bf16=True)
    A = dense_intra_adjacency(n, eu, ev, part)
    Ahat = (A + np.eye(n)) / (A.sum(1) + 1.0)[:, None]
    M1 = _bf16_lib(Ahat @ X)
    Z1 = np.stack([M1[i] @ W[0][part[i]] for i in range(n)])
    H1 = _bf16_lib(np.maximum(Z1, 0.0))
    M2 = Ahat @ H1
    z = np.array([M2[i] @ W[1][part[i]][:, 0] for i in range(n)])
    p = 1.0 / (1.0 + np.exp(-z))
    dz = (ALPHA * (A @ p) - BETA) * p * (1 - p)
    g = Ahat.T @ dz
    for s in range(S):
        msk = part == s
        np.testing.assert_allclose(r["dW"][1][s][:, 0], M2[msk].T @ dz[msk], rtol=1e-10, atol=1e-12)
        dZ1 = np.outer(g[msk], W[1][s][:, 0]) * (Z1[msk] > 0)
        np.testing.assert_allclose(r["dW"][0][s], M1[msk].T @ dZ1, rtol=1e-10, atol=1e-12)


# ----------------------------------------------------------- block-diagonal batch pin
def test_batch_equals_independent_subgraph_runs_bit_for_bit():
    n, S, dims = 90, 6, [6, 5, 4, 1]
    eu, ev, part = tiny_graph(n, 0.12, S, seed=91)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    X = rand_features(n, dims[0], 33)
    W = rand_weights(dims, S, 35)
    pen = (si.uniform01(7, 0, n) < 0.2).astype(np.float64)
    r = oracle.train_step(b, dims, X[b["perm"]], W, ALPHA, BETA, 0.5, pen[b["perm"]], want_dX=True, threads=3)
    for s in range(S):
        nodes = np.where(part == s)[0]                      # ascending original ids = new order inside s
        loc = {int(v): i for i, v in enumerate(nodes)}
        nbrs = [[] for _ in nodes]
        for a, c in zip(eu.tolist(), ev.tolist()):
            if a in loc and c in loc:
                nbrs[loc[a]].append(loc[c])
                nbrs[loc[c]].append(loc[a])
        rp = np.concatenate([[0], np.cumsum([len(x) for x in nbrs])]).astype(np.int32)
        ci = np.array([j for x in nbrs for j in sorted(x)], np.int32)
        one = oracle.subgraph_step(rp, ci, dims, X[nodes], [w[s] for w in W], ALPHA, BETA, 0.5, pen[nodes],
                                   want_dX=True)
        lo, hi = b["part_ptr"][s], b["part_ptr"][s + 1]
        assert one["loss"] == r["loss"][s]
        assert np.array_equal(one["p"], r["p"][lo:hi])
        assert np.array_equal(one["dX"], r["dX"][lo:hi])
        for l in range(len(W)):
            assert np.array_equal(one["dW"][l], r["dW"][l][s])


def test_shared_weight_gradient_is_sum_over_subgraphs():
    n, S, dims = 60, 4, [5, 3, 1]
    eu, ev, part = tiny_graph(n, 0.15, S, seed=95)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    X = rand_features(n, 5, 1)
    W1 = rand_weights(dims, 1, 2)
    WS = [np.tile(w, (S, 1, 1)) for w in W1]
    shared = oracle.train_step(b, dims, X, W1, ALPHA, BETA)
    per = oracle.train_step(b, dims, X, WS, ALPHA, BETA)
    for l in range(2):
        np.testing.assert_allclose(shared["dW"][l][0], per["dW"][l].sum(0), rtol=1e-12, atol=1e-14)
    assert np.array_equal(shared["p"], per["p"])


# ------------------------------------------------------------------------ Adam (a7)
def test_adam_two_steps_against_exact_rational_arithmetic():
    decimal.getcontext().prec = 60
    lr, b1, b2, eps = Fraction(1, 10), Fraction(9, 10), Fraction(999, 1000), Fraction(1, 10 ** 8)
    g = [Fraction(1, 2), Fraction(-1, 4)]
    W, m, v = Fraction(3, 10), Fraction(0), Fraction(0)
    expect = []
    for t in (1, 2):
        m = b1 * m + (1 - b1) * g[t - 1]
        v = b2 * v + (1 - b2) * g[t - 1] ** 2
        mh, vh = m / (1 - b1 ** t), v / (1 - b2 ** t)
        root = decimal.Decimal(vh.numerator) / decimal.Decimal(vh.denominator)
        root = root.sqrt()
        step = (decimal.Decimal(mh.numerator) / decimal.Decimal(mh.denominator)) / (
            root + decimal.Decimal(eps.numerator) / decimal.Decimal(eps.denominator))
        W = W - lr * Fraction(step)
        expect.append(float(W))
    Wd, md, vd = np.array([0.3]), np.zeros(1), np.zeros(1)
    got = []
    for t in (1, 2):
        oracle.adam(Wd, md, vd, np.array([float(g[t - 1])]), 0.1, t, 0.9, 0.999, 1e-8)
        got.append(float(Wd[0]))
    np.testing.assert_allclose(got, expect, rtol=1e-14)
    # the first step moves by lr*g/(|g|+eps): almost exactly lr against the gradient sign
    assert abs((0.3 - got[0]) - 0.1 * 0.5 / (0.5 + 1e-8)) < 1e-15


def test_adam_first_step_is_sign_step_and_zero_gradient_stays():
    g = np.array([3.0, -0.02, 0.0, 1e-3])
    W, m, v = np.ones(4), np.zeros(4), np.zeros(4)
    oracle.adam(W, m, v, g, 1e-3, 1)
    np.testing.assert_allclose(1.0 - W, 1e-3 * g / (np.abs(g) + 1e-8), rtol=1e-12, atol=0)
    assert W[2] == 1.0


# ------------------------------------------------------------- partition quality (Section 3.1)
@pytest.mark.parametrize("n,p,S,seed", [(30, 0.2, 4, 1), (60, 0.1, 7, 2), (25, 0.3, 1, 3), (40, 0.15, 40, 4)])
def test_partition_quality_matches_networkx_and_the_pairwise_definition(n, p, S, seed):
    import networkx as nx
    eu, ev, part = tiny_graph(n, p, S, seed=700 + seed)
    S = max(S, int(part.max()) + 1)
    r = oracle.partition_quality(eu, ev, part, S)
    G = nx.Graph()
    G.add_nodes_from(range(n))
    G.add_edges_from(zip(eu.tolist(), ev.tolist()))
    groups = [set(np.nonzero(part == s)[0].tolist()) for s in range(S)]
    groups = [g for g in groups if g]
    np.testing.assert_allclose(r["Q"], nx.community.modularity(G, groups), rtol=1e-12, atol=1e-15)
    # pairwise definition: Q = 1/(2m) sum_ij [A_ij - k_i k_j / 2m] [c_i = c_j]
    A = np.zeros((n, n))
    A[eu, ev] = 1.0
    A[ev, eu] = 1.0
    k = A.sum(axis=1)
    m = eu.size
    same = part[:, None] == part[None, :]
    np.testing.assert_allclose(r["Q"], ((A - np.outer(k, k) / (2 * m)) * same).sum() / (2 * m), rtol=1e-12, atol=1e-15)
    # integer parts, brute force
    for s in range(S):
        inside = sum(1 for a, c in zip(eu.tolist(), ev.tolist()) if part[a] == s and part[c] == s)
        assert r["in_edges"][s] == inside and r["tot"][s] == int(k[part == s].sum())
    assert r["tot"].sum() == 2 * m


def test_delta_q_is_the_exact_change_of_modularity():
    # move node i out of its own singleton community into a neighbour's community: Q changes by Eq. 2
    n, S0 = 24, 3
    eu, ev, part = tiny_graph(n, 0.25, S0, seed=801)
    m = eu.size
    deg = np.bincount(np.concatenate([eu, ev]), minlength=n)
    for i in (2, 7, 13):
        alone = part.copy()
        alone[i] = S0                                    # i in a community of its own
        before = oracle.partition_quality(eu, ev, alone, S0 + 1)
        for target in range(S0):
            joined = alone.copy()
            joined[i] = target
            after = oracle.partition_quality(eu, ev, joined, S0 + 1)
            k_i_in = sum(1 for a, c in zip(eu.tolist(), ev.tolist())
                         if (a == i and alone[c] == target) or (c == i and alone[a] == target))
            gain = oracle.delta_q(k_i_in, before["tot"][target], deg[i], m)
            np.testing.assert_allclose(after["Q"] - before["Q"], gain, rtol=1e-10, atol=1e-14)


# ------------------------------------------------- Gumbel-softmax input processing (Section 3.2)
def test_gumbel_softmax_without_noise_is_the_library_softmax():
    from scipy.special import softmax
    E = rand_features(37, 12, 5)
    for tau in (0.3, 1.0, 4.0):
        np.testing.assert_allclose(oracle.gumbel_softmax(E, None, tau), softmax(E / tau, axis=1), rtol=1e-13, atol=0)


def test_gumbel_softmax_two_features_closed_form():
    # e = (0, 0), tau = 1:  x_0 = 1 / (1 + exp(g_1 - g_0)) with exp(-g) = -ln u, i.e. x_0 = ln u_1 / ln(u_0 u_1)
    U = np.array([[0.2, 0.7], [0.9, 0.05], [0.5, 0.5]])
    x = oracle.gumbel_softmax(np.zeros((3, 2)), U, 1.0)
    expect0 = np.log(U[:, 1]) / np.log(U[:, 0] * U[:, 1])
    np.testing.assert_allclose(x[:, 0], expect0, rtol=1e-13)
    np.testing.assert_allclose(x[:, 1], 1.0 - expect0, rtol=1e-13)
    # temperature divides BOTH the embedding and the noise: e = (ln 3, 0), tau = 1/2, no noise -> odds 9 : 1
    y = oracle.gumbel_softmax(np.array([[np.log(3.0), 0.0]]), None, 0.5)
    np.testing.assert_allclose(y, [[0.9, 0.1]], rtol=1e-13)
    z = oracle.gumbel_softmax(np.zeros((1, 2)), np.array([[0.2, 0.7]]), 0.5)
    odds = (np.log(0.7) / np.log(0.2)) ** 2                      # exp((g_0 - g_1) / tau)
    np.testing.assert_allclose(z[0, 0] / z[0, 1], odds, rtol=1e-12)


def test_gumbel_softmax_invariants_and_temperature_limits():
    n, F = 50, 9
    E = rand_features(n, F, 8)
    U = si.uniform01(91, 0, n * F).reshape(n, F)
    x = oracle.gumbel_softmax(E, U, 0.7)
    assert np.all(x > 0) and np.all(x < 1)
    np.testing.assert_allclose(x.sum(axis=1), 1.0, rtol=1e-14)
    # a constant added to a row changes nothing; rows do not interact
    np.testing.assert_allclose(oracle.gumbel_softmax(E + 3.25, U, 0.7), x, rtol=1e-12)
    np.testing.assert_allclose(oracle.gumbel_softmax(E[7:8], U[7:8], 0.7), x[7:8], rtol=1e-14)
    # hot: close to uniform; cold: one-hot at the arg max of embedding + noise
    hot = oracle.gumbel_softmax(E, U, 1e6)
    assert np.max(np.abs(hot - 1.0 / F)) < 1e-4
    cold = oracle.gumbel_softmax(E, U, 1e-3)
    winner = np.argmax(E - np.log(-np.log(U)), axis=1)
    assert np.array_equal(np.argmax(cold, axis=1), winner) and np.all(cold.max(axis=1) > 1 - 1e-3)


def test_gumbel_max_trick_reproduces_the_softmax_distribution():
    # arg max of (e + g) is distributed as softmax(e): pins the noise law -log(-log u) statistically
    from scipy.special import softmax
    e = np.array([0.5, -1.0, 1.5, 0.0])
    N = 200_000
    U = si.uniform01(123, 0, N * 4).reshape(N, 4)
    cold = oracle.gumbel_softmax(np.broadcast_to(e, (N, 4)), U, 1e-2)
    freq = np.bincount(np.argmax(cold, axis=1), minlength=4) / N
    prob = softmax(e)
    sigma = np.sqrt(prob * (1 - prob) / N)
    assert np.all(np.abs(freq - prob) < 5 * sigma)


# --------------------------------------------------------------------- decode (a8, a9)
@pytest.mark.parametrize("seed", [1, 2, 3])
def test_decode_brute_force(seed):
    n, S = 45, 5
    eu, ev, part = tiny_graph(n, 0.2, S, seed=100 + seed)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    p_orig = si.uniform01(seed, 0, n).astype(np.float32)
    p_orig[::7] = 0.5                                             # ties go to "selected"
    d = oracle.decode(b, p_orig[b["perm"]])
    x = (p_orig >= np.float32(0.5)).astype(np.uint8)
    assert np.array_equal(d["x"], x[b["perm"]])
    intra = bnd = 0
    per = np.zeros(S, np.int64)
    for a, c in zip(eu.tolist(), ev.tolist()):
        if x[a] and x[c]:
            if part[a] == part[c]:
                intra += 1
            else:
                bnd += 1
                per[part[a]] += 1
                per[part[c]] += 1
    assert (d["set_size"], d["intra_viol"], d["boundary_viol"]) == (int(x.sum()), intra, bnd)
    assert np.array_equal(d["per_part"], per) and d["per_part"].sum() == 2 * bnd
    for e in range(b["E_b"]):
        u, v = b["perm"][b["bnd_u"][e]], b["perm"][b["bnd_v"][e]]
        assert d["viol"][e] == (x[u] & x[v])


# ------------------------------------------------------------- trajectory (sanity only)
def test_config1_training_lowers_every_subgraph_loss():
    w = si.make_workload(1)
    b = oracle.bookkeeping(w.n, w.eu, w.ev, w.part, w.S)
    X = w.features_f32()[b["perm"]].astype(np.float64)
    W = [w.weights(l).astype(np.float64) for l in range(w.L)]
    m = [np.zeros_like(x) for x in W]
    v = [np.zeros_like(x) for x in W]
    first = None
    for t in range(1, w.steps + 1):
        r = oracle.train_step(b, w.dims, X, W, w.alpha, w.beta, threads=4)
        if first is None:
            first = r["loss"].copy()
        for l in range(w.L):
            oracle.adam(W[l], m[l], v[l], r["dW"][l], w.lr, t)
    last = oracle.train_step(b, w.dims, X, W, w.alpha, w.beta, want_dW=False)["loss"]
    assert np.all(last < first)


# ------------------------------------------------- Stage-3 glue (conflicts -> fine-tune inputs)
@pytest.mark.parametrize("seed", [1, 2, 3])
def test_conflict_list_base_action_and_penalty_brute_force(seed):
    n, S = 60, 6
    eu, ev, part = tiny_graph(n, 0.15, S, seed=200 + seed)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    # three probability levels only, so that many conflict edges join endpoints with EQUAL p
    p_orig = np.array([0.2, 0.6, 0.9], np.float32)[(si.u64(300 + seed, 0, n) % np.uint64(3)).astype(int)]
    p_new = p_orig[b["perm"]]
    d = oracle.decode(b, p_new)
    conf = oracle.conflict_list(b, d["viol"])
    # brute force over the ORIGINAL edge list
    x = p_orig >= np.float32(0.5)
    want = set()
    for a, c in zip(eu.tolist(), ev.tolist()):
        if part[a] != part[c] and x[a] and x[c]:
            na, nc = int(b["inv_perm"][a]), int(b["inv_perm"][c])
            want.add((min(na, nc), max(na, nc)))
    got = [(int(b["bnd_u"][e]), int(b["bnd_v"][e])) for e in conf]
    assert got == sorted(want) and len(conf) == d["boundary_viol"]
    assert np.all(np.diff(conf) > 0)
    act = oracle.base_action(b, conf, p_new)
    assert any(p_new[b["bnd_u"][e]] == p_new[b["bnd_v"][e]] for e in conf)      # ties are exercised
    chosen = set()
    for e, a in zip(conf.tolist(), act.tolist()):
        u, v = int(b["bnd_u"][e]), int(b["bnd_v"][e])
        lower = u if p_new[u] < p_new[v] else v                 # smaller probability, ties -> larger id (v > u)
        assert (u, v)[a] == lower
        chosen.add(lower)
    r = oracle.apply_actions(b, conf, act)
    assert r["chosen"] == len(chosen)
    assert set(np.nonzero(r["pen"])[0].tolist()) == chosen and set(np.unique(r["pen"]).tolist()) <= {0.0, 1.0}
    assert set(np.nonzero(r["active"])[0].tolist()) == {int(b["node_part"][i]) for i in chosen}
    # removing the chosen nodes resolves every boundary conflict and touches nothing else
    p_fixed = p_new.copy()
    p_fixed[sorted(chosen)] = 0.0
    d2 = oracle.decode(b, p_fixed)
    assert d2["boundary_viol"] == 0 and d2["set_size"] == d["set_size"] - len(chosen)
    # the opposite choice is also a valid action vector and gives its own node list
    r2 = oracle.apply_actions(b, conf, 1 - act)
    other = {(int(b["bnd_u"][e]), int(b["bnd_v"][e]))[1 - a] for e, a in zip(conf.tolist(), act.tolist())}
    assert set(np.nonzero(r2["pen"])[0].tolist()) == other


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_repair_removes_exactly_the_chosen_nodes_brute_force(seed):
    n, S = 70, 5
    eu, ev, part = tiny_graph(n, 0.15, S, seed=400 + seed)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    p_new = si.uniform01(500 + seed, 0, n).astype(np.float32)
    d = oracle.decode(b, p_new)
    conf = oracle.conflict_list(b, d["viol"])
    assert conf.size > 0
    for act in (oracle.base_action(b, conf, p_new), (si.u64(600 + seed, 0, conf.size) & np.uint64(1)).astype(np.uint8)):
        pen = oracle.apply_actions(b, conf, act)["pen"]
        r = oracle.repair(d["x"], pen)
        # brute force on the ORIGINAL graph: drop the chosen endpoint of every violated cross edge
        x0 = p_new[b["inv_perm"]] >= np.float32(0.5)                 # original order
        drop = set()
        for e, a in zip(conf.tolist(), act.tolist()):
            drop.add(int(b["perm"][(int(b["bnd_u"][e]), int(b["bnd_v"][e]))[a]]))
        x1 = x0.copy()
        x1[sorted(drop)] = False
        assert np.array_equal(r["x"], x1[b["perm"]].astype(np.uint8)) and r["removed"] == len(drop)
        # no cross edge of the original graph has both ends selected any more; intra conflicts are untouched
        cross_left = sum(1 for a, c in zip(eu.tolist(), ev.tolist()) if part[a] != part[c] and x1[a] and x1[c])
        assert cross_left == 0
        d2 = oracle.decode(b, r["x"].astype(np.float32))
        assert d2["boundary_viol"] == 0 and d2["set_size"] == d["set_size"] - len(drop)
        assert d2["intra_viol"] <= d["intra_viol"]
    # nodes that are not selected are not counted, and a zero vector changes nothing
    pen = np.zeros(n, np.float32)
    pen[np.nonzero(d["x"] == 0)[0][:3]] = 1.0
    r = oracle.repair(d["x"], pen)
    assert r["removed"] == 0 and np.array_equal(r["x"], d["x"])


def test_stage3_glue_on_empty_conflict_set():
    n, S = 20, 4
    eu, ev, part = tiny_graph(n, 0.2, S, seed=7)
    b = oracle.bookkeeping(n, eu, ev, part, S)
    d = oracle.decode(b, np.zeros(n, np.float32))
    conf = oracle.conflict_list(b, d["viol"])
    assert conf.size == 0
    r = oracle.apply_actions(b, conf, np.zeros(0, np.uint8))
    assert r["chosen"] == 0 and not r["pen"].any() and not r["active"].any()
