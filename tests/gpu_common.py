"""Helpers of the GPU parity tests: run the CUDA library through its binding and the
oracle on the same seeded inputs, and compare element by element."""
import numpy as np

import oracle
import synth_inputs as si

# Tolerances.  The acceptance criteria state: float32 features rtol 1e-4 / atol 1e-5; bfloat16
# features rtol 2e-2.  They are applied FLAT (exactly as stated) to every tensor first:
#   float32:   |err| <= 1e-4 |ref| + 1e-5
#   bfloat16:  |err| <= 2e-2 |ref| + BF16_ATOL   (the criteria give bfloat16 no absolute part; a value
#              next to zero needs one.  A stored bf16 value carries 2^-9 relative rounding; both sides
#              round the same tensors, so they differ only where float32 and double sums fall on two
#              sides of a rounding boundary: one bf16 ulp (2^-8) of one O(1) activation times one
#              O(0.1) weight, a few 1e-4 in z.  BF16_ATOL = 2e-3 leaves a margin over that.)
# loss, p and z are held to the flat bound, always.
# GRADIENT tensors that miss the flat bound get a second, scaled bound, and every use of it is
# counted and printed (``Report``): the absolute part is taken in units of the scale of the entry's
# own group -- the subgraph's matrix for dW, the node's row for dX:
#   float32:   atol = 1e-5 * max(1, largest |ref| of the group).  A gradient entry is a sum of up to
#              thousands of products; in hub subgraphs entries reach the hundreds, and a float32 sum
#              cannot resolve 1e-5 of a cancelling entry (round-off eps * sqrt(terms) * partial sums).
#   bfloat16:  atol = 2^-6 * largest |ref| of the group (an entry that is a cancelling sum of K stored
#              values inherits 2^-9 * sum |terms| per rounding along the chain).
# bfloat16 gradients only: a hidden activation on a bf16 rounding boundary can differ by one ulp between
# the float32-accumulating kernel and the double-accumulating oracle; the next layer's pre-activations
# move by ~1e-4 and the few units that close to zero flip their ReLU mask, which changes a handful of
# gradient rows by a few percent.  Neither side is wrong, so at most BF16_GRAD_OUTLIER_FRAC of a bf16
# gradient tensor's entries may miss the scaled bound provided ||err||_F <= BF16_GRAD_NORM_RTOL ||ref||_F.
F32_RTOL, F32_ATOL = 1e-4, 1e-5
BF16_RTOL, BF16_ATOL = 2e-2, 2e-3
BF16_GROUP_ATOL_SCALE = 2.0 ** -6
BF16_GRAD_OUTLIER_FRAC = 2e-3
BF16_GRAD_NORM_RTOL = 2e-2


class Report:
    """Which bound each compared tensor needed; printed by the tests so that a drift inside the
    wider bounds is seen."""

    def __init__(self):
        self.rows = {}

    def add(self, name, entries, worst, scaled, outliers):
        r = self.rows.setdefault(name, dict(entries=0, worst=0.0, scaled=0, outliers=0))
        r["entries"] += entries
        r["worst"] = max(r["worst"], worst)
        r["scaled"] += scaled
        r["outliers"] += outliers

    def needs_only_flat(self, name):
        r = self.rows.get(name)
        return r is None or (r["scaled"] == 0 and r["outliers"] == 0)

    def __str__(self):
        out = []
        for name in sorted(self.rows):
            r = self.rows[name]
            how = "flat bound" if not (r["scaled"] or r["outliers"]) else (
                "%d entries needed the group-scaled bound, %d outliers under the norm rule" % (r["scaled"], r["outliers"]))
            out.append("  %-6s %10d entries, worst |err| %.3g: %s" % (name, r["entries"], r["worst"], how))
        return "\n".join(out)


def flat_tolerances(dtype):
    return (BF16_RTOL, BF16_ATOL) if dtype == "bf16" else (F32_RTOL, F32_ATOL)


def assert_close(got, ref, dtype, what, skip_mask=None, group_axes=None, report=None, name=None):
    """Element-wise comparison.  Without ``group_axes`` only the flat bound applies (loss, p, z).
    ``group_axes`` (gradient tensors) names the axes over which an entry's group extends -- (1, 2) for
    dW [sets, F_in, F_out], (1,) for dX [rows, F] -- and enables the scaled bound and, for bfloat16,
    the outlier rule.  Returns the largest absolute error."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    rtol, atol = flat_tolerances(dtype)
    err = np.abs(got - ref)
    checked = np.ones(err.shape, bool) if skip_mask is None else ~skip_mask
    bad = (err > atol + rtol * np.abs(ref)) & checked
    n_scaled = n_out = 0
    if bad.any() and group_axes is not None:
        top = np.abs(ref).max(axis=tuple(group_axes), keepdims=True) if ref.size else 0.0
        wide = BF16_GROUP_ATOL_SCALE * top + atol if dtype == "bf16" else F32_ATOL * np.maximum(1.0, top)
        still = (err > wide + rtol * np.abs(ref)) & checked
        n_scaled = int(bad.sum() - still.sum())
        bad = still
        if bad.any() and dtype == "bf16":
            frac = bad.sum() / max(1, checked.sum())
            rel = float(np.linalg.norm((got - ref)[checked]) / max(np.linalg.norm(ref[checked]), 1e-30))
            assert frac <= BF16_GRAD_OUTLIER_FRAC and rel <= BF16_GRAD_NORM_RTOL, (
                "%s: %.3g of entries outside the scaled bound, norm-wise error %.3g" % (what, frac, rel))
            n_out = int(bad.sum())
            bad = np.zeros_like(bad)
    if bad.any():
        k = np.unravel_index(np.argmax(np.where(bad, err, 0)), err.shape)
        raise AssertionError("%s: %d of %d entries outside rtol=%g atol=%g%s; worst at %s: got %r, expected %r"
                             % (what, int(bad.sum()), bad.size, rtol, atol,
                                " (group-scaled)" if group_axes is not None else "", k, got[k], ref[k]))
    worst = float(err[checked].max()) if checked.any() else 0.0
    if report is not None:
        report.add(name or what, int(checked.sum()), worst, n_scaled, n_out)
    return worst


def _adam_hyper(adam):
    """(lr, step, beta1, beta2, eps) as the float32 values the C ABI carries."""
    f = lambda x: float(np.float32(x))
    return f(adam["lr"]), adam["step"], f(0.9), f(0.999), f(1e-8)


def torch_dev():
    import torch
    return torch.device("cuda:0")


def to_dev(a, dtype=None):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a)).to(torch_dev())
    return t if dtype is None else t.to(dtype)


def load_graph(n, eu, ev, part, S):
    import paper_2511_09261_b200 as gnnco
    return gnnco.gnnco_partition_load(to_dev(eu.astype(np.int32)), to_dev(ev.astype(np.int32)),
                                      to_dev(part.astype(np.int32)), S)


def check_bookkeeping(graph, book):
    """Bit-exact comparison of every array gnnco_partition_load builds."""
    assert (graph.n, graph.S, graph.E_in, graph.E_b) == (book["n"], book["S"], book["E_in"], book["E_b"])
    arr = graph.arrays()
    for key in ("perm", "inv_perm", "part_ptr", "node_part", "rowptr", "colidx", "bnd_u", "bnd_v", "is_boundary"):
        got = arr[key].cpu().numpy()
        assert np.array_equal(got, book[key]), key
    got = arr["inv_deg"].cpu().numpy()
    assert np.array_equal(got.view(np.uint32), book["inv_deg"].view(np.uint32)), "inv_deg"
    deg = np.diff(book["rowptr"])
    assert graph.max_row == (int(deg.max()) if deg.size else 0)


class StepCase:
    """One teacher-forced step: same X, W, (m, v) on both sides; compares loss, p, z,
    every dW, dX and the Adam-updated weights."""

    def __init__(self, book, dims, dtype="f32", sets=None, alpha=2.0, beta=1.0, lam=0.0):
        self.book, self.dims, self.dtype = book, list(dims), dtype
        self.L = len(dims) - 1
        self.S, self.n = int(book["S"]), int(book["n"])
        self.sets = self.S if sets is None else sets
        self.alpha, self.beta, self.lam = alpha, beta, lam
        self.report = Report()
        self.extra_flags = 0                      # ORed into the step's flags (e.g. ONE_KERNEL_LAYERS)

    def run(self, graph, X_new, W, pen_new=None, want_dx=True, adam=None, threads=4, parts=None, label=""):
        """X_new [n,F0] float32 numpy (bf16-representable when dtype is bf16), W list of
        float32 numpy [sets,Fi,Fo]; adam = dict(m=[...], v=[...], step=t, lr=...) or None.
        parts: compare only these subgraphs (the oracle then runs only them)."""
        import torch
        import paper_2511_09261_b200 as gnnco
        bf16 = self.dtype == "bf16"
        fd = gnnco.BF16 if bf16 else gnnco.F32
        Xd = to_dev(X_new, torch.bfloat16 if bf16 else torch.float32)
        Wd = [to_dev(w) for w in W]
        model = gnnco.Model(self.dims, Wd, fd)
        opt = None
        if adam is not None:
            opt = gnnco.Adam(model, lr=adam["lr"])
            opt.step = adam["step"]
            opt.m = [to_dev(m) for m in adam["m"]]
            opt.v = [to_dev(v) for v in adam["v"]]
        dW = [torch.full_like(w, float("nan")) for w in Wd]
        z = torch.full((self.n,), float("nan"), device=Xd.device)
        dX = torch.full_like(Xd, float("nan")) if want_dx else None
        pen_d = to_dev(pen_new.astype(np.float32)) if pen_new is not None else None
        flags = (gnnco.WANT_DX if want_dx else 0) | self.extra_flags
        loss, p = graph.train_step(model, Xd, self.alpha, self.beta, self.lam, pen_d, opt, z=z, dW=dW, dX=dX,
                                   flags=flags)
        torch.cuda.synchronize()
        assert graph.async_status() == 0
        g = dict(loss=loss.cpu().numpy(), p=p.cpu().numpy(), z=z.cpu().numpy(),
                 dW=[t.cpu().numpy() for t in dW], dX=None if dX is None else dX.float().cpu().numpy(),
                 W=[t.cpu().numpy() for t in Wd])
        if opt is not None:
            g["m"] = [t.cpu().numpy() for t in opt.m]
            g["v"] = [t.cpu().numpy() for t in opt.v]
        # ---- oracle (weights as the matrix products see them: bf16-rounded for bf16 runs)
        Wc = [si.round_to_bf16(w) if bf16 else w for w in W]
        stats = {}
        if parts is None:
            r = oracle.train_step(self.book, self.dims, X_new, Wc, self.alpha, self.beta, self.lam, pen_new,
                                  want_dX=want_dx, want_Z=True, threads=threads, store_bf16=bf16)
            self._compare(g, r, slice(None), None, W, adam, stats, label)
        else:
            for s in parts:
                lo, hi = int(self.book["part_ptr"][s]), int(self.book["part_ptr"][s + 1])
                if hi == lo:
                    continue
                rp = self.book["rowptr"][lo:hi + 1] - self.book["rowptr"][lo]
                ci = self.book["colidx"][self.book["rowptr"][lo]:self.book["rowptr"][hi]] - lo
                ws = [w[s if self.sets > 1 else 0] for w in Wc]
                one = oracle.subgraph_step(rp, ci, self.dims, X_new[lo:hi], ws, self.alpha, self.beta, self.lam,
                                           None if pen_new is None else pen_new[lo:hi], want_dX=want_dx,
                                           want_Z=True, store_bf16=bf16)
                r = dict(loss=np.array([one["loss"]]), p=one["p"], z=one["z"], dX=one["dX"],
                         dW=[d[None] for d in one["dW"]], Z=one["Z"])
                self._compare(g, r, slice(lo, hi), s, W, adam, stats, "%s part %d" % (label, s))
        return g, stats

    def _compare(self, g, r, rows, s, W, adam, stats, label):
        dt = self.dtype
        sel = slice(None) if s is None else slice(s, s + 1)
        rep = self.report
        stats["loss"] = max(stats.get("loss", 0), assert_close(g["loss"][sel], r["loss"], dt, label + " loss", report=rep, name="loss"))
        stats["p"] = max(stats.get("p", 0), assert_close(g["p"][rows], r["p"], dt, label + " p", report=rep, name="p"))
        stats["z"] = max(stats.get("z", 0), assert_close(g["z"][rows], r["z"], dt, label + " z", report=rep, name="z"))
        # A pre-activation that sits on a ReLU kink (|Z| below float32 round-off) decides a 0/1
        # mask that the two sides may round differently.  Such an entry of hidden layer l, in
        # subgraph q and unit h, can only touch column h of dW[l][q], all of dW[l'][q] for
        # l' < l, and the dX rows of q: those are excluded from the comparison and counted.
        base = 0 if s is None else rows.start
        kinks = [set() for _ in range(self.L)]
        for l, Z in enumerate(r["Z"] or []):
            near = np.abs(Z) < 1e-6 * (1.0 + np.abs(Z))
            for i, h in zip(*np.nonzero(near)):
                kinks[l].add((int(self.book["node_part"][i + base]), int(h)))
        kink_parts = set(q for ks in kinks for q, _ in ks)
        stats["kink_units"] = stats.get("kink_units", 0) + sum(len(ks) for ks in kinks)
        shared = self.sets == 1
        if shared and (s is not None or kink_parts):
            return
        for l in range(self.L):
            gd = g["dW"][l][sel] if not shared else g["dW"][l]
            rd = r["dW"][l]
            skip = np.zeros(rd.shape, bool)
            for l2 in range(l, self.L):
                for q, h in kinks[l2]:
                    k = q if s is None else 0
                    if l2 == l:
                        skip[k, :, h] = True
                    else:
                        skip[k] = True
            # after training, dying units pile up just below zero, so a few such entries are
            # expected; most of the tensor must still be compared
            stats["kink_skipped_frac"] = max(stats.get("kink_skipped_frac", 0), float(skip.mean()))
            assert skip.mean() <= 0.3, "too many gradient entries sit behind a ReLU kink"
            stats["dW%d" % l] = max(stats.get("dW%d" % l, 0), assert_close(gd, rd, dt, label + " dW[%d]" % l, skip, (1, 2), rep, "dW%d" % l))
        if r["dX"] is not None and g["dX"] is not None:
            skip = np.zeros(r["dX"].shape, bool)
            for kp in kink_parts:
                lo, hi = int(self.book["part_ptr"][kp]) - base, int(self.book["part_ptr"][kp + 1]) - base
                skip[max(lo, 0):max(hi, 0)] = True
            stats["dX"] = max(stats.get("dX", 0), assert_close(g["dX"][rows], r["dX"], dt, label + " dX", skip, (1,), rep, "dX"))
        if adam is not None and s is None:
            for l in range(self.L):
                # (a) the update rule itself: the oracle's Adam fed with the GPU's own float32
                # gradient must reproduce the GPU's new m, v, W to float32 rounding.  (Adam divides
                # by sqrt(v): where |g| is below its own rounding error the sign of the step is
                # not determined by the mathematics, so the rule is checked on identical gradients.)
                Wn = W[l].astype(np.float64).copy()
                mn, vn = adam["m"][l].astype(np.float64).copy(), adam["v"][l].astype(np.float64).copy()
                oracle.adam(Wn, mn, vn, g["dW"][l].astype(np.float64), *_adam_hyper(adam))
                # float32 rounding of each product: a few 1e-7 of the operands' magnitude
                for key, ref in (("m", mn), ("v", vn), ("W", Wn)):
                    np.testing.assert_allclose(g[key][l], ref, rtol=2e-6, atol=5e-7 * float(np.abs(ref).max()) + 1e-30,
                                               err_msg=label + " adam " + key)
                # (b) end to end with the oracle's own gradient, float32 runs only
                if dt == "f32" and not kink_parts:
                    Wn = W[l].astype(np.float64).copy()
                    mn, vn = adam["m"][l].astype(np.float64).copy(), adam["v"][l].astype(np.float64).copy()
                    oracle.adam(Wn, mn, vn, r["dW"][l], *_adam_hyper(adam))
                    assert_close(g["m"][l], mn, dt, label + " adam m[%d]" % l, None, (1, 2), rep, "adam m")
                    assert_close(g["v"][l], vn, dt, label + " adam v[%d]" % l, None, (1, 2), rep, "adam v")
                    assert_close(g["W"][l], Wn, dt, label + " adam W[%d]" % l, report=rep, name="adam W")


def check_decode(graph, book, p_new_f32):
    """Bit-exact decode parity on the given float32 probabilities (new order)."""
    import torch
    d = graph.decode_boundary(to_dev(p_new_f32.astype(np.float32)))
    torch.cuda.synchronize()
    ref = oracle.decode(book, p_new_f32.astype(np.float32))
    assert np.array_equal(d["x"].cpu().numpy(), ref["x"])
    assert np.array_equal(d["viol"].cpu().numpy(), ref["viol"])
    assert np.array_equal(d["per_part"].cpu().numpy(), ref["per_part"])
    c = d["counts"].cpu().numpy().tolist()
    assert c == [ref["set_size"], ref["intra_viol"], ref["boundary_viol"]]
    assert int(ref["per_part"].sum()) == 2 * ref["boundary_viol"]
    return ref


def check_stage3(graph, book, p, policy_seed=None):
    """Bit-exact parity of conflict list, base action and actions -> (penalty list, active
    subgraphs, number of chosen nodes), for the base action and for a seeded 0/1 policy."""
    import torch
    ref_dec = oracle.decode(book, p)
    pd = to_dev(p)
    d = graph.decode_boundary(pd)
    ca = graph.conflict_actions(d["viol"], pd)
    torch.cuda.synchronize()
    conf = oracle.conflict_list(book, ref_dec["viol"])
    act = oracle.base_action(book, conf, p)
    C = int(ca["count"].item())
    assert C == conf.size == ref_dec["boundary_viol"]
    assert np.array_equal(ca["conflict_idx"].cpu().numpy()[:C], conf)
    assert np.array_equal(ca["action"].cpu().numpy()[:C], act)
    # list only (no probabilities)
    only = graph.conflict_actions(d["viol"], None, want_action=False)
    assert int(only["count"].item()) == C and only["action"] is None
    assert np.array_equal(only["conflict_idx"].cpu().numpy()[:C], conf)
    # the base action, then an arbitrary caller policy
    policies = [act]
    if policy_seed is not None and C:
        policies.append((si.u64(policy_seed, 0, C) & np.uint64(1)).astype(np.uint8))
    outs = []
    for a in policies:
        a_dev = ca["action"].clone()
        a_dev[:C] = to_dev(a)
        ap = graph.apply_actions(ca["conflict_idx"], a_dev, ca["count"])
        torch.cuda.synchronize()
        ref = oracle.apply_actions(book, conf, a)
        assert np.array_equal(ap["pen"].cpu().numpy(), ref["pen"])
        assert np.array_equal(ap["active"].cpu().numpy(), ref["active"])
        assert int(ap["chosen"].item()) == ref["chosen"]
        # the non-learned repair: clear the chosen nodes from the mask, then no boundary conflict is left
        xr = d["x"].clone()
        removed = graph.repair_boundary(ap["pen"], xr)
        fix = oracle.repair(ref_dec["x"], ref["pen"])
        assert np.array_equal(xr.cpu().numpy(), fix["x"]) and int(removed.item()) == fix["removed"] == ref["chosen"]
        again = graph.decode_boundary(xr.float())
        counts = again["counts"].cpu().tolist()
        assert counts[2] == 0 and counts[0] == ref_dec["set_size"] - fix["removed"]
        outs.append(ap)
    return conf, act, outs[0]


def sampled_step_check(graph, book, dims, dtype, Xd, Wd, parts, x_rows, w_part, alpha=2.0, beta=1.0, lam=0.0,
                       pen_d=None, pen_rows=None, opt=None, want_dx=True, label="", report=None):
    """Full-size parity on sampled subgraphs.  The GPU runs one step on the whole batch
    (device tensors Xd, Wd, optional gnnco.Adam ``opt``); for every subgraph in ``parts``
    the oracle runs that subgraph alone and is compared on loss, p, z, dW, dX and the Adam
    rule.  ``x_rows(lo, hi)`` / ``w_part(l, s)`` / ``pen_rows(lo, hi)`` give the oracle its
    inputs as float32 numpy arrays (for step 0 they come straight from the generators)."""
    import torch
    import paper_2511_09261_b200 as gnnco
    bf16 = dtype == "bf16"
    L = len(dims) - 1
    S = int(book["S"])
    sets = int(Wd[0].shape[0])
    model = gnnco.Model(dims, Wd, gnnco.BF16 if bf16 else gnnco.F32)
    dW = [torch.zeros_like(w) for w in Wd]
    z = torch.empty(int(book["n"]), device=Xd.device)
    dX = torch.empty_like(Xd) if want_dx else None
    before = {}
    if opt is not None:
        for s in parts:
            k = s if sets > 1 else 0
            before[s] = [(Wd[l][k].cpu().numpy().copy(), opt.m[l][k].cpu().numpy().copy(),
                          opt.v[l][k].cpu().numpy().copy()) for l in range(L)]
        step_no, lr = opt.step, opt.lr
    loss, p = graph.train_step(model, Xd, alpha, beta, lam, pen_d, opt, z=z, dW=dW, dX=dX,
                               flags=gnnco.WANT_DX if want_dx else 0)
    torch.cuda.synchronize()
    assert graph.async_status() == 0
    stats = {}
    # the oracle runs the sampled subgraphs one by one, several at a time on host threads (the C
    # call releases the interpreter lock; nothing inside a subgraph's arithmetic changes)
    import os
    from concurrent.futures import ThreadPoolExecutor

    def oracle_part(s):
        lo, hi = int(book["part_ptr"][s]), int(book["part_ptr"][s + 1])
        if hi == lo:
            return None
        Xs = x_rows(lo, hi)
        ws = [w_part(l, s) for l in range(L)]
        wc = [si.round_to_bf16(w) if bf16 else w for w in ws]
        rp = book["rowptr"][lo:hi + 1] - book["rowptr"][lo]
        ci = book["colidx"][book["rowptr"][lo]:book["rowptr"][hi]] - lo
        one = oracle.subgraph_step(rp, ci, dims, Xs, wc, alpha, beta, lam, None if pen_rows is None else pen_rows(lo, hi),
                                   want_dX=want_dx, want_Z=True, store_bf16=bf16)
        return Xs, one

    with ThreadPoolExecutor(max_workers=min(16, len(os.sched_getaffinity(0)))) as pool:
        oracle_out = dict(zip(parts, pool.map(oracle_part, parts)))
    for s in parts:
        lo, hi = int(book["part_ptr"][s]), int(book["part_ptr"][s + 1])
        if oracle_out[s] is None:
            continue
        k = s if sets > 1 else 0
        Xs, one = oracle_out[s]
        got_x = Xd[lo:hi].float().cpu().numpy()
        assert np.array_equal(got_x, Xs), "device X rows differ from the generator's"
        r = dict(loss=np.array([one["loss"]]), p=one["p"], z=one["z"], dX=one["dX"], dW=[d[None] for d in one["dW"]],
                 Z=one["Z"])
        g = dict(loss=loss[s:s + 1].cpu().numpy(), p=p[lo:hi].cpu().numpy(), z=z[lo:hi].cpu().numpy(),
                 dW=[dW[l][k:k + 1].cpu().numpy() for l in range(L)],
                 dX=None if dX is None else dX[lo:hi].float().cpu().numpy())
        tag = "%s part %d" % (label, s)
        stats["loss"] = max(stats.get("loss", 0), assert_close(g["loss"], r["loss"], dtype, tag + " loss", report=report, name="loss"))
        stats["p"] = max(stats.get("p", 0), assert_close(g["p"], r["p"], dtype, tag + " p", report=report, name="p"))
        stats["z"] = max(stats.get("z", 0), assert_close(g["z"], r["z"], dtype, tag + " z", report=report, name="z"))
        kinks = [set(np.nonzero((np.abs(Z) < 1e-6 * (1.0 + np.abs(Z))).any(axis=0))[0].tolist()) for Z in (r["Z"] or [])]
        kinks += [set()] * (L - len(kinks))
        near = any(kinks)
        stats["kink_units"] = stats.get("kink_units", 0) + sum(len(x) for x in kinks)
        if sets == 1:
            continue
        for l in range(L):
            skip = np.zeros(r["dW"][l].shape, bool)
            for l2 in range(l, L):
                if kinks[l2]:
                    if l2 == l:
                        skip[0][:, sorted(kinks[l2])] = True
                    else:
                        skip[:] = True
            stats["dW%d" % l] = max(stats.get("dW%d" % l, 0),
                                    assert_close(g["dW"][l], r["dW"][l], dtype, tag + " dW[%d]" % l, skip, (1, 2), report, "dW%d" % l))
        if want_dx and not near:
            stats["dX"] = max(stats.get("dX", 0), assert_close(g["dX"], r["dX"], dtype, tag + " dX", None, (1,), report, "dX"))
        if opt is not None:
            hyper = _adam_hyper(dict(lr=lr, step=step_no))
            for l in range(L):
                W0, m0, v0 = (a.astype(np.float64) for a in before[s][l])
                oracle.adam(W0, m0, v0, g["dW"][l][0].astype(np.float64), *hyper)
                for key, ref, got in (("m", m0, opt.m[l][k]), ("v", v0, opt.v[l][k]), ("W", W0, Wd[l][k])):
                    np.testing.assert_allclose(got.cpu().numpy(), ref, rtol=2e-6,
                                               atol=5e-7 * float(np.abs(ref).max()) + 1e-30, err_msg=tag + " adam " + key)
    return stats, loss, p


def pick_parts(book, count, seed):
    """Seeded sample of ``count`` subgraphs plus the first, the last, the one with the most intra
    edges and the one that holds the longest row."""
    S = int(book["S"])
    pp = book["part_ptr"].astype(np.int64)
    nnz = book["rowptr"][pp[1:]].astype(np.int64) - book["rowptr"][pp[:-1]].astype(np.int64)
    deg = np.diff(book["rowptr"])
    picks = {0, S - 1, int(np.argmax(nnz)), int(book["node_part"][int(np.argmax(deg))])}
    want = min(S, len(picks) + count)
    for r in si.u64(seed, 0, 8 * count + 64).tolist():
        if len(picks) >= want:
            break
        picks.add(int(r % S))
    return sorted(picks)
