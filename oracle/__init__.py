"""ctypes front end of the CPU oracle (``gnnco_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares nothing with the CUDA library: it loads its own shared object,
built by gcc from the C file beside it, and works on numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gnnco_oracle.c")
_LIB = os.path.join(_HERE, "libgnnco_oracle.so")
_lib = None

OK, BAD_ARG, OUT_OF_RANGE, NOT_SIMPLE = 0, -1, -2, -3


def build(force: bool = False) -> str:
    """Compile the oracle next to its source (gcc -O2, no fast-math, OpenMP for the
    outer loop over subgraphs)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _native():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32, dbl, vp, flt = ctypes.c_int64, ctypes.c_int32, ctypes.c_double, ctypes.c_void_p, ctypes.c_float
        lib.oracle_bookkeeping.argtypes = [i64, i64, vp, vp, vp, i32] + [vp] * 12
        lib.oracle_bookkeeping.restype = ctypes.c_int
        lib.oracle_subgraph_step.argtypes = [i32, vp, vp, i32, vp, vp, vp, dbl, dbl, dbl, vp, vp, vp, vp, vp, vp, vp, i32]
        lib.oracle_subgraph_step.restype = ctypes.c_int
        lib.oracle_train_step.argtypes = [i64, i32, vp, vp, vp, i32, vp, i32, vp, vp, dbl, dbl, dbl,
                                          vp, vp, vp, vp, vp, vp, vp, i32, i32]
        lib.oracle_train_step.restype = ctypes.c_int
        lib.oracle_adam.argtypes = [i64, vp, vp, vp, vp, dbl, dbl, dbl, dbl, i64]
        lib.oracle_adam.restype = None
        lib.oracle_decode.argtypes = [i64, i32, vp, vp, vp, i64, vp, vp, vp, flt, vp, vp, vp, vp]
        lib.oracle_decode.restype = None
        lib.oracle_conflict_list.argtypes = [i64, vp, vp]
        lib.oracle_conflict_list.restype = i64
        lib.oracle_base_action.argtypes = [i64, vp, vp, vp, vp, vp]
        lib.oracle_base_action.restype = None
        lib.oracle_apply_actions.argtypes = [i64, i32, i64, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_apply_actions.restype = i64
        lib.oracle_partition_quality.argtypes = [i64, vp, vp, vp, i32, vp, vp]
        lib.oracle_partition_quality.restype = dbl
        lib.oracle_repair.argtypes = [i64, vp, vp]
        lib.oracle_repair.restype = i64
        lib.oracle_round_bf16.argtypes = [dbl]
        lib.oracle_round_bf16.restype = dbl
        lib.oracle_louvain.argtypes = [i64, i64, vp, vp, i32, i32, vp, vp, vp, vp, vp]
        lib.oracle_louvain.restype = i64
        lib.oracle_louvain_sweep.argtypes = [i64, i64, vp, vp, vp, vp]
        lib.oracle_louvain_sweep.restype = i64
        _lib = lib
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s failed with status %d" % (what, code))
        self.code = code


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


def _ptr_array(arrs: Sequence[Optional[np.ndarray]]):
    t = (ctypes.c_void_p * max(1, len(arrs)))()
    for k, a in enumerate(arrs):
        t[k] = None if a is None else a.ctypes.data
    return t


def bookkeeping(n: int, eu: np.ndarray, ev: np.ndarray, part: np.ndarray, S: int) -> Dict[str, np.ndarray]:
    """Renumber nodes by (part, id), split edges into intra (CSR) and boundary (list)."""
    eu = np.ascontiguousarray(eu, dtype=np.int32)
    ev = np.ascontiguousarray(ev, dtype=np.int32)
    part = np.ascontiguousarray(part, dtype=np.int32)
    E = int(eu.size)
    out = dict(
        perm=np.empty(n, np.int32), inv_perm=np.empty(n, np.int32), part_ptr=np.empty(S + 1, np.int32),
        node_part=np.empty(n, np.int32), rowptr=np.empty(n + 1, np.int32), colidx=np.empty(max(1, 2 * E), np.int32),
        bnd_u=np.empty(max(1, E), np.int32), bnd_v=np.empty(max(1, E), np.int32), inv_deg=np.empty(n, np.float32),
        is_boundary=np.empty(n, np.uint8),
    )
    e_in, e_b = ctypes.c_int64(0), ctypes.c_int64(0)
    rc = _native().oracle_bookkeeping(
        n, E, _ptr(eu), _ptr(ev), _ptr(part), S, _ptr(out["perm"]), _ptr(out["inv_perm"]), _ptr(out["part_ptr"]),
        _ptr(out["node_part"]), _ptr(out["rowptr"]), _ptr(out["colidx"]), _ptr(out["bnd_u"]), _ptr(out["bnd_v"]),
        _ptr(out["inv_deg"]), _ptr(out["is_boundary"]), ctypes.addressof(e_in), ctypes.addressof(e_b))
    if rc != 0:
        raise OracleError(rc, "oracle_bookkeeping")
    out["E_in"], out["E_b"] = int(e_in.value), int(e_b.value)
    out["colidx"] = out["colidx"][: 2 * out["E_in"]].copy()
    out["bnd_u"] = out["bnd_u"][: out["E_b"]].copy()
    out["bnd_v"] = out["bnd_v"][: out["E_b"]].copy()
    out["n"], out["S"] = n, S
    return out


def _as_f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def subgraph_step(rowptr, colidx, dims: Sequence[int], X, W: Sequence[np.ndarray], alpha: float, beta: float,
                  lam: float = 0.0, pen=None, want_dW: bool = True, want_dX: bool = False,
                  want_Z: bool = False, store_bf16: bool = False) -> Dict[str, object]:
    """One standalone subgraph with local ids: forward, loss and exact gradients.
    ``store_bf16`` rounds the stored hidden tensors (M_l, H_l) to bfloat16."""
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    colidx = np.ascontiguousarray(colidx, dtype=np.int32)
    ns, L = rowptr.size - 1, len(dims) - 1
    dims_a = np.asarray(dims, dtype=np.int32)
    X = _as_f64(X)
    Wd = [_as_f64(w) for w in W]
    pen = _as_f64(pen)
    loss = np.zeros(1)
    z, p = np.empty(ns), np.empty(ns)
    dW = [np.zeros((dims[l], dims[l + 1])) for l in range(L)] if want_dW else None
    dX = np.zeros((ns, dims[0])) if want_dX else None
    Z = [np.zeros((ns, dims[l + 1])) for l in range(L - 1)] if want_Z else None
    rc = _native().oracle_subgraph_step(
        ns, _ptr(rowptr), _ptr(colidx), L, _ptr(dims_a), _ptr(X), _ptr_array(Wd), alpha, beta, lam, _ptr(pen),
        _ptr(loss), _ptr(z), _ptr(p), _ptr_array(dW) if dW is not None else None, _ptr(dX),
        _ptr_array(Z + [None]) if Z is not None else None, int(store_bf16))
    if rc != 0:
        raise OracleError(rc, "oracle_subgraph_step")
    return dict(loss=float(loss[0]), z=z, p=p, dW=dW, dX=dX, Z=Z)


def train_step(book: Dict[str, np.ndarray], dims: Sequence[int], X, W: Sequence[np.ndarray], alpha: float, beta: float,
               lam: float = 0.0, pen=None, want_dW: bool = True, want_dX: bool = False, want_Z: bool = False,
               threads: int = 1, store_bf16: bool = False) -> Dict[str, object]:
    """Block-diagonal batch over all subgraphs of ``book`` (the dict returned by
    ``bookkeeping``).  ``X`` is [n, F_0] in the NEW node order; ``W[l]`` is
    [S, F_l, F_{l+1}] (one set per subgraph) or [1, F_l, F_{l+1}] (shared)."""
    n, S = int(book["n"]), int(book["S"])
    L = len(dims) - 1
    dims_a = np.asarray(dims, dtype=np.int32)
    X = _as_f64(X)
    assert X.shape == (n, dims[0])
    Wd = [_as_f64(w) for w in W]
    sets = Wd[0].shape[0]
    for l in range(L):
        assert Wd[l].shape == (sets, dims[l], dims[l + 1]), (Wd[l].shape, l)
    pen = _as_f64(pen)
    loss, z, p = np.zeros(S), np.empty(n), np.empty(n)
    dW = [np.zeros_like(w) for w in Wd] if want_dW else None
    dX = np.zeros((n, dims[0])) if want_dX else None
    Z = [np.zeros((n, dims[l + 1])) for l in range(L - 1)] if want_Z else None
    rc = _native().oracle_train_step(
        n, S, _ptr(book["part_ptr"]), _ptr(book["rowptr"]), _ptr(book["colidx"]), L, _ptr(dims_a), sets, _ptr(X),
        _ptr_array(Wd), alpha, beta, lam, _ptr(pen), _ptr(loss), _ptr(z), _ptr(p),
        _ptr_array(dW) if dW is not None else None, _ptr(dX), _ptr_array(Z + [None]) if Z is not None else None,
        threads, int(store_bf16))
    if rc <= 0:
        raise OracleError(rc, "oracle_train_step")
    return dict(loss=loss, z=z, p=p, dW=dW, dX=dX, Z=Z, threads=rc)


def round_bf16(x: float) -> float:
    """The rounding that the bfloat16-storage mode applies to a stored value: double ->
    nearest float -> nearest bfloat16 (ties to even both times), as a Python float."""
    return float(_native().oracle_round_bf16(float(x)))


def adam(W: np.ndarray, m: np.ndarray, v: np.ndarray, g: np.ndarray, lr: float, t: int, b1: float = 0.9,
         b2: float = 0.999, eps: float = 1e-8) -> None:
    """In-place bias-corrected Adam on float64 arrays; ``t`` is the 1-based step."""
    for a in (W, m, v):
        assert a.dtype == np.float64 and a.flags.c_contiguous
    g = _as_f64(g)
    _native().oracle_adam(W.size, _ptr(W), _ptr(m), _ptr(v), _ptr(g), lr, b1, b2, eps, t)


def partition_quality(eu: np.ndarray, ev: np.ndarray, part: np.ndarray, S: int) -> Dict[str, object]:
    """Per-community internal edge counts and degree sums (the Sigma of Eq. 1) and the
    modularity Q of the partition, from the original edge list."""
    eu = np.ascontiguousarray(eu, dtype=np.int32)
    ev = np.ascontiguousarray(ev, dtype=np.int32)
    part = np.ascontiguousarray(part, dtype=np.int32)
    in_edges, tot = np.empty(S, np.int64), np.empty(S, np.int64)
    q = _native().oracle_partition_quality(eu.size, _ptr(eu), _ptr(ev), _ptr(part), S, _ptr(in_edges), _ptr(tot))
    return dict(in_edges=in_edges, tot=tot, Q=float(q))


def louvain(n: int, eu: np.ndarray, ev: np.ndarray, max_levels: int = 32, max_sweeps: int = 64) -> Dict[str, object]:
    """Deterministic Louvain partition (Section 3.1; synchronous sweeps, exact integer gains --
    see the C source).  Returns part [n] int32, S, the exact modularity numerator ``qnum`` and
    ``two_m`` (Q = qnum / two_m**2), the levels that moved something and the accepted sweeps."""
    eu = np.ascontiguousarray(eu, dtype=np.int32)
    ev = np.ascontiguousarray(ev, dtype=np.int32)
    part = np.empty(n, np.int32)
    qnum, two_m = ctypes.c_int64(0), ctypes.c_int64(0)
    levels, sweeps = ctypes.c_int32(0), ctypes.c_int32(0)
    S = _native().oracle_louvain(n, eu.size, _ptr(eu), _ptr(ev), max_levels, max_sweeps, _ptr(part),
                                 ctypes.addressof(qnum), ctypes.addressof(two_m), ctypes.addressof(levels),
                                 ctypes.addressof(sweeps))
    if S < 0:
        raise OracleError(int(S), "oracle_louvain")
    q = qnum.value / float(two_m.value) ** 2 if two_m.value else 0.0
    return dict(part=part, S=int(S), qnum=int(qnum.value), two_m=int(two_m.value), Q=q, levels=int(levels.value),
                sweeps=int(sweeps.value))


def louvain_sweep(n: int, eu: np.ndarray, ev: np.ndarray, comm: np.ndarray) -> Dict[str, object]:
    """One frozen-state sweep on the input graph from the community vector ``comm``: every node's
    next community and the number of nodes that move."""
    eu = np.ascontiguousarray(eu, dtype=np.int32)
    ev = np.ascontiguousarray(ev, dtype=np.int32)
    comm = np.ascontiguousarray(comm, dtype=np.int32)
    nxt = np.empty(n, np.int32)
    moves = _native().oracle_louvain_sweep(n, eu.size, _ptr(eu), _ptr(ev), _ptr(comm), _ptr(nxt))
    if moves < 0:
        raise OracleError(int(moves), "oracle_louvain_sweep")
    return dict(next=nxt, moves=int(moves))


def delta_q(k_i_in: float, sigma_tot: float, k_i: float, m: float) -> float:
    """Gain in modularity when an isolated node i joins a community (Section 3.1, the
    simplified form, Eq. 2):  k_i_in / m - sigma_tot * k_i / (2 m^2).  Eq. 1 as printed differs
    from it by a factor of two in its first term unless k_i_in and Sigma_in count every edge
    from both ends; Eq. 2 is the one that equals the exact difference of Q."""
    return k_i_in / m - sigma_tot * k_i / (2.0 * m * m)


def repair(x: np.ndarray, pen: np.ndarray) -> Dict[str, object]:
    """Carry the chosen actions out on the mask: a copy of ``x`` with every chosen node
    (``pen`` != 0) cleared, and the number of selected nodes that were removed."""
    out = np.ascontiguousarray(x, dtype=np.uint8).copy()
    pen = np.ascontiguousarray(pen, dtype=np.float32)
    removed = _native().oracle_repair(out.size, _ptr(pen), _ptr(out))
    return dict(x=out, removed=int(removed))


def gumbel_softmax(E: np.ndarray, U: Optional[np.ndarray], tau: float) -> np.ndarray:
    """Gumbel-softmax processing of the initial embeddings (Section 3.2, first paragraph of
    "Subgraph training"): row i of the result is softmax((e_i + g_i) / tau) over the feature
    axis, with Gumbel noise g = -log(-log u) from uniforms u in (0, 1) that the caller passes
    in (``U`` None: no noise).  Reading of the paper where it is silent: the soft (relaxed)
    form, one temperature ``tau`` for all nodes, noise drawn once with the embeddings.
    Plain float64 numpy; the row maximum is subtracted before exponentiating, which changes
    nothing in exact arithmetic."""
    a = np.asarray(E, dtype=np.float64)
    if U is not None:
        a = a + (-np.log(-np.log(np.asarray(U, dtype=np.float64))))
    a = a / float(tau)
    a = a - a.max(axis=1, keepdims=True)
    e = np.exp(a)
    return e / e.sum(axis=1, keepdims=True)


def decode(book: Dict[str, np.ndarray], p: np.ndarray, threshold: float = 0.5) -> Dict[str, object]:
    """Threshold float32 probabilities and count selected nodes and violated edges."""
    n, S = int(book["n"]), int(book["S"])
    p = np.ascontiguousarray(p, dtype=np.float32)
    assert p.shape == (n,)
    x = np.empty(n, np.uint8)
    viol = np.empty(max(1, book["E_b"]), np.uint8)
    per_part = np.empty(S, np.int32)
    counts = np.zeros(3, np.int64)
    _native().oracle_decode(n, S, _ptr(book["node_part"]), _ptr(book["rowptr"]), _ptr(book["colidx"]), book["E_b"],
                            _ptr(book["bnd_u"]), _ptr(book["bnd_v"]), _ptr(p), threshold, _ptr(x), _ptr(viol),
                            _ptr(per_part), _ptr(counts))
    return dict(x=x, viol=viol[: book["E_b"]], per_part=per_part, set_size=int(counts[0]), intra_viol=int(counts[1]),
                boundary_viol=int(counts[2]))


def conflict_list(book: Dict[str, np.ndarray], viol: np.ndarray) -> np.ndarray:
    """Ascending indices (into the boundary list) of the violated boundary edges."""
    viol = np.ascontiguousarray(viol, dtype=np.uint8)
    idx = np.empty(max(1, viol.size), np.int32)
    c = _native().oracle_conflict_list(viol.size, _ptr(viol), _ptr(idx))
    return idx[:c].copy()


def base_action(book: Dict[str, np.ndarray], conflicts: np.ndarray, p: np.ndarray) -> np.ndarray:
    """0/1 per conflict: which endpoint (u or v of the stored pair) to push below the threshold."""
    conflicts = np.ascontiguousarray(conflicts, dtype=np.int32)
    p = np.ascontiguousarray(p, dtype=np.float32)
    act = np.empty(max(1, conflicts.size), np.uint8)
    _native().oracle_base_action(conflicts.size, _ptr(conflicts), _ptr(book["bnd_u"]), _ptr(book["bnd_v"]), _ptr(p),
                                 _ptr(act))
    return act[:conflicts.size].copy()


def apply_actions(book: Dict[str, np.ndarray], conflicts: np.ndarray, action: np.ndarray) -> Dict[str, object]:
    """Penalty node list (0/1 float per node), active-subgraph mask and number of chosen nodes."""
    n, S = int(book["n"]), int(book["S"])
    conflicts = np.ascontiguousarray(conflicts, dtype=np.int32)
    action = np.ascontiguousarray(action, dtype=np.uint8)
    pen, active = np.empty(n, np.float32), np.empty(S, np.uint8)
    chosen = _native().oracle_apply_actions(n, S, conflicts.size, _ptr(conflicts), _ptr(action), _ptr(book["bnd_u"]),
                                            _ptr(book["bnd_v"]), _ptr(book["node_part"]), _ptr(pen), _ptr(active))
    return dict(pen=pen, active=active, chosen=int(chosen))
