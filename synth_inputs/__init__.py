"""Seeded synthetic inputs: graphs, partitions, embeddings and initial weights.

Everything here is *data generation*.  None of the method's arithmetic (aggregation,
transform, objective, decoding, intra/boundary bookkeeping) is implemented in this
module, so it can feed both the CUDA library and the CPU oracle without coupling them.

All randomness is drawn from SplitMix64 streams (see ``_native.c``), addressed by
``(seed, index)``, so any slice of a tensor can be regenerated on its own.

The graphs are stand-ins for the paper's workloads (Section 4, Tables 1-2): they take
the node/edge counts and the degree shape of those datasets, not their contents.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "_native.c")
_LIB = os.path.join(_HERE, "libsynth_inputs.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the native helper next to this file (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _native():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64, i64, i32, f32 = ctypes.c_uint64, ctypes.c_int64, ctypes.c_int32, ctypes.c_float
        vp = ctypes.c_void_p
        lib.synth_u64.argtypes = [u64, u64, i64, vp]
        lib.synth_fill_normal_f32.argtypes = [u64, u64, i64, vp]
        lib.synth_fill_normal_bf16.argtypes = [u64, u64, i64, vp]
        lib.synth_fill_uniform_f32.argtypes = [u64, u64, i64, f32, f32, vp]
        lib.synth_bfs_partition.argtypes = [i64, i64, vp, vp, i32, vp]
        lib.synth_bfs_partition.restype = ctypes.c_int
        for f in (lib.synth_u64, lib.synth_fill_normal_f32, lib.synth_fill_normal_bf16, lib.synth_fill_uniform_f32):
            f.restype = None
        _lib = lib
    return _lib


# ----------------------------------------------------------------------------- streams
def _stream(seed: int, tag: int) -> int:
    """Derive an independent stream id from a workload seed and a purpose tag."""
    return (seed * 0x1000003 + tag * 0x10001 + 0x5EED) & 0xFFFFFFFFFFFFFFFF


def u64(stream: int, start: int, count: int) -> np.ndarray:
    out = np.empty(count, dtype=np.uint64)
    _native().synth_u64(stream, start, count, out.ctypes.data)
    return out


def uniform01(stream: int, start: int, count: int) -> np.ndarray:
    """Doubles in [0, 1) with 53 random bits."""
    return (u64(stream, start, count) >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def normal_f32(stream: int, start: int, count: int) -> np.ndarray:
    out = np.empty(count, dtype=np.float32)
    _native().synth_fill_normal_f32(stream, start, count, out.ctypes.data)
    return out


def normal_bf16_bits(stream: int, start: int, count: int, out: Optional[np.ndarray] = None) -> np.ndarray:
    """N(0,1) rounded to bfloat16; returns the raw uint16 patterns."""
    if out is None:
        out = np.empty(count, dtype=np.uint16)
    assert out.dtype == np.uint16 and out.size == count and out.flags.c_contiguous
    _native().synth_fill_normal_bf16(stream, start, count, out.ctypes.data)
    return out


def uniform_f32(stream: int, start: int, count: int, lo: float, hi: float) -> np.ndarray:
    out = np.empty(count, dtype=np.float32)
    _native().synth_fill_uniform_f32(stream, start, count, lo, hi, out.ctypes.data)
    return out


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest-even bfloat16 and return them as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32).reshape(x.shape)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    return (round_to_bf16(x).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


# ------------------------------------------------------------------------------ graphs
def _unique_sorted(keys: np.ndarray) -> np.ndarray:
    """Sorted distinct values (np.sort + neighbour compare; much faster than np.unique
    on tens of millions of int64 keys)."""
    if keys.size == 0:
        return keys
    s = np.sort(keys)
    keep = np.empty(s.size, dtype=bool)
    keep[0] = True
    np.not_equal(s[1:], s[:-1], out=keep[1:])
    return s[keep]


def _random_perm(stream: int, start: int, m: int) -> np.ndarray:
    """Random permutation of range(m): sort (random high bits | index) and read the
    index back from the low bits (ties cannot occur, the index makes keys distinct)."""
    bits = max(1, int(m - 1).bit_length())
    key = (u64(stream, start, m) >> np.uint64(bits) << np.uint64(bits)) | np.arange(m, dtype=np.uint64)
    key.sort()
    return (key & np.uint64((1 << bits) - 1)).astype(np.int64)


def _finish_edges(keys: np.ndarray, n: int, stream: int) -> Tuple[np.ndarray, np.ndarray]:
    """Unique (lo*n+hi) keys -> edge arrays in shuffled order with random orientation."""
    m = keys.size
    keys = keys[_random_perm(stream, 1 << 40, m)]
    lo = (keys // n).astype(np.int32)
    hi = (keys % n).astype(np.int32)
    flip = (u64(stream, 1 << 41, m) & np.uint64(1)).astype(bool)
    eu = np.where(flip, hi, lo).astype(np.int32)
    ev = np.where(flip, lo, hi).astype(np.int32)
    return eu, ev


def erdos_renyi(n: int, p: float, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """G(n, p): pair number k (row-major over i<j) is kept when its draw is below p."""
    stream = _stream(seed, 1)
    iu, ju = np.triu_indices(n, k=1)
    keep = uniform01(stream, 0, iu.size) < p
    keys = iu[keep].astype(np.int64) * n + ju[keep].astype(np.int64)
    return _finish_edges(keys, n, stream)


def random_regular(n: int, d: int, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """Configuration model: d stubs per node, random stub permutation, consecutive stubs
    paired; self loops and repeated edges dropped (a few nodes end below degree d)."""
    stream = _stream(seed, 2)
    stubs = np.repeat(np.arange(n, dtype=np.int64), d)
    if stubs.size % 2:
        stubs = stubs[:-1]
    s = stubs[_random_perm(stream, 0, stubs.size)]
    a, b = s[0::2], s[1::2]
    ok = a != b
    lo, hi = np.minimum(a[ok], b[ok]), np.maximum(a[ok], b[ok])
    keys = _unique_sorted(lo * n + hi)
    return _finish_edges(keys, n, stream)


def _chung_lu_i0(n: int, n_edges: int, gamma: float, max_degree: float) -> float:
    """Offset i0 of the weight law w_i ~ (i+i0)^(-1/(gamma-1)) giving node 0 the wanted
    expected degree."""
    a = 1.0 / (gamma - 1.0)
    e = 1.0 - a

    def deg0(i0: float) -> float:
        lo, hi = i0 ** e, (n + i0) ** e
        return 2.0 * n_edges * ((i0 + 1.0) ** e - lo) / (hi - lo)

    lo, hi = 1e-9, float(n)
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if deg0(mid) > max_degree:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def chung_lu(n: int, n_edges: int, gamma: float, max_degree: float, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """Power-law graph: both endpoints of every edge drawn with probability proportional
    to w_i = (i+i0)^(-1/(gamma-1)) (inverse transform of the continuous law, floored);
    self loops and repeats rejected; redrawn until n_edges distinct edges exist."""
    stream = _stream(seed, 3)
    a = 1.0 / (gamma - 1.0)
    e = 1.0 - a
    i0 = _chung_lu_i0(n, n_edges, gamma, max_degree)
    lo_c, hi_c = i0 ** e, (n + i0) ** e
    keys = np.empty(0, dtype=np.int64)
    cursor = 0
    while keys.size < n_edges:
        need = n_edges - keys.size
        m = int(need * 1.08) + 1024
        u = uniform01(stream, cursor, 2 * m)
        cursor += 2 * m
        idx = np.floor((lo_c + u * (hi_c - lo_c)) ** (1.0 / e) - i0).astype(np.int64)
        np.clip(idx, 0, n - 1, out=idx)
        p, q = idx[:m], idx[m:]
        ok = p != q
        k = np.minimum(p[ok], q[ok]) * n + np.maximum(p[ok], q[ok])
        keys = _unique_sorted(np.concatenate([keys, k]))
    if keys.size > n_edges:
        # drop a seeded random subset of the surplus
        keep = np.sort(_random_perm(stream, 1 << 42, keys.size)[:n_edges])
        keys = keys[keep]
    return _finish_edges(keys, n, stream)


def triangle_closure(n: int, eu: np.ndarray, ev: np.ndarray, n_edges: int, seed: int) -> Tuple[np.ndarray, np.ndarray]:
    """Raise clustering: repeatedly take a random existing edge (c, a), a random other
    neighbour b of c, and add the edge a-b if absent, until n_edges edges exist."""
    stream = _stream(seed, 4)
    nbr: List[List[int]] = [[] for _ in range(n)]
    have = set()
    ends: List[Tuple[int, int]] = []
    for a, b in zip(eu.tolist(), ev.tolist()):
        nbr[a].append(b)
        nbr[b].append(a)
        have.add((min(a, b), max(a, b)))
        ends.append((a, b))
    cursor = 0
    chunk = u64(stream, 0, 1 << 16)
    while len(have) < n_edges:
        if cursor + 3 > chunk.size:
            chunk = u64(stream, int(chunk[-1]) & 0xFFFFFFFF, 1 << 16)
            cursor = 0
        r0, r1, r2 = int(chunk[cursor]), int(chunk[cursor + 1]), int(chunk[cursor + 2])
        cursor += 3
        c, a = ends[r0 % len(ends)]
        if r1 & 1:
            c, a = a, c
        b = nbr[c][(r2 >> 8) % len(nbr[c])]
        if a == b:
            continue
        key = (min(a, b), max(a, b))
        if key in have:
            continue
        have.add(key)
        nbr[a].append(b)
        nbr[b].append(a)
        ends.append((a, b))
    keys = np.array(sorted(k[0] * n + k[1] for k in have), dtype=np.int64)
    return _finish_edges(keys, n, _stream(seed, 5))


# -------------------------------------------------------------------------- partitions
def contiguous_partition(n: int, S: int) -> np.ndarray:
    """Blocks of ceil(n/S) consecutive node ids."""
    size = -(-n // S)
    return (np.arange(n, dtype=np.int64) // size).astype(np.int32)


def bfs_partition(n: int, eu: np.ndarray, ev: np.ndarray, S: int) -> np.ndarray:
    """Breadth-first grown balanced parts (see ``synth_bfs_partition``)."""
    eu = np.ascontiguousarray(eu, dtype=np.int32)
    ev = np.ascontiguousarray(ev, dtype=np.int32)
    part = np.empty(n, dtype=np.int32)
    rc = _native().synth_bfs_partition(n, eu.size, eu.ctypes.data, ev.ctypes.data, S, part.ctypes.data)
    if rc != 0:
        raise ValueError("synth_bfs_partition failed (bad edge endpoint or out of memory)")
    return part


# --------------------------------------------------------------------------- workloads
@dataclass
class Workload:
    """One seeded problem instance: graph, partition and model shape."""
    name: str
    n: int
    eu: np.ndarray
    ev: np.ndarray
    part: np.ndarray
    S: int
    dims: List[int]                 # F_0, ..., F_{L-1}, 1
    dtype: str                      # "f32" or "bf16" (feature storage)
    steps: int
    seed: int
    lr: float = 1e-3
    alpha: float = 2.0
    beta: float = 1.0
    lam: float = 1.0
    extra: dict = field(default_factory=dict)

    @property
    def E(self) -> int:
        return int(self.eu.size)

    @property
    def L(self) -> int:
        return len(self.dims) - 1

    # Embeddings, in ORIGINAL node order: row i is the embedding of input node i.
    def features_f32(self, rows: Optional[np.ndarray] = None) -> np.ndarray:
        """Rows of the N(0,1) embedding matrix as float32 (bf16-representable values for
        bf16 workloads).  ``rows`` = original node ids, default all."""
        F = self.dims[0]
        st = _stream(self.seed, 10)
        if rows is None:
            if self.dtype == "bf16":
                return bf16_bits_to_f32(normal_bf16_bits(st, 0, self.n * F)).reshape(self.n, F)
            return normal_f32(st, 0, self.n * F).reshape(self.n, F)
        rows = np.asarray(rows, dtype=np.int64)
        out = np.empty((rows.size, F), dtype=np.float32)
        for k, r in enumerate(rows.tolist()):
            out[k] = normal_f32(st, r * F, F)
        return round_to_bf16(out) if self.dtype == "bf16" else out

    def features_bf16_bits(self, out: Optional[np.ndarray] = None) -> np.ndarray:
        F = self.dims[0]
        bits = normal_bf16_bits(_stream(self.seed, 10), 0, self.n * F, None if out is None else out.reshape(-1))
        return bits.reshape(self.n, F)

    def weights(self, layer: int, parts: Optional[np.ndarray] = None) -> np.ndarray:
        """Glorot-uniform start weights of layer ``layer`` (0-based), one set per part:
        array [len(parts), F_in, F_out], U(-a, a) with a = sqrt(6/(F_in+F_out)).
        Rounded to bf16-representable values for bf16 workloads."""
        fi, fo = self.dims[layer], self.dims[layer + 1]
        a = float(np.sqrt(6.0 / (fi + fo)))
        st = _stream(self.seed, 20 + layer)
        if parts is None:
            w = uniform_f32(st, 0, self.S * fi * fo, -a, a).reshape(self.S, fi, fo)
        else:
            parts = np.asarray(parts, dtype=np.int64)
            w = np.empty((parts.size, fi, fo), dtype=np.float32)
            for k, s in enumerate(parts.tolist()):
                w[k] = uniform_f32(st, s * fi * fo, fi * fo, -a, a).reshape(fi, fo)
        return round_to_bf16(w) if self.dtype == "bf16" else w

    def penalty(self, density: float = 0.05) -> np.ndarray:
        """A 0/1 per-node penalty selection in original node order (Section 3.3's
        fine-tuning node list), each node chosen with probability ``density``."""
        return (uniform01(_stream(self.seed, 30), 0, self.n) < density).astype(np.float32)


def make_workload(index: int, scale: float = 1.0) -> Workload:
    """The five benchmark configurations (index 1..5).  ``scale`` < 1 shrinks the node
    count, edge count and part count of configurations 4 and 5 proportionally, for
    tests that must finish quickly; 1.0 gives the full size."""
    if index == 1:
        n, S = 1000, 8
        eu, ev = erdos_renyi(n, 0.01, seed=0)
        return Workload("C1-er1k", n, eu, ev, contiguous_partition(n, S), S, [64, 32, 1], "f32", 100, 0)
    if index == 2:
        n, S = 100_000, 64
        eu, ev = random_regular(n, 3, seed=2)
        return Workload("C2-reg3-100k", n, eu, ev, bfs_partition(n, eu, ev, S), S, [128, 64, 1], "f32", 500, 2)
    if index == 3:
        n, S = 4039, 16
        eu, ev = chung_lu(n, 60_000, 2.5, 700.0, seed=3)
        eu, ev = triangle_closure(n, eu, ev, 88_000, seed=3)
        return Workload("C3-chunglu-4k", n, eu, ev, bfs_partition(n, eu, ev, S), S, [128, 128, 128, 1], "f32", 100, 3)
    if index == 4:
        n = max(2048, int(1_130_000 * scale))
        S = max(2, int(round(1024 * scale)))
        E = int(3_000_000 * scale)
        eu, ev = chung_lu(n, E, 2.1, min(43_000.0, n / 4), seed=4)
        return Workload("C4-chunglu-1.13M" if scale == 1.0 else "C4-scaled-%g" % scale,
                        n, eu, ev, bfs_partition(n, eu, ev, S), S, [128, 128, 1], "f32", 20, 4)
    if index == 5:
        n = max(4096, int(10_000_000 * scale))
        S = max(2, int(round(4096 * scale)))
        E = 4 * n
        eu, ev = chung_lu(n, E, 2.3, min(50_000.0, n / 4), seed=5)
        return Workload("C5-chunglu-10M" if scale == 1.0 else "C5-scaled-%g" % scale,
                        n, eu, ev, bfs_partition(n, eu, ev, S), S, [256, 256, 256, 1], "bf16", 5, 5)
    raise ValueError("workload index must be 1..5")


def small_regular_workload(n: int, d: int, S: int, dims: List[int], seed: int) -> Workload:
    """d-regular graphs of the paper's small-graph experiment shape (Section 4:
    100..1000 nodes, degree 10..40), contiguous parts."""
    eu, ev = random_regular(n, d, seed)
    return Workload("reg%d-%d" % (d, n), n, eu, ev, contiguous_partition(n, S), S, dims, "f32", 10, seed)
