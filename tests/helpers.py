"""Shared test helpers: tiny graphs and brute-force restatements that use neither the
oracle nor the CUDA library."""
import numpy as np

import synth_inputs as si


def tiny_graph(n, p, S, seed, contiguous=False):
    """Erdos-Renyi graph with a random (or contiguous) partition into S parts."""
    eu, ev = si.erdos_renyi(n, p, seed)
    if contiguous:
        part = si.contiguous_partition(n, S)
    else:
        part = (si.u64(seed * 77 + 5, 0, n) % np.uint64(S)).astype(np.int32)
    return eu, ev, part


def dense_intra_adjacency(n, eu, ev, part):
    """Dense 0/1 adjacency of the intra-partition edges, ORIGINAL node order."""
    A = np.zeros((n, n))
    for a, b in zip(eu.tolist(), ev.tolist()):
        if part[a] == part[b]:
            A[a, b] = 1.0
            A[b, a] = 1.0
    return A


def rand_weights(dims, sets, seed, scale=1.0):
    out = []
    for l in range(len(dims) - 1):
        a = scale * np.sqrt(6.0 / (dims[l] + dims[l + 1]))
        w = si.uniform_f32(seed * 131 + l, 0, sets * dims[l] * dims[l + 1], -a, a)
        out.append(w.reshape(sets, dims[l], dims[l + 1]).astype(np.float64))
    return out


def rand_features(n, F, seed):
    return si.normal_f32(seed * 977 + 3, 0, n * F).reshape(n, F).astype(np.float64)
