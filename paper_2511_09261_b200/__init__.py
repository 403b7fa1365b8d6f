"""Python binding of libgnnco (argument marshalling only).

Every step of the path runs inside the CUDA library; this module turns torch tensors
into raw pointers and calls the C ABI declared in ``include/gnnco.h`` with the same
names.  PyTorch is used for device memory and streams, nothing else.  There is no CPU
fallback: if the shared library is missing or cannot be loaded, importing the binding's
entry points raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

from . import _build

MAX_LAYERS = 8
OK = 0
INVALID_ARGUMENT, OUT_OF_RANGE, NOT_SIMPLE_GRAPH, UNSUPPORTED, WORKSPACE_TOO_SMALL, CUDA_ERROR, INTERNAL = (
    -1, -2, -3, -4, -5, -6, -7)
F32, BF16 = 0, 1
WANT_DX, FORWARD_ONLY, AX_STORE, AX_REUSE, WEIGHTS_UNTOUCHED, ACTIVE_ONLY, ONE_KERNEL_LAYERS = 1, 2, 4, 8, 16, 32, 64

EXPORTS = [
    "gnnco_status_string", "gnnco_partition_workspace_bytes", "gnnco_partition_load", "gnnco_graph_info",
    "gnnco_gather_rows", "gnnco_train_workspace_bytes", "gnnco_train_step", "gnnco_train_host_workspace_bytes",
    "gnnco_train_step_host", "gnnco_decode_boundary", "gnnco_async_status", "gnnco_launch_count", "gnnco_destroy",
    "gnnco_profile_begin", "gnnco_profile_end", "gnnco_objective_static", "gnnco_conflict_workspace_bytes",
    "gnnco_conflict_actions", "gnnco_apply_actions", "gnnco_gumbel_softmax", "gnnco_embedding_update",
    "gnnco_repair_boundary", "gnnco_partition_quality", "gnnco_active_plan_bytes", "gnnco_active_plan",
    "gnnco_louvain_workspace_bytes", "gnnco_louvain",
]

_vp, _i32, _i64, _u32, _f32, _sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32, ctypes.c_float,
                                    ctypes.c_size_t)


class GraphDesc(ctypes.Structure):
    _fields_ = [("n", _i64), ("E", _i64), ("S", _i32), ("edge_u", _vp), ("edge_v", _vp), ("part", _vp)]


class GraphView(ctypes.Structure):
    _fields_ = [("n", _i64), ("S", _i32), ("E_in", _i64), ("E_b", _i64), ("max_row", _i32), ("perm", _vp),
                ("inv_perm", _vp), ("part_ptr", _vp), ("node_part", _vp), ("rowptr", _vp), ("colidx", _vp),
                ("bnd_u", _vp), ("bnd_v", _vp), ("inv_deg", _vp), ("is_boundary", _vp)]


class ModelDesc(ctypes.Structure):
    _fields_ = [("L", _i32), ("dims", _i32 * (MAX_LAYERS + 1)), ("feat_dtype", _i32), ("weight_sets", _i32),
                ("W", _vp * MAX_LAYERS)]


class Objective(ctypes.Structure):
    _fields_ = [("alpha", _f32), ("beta", _f32), ("lam", _f32), ("pen", _vp)]


class AdamState(ctypes.Structure):
    _fields_ = [("lr", _f32), ("beta1", _f32), ("beta2", _f32), ("eps", _f32), ("step", _i64),
                ("m", _vp * MAX_LAYERS), ("v", _vp * MAX_LAYERS), ("active", _vp), ("step_dev", _vp)]


class TrainOut(ctypes.Structure):
    _fields_ = [("loss", _vp), ("p", _vp), ("z", _vp), ("dW", _vp * MAX_LAYERS), ("dX", _vp), ("ax_cache", _vp)]


class ProfileEntry(ctypes.Structure):
    _fields_ = [("name", ctypes.c_char * 32), ("calls", _i64), ("total_ms", ctypes.c_double)]


class GnncoError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__("%s: %s (status %d)" % (what, status_string(status), status))
        self.status = status


_lib = None


def lib_path() -> str:
    return _build.LIB_PATH


def load_library(build_if_missing: bool = True):
    """Load libgnnco.so (building it in-tree first if it is absent or stale and nvcc is
    available).  Raises if the library cannot be produced or loaded."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing and _build.needs_build():
        _build.build()
    if not os.path.exists(_build.LIB_PATH):
        raise RuntimeError("libgnnco.so is missing: build it with paper_2511_09261_b200._build.build()")
    lib = ctypes.CDLL(_build.LIB_PATH)
    lib.gnnco_status_string.argtypes = [_i32]
    lib.gnnco_status_string.restype = ctypes.c_char_p
    lib.gnnco_partition_workspace_bytes.argtypes = [_i64, _i64, _i32, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]
    lib.gnnco_partition_load.argtypes = [ctypes.POINTER(GraphDesc), _vp, _sz, _vp, _sz, _vp, ctypes.POINTER(_vp)]
    lib.gnnco_graph_info.argtypes = [_vp, ctypes.POINTER(GraphView)]
    lib.gnnco_gather_rows.argtypes = [_vp, _vp, _vp, _vp, _i64, _i64, _vp]
    lib.gnnco_train_workspace_bytes.argtypes = [_vp, ctypes.POINTER(ModelDesc), _u32, ctypes.POINTER(_sz)]
    lib.gnnco_train_host_workspace_bytes.argtypes = [_vp, ctypes.POINTER(ModelDesc), _u32, ctypes.POINTER(_sz)]
    lib.gnnco_train_step.argtypes = [_vp, ctypes.POINTER(ModelDesc), _vp, ctypes.POINTER(Objective),
                                     ctypes.POINTER(AdamState), ctypes.POINTER(TrainOut), _u32, _vp, _sz, _vp]
    lib.gnnco_train_step_host.argtypes = [_vp, ctypes.POINTER(ModelDesc), _vp, _f32, _f32, _f32, _vp,
                                          ctypes.POINTER(AdamState), _vp, _vp, _u32, _vp, _sz, _vp]
    lib.gnnco_decode_boundary.argtypes = [_vp, _vp, _f32, _vp, _vp, _vp, _vp, _vp]
    lib.gnnco_async_status.argtypes = [_vp, _vp, ctypes.POINTER(_i32)]
    lib.gnnco_launch_count.argtypes = [_vp]
    lib.gnnco_launch_count.restype = _i64
    lib.gnnco_destroy.argtypes = [_vp]
    lib.gnnco_objective_static.argtypes = [_vp, _vp, ctypes.POINTER(Objective), _vp, _vp]
    lib.gnnco_profile_begin.argtypes = [_vp]
    lib.gnnco_profile_end.argtypes = [_vp, _vp, ctypes.POINTER(ProfileEntry), _i32, ctypes.POINTER(_i32)]
    lib.gnnco_conflict_workspace_bytes.argtypes = [_vp, ctypes.POINTER(_sz)]
    lib.gnnco_conflict_actions.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
    lib.gnnco_apply_actions.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
    lib.gnnco_partition_quality.argtypes = [_vp, _vp, _vp, _vp, _vp]
    lib.gnnco_repair_boundary.argtypes = [_vp, _vp, _vp, _vp, _vp]
    lib.gnnco_louvain_workspace_bytes.argtypes = [_i64, _i64, ctypes.POINTER(_sz)]
    lib.gnnco_louvain.argtypes = [_i64, _i64, _vp, _vp, _i32, _i32, _vp, ctypes.POINTER(_i32), ctypes.POINTER(_i64),
                                  ctypes.POINTER(_i64), ctypes.POINTER(_i32), ctypes.POINTER(_i32), _vp, _sz, _vp]
    lib.gnnco_active_plan_bytes.argtypes = [_vp, ctypes.POINTER(_sz)]
    lib.gnnco_active_plan.argtypes = [_vp, _vp, _vp, _sz, _vp, ctypes.POINTER(_i32)]
    lib.gnnco_gumbel_softmax.argtypes = [_vp, _i32, _i32, _vp, _vp, _f32, _vp, _vp]
    lib.gnnco_embedding_update.argtypes = [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _f32, _f32, _f32, _f32, _i64, _vp]
    for name in EXPORTS:
        if name not in ("gnnco_status_string", "gnnco_launch_count"):
            getattr(lib, name).restype = _i32
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().gnnco_status_string(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != OK:
        raise GnncoError(status, what)


def _stream_ptr(stream=None) -> int:
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _dptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _require(t, dtype, what: str, device_type: str = "cuda"):
    import torch
    if not isinstance(t, torch.Tensor) or t.dtype != dtype or not t.is_contiguous() or t.device.type != device_type:
        raise TypeError("%s must be a contiguous %s tensor of dtype %s" % (what, device_type, dtype))
    return t


class Model:
    """Shape and weights of the GCN (``gnnco_model_desc``).  ``W[l]`` is a float32 CUDA
    tensor [weight_sets, dims[l], dims[l+1]]."""

    def __init__(self, dims: Sequence[int], W: Sequence, feat_dtype: int = F32):
        import torch
        self.dims = [int(d) for d in dims]
        self.L = len(self.dims) - 1
        if self.L < 1 or self.L > MAX_LAYERS or len(W) != self.L:
            raise ValueError("need 1..%d layers and one weight tensor per layer" % MAX_LAYERS)
        self.W = [_require(w, torch.float32, "W[%d]" % l) for l, w in enumerate(W)]
        self.weight_sets = int(self.W[0].shape[0])
        for l, w in enumerate(self.W):
            if tuple(w.shape) != (self.weight_sets, self.dims[l], self.dims[l + 1]):
                raise ValueError("W[%d] has shape %s" % (l, tuple(w.shape)))
        self.feat_dtype = int(feat_dtype)

    def desc(self) -> ModelDesc:
        d = ModelDesc()
        d.L = self.L
        for k, v in enumerate(self.dims):
            d.dims[k] = v
        d.feat_dtype = self.feat_dtype
        d.weight_sets = self.weight_sets
        for l, w in enumerate(self.W):
            d.W[l] = w.data_ptr()
        return d

    @property
    def torch_feat_dtype(self):
        import torch
        return torch.bfloat16 if self.feat_dtype == BF16 else torch.float32


class Adam:
    """Adam moments and hyper-parameters (``gnnco_adam_state``); ``step`` is advanced by
    ``PartitionedGraph.train_step`` after each update."""

    def __init__(self, model: Model, lr: float = 1e-3, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                 device_step: bool = False):
        import torch
        self.lr, self.beta1, self.beta2, self.eps = lr, beta1, beta2, eps
        self.step = 1
        self.active = None          # uint8 [S] device tensor: subgraphs being fine-tuned (None = all)
        # ``gnnco_adam_state.step_dev``: number of updates done so far, kept on the device (steps that use it can be
        # recorded in a CUDA graph and replayed)
        self.step_dev = torch.zeros(1, dtype=torch.int32, device=model.W[0].device) if device_step else None
        self.m = [torch.zeros_like(w) for w in model.W]
        self.v = [torch.zeros_like(w) for w in model.W]

    def desc(self) -> AdamState:
        a = AdamState()
        a.lr, a.beta1, a.beta2, a.eps, a.step = self.lr, self.beta1, self.beta2, self.eps, self.step
        for l in range(len(self.m)):
            a.m[l] = self.m[l].data_ptr()
            a.v[l] = self.v[l].data_ptr()
        a.active = _dptr(self.active)
        a.step_dev = _dptr(self.step_dev)
        return a


class PartitionedGraph:
    """Handle returned by ``gnnco_partition_load`` plus the torch buffers it lives in."""

    def __init__(self, edge_u, edge_v, part, S: int, stream=None):
        import torch
        lib = load_library()
        self._lib = lib
        self._handle = None
        n, E = int(part.numel()), int(edge_u.numel())
        _require(part, torch.int32, "part")
        _require(edge_u, torch.int32, "edge_u")
        _require(edge_v, torch.int32, "edge_v")
        if int(edge_v.numel()) != E:
            raise ValueError("edge_u and edge_v differ in length")
        self.device = part.device
        pb, sb = _sz(0), _sz(0)
        _check(lib.gnnco_partition_workspace_bytes(n, E, S, ctypes.byref(pb), ctypes.byref(sb)),
               "gnnco_partition_workspace_bytes")
        self._persistent = torch.empty(pb.value, dtype=torch.uint8, device=self.device)
        scratch = torch.empty(sb.value, dtype=torch.uint8, device=self.device)
        g = GraphDesc(n, E, S, _dptr(edge_u) if E else None, _dptr(edge_v) if E else None, _dptr(part))
        hp = _vp(0)
        st = lib.gnnco_partition_load(ctypes.byref(g), self._persistent.data_ptr(), pb.value, scratch.data_ptr(),
                                      sb.value, _stream_ptr(stream), ctypes.byref(hp))
        _check(st, "gnnco_partition_load")
        self._handle = hp
        del scratch
        v = GraphView()
        _check(lib.gnnco_graph_info(self._handle, ctypes.byref(v)), "gnnco_graph_info")
        self.n, self.S, self.E_in, self.E_b, self.max_row = int(v.n), int(v.S), int(v.E_in), int(v.E_b), int(v.max_row)
        self._view = v
        self._ws = None
        self._ws_key = None
        self._plan_ws = None
        self._plan_active = None

    # ---- views of the persistent area as torch tensors (no copies)
    def _view_tensor(self, ptr: int, count: int, dtype):
        import torch
        esz = torch.empty(0, dtype=dtype).element_size()
        off = ptr - self._persistent.data_ptr()
        return self._persistent[off: off + count * esz].view(dtype)

    def arrays(self) -> dict:
        import torch
        v = self._view
        return dict(
            perm=self._view_tensor(v.perm, self.n, torch.int32),
            inv_perm=self._view_tensor(v.inv_perm, self.n, torch.int32),
            part_ptr=self._view_tensor(v.part_ptr, self.S + 1, torch.int32),
            node_part=self._view_tensor(v.node_part, self.n, torch.int32),
            rowptr=self._view_tensor(v.rowptr, self.n + 1, torch.int32),
            colidx=self._view_tensor(v.colidx, 2 * self.E_in, torch.int32),
            bnd_u=self._view_tensor(v.bnd_u, self.E_b, torch.int32),
            bnd_v=self._view_tensor(v.bnd_v, self.E_b, torch.int32),
            inv_deg=self._view_tensor(v.inv_deg, self.n, torch.float32),
            is_boundary=self._view_tensor(v.is_boundary, self.n, torch.uint8),
        )

    def gather_rows(self, src, index, out=None, stream=None):
        """out[i] = src[index[i]] (``gnnco_gather_rows``)."""
        import torch
        rows = int(index.numel())
        row_bytes = src[0].numel() * src.element_size() if src.dim() > 1 else src.element_size()
        if out is None:
            out = torch.empty((rows,) + tuple(src.shape[1:]), dtype=src.dtype, device=src.device)
        _check(self._lib.gnnco_gather_rows(self._handle, src.data_ptr(), out.data_ptr(), index.data_ptr(), rows,
                                           row_bytes, _stream_ptr(stream)), "gnnco_gather_rows")
        return out

    def _workspace(self, model: Model, flags: int, host: bool):
        import torch
        key = (tuple(model.dims), model.feat_dtype, model.weight_sets, flags & FORWARD_ONLY, host)
        if self._ws_key != key:
            b = _sz(0)
            md = model.desc()
            fn = self._lib.gnnco_train_host_workspace_bytes if host else self._lib.gnnco_train_workspace_bytes
            _check(fn(self._handle, ctypes.byref(md), flags, ctypes.byref(b)), "gnnco_train_workspace_bytes")
            self._ws = None
            self._ws = torch.empty(max(256, b.value), dtype=torch.uint8, device=self.device)
            self._ws_key = key
        return self._ws

    def train_step(self, model: Model, X, alpha: float, beta: float, lam: float = 0.0, pen=None,
                   opt: Optional[Adam] = None, loss=None, p=None, z=None, dW: Optional[List] = None, dX=None,
                   flags: int = 0, stream=None, ax_cache=None):
        """One ``gnnco_train_step``.  Returns (loss, p).  Optional outputs are written
        into the tensors passed as ``z``, ``dW`` (list, entries may be None) and ``dX``;
        ``ax_cache`` ([n, dims[0]], the features' type) goes with AX_STORE / AX_REUSE."""
        import torch
        _require(X, model.torch_feat_dtype, "X")
        if tuple(X.shape) != (self.n, model.dims[0]):
            raise ValueError("X must be [n, dims[0]]")
        if loss is None:
            loss = torch.empty(self.S, dtype=torch.float32, device=self.device)
        if p is None:
            p = torch.empty(self.n, dtype=torch.float32, device=self.device)
        ws = self._workspace(model, flags, host=False)
        md = model.desc()
        obj = Objective(alpha, beta, lam, _dptr(pen))
        out = TrainOut()
        out.loss, out.p, out.z, out.dX = _dptr(loss), _dptr(p), _dptr(z), _dptr(dX)
        if ax_cache is not None:
            _require(ax_cache, model.torch_feat_dtype, "ax_cache")
            if tuple(ax_cache.shape) != (self.n, model.dims[0]):
                raise ValueError("ax_cache must be [n, dims[0]]")
            out.ax_cache = ax_cache.data_ptr()
        if dW is not None:
            for l, t in enumerate(dW):
                out.dW[l] = _dptr(t)
        ad = opt.desc() if opt is not None else None
        st = self._lib.gnnco_train_step(self._handle, ctypes.byref(md), X.data_ptr(), ctypes.byref(obj),
                                        ctypes.byref(ad) if ad is not None else None, ctypes.byref(out), flags,
                                        ws.data_ptr(), ws.numel(), _stream_ptr(stream))
        _check(st, "gnnco_train_step")
        if opt is not None and not (flags & FORWARD_ONLY):
            opt.step += 1
        return loss, p

    def train_step_host(self, model: Model, X_host, alpha: float, beta: float, lam: float = 0.0, pen_host=None,
                        opt: Optional[Adam] = None, loss_host=None, p_host=None, flags: int = 0, stream=None):
        """``gnnco_train_step_host``: per-step inputs and outputs are HOST tensors (pinned
        recommended); returns (loss_host, p_host) after the stream has been synchronised."""
        import torch
        _require(X_host, model.torch_feat_dtype, "X_host", "cpu")
        if loss_host is None:
            loss_host = torch.empty(self.S, dtype=torch.float32).pin_memory()
        if p_host is None:
            p_host = torch.empty(self.n, dtype=torch.float32).pin_memory()
        ws = self._workspace(model, flags, host=True)
        md = model.desc()
        ad = opt.desc() if opt is not None else None
        st = self._lib.gnnco_train_step_host(self._handle, ctypes.byref(md), X_host.data_ptr(), alpha, beta, lam,
                                             _dptr(pen_host), ctypes.byref(ad) if ad is not None else None,
                                             loss_host.data_ptr(), p_host.data_ptr(), flags, ws.data_ptr(),
                                             ws.numel(), _stream_ptr(stream))
        _check(st, "gnnco_train_step_host")
        if opt is not None and not (flags & FORWARD_ONLY):
            opt.step += 1
        return loss_host, p_host

    def decode_boundary(self, p, threshold: float = 0.5, x=None, viol=None, per_part=None, counts=None,
                        want_viol: bool = True, want_per_part: bool = True, stream=None):
        """``gnnco_decode_boundary``.  Returns dict(x, viol, per_part, counts) of device
        tensors; counts = int64[3] (set size, intra violations, boundary violations)."""
        import torch
        _require(p, torch.float32, "p")
        if x is None:
            x = torch.empty(self.n, dtype=torch.uint8, device=self.device)
        if viol is None and want_viol:
            viol = torch.empty(self.E_b, dtype=torch.uint8, device=self.device)
        if per_part is None and want_per_part:
            per_part = torch.empty(self.S, dtype=torch.int32, device=self.device)
        if counts is None:
            counts = torch.empty(3, dtype=torch.int64, device=self.device)
        st = self._lib.gnnco_decode_boundary(self._handle, p.data_ptr(), threshold, x.data_ptr(), _dptr(viol),
                                             _dptr(per_part), counts.data_ptr(), _stream_ptr(stream))
        _check(st, "gnnco_decode_boundary")
        return dict(x=x, viol=viol, per_part=per_part, counts=counts)

    def active_plan(self, active, stream=None) -> int:
        """``gnnco_active_plan``: work lists of the subgraphs with ``active[s] != 0`` (uint8 [S] device tensor,
        kept alive by the caller while the plan is in use) for steps with ACTIVE_ONLY.  Synchronises the
        stream; returns the number of active subgraphs."""
        import torch
        _require(active, torch.uint8, "active")
        if tuple(active.shape) != (self.S,):
            raise ValueError("active must be [S]")
        need = _sz(0)
        _check(self._lib.gnnco_active_plan_bytes(self._handle, ctypes.byref(need)), "gnnco_active_plan_bytes")
        if self._plan_ws is None or self._plan_ws.numel() < need.value:
            self._plan_ws = torch.empty(max(256, need.value), dtype=torch.uint8, device=self.device)
        count = _i32(0)
        _check(self._lib.gnnco_active_plan(self._handle, active.data_ptr(), self._plan_ws.data_ptr(),
                                           self._plan_ws.numel(), _stream_ptr(stream), ctypes.byref(count)),
               "gnnco_active_plan")
        self._plan_active = active
        return int(count.value)

    def conflict_actions(self, viol, p=None, want_action: bool = True, stream=None):
        """``gnnco_conflict_actions``.  Returns dict(conflict_idx, action, count): int32 [E_b]
        and uint8 [E_b] buffers of which the first ``count`` entries are valid, and the device
        int32 count itself (no host synchronisation)."""
        import torch
        _require(viol, torch.uint8, "viol")
        if want_action:
            _require(p, torch.float32, "p")
        need = _sz(0)
        _check(self._lib.gnnco_conflict_workspace_bytes(self._handle, ctypes.byref(need)),
               "gnnco_conflict_workspace_bytes")
        ws = torch.empty(need.value, dtype=torch.uint8, device=self.device)
        idx = torch.empty(self.E_b, dtype=torch.int32, device=self.device)
        action = torch.empty(self.E_b, dtype=torch.uint8, device=self.device) if want_action else None
        count = torch.empty(1, dtype=torch.int32, device=self.device)
        _check(self._lib.gnnco_conflict_actions(self._handle, viol.data_ptr(), _dptr(p) if want_action else None,
                                                idx.data_ptr(), _dptr(action), count.data_ptr(), ws.data_ptr(),
                                                need.value, _stream_ptr(stream)), "gnnco_conflict_actions")
        return dict(conflict_idx=idx, action=action, count=count)

    def apply_actions(self, conflict_idx, action, count, pen=None, active=None, stream=None):
        """``gnnco_apply_actions``.  Returns dict(pen, active, chosen): float32 [n], uint8 [S]
        and a device int32 with the number of distinct chosen nodes."""
        import torch
        _require(conflict_idx, torch.int32, "conflict_idx")
        _require(action, torch.uint8, "action")
        _require(count, torch.int32, "count")
        if pen is None:
            pen = torch.empty(self.n, dtype=torch.float32, device=self.device)
        if active is None:
            active = torch.empty(self.S, dtype=torch.uint8, device=self.device)
        chosen = torch.empty(1, dtype=torch.int32, device=self.device)
        _check(self._lib.gnnco_apply_actions(self._handle, conflict_idx.data_ptr(), action.data_ptr(),
                                             count.data_ptr(), pen.data_ptr(), active.data_ptr(), chosen.data_ptr(),
                                             _stream_ptr(stream)), "gnnco_apply_actions")
        return dict(pen=pen, active=active, chosen=chosen)

    def partition_quality(self, stream=None):
        """``gnnco_partition_quality``: dict(in_edges int64 [S], tot int64 [S], Q float64 [1]) on the device."""
        import torch
        in_edges = torch.empty(self.S, dtype=torch.int64, device=self.device)
        tot = torch.empty(self.S, dtype=torch.int64, device=self.device)
        Q = torch.empty(1, dtype=torch.float64, device=self.device)
        _check(self._lib.gnnco_partition_quality(self._handle, in_edges.data_ptr(), tot.data_ptr(), Q.data_ptr(),
                                                 _stream_ptr(stream)), "gnnco_partition_quality")
        return dict(in_edges=in_edges, tot=tot, Q=Q)

    def repair_boundary(self, pen, x, stream=None):
        """``gnnco_repair_boundary``: clears, in place, every chosen node (``pen`` != 0) from the
        mask ``x``; returns a device int32 with the number of selected nodes removed."""
        import torch
        _require(pen, torch.float32, "pen")
        _require(x, torch.uint8, "x")
        removed = torch.empty(1, dtype=torch.int32, device=self.device)
        _check(self._lib.gnnco_repair_boundary(self._handle, pen.data_ptr(), x.data_ptr(), removed.data_ptr(),
                                               _stream_ptr(stream)), "gnnco_repair_boundary")
        return removed

    def gumbel_softmax(self, E, U=None, tau: float = 1.0, out=None, stream=None):
        """``gnnco_gumbel_softmax``: rows of ``E`` ([n, F], float32 or bfloat16) through the
        Gumbel-softmax with uniforms ``U`` ([n, F] float32 in (0, 1), or None for no noise)."""
        import torch
        if E.dtype not in (torch.float32, torch.bfloat16) or E.dim() != 2 or E.shape[0] != self.n:
            raise ValueError("E must be [n, F] float32 or bfloat16")
        _require(E, E.dtype, "E")
        if U is not None:
            _require(U, torch.float32, "U")
            if tuple(U.shape) != tuple(E.shape):
                raise ValueError("U must have the shape of E")
        if out is None:
            out = torch.empty_like(E)
        _require(out, E.dtype, "out")
        dt = BF16 if E.dtype == torch.bfloat16 else F32
        _check(self._lib.gnnco_gumbel_softmax(self._handle, dt, int(E.shape[1]), E.data_ptr(), _dptr(U), float(tau),
                                              out.data_ptr(), _stream_ptr(stream)), "gnnco_gumbel_softmax")
        return out

    def embedding_update(self, dX, X_master, m, v, X, lr: float, step: int, beta1: float = 0.9,
                         beta2: float = 0.999, eps: float = 1e-8, stream=None):
        """``gnnco_embedding_update``: one Adam step on the float32 master embeddings with the
        gradient ``dX`` of a WANT_DX training step; ``X`` receives them in the features' type."""
        import torch
        for t, what in ((X_master, "X_master"), (m, "m"), (v, "v")):
            _require(t, torch.float32, what)
        _require(dX, X.dtype, "dX")
        _require(X, X.dtype, "X")
        if X.dtype not in (torch.float32, torch.bfloat16) or X.dim() != 2 or X.shape[0] != self.n:
            raise ValueError("X must be [n, F] float32 or bfloat16")
        for t in (dX, X_master, m, v):
            if tuple(t.shape) != tuple(X.shape):
                raise ValueError("dX, X_master, m, v and X must have the same shape")
        dt = BF16 if X.dtype == torch.bfloat16 else F32
        _check(self._lib.gnnco_embedding_update(self._handle, dt, int(X.shape[1]), dX.data_ptr(), X_master.data_ptr(),
                                                m.data_ptr(), v.data_ptr(), X.data_ptr(), float(lr), float(beta1),
                                                float(beta2), float(eps), int(step), _stream_ptr(stream)),
               "gnnco_embedding_update")
        return X

    def objective_static(self, p, alpha: float, beta: float, lam: float = 0.0, pen=None, loss=None, stream=None):
        """``gnnco_objective_static``: per-subgraph objective of given probabilities, with no
        work area and no allocation inside the library (``loss`` must be passed by callers
        that cannot allocate; it is created here only as a convenience)."""
        import torch
        _require(p, torch.float32, "p")
        if loss is None:
            loss = torch.empty(self.S, dtype=torch.float32, device=self.device)
        obj = Objective(alpha, beta, lam, _dptr(pen))
        _check(self._lib.gnnco_objective_static(self._handle, p.data_ptr(), ctypes.byref(obj), loss.data_ptr(),
                                                _stream_ptr(stream)), "gnnco_objective_static")
        return loss

    def async_status(self, stream=None) -> int:
        s = _i32(0)
        _check(self._lib.gnnco_async_status(self._handle, _stream_ptr(stream), ctypes.byref(s)), "gnnco_async_status")
        return int(s.value)

    def profile_begin(self) -> None:
        _check(self._lib.gnnco_profile_begin(self._handle), "gnnco_profile_begin")

    def profile_end(self, stream=None) -> dict:
        """``gnnco_profile_end``: {kernel family: (calls, total_ms)} since profile_begin."""
        entries = (ProfileEntry * 32)()
        count = _i32(0)
        _check(self._lib.gnnco_profile_end(self._handle, _stream_ptr(stream), entries, 32, ctypes.byref(count)),
               "gnnco_profile_end")
        return {entries[k].name.decode(): (int(entries[k].calls), float(entries[k].total_ms))
                for k in range(count.value)}

    def launch_count(self) -> int:
        return int(self._lib.gnnco_launch_count(self._handle))

    def close(self) -> None:
        if self._handle is not None:
            self._lib.gnnco_destroy(self._handle)
            self._handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def gnnco_partition_load(edge_u, edge_v, part, S: int, stream=None) -> PartitionedGraph:
    return PartitionedGraph(edge_u, edge_v, part, S, stream)


def gnnco_train_step(graph: PartitionedGraph, *args, **kwargs):
    return graph.train_step(*args, **kwargs)


def gnnco_decode_boundary(graph: PartitionedGraph, *args, **kwargs):
    return graph.decode_boundary(*args, **kwargs)


def gnnco_louvain(edge_u, edge_v, n: int, max_levels: int = 32, max_sweeps: int = 64, stream=None):
    """``gnnco_louvain``: deterministic Louvain partition of the graph (int32 device tensors ``edge_u``,
    ``edge_v``).  Returns dict(part [n] int32 device tensor, S, qnum, two_m, Q, levels, sweeps)."""
    import torch
    lib = load_library()
    _require(edge_u, torch.int32, "edge_u")
    _require(edge_v, torch.int32, "edge_v")
    E = int(edge_u.numel())
    need = _sz(0)
    _check(lib.gnnco_louvain_workspace_bytes(n, E, ctypes.byref(need)), "gnnco_louvain_workspace_bytes")
    ws = torch.empty(max(256, need.value), dtype=torch.uint8, device=edge_u.device)
    part = torch.empty(n, dtype=torch.int32, device=edge_u.device)
    S, levels, sweeps = _i32(0), _i32(0), _i32(0)
    qnum, two_m = _i64(0), _i64(0)
    _check(lib.gnnco_louvain(n, E, edge_u.data_ptr() if E else None, edge_v.data_ptr() if E else None, max_levels,
                             max_sweeps, part.data_ptr(), ctypes.byref(S), ctypes.byref(qnum), ctypes.byref(two_m),
                             ctypes.byref(levels), ctypes.byref(sweeps), ws.data_ptr(), ws.numel(), _stream_ptr(stream)),
           "gnnco_louvain")
    q = qnum.value / float(two_m.value) ** 2 if two_m.value else 0.0
    return dict(part=part, S=int(S.value), qnum=int(qnum.value), two_m=int(two_m.value), Q=q, levels=int(levels.value),
                sweeps=int(sweeps.value))
