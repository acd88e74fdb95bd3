"""Python binding of libtreeverify (argument marshalling only).

Every function here has the name of the C entry point it forwards to
(``include/tree_verify.h``) minus the ``tv_`` prefix; all arithmetic runs in
the CUDA kernels of the shared library.  PyTorch supplies device memory and
the current stream, nothing else.  If the shared library has not been built
the first call raises: there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

GATED, DELTA = 0, 1
F32, BF16 = 0, 1
IMPL_AUTO, IMPL_SIMT, IMPL_TC = 0, 1, 2
MAX_NODES = 128
STATIC_MAX_TREES = 128

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtreeverify.so")
_lib = None


class TreeVerifyError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().tv_strerror(status).decode()
        if status == -4:
            msg += f" [cudaError {lib().tv_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({status})")


class _Strides(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in ("b", "h", "t")]


class _Dims(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("L", "B", "H", "T", "dk", "dv", "rule", "qkv_dtype", "impl", "Hk")] + \
               [(n, _Strides) for n in ("qk", "v", "gate", "out")]


class _ConvDims(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("B", "H", "T", "dk", "dv", "W", "io_dtype", "normalize_qk")] + [("eps", ctypes.c_float),
                                                                                   ("impl", ctypes.c_int32)]


def lib() -> ctypes.CDLL:
    """Load libtreeverify.so; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2608_01651_b200.build` "
            "(there is no non-CUDA fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, p = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER
    L.tv_strerror.restype = ctypes.c_char_p
    L.tv_strerror.argtypes = [ctypes.c_int]
    L.tv_version.restype = ctypes.c_int
    L.tv_last_cuda_error.restype = ctypes.c_int
    L.tv_tree_build.argtypes = [vp, i32, i32, p(vp)]
    L.tv_tree_rebuild.argtypes = [vp, vp]
    L.tv_forest_build.argtypes = [vp, vp, i32, i32, i32, p(vp)]
    L.tv_forest_rebuild.argtypes = [vp, vp, vp]
    L.tv_budget_workspace_bytes.argtypes = [i32, i32]
    L.tv_budget_workspace_bytes.restype = ctypes.c_size_t
    L.tv_budget_select.argtypes = [vp, vp, i32, i32, i32] + [vp] * 8
    L.tv_budget_select.restype = ctypes.c_int
    L.tv_forest_upload_device.argtypes = [vp, vp, vp, i32, vp]
    L.tv_forest_upload_device.restype = ctypes.c_int
    L.tv_forest_build.restype = ctypes.c_int
    L.tv_forest_rebuild.restype = ctypes.c_int
    L.tv_tree_meta.argtypes = [vp, vp, vp, vp]
    L.tv_tree_info.argtypes = [vp, p(i32), p(i32), p(i32)]
    L.tv_tree_path.argtypes = [vp, vp, i32, vp, i32, vp]
    L.tv_tree_upload.argtypes = [vp, vp]
    L.tv_tree_free.argtypes = [vp]
    L.tv_tree_device_status.argtypes = [vp, vp]
    L.tv_selftest_wait_timeout.argtypes = [vp, vp]
    L.tv_selftest_wait_timeout.restype = ctypes.c_int
    L.tv_tree_meta_device.argtypes = [vp, vp, vp, vp]
    L.tv_tree_meta_device.restype = ctypes.c_int
    L.tv_tree_device_status.restype = ctypes.c_int
    L.tv_tree_verify.argtypes = [vp, p(_Dims)] + [vp] * 9
    L.tv_commit_path.argtypes = [vp, p(_Dims)] + [vp] * 9
    L.tv_commit_path_layers.argtypes = [vp, p(_Dims), vp, i32] + [vp] * 8
    L.tv_commit_path_layers.restype = ctypes.c_int
    L.tv_tree_verify_static.argtypes = [vp, i32, p(_Dims)] + [vp] * 10
    L.tv_tree_verify_static.restype = ctypes.c_int
    L.tv_tree_conv.argtypes = [vp, p(_ConvDims)] + [vp] * 14
    L.tv_conv_commit.argtypes = [vp, p(_ConvDims)] + [vp] * 5
    L.tv_tree_conv.restype = ctypes.c_int
    L.tv_conv_commit.restype = ctypes.c_int
    L.tv_session_create.argtypes = [p(_Dims), i32, p(vp)]
    L.tv_session_round.argtypes = [vp] + [vp] * 11
    L.tv_session_free.argtypes = [vp]
    for name in ("tv_session_create", "tv_session_round", "tv_session_free"):
        getattr(L, name).restype = ctypes.c_int
    for name in ("tv_tree_build", "tv_tree_rebuild", "tv_tree_meta", "tv_tree_info", "tv_tree_path",
                 "tv_tree_upload", "tv_tree_free", "tv_tree_verify", "tv_commit_path"):
        getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


def _check(st: int, where: str):
    if st != 0:
        raise TreeVerifyError(st, where)


def _np_i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.int32)


class Tree:
    """Handle of a library-owned ``tv_tree`` (metadata of 1 or B proposal trees)."""

    def __init__(self, handle, n_trees, n):
        self._h = handle
        self.n_trees = n_trees
        self.n = n
        self.offsets = None     # packed forest (forest_build): int32 [n_trees + 1]
        self.capacity = None    # packed forest: rows of one (layer, head) plane

    def rebuild_forest(self, parents):
        """``tv_forest_rebuild``: new per-request parent arrays (lengths may change)."""
        parts = [_np_i32(p).reshape(-1) for p in parents]
        offsets = np.zeros(len(parts) + 1, dtype=np.int32)
        offsets[1:] = np.cumsum([len(p) for p in parts])
        flat = np.ascontiguousarray(np.concatenate(parts), dtype=np.int32)
        _check(lib().tv_forest_rebuild(self._h, flat.ctypes.data, offsets.ctypes.data), "tv_forest_rebuild")
        self.offsets = offsets
        return self

    def rebuild(self, parent):
        par = _np_i32(parent).reshape(self.n_trees, self.n)
        _check(lib().tv_tree_rebuild(self._h, par.ctypes.data), "tv_tree_rebuild")
        return self

    def meta(self):
        """(anc uint64 [n_trees,n,2], depth int32 [n_trees,n], max_depth int32 [n_trees])."""
        anc = np.zeros((self.n_trees, self.n, 2), dtype=np.uint64)
        depth = np.zeros((self.n_trees, self.n), dtype=np.int32)
        md = np.zeros(self.n_trees, dtype=np.int32)
        _check(lib().tv_tree_meta(self._h, anc.ctypes.data, depth.ctypes.data, md.ctypes.data),
               "tv_tree_meta")
        return anc, depth, md

    def meta_device(self, stream=None):
        """``tv_tree_meta_device``: the masks and depths as built on the device."""
        anc = np.zeros((self.n_trees, self.n, 2), dtype=np.uint64)
        depth = np.zeros((self.n_trees, self.n), dtype=np.int32)
        _check(lib().tv_tree_meta_device(self._h, anc.ctypes.data, depth.ctypes.data, _stream_ptr(stream)),
               "tv_tree_meta_device")
        return anc, depth

    @property
    def max_depth(self) -> int:
        md = ctypes.c_int32()
        _check(lib().tv_tree_info(self._h, None, None, ctypes.byref(md)), "tv_tree_info")
        return md.value

    def path(self, accepted):
        """(path int32 [n_req, max_depth+1] padded with -1, len int32 [n_req])."""
        acc = _np_i32(accepted).reshape(-1)
        stride = self.max_depth + 1
        path = np.zeros((len(acc), stride), dtype=np.int32)
        ln = np.zeros(len(acc), dtype=np.int32)
        _check(lib().tv_tree_path(self._h, acc.ctypes.data, len(acc), path.ctypes.data, stride,
                                  ln.ctypes.data), "tv_tree_path")
        return path, ln

    def upload(self, stream=None):
        _check(lib().tv_tree_upload(self._h, _stream_ptr(stream)), "tv_tree_upload")
        return self

    def prepare_refresh(self, parent, stream=None):
        """``tv_tree_rebuild`` + ``tv_tree_upload`` with pre-marshalled arguments: returns a
        callable that re-reads ``parent`` (an int32 C-contiguous numpy array that the caller
        updates in place) and uploads the new metadata."""
        par = np.asarray(parent)
        if par.dtype != np.int32 or not par.flags["C_CONTIGUOUS"] or par.size != self.n_trees * self.n:
            raise ValueError("parent must be a C-contiguous int32 array of n_trees * n entries")
        L = lib()
        h, pp, sp = self._h, ctypes.c_void_p(par.ctypes.data), _stream_ptr(stream)
        rebuild, upload = L.tv_tree_rebuild, L.tv_tree_upload

        def refresh(_keep=(par, self)):
            st = rebuild(h, pp)
            if st == 0:
                st = upload(h, sp)
            if st != 0:
                raise TreeVerifyError(st, "tv_tree_rebuild/tv_tree_upload")
        return refresh

    def upload_device(self, parent_padded, offsets, max_depth_bound, stream=None):
        """``tv_forest_upload_device``: metadata from CUDA int32 tensors (as ``budget_select`` leaves
        them); the host-side metadata of the handle is stale afterwards."""
        import torch
        _require(parent_padded, "parent_padded", torch.int32)
        _require(offsets, "offsets", torch.int32)
        _check(lib().tv_forest_upload_device(self._h, _ptr(parent_padded), _ptr(offsets), int(max_depth_bound),
                                             _stream_ptr(stream)), "tv_forest_upload_device")
        return self

    def prepare_refresh_forest(self, parent_flat, offsets, stream=None):
        """``tv_forest_rebuild`` + ``tv_tree_upload`` with pre-marshalled arguments; the caller
        updates the two int32 arrays in place between calls."""
        flat, off = np.asarray(parent_flat), np.asarray(offsets)
        for a in (flat, off):
            if a.dtype != np.int32 or not a.flags["C_CONTIGUOUS"]:
                raise ValueError("parent_flat and offsets must be C-contiguous int32 arrays")
        L = lib()
        h, pp, po, sp = self._h, ctypes.c_void_p(flat.ctypes.data), ctypes.c_void_p(off.ctypes.data), _stream_ptr(stream)
        rebuild, upload = L.tv_forest_rebuild, L.tv_tree_upload

        def refresh(_keep=(flat, off, self)):
            st = rebuild(h, pp, po)
            if st == 0:
                st = upload(h, sp)
            if st != 0:
                raise TreeVerifyError(st, "tv_forest_rebuild/tv_tree_upload")
        return refresh

    def device_status(self, stream=None):
        """``tv_tree_device_status``: synchronise and raise if a device wait timed out."""
        _check(lib().tv_tree_device_status(self._h, _stream_ptr(stream)), "tv_tree_device_status")

    def free(self):
        if self._h:
            lib().tv_tree_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def tree_build(parent) -> Tree:
    """``tv_tree_build``: parent int32 [n] or [n_trees, n], -1 <= parent[i] < i."""
    par = _np_i32(parent)
    if par.ndim == 1:
        par = par[None]
    n_trees, n = par.shape
    h = ctypes.c_void_p()
    _check(lib().tv_tree_build(par.ctypes.data, n_trees, n, ctypes.byref(h)), "tv_tree_build")
    return Tree(h, n_trees, n)


def forest_build(parents, n_max=None, capacity=None) -> Tree:
    """``tv_forest_build``: ``parents`` is a list of per-request parent arrays (local indices) of
    different lengths; they are packed in order.  Returns a ``Tree`` with ``offsets`` (int32
    [B+1]) and ``capacity``; node-indexed tensors are then [L][H][capacity][d] planes."""
    parts = [_np_i32(p).reshape(-1) for p in parents]
    offsets = np.zeros(len(parts) + 1, dtype=np.int32)
    offsets[1:] = np.cumsum([len(p) for p in parts])
    flat = np.ascontiguousarray(np.concatenate(parts), dtype=np.int32)
    n_max = int(max(len(p) for p in parts)) if n_max is None else int(n_max)
    capacity = int(offsets[-1]) if capacity is None else int(capacity)
    h = ctypes.c_void_p()
    _check(lib().tv_forest_build(flat.ctypes.data, offsets.ctypes.data, len(parts), n_max, capacity,
                                 ctypes.byref(h)), "tv_forest_build")
    t = Tree(h, len(parts), n_max)
    t.offsets, t.capacity = offsets, capacity
    return t


def budget_select(parent, p_draft, budget, *, status=None, stream=None, out=None):
    """``tv_budget_select``: ``parent`` int32 and ``p_draft`` float32 CUDA tensors [B, Tc].  Returns a
    dict of CUDA tensors: rho, counts, offsets, parent_packed, node_id (``out``: the dict of an
    earlier call with the same sizes, to reuse its tensors)."""
    import torch
    _require(parent, "parent", torch.int32)
    _require(p_draft, "p_draft", torch.float32)
    _require(status, "status", torch.int32)
    B, Tc = parent.shape
    dev = parent.device
    if out is not None:
        if out["node_id"].numel() != int(budget) or tuple(out["rho"].shape) != (B, Tc):
            raise ValueError("out does not match these sizes")
        _check(lib().tv_budget_select(_ptr(parent), _ptr(p_draft), B, Tc, int(budget), _ptr(out["rho"]),
                                      _ptr(out["counts"]), _ptr(out["offsets"]), _ptr(out["parent_packed"]),
                                      _ptr(out["node_id"]), _ptr(out["_workspace"]), _ptr(status),
                                      _stream_ptr(stream)), "tv_budget_select")
        return out
    out = {"rho": torch.empty(B, Tc, device=dev, dtype=torch.float32),
           "counts": torch.empty(B, device=dev, dtype=torch.int32),
           "offsets": torch.empty(B + 1, device=dev, dtype=torch.int32),
           "parent_packed": torch.empty(B, Tc, device=dev, dtype=torch.int32),
           "node_id": torch.empty(int(budget), device=dev, dtype=torch.int32)}
    ws = torch.empty(lib().tv_budget_workspace_bytes(B, Tc), device=dev, dtype=torch.uint8)
    _check(lib().tv_budget_select(_ptr(parent), _ptr(p_draft), B, Tc, int(budget), _ptr(out["rho"]),
                                  _ptr(out["counts"]), _ptr(out["offsets"]), _ptr(out["parent_packed"]),
                                  _ptr(out["node_id"]), _ptr(ws), _ptr(status), _stream_ptr(stream)),
           "tv_budget_select")
    out["_workspace"] = ws   # keep it alive until the stream has run the kernels
    return out


def _stream_ptr(stream):
    if stream is None:
        import torch
        if torch.cuda.is_available():
            return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
        return ctypes.c_void_p(0)
    if hasattr(stream, "cuda_stream"):
        return ctypes.c_void_p(stream.cuda_stream)
    return ctypes.c_void_p(int(stream))


def _ptr(t):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _strides_of(t, tail, B):
    """Element strides (b, h, t) of a node-indexed tensor [(L,) B, heads, T(, d)]; all zero for a
    contiguous one (the library's dense layout).  ``tail`` = 1 when the tensor has a channel axis."""
    if t is None or t.is_contiguous():
        return _Strides(0, 0, 0)
    if tail and t.stride(-1) != 1:
        raise ValueError("the channel axis must be contiguous")
    st = t.stride()
    b, h, n = st[-3 - tail], st[-2 - tail], st[-1 - tail]
    if t.dim() == 4 + tail and t.shape[0] > 1 and st[0] != B * b:
        raise ValueError("layers must be stacked with a stride of B batch strides")
    return _Strides(b, h, n)


def _same(a, b):
    return (a.b, a.h, a.t) == (b.b, b.h, b.t)


def _dims(S_pre, k, v, rule, impl, tree=None, q=None, gates=(), outs=()) -> _Dims:
    import torch
    if S_pre.dim() == 4:
        L = 1
        B, H, dv, dk = S_pre.shape
    elif S_pre.dim() == 5:
        L, B, H, dv, dk = S_pre.shape
    else:
        raise ValueError("S_pre must be [B,H,dv,dk] or [L,B,H,dv,dk]")
    T = k.shape[-2]
    if k.dtype == torch.bfloat16:
        dt = BF16
    elif k.dtype == torch.float32:
        dt = F32
    else:
        raise ValueError("q/k/v must be float32 or bfloat16")
    if tree is not None and getattr(tree, "capacity", None) is not None:
        # packed forest: [L][H][capacity][d] planes; the per-request node limit comes from the handle
        if T != tree.capacity or k.dim() != S_pre.dim() - 1:
            raise ValueError("packed-forest tensors must be [L][H][capacity][d] (or [H][capacity][d])")
        T = tree.n
    Hk = k.shape[-3]
    if H % Hk:
        raise ValueError("the number of state heads must be a multiple of the number of key heads")
    d = _Dims(L, B, H, T, dk, dv, rule, dt, impl, 0 if Hk == H else Hk)
    # strided views (token-major projections, slices of a fused projection) are passed as they are
    d.qk = _strides_of(k, 1, B)
    if q is not None and not _same(_strides_of(q, 1, B), d.qk):
        raise ValueError("q and k must share one layout")
    d.v = _strides_of(v, 1, B)
    gs = [_strides_of(g, 0, B) for g in gates if g is not None]
    os_ = [_strides_of(o, 1, B) for o in outs if o is not None]
    if any(not _same(x, gs[0]) for x in gs) or any(not _same(x, os_[0]) for x in os_):
        raise ValueError("alpha and beta (and O and U) must share one layout")
    if gs:
        d.gate = gs[0]
    if os_:
        d.out = os_[0]
    return d


def _require(t, name, dtype=None, strided=False):
    if t is None:
        return
    if not t.is_cuda or not (strided or t.is_contiguous()):
        raise ValueError(f"{name} must be a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}")


def tree_verify(tree: Tree, S_pre, q, k, v, alpha, beta=None, *, rule=GATED, O=None, U=None,
                want_U=False, impl=IMPL_AUTO, stream=None):
    """``tv_tree_verify``: per-node outputs O (and corrections U) for all nodes.

    Tensors are CUDA, contiguous, in the layout of ``tree_verify.h``.  Returns
    ``O`` or ``(O, U)``.
    """
    import torch
    _require(S_pre, "S_pre", torch.float32)
    for t, n in ((alpha, "alpha"), (beta, "beta")):
        _require(t, n, torch.float32, strided=True)
    for t, n in ((q, "q"), (k, "k"), (v, "v")):
        _require(t, n, k.dtype, strided=True)
    if O is None:
        O = torch.empty(*v.shape[:-1], v.shape[-1], device=v.device, dtype=torch.float32)
    if U is None and want_U:
        U = torch.empty_like(O)
    _require(O, "O", torch.float32, strided=True)
    _require(U, "U", torch.float32, strided=True)
    d = _dims(S_pre, k, v, rule, impl, tree, q=q, gates=(alpha, beta), outs=(O, U))
    _check(lib().tv_tree_verify(tree._h, ctypes.byref(d), _ptr(S_pre), _ptr(q), _ptr(k), _ptr(v),
                                _ptr(alpha), _ptr(beta), _ptr(O), _ptr(U), _stream_ptr(stream)),
           "tv_tree_verify")
    return (O, U) if U is not None else O


def commit_path(tree: Tree, accepted, S_pre, k, v, alpha, beta=None, *, rule=GATED, U=None,
                S_new=None, stream=None):
    """``tv_commit_path``: write the state at the end of the accepted path.

    ``accepted`` is a CUDA int32 tensor [B].  ``S_new=None`` commits in place
    and returns ``S_pre``.
    """
    import torch
    _require(accepted, "accepted", torch.int32)
    for t, n in ((S_pre, "S_pre"), (S_new, "S_new")):
        _require(t, n, torch.float32)
    for t, n in ((alpha, "alpha"), (beta, "beta"), (U, "U")):
        _require(t, n, torch.float32, strided=True)
    for t, n in ((k, "k"), (v, "v")):
        _require(t, n, k.dtype, strided=True)
    d = _dims(S_pre, k, v, rule, IMPL_AUTO, tree, gates=(alpha, beta), outs=(U,))
    out = S_pre if S_new is None else S_new
    _check(lib().tv_commit_path(tree._h, ctypes.byref(d), _ptr(accepted), _ptr(S_pre), _ptr(k),
                                _ptr(v), _ptr(alpha), _ptr(beta), _ptr(U), _ptr(out),
                                _stream_ptr(stream)), "tv_commit_path")
    return out


def commit_path_layers(tree: Tree, accepted, S_pre, k, v, alpha, beta=None, *, rule=GATED, U=None,
                       S_new=None, stream=None):
    """``tv_commit_path_layers``: one commit launch over layers that own their tensors separately.

    ``S_pre``, ``k``, ``v``, ``alpha`` (and ``beta``, ``U``, ``S_new`` when given) are lists with
    one tensor per layer, each shaped like a single layer of ``commit_path``; all layers share
    the tree, the accepted nodes, the shapes and the layout.  ``S_new=None`` commits in place.
    """
    import torch
    _require(accepted, "accepted", torch.int32)
    n = len(S_pre)
    lists = {"k": k, "v": v, "alpha": alpha, "beta": beta, "U": U, "S_new": S_new}
    for name, lst in lists.items():
        if lst is not None and len(lst) != n:
            raise ValueError(f"{name} must list one tensor per layer")
    for l in range(n):
        for t, nm in ((S_pre[l], "S_pre"), (None if S_new is None else S_new[l], "S_new")):
            _require(t, nm, torch.float32)
        for lst, nm in ((alpha, "alpha"), (beta, "beta"), (U, "U")):
            _require(None if lst is None else lst[l], nm, torch.float32, strided=True)
        for lst, nm in ((k, "k"), (v, "v")):
            _require(None if lst is None else lst[l], nm, k[0].dtype, strided=True)
    d = _dims(S_pre[0], k[0], v[0], rule, IMPL_AUTO, tree, gates=(alpha[0], None if beta is None else beta[0]),
              outs=(None if U is None else U[0],))
    for l in range(1, n):
        dl = _dims(S_pre[l], k[l], v[l], rule, IMPL_AUTO, tree, gates=(alpha[l], None if beta is None else beta[l]),
                   outs=(None if U is None else U[l],))
        if bytes(dl) != bytes(d):
            raise ValueError("all layers must share shapes and layout")
    out = S_pre if S_new is None else S_new
    table = lambda lst: None if lst is None else (ctypes.c_void_p * n)(*[t.data_ptr() for t in lst])
    tabs = [table(x) for x in (S_pre, k, v, alpha, beta, U, out)]
    _check(lib().tv_commit_path_layers(tree._h, ctypes.byref(d), _ptr(accepted), n,
                                       *[None if t is None else ctypes.cast(t, ctypes.c_void_p) for t in tabs],
                                       _stream_ptr(stream)), "tv_commit_path_layers")
    return out


def tree_verify_static(parent, S_pre, q, k, v, alpha, beta=None, *, rule=GATED, O, U=None, status=None,
                       impl=IMPL_AUTO, stream=None):
    """``tv_tree_verify_static``: verification for callers that must not allocate.

    ``parent`` is a CUDA int32 tensor [n_trees, T] (n_trees = 1 or B); ``O`` (and ``U``,
    ``status`` if wanted) are preallocated CUDA tensors.  Nothing is allocated here or in the
    library: the tree metadata lives in a fixed device array (at most 128 trees of 128 nodes).
    """
    import torch
    _require(parent, "parent", torch.int32)
    _require(status, "status", torch.int32)
    for t, n in ((S_pre, "S_pre"), (alpha, "alpha"), (beta, "beta"), (O, "O"), (U, "U")):
        _require(t, n, torch.float32)
    for t, n in ((q, "q"), (k, "k"), (v, "v")):
        _require(t, n, k.dtype)
    d = _dims(S_pre, k, v, rule, impl)
    n_trees = parent.shape[0] if parent.dim() == 2 else 1
    if parent.dim() not in (1, 2) or parent.shape[-1] != d.T:
        raise ValueError("parent must be [T] or [n_trees, T] with T = the node count of q/k/v")
    if n_trees not in (1, d.B):
        raise ValueError("parent must hold one tree or one tree per request")
    _check(lib().tv_tree_verify_static(_ptr(parent), n_trees, ctypes.byref(d), _ptr(S_pre), _ptr(q),
                                       _ptr(k), _ptr(v), _ptr(alpha), _ptr(beta), _ptr(O), _ptr(U),
                                       _ptr(status), _stream_ptr(stream)), "tv_tree_verify_static")
    return O


def _conv_dims(x, H, dk, dv, W, normalize_qk, eps, tree=None, impl=IMPL_AUTO) -> _ConvDims:
    import torch
    if tree is not None and tree.capacity is not None:
        # packed forest: x is [capacity, C]; request count and node limit come from the handle
        if x.dim() != 2 or x.shape[0] != tree.capacity or x.shape[1] != H * (2 * dk + dv):
            raise ValueError("packed-forest x must be [capacity, H*(2*dk+dv)]")
        dt = BF16 if x.dtype == torch.bfloat16 else F32 if x.dtype == torch.float32 else None
        if dt is None:
            raise ValueError("x must be float32 or bfloat16")
        return _ConvDims(tree.n_trees, H, tree.n, dk, dv, W, dt, int(bool(normalize_qk)), float(eps), int(impl))
    if x.dim() != 3 or x.shape[2] != H * (2 * dk + dv):
        raise ValueError("x must be [B, T, H*(2*dk+dv)]")
    if x.dtype == torch.bfloat16:
        dt = BF16
    elif x.dtype == torch.float32:
        dt = F32
    else:
        raise ValueError("x must be float32 or bfloat16")
    return _ConvDims(x.shape[0], H, x.shape[1], dk, dv, W, dt, int(bool(normalize_qk)), float(eps), int(impl))


def _conv_args(tree, x, ctx, weight, bias, H, dk, dv, gate_a, gate_b, A_log, dt_bias, normalize_qk, eps,
               q, k, v, alpha, beta, stream, impl=IMPL_AUTO):
    import torch
    for t, n in ((x, "x"), (ctx, "ctx"), (gate_a, "gate_a"), (gate_b, "gate_b"), (q, "q"), (k, "k"), (v, "v")):
        _require(t, n, x.dtype)
    for t, n in ((weight, "weight"), (bias, "bias"), (A_log, "A_log"), (dt_bias, "dt_bias"),
                 (alpha, "alpha"), (beta, "beta")):
        _require(t, n, torch.float32)
    if weight.dim() != 2 or weight.shape[0] != x.shape[-1]:
        raise ValueError("weight must be [C, W]")
    W = weight.shape[1]
    n_req = tree.n_trees if tree.capacity is not None else x.shape[0]
    if W > 1 and (ctx is None or tuple(ctx.shape) != (n_req, W - 1, x.shape[-1])):
        raise ValueError("ctx must be [B, W-1, C]")
    d = _conv_dims(x, H, dk, dv, W, normalize_qk, eps, tree, impl)
    args = (tree._h, ctypes.byref(d), _ptr(x), _ptr(ctx), _ptr(weight), _ptr(bias), _ptr(gate_a), _ptr(gate_b),
            _ptr(A_log), _ptr(dt_bias), _ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(beta), _stream_ptr(stream))
    keep = (tree, d, x, ctx, weight, bias, gate_a, gate_b, A_log, dt_bias, q, k, v, alpha, beta)
    return args, keep


def tree_conv(tree: Tree, x, ctx, weight, bias=None, *, H, dk, dv, gate_a=None, gate_b=None, A_log=None,
              dt_bias=None, normalize_qk=False, eps=1e-6, q=None, k=None, v=None, alpha=None, beta=None,
              stream=None, impl=IMPL_AUTO):
    """``tv_tree_conv``: tree-parallel causal convolution + bias + SiLU (+ q/k normalisation, + gates).

    ``x`` [B,T,C], ``ctx`` [B,W-1,C], ``weight`` f32 [C,W]; returns ``(q, k, v)`` head-major, and
    ``(q, k, v, alpha, beta)`` when ``gate_a`` is given (``beta`` None without ``gate_b``).
    """
    import torch
    lead = (H, tree.capacity) if tree.capacity is not None else (x.shape[0], H, x.shape[1])
    q = torch.empty(*lead, dk, device=x.device, dtype=x.dtype) if q is None else q
    k = torch.empty(*lead, dk, device=x.device, dtype=x.dtype) if k is None else k
    v = torch.empty(*lead, dv, device=x.device, dtype=x.dtype) if v is None else v
    if gate_a is not None and alpha is None:
        alpha = torch.empty(*lead, device=x.device, dtype=torch.float32)
    if gate_b is not None and beta is None:
        beta = torch.empty(*lead, device=x.device, dtype=torch.float32)
    args, _keep = _conv_args(tree, x, ctx, weight, bias, H, dk, dv, gate_a, gate_b, A_log, dt_bias,
                             normalize_qk, eps, q, k, v, alpha, beta, stream, impl)
    _check(lib().tv_tree_conv(*args), "tv_tree_conv")
    return (q, k, v) if gate_a is None else (q, k, v, alpha, beta)


def prepare_tree_conv(tree: Tree, x, ctx, weight, bias=None, *, H, dk, dv, gate_a=None, gate_b=None,
                      A_log=None, dt_bias=None, normalize_qk=False, eps=1e-6, q, k, v, alpha=None, beta=None,
                      stream=None, impl=IMPL_AUTO) -> "Prepared":
    """``tv_tree_conv`` with pre-marshalled arguments; outputs must be given."""
    args, keep = _conv_args(tree, x, ctx, weight, bias, H, dk, dv, gate_a, gate_b, A_log, dt_bias,
                            normalize_qk, eps, q, k, v, alpha, beta, stream, impl)
    return Prepared(lib().tv_tree_conv, "tv_tree_conv", args, keep)


def conv_commit(tree: Tree, accepted, x, ctx, *, H, dk, dv, ctx_new=None, stream=None):
    """``tv_conv_commit``: context rows after the accepted path (in place when ``ctx_new`` is None)."""
    import torch
    _require(accepted, "accepted", torch.int32)
    for t, n in ((x, "x"), (ctx, "ctx"), (ctx_new, "ctx_new")):
        _require(t, n, x.dtype)
    out = ctx if ctx_new is None else ctx_new
    d = _conv_dims(x, H, dk, dv, ctx.shape[1] + 1, False, 0.0, tree)
    _check(lib().tv_conv_commit(tree._h, ctypes.byref(d), _ptr(accepted), _ptr(x), _ptr(ctx), _ptr(out),
                                _stream_ptr(stream)), "tv_conv_commit")
    return out


def selftest_wait_timeout(status, stream=None):
    """``tv_selftest_wait_timeout``: make a bounded device wait run out; ``status`` is a CUDA int32[1]."""
    _check(lib().tv_selftest_wait_timeout(_ptr(status), _stream_ptr(stream)), "tv_selftest_wait_timeout")


class Prepared:
    """A C-ABI call with its arguments marshalled once (for loops that repeat the same call:
    validation and ctypes conversion are paid at construction, the call itself is one foreign
    call).  Holds references to every tensor it points into."""

    def __init__(self, fn, name, args, keep):
        self._fn, self._name, self._args, self._keep = fn, name, args, keep

    def __call__(self):
        st = self._fn(*self._args)
        if st != 0:
            raise TreeVerifyError(st, self._name)


def prepare_tree_verify(tree: Tree, S_pre, q, k, v, alpha, beta=None, *, rule=GATED, O=None, U=None,
                        impl=IMPL_AUTO, stream=None) -> Prepared:
    """``tv_tree_verify`` with pre-marshalled arguments; ``O`` (and ``U``) must be given."""
    import torch
    for t, n in ((S_pre, "S_pre"), (alpha, "alpha"), (beta, "beta"), (O, "O"), (U, "U")):
        _require(t, n, torch.float32)
    for t, n in ((q, "q"), (k, "k"), (v, "v")):
        _require(t, n, k.dtype)
    if O is None:
        raise ValueError("O must be preallocated")
    d = _dims(S_pre, k, v, rule, impl, tree)
    args = (tree._h, ctypes.byref(d), _ptr(S_pre), _ptr(q), _ptr(k), _ptr(v), _ptr(alpha), _ptr(beta),
            _ptr(O), _ptr(U), _stream_ptr(stream))
    return Prepared(lib().tv_tree_verify, "tv_tree_verify", args, (tree, d, S_pre, q, k, v, alpha, beta, O, U))


def prepare_commit_path(tree: Tree, accepted, S_pre, k, v, alpha, beta=None, *, rule=GATED, U=None,
                        S_new=None, stream=None) -> Prepared:
    """``tv_commit_path`` with pre-marshalled arguments (in place when ``S_new`` is None)."""
    import torch
    _require(accepted, "accepted", torch.int32)
    for t, n in ((S_pre, "S_pre"), (alpha, "alpha"), (beta, "beta"), (U, "U"), (S_new, "S_new")):
        _require(t, n, torch.float32)
    for t, n in ((k, "k"), (v, "v")):
        _require(t, n, k.dtype)
    d = _dims(S_pre, k, v, rule, IMPL_AUTO, tree)
    out = S_pre if S_new is None else S_new
    args = (tree._h, ctypes.byref(d), _ptr(accepted), _ptr(S_pre), _ptr(k), _ptr(v), _ptr(alpha),
            _ptr(beta), _ptr(U), _ptr(out), _stream_ptr(stream))
    return Prepared(lib().tv_commit_path, "tv_commit_path", args,
                    (tree, d, accepted, S_pre, k, v, alpha, beta, U, out))


class Session:
    """Handle of a ``tv_session``: device copies for host-buffer rounds."""

    def __init__(self, L, B, H, T, dk, dv, *, rule=GATED, qkv_dtype=BF16, n_trees=None,
                 impl=IMPL_AUTO, Hk=None):
        self.dims = _Dims(L, B, H, T, dk, dv, rule, qkv_dtype, impl, 0 if Hk in (None, H) else Hk)
        self._h = ctypes.c_void_p()
        _check(lib().tv_session_create(ctypes.byref(self.dims), B if n_trees is None else n_trees,
                                       ctypes.byref(self._h)), "tv_session_create")

    def round(self, parent, accepted, S_pre, q, k, v, alpha, beta, O, S_new, stream=None):
        """``tv_session_round``: all arguments are HOST tensors/arrays (torch CPU
        tensors, ideally pinned; parent/accepted int32 numpy arrays)."""
        par = _np_i32(parent)
        acc = _np_i32(accepted)
        _check(lib().tv_session_round(self._h, par.ctypes.data, acc.ctypes.data, _ptr(S_pre), _ptr(q),
                                      _ptr(k), _ptr(v), _ptr(alpha), _ptr(beta), _ptr(O), _ptr(S_new),
                                      _stream_ptr(stream)), "tv_session_round")
        return O, S_new

    def free(self):
        if self._h:
            lib().tv_session_free(self._h)
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def session_create(*args, **kw) -> Session:
    return Session(*args, **kw)
