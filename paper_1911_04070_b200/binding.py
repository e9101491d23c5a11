"""Thin Python binding of the C ABI in include/bpt.h (argument marshalling only).

PyTorch supplies device memory and the current stream; every step of the path
runs in the CUDA kernels of libbpt.so.  There is no CPU fallback: a missing
library or a failing call raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbpt.so")
CHECK_LIB_PATH = os.path.join(_HERE, "libbpt_check.so")   # the build with index checks; set LIB_PATH to it before the first call

BPT_BIDIR, BPT_LEFT_ONLY, BPT_MODE_PAD, BPT_MODE_ALG1 = 0, 1, 0, 2
BPT_F32, BPT_BF16 = 0, 1
BPT_PATH_AUTO, BPT_PATH_MMA, BPT_PATH_TC5 = 0, 1, 2

EXPORTS = ("bpt_graph_dims_query", "bpt_build_graph", "bpt_attn_workspace_bytes", "bpt_attn_fwd",
           "bpt_attn_bwd", "bpt_status_str", "bpt_trace_begin", "bpt_trace_end",
           "bpt_static_scratch_bytes", "bpt_attn_bwd_static_scratch", "bpt_attn_fwd_varlen", "bpt_attn_bwd_varlen",
           "bpt_attn_fwd_ex", "bpt_attn_bwd_ex", "bpt_attn_fwd_rows", "bpt_attn_bwd_min_workspace_bytes", "bpt_check",
           "bpt_selftest_wait_timeout", "bpt_debug_bounds", "bpt_out_proj_norm")


class BptError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (where, status_str(status), status))


class GraphDims(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int32), ("k", ctypes.c_int32), ("flags", ctypes.c_uint32),
                ("n_levels", ctypes.c_int32), ("n_nodes", ctypes.c_int32), ("n_rel", ctypes.c_int32),
                ("n_edges", ctypes.c_int64), ("build_workspace_bytes", ctypes.c_size_t)]


class GraphStruct(ctypes.Structure):
    _fields_ = [("row_ptr", ctypes.c_void_p), ("col", ctypes.c_void_p), ("rel", ctypes.c_void_p),
                ("t_ptr", ctypes.c_void_p), ("t_dst", ctypes.c_void_p), ("t_eid", ctypes.c_void_p),
                ("dims", GraphDims)]


class AttnOptions(ctypes.Structure):
    _fields_ = [("lengths", ctypes.c_void_p), ("dropout_p", ctypes.c_float), ("dropout_seed", ctypes.c_uint64),
                ("path", ctypes.c_uint32)]


# When set, the autograd wrapper in layer.py asks bpt_check after every attention call (a stream
# synchronisation per call): for debugging; training loops normally check once per step.
CHECK_DEVICE_STATUS = False

_lib = None


def load_library() -> ctypes.CDLL:
    """Load libbpt.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libbpt.so is missing: run `python -m paper_1911_04070_b200.build` "
                              "(there is no fallback implementation)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, u32, sz, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint32, ctypes.c_size_t, ctypes.c_float
        lib.bpt_graph_dims_query.restype = ctypes.c_int
        lib.bpt_graph_dims_query.argtypes = [i32, i32, u32, ctypes.POINTER(GraphDims)]
        lib.bpt_build_graph.restype = ctypes.c_int
        lib.bpt_build_graph.argtypes = [ctypes.POINTER(GraphDims), vp, vp, vp, vp, vp, vp, vp, vp, ctypes.POINTER(GraphStruct)]
        lib.bpt_attn_workspace_bytes.restype = sz
        lib.bpt_attn_workspace_bytes.argtypes = [ctypes.POINTER(GraphStruct), i32, i32, i32, ctypes.c_int, ctypes.c_int]
        lib.bpt_attn_bwd_min_workspace_bytes.restype = sz
        lib.bpt_attn_bwd_min_workspace_bytes.argtypes = [ctypes.POINTER(GraphStruct), i32, i32, i32, ctypes.c_int]
        lib.bpt_check.restype = ctypes.c_int
        lib.bpt_check.argtypes = [vp, vp]
        lib.bpt_selftest_wait_timeout.restype = ctypes.c_int
        lib.bpt_selftest_wait_timeout.argtypes = [vp, ctypes.c_int64, i32, vp]
        lib.bpt_out_proj_norm.restype = ctypes.c_int
        lib.bpt_out_proj_norm.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_int64, i32, f32, vp, vp]
        lib.bpt_debug_bounds.restype = ctypes.c_int
        lib.bpt_debug_bounds.argtypes = [ctypes.POINTER(ctypes.c_uint32), vp]
        lib.bpt_attn_fwd.restype = ctypes.c_int
        lib.bpt_attn_fwd.argtypes = [ctypes.POINTER(GraphStruct), i32, i32, i32, ctypes.c_int, vp, vp, vp, vp, f32,
                                     vp, vp, vp, sz, vp]
        lib.bpt_attn_bwd.restype = ctypes.c_int
        lib.bpt_attn_bwd.argtypes = [ctypes.POINTER(GraphStruct), i32, i32, i32, ctypes.c_int, vp, vp, vp, vp, f32,
                                     vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.bpt_attn_fwd_varlen.restype = ctypes.c_int
        lib.bpt_attn_fwd_varlen.argtypes = [ctypes.POINTER(GraphStruct), i32, i32, i32, ctypes.c_int, vp, vp, vp, vp, f32,
                                            vp, vp, vp, vp, sz, vp]
        lib.bpt_attn_bwd_varlen.restype = ctypes.c_int
        lib.bpt_attn_bwd_varlen.argtypes = [ctypes.POINTER(GraphStruct), i32, i32, i32, ctypes.c_int, vp, vp, vp, vp, f32,
                                            vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.bpt_attn_fwd_ex.restype = ctypes.c_int
        lib.bpt_attn_fwd_ex.argtypes = [ctypes.POINTER(GraphStruct), i32, i32, i32, ctypes.c_int, vp, vp, vp, vp, f32,
                                        ctypes.POINTER(AttnOptions), vp, vp, vp, sz, vp]
        lib.bpt_attn_bwd_ex.restype = ctypes.c_int
        lib.bpt_attn_bwd_ex.argtypes = [ctypes.POINTER(GraphStruct), i32, i32, i32, ctypes.c_int, vp, vp, vp, vp, f32,
                                        ctypes.POINTER(AttnOptions), vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.bpt_attn_fwd_rows.restype = ctypes.c_int
        lib.bpt_attn_fwd_rows.argtypes = [ctypes.POINTER(GraphStruct), i32, i32, i32, ctypes.c_int, vp, vp, vp, vp, f32,
                                          ctypes.POINTER(AttnOptions), vp, i32, vp, vp, vp]
        lib.bpt_static_scratch_bytes.restype = sz
        lib.bpt_static_scratch_bytes.argtypes = []
        lib.bpt_attn_bwd_static_scratch.restype = ctypes.c_int
        lib.bpt_attn_bwd_static_scratch.argtypes = [ctypes.POINTER(GraphStruct), i32, i32, i32, ctypes.c_int, vp, vp, vp, vp,
                                                    f32, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.bpt_trace_begin.restype = ctypes.c_int
        lib.bpt_trace_begin.argtypes = [i32, vp]
        lib.bpt_trace_end.restype = ctypes.c_int
        lib.bpt_trace_end.argtypes = [ctypes.POINTER(i32), ctypes.POINTER(f32), ctypes.POINTER(ctypes.c_char_p), i32]
        lib.bpt_status_str.restype = ctypes.c_char_p
        lib.bpt_status_str.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def status_str(status: int) -> str:
    return load_library().bpt_status_str(int(status)).decode()


def _check(status: int, where: str):
    if status != 0:
        raise BptError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return BPT_F32
    if t.dtype == torch.bfloat16:
        return BPT_BF16
    raise TypeError("only float32 and bfloat16 tensors are supported, got %s" % t.dtype)


def bpt_graph_dims_query(n: int, k: int, flags: int = 0) -> GraphDims:
    dims = GraphDims()
    _check(load_library().bpt_graph_dims_query(n, k, flags, ctypes.byref(dims)), "bpt_graph_dims_query")
    return dims


class Graph:
    """Device-resident BPT graph: owns the index tensors the C struct points at."""

    def __init__(self, dims: GraphDims, device, with_transpose: bool):
        E, N = dims.n_edges, dims.n_nodes
        i32 = dict(dtype=torch.int32, device=device)
        self.dims = dims
        self.row_ptr = torch.empty(N + 1, **i32)
        self.col = torch.empty(E, **i32)
        self.rel = torch.empty(E, **i32)
        self.t_ptr = torch.empty(N + 1, **i32) if with_transpose else None
        self.t_dst = torch.empty(E, **i32) if with_transpose else None
        self.t_eid = torch.empty(E, **i32) if with_transpose else None
        self.c = GraphStruct()

    n = property(lambda s: s.dims.n)
    k = property(lambda s: s.dims.k)
    n_nodes = property(lambda s: s.dims.n_nodes)
    n_edges = property(lambda s: s.dims.n_edges)
    n_rel = property(lambda s: s.dims.n_rel)


def bpt_build_graph(n: int, k: int, flags: int = 0, device="cuda", with_transpose: bool = True) -> Graph:
    """Builds the graph of (n, k, flags) on `device` with the library's kernels."""
    lib = load_library()
    dims = bpt_graph_dims_query(n, k, flags)
    device = torch.device(device)
    with torch.cuda.device(device):
        g = Graph(dims, device, with_transpose)
        ws = torch.empty(max(int(dims.build_workspace_bytes), 1), dtype=torch.uint8, device=device)
        _check(lib.bpt_build_graph(ctypes.byref(dims), _ptr(g.row_ptr), _ptr(g.col), _ptr(g.rel),
                                   _ptr(g.t_ptr), _ptr(g.t_dst), _ptr(g.t_eid), _ptr(ws), _stream(),
                                   ctypes.byref(g.c)), "bpt_build_graph")
        g._build_ws = ws  # keep alive until the stream has run the build
    return g


def bpt_attn_workspace_bytes(g: Graph, B: int, H: int, d: int, dtype_code: int, backward: bool) -> int:
    return int(load_library().bpt_attn_workspace_bytes(ctypes.byref(g.c), B, H, d, dtype_code, int(backward)))


def bpt_attn_bwd_min_workspace_bytes(g: Graph, B: int, H: int, d: int, dtype_code: int) -> int:
    """The smallest workspace bpt_attn_bwd accepts (it then works through the problem in more passes)."""
    return int(load_library().bpt_attn_bwd_min_workspace_bytes(ctypes.byref(g.c), B, H, d, dtype_code))


def bpt_check(workspace) -> int:
    """Waits for the current stream and returns the status the last attention call left in `workspace`
    (0 = ok, 5 = a bounded device-side wait expired: that call's results are invalid)."""
    dev = torch.cuda.current_device() if workspace is None else workspace.device
    with torch.cuda.device(dev):
        return int(load_library().bpt_check(_ptr(workspace), _stream()))


def bpt_out_proj_norm(a, w_o, h, gamma, beta, eps: float = 1e-5, z=None, workspace=None):
    """z = LayerNorm(h + a @ w_o.T) * gamma + beta over the last axis, in one kernel (bf16 in and out, fp32
    accumulation and statistics).  a, h: [..., D] bfloat16 contiguous; w_o: [D, D] bfloat16; gamma, beta: [D]
    float32; D in (128, 256, 512).  Forward only."""
    D = a.shape[-1]
    for t in (a, h):
        if t.dtype != torch.bfloat16 or not t.is_contiguous() or t.shape != a.shape or not t.is_cuda:
            raise ValueError("a and h must be contiguous bfloat16 CUDA tensors of one shape")
    if w_o.dtype != torch.bfloat16 or w_o.shape != (D, D) or not w_o.is_contiguous():
        raise ValueError("w_o must be a contiguous bfloat16 [D, D] tensor")
    for t in (gamma, beta):
        if t.dtype != torch.float32 or t.shape != (D,) or not t.is_contiguous():
            raise ValueError("gamma and beta must be contiguous float32 [D] tensors")
    rows = a.numel() // D
    with torch.cuda.device(a.device):
        z = torch.empty_like(a) if z is None else z
        _check(load_library().bpt_out_proj_norm(_ptr(a), _ptr(w_o), _ptr(h), _ptr(gamma), _ptr(beta), _ptr(z), rows, D, float(eps),
                                                _ptr(workspace), _stream()), "bpt_out_proj_norm")
    return z


def bpt_debug_bounds():
    """The index-check record of the checking build as (violations, site, index, limit); raises BptError
    with status 2 on the normal build, which carries no checks."""
    rec = (ctypes.c_uint32 * 4)()
    _check(load_library().bpt_debug_bounds(rec, _stream()), "bpt_debug_bounds")
    return tuple(int(x) for x in rec)


def bpt_selftest_wait_timeout(workspace, limit_cycles: int, arrive: bool):
    """Launches the library's wait self-test (see include/bpt.h); read the outcome with bpt_check."""
    with torch.cuda.device(workspace.device):
        _check(load_library().bpt_selftest_wait_timeout(_ptr(workspace), int(limit_cycles), int(arrive), _stream()),
               "bpt_selftest_wait_timeout")


def _check_layout(g: Graph, q, *same):
    if q.dim() != 4 or q.shape[1] != g.n_nodes:
        raise ValueError("expected [B, n_nodes=%d, H, d], got %s" % (g.n_nodes, tuple(q.shape)))
    for t in same:
        if t.shape != q.shape or t.dtype != q.dtype or t.device != q.device:
            raise ValueError("q, k, v, out, d_out must share shape, dtype and device")
    for t in (q,) + same:
        if not t.is_contiguous():
            raise ValueError("tensors must be contiguous")
        if not t.is_cuda:
            raise ValueError("tensors must live on a CUDA device")


def _check_lengths(lengths, q):
    if lengths.dtype != torch.int32 or lengths.shape != (q.shape[0],) or lengths.device != q.device or not lengths.is_contiguous():
        raise ValueError("lengths must be a contiguous int32 tensor [B] on the device of q")


def bpt_attn_fwd(g: Graph, q, k, v, rel_emb, scale: float, out=None, lse=None, workspace=None, lengths=None,
                 dropout_p: float = 0.0, dropout_seed: int = 0, path: int = BPT_PATH_AUTO):
    """Returns (out [B,N,H,d], lse [B,N,H] fp32).  With `lengths` (int32 [B] on the device) batch entry b
    has lengths[b] real tokens; with dropout_p > 0 the attention weights are dropped (mask defined by
    dropout_seed); `path` forces a kernel family; see bpt_attn_fwd_varlen / bpt_attn_fwd_ex in include/bpt.h.
    A workspace the wrapper allocates itself stays reachable as `out._bpt_workspace` for bpt_check."""
    lib = load_library()
    _check_layout(g, q, k, v)
    B, N, H, d = q.shape
    code = _dtype_code(q)
    if rel_emb.shape != (g.n_rel, d) or rel_emb.dtype != q.dtype or not rel_emb.is_contiguous():
        raise ValueError("rel_emb must be contiguous [n_rel=%d, d] of the same dtype" % g.n_rel)
    with torch.cuda.device(q.device):
        out = torch.empty_like(q) if out is None else out
        lse = torch.empty((B, N, H), dtype=torch.float32, device=q.device) if lse is None else lse
        need = bpt_attn_workspace_bytes(g, B, H, d, code, False)
        if workspace is None and need:
            workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
        ws_n = 0 if workspace is None else workspace.numel()
        out._bpt_workspace = workspace
        if dropout_p or path:
            if lengths is not None:
                _check_lengths(lengths, q)
            opt = AttnOptions(_ptr(lengths), float(dropout_p), int(dropout_seed), int(path))
            _check(lib.bpt_attn_fwd_ex(ctypes.byref(g.c), B, H, d, code, _ptr(q), _ptr(k), _ptr(v), _ptr(rel_emb),
                                       float(scale), ctypes.byref(opt), _ptr(out), _ptr(lse), _ptr(workspace), ws_n,
                                       _stream()), "bpt_attn_fwd_ex")
        elif lengths is None:
            _check(lib.bpt_attn_fwd(ctypes.byref(g.c), B, H, d, code, _ptr(q), _ptr(k), _ptr(v), _ptr(rel_emb),
                                    float(scale), _ptr(out), _ptr(lse), _ptr(workspace), ws_n, _stream()), "bpt_attn_fwd")
        else:
            _check_lengths(lengths, q)
            _check(lib.bpt_attn_fwd_varlen(ctypes.byref(g.c), B, H, d, code, _ptr(q), _ptr(k), _ptr(v), _ptr(rel_emb),
                                           float(scale), _ptr(lengths), _ptr(out), _ptr(lse), _ptr(workspace), ws_n,
                                           _stream()), "bpt_attn_fwd_varlen")
    return out, lse


def bpt_attn_bwd(g: Graph, q, k, v, rel_emb, scale: float, out, lse, d_out, workspace=None,
                 dq=None, dk=None, dv=None, d_rel=None, lengths=None, dropout_p: float = 0.0, dropout_seed: int = 0,
                 path: int = BPT_PATH_AUTO):
    """Returns (dq, dk, dv [B,N,H,d], d_rel [n_rel, d] fp32).  `lengths`, `dropout_p`, `dropout_seed` as for
    bpt_attn_fwd (pass what the forward had).  A workspace the wrapper allocates itself stays reachable as
    `dq._bpt_workspace` for bpt_check."""
    lib = load_library()
    _check_layout(g, q, k, v, out, d_out)
    B, N, H, d = q.shape
    code = _dtype_code(q)
    with torch.cuda.device(q.device):
        dq = torch.empty_like(q) if dq is None else dq
        dk = torch.empty_like(q) if dk is None else dk
        dv = torch.empty_like(q) if dv is None else dv
        d_rel = torch.empty((g.n_rel, d), dtype=torch.float32, device=q.device) if d_rel is None else d_rel
        need = bpt_attn_workspace_bytes(g, B, H, d, code, True)
        if workspace is None and need:
            workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
        ws_n = 0 if workspace is None else workspace.numel()
        dq._bpt_workspace = workspace
        if dropout_p or path:
            if lengths is not None:
                _check_lengths(lengths, q)
            opt = AttnOptions(_ptr(lengths), float(dropout_p), int(dropout_seed), int(path))
            _check(lib.bpt_attn_bwd_ex(ctypes.byref(g.c), B, H, d, code, _ptr(q), _ptr(k), _ptr(v), _ptr(rel_emb),
                                       float(scale), ctypes.byref(opt), _ptr(out), _ptr(lse), _ptr(d_out), _ptr(dq),
                                       _ptr(dk), _ptr(dv), _ptr(d_rel), _ptr(workspace), ws_n, _stream()), "bpt_attn_bwd_ex")
        elif lengths is None:
            _check(lib.bpt_attn_bwd(ctypes.byref(g.c), B, H, d, code, _ptr(q), _ptr(k), _ptr(v), _ptr(rel_emb),
                                    float(scale), _ptr(out), _ptr(lse), _ptr(d_out), _ptr(dq), _ptr(dk), _ptr(dv),
                                    _ptr(d_rel), _ptr(workspace), ws_n, _stream()), "bpt_attn_bwd")
        else:
            _check_lengths(lengths, q)
            _check(lib.bpt_attn_bwd_varlen(ctypes.byref(g.c), B, H, d, code, _ptr(q), _ptr(k), _ptr(v), _ptr(rel_emb),
                                           float(scale), _ptr(lengths), _ptr(out), _ptr(lse), _ptr(d_out), _ptr(dq),
                                           _ptr(dk), _ptr(dv), _ptr(d_rel), _ptr(workspace), ws_n, _stream()),
                   "bpt_attn_bwd_varlen")
    return dq, dk, dv, d_rel


def bpt_attn_fwd_rows(g: Graph, q, k, v, rel_emb, scale: float, rows, out, lse, lengths=None,
                      dropout_p: float = 0.0, dropout_seed: int = 0):
    """Recomputes the listed destination rows of (out, lse) in place.  rows: int32 [B, n_rows] node ids on the
    device (one list per batch entry).  The building block of step-by-step decoding: token i and its
    ancestors, with lengths = i + 1."""
    _check_layout(g, q, k, v, out)
    B, N, H, d = q.shape
    if rows.dtype != torch.int32 or rows.dim() != 2 or rows.shape[0] != B or not rows.is_contiguous() or rows.device != q.device:
        raise ValueError("rows must be a contiguous int32 tensor [B, n_rows] on the device of q")
    if lengths is not None:
        _check_lengths(lengths, q)
    opt = AttnOptions(_ptr(lengths), float(dropout_p), int(dropout_seed), 0)
    with torch.cuda.device(q.device):
        _check(load_library().bpt_attn_fwd_rows(ctypes.byref(g.c), B, H, d, _dtype_code(q), _ptr(q), _ptr(k), _ptr(v),
                                                _ptr(rel_emb), float(scale), ctypes.byref(opt), _ptr(rows), rows.shape[1],
                                                _ptr(out), _ptr(lse), _stream()), "bpt_attn_fwd_rows")
    return out, lse


def bpt_static_scratch_bytes() -> int:
    return int(load_library().bpt_static_scratch_bytes())


def bpt_attn_bwd_static_scratch(g: Graph, q, k, v, rel_emb, scale: float, out, lse, d_out, dq, dk, dv, d_rel):
    """Backward pass that takes its scratch from the library's built-in device array instead
    of a workspace tensor, for callers that are not allowed to allocate device memory.  The
    caller passes every input and output (this wrapper allocates nothing either); a problem
    of which one (batch entry, head) pair alone needs more than bpt_static_scratch_bytes() raises
    BptError with status 7.  Calls share the array:
    keep them ordered on one stream."""
    _check_layout(g, q, k, v, out, d_out, dq, dk, dv)
    B, N, H, d = q.shape
    with torch.cuda.device(q.device):
        _check(load_library().bpt_attn_bwd_static_scratch(
            ctypes.byref(g.c), B, H, d, _dtype_code(q), _ptr(q), _ptr(k), _ptr(v), _ptr(rel_emb), float(scale),
            _ptr(out), _ptr(lse), _ptr(d_out), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(d_rel), _stream()),
            "bpt_attn_bwd_static_scratch")
    return dq, dk, dv, d_rel


def bpt_trace_begin(capacity: int):
    """Start recording one CUDA event after every kernel the library launches."""
    _check(load_library().bpt_trace_begin(capacity, _stream()), "bpt_trace_begin")


def bpt_trace_end(capacity: int):
    """Stop recording; returns [(kernel name, milliseconds), ...] in launch order."""
    n = ctypes.c_int32(0)
    ms = (ctypes.c_float * capacity)()
    names = (ctypes.c_char_p * capacity)()
    _check(load_library().bpt_trace_end(ctypes.byref(n), ms, names, capacity), "bpt_trace_end")
    return [(names[i].decode(), float(ms[i])) for i in range(min(n.value, capacity))]
