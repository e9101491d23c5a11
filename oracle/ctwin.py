"""ctypes access to the plain-C twin of the oracle (oracle/bpt_oracle_c.c).

TEST INFRASTRUCTURE ONLY -- used by the tests, the smoke check and the
benchmark's CPU-baseline leg for sizes the NumPy oracle is too slow for.
``build()`` compiles the C file with gcc next to itself; nothing here touches
the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bpt_oracle_c.c")
_LIB = os.path.join(_HERE, "libbpt_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C twin if it is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, u32, dbl = ctypes.c_int64, ctypes.c_uint32, ctypes.c_double
        p = ctypes.c_void_p
        lib.orc_threads.restype = ctypes.c_int
        lib.orc_count_edges.restype = i64
        lib.orc_count_edges.argtypes = [i64, i64, u32]
        lib.orc_build_csr.restype = None
        lib.orc_build_csr.argtypes = [i64, i64, u32, p, p, p]
        lib.orc_transpose.restype = None
        lib.orc_transpose.argtypes = [i64, p, p, p, p, p]
        lib.orc_attn_fwd.restype = None
        lib.orc_attn_fwd.argtypes = [i64, p, p, p, i64, i64, i64, i64, i64, p, p, p, p, dbl, p, p, dbl, ctypes.c_uint64]
        lib.orc_attn_bwd.restype = None
        lib.orc_attn_bwd.argtypes = [i64, i64, p, p, p, i64, i64, i64, i64, i64, p, p, p, p, dbl, p, p, p, p, p, p, dbl, ctypes.c_uint64]
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().orc_threads())


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


class CGraph:
    """Same fields as oracle.bpt_oracle.Graph, produced by the C twin."""

    def __init__(self, n: int, k: int, flags: int = 0):
        lib = _load()
        self.n, self.k, self.flags = n, k, flags
        self.L = n.bit_length() - 1
        self.n_nodes = 2 * n - 1
        self.n_rel = 1 + 2 * self.L * (k + 1) + self.L
        E = int(lib.orc_count_edges(n, k, flags))
        self.n_edges = E
        self.row_ptr = np.zeros(2 * n, dtype=np.int32)
        self.col = np.zeros(E, dtype=np.int32)
        self.rel = np.zeros(E, dtype=np.int32)
        lib.orc_build_csr(n, k, flags, _ptr(self.row_ptr), _ptr(self.col), _ptr(self.rel))
        self.t_ptr = np.zeros(2 * n, dtype=np.int32)
        self.t_dst = np.zeros(E, dtype=np.int32)
        self.t_eid = np.zeros(E, dtype=np.int32)
        lib.orc_transpose(self.n_nodes, _ptr(self.row_ptr), _ptr(self.col),
                          _ptr(self.t_ptr), _ptr(self.t_dst), _ptr(self.t_eid))


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def attn_fwd(g, q, k, v, r, scale, b0=0, b1=None, p_drop=0.0, seed=0):
    """fp64 forward on batch entries [b0, b1); other entries of the outputs stay 0.
    p_drop, seed: attention dropout as defined in oracle/bpt_oracle.py (0 = none)."""
    q, k, v, r = _f64(q), _f64(k), _f64(v), _f64(r)
    B, N, H, d = q.shape
    b1 = B if b1 is None else b1
    out = np.zeros_like(q)
    lse = np.zeros((B, N, H))
    _load().orc_attn_fwd(N, _ptr(g.row_ptr), _ptr(g.col), _ptr(g.rel), B, H, d, b0, b1,
                         _ptr(q), _ptr(k), _ptr(v), _ptr(r), float(scale), _ptr(out), _ptr(lse), float(p_drop), int(seed))
    return out, lse


def attn_bwd(g, q, k, v, r, scale, d_out, b0=0, b1=None, out=None, p_drop=0.0, seed=0):
    """fp64 backward on batch entries [b0, b1); dr sums over those entries only.
    ``out``: optional stored forward output to use in the row term (see the C source)."""
    q, k, v, r, d_out = _f64(q), _f64(k), _f64(v), _f64(r), _f64(d_out)
    B, N, H, d = q.shape
    b1 = B if b1 is None else b1
    dq, dk, dv = np.zeros_like(q), np.zeros_like(q), np.zeros_like(q)
    dr = np.zeros_like(r)
    _out = None if out is None else _f64(out)
    _load().orc_attn_bwd(N, r.shape[0], _ptr(g.row_ptr), _ptr(g.col), _ptr(g.rel), B, H, d, b0, b1,
                         _ptr(q), _ptr(k), _ptr(v), _ptr(r), float(scale), _ptr(d_out),
                         None if out is None else _ptr(_out),
                         _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dr), float(p_drop), int(seed))
    return dq, dk, dv, dr


class MaskedGraph:
    """CSR of a CGraph restricted to the nodes that cover at least one of the first `length`
    tokens (same reading as oracle.bpt_oracle.mask_graph, written independently of it: a node id
    is decoded level by level, its first token is index << level)."""

    def __init__(self, g: CGraph, length: int):
        n, N = g.n, g.n_nodes
        first = np.zeros(N, dtype=np.int64)
        base, width, level = 0, n, 0
        while width >= 1:
            first[base:base + width] = np.arange(width, dtype=np.int64) << level
            base, width, level = base + width, width >> 1, level + 1
        real = first < length
        dst = np.repeat(np.arange(N), np.diff(g.row_ptr))
        keep = real[dst] & real[g.col]
        self.n, self.k, self.flags, self.L, self.n_nodes, self.n_rel = g.n, g.k, g.flags, g.L, N, g.n_rel
        self.row_ptr = np.zeros(N + 1, dtype=np.int32)
        np.cumsum(np.bincount(dst[keep], minlength=N), out=self.row_ptr[1:])
        self.col = np.ascontiguousarray(g.col[keep])
        self.rel = np.ascontiguousarray(g.rel[keep])
        self.n_edges = int(self.col.shape[0])


def attn_fwd_varlen(g, q, k, v, r, scale, lengths, p_drop=0.0, seed=0):
    """Forward with one length per batch entry (and, optionally, attention dropout)."""
    q = _f64(q)
    out = np.zeros_like(q)
    lse = np.zeros(q.shape[:3])
    for b, length in enumerate(lengths):
        o, l = attn_fwd(MaskedGraph(g, int(length)), q, k, v, r, scale, b0=b, b1=b + 1, p_drop=p_drop, seed=seed)
        out[b], lse[b] = o[b], l[b]
    return out, lse


def attn_bwd_varlen(g, q, k, v, r, scale, d_out, lengths, out=None, p_drop=0.0, seed=0):
    """Backward with one length per batch entry (and, optionally, attention dropout); dr sums over the batch."""
    q = _f64(q)
    dq, dk, dv = np.zeros_like(q), np.zeros_like(q), np.zeros_like(q)
    dr = np.zeros_like(_f64(r))
    for b, length in enumerate(lengths):
        a = attn_bwd(MaskedGraph(g, int(length)), q, k, v, r, scale, d_out, b0=b, b1=b + 1, out=out, p_drop=p_drop, seed=seed)
        dq[b], dk[b], dv[b] = a[0][b], a[1][b], a[2][b]
        dr += a[3]
    return dq, dk, dv, dr
