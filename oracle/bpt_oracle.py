"""CPU oracle for BP-Transformer graph self-attention (arXiv 1911.04070).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  It must never be imported by the product
package; only the tests, the smoke check and the benchmark's CPU-baseline leg
use it.  It shares no code with the CUDA path.

Everything here is fp64 NumPy written straight from the paper:

* ``enumerate_graph``  -- Section 3.2 (node construction, affiliated edges,
  contextual edges incl. the parity pad rule, Algorithm 1) and Section 3.4
  (one relation label per edge).
* ``attn_fwd``         -- Graph self-attention with tree relative positions,
  Section 3.1 / 3.4 (the softmax((Q (K+R)^T)/sqrt(d)) V equation of 3.4).
* ``attn_bwd``         -- the analytic gradient of that equation.

Conventions (0-indexed everywhere): ``n`` tokens (a power of two),
``L = log2 n`` levels above the tokens, node ``(l, m)`` is the m-th node of
level ``l`` and covers tokens ``[m*2^l, (m+1)*2^l)``; ``parent(l, m) =
(l+1, m >> 1)``.  Node ids are level-major: ``id(l, m) = 2n - (2n >> l) + m``
(tokens ``0..n-1``, root ``2n-2``).  An edge ``v -> u`` means ``u`` attends to
``v``.

Parity pins: every function in this file is pinned by tests/test_oracle_*.py
(coverage invariants, hand-derived worked example, dense masked attention,
closed forms, finite differences).  Nothing is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

BIDIR = 0
LEFT_ONLY = 1
MODE_PAD = 0
MODE_ALG1 = 2


def log2_exact(n: int) -> int:
    if n < 2 or (n & (n - 1)) != 0:
        raise ValueError("n must be a power of two >= 2")
    return n.bit_length() - 1


def node_id(n: int, l: int, m: int) -> int:
    """Level-major id of node (l, m) in the binary partition tree (Sec. 3.2.1)."""
    return 2 * n - ((2 * n) >> l) + m


def node_level_index(n: int, u: int):
    """Inverse of node_id."""
    l = 0
    base = 0
    width = n
    while u >= base + width:
        base += width
        width >>= 1
        l += 1
    return l, u - base


# ---- relation labels (Sec. 3.4) -------------------------------------------

def rel_self() -> int:
    return 0


def rel_left(L: int, k: int, j: int, o: int) -> int:
    """o-th node (nearest first) to join on the left at level j."""
    return 1 + j * (k + 1) + o


def rel_right(L: int, k: int, j: int, o: int) -> int:
    return 1 + L * (k + 1) + j * (k + 1) + o


def rel_anc(L: int, k: int, j: int) -> int:
    """Token -> its ancestor at level j (1 <= j <= L)."""
    return 1 + 2 * L * (k + 1) + (j - 1)


def num_relations(L: int, k: int) -> int:
    return 1 + 2 * L * (k + 1) + L


# ---- contextual nodes of one token (Sec. 3.2.2, Algorithm 1) ---------------

def right_context(n: int, k: int, i: int, pad: bool):
    """Right contextual nodes of token i in joining order.

    Returns a list of (level, index, offset).  Level l contributes the nodes
    p_l .. p_l+k-1; with the pad rule one more node is taken when the last one
    is a left child, so that the next level starts at a whole parent.
    """
    out = []
    p, l = i + 1, 0
    while p < (n >> l):
        last = p + k - 1
        if pad and last % 2 == 0:
            last += 1
        last = min(last, (n >> l) - 1)
        for m in range(p, last + 1):
            out.append((l, m, m - p))
        nxt = last + 1
        if nxt >= (n >> l):
            break
        p, l = nxt >> 1, l + 1
    return out


def left_context(n: int, k: int, i: int, pad: bool):
    """Mirror image of right_context; offsets count from the nearest node."""
    out = []
    q, l = i - 1, 0
    while q >= 0:
        last = q - k + 1
        if pad and last % 2 == 1:
            last -= 1
        last = max(last, 0)
        for m in range(q, last - 1, -1):
            out.append((l, m, q - m))
        nxt = last - 1
        if nxt < 0:
            break
        q, l = nxt >> 1, l + 1
    return out


class Graph:
    """CSR by destination plus its by-source transpose."""

    def __init__(self, n, k, flags, row_ptr, col, rel):
        self.n, self.k, self.flags = n, k, flags
        self.L = log2_exact(n)
        self.n_nodes = 2 * n - 1
        self.n_rel = num_relations(self.L, k)
        self.row_ptr = row_ptr
        self.col = col
        self.rel = rel
        self.n_edges = int(col.shape[0])
        self._transpose()

    def _transpose(self):
        """By-source lists: for source v the (destination, edge id) pairs,
        destinations ascending (a stable sort of the CSR by source)."""
        N = self.n_nodes
        dst_of_edge = np.repeat(np.arange(N, dtype=np.int64), np.diff(self.row_ptr))
        order = np.argsort(self.col, kind="stable")
        self.t_dst = dst_of_edge[order].astype(np.int32)
        self.t_eid = order.astype(np.int32)
        counts = np.bincount(self.col, minlength=N)
        self.t_ptr = np.zeros(N + 1, dtype=np.int32)
        np.cumsum(counts, out=self.t_ptr[1:])


def enumerate_graph(n: int, k: int, flags: int = 0) -> Graph:
    """All edges of the BPT graph, destination-major, sources ascending by id."""
    L = log2_exact(n)
    if k < 1:
        raise ValueError("k must be >= 1")
    pad = (flags & MODE_ALG1) == 0
    left_only = (flags & LEFT_ONLY) != 0
    rows_col, rows_rel = [], []
    for i in range(n):
        entries = [(i, rel_self())]                       # Algorithm 1: N <- {u}
        for (l, m, o) in left_context(n, k, i, pad):
            entries.append((node_id(n, l, m), rel_left(L, k, l, o)))
        if not left_only:
            for (l, m, o) in right_context(n, k, i, pad):
                entries.append((node_id(n, l, m), rel_right(L, k, l, o)))
        entries.sort()
        rows_col.append([e[0] for e in entries])
        rows_rel.append([e[1] for e in entries])
    for l in range(1, L + 1):                              # affiliated edges
        for m in range(n >> l):
            toks = list(range(m << l, (m + 1) << l))
            rows_col.append(toks)
            rows_rel.append([rel_anc(L, k, l)] * len(toks))
    deg = np.array([len(r) for r in rows_col], dtype=np.int64)
    row_ptr = np.zeros(2 * n, dtype=np.int32)
    np.cumsum(deg, out=row_ptr[1:])
    col = np.fromiter((c for r in rows_col for c in r), dtype=np.int32, count=int(deg.sum()))
    rel = np.fromiter((c for r in rows_rel for c in r), dtype=np.int32, count=int(deg.sum()))
    return Graph(n, k, flags, row_ptr, col, rel)


# ---- attention (Sec. 3.1 GSA, Sec. 3.4 relative positions) -----------------

def attn_fwd(g: Graph, q, k, v, r, scale):
    """q, k, v: [B, N, H, d]; r: [n_rel, d] (shared by heads).  fp64.

    For every node u and head: s_e = scale * q_u . (k_v + r_rel(e)) over the
    predecessors v of u, softmax over them, o_u = sum_e P_e v_v.
    Returns (out [B,N,H,d], lse [B,N,H]).
    """
    q, k, v, r = (np.asarray(a, dtype=np.float64) for a in (q, k, v, r))
    B, N, H, d = q.shape
    out = np.zeros_like(q)
    lse = np.zeros((B, N, H))
    for u in range(N):
        a, b = g.row_ptr[u], g.row_ptr[u + 1]
        if a == b:                                             # a node without predecessors (only in a
            continue                                           # length-masked graph): out = 0, lse = 0
        src, rl = g.col[a:b], g.rel[a:b]
        kk = k[:, src] + r[rl][None, :, None, :]               # [B, deg, H, d]
        s = scale * np.einsum("bhc,behc->bhe", q[:, u], kk)
        mx = s.max(axis=2, keepdims=True)
        p = np.exp(s - mx)
        z = p.sum(axis=2, keepdims=True)
        p = p / z
        out[:, u] = np.einsum("bhe,behc->bhc", p, v[:, src])
        lse[:, u] = (mx + np.log(z))[:, :, 0]
    return out, lse


def attn_bwd(g: Graph, q, k, v, r, scale, d_out, out=None):
    """Gradient of sum(out * d_out) w.r.t. q, k, v, r.  fp64.

    With P the softmax weights of a row: dP_e = d_out_u . v_v,
    dS_e = P_e (dP_e - sum_e' P_e' dP_e'), dq_u = scale sum_e dS_e (k_v + r_e),
    dk_v += scale dS_e q_u, dv_v += P_e d_out_u, dr_rel(e) += scale dS_e q_u
    (summed over batch and heads, the table being shared).

    The row term sum_e' P_e' dP_e' equals d_out_u . out_u.  When ``out`` is
    given (e.g. a forward result that was rounded to bf16 for storage) that
    second form is evaluated with it, which is what a backward pass that
    receives a stored forward output computes; with ``out=None`` the gradient
    is exact.
    """
    q, k, v, r, d_out = (np.asarray(a, dtype=np.float64) for a in (q, k, v, r, d_out))
    B, N, H, d = q.shape
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    dr = np.zeros_like(r)
    for u in range(N):
        a, b = g.row_ptr[u], g.row_ptr[u + 1]
        if a == b:
            continue
        src, rl = g.col[a:b], g.rel[a:b]
        kk = k[:, src] + r[rl][None, :, None, :]
        s = scale * np.einsum("bhc,behc->bhe", q[:, u], kk)
        s -= s.max(axis=2, keepdims=True)
        p = np.exp(s)
        p /= p.sum(axis=2, keepdims=True)
        dp = np.einsum("bhc,behc->bhe", d_out[:, u], v[:, src])
        if out is None:
            row_term = (p * dp).sum(axis=2, keepdims=True)
        else:
            row_term = (d_out[:, u] * np.asarray(out, dtype=np.float64)[:, u]).sum(axis=2)[:, :, None]
        ds = p * (dp - row_term)
        dq[:, u] = scale * np.einsum("bhe,behc->bhc", ds, kk)
        dk[:, src] += scale * np.einsum("bhe,bhc->behc", ds, q[:, u])    # src unique per row
        dv[:, src] += np.einsum("bhe,bhc->behc", p, d_out[:, u])
        np.add.at(dr, rl, scale * np.einsum("bhe,bhc->ec", ds, q[:, u]))
    return dq, dk, dv, dr


# ---- sequences shorter than n (placeholder tokens) ---------------------------
#
# The paper's tree is a perfect binary tree over n = 2^L tokens (Sec. 3.2.1) and says nothing
# about padding.  Reading taken here: a sequence of `length` <= n real tokens occupies the first
# `length` leaves; a node is real when it covers at least one real token.  Edges whose source or
# destination is not real are dropped, everything else (node ids, relation ids, offsets) stays as
# in the full graph.  Rows of nodes that are not real have no predecessors: their output and lse
# are 0 and they receive and send no gradient.

def first_token(n: int, u: int) -> int:
    """First token covered by node id u."""
    l, m = node_level_index(n, u)
    return m << l


def mask_graph(g: Graph, length: int) -> Graph:
    """The graph restricted to the nodes that cover at least one of the first `length` tokens."""
    if not (1 <= length <= g.n):
        raise ValueError("length must be in [1, n]")
    real = np.array([first_token(g.n, u) < length for u in range(g.n_nodes)])
    dst = np.repeat(np.arange(g.n_nodes), np.diff(g.row_ptr))
    keep = real[dst] & real[g.col]
    deg = np.bincount(dst[keep], minlength=g.n_nodes)
    row_ptr = np.zeros(g.n_nodes + 1, dtype=np.int32)
    np.cumsum(deg, out=row_ptr[1:])
    return Graph(g.n, g.k, g.flags, row_ptr, g.col[keep].copy(), g.rel[keep].copy())


def attn_fwd_varlen(g: Graph, q, k, v, r, scale, lengths):
    """attn_fwd with one length per batch entry (see above)."""
    q = np.asarray(q, dtype=np.float64)
    out = np.zeros_like(q)
    lse = np.zeros(q.shape[:3])
    for b, length in enumerate(lengths):
        o, l = attn_fwd(mask_graph(g, int(length)), q[b:b + 1], np.asarray(k)[b:b + 1], np.asarray(v)[b:b + 1], r, scale)
        out[b], lse[b] = o[0], l[0]
    return out, lse


def attn_bwd_varlen(g: Graph, q, k, v, r, scale, d_out, lengths, out=None):
    """attn_bwd with one length per batch entry; dr sums over the batch."""
    q = np.asarray(q, dtype=np.float64)
    dq, dk, dv = np.zeros_like(q), np.zeros_like(q), np.zeros_like(q)
    dr = np.zeros_like(np.asarray(r, dtype=np.float64))
    for b, length in enumerate(lengths):
        ob = None if out is None else np.asarray(out)[b:b + 1]
        a = attn_bwd(mask_graph(g, int(length)), q[b:b + 1], np.asarray(k)[b:b + 1], np.asarray(v)[b:b + 1], r, scale,
                     np.asarray(d_out)[b:b + 1], out=ob)
        dq[b], dk[b], dv[b] = a[0][0], a[1][0], a[2][0]
        dr += a[3]
    return dq, dk, dv, dr


# ---- attention dropout (App. A.1 lists an attention dropout rate p_a for every experiment) --------
#
# The paper does not say how its masks are drawn.  Here every edge weight of every (batch entry,
# head) is kept with probability 1 - p and divided by 1 - p (inverted dropout, applied after the
# softmax, before the product with V), and the mask is a pure function of (seed, batch entry, head,
# destination node, source node) so that the backward pass and another implementation can rebuild
# it: Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as
# 1, 2, 3", SC'11), key = (seed & 0xffffffff, seed >> 32), counter = (destination node, source node,
# batch entry * H + head, PHILOX_TAG), first output word u; the edge is kept iff u >= floor(p * 2^32).

PHILOX_M0, PHILOX_M1 = 0xD2511F53, 0xCD9E8D57
PHILOX_W0, PHILOX_W1 = 0x9E3779B9, 0xBB67AE85
PHILOX_TAG = 0x42505431


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Philox4x32-10 on arrays (or scalars) of 32-bit words; returns the four output words."""
    c0, c1, c2, c3 = (np.asarray(a, dtype=np.uint64) & np.uint64(0xFFFFFFFF) for a in (c0, c1, c2, c3))
    k0, k1 = np.uint64(k0 & 0xFFFFFFFF), np.uint64(k1 & 0xFFFFFFFF)
    mask = np.uint64(0xFFFFFFFF)
    for _ in range(10):
        p0 = np.uint64(PHILOX_M0) * c0          # 64-bit products of 32-bit words
        p1 = np.uint64(PHILOX_M1) * c2
        hi0, lo0, hi1, lo1 = p0 >> np.uint64(32), p0 & mask, p1 >> np.uint64(32), p1 & mask
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + np.uint64(PHILOX_W0)) & mask
        k1 = (k1 + np.uint64(PHILOX_W1)) & mask
    return c0, c1, c2, c3


def dropout_keep(seed: int, p: float, b: int, h: int, H: int, dst, src):
    """Boolean keep mask of the edges src[i] -> dst[i] for batch entry b and head h."""
    thr = np.uint64(min(int(np.floor(float(p) * 4294967296.0)), 0xFFFFFFFF))
    u = philox4x32_10(dst, src, np.full(np.shape(src), b * H + h), np.full(np.shape(src), PHILOX_TAG),
                      seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)[0]
    return u >= thr


def attn_fwd_dropout(g: Graph, q, k, v, r, scale, p_drop, seed):
    """attn_fwd with attention dropout: out_u = sum_e keep_e / (1 - p) P_e v_v; lse is that of the softmax."""
    q, k, v, r = (np.asarray(a, dtype=np.float64) for a in (q, k, v, r))
    B, N, H, d = q.shape
    out = np.zeros_like(q)
    lse = np.zeros((B, N, H))
    for u in range(N):
        a, b_ = g.row_ptr[u], g.row_ptr[u + 1]
        if a == b_:
            continue
        src, rl = g.col[a:b_], g.rel[a:b_]
        kk = k[:, src] + r[rl][None, :, None, :]
        s = scale * np.einsum("bhc,behc->bhe", q[:, u], kk)
        mx = s.max(axis=2, keepdims=True)
        pr = np.exp(s - mx)
        z = pr.sum(axis=2, keepdims=True)
        pr = pr / z
        lse[:, u] = (mx + np.log(z))[:, :, 0]
        for b in range(B):
            for h in range(H):
                keep = dropout_keep(seed, p_drop, b, h, H, np.full(src.shape, u), src)
                w = pr[b, h] * keep / (1.0 - p_drop)
                out[b, u, h] = w @ v[b, src, h]
    return out, lse


def attn_bwd_dropout(g: Graph, q, k, v, r, scale, d_out, p_drop, seed, out=None):
    """Gradient of sum(out * d_out) for attn_fwd_dropout (the mask does not depend on the inputs).
    With W_e = keep_e / (1 - p): dP_e = W_e d_out_u . v_v, dS_e = P_e (dP_e - sum_e' P_e' dP_e'),
    dv_v += W_e P_e d_out_u; dq, dk, dr from dS as without dropout.  The row term equals
    d_out_u . out_u; `out` as in attn_bwd."""
    q, k, v, r, d_out = (np.asarray(a, dtype=np.float64) for a in (q, k, v, r, d_out))
    B, N, H, d = q.shape
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    dr = np.zeros_like(r)
    for u in range(N):
        a, b_ = g.row_ptr[u], g.row_ptr[u + 1]
        if a == b_:
            continue
        src, rl = g.col[a:b_], g.rel[a:b_]
        kk = k[:, src] + r[rl][None, :, None, :]
        s = scale * np.einsum("bhc,behc->bhe", q[:, u], kk)
        s -= s.max(axis=2, keepdims=True)
        pr = np.exp(s)
        pr /= pr.sum(axis=2, keepdims=True)
        w = np.zeros_like(pr)
        for b in range(B):
            for h in range(H):
                w[b, h] = dropout_keep(seed, p_drop, b, h, H, np.full(src.shape, u), src) / (1.0 - p_drop)
        dp = w * np.einsum("bhc,behc->bhe", d_out[:, u], v[:, src])
        if out is None:
            row_term = (pr * dp).sum(axis=2, keepdims=True)
        else:
            row_term = (d_out[:, u] * np.asarray(out, dtype=np.float64)[:, u]).sum(axis=2)[:, :, None]
        ds = pr * (dp - row_term)
        dq[:, u] = scale * np.einsum("bhe,behc->bhc", ds, kk)
        dk[:, src] += scale * np.einsum("bhe,bhc->behc", ds, q[:, u])
        dv[:, src] += np.einsum("bhe,bhc->behc", w * pr, d_out[:, u])
        np.add.at(dr, rl, scale * np.einsum("bhe,bhc->ec", ds, q[:, u]))
    return dq, dk, dv, dr
