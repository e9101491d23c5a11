"""Pins of the oracle's reading of sequences shorter than n (placeholder tokens).

The paper's tree is a perfect binary tree over n = 2^L leaves and is silent about padding; the
reading (see oracle/bpt_oracle.py) keeps the full graph's node and relation numbering and drops
every edge that touches a node covering no real token.  None of these tests re-uses the masking
code to produce its expectation: they compare with the unmasked oracle on another tree, with
finite differences, or check properties the reading must have."""
import numpy as np
import pytest

from oracle import bpt_oracle as orc
from oracle import ctwin


def _inputs(g, B, H, d, seed):
    rng = np.random.default_rng(seed)
    shape = (B, g.n_nodes, H, d)
    return (rng.standard_normal(shape), rng.standard_normal(shape), rng.standard_normal(shape),
            0.5 * rng.standard_normal((g.n_rel, d)), rng.standard_normal(shape))


@pytest.mark.parametrize("flags", [0, 1, 2])
def test_full_length_is_the_plain_graph(flags):
    g = orc.enumerate_graph(16, 2, flags)
    m = orc.mask_graph(g, 16)
    for name in ("row_ptr", "col", "rel"):
        assert np.array_equal(getattr(g, name), getattr(m, name))


@pytest.mark.parametrize("n,k,flags", [(16, 2, 0), (32, 3, 1), (16, 1, 2), (32, 40, 0)])
def test_half_length_equals_the_half_size_tree(n, k, flags):
    """With length n/2 the real nodes are the first half of every level below the root, and what
    they compute must be what the tree over n/2 tokens computes, once the relation table is
    re-indexed (right and ancestor ids depend on the number of levels)."""
    big, small = orc.enumerate_graph(n, k, flags), orc.enumerate_graph(n // 2, k, flags)
    B, H, d = 2, 2, 4
    q, kk, v, r, go = _inputs(big, B, H, d, 5)
    Lb, Ls, W = big.L, small.L, k + 1
    ids_big, ids_small = [], []
    for l in range(0, Ls + 1):
        for m in range((n // 2) >> l):
            ids_big.append(orc.node_id(n, l, m)); ids_small.append(orc.node_id(n // 2, l, m))
    r_small = np.zeros((small.n_rel, d))
    r_small[0] = r[0]
    for j in range(Ls):
        for o in range(W):
            r_small[orc.rel_left(Ls, k, j, o)] = r[orc.rel_left(Lb, k, j, o)]
            r_small[orc.rel_right(Ls, k, j, o)] = r[orc.rel_right(Lb, k, j, o)]
    for j in range(1, Ls + 1):
        r_small[orc.rel_anc(Ls, k, j)] = r[orc.rel_anc(Lb, k, j)]
    sub = lambda a: np.ascontiguousarray(a[:, ids_big][:, np.argsort(ids_small)])
    lengths = [n // 2] * B
    out, lse = orc.attn_fwd_varlen(big, q, kk, v, r, 0.4, lengths)
    o_s, l_s = orc.attn_fwd(small, sub(q), sub(kk), sub(v), r_small, 0.4)
    assert np.allclose(sub(out), o_s, rtol=1e-11, atol=1e-12)
    assert np.allclose(sub(lse), l_s, rtol=1e-11, atol=1e-12)
    # gradients: the upstream gradient of the big root (real, but without a counterpart) is set to zero
    go = go.copy(); go[:, orc.node_id(n, Lb, 0)] = 0.0
    dq, dk, dv, dr = orc.attn_bwd_varlen(big, q, kk, v, r, 0.4, go, lengths)
    sq, sk, sv, sr = orc.attn_bwd(small, sub(q), sub(kk), sub(v), r_small, 0.4, sub(go))
    for a, b in ((dq, sq), (dk, sk), (dv, sv)):
        assert np.allclose(sub(a), b, rtol=1e-10, atol=1e-12)
    assert np.allclose(dr[0], sr[0], rtol=1e-10, atol=1e-12)
    for j in range(Ls):
        for o in range(W):
            assert np.allclose(dr[orc.rel_left(Lb, k, j, o)], sr[orc.rel_left(Ls, k, j, o)], rtol=1e-10, atol=1e-12)
            assert np.allclose(dr[orc.rel_right(Lb, k, j, o)], sr[orc.rel_right(Ls, k, j, o)], rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("n,k,flags,length", [(16, 2, 0, 5), (32, 3, 1, 21), (16, 4, 0, 1), (32, 2, 2, 31)])
def test_placeholders_neither_influence_nor_receive(n, k, flags, length):
    g = orc.enumerate_graph(n, k, flags)
    B, H, d = 1, 2, 4
    q, kk, v, r, go = _inputs(g, B, H, d, 9)
    real = np.array([orc.first_token(n, u) < length for u in range(g.n_nodes)])
    assert real[: length].all() and not real[length:n].any() and real[g.n_nodes - 1]
    out, lse = orc.attn_fwd_varlen(g, q, kk, v, r, 0.3, [length])
    grads = orc.attn_bwd_varlen(g, q, kk, v, r, 0.3, go, [length])
    assert (out[:, ~real] == 0).all() and (lse[:, ~real] == 0).all()
    for a in grads[:3]:
        assert (a[:, ~real] == 0).all()
    rng = np.random.default_rng(1)
    q2, k2, v2, go2 = (a.copy() for a in (q, kk, v, go))
    for a in (q2, k2, v2, go2):
        a[:, ~real] = rng.standard_normal(a[:, ~real].shape) * 50.0
    out2, lse2 = orc.attn_fwd_varlen(g, q2, k2, v2, r, 0.3, [length])
    grads2 = orc.attn_bwd_varlen(g, q2, k2, v2, r, 0.3, go2, [length])
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)
    for a, b in zip(grads, grads2):
        assert np.array_equal(a, b)
    # every real token still reaches every other real token within two hops (Sec. 3.2.2), left-only: earlier ones
    m = orc.mask_graph(g, length)
    preds = [set(m.col[m.row_ptr[u]:m.row_ptr[u + 1]].tolist()) for u in range(g.n_nodes)]
    for b in range(length):
        for a in range(length):
            if a == b or ((flags & 1) and a > b):
                continue
            assert a in preds[b] or any(a in preds[s] for s in preds[b] if s >= n), (a, b)


def test_gradient_of_a_short_sequence_by_finite_differences():
    g = orc.enumerate_graph(8, 1, 0)
    B, H, d = 1, 1, 3
    q, kk, v, r, go = _inputs(g, B, H, d, 3)
    lengths = [5]
    f = lambda q_, k_, v_, r_: float((orc.attn_fwd_varlen(g, q_, k_, v_, r_, 0.7, lengths)[0] * go).sum())
    grads = orc.attn_bwd_varlen(g, q, kk, v, r, 0.7, go, lengths)
    eps = 1e-6
    rng = np.random.default_rng(0)
    for which, arr in enumerate((q, kk, v, r)):
        for _ in range(12):
            idx = tuple(rng.integers(0, s) for s in arr.shape)
            args = [q, kk, v, r]
            hi, lo = arr.copy(), arr.copy()
            hi[idx] += eps; lo[idx] -= eps
            args[which] = hi; fh = f(*args)
            args[which] = lo; fl = f(*args)
            assert abs((fh - fl) / (2 * eps) - grads[which][idx]) < 1e-6, (which, idx)


def test_c_twin_agrees_on_short_sequences():
    n, k, flags = 64, 3, 0
    g, cg = orc.enumerate_graph(n, k, flags), ctwin.CGraph(n, k, flags)
    B, H, d = 3, 2, 8
    q, kk, v, r, go = _inputs(g, B, H, d, 11)
    lengths = [64, 37, 1]
    o1, l1 = orc.attn_fwd_varlen(g, q, kk, v, r, 0.35, lengths)
    o2, l2 = ctwin.attn_fwd_varlen(cg, q, kk, v, r, 0.35, lengths)
    assert np.allclose(o1, o2, rtol=1e-12, atol=1e-13) and np.allclose(l1, l2, rtol=1e-12, atol=1e-13)
    g1 = orc.attn_bwd_varlen(g, q, kk, v, r, 0.35, go, lengths)
    g2 = ctwin.attn_bwd_varlen(cg, q, kk, v, r, 0.35, go, lengths)
    for a, b in zip(g1, g2):
        assert np.allclose(a, b, rtol=1e-11, atol=1e-12)
