"""Pins for the oracle's attention forward/backward (Sec. 3.1 GSA equations,
Sec. 3.4 equation with relative positions).  References used here are written
independently of the oracle: dense masked softmax attention (textbook),
closed forms, and central finite differences."""
import numpy as np
import pytest

from oracle import bpt_oracle as orc


def _rand(n, k, flags, B, H, d, seed, std_r=0.3):
    g = orc.enumerate_graph(n, k, flags)
    rng = np.random.default_rng(seed)
    q, kk, v, go = (rng.standard_normal((B, g.n_nodes, H, d)) for _ in range(4))
    r = rng.standard_normal((g.n_rel, d)) * std_r
    return g, q, kk, v, r, go


def _dense_reference(g, q, k, v, r, scale):
    """Masked dense attention over all N nodes: S = scale (Q K^T + bias) with
    bias[u, v] = q_u . r_{v,u}, -inf outside the adjacency."""
    B, N, H, d = q.shape
    adj = np.zeros((N, N), dtype=bool)
    relm = np.zeros((N, N), dtype=np.int64)
    for u in range(N):
        for e in range(g.row_ptr[u], g.row_ptr[u + 1]):
            adj[u, g.col[e]] = True
            relm[u, g.col[e]] = g.rel[e]
    out = np.zeros_like(q)
    lse = np.zeros((B, N, H))
    for b in range(B):
        for h in range(H):
            Q, K, V = q[b, :, h], k[b, :, h], v[b, :, h]
            S = Q @ K.T
            bias = (Q @ r.T)[np.arange(N)[:, None], relm]          # [N, N]
            S = scale * (S + bias)
            S[~adj] = -np.inf
            m = S.max(axis=1, keepdims=True)
            P = np.exp(S - m)
            z = P.sum(axis=1, keepdims=True)
            out[b, :, h] = (P / z) @ V
            lse[b, :, h] = (m + np.log(z))[:, 0]
    return out, lse


@pytest.mark.parametrize("n,k,flags", [(8, 1, 0), (16, 2, 0), (32, 3, 1), (64, 4, 0), (16, 2, 2), (16, 20, 0)])
def test_forward_equals_dense_masked_attention(n, k, flags):
    g, q, kk, v, r, _ = _rand(n, k, flags, B=2, H=2, d=8, seed=n + k)
    scale = 1 / np.sqrt(8)
    out, lse = orc.attn_fwd(g, q, kk, v, r, scale)
    ref_out, ref_lse = _dense_reference(g, q, kk, v, r, scale)
    np.testing.assert_allclose(out, ref_out, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(lse, ref_lse, rtol=1e-12, atol=1e-12)


def test_constant_values_give_constant_output():
    g, q, kk, v, r, _ = _rand(32, 2, 0, 1, 2, 4, 1)
    v[:] = np.array([1.0, -2.0, 3.0, 0.5])
    out, _ = orc.attn_fwd(g, q, kk, v, r, 0.5)
    np.testing.assert_allclose(out, np.broadcast_to(v[0, 0, 0], out.shape), rtol=1e-13)


def test_zero_queries_average_the_predecessors():
    """Q = 0 makes every score 0: a span's output is the mean of its tokens
    (Sec. 3.3: a span's predecessors are exactly its contained tokens)."""
    n = 16
    g, q, kk, v, r, _ = _rand(n, 2, 0, 1, 1, 4, 2)
    q[:] = 0
    out, lse = orc.attn_fwd(g, q, kk, v, r, 1.0)
    for l in range(1, g.L + 1):
        for m in range(n >> l):
            u = orc.node_id(n, l, m)
            np.testing.assert_allclose(out[0, u, 0], v[0, m << l:(m + 1) << l, 0].mean(axis=0), rtol=1e-13)
            assert abs(lse[0, u, 0] - np.log(2.0 ** l)) < 1e-13
    for i in range(n):
        cols = g.col[g.row_ptr[i]:g.row_ptr[i + 1]]
        np.testing.assert_allclose(out[0, i, 0], v[0, cols, 0].mean(axis=0), rtol=1e-13)


def test_large_k_is_vanilla_attention_with_relative_positions():
    """Sec. 3.4 closing remark: k >= length degenerates to the vanilla
    Transformer with (Shaw-style) relative position terms on the keys."""
    n, k, d = 16, 16, 8
    g, q, kk, v, r, _ = _rand(n, k, 0, 1, 2, d, 3)
    scale = 1 / np.sqrt(d)
    out, _ = orc.attn_fwd(g, q, kk, v, r, scale)
    L = g.L
    # relative embedding as a function of signed distance j - i only
    a = np.zeros((2 * n - 1, d))
    for dist in range(-(n - 1), n):
        if dist == 0:
            a[dist + n - 1] = r[0]
        elif dist < 0:
            a[dist + n - 1] = r[1 + (-dist - 1)]                     # left, level 0, offset |dist|-1
        else:
            a[dist + n - 1] = r[1 + L * (k + 1) + (dist - 1)]        # right, level 0
    for h in range(2):
        Q, K, V = q[0, :n, h], kk[0, :n, h], v[0, :n, h]
        S = np.array([[Q[i] @ (K[j] + a[j - i + n - 1]) for j in range(n)] for i in range(n)]) * scale
        P = np.exp(S - S.max(1, keepdims=True))
        P /= P.sum(1, keepdims=True)
        np.testing.assert_allclose(out[0, :n, h], P @ V, rtol=1e-12, atol=1e-13)


def test_output_ignores_ancestor_relation_embedding():
    """All edges into a span carry the same r^anc_j: a softmax shift."""
    g, q, kk, v, r, _ = _rand(16, 2, 0, 1, 2, 4, 4)
    out0, lse0 = orc.attn_fwd(g, q, kk, v, r, 0.5)
    r2 = r.copy()
    r2[orc.rel_anc(g.L, 2, 1):] += 7.0
    out1, _ = orc.attn_fwd(g, q, kk, v, r2, 0.5)
    np.testing.assert_allclose(out0, out1, rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("n,k,flags,H", [(8, 1, 0, 1), (16, 2, 0, 2), (16, 3, 1, 2), (8, 2, 2, 1)])
def test_backward_matches_finite_differences(n, k, flags, H):
    g, q, kk, v, r, go = _rand(n, k, flags, B=2, H=H, d=4, seed=10 + n + k)
    scale = 0.5
    dq, dk, dv, dr = orc.attn_bwd(g, q, kk, v, r, scale, go)

    def loss(q_, k_, v_, r_):
        return float((orc.attn_fwd(g, q_, k_, v_, r_, scale)[0] * go).sum())

    rng = np.random.default_rng(0)
    eps = 1e-6
    args = [q, kk, v, r]
    grads = [dq, dk, dv, dr]
    for which in range(4):
        x = args[which]
        flat_idx = rng.choice(x.size, size=min(40, x.size), replace=False)
        for fi in flat_idx:
            idx = np.unravel_index(fi, x.shape)
            old = x[idx]
            x[idx] = old + eps
            lp = loss(*args)
            x[idx] = old - eps
            lm = loss(*args)
            x[idx] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - grads[which][idx]) <= 1e-6 * max(1.0, abs(fd)), (which, idx, fd, grads[which][idx])


def test_backward_structure():
    g, q, kk, v, r, go = _rand(16, 2, 0, B=1, H=2, d=4, seed=5)
    dq, dk, dv, dr = orc.attn_bwd(g, q, kk, v, r, 0.5, go)
    L = g.L
    # gradient of the ancestor relations vanishes (softmax shift invariance)
    assert np.abs(dr[orc.rel_anc(L, 2, 1):]).max() <= 1e-12 * np.abs(dr).max()
    # rows of the table no edge uses get no gradient
    used = np.zeros(g.n_rel, dtype=bool)
    used[g.rel] = True
    assert (dr[~used] == 0).all()
    # R is shared over batch and heads: doubling the batch with the same data doubles dR only
    q2, k2, v2, go2 = (np.concatenate([a, a], axis=0) for a in (q, kk, v, go))
    dq2, dk2, dv2, dr2 = orc.attn_bwd(g, q2, k2, v2, r, 0.5, go2)
    np.testing.assert_allclose(dr2, 2 * dr, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(dq2[1], dq[0], rtol=1e-12)
    np.testing.assert_allclose(dk2[0], dk[0], rtol=1e-12)
    np.testing.assert_allclose(dv2[1], dv[0], rtol=1e-12)


def test_backward_row_term_from_stored_output():
    """sum_e P_e dP_e = d_out_u . out_u: passing the exact forward output reproduces the
    exact gradient; passing a perturbed one changes dq, dk, d_rel but never dv."""
    g, q, kk, v, r, go = _rand(16, 2, 0, B=2, H=2, d=4, seed=6)
    out, _ = orc.attn_fwd(g, q, kk, v, r, 0.5)
    exact = orc.attn_bwd(g, q, kk, v, r, 0.5, go)
    same = orc.attn_bwd(g, q, kk, v, r, 0.5, go, out=out)
    for a, b in zip(exact, same):
        np.testing.assert_allclose(b, a, rtol=1e-11, atol=1e-13)
    pert = orc.attn_bwd(g, q, kk, v, r, 0.5, go, out=out * 1.01)
    np.testing.assert_allclose(pert[2], exact[2], rtol=1e-12, atol=1e-14)
    assert np.abs(pert[0] - exact[0]).max() > 1e-6
