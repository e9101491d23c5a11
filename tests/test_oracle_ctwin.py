"""The plain-C twin of the oracle must agree with the pinned NumPy oracle."""
import numpy as np
import pytest

from oracle import bpt_oracle as orc
from oracle import ctwin


@pytest.mark.parametrize("n,k,flags", [(2, 1, 0), (8, 1, 0), (8, 9, 0), (64, 3, 1), (64, 4, 2), (128, 5, 3), (256, 4, 0), (512, 64, 1)])
def test_graph(n, k, flags):
    g, c = orc.enumerate_graph(n, k, flags), ctwin.CGraph(n, k, flags)
    assert g.n_edges == c.n_edges and g.n_rel == c.n_rel
    for name in ("row_ptr", "col", "rel", "t_ptr", "t_dst", "t_eid"):
        assert np.array_equal(getattr(g, name), getattr(c, name)), name


def test_mid_size_edge_counts():
    # E = E_ctx + n + n log2 n; E_aff and E_self are fixed by Sec. 3.2.2, so this pins E_ctx of the twin
    # against the NumPy enumeration on a mid-sized case and the twin's own count routine elsewhere.
    c = ctwin.CGraph(2048, 8, 0)
    g = orc.enumerate_graph(2048, 8, 0)
    assert c.n_edges == g.n_edges == int(g.row_ptr[-1])


@pytest.mark.parametrize("n,k,flags", [(16, 2, 0), (64, 3, 1), (32, 40, 0)])
def test_attention(n, k, flags):
    g = orc.enumerate_graph(n, k, flags)
    rng = np.random.default_rng(7)
    B, H, d = 3, 2, 8
    q, kk, v, go = (rng.standard_normal((B, g.n_nodes, H, d)) for _ in range(4))
    r = rng.standard_normal((g.n_rel, d)) * 0.3
    out, lse = orc.attn_fwd(g, q, kk, v, r, 0.3)
    cout, clse = ctwin.attn_fwd(g, q, kk, v, r, 0.3)
    np.testing.assert_allclose(cout, out, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(clse, lse, rtol=1e-12, atol=1e-13)
    grads = orc.attn_bwd(g, q, kk, v, r, 0.3, go)
    cgrads = ctwin.attn_bwd(g, q, kk, v, r, 0.3, go)
    for a, b in zip(grads, cgrads):
        np.testing.assert_allclose(b, a, rtol=1e-11, atol=1e-12)
    rounded = np.round(out * 64) / 64
    for a, b in zip(orc.attn_bwd(g, q, kk, v, r, 0.3, go, out=rounded), ctwin.attn_bwd(g, q, kk, v, r, 0.3, go, out=rounded)):
        np.testing.assert_allclose(b, a, rtol=1e-11, atol=1e-12)
    # batch slicing: entries outside [b0, b1) untouched, dr sums the slice only
    part = ctwin.attn_bwd(g, q, kk, v, r, 0.3, go, b0=1, b1=2)
    one = orc.attn_bwd(g, q[1:2], kk[1:2], v[1:2], r, 0.3, go[1:2])
    np.testing.assert_allclose(part[3], one[3], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(part[0][1], one[0][0], rtol=1e-11, atol=1e-12)
    assert (part[0][0] == 0).all() and (part[1][2] == 0).all()
