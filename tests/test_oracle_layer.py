"""Pins of the layer oracle: its dense masked attention against the edge-by-edge oracle (two
independent writings of the Sec. 3.4 equation), with and without lengths, and the layer against a
hand-assembled computation from NumPy pieces."""
import numpy as np
import torch

from oracle import bpt_layer, bpt_oracle as orc


def test_dense_attention_equals_edge_by_edge_oracle():
    g = orc.enumerate_graph(16, 2, 0)
    rng = np.random.default_rng(0)
    B, H, d = 2, 2, 4
    q, k, v = (rng.standard_normal((B, g.n_nodes, H, d)) for _ in range(3))
    r = rng.standard_normal((g.n_rel, d))
    for lengths in (None, [11, 3]):
        mask, rel = bpt_layer.dense_tables(g, lengths, B)
        got = bpt_layer.attention(*(torch.from_numpy(a) for a in (q, k, v, r)), mask, rel, 0.3).numpy()
        want = orc.attn_fwd(g, q, k, v, r, 0.3)[0] if lengths is None else orc.attn_fwd_varlen(g, q, k, v, r, 0.3, lengths)[0]
        assert np.allclose(got, want, rtol=1e-11, atol=1e-12)


def test_layer_matches_numpy_assembly():
    g = orc.enumerate_graph(8, 1, 1)
    rng = np.random.default_rng(1)
    B, H, D, F = 1, 2, 8, 12
    w = {"wq": (D, D), "wk": (D, D), "wv": (D, D), "wo": (D, D), "rel_emb": (g.n_rel, D // H), "ln1_w": (D,), "ln1_b": (D,),
         "ln2_w": (D,), "ln2_b": (D,), "ff1_w": (F, D), "ff1_b": (F,), "ff2_w": (D, F), "ff2_b": (D,)}
    w = {a: rng.standard_normal(s) * 0.5 for a, s in w.items()}
    h = rng.standard_normal((B, g.n_nodes, D))
    mask, rel = bpt_layer.dense_tables(g, None, B)
    got = bpt_layer.layer_forward(torch.from_numpy(h), {a: torch.from_numpy(b) for a, b in w.items()}, mask, rel, H).numpy()

    def ln(x, gam, bet):
        mu = x.mean(-1, keepdims=True); var = ((x - mu) ** 2).mean(-1, keepdims=True)
        return (x - mu) / np.sqrt(var + 1e-5) * gam + bet
    sp = lambda x: x.reshape(B, g.n_nodes, H, D // H)
    a = orc.attn_fwd(g, sp(h @ w["wq"].T), sp(h @ w["wk"].T), sp(h @ w["wv"].T), w["rel_emb"], (D // H) ** -0.5)[0]
    z = ln(h + a.reshape(B, g.n_nodes, D) @ w["wo"].T, w["ln1_w"], w["ln1_b"])
    want = ln(z + np.maximum(z @ w["ff1_w"].T + w["ff1_b"], 0) @ w["ff2_w"].T + w["ff2_b"], w["ln2_w"], w["ln2_b"])
    assert np.allclose(got, want, rtol=1e-10, atol=1e-11)


def test_out_proj_norm_pins():
    """The NumPy statement of z = LayerNorm(h + a w_o^T) against what fixes it: PyTorch's own float64 operators
    (a library routine written independently of it), the normalisation's invariants, and two special cases."""
    import numpy as np
    import torch
    from oracle import bpt_layer
    rng = np.random.default_rng(0)
    rows, D = 7, 16
    a, h = rng.normal(size=(rows, D)), rng.normal(size=(rows, D))
    w = rng.normal(size=(D, D)) / 4
    gamma, beta = rng.normal(size=D), rng.normal(size=D)
    z = bpt_layer.out_proj_norm(a, w, h, gamma, beta, 1e-5)
    lin = torch.nn.functional.linear(torch.from_numpy(a), torch.from_numpy(w))             # a @ w.T
    want = torch.nn.functional.layer_norm(torch.from_numpy(h) + lin, (D,), torch.from_numpy(gamma), torch.from_numpy(beta), 1e-5)
    assert np.abs(z - want.numpy()).max() < 1e-12
    plain = bpt_layer.out_proj_norm(a, w, h, np.ones(D), np.zeros(D), 1e-12)
    assert np.abs(plain.mean(axis=-1)).max() < 1e-12 and np.abs(plain.var(axis=-1) - 1).max() < 1e-9
    # w_o = 0: the normalised residual; a transposed weight would change the next one
    assert np.abs(bpt_layer.out_proj_norm(a, np.zeros((D, D)), h, gamma, beta) - bpt_layer.out_proj_norm(0 * a, w, h, gamma, beta)).max() < 1e-12
    e = np.zeros((D, D)); e[3, 5] = 1.0          # output channel 3 reads input channel 5
    x = h.copy(); x[:, 3] += a[:, 5]
    m, v = x.mean(-1, keepdims=True), x.var(-1, keepdims=True)
    assert np.abs(bpt_layer.out_proj_norm(a, e, h, np.ones(D), np.zeros(D), 1e-5) - (x - m) / np.sqrt(v + 1e-5)).max() < 1e-12
    # shift invariance of the normalisation: adding a constant to every channel of h changes nothing
    assert np.abs(bpt_layer.out_proj_norm(a, w, h + 3.0, gamma, beta) - z).max() < 1e-9
