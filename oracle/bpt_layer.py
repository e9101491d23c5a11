"""Oracle of one BP-Transformer layer and of a stack of them (arXiv 1911.04070, Sec. 3.3, Algorithm 2).

TEST INFRASTRUCTURE ONLY.  Plain PyTorch CPU operators in float64; the attention is the dense
definition -- scores of all node pairs, the pairs that are not edges of the BPT graph masked out --
so it shares nothing with the edge-by-edge oracle in bpt_oracle.py (which pins it) nor with the
CUDA library.  Gradients come from autograd on these operators.

Layer (Algorithm 2, with the multi-head attention of Sec. 3.1 and the relative positions of Sec. 3.4):
    A   = concat_h softmax_over_predecessors( (H Wq_h) ((H Wk_h) + R[rel])^T / sqrt(d_h) ) (H Wv_h)  Wo
    Z   = LayerNorm(H + A)
    H'  = LayerNorm(Z + W2 relu(W1 Z + b1) + b2)
"""
import numpy as np
import torch


def dense_tables(g, lengths=None, B=1):
    """mask [B, N, N] (True where v -> u is an edge, u the row) and rel [N, N] (relation id, 0 where no edge).
    With lengths, edges touching a node that covers no real token are removed (see bpt_oracle.mask_graph)."""
    N = g.n_nodes
    adj = np.zeros((N, N), dtype=bool)
    rel = np.zeros((N, N), dtype=np.int64)
    for u in range(N):
        a, b = g.row_ptr[u], g.row_ptr[u + 1]
        adj[u, g.col[a:b]] = True
        rel[u, g.col[a:b]] = g.rel[a:b]
    mask = np.broadcast_to(adj, (B, N, N)).copy()
    if lengths is not None:
        first = np.zeros(N, dtype=np.int64)
        base, width, level = 0, g.n, 0
        while width >= 1:
            first[base:base + width] = np.arange(width) << level
            base, width, level = base + width, width >> 1, level + 1
        for b, length in enumerate(lengths):
            real = first < int(length)
            mask[b] &= real[:, None] & real[None, :]
    return torch.from_numpy(mask), torch.from_numpy(rel)


def attention(q, k, v, r, mask, rel, scale):
    """q, k, v: [B, N, H, d]; r: [n_rel, d]; mask [B, N, N]; rel [N, N].  Rows without edges give zeros."""
    bias = torch.einsum("buhc,uvc->bhuv", q, r[rel])                       # q_u . r[rel(u, v)]
    s = scale * (torch.einsum("buhc,bvhc->bhuv", q, k) + bias)
    s = s.masked_fill(~mask[:, None], float("-inf"))
    any_edge = mask.any(dim=2)[:, None, :, None]
    p = torch.softmax(torch.where(any_edge, s, torch.zeros_like(s)), dim=-1)
    p = torch.where(mask[:, None], p, torch.zeros_like(p)) * any_edge
    return torch.einsum("bhuv,bvhc->buhc", p, v)


def out_proj_norm(a, w_o, h, gamma, beta, eps=1e-5):
    """The middle of Algorithm 2 written out in NumPy float64: z = LayerNorm(h + a w_o^T) * gamma + beta over the
    last axis, with the biased variance about the mean (the definition of layer normalisation)."""
    x = np.asarray(h, dtype=np.float64) + np.asarray(a, dtype=np.float64) @ np.asarray(w_o, dtype=np.float64).T
    mean = x.mean(axis=-1, keepdims=True)
    var = ((x - mean) ** 2).mean(axis=-1, keepdims=True)
    return (x - mean) / np.sqrt(var + eps) * np.asarray(gamma, dtype=np.float64) + np.asarray(beta, dtype=np.float64)


def layer_forward(h, w, mask, rel, n_heads):
    """h: [B, N, D]; w: dict of float64 tensors wq, wk, wv, wo [D, D] (applied as x @ w.T), rel_emb [n_rel, D/H],
    ln1_w, ln1_b, ln2_w, ln2_b [D], ff1_w [F, D], ff1_b [F], ff2_w [D, F], ff2_b [D]."""
    B, N, D = h.shape
    dh = D // n_heads
    split = lambda x: x.view(B, N, n_heads, dh)
    a = attention(split(h @ w["wq"].T), split(h @ w["wk"].T), split(h @ w["wv"].T), w["rel_emb"], mask, rel, dh ** -0.5)
    z = torch.nn.functional.layer_norm(h + a.reshape(B, N, D) @ w["wo"].T, (D,), w["ln1_w"], w["ln1_b"])
    f = torch.relu(z @ w["ff1_w"].T + w["ff1_b"]) @ w["ff2_w"].T + w["ff2_b"]
    return torch.nn.functional.layer_norm(z + f, (D,), w["ln2_w"], w["ln2_b"])


def encoder_forward(tokens, layers, g, n_heads, lengths=None, readout="tokens"):
    """Token states [B, n, D] -> stack of layers over all 2n-1 nodes, span nodes starting from zero (Sec. 3.3)."""
    B, n, D = tokens.shape
    mask, rel = dense_tables(g, lengths, B)
    h = torch.cat([tokens, torch.zeros(B, n - 1, D, dtype=tokens.dtype)], dim=1)
    for w in layers:
        h = layer_forward(h, w, mask, rel, n_heads)
    return h[:, :n] if readout == "tokens" else h[:, -1]
