"""BP-Transformer layers on top of the graph self-attention library (arXiv 1911.04070, Sec. 3.3,
Algorithm 2): PyTorch modules whose attention runs in libbpt.so.

Only the graph self-attention is this package's own code; the projections, the feed-forward block
and the layer normalisation are plain PyTorch operators around it, so that the operator can be
dropped into a model and trained.  Nothing here falls back to another attention implementation.
"""
from __future__ import annotations

import math

import torch
from torch import nn

from . import binding


# Inference (no gradient, bfloat16, model width 128 / 256 / 512): the output projection, the residual and the first
# layer normalisation of a layer run in the library's fused kernel (bpt_out_proj_norm) instead of three operators.
FUSE_OUT_PROJ_NORM = True


class _GraphSelfAttention(torch.autograd.Function):
    """out = GSA(q, k, v, rel_emb) over the BPT graph; backward through bpt_attn_bwd."""

    @staticmethod
    def forward(ctx, q, k, v, rel_emb, g, scale, lengths, dropout_p, dropout_seed):
        q, k, v, rel_emb = q.contiguous(), k.contiguous(), v.contiguous(), rel_emb.contiguous()
        out, lse = binding.bpt_attn_fwd(g, q, k, v, rel_emb, scale, lengths=lengths, dropout_p=dropout_p,
                                        dropout_seed=dropout_seed)
        if binding.CHECK_DEVICE_STATUS and binding.bpt_check(getattr(out, "_bpt_workspace", None)):
            raise RuntimeError("graph self-attention forward: a device-side wait timed out, results are invalid")
        ctx.save_for_backward(q, k, v, rel_emb, out, lse)
        ctx.g, ctx.scale, ctx.lengths, ctx.drop = g, scale, lengths, (dropout_p, dropout_seed)
        return out

    @staticmethod
    def backward(ctx, d_out):
        q, k, v, rel_emb, out, lse = ctx.saved_tensors
        dq, dk, dv, d_rel = binding.bpt_attn_bwd(ctx.g, q, k, v, rel_emb, ctx.scale, out, lse, d_out.contiguous(),
                                                 lengths=ctx.lengths, dropout_p=ctx.drop[0], dropout_seed=ctx.drop[1])
        if binding.CHECK_DEVICE_STATUS and binding.bpt_check(getattr(dq, "_bpt_workspace", None)):
            raise RuntimeError("graph self-attention backward: a device-side wait timed out, results are invalid")
        return dq, dk, dv, d_rel.to(rel_emb.dtype), None, None, None, None, None


def graph_self_attention(g: binding.Graph, q, k, v, rel_emb, scale=None, lengths=None, dropout_p=0.0, dropout_seed=0):
    """Differentiable graph self-attention with tree relative positions (Sec. 3.1, 3.4).

    q, k, v: [B, 2n-1, H, d] (float32 or bfloat16, on the graph's device); rel_emb: [n_rel, d], shared
    by the heads; lengths: optional int32 [B]; dropout_p / dropout_seed: attention dropout (the mask is a
    function of the seed, so the backward pass rebuilds it).  Returns [B, 2n-1, H, d]."""
    scale = 1.0 / math.sqrt(q.shape[-1]) if scale is None else float(scale)
    return _GraphSelfAttention.apply(q, k, v, rel_emb, g, scale, lengths, float(dropout_p), int(dropout_seed))


class BPTLayer(nn.Module):
    """One layer of Algorithm 2:  Z = norm(H + GSA(H)),  H' = norm(Z + FFN(Z)).

    H holds the states of all 2n-1 nodes.  The relation embeddings are a parameter of the layer
    (Sec. 3.4: not shared between layers, shared between the heads)."""

    def __init__(self, g: binding.Graph, d_model: int, n_heads: int, d_ff: int, rel_std: float = 0.02,
                 attn_dropout: float = 0.0):
        super().__init__()
        self.attn_dropout = attn_dropout
        if d_model % n_heads:
            raise ValueError("d_model must be a multiple of n_heads")
        self.g, self.h, self.dh = g, n_heads, d_model // n_heads
        self.wq, self.wk, self.wv, self.wo = (nn.Linear(d_model, d_model, bias=False) for _ in range(4))
        self.rel_emb = nn.Parameter(torch.randn(g.n_rel, self.dh) * rel_std)
        self.norm1, self.norm2 = nn.LayerNorm(d_model), nn.LayerNorm(d_model)
        self.ff1, self.ff2 = nn.Linear(d_model, d_ff), nn.Linear(d_ff, d_model)

    def forward(self, h, lengths=None):
        B, N, D = h.shape
        split = lambda x: x.view(B, N, self.h, self.dh)
        p_drop = self.attn_dropout if self.training else 0.0
        seed = int(torch.randint(0, 2 ** 62, (1,)).item()) if p_drop else 0   # a fresh mask per call, from torch's CPU generator
        a = graph_self_attention(self.g, split(self.wq(h)), split(self.wk(h)), split(self.wv(h)),
                                 self.rel_emb.to(h.dtype), lengths=lengths, dropout_p=p_drop, dropout_seed=seed)
        if (FUSE_OUT_PROJ_NORM and not torch.is_grad_enabled() and h.dtype == torch.bfloat16 and D in (128, 256, 512)
                and self.wo.weight.dtype == torch.bfloat16):
            z = binding.bpt_out_proj_norm(a.reshape(B, N, D), self.wo.weight.contiguous(), h.contiguous(), self.norm1.weight.float(),
                                          self.norm1.bias.float(), self.norm1.eps)
        else:
            z = self.norm1(h + self.wo(a.reshape(B, N, D)))
        return self.norm2(z + self.ff2(torch.relu(self.ff1(z))))


class BPTEncoder(nn.Module):
    """A stack of BPT layers over one sequence length n (a power of two).

    Token nodes start from the given token states, span nodes from zero, and all nodes are updated
    together in every layer (Sec. 3.3).  `readout`: "tokens" returns the token states [B, n, D]
    (language modelling, translation), "root" the root node's state [B, D] (classification)."""

    def __init__(self, n: int, k: int, d_model: int, n_heads: int, d_ff: int, n_layers: int, left_only: bool = False,
                 device="cuda", attn_dropout: float = 0.0):
        super().__init__()
        self.n = n
        self.g = binding.bpt_build_graph(n, k, binding.BPT_LEFT_ONLY if left_only else 0, device=device)
        self.layers = nn.ModuleList(BPTLayer(self.g, d_model, n_heads, d_ff, attn_dropout=attn_dropout) for _ in range(n_layers))

    def forward(self, tokens, lengths=None, readout: str = "tokens"):
        B, n, D = tokens.shape
        if n != self.n:
            raise ValueError("expected %d token states per sequence, got %d" % (self.n, n))
        h = torch.cat([tokens, tokens.new_zeros(B, n - 1, D)], dim=1)
        for layer in self.layers:
            h = layer(h, lengths)
        if readout == "tokens":
            return h[:, :n]
        if readout == "root":
            return h[:, -1]
        raise ValueError("readout must be 'tokens' or 'root'")


class BPTDecoder:
    """Step-by-step evaluation of a left-only BPTEncoder with cached per-layer state, for autoregressive use
    (Sec. 4.2 trains BPT as a language model; generation feeds it one token at a time).

    When token i arrives, the only nodes whose state changes in any layer are token i and its log2(n)
    ancestors: every other token lies to its left and attends only nodes that lie wholly to its own left.
    The decoder therefore keeps, per layer, the input states of all 2n-1 nodes and their key / value
    rows, recomputes those log2(n) + 1 rows per layer with `bpt_attn_fwd_rows` and lengths = i + 1 (the
    ancestors then attend exactly the tokens seen so far), and returns the last layer's state of token i.
    A span is complete once its last token has arrived; from then on its cached state is the one a full
    forward pass over the finished sequence computes, so the token outputs of the steps equal the token
    rows of `BPTEncoder.forward` on the whole sequence."""

    def __init__(self, enc: BPTEncoder, batch: int, dtype=torch.float32):
        g = enc.g
        if not (g.dims.flags & binding.BPT_LEFT_ONLY):
            raise ValueError("step-by-step decoding needs the left-only graph")
        self.enc, self.g, self.n, self.batch = enc, g, enc.n, batch
        first = enc.layers[0]
        dev = first.rel_emb.device
        D, H, dh, N = first.h * first.dh, first.h, first.dh, g.n_nodes
        self.L = g.dims.n_levels
        self.h = [torch.zeros(batch, N, D, device=dev, dtype=dtype) for _ in range(len(enc.layers) + 1)]
        heads = lambda: torch.zeros(batch, N, H, dh, device=dev, dtype=dtype)
        self.q, self.k, self.v, self.a = ([heads() for _ in enc.layers] for _ in range(4))
        self.lse = torch.zeros(batch, N, H, device=dev, dtype=torch.float32)
        self.pos = 0

    def rows_of_step(self, i: int):
        """Token i and its ancestors, finest first."""
        n = self.n
        return [i] + [2 * n - ((2 * n) >> j) + (i >> j) for j in range(1, self.L + 1)]

    @torch.no_grad()
    def step(self, token_state):
        """token_state: [batch, D], the input state of the next token.  Returns its output state [batch, D]."""
        i = self.pos
        if i >= self.n:
            raise ValueError("the sequence is full (n = %d)" % self.n)
        rows = self.rows_of_step(i)
        B, R = self.batch, len(rows)
        dev = self.h[0].device
        idx = torch.tensor(rows, device=dev)
        rows_t = torch.tensor([rows] * B, dtype=torch.int32, device=dev)
        lens = torch.full((B,), i + 1, dtype=torch.int32, device=dev)
        self.h[0][:, i] = token_state.to(self.h[0].dtype)
        for li, layer in enumerate(self.enc.layers):
            hr = self.h[li][:, idx]                                     # [B, R, D]; span rows of layer 0 are zero
            split = lambda x: x.view(B, R, layer.h, layer.dh)
            self.q[li][:, idx] = split(layer.wq(hr))
            self.k[li][:, idx] = split(layer.wk(hr))
            self.v[li][:, idx] = split(layer.wv(hr))
            binding.bpt_attn_fwd_rows(self.g, self.q[li], self.k[li], self.v[li], layer.rel_emb.to(hr.dtype).contiguous(),
                                      1.0 / math.sqrt(layer.dh), rows_t, self.a[li], self.lse, lengths=lens)
            a = self.a[li][:, idx].reshape(B, R, -1)
            z = layer.norm1(hr + layer.wo(a))
            self.h[li + 1][:, idx] = layer.norm2(z + layer.ff2(torch.relu(layer.ff1(z))))
        self.pos += 1
        return self.h[-1][:, i]
