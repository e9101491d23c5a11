"""Seeded synthetic inputs for BPT graph self-attention.

This module only draws random tensors of a given shape; it contains none of
the method's arithmetic (no graph, no attention), so both the CUDA binding's
callers and the CPU oracle's callers may use it without the two sharing code.

The workloads stand in for the paper's text-classification, document
translation and character-level language-modelling inputs (Sec. 4): only the
shapes matter for the operator, so values are i.i.d. normal.
"""
from __future__ import annotations

import numpy as np


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16-representable value (ties to even);
    the result is still stored as fp32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) & np.uint32(0xFFFF0000)).view(np.float32)


def make_inputs(B: int, n_nodes: int, H: int, d: int, n_rel: int, *, seed: int,
                std_qkv: float, std_rel: float = 0.02, bf16: bool, with_grad: bool = True):
    """Returns a dict of fp32 arrays q, k, v [B, n_nodes, H, d], rel_emb
    [n_rel, d] and (optionally) d_out [B, n_nodes, H, d] ~ N(0, 1).

    With ``bf16`` every value is already rounded to bf16, so converting to
    torch.bfloat16 (GPU side) or to float64 (oracle side) is exact.
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    shape = (B, n_nodes, H, d)
    out = {}
    for name in ("q", "k", "v"):
        out[name] = rng.standard_normal(shape, dtype=np.float32) * np.float32(std_qkv)
    out["rel_emb"] = rng.standard_normal((n_rel, d), dtype=np.float32) * np.float32(std_rel)
    if with_grad:
        out["d_out"] = rng.standard_normal(shape, dtype=np.float32)
    if bf16:
        out = {name: round_to_bf16(a) for name, a in out.items()}
    return out


# The five workloads of the benchmark definition.  ``flags`` bit 0 = left-only.
CONFIGS = {
    "cfg1_tiny": dict(B=1, n=256, k=4, flags=0, H=2, d=32, bf16=False, seed=0, std_qkv=1.0, backward=True),
    "cfg2_cls": dict(B=32, n=512, k=4, flags=0, H=8, d=64, bf16=True, seed=2, std_qkv=0.125, backward=False),
    "cfg3_doc_mt": dict(B=16, n=2048, k=8, flags=0, H=8, d=64, bf16=True, seed=3, std_qkv=0.125, backward=True),
    "cfg4_char_lm": dict(B=4, n=8192, k=64, flags=1, H=8, d=64, bf16=True, seed=4, std_qkv=0.125, backward=True),
}


def sweep_configs():
    """Scaling sweep: n x k grid, bidirectional, batch * n = 262144 tokens."""
    out = {}
    for n in (1024, 4096, 16384, 65536):
        for k in (4, 16, 64):
            out["cfg5_n%d_k%d" % (n, k)] = dict(B=262144 // n, n=n, k=k, flags=0, H=8, d=64, bf16=True,
                                                seed=5, std_qkv=0.125, backward=True)
    return out
