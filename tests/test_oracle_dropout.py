"""Pins of the oracle's attention dropout: the generator against the published known-answer vectors
of Philox4x32-10, the mask's statistics, p = 0, finite differences with the (input-independent)
mask, and the C twin."""
import numpy as np
import pytest

from oracle import bpt_oracle as orc
from oracle import ctwin

# known-answer vectors distributed with the generator's reference implementation (Random123, kat_vectors):
# counter words, key words -> output words
KAT = [
    ((0, 0, 0, 0), (0, 0), (0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8)),
    ((0xffffffff,) * 4, (0xffffffff,) * 2, (0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd)),
    ((0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344), (0xa4093822, 0x299f31d0), (0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1)),
]


@pytest.mark.parametrize("ctr,key,want", KAT)
def test_philox_known_answers(ctr, key, want):
    assert tuple(int(x) for x in orc.philox4x32_10(*ctr, *key)) == want


def test_mask_statistics_and_determinism():
    dst, src = np.meshgrid(np.arange(300), np.arange(300), indexing="ij")
    for p in (0.1, 0.3, 0.75):
        keep = orc.dropout_keep(12345, p, 1, 2, 8, dst.ravel(), src.ravel())
        assert abs(keep.mean() - (1 - p)) < 4 * np.sqrt(p * (1 - p) / keep.size)
        assert np.array_equal(keep, orc.dropout_keep(12345, p, 1, 2, 8, dst.ravel(), src.ravel()))
        other = orc.dropout_keep(12346, p, 1, 2, 8, dst.ravel(), src.ravel())
        assert 0.2 < (keep != other).mean() / (2 * p * (1 - p)) < 1.8      # another seed: an independent mask
    assert orc.dropout_keep(7, 0.0, 0, 0, 1, dst.ravel(), src.ravel()).all()


def _inputs(g, B, H, d, seed):
    rng = np.random.default_rng(seed)
    sh = (B, g.n_nodes, H, d)
    return rng.standard_normal(sh), rng.standard_normal(sh), rng.standard_normal(sh), 0.5 * rng.standard_normal((g.n_rel, d)), rng.standard_normal(sh)


def test_zero_rate_is_plain_attention_and_mean_over_seeds_approaches_it():
    g = orc.enumerate_graph(16, 2, 0)
    q, k, v, r, go = _inputs(g, 1, 2, 4, 0)
    o0, l0 = orc.attn_fwd(g, q, k, v, r, 0.4)
    o1, l1 = orc.attn_fwd_dropout(g, q, k, v, r, 0.4, 0.0, 99)
    assert np.allclose(o0, o1, rtol=1e-13, atol=1e-14) and np.allclose(l0, l1)
    acc = np.zeros_like(o0)
    n_seeds = 400
    for s in range(n_seeds):
        acc += orc.attn_fwd_dropout(g, q, k, v, r, 0.4, 0.25, 1000 + s)[0]
    assert np.abs(acc / n_seeds - o0).max() < 0.25          # inverted dropout is unbiased


def test_gradient_by_finite_differences_with_a_fixed_mask():
    g = orc.enumerate_graph(8, 1, 0)
    q, k, v, r, go = _inputs(g, 1, 2, 3, 3)
    p, seed = 0.3, 2024
    f = lambda q_, k_, v_, r_: float((orc.attn_fwd_dropout(g, q_, k_, v_, r_, 0.7, p, seed)[0] * go).sum())
    grads = orc.attn_bwd_dropout(g, q, k, v, r, 0.7, go, p, seed)
    eps = 1e-6
    rng = np.random.default_rng(0)
    for which, arr in enumerate((q, k, v, r)):
        for _ in range(12):
            idx = tuple(rng.integers(0, s) for s in arr.shape)
            args = [q, k, v, r]
            hi, lo = arr.copy(), arr.copy()
            hi[idx] += eps; lo[idx] -= eps
            args[which] = hi; fh = f(*args)
            args[which] = lo; fl = f(*args)
            assert abs((fh - fl) / (2 * eps) - grads[which][idx]) < 1e-6, (which, idx)


def test_c_twin_draws_the_same_masks():
    n, k, flags = 64, 3, 1
    g, cg = orc.enumerate_graph(n, k, flags), ctwin.CGraph(n, k, flags)
    q, kk, v, r, go = _inputs(g, 2, 2, 8, 11)
    p, seed = 0.2, (7 << 32) | 12345
    o1, l1 = orc.attn_fwd_dropout(g, q, kk, v, r, 0.35, p, seed)
    o2, l2 = ctwin.attn_fwd(cg, q, kk, v, r, 0.35, p_drop=p, seed=seed)
    assert np.allclose(o1, o2, rtol=1e-12, atol=1e-13) and np.allclose(l1, l2, rtol=1e-12, atol=1e-13)
    g1 = orc.attn_bwd_dropout(g, q, kk, v, r, 0.35, go, p, seed)
    g2 = ctwin.attn_bwd(cg, q, kk, v, r, 0.35, go, p_drop=p, seed=seed)
    for a, b in zip(g1, g2):
        assert np.allclose(a, b, rtol=1e-11, atol=1e-12)
