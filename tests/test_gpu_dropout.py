"""Attention dropout through the C ABI (bpt_attn_fwd_ex / bpt_attn_bwd_ex) against the fp64 oracle: the
library must draw exactly the oracle's masks (Philox4x32-10 keyed on seed, batch entry, head,
destination, source), so outputs and gradients are compared element by element as in the other
parity tests."""
import numpy as np
import pytest

from parity import TOL, assert_close, assert_max_norm

pytestmark = pytest.mark.gpu


def _np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


CASES = [
    # n, k, flags, B, H, d, bf16, p, seed
    (16, 2, 0, 2, 2, 32, False, 0.3, 7),                       # general row kernels
    (128, 3, 1, 1, 3, 64, False, 0.1, (5 << 32) | 9),
    (64, 4, 0, 2, 2, 64, True, 0.25, 11),                      # tiled kernels, one tile
    (512, 16, 1, 2, 3, 64, True, 0.1, 12345678901234),
    (1024, 64, 0, 1, 2, 64, True, 0.3, 3),                     # k = 64: tensor-memory forward
    (2048, 8, 0, 1, 2, 64, True, 0.5, 99),
]


@pytest.mark.parametrize("n,k,flags,B,H,d,bf16,p,seed", CASES)
def test_dropout_parity(n, k, flags, B, H, d, bf16, p, seed):
    _dropout_case(n, k, flags, B, H, d, bf16, p, seed, 0)


@pytest.mark.parametrize("n,k,flags,B,H,p,seed", [(128, 64, 0, 1, 2, 0.3, 3), (512, 16, 1, 2, 3, 0.1, 12345678901234),
                                                   (1024, 63, 0, 1, 2, 0.25, (7 << 32) | 5)])
def test_dropout_parity_tensor_memory_kernels(n, k, flags, B, H, p, seed):
    from paper_1911_04070_b200 import binding
    _dropout_case(n, k, flags, B, H, 64, True, p, seed, binding.BPT_PATH_TC5)


def _dropout_case(n, k, flags, B, H, d, bf16, p, seed, path):
    import torch
    from oracle import ctwin
    from paper_1911_04070_b200 import binding, synth
    tol = TOL["bf16" if bf16 else "fp32"]
    ref = ctwin.CGraph(n, k, flags)
    x = synth.make_inputs(B, ref.n_nodes, H, d, ref.n_rel, seed=500 + n, std_qkv=0.5, std_rel=0.3, bf16=bf16)
    dt = torch.bfloat16 if bf16 else torch.float32
    t = {a: torch.from_numpy(v).to("cuda:0", dt) for a, v in x.items()}
    g = binding.bpt_build_graph(n, k, flags, device="cuda:0")
    scale = d ** -0.5
    out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, dropout_p=p, dropout_seed=seed, path=path)
    assert binding.bpt_check(out._bpt_workspace) == 0
    o_ref, lse_ref = ctwin.attn_fwd(ref, x["q"], x["k"], x["v"], x["rel_emb"], scale, p_drop=p, seed=seed)
    o_plain, _ = ctwin.attn_fwd(ref, x["q"], x["k"], x["v"], x["rel_emb"], scale)
    assert np.abs(o_ref - o_plain).max() > 10 * tol * np.abs(o_plain).max()      # the masks do change the result
    assert_close("out", _np(out), o_ref, tol)
    assert_close("lse", _np(lse), lse_ref, tol)
    dq, dk, dv, dr = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"],
                                          dropout_p=p, dropout_seed=seed, path=path)
    assert binding.bpt_check(dq._bpt_workspace) == 0
    first_anc = 1 + 2 * ref.L * (k + 1)
    exact = ctwin.attn_bwd(ref, x["q"], x["k"], x["v"], x["rel_emb"], scale, x["d_out"], p_drop=p, seed=seed)
    for name, a, b_ in zip(("dq", "dk", "dv"), (dq, dk, dv), exact[:3]):
        assert_max_norm(name, _np(a), b_, tol)
    assert_max_norm("d_rel", _np(dr)[:first_anc], exact[3][:first_anc], tol)
    rq, rk, rv, rr = ctwin.attn_bwd(ref, x["q"], x["k"], x["v"], x["rel_emb"], scale, x["d_out"], out=_np(out), p_drop=p, seed=seed)
    assert_close("dq", _np(dq), rq, tol, row_rms=True)
    assert_close("dk", _np(dk), rk, tol, row_rms=True)
    assert_close("dv", _np(dv), rv, tol, row_rms=True)
    assert_close("d_rel", _np(dr)[:first_anc], rr[:first_anc], tol)


def test_bad_rate_is_refused():
    import torch
    from paper_1911_04070_b200 import binding
    g = binding.bpt_build_graph(64, 2, 0, device="cuda:0")
    q = torch.zeros((1, g.n_nodes, 2, 64), device="cuda:0")
    r = torch.zeros((g.n_rel, 64), device="cuda:0")
    with pytest.raises(binding.BptError) as ei:
        binding.bpt_attn_fwd(g, q, q, q, r, 1.0, dropout_p=1.0)
    assert ei.value.status == 1
