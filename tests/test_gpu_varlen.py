"""Sequences shorter than n through the C ABI (bpt_attn_fwd_varlen / bpt_attn_bwd_varlen) against the
fp64 oracle's reading: a node is real when it covers a real token, edges touching other nodes do not
exist, rows of such nodes are zero.  The placeholder rows of the inputs hold large finite values, so a
kernel that let them leak into a result would fail."""
import numpy as np
import pytest

from parity import TOL, assert_close, assert_max_norm

pytestmark = pytest.mark.gpu


def _np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def run_case(n, k, flags, H, d, bf16, lengths, seed, path=0):
    import torch
    from oracle import ctwin
    from paper_1911_04070_b200 import binding, synth
    tol = TOL["bf16" if bf16 else "fp32"]
    B = len(lengths)
    ref = ctwin.CGraph(n, k, flags)
    x = synth.make_inputs(B, ref.n_nodes, H, d, ref.n_rel, seed=seed, std_qkv=0.5, std_rel=0.3, bf16=bf16)
    # placeholder rows: large but finite (they must not matter)
    first = np.zeros(ref.n_nodes, dtype=np.int64)
    base, width, level = 0, n, 0
    while width >= 1:
        first[base:base + width] = np.arange(width) << level
        base, width, level = base + width, width >> 1, level + 1
    for b, length in enumerate(lengths):
        for name in ("q", "k", "v", "d_out"):
            x[name][b, first >= length] = 96.0
    dt = torch.bfloat16 if bf16 else torch.float32
    t = {a: torch.from_numpy(v).to("cuda:0", dt) for a, v in x.items()}
    lens = torch.tensor(lengths, dtype=torch.int32, device="cuda:0")
    g = binding.bpt_build_graph(n, k, flags, device="cuda:0")
    scale = d ** -0.5
    out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, lengths=lens, path=path)
    assert binding.bpt_check(out._bpt_workspace) == 0
    o_ref, lse_ref = ctwin.attn_fwd_varlen(ref, x["q"], x["k"], x["v"], x["rel_emb"], scale, lengths)
    assert_close("out", _np(out), o_ref, tol)
    assert_close("lse", _np(lse), lse_ref, tol)
    for b, length in enumerate(lengths):      # rows of nodes without real tokens are exact zeros
        assert (out[b][torch.from_numpy(first >= length).to("cuda:0")] == 0).all()
    dq, dk, dv, dr = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"], lengths=lens, path=path)
    assert binding.bpt_check(dq._bpt_workspace) == 0
    exact = ctwin.attn_bwd_varlen(ref, x["q"], x["k"], x["v"], x["rel_emb"], scale, x["d_out"], lengths)
    first_anc = 1 + 2 * ref.L * (k + 1)
    for name, a, b_ in zip(("dq", "dk", "dv"), (dq, dk, dv), exact[:3]):
        assert_max_norm(name, _np(a), b_, tol)
    assert_max_norm("d_rel", _np(dr)[:first_anc], exact[3][:first_anc], tol)
    rq, rk, rv, rr = ctwin.attn_bwd_varlen(ref, x["q"], x["k"], x["v"], x["rel_emb"], scale, x["d_out"], lengths, out=_np(out))
    assert_close("dq", _np(dq), rq, tol, row_rms=True)
    assert_close("dk", _np(dk), rk, tol, row_rms=True)
    assert_close("dv", _np(dv), rv, tol, row_rms=True)
    assert_close("d_rel", _np(dr)[:first_anc], rr[:first_anc], tol)
    for b, length in enumerate(lengths):
        m = torch.from_numpy(first >= length).to("cuda:0")
        assert (dq[b][m] == 0).all() and (dk[b][m] == 0).all() and (dv[b][m] == 0).all()


CASES = [
    # n, k, flags, H, d, bf16, lengths
    (16, 2, 0, 2, 32, False, [16, 5, 1]),                 # general row kernels
    (256, 4, 1, 3, 64, False, [200, 64, 255]),
    (64, 4, 0, 2, 64, True, [64, 37, 1]),                 # one tile
    (256, 4, 0, 3, 64, True, [256, 100, 65, 64]),         # tile boundaries
    (512, 16, 1, 2, 64, True, [300, 511]),
    (1024, 64, 0, 1, 64, True, [1000, 129]),              # k = 64: tensor-memory forward
    (2048, 8, 2, 2, 64, True, [1500, 2048, 7]),
    (4096, 3, 0, 1, 64, True, [4000, 2049]),              # outer ancestors with and without real tokens
]


@pytest.mark.parametrize("n,k,flags,H,d,bf16,lengths", CASES)
def test_short_sequences(n, k, flags, H, d, bf16, lengths):
    run_case(n, k, flags, H, d, bf16, lengths, seed=300 + n + k)


@pytest.mark.parametrize("n,k,flags,H,lengths", [(128, 64, 0, 2, [128, 77, 1]), (256, 4, 1, 3, [256, 100, 129, 128]),
                                                 (1024, 64, 0, 1, [1000, 129]), (2048, 33, 1, 2, [1500, 2048, 7])])
def test_short_sequences_tensor_memory_kernels(n, k, flags, H, lengths):
    from paper_1911_04070_b200 import binding
    run_case(n, k, flags, H, 64, True, lengths, seed=400 + n + k, path=binding.BPT_PATH_TC5)


def test_full_lengths_give_the_plain_result_bitwise():
    import torch
    from paper_1911_04070_b200 import binding, synth
    n, k, B, H, d = 512, 8, 2, 4, 64
    g = binding.bpt_build_graph(n, k, 0, device="cuda:0")
    x = synth.make_inputs(B, g.n_nodes, H, d, g.n_rel, seed=5, std_qkv=0.125, bf16=True)
    t = {a: torch.from_numpy(v).to("cuda:0", torch.bfloat16) for a, v in x.items()}
    lens = torch.full((B,), n, dtype=torch.int32, device="cuda:0")
    o1, l1 = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125)
    o2, l2 = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, lengths=lens)
    assert torch.equal(o1, o2) and torch.equal(l1, l2)
    g1 = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, o1, l1, t["d_out"])
    g2 = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, o1, l1, t["d_out"], lengths=lens)
    for a, b in zip(g1, g2):
        assert torch.equal(a, b)
