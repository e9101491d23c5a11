"""bpt_attn_fwd_rows: the forward restricted to listed destination rows (the decoding building block).
A decoding step for token i of a left-only graph recomputes token i and its ancestors with lengths = i + 1."""
import numpy as np
import pytest

from parity import TOL, assert_close

pytestmark = pytest.mark.gpu


def _rows_of_step(n, i):
    L = n.bit_length() - 1
    return [i] + [2 * n - ((2 * n) >> j) + (i >> j) for j in range(1, L + 1)]


@pytest.mark.parametrize("bf16,d", [(False, 32), (True, 64)])
def test_decoding_steps_match_the_full_forward(bf16, d):
    import torch
    from oracle import ctwin
    from paper_1911_04070_b200 import binding, synth
    n, k, B, H = 128, 3, 2, 2
    ref = ctwin.CGraph(n, k, 1)
    x = synth.make_inputs(B, ref.n_nodes, H, d, ref.n_rel, seed=8, std_qkv=0.5, std_rel=0.3, bf16=bf16, with_grad=False)
    dt = torch.bfloat16 if bf16 else torch.float32
    t = {a: torch.from_numpy(v).to("cuda:0", dt) for a, v in x.items()}
    g = binding.bpt_build_graph(n, k, 1, device="cuda:0", with_transpose=False)
    scale = d ** -0.5
    for steps in ([0, 5], [63, 64], [100, 127]):          # one position per batch entry
        lengths = [i + 1 for i in steps]
        rows = torch.tensor([_rows_of_step(n, i) for i in steps], dtype=torch.int32, device="cuda:0")
        lens = torch.tensor(lengths, dtype=torch.int32, device="cuda:0")
        out = torch.full_like(t["q"], 7.0)
        lse = torch.full((B, ref.n_nodes, H), 7.0, device="cuda:0")
        binding.bpt_attn_fwd_rows(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, rows, out, lse, lengths=lens)
        torch.cuda.synchronize()
        o_ref, l_ref = ctwin.attn_fwd_varlen(ref, x["q"], x["k"], x["v"], x["rel_emb"], scale, lengths)
        touched = torch.zeros((B, ref.n_nodes), dtype=torch.bool, device="cuda:0")
        for b in range(B):
            touched[b, rows[b].long()] = True
        assert (out[~touched] == 7.0).all() and (lse[~touched] == 7.0).all()      # other rows are left alone
        for b in range(B):
            idx = rows[b].long().cpu().numpy()
            assert_close("out", out[b].float().cpu().numpy()[idx], o_ref[b][idx], TOL["bf16" if bf16 else "fp32"])
            assert_close("lse", lse[b].cpu().numpy()[idx], l_ref[b][idx], TOL["bf16" if bf16 else "fp32"])
        if not bf16:      # the full forward of this shape runs the same general kernel: identical bits
            o_full, l_full = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, lengths=lens)
            assert torch.equal(out[touched], o_full[touched]) and torch.equal(lse[touched], l_full[touched])
