"""The tiled backward works through the (batch entry, head) pairs in passes when the workspace it is
given holds the partial rows of only some of them, adding d_rel up over the passes.  With a workspace
a third of the planned size a mid-sized problem takes several passes and must still match the oracle,
and the single-pass result bit for bit."""
import numpy as np
import pytest

from parity import TOL, assert_close

pytestmark = pytest.mark.gpu


def _backward(g, t, out, lse, ws_bytes):
    import torch
    from paper_1911_04070_b200 import binding
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda:0")
    binding.bpt_trace_begin(400)
    grads = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, out, lse, t["d_out"], workspace=ws,
                                 path=binding.BPT_PATH_MMA)
    passes = sum(1 for a, _ in binding.bpt_trace_end(400) if a == "bwd_tile")
    assert binding.bpt_check(ws) == 0
    return grads, passes


def test_many_passes_match_one_pass():
    import torch
    from oracle import ctwin
    from paper_1911_04070_b200 import binding, synth
    n, k, flags, B, H, d = 1024, 16, 0, 3, 5, 64
    ref = ctwin.CGraph(n, k, flags)
    x = synth.make_inputs(B, ref.n_nodes, H, d, ref.n_rel, seed=21, std_qkv=0.5, std_rel=0.3, bf16=True)
    t = {a: torch.from_numpy(b).to("cuda:0", torch.bfloat16) for a, b in x.items()}
    g = binding.bpt_build_graph(n, k, flags, device="cuda:0")
    ws_one = binding.bpt_attn_workspace_bytes(g, B, H, d, binding.BPT_BF16, True)
    ws_min = binding.bpt_attn_bwd_min_workspace_bytes(g, B, H, d, binding.BPT_BF16)
    ws_many = max(ws_one // 3, ws_min)
    assert ws_min <= ws_many < ws_one
    out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125)
    one, passes_one = _backward(g, t, out, lse, ws_one)
    many, passes_many = _backward(g, t, out, lse, ws_many)
    least, passes_least = _backward(g, t, out, lse, ws_min)
    assert passes_one == 1 and 1 < passes_many <= passes_least <= B * H and passes_least > 2

    o64 = out.float().cpu().numpy().astype(np.float64)
    want = ctwin.attn_bwd(ref, x["q"], x["k"], x["v"], x["rel_emb"], 0.125, x["d_out"], out=o64)
    fa = 1 + 2 * ref.L * (k + 1)
    for grads in (many, least):
        for name, a, b in zip(("dq", "dk", "dv"), grads[:3], want[:3]):
            assert_close(name, a.float().cpu().numpy(), b, TOL["bf16"], row_rms=True)
        assert_close("d_rel", grads[3].cpu().numpy()[:fa], want[3][:fa], TOL["bf16"])
        for name, x1, y1 in zip(("dq", "dk", "dv"), one[:3], grads[:3]):
            assert torch.equal(x1, y1), name       # per-pair work does not depend on the pass it runs in
        # d_rel is summed pass by pass (another, still fixed, order): equal up to fp32 rounding
        assert torch.allclose(one[3], grads[3], rtol=1e-4, atol=1e-6 * float(one[3].abs().max()))

    # a workspace below the minimum is refused on the host
    with pytest.raises(binding.BptError) as ei:
        binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, out, lse, t["d_out"],
                             workspace=torch.empty(ws_min - 256, dtype=torch.uint8, device="cuda:0"), path=binding.BPT_PATH_MMA)
    assert ei.value.status == 3
