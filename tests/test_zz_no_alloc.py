"""The allocation-free backward entry point (scratch inside the library's device image).

Some callers may hand the library tensors but cannot call cudaMalloc themselves (plugins
without an allocator, loops that must not allocate after start-up, processes whose pool
owns the whole device).  For them bpt_attn_bwd_static_scratch must give what bpt_attn_bwd
gives with a caller-supplied workspace.  This file is collected last on purpose: a run that
stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest

from parity import TOL, assert_close

pytestmark = pytest.mark.gpu


def _problem(seed):
    import torch
    from paper_1911_04070_b200 import binding, synth
    n, k, flags, B, H, d = 256, 4, 0, 2, 8, 64
    g = binding.bpt_build_graph(n, k, flags, device="cuda:0")
    x = synth.make_inputs(B, g.n_nodes, H, d, g.n_rel, seed=seed, std_qkv=0.125, bf16=True)
    t = {a: torch.from_numpy(b).to("cuda:0", torch.bfloat16) for a, b in x.items()}
    return g, t, d ** -0.5


def test_static_scratch_backward_matches_workspace_backward_twice():
    import torch
    from paper_1911_04070_b200 import binding
    g, t, scale = _problem(21)
    B, N, H, d = t["q"].shape
    assert binding.bpt_attn_workspace_bytes(g, B, H, d, binding.BPT_BF16, True) <= binding.bpt_static_scratch_bytes()
    out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale)
    want = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"])
    torch.cuda.synchronize()
    for call in range(2):      # the second call finds the first call's leftovers in the array
        dq, dk, dv = (torch.full_like(t["q"], float("nan")) for _ in range(3))
        d_rel = torch.full((g.n_rel, d), float("nan"), dtype=torch.float32, device="cuda:0")
        binding.bpt_attn_bwd_static_scratch(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"],
                                            dq, dk, dv, d_rel)
        torch.cuda.synchronize()
        first_anc = 1 + 2 * g.dims.n_levels * (g.k + 1)
        for name, a, b in zip(("dq", "dk", "dv"), (dq, dk, dv), want[:3]):
            assert_close("%s (call %d)" % (name, call), a.float().cpu().numpy(), b.float().cpu().numpy(), TOL["bf16"])
        assert_close("d_rel (call %d)" % call, d_rel[:first_anc].cpu().numpy(), want[3][:first_anc].cpu().numpy(), TOL["bf16"])
        assert (d_rel[first_anc:] == 0).all()
        # a different problem in between, so that the leftovers really differ
        g2, t2, s2 = _problem(22 + call)
        o2, l2 = binding.bpt_attn_fwd(g2, t2["q"], t2["k"], t2["v"], t2["rel_emb"], s2)
        binding.bpt_attn_bwd_static_scratch(g2, t2["q"], t2["k"], t2["v"], t2["rel_emb"], s2, o2, l2, t2["d_out"],
                                            torch.empty_like(t2["q"]), torch.empty_like(t2["q"]), torch.empty_like(t2["q"]),
                                            torch.empty((g2.n_rel, d), dtype=torch.float32, device="cuda:0"))


def test_static_scratch_refuses_problems_beyond_its_limit():
    import torch
    from paper_1911_04070_b200 import binding
    n, k, B, H, d = 2048, 8, 4, 8, 64
    g = binding.bpt_build_graph(n, k, 0, device="cuda:0")
    assert binding.bpt_attn_workspace_bytes(g, B, H, d, binding.BPT_BF16, True) > binding.bpt_static_scratch_bytes()
    q = torch.zeros((B, g.n_nodes, H, d), dtype=torch.bfloat16, device="cuda:0")
    r = torch.zeros((g.n_rel, d), dtype=torch.bfloat16, device="cuda:0")
    lse = torch.zeros((B, g.n_nodes, H), dtype=torch.float32, device="cuda:0")
    d_rel = torch.zeros((g.n_rel, d), dtype=torch.float32, device="cuda:0")
    with pytest.raises(binding.BptError) as ei:
        binding.bpt_attn_bwd_static_scratch(g, q, q, q, r, 1.0, q, lse, q, q.clone(), q.clone(), q.clone(), d_rel)
    assert ei.value.status == 7
    assert "static" in str(ei.value)
