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


def _problem(seed, n=256, k=4, flags=0, B=2, H=8, d=64, bf16=True):
    import torch
    from paper_1911_04070_b200 import binding, synth
    g = binding.bpt_build_graph(n, k, flags, device="cuda:0")
    x = synth.make_inputs(B, g.n_nodes, H, d, g.n_rel, seed=seed, std_qkv=0.125, bf16=bf16)
    dt = torch.bfloat16 if bf16 else torch.float32
    t = {a: torch.from_numpy(b).to("cuda:0", dt) for a, b in x.items()}
    return g, t, d ** -0.5


def _outputs(g, t):
    import torch
    d = t["q"].shape[-1]
    dq, dk, dv = (torch.full_like(t["q"], float("nan")) for _ in range(3))
    d_rel = torch.full((g.n_rel, d), float("nan"), dtype=torch.float32, device="cuda:0")
    return dq, dk, dv, d_rel


def _compare(tag, g, got, want, tol):
    first_anc = 1 + 2 * g.dims.n_levels * (g.k + 1)
    for name, a, b in zip(("dq", "dk", "dv"), got[:3], want[:3]):
        assert_close("%s (%s)" % (name, tag), a.float().cpu().numpy(), b.float().cpu().numpy(), tol)
    assert_close("d_rel (%s)" % tag, got[3][:first_anc].cpu().numpy(), want[3][:first_anc].cpu().numpy(), tol)
    assert (got[3][first_anc:] == 0).all()


def test_static_scratch_backward_matches_workspace_backward_twice():
    import torch
    from paper_1911_04070_b200 import binding
    g, t, scale = _problem(21)
    B, N, H, d = t["q"].shape
    out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale)
    want = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"])
    # problems of another shape, graph, type and kernel family, run through the same array in between,
    # so that what one call leaves behind has a different layout from what the next one expects
    others = [_problem(22, n=512, k=16, flags=1, B=1, H=3), _problem(23, n=32, k=3, B=2, H=2, d=32, bf16=False)]
    prepared = []
    for g2, t2, s2 in others:
        o2, l2 = binding.bpt_attn_fwd(g2, t2["q"], t2["k"], t2["v"], t2["rel_emb"], s2)
        w2 = binding.bpt_attn_bwd(g2, t2["q"], t2["k"], t2["v"], t2["rel_emb"], s2, o2, l2, t2["d_out"])
        prepared.append((g2, t2, s2, o2, l2, w2, _outputs(g2, t2)))
    bufs = [_outputs(g, t) for _ in range(2)]
    torch.cuda.synchronize()
    binding.bpt_attn_bwd_static_scratch(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"], *_outputs(g, t))
    torch.cuda.synchronize()       # the first call on the device has looked the array up; from here on nothing may allocate
    free_before = torch.cuda.mem_get_info()[0]
    reserved_before = torch.cuda.memory_reserved()
    for call in range(2):          # the second call finds the leftovers of the calls before it
        binding.bpt_attn_bwd_static_scratch(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"], *bufs[call])
        g2, t2, s2, o2, l2, w2, outs2 = prepared[call]
        binding.bpt_attn_bwd_static_scratch(g2, t2["q"], t2["k"], t2["v"], t2["rel_emb"], s2, o2, l2, t2["d_out"], *outs2)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_reserved() == reserved_before
    for call in range(2):
        _compare("call %d" % call, g, bufs[call], want, TOL["bf16"])
        g2, t2, s2, o2, l2, w2, outs2 = prepared[call]
        _compare("other problem %d" % call, g2, outs2, w2, TOL["bf16"] if t2["q"].dtype == torch.bfloat16 else TOL["fp32"])


def test_static_scratch_takes_more_passes_instead_of_refusing():
    """A problem whose planned workspace is far above the array's size still runs: the backward fits its
    passes to the array.  Same dq, dk, dv bits as with a large workspace."""
    import torch
    from paper_1911_04070_b200 import binding
    g, t, scale = _problem(31, n=2048, k=8, B=2, H=8)
    B, N, H, d = t["q"].shape
    assert binding.bpt_attn_workspace_bytes(g, B, H, d, binding.BPT_BF16, True) > binding.bpt_static_scratch_bytes()
    assert binding.bpt_attn_bwd_min_workspace_bytes(g, B, H, d, binding.BPT_BF16) <= binding.bpt_static_scratch_bytes()
    out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale)
    want = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"])
    got = _outputs(g, t)
    binding.bpt_attn_bwd_static_scratch(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"], *got)
    torch.cuda.synchronize()
    _compare("many passes", g, got, want, TOL["bf16"])


def test_static_scratch_refuses_problems_beyond_its_limit():
    import torch
    from paper_1911_04070_b200 import binding
    n, k, B, H, d = 65536, 64, 1, 1, 64          # one (batch entry, head) pair alone needs more than the array holds
    g = binding.bpt_build_graph(n, k, 0, device="cuda:0")
    assert binding.bpt_attn_bwd_min_workspace_bytes(g, B, H, d, binding.BPT_BF16) > binding.bpt_static_scratch_bytes()
    q = torch.zeros((B, g.n_nodes, H, d), dtype=torch.bfloat16, device="cuda:0")
    r = torch.zeros((g.n_rel, d), dtype=torch.bfloat16, device="cuda:0")
    lse = torch.zeros((B, g.n_nodes, H), dtype=torch.float32, device="cuda:0")
    d_rel = torch.zeros((g.n_rel, d), dtype=torch.float32, device="cuda:0")
    with pytest.raises(binding.BptError) as ei:
        binding.bpt_attn_bwd_static_scratch(g, q, q, q, r, 1.0, q, lse, q, q.clone(), q.clone(), q.clone(), d_rel)
    assert ei.value.status == 7
    assert "static" in str(ei.value)
