"""The tensor-memory (tcgen05) kernels for the token rows, forced with path = BPT_PATH_TC5 on shapes
that the automatic choice would give to the warp-level kernels as well; compared with the fp64 oracle
exactly as the other parity tests do."""
import numpy as np
import pytest

from parity import TOL, assert_close

pytestmark = pytest.mark.gpu

CASES = [(128, 64, 0, 2, 2), (256, 4, 0, 2, 9), (256, 33, 1, 1, 3), (512, 63, 2, 1, 2), (2048, 3, 3, 1, 2),
         (4096, 64, 0, 1, 1), (8192, 64, 1, 1, 8), (16384, 4, 0, 1, 2)]


@pytest.mark.parametrize("n,k,flags,B,H", CASES)
def test_tensor_memory_forward_matches_oracle(n, k, flags, B, H):
    import torch
    from oracle import ctwin
    from paper_1911_04070_b200 import binding, synth
    ref = ctwin.CGraph(n, k, flags)
    x = synth.make_inputs(B, ref.n_nodes, H, 64, ref.n_rel, seed=7 + n + k, std_qkv=0.5, std_rel=0.3, bf16=True, with_grad=False)
    g = binding.bpt_build_graph(n, k, flags, device="cuda:0", with_transpose=False)
    t = {a: torch.from_numpy(b).to("cuda:0", torch.bfloat16) for a, b in x.items()}
    ws = torch.empty(binding.bpt_attn_workspace_bytes(g, B, H, 64, binding.BPT_BF16, False), dtype=torch.uint8, device="cuda:0")
    binding.bpt_trace_begin(8)
    out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, workspace=ws, path=binding.BPT_PATH_TC5)
    names = [a for a, _ in binding.bpt_trace_end(8)]
    assert "fwd_tc5" in names, names          # the tensor-memory kernel really ran
    assert binding.bpt_check(ws) == 0         # no bounded wait gave up
    o_ref, lse_ref = ctwin.attn_fwd(ref, x["q"], x["k"], x["v"], x["rel_emb"], 0.125)
    assert_close("out", out.float().cpu().numpy(), o_ref, TOL["bf16"])
    assert_close("lse", lse.cpu().numpy(), lse_ref, TOL["bf16"])
    out2, lse2 = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, path=binding.BPT_PATH_TC5)
    assert torch.equal(out, out2) and torch.equal(lse, lse2)


@pytest.mark.parametrize("n,k,flags,B,H,std", [(256, 33, 1, 1, 3, 3.0), (1024, 64, 0, 1, 2, 3.0), (2048, 16, 0, 1, 2, 8.0),
                                               (8192, 64, 1, 1, 2, 8.0)])
def test_tensor_memory_forward_wide_logits(n, k, flags, B, H, std):
    """Scores that differ by tens to hundreds of binary orders of magnitude between a row's items: the kernel keeps
    its output accumulator in tensor memory and raises the row's reference exponent (rescaling the accumulator in
    place) when a later item exceeds it, so this is the case that exercises the rescale."""
    import torch
    from oracle import ctwin
    from paper_1911_04070_b200 import binding, synth
    ref = ctwin.CGraph(n, k, flags)
    x = synth.make_inputs(B, ref.n_nodes, H, 64, ref.n_rel, seed=11 + n + k, std_qkv=std, std_rel=0.3, bf16=True, with_grad=False)
    g = binding.bpt_build_graph(n, k, flags, device="cuda:0", with_transpose=False)
    t = {a: torch.from_numpy(b).to("cuda:0", torch.bfloat16) for a, b in x.items()}
    ws = torch.empty(binding.bpt_attn_workspace_bytes(g, B, H, 64, binding.BPT_BF16, False), dtype=torch.uint8, device="cuda:0")
    out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, workspace=ws, path=binding.BPT_PATH_TC5)
    assert binding.bpt_check(ws) == 0
    o_ref, lse_ref = ctwin.attn_fwd(ref, x["q"], x["k"], x["v"], x["rel_emb"], 0.125)
    assert np.isfinite(out.float().cpu().numpy()).all()
    assert_close("out", out.float().cpu().numpy(), o_ref, TOL["bf16"])
    assert_close("lse", lse.cpu().numpy(), lse_ref, TOL["bf16"])
    out_m, lse_m = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, path=binding.BPT_PATH_MMA)
    assert_close("out vs warp-level kernel", out.float().cpu().numpy(), out_m.float().cpu().numpy(), TOL["bf16"])


BWD_CASES = [
    # n, k, flags, B, H
    (128, 64, 0, 2, 2),       # one tile per kernel, k = 64 on both sides
    (128, 1, 1, 1, 3),        # thinnest graph
    (256, 33, 1, 1, 3),       # odd k, left only
    (512, 63, 2, 1, 2),       # Algorithm-1 graph, k + 1 = 64 relation rows exactly
    (1024, 16, 0, 2, 3),
    (2048, 3, 3, 1, 2),
    (4096, 64, 0, 1, 1),      # level-0 ranges split into several items
    (8192, 64, 1, 1, 8),      # the metric shape at batch 1
]


@pytest.mark.parametrize("n,k,flags,B,H", BWD_CASES)
def test_tensor_memory_backward_matches_oracle(n, k, flags, B, H):
    """Both passes forced onto the tensor-memory kernels (query-side and key-side backward), with the same
    criteria as the general parity tests, including the bit-for-bit repeat."""
    from paper_1911_04070_b200 import binding
    from test_gpu_attention import run_case
    run_case(n, k, flags, B, H, 64, True, seed=100 + n + k, std_qkv=0.5, std_rel=0.3, path=binding.BPT_PATH_TC5)


def test_tensor_memory_backward_in_passes():
    """A workspace that holds one (batch entry, head) pair at a time: same dq, dk, dv bits as the single pass."""
    import torch
    from paper_1911_04070_b200 import binding, synth
    n, k, B, H, d = 1024, 48, 2, 3, 64
    g = binding.bpt_build_graph(n, k, 0, device="cuda:0")
    x = synth.make_inputs(B, g.n_nodes, H, d, g.n_rel, seed=77, std_qkv=0.5, std_rel=0.3, bf16=True)
    t = {a: torch.from_numpy(b).to("cuda:0", torch.bfloat16) for a, b in x.items()}
    out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, path=binding.BPT_PATH_TC5)
    one = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, out, lse, t["d_out"], path=binding.BPT_PATH_TC5)
    ws = torch.empty(binding.bpt_attn_bwd_min_workspace_bytes(g, B, H, d, binding.BPT_BF16), dtype=torch.uint8, device="cuda:0")
    binding.bpt_trace_begin(200)
    many = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, out, lse, t["d_out"], workspace=ws, path=binding.BPT_PATH_TC5)
    names = [a for a, _ in binding.bpt_trace_end(200)]
    assert names.count("bwd_kv_tc5") > 1 and names.count("bwd_q_tc5") == 1
    assert binding.bpt_check(ws) == 0
    for a, b in zip(one[:3], many[:3]):
        assert torch.equal(a, b)
    assert torch.allclose(one[3], many[3], rtol=1e-4, atol=1e-6 * float(one[3].abs().max()))
