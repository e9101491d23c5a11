"""bpt_attn_fwd / bpt_attn_bwd only enqueue kernels on the caller's stream (no allocation, no
synchronisation), so a forward + backward can be captured in a CUDA graph and replayed: the replay
must give the bits of the plain calls.  Useful where a step is a few short launches."""
import pytest

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,k,flags,B,H,d,bf16", [(256, 4, 0, 1, 2, 32, False), (512, 8, 0, 2, 3, 64, True), (1024, 64, 1, 1, 2, 64, True)])
def test_forward_backward_replay_from_a_graph(n, k, flags, B, H, d, bf16):
    import torch
    from paper_1911_04070_b200 import binding, synth
    g = binding.bpt_build_graph(n, k, flags, device="cuda:0")
    x = synth.make_inputs(B, g.n_nodes, H, d, g.n_rel, seed=3, std_qkv=0.5, bf16=bf16)
    dt = torch.bfloat16 if bf16 else torch.float32
    t = {a: torch.from_numpy(b).to("cuda:0", dt) for a, b in x.items()}
    code = binding.BPT_BF16 if bf16 else binding.BPT_F32
    ws = torch.zeros(max(binding.bpt_attn_workspace_bytes(g, B, H, d, code, True),
                         binding.bpt_attn_workspace_bytes(g, B, H, d, code, False), 1), dtype=torch.uint8, device="cuda:0")
    out = torch.empty_like(t["q"])
    lse = torch.empty((B, g.n_nodes, H), device="cuda:0")
    dq, dk, dv = (torch.empty_like(t["q"]) for _ in range(3))
    dr = torch.empty((g.n_rel, d), device="cuda:0")
    res = (out, lse, dq, dk, dv, dr)

    def step():
        binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], d ** -0.5, out=out, lse=lse, workspace=ws)
        binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], d ** -0.5, out, lse, t["d_out"], workspace=ws,
                             dq=dq, dk=dk, dv=dv, d_rel=dr)

    step()
    torch.cuda.synchronize()
    want = [a.clone() for a in res]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):        # warm-up on a side stream, as graph capture asks for
        step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for a in res:
        a.zero_()
    graph.replay()
    torch.cuda.synchronize()
    for a, b in zip(res, want):
        assert torch.equal(a, b)
