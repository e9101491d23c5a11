"""A forward + backward step recorded once into a CUDA graph and replayed: the library's calls are plain stream
work (kernel launches and one memset of the status block), so a replay must reproduce the eager results bit for
bit on every kernel family."""
import pytest

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,k,flags,B,H,d,bf16", [
    (256, 4, 0, 1, 2, 32, False),     # general row kernels (fp32)
    (512, 4, 0, 2, 2, 64, True),      # warp-level tile kernels
    (1024, 24, 1, 1, 2, 64, True),    # tensor-memory forward, warp-level backward
    (512, 64, 0, 1, 2, 64, True),     # tensor-memory kernels in both passes
])
def test_graph_replay_equals_eager(n, k, flags, B, H, d, bf16):
    import torch
    from paper_1911_04070_b200 import binding, synth
    dev = "cuda:0"
    g = binding.bpt_build_graph(n, k, flags, device=dev)
    x = synth.make_inputs(B, g.n_nodes, H, d, g.n_rel, seed=5, std_qkv=0.5, std_rel=0.3, bf16=bf16)
    dt = torch.bfloat16 if bf16 else torch.float32
    t = {a: torch.from_numpy(b).to(dev, dt) for a, b in x.items()}
    code = binding.BPT_BF16 if bf16 else binding.BPT_F32
    ws = torch.empty(max(binding.bpt_attn_workspace_bytes(g, B, H, d, code, True),
                         binding.bpt_attn_workspace_bytes(g, B, H, d, code, False), 256), dtype=torch.uint8, device=dev)
    out = torch.empty_like(t["q"]); lse = torch.empty((B, g.n_nodes, H), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty_like(t["q"]) for _ in range(3))
    d_rel = torch.empty((g.n_rel, d), dtype=torch.float32, device=dev)
    scale = d ** -0.5

    def step():
        binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out=out, lse=lse, workspace=ws)
        binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"], workspace=ws,
                             dq=dq, dk=dk, dv=dv, d_rel=d_rel)

    step()                                   # eager: also the one-time lookups and attribute settings
    torch.cuda.synchronize()
    want = [r.clone() for r in (out, lse, dq, dk, dv, d_rel)]
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        for r in (out, lse, dq, dk, dv, d_rel):
            r.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert binding.bpt_check(ws) == 0
        for name, a, b in zip(("out", "lse", "dq", "dk", "dv", "d_rel"), (out, lse, dq, dk, dv, d_rel), want):
            assert torch.equal(a, b), name
