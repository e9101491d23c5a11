"""The device-side failure report: a bounded wait that runs out makes the kernel store BPT_ERR_TIMEOUT
in the workspace's status block and return, and bpt_check hands that to the host.  The library's
self-test kernel waits, with a limit of a few thousand cycles, on a barrier nobody arrives on -- the
wait is bounded by construction, nothing faults or hangs -- and the context stays usable afterwards."""
import pytest

pytestmark = pytest.mark.gpu


def test_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    import torch
    from paper_1911_04070_b200 import binding
    ws = torch.full((256,), 0xFF, dtype=torch.uint8, device="cuda:0")
    binding.bpt_selftest_wait_timeout(ws, 20000, arrive=False)
    assert binding.bpt_check(ws) == 5                      # BPT_ERR_TIMEOUT
    assert binding.status_str(5) == "device-side wait timed out"
    binding.bpt_selftest_wait_timeout(ws, 20000, arrive=True)
    assert binding.bpt_check(ws) == 0                      # the barrier completed: cleared block stays clear
    # the context is intact: a real forward runs and reports no give-up
    g = binding.bpt_build_graph(128, 64, 0, device="cuda:0", with_transpose=False)
    q = torch.randn((1, g.n_nodes, 2, 64), device="cuda:0").bfloat16()
    r = torch.zeros((g.n_rel, 64), device="cuda:0", dtype=torch.bfloat16)
    out, lse = binding.bpt_attn_fwd(g, q, q, q, r, 0.125)
    assert binding.bpt_check(out._bpt_workspace) == 0
    assert torch.isfinite(out.float()).all()


def test_every_attention_call_clears_the_block_it_is_given():
    import torch
    from paper_1911_04070_b200 import binding
    g = binding.bpt_build_graph(128, 8, 0, device="cuda:0")
    q = torch.randn((1, g.n_nodes, 2, 64), device="cuda:0").bfloat16()
    r = torch.zeros((g.n_rel, 64), device="cuda:0", dtype=torch.bfloat16)
    need = max(binding.bpt_attn_workspace_bytes(g, 1, 2, 64, binding.BPT_BF16, b) for b in (False, True))
    ws = torch.empty(need, dtype=torch.uint8, device="cuda:0")
    binding.bpt_selftest_wait_timeout(ws, 1000, arrive=False)
    assert binding.bpt_check(ws) == 5
    out, lse = binding.bpt_attn_fwd(g, q, q, q, r, 0.125, workspace=ws)
    assert binding.bpt_check(ws) == 0
    binding.bpt_selftest_wait_timeout(ws, 1000, arrive=False)
    binding.bpt_attn_bwd(g, q, q, q, r, 0.125, out, lse, q, workspace=ws)
    assert binding.bpt_check(ws) == 0
    assert binding.bpt_check(None) == 0
