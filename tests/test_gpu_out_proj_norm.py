"""bpt_out_proj_norm (output projection + residual + layer normalisation of Algorithm 2 in one kernel)
against the float64 oracle, element by element, over row counts with ragged tails and the three widths."""
import numpy as np
import pytest

from parity import TOL, assert_close

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,D", [(1, 128), (100, 256), (128, 512), (129, 128), (1000, 512), (4 * 1023, 256), (2 * 16383, 512)])
def test_matches_the_oracle(rows, D):
    import torch
    from oracle import bpt_layer
    from paper_1911_04070_b200 import binding
    g = torch.Generator().manual_seed(rows + D)
    bf = lambda *shape, s=1.0: (torch.randn(*shape, generator=g) * s).bfloat16()
    a, h, w = bf(rows, D), bf(rows, D), bf(D, D, s=D ** -0.5)
    gamma, beta = 1 + 0.5 * torch.randn(D, generator=g), 0.5 * torch.randn(D, generator=g)
    ws = torch.full((256,), 0xFF, dtype=torch.uint8, device="cuda:0")
    z = binding.bpt_out_proj_norm(a.cuda(), w.cuda(), h.cuda(), gamma.cuda(), beta.cuda(), 1e-5, workspace=ws)
    assert binding.bpt_check(ws) == 0
    want = bpt_layer.out_proj_norm(a.float().numpy(), w.float().numpy(), h.float().numpy(), gamma.numpy(), beta.numpy(), 1e-5)
    assert_close("z", z.float().cpu().numpy(), want, TOL["bf16"])
    z2 = binding.bpt_out_proj_norm(a.cuda(), w.cuda(), h.cuda(), gamma.cuda(), beta.cuda(), 1e-5)
    assert torch.equal(z, z2)


def test_argument_errors():
    import torch
    from paper_1911_04070_b200 import binding
    a = torch.zeros(4, 192, dtype=torch.bfloat16, device="cuda:0")
    w = torch.zeros(192, 192, dtype=torch.bfloat16, device="cuda:0")
    v = torch.zeros(192, device="cuda:0")
    with pytest.raises(binding.BptError) as ei:      # width 192 is not supported
        binding.bpt_out_proj_norm(a, w, a, v, v)
    assert ei.value.status == 2


def test_layer_in_eval_mode_uses_the_fused_kernel_and_agrees_with_the_operators():
    import torch
    from paper_1911_04070_b200 import binding, layer
    torch.manual_seed(0)
    enc = layer.BPTEncoder(128, 4, 128, 2, 128, 2, device="cuda:0").to("cuda:0", torch.bfloat16).eval()
    x = torch.randn(2, 128, 128, device="cuda:0", dtype=torch.bfloat16)
    with torch.no_grad():
        binding.bpt_trace_begin(64)
        y = enc(x)
        names = [a for a, _ in binding.bpt_trace_end(64)]
        assert names.count("out_proj_norm") == 2, names
        layer.FUSE_OUT_PROJ_NORM = False
        try:
            y_ref = enc(x)
        finally:
            layer.FUSE_OUT_PROJ_NORM = True
    err = (y.float() - y_ref.float()).abs().max().item()
    assert err <= 5e-2 * y_ref.float().abs().max().item(), err     # two bf16 pipelines with different rounding points
