"""BPTLayer / BPTEncoder (Algorithm 2 around the library's graph self-attention) against the fp64
layer oracle: outputs and the gradients of every parameter and of the input."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

NAMES = {"wq": "wq.weight", "wk": "wk.weight", "wv": "wv.weight", "wo": "wo.weight", "rel_emb": "rel_emb",
         "ln1_w": "norm1.weight", "ln1_b": "norm1.bias", "ln2_w": "norm2.weight", "ln2_b": "norm2.bias",
         "ff1_w": "ff1.weight", "ff1_b": "ff1.bias", "ff2_w": "ff2.weight", "ff2_b": "ff2.bias"}


def _run(n, k, left_only, D, H, F, n_layers, dtype, lengths, readout, tol):
    import torch
    from oracle import bpt_layer, bpt_oracle as orc
    from paper_1911_04070_b200 import layer
    torch.manual_seed(0)
    B = 2
    enc = layer.BPTEncoder(n, k, D, H, F, n_layers, left_only=left_only, device="cuda:0").to("cuda:0")
    with torch.no_grad():
        for l in enc.layers:                      # relation embeddings large enough to matter; parameters representable in dtype
            l.rel_emb.mul_(10.0)
        for p in enc.parameters():
            p.copy_(p.to(dtype).float())
    tokens = torch.randn(B, n, D).to(dtype).float()
    g_up = torch.randn(B, n, D) if readout == "tokens" else torch.randn(B, D)
    lens_dev = None if lengths is None else torch.tensor(lengths, dtype=torch.int32, device="cuda:0")

    enc_d = enc.to(dtype)
    x = tokens.to("cuda:0", dtype).requires_grad_(True)
    y = enc_d(x, lens_dev, readout)
    (y.float() * g_up.to("cuda:0")).sum().backward()

    ref_g = orc.enumerate_graph(n, k, 1 if left_only else 0)
    ws = []
    for l in enc.layers:
        sd = dict(l.named_parameters())
        ws.append({a: sd[b].detach().double().cpu().requires_grad_(True) for a, b in NAMES.items()})
    xr = tokens.double().requires_grad_(True)
    yr = bpt_layer.encoder_forward(xr, ws, ref_g, H, lengths, readout)
    (yr * g_up.double()).sum().backward()

    def close(name, got, want):
        got, want = got.detach().double().cpu().numpy(), want.detach().numpy()
        assert np.isfinite(got).all(), name
        if dtype == torch.float32:      # max-norm
            err, scale = np.abs(got - want).max(), np.abs(want).max()
        else:                           # bf16 layer: PyTorch's own bf16 linear / norm / relu steps flip single relu
            err, scale = np.linalg.norm(got - want), np.linalg.norm(want)   # gates, so the 2-norm is compared
        assert err <= tol * max(scale, 1e-30), "%s: %.3e vs scale %.3e" % (name, err, scale)

    close("output", y, yr)
    close("d tokens", x.grad, xr.grad)
    for li, l in enumerate(enc_d.layers):
        sd = dict(l.named_parameters())
        for a, b in NAMES.items():
            close("layer %d d %s" % (li, a), sd[b].grad, ws[li][a].grad)


def test_fp32_layer_general_kernels():
    import torch
    _run(n=32, k=2, left_only=False, D=64, H=2, F=96, n_layers=2, dtype=torch.float32, lengths=None, readout="tokens", tol=2e-4)


def test_fp32_left_only_with_lengths_root_readout():
    import torch
    _run(n=32, k=3, left_only=True, D=64, H=2, F=64, n_layers=1, dtype=torch.float32, lengths=[32, 19], readout="root", tol=2e-4)


def test_bf16_layer_tiled_kernels(monkeypatch):
    """The layer in bf16 runs the tiled kernels with lengths.  What those kernels produce inside the layer is
    compared element by element: the attention's inputs and output are recorded on the way through the layer
    and the oracle is evaluated on exactly those inputs.  The layer's own output and parameter gradients also pass
    through PyTorch's bf16 linear / norm / relu operators and are held to a 2-norm bound only."""
    import torch
    from oracle import ctwin
    from paper_1911_04070_b200 import binding, layer
    from parity import TOL, assert_close
    seen = []
    real_fwd, real_bwd = binding.bpt_attn_fwd, binding.bpt_attn_bwd

    def rec_fwd(g, q, k, v, rel_emb, scale, **kw):
        out, lse = real_fwd(g, q, k, v, rel_emb, scale, **kw)
        seen.append(dict(kind="fwd", g=g, q=q, k=k, v=v, r=rel_emb, scale=scale, lengths=kw.get("lengths"), out=out, lse=lse))
        return out, lse

    def rec_bwd(g, q, k, v, rel_emb, scale, out, lse, d_out, **kw):
        grads = real_bwd(g, q, k, v, rel_emb, scale, out, lse, d_out, **kw)
        seen.append(dict(kind="bwd", g=g, q=q, k=k, v=v, r=rel_emb, scale=scale, lengths=kw.get("lengths"), out=out,
                         d_out=d_out, grads=grads))
        return grads

    monkeypatch.setattr(binding, "bpt_attn_fwd", rec_fwd)
    monkeypatch.setattr(binding, "bpt_attn_bwd", rec_bwd)
    _run(n=128, k=4, left_only=False, D=128, H=2, F=128, n_layers=1, dtype=torch.bfloat16, lengths=[128, 77], readout="tokens", tol=1e-1)
    assert [s["kind"] for s in seen] == ["fwd", "bwd"]
    f64 = lambda t: t.detach().float().cpu().numpy().astype(np.float64)
    for s in seen:
        ref = ctwin.CGraph(s["g"].n, s["g"].k, 0)
        lens = s["lengths"].cpu().numpy()
        q, k, v, r = (f64(s[a]) for a in ("q", "k", "v", "r"))
        if s["kind"] == "fwd":
            o_ref, lse_ref = ctwin.attn_fwd_varlen(ref, q, k, v, r, s["scale"], lens)
            assert_close("attention out inside the layer", f64(s["out"]), o_ref, TOL["bf16"])
            assert_close("attention lse inside the layer", f64(s["lse"]), lse_ref, TOL["bf16"])
        else:
            want = ctwin.attn_bwd_varlen(ref, q, k, v, r, s["scale"], f64(s["d_out"]), lens, out=f64(s["out"]))
            fa = 1 + 2 * ref.L * (s["g"].k + 1)
            for name, a, b in zip(("dq", "dk", "dv"), s["grads"][:3], want[:3]):
                assert_close("attention %s inside the layer" % name, f64(a), b, TOL["bf16"], row_rms=True)
            assert_close("attention d_rel inside the layer", f64(s["grads"][3])[:fa], want[3][:fa], TOL["bf16"])
