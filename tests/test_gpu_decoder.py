"""BPTDecoder: decoding a sequence token by token with cached per-layer state gives the token rows of a full
forward pass of the left-only encoder over the finished sequence (autoregressive use, Sec. 4.2), and both
agree with the fp64 layer oracle."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

NAMES = {"wq": "wq.weight", "wk": "wk.weight", "wv": "wv.weight", "wo": "wo.weight", "rel_emb": "rel_emb",
         "ln1_w": "norm1.weight", "ln1_b": "norm1.bias", "ln2_w": "norm2.weight", "ln2_b": "norm2.bias",
         "ff1_w": "ff1.weight", "ff1_b": "ff1.bias", "ff2_w": "ff2.weight", "ff2_b": "ff2.bias"}


@pytest.mark.parametrize("n,k,n_layers", [(64, 3, 2), (256, 2, 1)])
def test_step_by_step_decoding_reproduces_the_full_forward(n, k, n_layers):
    import torch
    from oracle import bpt_layer, bpt_oracle as orc
    from paper_1911_04070_b200 import layer
    torch.manual_seed(1)
    B, D, H, F = 2, 64, 2, 96
    enc = layer.BPTEncoder(n, k, D, H, F, n_layers, left_only=True, device="cuda:0").to("cuda:0").eval()
    with torch.no_grad():
        for l in enc.layers:
            l.rel_emb.mul_(10.0)            # relation embeddings large enough to matter
    tokens = torch.randn(B, n, D, device="cuda:0")
    with torch.no_grad():
        full = enc(tokens, readout="tokens")
    dec = layer.BPTDecoder(enc, B)
    steps = torch.stack([dec.step(tokens[:, i]) for i in range(n)], dim=1)
    assert dec.pos == n
    with pytest.raises(ValueError):
        dec.step(tokens[:, 0])
    # same kernels row by row, same operators on fewer rows: equal up to the rounding order of the dense operators
    err = (steps - full).abs().max().item()
    assert err <= 2e-5 * full.abs().max().item(), err
    # and both match the fp64 oracle of the layer stack over the whole sequence
    ref_g = orc.enumerate_graph(n, k, 1)
    ws = []
    for l in enc.layers:
        sd = dict(l.named_parameters())
        ws.append({a: sd[b].detach().double().cpu() for a, b in NAMES.items()})
    want = bpt_layer.encoder_forward(tokens.double().cpu(), ws, ref_g, H, None, "tokens").numpy()
    got = steps.double().cpu().numpy()
    assert np.abs(got - want).max() <= 2e-4 * np.abs(want).max()


def test_decoder_needs_the_left_only_graph():
    import torch
    from paper_1911_04070_b200 import layer
    enc = layer.BPTEncoder(32, 2, 32, 1, 32, 1, left_only=False, device="cuda:0").to("cuda:0")
    with pytest.raises(ValueError):
        layer.BPTDecoder(enc, 1)
