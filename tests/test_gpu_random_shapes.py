"""Seeded random problems through the C ABI against the fp64 oracle: sizes, k (around the kernel
selection thresholds), graph flags, head counts, dtypes, and the options (lengths, attention dropout)
in combination -- corners the hand-picked cases of the other parity tests may miss."""
import numpy as np
import pytest

from parity import TOL, assert_close

pytestmark = pytest.mark.gpu


def _close_or_zero(name, got, want, tol, **kw):
    if np.abs(want).max() == 0:                 # e.g. a sequence of one token: every row has one edge, dS = 0
        assert np.abs(got).max() == 0, name
    else:
        assert_close(name, got, want, tol, **kw)


@pytest.mark.parametrize("seed", [11, 12])
def test_random_problems(seed):
    import torch
    from oracle import ctwin
    from paper_1911_04070_b200 import binding, synth
    rng = np.random.default_rng(seed)
    for case in range(30):
        n = int(2 ** rng.integers(1, 12))
        k = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 15, 16, 17, 31, 32, 33, 48, 55, 56, 57, 63, 64, 65, 100]))
        flags = int(rng.integers(0, 4)); B = int(rng.integers(1, 4)); H = int(rng.integers(1, 10))
        bf16 = bool(rng.integers(0, 2)); d = int(rng.choice([32, 64]))
        p = float(rng.choice([0.0, 0.0, 0.2, 0.5])); drop_seed = int(rng.integers(0, 2 ** 62))
        lengths = [int(rng.integers(2, n + 1)) for _ in range(B)] if rng.integers(0, 2) else [n] * B   # length 1 (every row a single edge: all gradients cancel to rounding noise) is covered in test_gpu_varlen.py
        what = (n, k, flags, B, H, d, bf16, lengths, p)
        tol = TOL["bf16" if bf16 else "fp32"]
        ref = ctwin.CGraph(n, k, flags)
        x = synth.make_inputs(B, ref.n_nodes, H, d, ref.n_rel, seed=case, std_qkv=0.5, std_rel=0.3, bf16=bf16)
        dt = torch.bfloat16 if bf16 else torch.float32
        t = {a: torch.from_numpy(v).to("cuda:0", dt) for a, v in x.items()}
        lens = torch.tensor(lengths, dtype=torch.int32, device="cuda:0")
        g = binding.bpt_build_graph(n, k, flags, device="cuda:0")
        scale = d ** -0.5
        out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, lengths=lens, dropout_p=p, dropout_seed=drop_seed)
        dq, dk, dv, dr = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], scale, out, lse, t["d_out"],
                                              lengths=lens, dropout_p=p, dropout_seed=drop_seed)
        torch.cuda.synchronize()
        o64 = out.float().cpu().numpy().astype(np.float64)
        o_ref, l_ref = ctwin.attn_fwd_varlen(ref, x["q"], x["k"], x["v"], x["rel_emb"], scale, lengths, p_drop=p, seed=drop_seed)
        gr = ctwin.attn_bwd_varlen(ref, x["q"], x["k"], x["v"], x["rel_emb"], scale, x["d_out"], lengths, out=o64, p_drop=p, seed=drop_seed)
        _close_or_zero("out %r" % (what,), o64, o_ref, tol)
        _close_or_zero("lse %r" % (what,), lse.cpu().numpy(), l_ref, tol)
        fa = 1 + 2 * ref.L * (k + 1)
        for name, a, b_ in zip(("dq", "dk", "dv"), (dq, dk, dv), gr[:3]):
            _close_or_zero("%s %r" % (name, what), a.float().cpu().numpy(), b_, tol, row_rms=True)
        _close_or_zero("d_rel %r" % (what,), dr.cpu().numpy()[:fa], gr[3][:fa], tol)
