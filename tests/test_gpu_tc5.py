"""The tensor-memory (tcgen05) forward kernel for the token rows, selected with BPT_FWD_TOKENS=tc5.

The choice is read once per process, so these cases run in a child process with the variable set;
the child compares the forward output with the fp64 oracle exactly as the other parity tests do."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %(root)r); sys.path.insert(0, %(tests)r)
import numpy as np, torch
from oracle import ctwin
from paper_1911_04070_b200 import binding, synth
from parity import TOL, assert_close
cases = [(128, 64, 0, 2, 2), (256, 4, 0, 2, 9), (256, 33, 1, 1, 3), (512, 63, 2, 1, 2), (2048, 3, 3, 1, 2),
         (4096, 64, 0, 1, 1), (8192, 64, 1, 1, 8), (16384, 4, 0, 1, 2)]
for n, k, flags, B, H in cases:
    ref = ctwin.CGraph(n, k, flags)
    x = synth.make_inputs(B, ref.n_nodes, H, 64, ref.n_rel, seed=7 + n + k, std_qkv=0.5, std_rel=0.3, bf16=True, with_grad=False)
    g = binding.bpt_build_graph(n, k, flags, device="cuda:0", with_transpose=False)
    t = {a: torch.from_numpy(b).to("cuda:0", torch.bfloat16) for a, b in x.items()}
    ws = torch.zeros(binding.bpt_attn_workspace_bytes(g, B, H, 64, binding.BPT_BF16, False), dtype=torch.uint8, device="cuda:0")
    binding.bpt_trace_begin(8)
    out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125, workspace=ws)
    names = [a for a, _ in binding.bpt_trace_end(8)]
    assert "fwd_tc5" in names, names          # the tensor-memory kernel really ran
    assert binding.bpt_forward_status(ws) == 0   # no bounded wait gave up
    o_ref, lse_ref = ctwin.attn_fwd(ref, x["q"], x["k"], x["v"], x["rel_emb"], 0.125)
    assert_close("out", out.float().cpu().numpy(), o_ref, TOL["bf16"])
    assert_close("lse", lse.cpu().numpy(), lse_ref, TOL["bf16"])
    out2, lse2 = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], 0.125)
    assert torch.equal(out, out2) and torch.equal(lse, lse2)
print("tc5 cases ok")
"""


def test_tensor_memory_forward_matches_oracle():
    env = dict(os.environ, BPT_FWD_TOKENS="tc5")
    code = CHILD % {"root": ROOT, "tests": os.path.join(ROOT, "tests")}
    res = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    assert "tc5 cases ok" in res.stdout
