"""The index-checking build (libbpt_check.so, -DBPT_BOUNDS_CHECK): every gather index and CSR offset is tested
before the access, a violation is recorded instead of trapping.  Tiny cases -- every n <= 64 with every k <= n --
run through it in a child process (the library path is chosen before the first call); the record must stay empty
and the results must be those of the normal build, bit for bit."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %(root)r)
import torch
from paper_1911_04070_b200 import binding, synth
if %(check)d:
    binding.LIB_PATH = binding.CHECK_LIB_PATH
results = []
shapes = [(n, k, flags) for n in (2, 4, 8, 16, 32, 64) for k in range(1, n + 1) for flags in (0, 1)
          if k <= 4 or k %% 7 == 0 or k == n] + [(64, 5, 2), (64, 64, 3), (256, 9, 0), (512, 64, 1)]
for n, k, flags in shapes:
    g = binding.bpt_build_graph(n, k, flags, device="cuda:0")
    for bf16, d in ((False, 32), (True, 64)):
        if n < 8 and bf16:
            continue
        x = synth.make_inputs(2, g.n_nodes, 2, d, g.n_rel, seed=n + k, std_qkv=0.5, std_rel=0.3, bf16=bf16)
        dt = torch.bfloat16 if bf16 else torch.float32
        t = {a: torch.from_numpy(b).to("cuda:0", dt) for a, b in x.items()}
        for path in ((0, 2) if (bf16 and n >= 128) else (0,)):
            out, lse = binding.bpt_attn_fwd(g, t["q"], t["k"], t["v"], t["rel_emb"], d ** -0.5, path=path)
            grads = binding.bpt_attn_bwd(g, t["q"], t["k"], t["v"], t["rel_emb"], d ** -0.5, out, lse, t["d_out"], path=path)
            results.append([z.float().cpu() for z in (out, lse) + tuple(grads)])
    results.append([g.col.cpu().float(), g.rel.cpu().float(), g.t_dst.cpu().float(), g.t_eid.cpu().float()])
if %(check)d:
    rec = binding.bpt_debug_bounds()
    assert rec == (0, 0, 0, 0), rec
    print("violations", rec[0])
else:
    try:
        binding.bpt_debug_bounds()
        raise SystemExit("the normal build must not answer bpt_debug_bounds")
    except binding.BptError as e:
        assert e.status == 2
torch.save(results, %(dump)r)
print("cases", len(results))
"""


def _run(check, dump):
    code = CHILD % {"root": ROOT, "check": check, "dump": dump}
    res = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-2000:] + res.stderr[-4000:]
    return res.stdout


def test_tiny_cases_leave_the_record_empty_and_match_the_normal_build(tmp_path):
    import torch
    out = _run(1, str(tmp_path / "check.pt"))
    assert "violations 0" in out
    _run(0, str(tmp_path / "plain.pt"))
    a, b = torch.load(tmp_path / "check.pt"), torch.load(tmp_path / "plain.pt")
    assert len(a) == len(b) > 100
    for x, y in zip(a, b):
        for u, v in zip(x, y):
            assert torch.equal(u, v)
