"""The C-ABI library loads and exports every symbol include/bpt.h declares;
host-only entry points validate their arguments.  No GPU needed."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1911_04070_b200 import build, binding
    build.build()
    return binding.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "bpt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bpt_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_1911_04070_b200 import binding
    names = _declared()
    assert set(binding.EXPORTS) <= set(names)
    assert {"bpt_build_graph", "bpt_attn_fwd", "bpt_attn_bwd"} <= set(names)
    for name in names:
        assert getattr(lib, name) is not None, name


def test_dims_query_matches_closed_forms(lib):
    from paper_1911_04070_b200 import binding
    d = binding.bpt_graph_dims_query(8, 1, 0)
    assert (d.n_nodes, d.n_levels, d.n_edges, d.n_rel) == (15, 3, 68, 1 + 2 * 3 * 2 + 3)
    d = binding.bpt_graph_dims_query(8192, 64, binding.BPT_LEFT_ONLY)
    assert d.n_nodes == 16383 and d.n_rel == 1704 and d.n_edges > 8192 * 13


def test_argument_errors(lib):
    from paper_1911_04070_b200 import binding
    for args, status in [((7, 1, 0), 2), ((48, 4, 0), 2), ((8, 0, 0), 1), ((8, 1, 8), 1), ((1, 1, 0), 1), ((1 << 21, 1, 0), 2),
                         ((8, (1 << 20) + 1, 0), 2)]:
        with pytest.raises(binding.BptError) as ei:
            binding.bpt_graph_dims_query(*args)
        assert ei.value.status == status
    assert lib.bpt_graph_dims_query(8, 1, 0, None) == 1
    # null graph / bad head size are refused before any launch
    g = binding.GraphStruct()
    assert lib.bpt_attn_workspace_bytes(ctypes.byref(g), 1, 1, 64, 0, 0) == 0
    assert lib.bpt_attn_fwd(None, 1, 1, 64, 0, None, None, None, None, 1.0, None, None, None, 0, None) == 1
    assert binding.status_str(3) == "workspace missing or too small"
    assert lib.bpt_attn_bwd_min_workspace_bytes(ctypes.byref(g), 1, 1, 64, 0) == 0
    assert lib.bpt_selftest_wait_timeout(None, 1000, 0, None) == 1      # refused on the host: nothing is launched


def test_oracle_edge_count_agrees_with_host_query(lib):
    from oracle import ctwin
    from paper_1911_04070_b200 import binding
    for n, k, flags in [(2, 1, 0), (8, 3, 1), (256, 4, 0), (512, 600, 0), (2048, 8, 2), (8192, 64, 1)]:
        d = binding.bpt_graph_dims_query(n, k, flags)
        c = ctwin.CGraph(n, k, flags)
        assert d.n_edges == c.n_edges and d.n_rel == c.n_rel
