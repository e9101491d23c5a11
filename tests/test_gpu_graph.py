"""GPU graph builder vs the oracle: bit-exact CSR and by-source lists."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

CASES = [
    (2, 1, 0), (2, 5, 0), (4, 1, 1), (8, 1, 0), (8, 1, 2), (8, 2, 0), (16, 2, 3), (64, 3, 0), (64, 70, 0),
    (128, 5, 1), (256, 4, 0), (512, 4, 0), (512, 128, 1), (1024, 16, 2), (2048, 8, 0), (4096, 1, 0),
    (8192, 64, 1), (8192, 64, 0), (16384, 16, 0), (65536, 64, 0), (1 << 20, 1, 0),
]


@pytest.mark.parametrize("n,k,flags", CASES)
def test_graph_bit_exact(n, k, flags):
    import torch
    from oracle import ctwin
    from paper_1911_04070_b200 import binding
    g = binding.bpt_build_graph(n, k, flags, device="cuda:0")
    torch.cuda.synchronize()
    ref = ctwin.CGraph(n, k, flags)
    assert g.n_edges == ref.n_edges and g.n_rel == ref.n_rel and g.n_nodes == ref.n_nodes
    for name in ("row_ptr", "col", "rel", "t_ptr", "t_dst", "t_eid"):
        got = getattr(g, name).cpu().numpy()
        assert np.array_equal(got, getattr(ref, name)), name


def test_small_graphs_against_numpy_oracle():
    import torch
    from oracle import bpt_oracle as orc
    from paper_1911_04070_b200 import binding
    for n in (2, 4, 8, 16, 32):
        for k in (1, 2, 3, 7, 40):
            for flags in (0, 1, 2, 3):
                g = binding.bpt_build_graph(n, k, flags, device="cuda:0")
                ref = orc.enumerate_graph(n, k, flags)
                for name in ("row_ptr", "col", "rel", "t_ptr", "t_dst", "t_eid"):
                    assert np.array_equal(getattr(g, name).cpu().numpy(), getattr(ref, name)), (n, k, flags, name)


def test_forward_only_graph_and_bad_arguments():
    import ctypes
    import torch
    from paper_1911_04070_b200 import binding
    g = binding.bpt_build_graph(64, 2, 0, device="cuda:0", with_transpose=False)
    assert g.t_ptr is None and g.c.t_ptr is None
    lib = binding.load_library()
    dims = binding.bpt_graph_dims_query(64, 2, 0)
    bad = binding.GraphStruct()
    ws = torch.empty(256, dtype=torch.uint8, device="cuda:0")
    # missing outputs / workspace, inconsistent dims: refused on the host
    assert lib.bpt_build_graph(ctypes.byref(dims), None, None, None, None, None, None, ws.data_ptr(), None, ctypes.byref(bad)) == 1
    assert lib.bpt_build_graph(ctypes.byref(dims), g.row_ptr.data_ptr(), g.col.data_ptr(), g.rel.data_ptr(),
                               None, None, None, None, None, ctypes.byref(bad)) == 3
    dims.n_edges += 1
    assert lib.bpt_build_graph(ctypes.byref(dims), g.row_ptr.data_ptr(), g.col.data_ptr(), g.rel.data_ptr(),
                               None, None, None, ws.data_ptr(), None, ctypes.byref(bad)) == 1
