"""Pins for the oracle's graph enumeration (Sec. 3.2, Algorithm 1, Sec. 3.4).

Each test checks the enumeration against something the paper or plain
combinatorics fixes, not against the enumeration itself.
"""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import bpt_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(g):
    return [(g.col[g.row_ptr[u]:g.row_ptr[u + 1]], g.rel[g.row_ptr[u]:g.row_ptr[u + 1]]) for u in range(g.n_nodes)]


def _span_tokens(n, u):
    l, m = orc.node_level_index(n, u)
    return range(m << l, (m + 1) << l)


def test_node_ids_are_level_major():
    n = 16
    ids = [orc.node_id(n, l, m) for l in range(5) for m in range(n >> l)]
    assert ids == list(range(2 * n - 1))                      # 2n-1 partitions, Sec. 3.2.1
    for u in ids:
        l, m = orc.node_level_index(n, u)
        assert orc.node_id(n, l, m) == u


def test_worked_example_n8_k1():
    want = {}
    for line in open(os.path.join(GOLD, "graph_n8_k1_pad_bidir.txt")):
        if line.startswith("#") or not line.strip():
            continue
        tok, rest = line.split(":")
        left, right = rest.split("|")
        parse = lambda s: [tuple(int(x) for x in t.split(",")) for t in s.split()]
        want[int(tok)] = (parse(left), parse(right))
    for i in range(8):
        left = [(l, m) for (l, m, o) in orc.left_context(8, 1, i, True)]
        right = [(l, m) for (l, m, o) in orc.right_context(8, 1, i, True)]
        assert (left, right) == want[i]
        # joining order defines the offsets 0, 1, ... inside every level (Sec. 3.4)
        for ctx in (orc.left_context(8, 1, i, True), orc.right_context(8, 1, i, True)):
            for lvl, grp in itertools.groupby(ctx, key=lambda t: t[0]):
                assert [o for (_, _, o) in grp] == list(range(len([1 for t in ctx if t[0] == lvl])))


def test_edge_counts_golden():
    for line in open(os.path.join(GOLD, "edge_counts.txt")):
        if line.startswith("#") or not line.strip():
            continue
        n, k, flags, e_ctx, e_tot = (int(x) for x in line.split())
        g = orc.enumerate_graph(n, k, flags)
        assert g.n_edges == e_tot
        assert g.n_edges - n - n * g.L == e_ctx


@pytest.mark.parametrize("n", [2, 4, 8, 16, 32, 64, 128])
def test_pad_graph_partitions_each_side(n):
    """Sec. 3 opening: a token's context is grouped into non-overlapping spans
    whose scale grows with distance.  With the pad rule the nodes on each side
    tile that side's tokens exactly once; levels are consecutive from 0, each
    non-final level holds k or k+1 nodes and ends on a whole-parent boundary."""
    for k in range(1, min(n, 19) + 1):
        for i in range(n):
            for side, ctx in (("R", orc.right_context(n, k, i, True)), ("L", orc.left_context(n, k, i, True))):
                cover = np.zeros(n, dtype=int)
                levels = {}
                for (l, m, o) in ctx:
                    assert 0 <= m < (n >> l)
                    cover[m << l:(m + 1) << l] += 1
                    levels.setdefault(l, []).append(m)
                want = np.zeros(n, dtype=int)
                if side == "R":
                    want[i + 1:] = 1
                else:
                    want[:i] = 1
                assert np.array_equal(cover, want), (n, k, i, side)
                if not levels:
                    continue
                assert sorted(levels) == list(range(max(levels) + 1))
                prev_extent = None
                for l in sorted(levels):
                    ms = levels[l]
                    far = max(ms) if side == "R" else min(ms)
                    assert sorted(ms) == list(range(min(ms), max(ms) + 1))      # contiguous
                    if l != max(levels):
                        assert len(ms) in (k, k + 1)
                        assert far % 2 == (1 if side == "R" else 0)
                    else:
                        assert len(ms) <= k + 1
                    # fine -> coarse: each level lies beyond the previous one
                    lo_tok, hi_tok = min(ms) << l, ((max(ms) + 1) << l) - 1
                    if prev_extent is not None:
                        if side == "R":
                            assert lo_tok == prev_extent + 1
                        else:
                            assert hi_tok == prev_extent - 1
                    prev_extent = hi_tok if side == "R" else lo_tok


@pytest.mark.parametrize("n", [4, 8, 16, 32, 64])
def test_alg1_graph_exactly_k_per_level(n):
    """Algorithm 1 literal: k steps per level then parent(); every token of the
    side is covered at least once, the token itself never."""
    for k in range(1, min(n, 9) + 1):
        for i in range(n):
            ctx = orc.right_context(n, k, i, False)
            cover = np.zeros(n, dtype=int)
            levels = {}
            for (l, m, o) in ctx:
                cover[m << l:(m + 1) << l] += 1
                levels.setdefault(l, []).append(m)
            assert (cover[i + 1:] >= 1).all() and (cover[:i + 1] == 0).all()
            p = i + 1
            for l in sorted(levels):
                assert levels[l][0] == p                          # p_l = parent(p_{l-1} + k)
                if l != max(levels):
                    assert len(levels[l]) == k
                p = (p + k) >> 1
            lctx = orc.left_context(n, k, i, False)
            cover = np.zeros(n, dtype=int)
            for (l, m, o) in lctx:
                cover[m << l:(m + 1) << l] += 1
            assert (cover[:i] >= 1).all() and (cover[i:] == 0).all()


@pytest.mark.parametrize("flags", [0, orc.LEFT_ONLY, orc.MODE_ALG1, orc.MODE_ALG1 | orc.LEFT_ONLY])
def test_csr_structure(flags):
    n, k = 32, 3
    g = orc.enumerate_graph(n, k, flags)
    L = g.L
    assert g.n_nodes == 2 * n - 1 and g.row_ptr[0] == 0 and g.row_ptr[-1] == g.n_edges
    rows = _rows(g)
    for u, (cols, rels) in enumerate(rows):
        assert (np.diff(cols) > 0).all()                          # ascending, unique
        l, m = orc.node_level_index(n, u)
        if l == 0:
            assert (cols == u).sum() == 1                         # self loop (Algorithm 1: N <- {u})
            assert rels[list(cols).index(u)] == orc.rel_self()
            for c in cols:                                        # never an ancestor of the token
                if c != u:
                    assert u not in _span_tokens(n, c)
            if flags & orc.LEFT_ONLY:                             # causal: every source lies to the left
                for c in cols:
                    assert max(_span_tokens(n, c)) <= u
        else:
            assert list(cols) == list(range(m << l, (m + 1) << l))   # 2^l affiliated edges, Sec. 3.2.2
            assert (rels == orc.rel_anc(L, k, l)).all()
    # relation labels: distinct per (side, level, offset), inside the table
    assert g.rel.min() >= 0 and g.rel.max() < g.n_rel == 1 + 2 * L * (k + 1) + L
    for i in range(n):
        seen = {}
        pad = not (flags & orc.MODE_ALG1)
        for (l, m, o) in orc.left_context(n, k, i, pad):
            seen[orc.node_id(n, l, m)] = orc.rel_left(L, k, l, o)
        if not (flags & orc.LEFT_ONLY):
            for (l, m, o) in orc.right_context(n, k, i, pad):
                seen[orc.node_id(n, l, m)] = orc.rel_right(L, k, l, o)
        cols, rels = rows[i]
        assert len(set(seen.values())) == len(seen)
        for c, r in zip(cols, rels):
            if c != i:
                assert seen[c] == r
    ids = {orc.rel_self()} | {orc.rel_left(L, k, j, o) for j in range(L) for o in range(k + 1)} \
        | {orc.rel_right(L, k, j, o) for j in range(L) for o in range(k + 1)} | {orc.rel_anc(L, k, j) for j in range(1, L + 1)}
    assert ids == set(range(g.n_rel))


@pytest.mark.parametrize("flags", [0, orc.LEFT_ONLY])
def test_token_distance_at_most_two(flags):
    """Sec. 3.2.2 / 3.3: any two tokens are joined by at most two edges, i.e.
    b attends a directly or attends a span containing a."""
    for n, k in [(8, 1), (16, 2), (64, 1), (64, 3), (32, 5)]:
        g = orc.enumerate_graph(n, k, flags)
        rows = _rows(g)
        for b in range(n):
            reach = set()
            for c in rows[b][0]:
                reach.update(_span_tokens(n, c))
            want = set(range(b + 1)) if flags & orc.LEFT_ONLY else set(range(n))
            assert want <= reach


def test_edge_count_growth():
    """Number of edges is O(k n log(n/k)) (abstract, Sec. 3.2.2)."""
    for n in (256, 1024, 4096):
        for k in (1, 4, 16, 64):
            e_ctx = sum(len(orc.right_context(n, k, i, True)) + len(orc.left_context(n, k, i, True)) for i in range(0, n, 7))
            cnt = len(range(0, n, 7))
            bound = cnt * 2 * (k + 1) * (math.floor(math.log2(n / k)) + 1)
            assert e_ctx <= bound
            assert e_ctx >= 0.25 * cnt * 2 * k * max(1.0, math.log2(n / k))


def test_k_at_least_n_is_fully_connected():
    """Sec. 3.4 closing remark: k >= sentence length gives the vanilla Transformer."""
    n = 16
    for k in (n, n + 3):
        g = orc.enumerate_graph(n, k, 0)
        for i in range(n):
            cols = g.col[g.row_ptr[i]:g.row_ptr[i + 1]]
            assert list(cols) == list(range(n))


def test_transpose_is_consistent():
    g = orc.enumerate_graph(32, 2, 0)
    dst_of = np.repeat(np.arange(g.n_nodes), np.diff(g.row_ptr))
    for v in range(g.n_nodes):
        a, b = g.t_ptr[v], g.t_ptr[v + 1]
        assert (g.col[g.t_eid[a:b]] == v).all()
        assert (dst_of[g.t_eid[a:b]] == g.t_dst[a:b]).all()
        assert (np.diff(g.t_dst[a:b]) > 0).all()
    assert sorted(g.t_eid.tolist()) == list(range(g.n_edges))
    # a token feeds its L ancestors, one per level (Sec. 3.2.2 affiliated edges)
    for j in range(32):
        anc = [u for u in g.t_dst[g.t_ptr[j]:g.t_ptr[j + 1]] if u >= 32]
        assert anc == [orc.node_id(32, l, j >> l) for l in range(1, g.L + 1)]
