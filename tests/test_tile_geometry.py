"""Size bounds the tiled kernels rely on (shared-memory tiles, partial-row workspace, tensor-memory
columns), checked by brute force with the oracle's per-token context lists (Sec. 3.2.2):

* the nodes T consecutive tokens attend at one (side, level), with the self loop counted into the
  level-0 left range, span at most (T >> level) + min(k, n) + 3 consecutive node indices (T = 64: rows
  reserved per chunk in the backward workspace; T = 128: the tensor-memory forward stages at most 208 rows);
* 32 consecutive tokens reach at most 32 + k + 2 node indices per (side, level), so four 32-column
  pieces starting at a multiple of 8 cover a warp's rows in the tensor-memory forward;
* both ends of a token's range are non-decreasing in the token index (the per-tile range table of the
  backward is searched by bisection)."""
import pytest

from oracle import bpt_oracle as orc


def _ranges(n, k, pad, i):
    """{(side, level): (lo, hi)} of token i; the self loop extends the level-0 left range to i."""
    out = {}
    for side, ctx in ((0, orc.left_context(n, k, i, pad)), (1, orc.right_context(n, k, i, pad))):
        for (l, m, _o) in ctx:
            lo, hi = out.get((side, l), (m, m))
            out[(side, l)] = (min(lo, m), max(hi, m))
    lo, hi = out.get((0, 0), (i, i))
    out[(0, 0)] = (min(lo, i), i)
    return out


@pytest.mark.parametrize("n", [64, 128, 512, 2048])
@pytest.mark.parametrize("pad", [True, False])
def test_union_ranges_fit_the_reserved_sizes(n, pad):
    for k in (1, 2, 3, 4, 7, 8, 16, 31, 33, 63, 64):
        kc = min(k, n)
        per_token = [_ranges(n, k, pad, i) for i in range(n)]
        for T in (32, 64, 128):
            if T > n:
                continue
            for t0 in range(0, n, T):
                union = {}
                for i in range(t0, t0 + T):
                    for key, (lo, hi) in per_token[i].items():
                        a, b = union.get(key, (lo, hi))
                        union[key] = (min(a, lo), max(b, hi))
                for (side, level), (lo, hi) in union.items():
                    if T == 32:
                        assert hi - lo + 1 <= 32 + kc + 2, (n, k, pad, t0, side, level)
                    else:
                        assert hi - lo + 1 <= (T >> level) + kc + 3, (n, k, pad, T, t0, side, level)
                        if T == 128 and k <= 64:
                            assert ((hi - lo + 1 + 15) & ~15) <= 208
        for key in set().union(*[set(r) for r in per_token]):      # monotone ends over the tokens that have the level
            prev = None
            for i in range(n):
                if key in per_token[i]:
                    if prev is not None:
                        assert per_token[i][key][0] >= prev[0] and per_token[i][key][1] >= prev[1], (n, k, pad, key, i)
                    prev = per_token[i][key]
