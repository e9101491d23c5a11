// Index arithmetic of the binary partition tree and of a token's contextual
// nodes (arXiv 1911.04070, Sec. 3.2).  Host + device, integers only.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#define BPT_HD __host__ __device__ __forceinline__

namespace bpt {

constexpr int kMaxLevels = 21;  // n <= 2^20

struct TreeParams {
    int n;      // tokens
    int L;      // log2 n
    int k;      // connection density (relation ids use W = k + 1)
    int kc;     // min(k, n): same ranges after clipping, no overflow
    int pad;    // 1: pad rule of Sec. 3.2.2, 0: Algorithm 1 literal
    int left_only;
};

BPT_HD int node_id(int n, int l, int m) { return 2 * n - ((2 * n) >> l) + m; }

// level of node id u (0 = token)
BPT_HD int node_level(int n, int u) {
    int l = 0, base = 0, width = n;
    while (u >= base + width) { base += width; width >>= 1; ++l; }
    return l;
}

// first token covered by node id u
BPT_HD int node_first_token(int n, int u) {
    int l = 0, base = 0, width = n;
    while (u >= base + width) { base += width; width >>= 1; ++l; }
    return (u - base) << l;
}

BPT_HD int rel_left(const TreeParams& t, int j, int o) { return 1 + j * (t.k + 1) + o; }
BPT_HD int rel_right(const TreeParams& t, int j, int o) { return 1 + (t.L + j) * (t.k + 1) + o; }
BPT_HD int rel_anc(const TreeParams& t, int j) { return 1 + 2 * t.L * (t.k + 1) + (j - 1); }

// One side's walk over the levels (Sec. 3.2.2: start index p_0 = i + 1, k nodes per
// level, with the pad rule one more when the last node is a left child, then the
// parent of the next index).  Usage:
//   RightWalk w(t, i); while (w.valid()) { use w.l, w.lo..w.hi; w.next(); }
struct RightWalk {
    int l, lo, hi;
    bool ok;
    const TreeParams& t;
    BPT_HD RightWalk(const TreeParams& tp, int i) : l(0), lo(i + 1), hi(0), ok(true), t(tp) { settle(); }
    BPT_HD void settle() {
        const int nl = t.n >> l;
        if (lo >= nl) { ok = false; return; }
        hi = lo + t.kc - 1;
        if (t.pad && !(hi & 1)) ++hi;
        if (hi > nl - 1) hi = nl - 1;
    }
    BPT_HD bool valid() const { return ok; }
    BPT_HD void next() {
        const int nxt = hi + 1;
        if (nxt >= (t.n >> l)) { ok = false; return; }
        lo = nxt >> 1; ++l; settle();
    }
};

// Mirror image: nodes lo..hi with hi the nearest (first to join).
struct LeftWalk {
    int l, lo, hi;
    bool ok;
    const TreeParams& t;
    BPT_HD LeftWalk(const TreeParams& tp, int i) : l(0), lo(0), hi(i - 1), ok(true), t(tp) { settle(); }
    BPT_HD void settle() {
        if (hi < 0) { ok = false; return; }
        lo = hi - t.kc + 1;
        if (t.pad && (lo & 1)) --lo;
        if (lo < 0) lo = 0;
    }
    BPT_HD bool valid() const { return ok; }
    BPT_HD void next() {
        const int nxt = lo - 1;
        if (nxt < 0) { ok = false; return; }
        hi = nxt >> 1; ++l; settle();
    }
};

// Position inside token i's row (sources ascending by node id: level by level, inside a
// level left nodes ascending, then the token itself at level 0, then right nodes
// ascending) of the first node of (side, level), and how many nodes that block has.
// side: 0 = left, 1 = right, 2 = the self loop.  Returns false when the block is empty.
BPT_HD bool token_block(const TreeParams& t, int i, int side, int level, int* pos, int* cnt, int* first_m) {
    LeftWalk lw(t, i);
    RightWalk rw(t, i);
    const bool use_r = !t.left_only;
    int at = 0;
    for (int l = 0; l <= level; ++l) {
        const bool hl = lw.valid() && lw.l == l;
        const bool hr = use_r && rw.valid() && rw.l == l;
        const int cl = hl ? lw.hi - lw.lo + 1 : 0;
        const int cr = hr ? rw.hi - rw.lo + 1 : 0;
        if (l == level) {
            if (side == 0) { *pos = at; *cnt = cl; *first_m = hl ? lw.lo : 0; return cl > 0; }
            at += cl;
            if (side == 2) { *pos = at; *cnt = (l == 0); *first_m = i; return l == 0; }
            if (l == 0) ++at;
            *pos = at; *cnt = cr; *first_m = hr ? rw.lo : 0; return cr > 0;
        }
        at += cl + cr + (l == 0);
        if (hl) lw.next();
        if (hr) rw.next();
        if (!(lw.valid() || (use_r && rw.valid()))) break;
    }
    *pos = at; *cnt = 0; *first_m = 0;
    return false;
}

// Number of edges into token i.
BPT_HD int token_degree(const TreeParams& t, int i) {
    int deg = 1;
    for (LeftWalk w(t, i); w.valid(); w.next()) deg += w.hi - w.lo + 1;
    if (!t.left_only)
        for (RightWalk w(t, i); w.valid(); w.next()) deg += w.hi - w.lo + 1;
    return deg;
}

}  // namespace bpt
