// Geometry shared by the tiled (leaf-block) kernels: per token row and per
// (side, level) chunk, the contiguous range of nodes the token attends
// (arXiv 1911.04070, Sec. 3.2.2), kept in shared memory for a tile of 64 tokens.
#pragma once
#include "bpt_tree.cuh"

namespace bpt {

constexpr int kTileTokens = 64;  // tokens per CTA (4 warps x 16 rows)
constexpr int kTileMaxK = 64;    // largest k the tiled kernels stage (k + 2 relation rows, k + 67 nodes per level)

// The tiled kernels cover bf16, head size 64, at least one full tile of tokens and k <= 64;
// everything else runs on the general row kernels.
inline bool tile_path(int n, int k, int d, bool bf16) { return bf16 && d == 64 && n >= kTileTokens && k <= kTileMaxK; }

// Number of levels that carry left / right contextual nodes for at least one token.
inline void context_levels(const TreeParams& t, int* n_left, int* n_right) {
    int nl = 0, nr = 0;
    for (LeftWalk w(t, t.n - 1); w.valid(); w.next()) nl = w.l + 1;
    if (!t.left_only)
        for (RightWalk w(t, 0); w.valid(); w.next()) nr = w.l + 1;
    *n_left = nl;
    *n_right = nr;
}

// bnd[c * TILE + r] = (first, last) node index at the chunk's level that token t0 + r attends;
// chunks 0..n_left-1 are the left levels, n_left..n_left+n_right-1 the right levels.
// Rows that do not reach a level get an empty range that keeps the bounds monotone in r.
template <int TILE = kTileTokens>
__device__ __forceinline__ void fill_row_bounds(const TreeParams& t, int t0, int r, int n_left, int n_right, int2* bnd) {
    {
        LeftWalk w(t, t0 + r);
        for (int c = 0; c < n_left; ++c) {
            int2 v = make_int2(0, -1);
            if (w.valid()) { v = make_int2(w.lo, w.hi); w.next(); }
            bnd[c * TILE + r] = v;
        }
    }
    {
        RightWalk w(t, t0 + r);
        for (int c = 0; c < n_right; ++c) {
            const int n_l = t.n >> c;
            int2 v = make_int2(n_l, n_l - 1);
            if (w.valid()) { v = make_int2(w.lo, w.hi); w.next(); }
            bnd[(n_left + c) * TILE + r] = v;
        }
    }
}

// Sequences shorter than n: the first `len` tokens are real, a node is real when it covers a real
// token, i.e. node (level, m) with m <= (len - 1) >> level; edges that touch other nodes do not exist.
__device__ __forceinline__ int seq_len(const int32_t* lengths, int b, int n) {
    return lengths ? min(max(lengths[b], 0), n) : n;
}

// Applies a length to the row ranges fill_row_bounds wrote for token t0 + r: a placeholder token
// attends nothing; a real token's right-side ranges end at the last real node of the level (left-side
// nodes lie before the token and are real).  Empty ranges keep the encoding of fill_row_bounds.
template <int TILE = kTileTokens>
__device__ __forceinline__ void mask_row_bounds(const TreeParams& t, int t0, int r, int n_left, int n_right, int2* bnd, int len) {
    if (len >= t.n) return;
    const bool real = t0 + r < len;
    for (int c = 0; c < n_left; ++c)
        if (!real) bnd[c * TILE + r] = make_int2(0, -1);
    for (int c = 0; c < n_right; ++c) {
        const int n_l = t.n >> c;
        int2 v = bnd[(n_left + c) * TILE + r];
        if (real && v.x <= v.y) v.y = min(v.y, (len - 1) >> c);
        if (!real || v.x > v.y) v = make_int2(n_l, n_l - 1);
        bnd[(n_left + c) * TILE + r] = v;
    }
}

// Union of the non-empty ranges of rows [r0, r0 + cnt) of one chunk (lanes 0..cnt-1 each
// look at one row; cnt <= 32).  Returns (lo, hi) with lo > hi when all rows are empty.
__device__ __forceinline__ int2 rows_union(const int2* bnd_chunk, int r0, int cnt, int lane) {
    int lo = 0x7fffffff, hi = -1;
    if (lane < cnt) {
        const int2 v = bnd_chunk[r0 + lane];
        if (v.x <= v.y) { lo = v.x; hi = v.y; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    return make_int2(lo, hi);
}

}  // namespace bpt
