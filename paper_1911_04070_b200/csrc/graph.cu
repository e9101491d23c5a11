// Device-side builder of the BPT attention graph (arXiv 1911.04070, Sec. 3.2.2
// affiliated + contextual edges, Sec. 3.4 relation labels): CSR by destination and
// the by-source lists, bit-exact and without atomics.
#include "bounds_check.cuh"
#include "bpt_internal.cuh"

namespace bpt {

// ---------------------------------------------------------------------------------
// row_ptr
// ---------------------------------------------------------------------------------
__global__ void token_degree_kernel(TreeParams t, int32_t* __restrict__ row_ptr) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < t.n) row_ptr[i] = token_degree(t, i);
}

// In-place exclusive scan of a[0..len) by one block; a[len] receives the total.
__global__ void __launch_bounds__(1024) exclusive_scan_kernel(int32_t* __restrict__ a, int len) {
    __shared__ int32_t warp_sum[32];
    __shared__ int32_t block_carry;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int per = (len + blockDim.x - 1) / blockDim.x;
    const int beg = min(tid * per, len), end = min(beg + per, len);
    int32_t sum = 0;
    for (int j = beg; j < end; ++j) sum += a[j];
    int32_t incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    if (lane == 31) warp_sum[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        int32_t w = warp_sum[lane];
        int32_t wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t up = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += up;
        }
        warp_sum[lane] = wi - w;  // exclusive over warps
        if (lane == 31) block_carry = wi;
    }
    __syncthreads();
    int32_t run = warp_sum[wid] + incl - sum;
    for (int j = beg; j < end; ++j) {
        const int32_t x = a[j];
        a[j] = run;
        run += x;
    }
    if (tid == 0) a[len] = block_carry;
}

// Span rows: level l >= 1 occupies n consecutive edges after the token rows.
__global__ void span_row_ptr_kernel(TreeParams t, int32_t* __restrict__ row_ptr) {
    const int s = blockIdx.x * blockDim.x + threadIdx.x;  // span number 0..n-2, plus one for the end
    const int e_tok = row_ptr[t.n];
    if (s > t.n - 1) return;
    if (s == t.n - 1) { row_ptr[2 * t.n - 1] = e_tok + t.L * t.n; return; }
    const int u = t.n + s;
    const int l = node_level(t.n, u);
    const int m = u - node_id(t.n, l, 0);
    if (s > 0) row_ptr[u] = e_tok + (l - 1) * t.n + (m << l);  // s == 0 already holds e_tok
}

// ---------------------------------------------------------------------------------
// col / rel
// ---------------------------------------------------------------------------------
// One warp per token row.
__global__ void token_fill_kernel(TreeParams t, const int32_t* __restrict__ row_ptr,
                                  int32_t* __restrict__ col, int32_t* __restrict__ rel, int64_t E) {
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (i >= t.n) return;
    int at = row_ptr[i];
    LeftWalk lw(t, i);
    RightWalk rw(t, i);
    const bool use_r = !t.left_only;
    for (int l = 0; lw.valid() || (use_r && rw.valid()) || l == 0; ++l) {
        if (lw.valid()) {
            const int c = lw.hi - lw.lo + 1, base = node_id(t.n, l, lw.lo), r0 = rel_left(t, l, 0);
            for (int j = lane; j < c; j += 32)
                if (BPT_IDX_OK(at + j, E, BPT_SITE_GRAPH_WRITE)) { col[at + j] = base + j; rel[at + j] = r0 + (c - 1 - j); }
            at += c;
            lw.next();
        }
        if (l == 0) {
            if (lane == 0 && BPT_IDX_OK(at, E, BPT_SITE_GRAPH_WRITE)) { col[at] = i; rel[at] = 0; }
            ++at;
        }
        if (use_r && rw.valid()) {
            const int c = rw.hi - rw.lo + 1, base = node_id(t.n, l, rw.lo), r0 = rel_right(t, l, 0);
            for (int j = lane; j < c; j += 32)
                if (BPT_IDX_OK(at + j, E, BPT_SITE_GRAPH_WRITE)) { col[at + j] = base + j; rel[at + j] = r0 + j; }
            at += c;
            rw.next();
        }
    }
}

// Affiliated edges: inside level l the j-th edge comes from token j.
__global__ void span_fill_kernel(TreeParams t, const int32_t* __restrict__ row_ptr,
                                 int32_t* __restrict__ col, int32_t* __restrict__ rel, int64_t E) {
    const int64_t x = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= (int64_t)t.L * t.n) return;
    const int l = (int)(x / t.n) + 1, j = (int)(x % t.n);
    const int64_t e = (int64_t)row_ptr[t.n] + x;
    if (!BPT_IDX_OK(e, E, BPT_SITE_GRAPH_WRITE)) return;
    col[e] = j;
    rel[e] = rel_anc(t, l);
}

// ---------------------------------------------------------------------------------
// by-source lists
// ---------------------------------------------------------------------------------
// Tokens that see node (l, m) on their right form one interval, because the start and
// end index of a level are non-decreasing in the token index (and the level exists for a
// prefix of the tokens); likewise on the left (suffix).  Both ends by bisection.
__device__ bool right_level_range(const TreeParams& t, int i, int level, int* lo, int* hi) {
    RightWalk w(t, i);
    while (w.valid() && w.l < level) w.next();
    if (!w.valid()) return false;
    *lo = w.lo; *hi = w.hi;
    return true;
}
__device__ bool left_level_range(const TreeParams& t, int i, int level, int* lo, int* hi) {
    LeftWalk w(t, i);
    while (w.valid() && w.l < level) w.next();
    if (!w.valid()) return false;
    *lo = w.lo; *hi = w.hi;
    return true;
}

// tokens i (all < first token of the node) that have (l, m) in their right context: [*a, *b)
__device__ void seen_on_right_by(const TreeParams& t, int l, int m, int* a, int* b) {
    const int lim = m << l;  // candidates are tokens 0..lim-1
    int lo = 0, hi = lim;    // first i whose level-l range ends at or beyond m (a missing level counts as beyond)
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        int rl, rh;
        const bool ex = right_level_range(t, mid, l, &rl, &rh);
        if (!ex || rh >= m) hi = mid; else lo = mid + 1;
    }
    const int first = lo;
    lo = first; hi = lim;    // first i whose range starts beyond m (or has no level l)
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        int rl, rh;
        const bool ex = right_level_range(t, mid, l, &rl, &rh);
        if (!ex || rl > m) hi = mid; else lo = mid + 1;
    }
    *a = first; *b = lo;
}

// tokens i (all beyond the node) that have (l, m) in their left context: [*a, *b)
__device__ void seen_on_left_by(const TreeParams& t, int l, int m, int* a, int* b) {
    const int from = (m + 1) << l;
    int lo = from, hi = t.n;  // first i whose nearest level-l node is at or beyond m
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        int rl, rh;
        const bool ex = left_level_range(t, mid, l, &rl, &rh);
        if (ex && rh >= m) hi = mid; else lo = mid + 1;
    }
    const int first = lo;
    lo = first; hi = t.n;     // first i whose farthest level-l node lies beyond m
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        int rl, rh;
        const bool ex = left_level_range(t, mid, l, &rl, &rh);
        if (ex && rl > m) hi = mid; else lo = mid + 1;
    }
    *a = first; *b = lo;
}

struct SourceFan {
    int ra, rb;  // destinations (tokens) that see the node on their right: [ra, rb)
    int la, lb;  // ... on their left: [la, lb)
};

__device__ SourceFan source_fan(const TreeParams& t, int l, int m) {
    SourceFan f;
    f.ra = f.rb = 0;
    if (!t.left_only) seen_on_right_by(t, l, m, &f.ra, &f.rb);
    seen_on_left_by(t, l, m, &f.la, &f.lb);
    return f;
}

__global__ void source_degree_kernel(TreeParams t, int32_t* __restrict__ t_ptr) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= 2 * t.n - 1) return;
    const int l = node_level(t.n, v), m = v - node_id(t.n, l, 0);
    const SourceFan f = source_fan(t, l, m);
    int deg = (f.rb - f.ra) + (f.lb - f.la);
    if (l == 0) deg += 1 + t.L;  // self loop and one ancestor per level
    t_ptr[v] = deg;
}

// One warp per source node; destinations ascending.
__global__ void source_fill_kernel(TreeParams t, const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ t_ptr,
                                   int32_t* __restrict__ t_dst, int32_t* __restrict__ t_eid, int64_t E) {
    const int v = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
    const int lane = threadIdx.x & 31;
    if (v >= 2 * t.n - 1) return;
    const int l = node_level(t.n, v), m = v - node_id(t.n, l, 0);
    const SourceFan f = source_fan(t, l, m);
    int at = t_ptr[v];
    // tokens to the left of the node: it is in their right context
    for (int i = f.ra + lane; i < f.rb; i += 32) {
        int pos, cnt, first;
        token_block(t, i, 1, l, &pos, &cnt, &first);
        if (!BPT_IDX_OK(at + i - f.ra, E, BPT_SITE_GRAPH_WRITE)) continue;
        t_dst[at + i - f.ra] = i;
        t_eid[at + i - f.ra] = row_ptr[i] + pos + (m - first);
    }
    at += f.rb - f.ra;
    if (l == 0) {
        if (lane == 0) {
            int pos, cnt, first;
            token_block(t, m, 2, 0, &pos, &cnt, &first);
            if (BPT_IDX_OK(at, E, BPT_SITE_GRAPH_WRITE)) {
                t_dst[at] = m;
                t_eid[at] = row_ptr[m] + pos;
            }
        }
        ++at;
    }
    for (int i = f.la + lane; i < f.lb; i += 32) {
        int pos, cnt, first;
        token_block(t, i, 0, l, &pos, &cnt, &first);
        if (!BPT_IDX_OK(at + i - f.la, E, BPT_SITE_GRAPH_WRITE)) continue;
        t_dst[at + i - f.la] = i;
        t_eid[at + i - f.la] = row_ptr[i] + pos + (m - first);
    }
    at += f.lb - f.la;
    if (l == 0) {
        for (int j = 1 + lane; j <= t.L; j += 32) {
            const int u = node_id(t.n, j, m >> j);
            if (!BPT_IDX_OK(at + j - 1, E, BPT_SITE_GRAPH_WRITE)) continue;
            t_dst[at + j - 1] = u;
            t_eid[at + j - 1] = row_ptr[u] + (m & ((1 << j) - 1));
        }
    }
}

}  // namespace bpt

using namespace bpt;

static bool make_params(int32_t n, int32_t k, uint32_t flags, TreeParams* t) {
    if (n < 2 || (n & (n - 1)) != 0 || k < 1) return false;
    int L = 0;
    while ((1 << L) < n) ++L;
    t->n = n; t->L = L; t->k = k; t->kc = k < n ? k : n;
    t->pad = (flags & BPT_MODE_ALG1) ? 0 : 1;
    t->left_only = (flags & BPT_LEFT_ONLY) ? 1 : 0;
    return true;
}

bool bpt::tree_params_from_dims(const bpt_graph_dims& d, TreeParams* t) { return make_params(d.n, d.k, d.flags, t); }

extern "C" bpt_status bpt_graph_dims_query(int32_t n, int32_t k, uint32_t flags, bpt_graph_dims* out) {
    if (!out) return BPT_ERR_INVALID_ARG;
    if (flags & ~(uint32_t)(BPT_LEFT_ONLY | BPT_MODE_ALG1)) return BPT_ERR_INVALID_ARG;
    TreeParams t;
    if (n >= 2 && (n & (n - 1)) != 0) return BPT_ERR_UNSUPPORTED;  // the tree of Sec. 3.2.1 is perfect: shorter sequences go through the length arguments
    if (!make_params(n, k, flags, &t)) return BPT_ERR_INVALID_ARG;
    if (n > (1 << 20) || k > (1 << 20)) return BPT_ERR_UNSUPPORTED;
    int64_t e = (int64_t)n * t.L;
    for (int i = 0; i < n; ++i) e += token_degree(t, i);
    if (e >= (int64_t)INT32_MAX) return BPT_ERR_OVERFLOW;
    out->n = n; out->k = k; out->flags = flags;
    out->n_levels = t.L;
    out->n_nodes = 2 * n - 1;
    out->n_rel = 1 + 2 * t.L * (k + 1) + t.L;
    out->n_edges = e;
    out->build_workspace_bytes = 256;  // reserved; the build itself works in place
    return BPT_OK;
}

extern "C" bpt_status bpt_build_graph(const bpt_graph_dims* dims, int32_t* row_ptr, int32_t* col, int32_t* rel,
                                      int32_t* t_ptr, int32_t* t_dst, int32_t* t_eid,
                                      void* workspace, void* cuda_stream, bpt_graph* out) {
    if (!dims || !row_ptr || !col || !rel || !out) return BPT_ERR_INVALID_ARG;
    const bool want_t = t_ptr || t_dst || t_eid;
    if (want_t && !(t_ptr && t_dst && t_eid)) return BPT_ERR_INVALID_ARG;
    if (!workspace) return BPT_ERR_WORKSPACE;
    bpt_graph_dims chk;
    const bpt_status qs = bpt_graph_dims_query(dims->n, dims->k, dims->flags, &chk);
    if (qs != BPT_OK) return qs;
    if (chk.n_edges != dims->n_edges || chk.n_nodes != dims->n_nodes || chk.n_rel != dims->n_rel) return BPT_ERR_INVALID_ARG;
    TreeParams t;
    make_params(dims->n, dims->k, dims->flags, &t);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int n = t.n, N = 2 * n - 1;

    token_degree_kernel<<<(n + 255) / 256, 256, 0, st>>>(t, row_ptr);
    exclusive_scan_kernel<<<1, 1024, 0, st>>>(row_ptr, n);
    span_row_ptr_kernel<<<(n + 255) / 256, 256, 0, st>>>(t, row_ptr);
    token_fill_kernel<<<(n * 32 + 255) / 256, 256, 0, st>>>(t, row_ptr, col, rel, dims->n_edges);
    {
        const int64_t tot = (int64_t)t.L * n;
        span_fill_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, st>>>(t, row_ptr, col, rel, dims->n_edges);
    }
    if (want_t) {
        source_degree_kernel<<<(N + 127) / 128, 128, 0, st>>>(t, t_ptr);
        exclusive_scan_kernel<<<1, 1024, 0, st>>>(t_ptr, N);
        source_fill_kernel<<<(unsigned)(((int64_t)N * 32 + 255) / 256), 256, 0, st>>>(t, row_ptr, t_ptr, t_dst, t_eid, dims->n_edges);
    }
    if (cudaGetLastError() != cudaSuccess) return BPT_ERR_CUDA;
    out->row_ptr = row_ptr; out->col = col; out->rel = rel;
    out->t_ptr = want_t ? t_ptr : nullptr;
    out->t_dst = want_t ? t_dst : nullptr;
    out->t_eid = want_t ? t_eid : nullptr;
    out->dims = *dims;
    return BPT_OK;
}
