// Forward graph self-attention over the CSR (arXiv 1911.04070: GSA of Sec. 3.1 with the
// relative-position term of Sec. 3.4).  General row kernel: one CTA per (batch, node,
// head group); its warps take the row's edges in turns, each keeps an online softmax in
// registers, and the per-warp states are merged in a fixed order through shared memory.
#include <cstdlib>

#include "bounds_check.cuh"
#include "bpt_internal.cuh"
#include "row_map.cuh"
#include "tile_geom.cuh"

namespace bpt {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <typename T, int D, int U>
__global__ void __launch_bounds__(256)
fwd_rows_kernel(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col, const int32_t* __restrict__ rel,
                const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, const T* __restrict__ r,
                T* __restrict__ out, float* __restrict__ lse, int N, int row0, int nrows, int H, int ngroups,
                float scale_log2e, const int32_t* __restrict__ lengths, DropoutParams drop,
                const int32_t* __restrict__ row_list, int64_t E, int n_rel) {
    using M = RowMap<T, D>;
    constexpr int EPL = M::EPL;
    extern __shared__ float smem[];
    const int nw = blockDim.x >> 5, w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t bid = blockIdx.x;
    // rows [row0, row0 + nrows), long span rows first; or the nrows rows of row_list (per batch entry: [B][nrows])
    const int hg = (int)((bid / nrows) % ngroups);
    const int b = (int)(bid / ((int64_t)nrows * ngroups));
    const int u = row_list ? row_list[(size_t)b * nrows + (int)(bid % nrows)] : row0 + nrows - 1 - (int)(bid % nrows);
    if (u < 0 || u >= N) return;  // an entry of row_list outside the graph is skipped (uniform over the CTA)
    const int head = hg * M::HPW + lane / M::G;
    const bool head_ok = head < H;
    const int hc = head_ok ? head : H - 1;
    const int sub = lane % M::G;
    const size_t rs = (size_t)H * D;
    const size_t boff = (size_t)b * N * rs + (size_t)hc * D;

    float qv[EPL];
    M::load(q + boff + (size_t)u * rs, sub, qv);
#pragma unroll
    for (int c = 0; c < EPL; ++c) qv[c] *= scale_log2e;

    float m = -INFINITY, l = 0.f, acc[EPL];
#pragma unroll
    for (int c = 0; c < EPL; ++c) acc[c] = 0.f;

    // short sequence: edges that touch a node without real tokens do not exist
    const int n_tok = (N + 1) / 2;
    const int len = lengths ? min(max(lengths[b], 0), n_tok) : n_tok;
    const bool u_real = len >= n_tok || node_first_token(n_tok, u) < len;
    const int a = row_ptr[u], z = u_real ? row_ptr[u + 1] : row_ptr[u];
    for (int e0 = a + w * U; e0 < z; e0 += nw * U) {
        const int cnt = min(U, z - e0);
        int my_c = 0, my_r = 0;
        if (lane < cnt && BPT_IDX_OK(e0 + lane, E, BPT_SITE_CSR_OFFSET)) { my_c = col[e0 + lane]; my_r = rel[e0 + lane]; }
        float s[U], vv[U][EPL], wgt[U];
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const int c = __shfl_sync(0xffffffffu, my_c, j), rr = __shfl_sync(0xffffffffu, my_r, j);
            wgt[j] = (drop.thr && j < cnt) ? dropout_weight(drop, (uint32_t)(b * H + hc), (uint32_t)u, (uint32_t)c) : 1.f;
            if (j < cnt && BPT_IDX_OK(c, N, BPT_SITE_NODE) && BPT_IDX_OK(rr, n_rel, BPT_SITE_RELATION) &&
                (len >= n_tok || node_first_token(n_tok, c) < len)) {
                float kk[EPL], rv[EPL];
                M::load(k + boff + (size_t)c * rs, sub, kk);
                M::load(r + (size_t)rr * D, sub, rv);
                M::load(v + boff + (size_t)c * rs, sub, vv[j]);
                float d = 0.f;
#pragma unroll
                for (int x = 0; x < EPL; ++x) d = fmaf(qv[x], kk[x] + rv[x], d);
                s[j] = d;
            } else {
                s[j] = -INFINITY;
#pragma unroll
                for (int x = 0; x < EPL; ++x) vv[j][x] = 0.f;
            }
        }
        float m_new = m;
#pragma unroll
        for (int j = 0; j < U; ++j) {
            s[j] = M::head_sum(s[j]);
            m_new = fmaxf(m_new, s[j]);
        }
        const float m_ref = m_new == -INFINITY ? 0.f : m_new;  // nothing seen so far (only skipped edges): keep the empty state
        const float corr = fast_exp2(m - m_ref);
        l *= corr;
#pragma unroll
        for (int x = 0; x < EPL; ++x) acc[x] *= corr;
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const float p = fast_exp2(s[j] - m_ref);
            l += p;
            const float pw = p * wgt[j];  // dropout acts on the weight that reaches V, not on the softmax sum
#pragma unroll
            for (int x = 0; x < EPL; ++x) acc[x] = fmaf(pw, vv[j][x], acc[x]);
        }
        m = m_new;
    }

    if (nw > 1) {  // merge the warps' (m, l, acc) in warp order
        float* sm_m = smem;
        float* sm_l = smem + nw * 32;
        float* sm_a = smem + 2 * nw * 32;
        sm_m[w * 32 + lane] = m;
        sm_l[w * 32 + lane] = l;
#pragma unroll
        for (int x = 0; x < EPL; ++x) sm_a[(w * EPL + x) * 32 + lane] = acc[x];
        __syncthreads();
        if (w != 0) return;
        float mt = -INFINITY;
        for (int j = 0; j < nw; ++j) mt = fmaxf(mt, sm_m[j * 32 + lane]);
        if (mt == -INFINITY) mt = 0.f;  // a row without edges: every warp state is empty
        l = 0.f;
#pragma unroll
        for (int x = 0; x < EPL; ++x) acc[x] = 0.f;
        for (int j = 0; j < nw; ++j) {
            const float f = fast_exp2(sm_m[j * 32 + lane] - mt);
            l = fmaf(sm_l[j * 32 + lane], f, l);
#pragma unroll
            for (int x = 0; x < EPL; ++x) acc[x] = fmaf(sm_a[(j * EPL + x) * 32 + lane], f, acc[x]);
        }
        m = mt;
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll
    for (int x = 0; x < EPL; ++x) acc[x] *= inv;
    if (head_ok) {
        M::store(out + boff + (size_t)u * rs, sub, acc);
        if (sub == 0) lse[((size_t)b * N + u) * H + head] = l > 0.f ? (m + log2f(l)) * kLn2 : 0.f;
    }
}

int rows_kernel_warps(const bpt_graph& g) {
    const double avg = (double)g.dims.n_edges / (double)g.dims.n_nodes;
    return avg >= 96.0 ? 8 : (avg >= 24.0 ? 4 : 2);
}

template <typename T, int D>
static bpt_status launch_rows(const AttnProblem& p, int row0, int nrows, const int32_t* row_list = nullptr) {
    using M = RowMap<T, D>;
    constexpr int U = 4;
    const bpt_graph& g = *p.g;
    const int N = g.dims.n_nodes;
    const int ngroups = (p.H + M::HPW - 1) / M::HPW;
    const int nw = rows_kernel_warps(g);
    const int64_t blocks = (int64_t)p.B * nrows * ngroups;
    if (blocks > 0x7fffffffll) return BPT_ERR_UNSUPPORTED;
    const size_t smem = nw > 1 ? (size_t)nw * 32 * (2 + M::EPL) * sizeof(float) : 0;
    fwd_rows_kernel<T, D, U><<<(unsigned)blocks, nw * 32, smem, p.stream>>>(
        g.row_ptr, g.col, g.rel, (const T*)p.q, (const T*)p.k, (const T*)p.v, (const T*)p.rel_emb,
        (T*)p.out, p.lse, N, row0, nrows, p.H, ngroups, p.scale * kLog2e, p.lengths, p.drop, row_list, g.dims.n_edges, g.dims.n_rel);
    trace_mark(p.stream, "fwd_rows");
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

bpt_status launch_fwd_tile(const AttnProblem& p);
bool fwd_tc5_eligible(const AttnProblem& p);
bpt_status launch_fwd_tc5(const AttnProblem& p, int* status, int2* ranges);
size_t fwd_tc5_ranges_bytes(const TreeParams& t);
size_t fwd_span_workspace_bytes(const TreeParams& t, int B, int H);
bpt_status launch_fwd_span(const AttnProblem& p);

static size_t span_ws_bytes(const TreeParams& t, int B, int H) { return (fwd_span_workspace_bytes(t, B, H) + 255) & ~(size_t)255; }

size_t fwd_workspace_bytes(const bpt_graph& g, int B, int H, int d, bpt_dtype dtype) {
    if (!tile_path(g.dims.n, g.dims.k, d, dtype == BPT_BF16)) return 0;
    TreeParams t;
    tree_params_from_dims(g.dims, &t);
    // the span partials, then the node-range table of the tensor-memory kernel (never empty, so that the status block in front exists)
    return span_ws_bytes(t, B, H) + fwd_tc5_ranges_bytes(t) + 256;
}

// Two kernels cover the token rows: the warp-level one (mma.sync, 64-token tiles) and the tensor-memory
// one (tcgen05 + TMA, 128-token tiles, two CTAs per SM).  Measured at n = 8192, left-only, batch 4 (ms, warp-level /
// tensor-memory): k = 64 0.36 / 0.24, k = 48 0.32 / 0.22, k = 32 0.25 / 0.21, k = 24 0.25 / 0.21, k = 16 0.21 / 0.21,
// k = 8 0.18 / 0.21, k = 4 0.18 / 0.23; bidirectional n = 16384, k = 16: 0.42 / 0.38; n = 65536, k = 64: 1.92 / 1.14.
// The tensor-memory kernel therefore takes k >= 16.  bpt_attn_options.path forces one of them for comparison runs.
static bool want_tc5(int k, uint32_t path) { return path == BPT_PATH_TC5 || (path == BPT_PATH_AUTO && k >= 16); }

bpt_status launch_fwd(const AttnProblem& p) {
    if (tile_path(p.tree.n, p.tree.k, p.d, p.dtype == BPT_BF16)) {  // token rows and span rows on the tensor cores
        int2* ranges = reinterpret_cast<int2*>(static_cast<char*>(p.workspace) + span_ws_bytes(p.tree, p.B, p.H));
        const bpt_status s = (want_tc5(p.tree.k, p.path) && fwd_tc5_eligible(p)) ? launch_fwd_tc5(p, p.status, ranges) : launch_fwd_tile(p);
        return s != BPT_OK ? s : launch_fwd_span(p);
    }
    const int row0 = 0, nrows = p.g->dims.n_nodes;
    if (p.dtype == BPT_F32) return p.d == 64 ? launch_rows<float, 64>(p, row0, nrows) : launch_rows<float, 32>(p, row0, nrows);
    return p.d == 64 ? launch_rows<__nv_bfloat16, 64>(p, row0, nrows) : launch_rows<__nv_bfloat16, 32>(p, row0, nrows);
}

// The listed destination rows only, through the general row kernel (any dtype / head size the library takes).
bpt_status launch_fwd_row_list(const AttnProblem& p, const int32_t* rows, int n_rows) {
    if (p.dtype == BPT_F32) return p.d == 64 ? launch_rows<float, 64>(p, 0, n_rows, rows) : launch_rows<float, 32>(p, 0, n_rows, rows);
    return p.d == 64 ? launch_rows<__nv_bfloat16, 64>(p, 0, n_rows, rows) : launch_rows<__nv_bfloat16, 32>(p, 0, n_rows, rows);
}

}  // namespace bpt
