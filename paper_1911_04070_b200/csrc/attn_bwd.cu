// Backward of graph self-attention with relative positions (arXiv 1911.04070, Sec. 3.4
// equation; the relation embeddings are trainable and shared across heads).
//
// General path, four launches, no atomics, every sum in a fixed order:
//   A  by destination: dq, and per edge P and dS into the workspace
//   B  by source (transposed lists): dk, dv from the stored P / dS
//   C  per (side, level) block of the relation table: partial d_rel over token chunks
//   D  sum of the partials
// The rows of d_rel that belong to the ancestor relations are written as exact zeros:
// every edge into a span carries the same relation, so its embedding shifts all scores of
// the row alike and the softmax does not depend on it.
#include "bounds_check.cuh"
#include "bpt_internal.cuh"
#include "row_map.cuh"

namespace bpt {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kRelChunks = 64;  // token chunks of stage C (upper bound)

int rows_kernel_warps(const bpt_graph& g);

struct BwdWorkspace {
    float* p;        // [B, E, H]
    float* ds;       // [B, E, H]
    float* part;     // [chunks, n_rel, d]
    size_t bytes;
};

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

static int rel_chunks(int n) { return n < kRelChunks ? n : kRelChunks; }

static BwdWorkspace carve(const bpt_graph& g, int B, int H, int d, void* base) {
    const size_t E = (size_t)g.dims.n_edges, n = (size_t)g.dims.n;
    char* c = (char*)base;
    BwdWorkspace w;
    size_t off = 0;
    w.p = (float*)(c + off); off += align256(sizeof(float) * B * E * H);
    w.ds = (float*)(c + off); off += align256(sizeof(float) * B * E * H);
    w.part = (float*)(c + off); off += align256(sizeof(float) * rel_chunks((int)n) * (size_t)g.dims.n_rel * d);
    w.bytes = off;
    return w;
}


// ---------------------------------------------------------------------------------
// A: by destination
// ---------------------------------------------------------------------------------
template <typename T, int D, int U>
__global__ void __launch_bounds__(256)
bwd_dst_kernel(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col, const int32_t* __restrict__ rel,
               const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, const T* __restrict__ r,
               const T* __restrict__ out, const float* __restrict__ lse, const T* __restrict__ d_out,
               T* __restrict__ dq, float* __restrict__ ws_p, float* __restrict__ ws_ds,
               int N, int row0, int nrows, int H, int ngroups, int64_t e_first, int64_t E, float scale,
               const int32_t* __restrict__ lengths, DropoutParams drop, int n_rel) {
    using M = RowMap<T, D>;
    constexpr int EPL = M::EPL;
    extern __shared__ float smem[];
    const int nw = blockDim.x >> 5, w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t bid = blockIdx.x;
    const int u = row0 + nrows - 1 - (int)(bid % nrows);  // rows [row0, row0 + nrows), long span rows first
    const int hg = (int)((bid / nrows) % ngroups);
    const int b = (int)(bid / ((int64_t)nrows * ngroups));
    const int head = hg * M::HPW + lane / M::G;
    const bool head_ok = head < H;
    const int hc = head_ok ? head : H - 1;
    const int sub = lane % M::G;
    const size_t rs = (size_t)H * D;
    const size_t boff = (size_t)b * N * rs + (size_t)hc * D;
    const size_t uoff = boff + (size_t)u * rs;

    float qv[EPL], gv[EPL], acc[EPL];
    M::load(q + uoff, sub, qv);
    M::load(d_out + uoff, sub, gv);
    float delta = 0.f;  // d_out_u . out_u
    {
        float ov[EPL];
        M::load(out + uoff, sub, ov);
#pragma unroll
        for (int x = 0; x < EPL; ++x) delta = fmaf(gv[x], ov[x], delta);
        delta = M::head_sum(delta);
    }
    const float lse2 = lse[((size_t)b * N + u) * H + hc] * kLog2e;
    const float sc2 = scale * kLog2e;
#pragma unroll
    for (int x = 0; x < EPL; ++x) acc[x] = 0.f;

    // short sequence: edges that touch a node without real tokens do not exist (their P and dS are stored as 0)
    const int n_tok = (N + 1) / 2;
    const int len = lengths ? min(max(lengths[b], 0), n_tok) : n_tok;
    const bool u_real = len >= n_tok || node_first_token(n_tok, u) < len;
    const int a = row_ptr[u], z = row_ptr[u + 1];
    const size_t eoff = (size_t)b * E;
    for (int e0 = a + w * U; e0 < z; e0 += nw * U) {
        const int cnt = min(U, z - e0);
        int my_c = 0, my_r = 0;
        if (lane < cnt && BPT_IDX_OK(e0 + lane, E, BPT_SITE_CSR_OFFSET)) { my_c = col[e0 + lane]; my_r = rel[e0 + lane]; }
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const int c = __shfl_sync(0xffffffffu, my_c, j), rr = __shfl_sync(0xffffffffu, my_r, j);
            if (j < cnt && !(u_real && (len >= n_tok || node_first_token(n_tok, c) < len))) {
                if (sub == 0 && head_ok) {
                    const size_t o = (eoff + (size_t)(e0 + j - e_first)) * H + head;
                    ws_p[o] = 0.f;
                    ws_ds[o] = 0.f;
                }
            } else if (j < cnt && BPT_IDX_OK(c, N, BPT_SITE_NODE) && BPT_IDX_OK(rr, n_rel, BPT_SITE_RELATION)) {  // uniform over the warp
                float kk[EPL], rv[EPL], vv[EPL];
                M::load(k + boff + (size_t)c * rs, sub, kk);
                M::load(r + (size_t)rr * D, sub, rv);
                M::load(v + boff + (size_t)c * rs, sub, vv);
                float s = 0.f, dp = 0.f;
#pragma unroll
                for (int x = 0; x < EPL; ++x) {
                    kk[x] += rv[x];
                    s = fmaf(qv[x], kk[x], s);
                    dp = fmaf(gv[x], vv[x], dp);
                }
                s = M::head_sum(s);
                dp = M::head_sum(dp);
                float p = fast_exp2(fmaf(s, sc2, -lse2));
                // dropout: dP = W d_out.v and the weight that reaches dv is W P; dS keeps the undropped P
                const float wgt = drop.thr ? dropout_weight(drop, (uint32_t)(b * H + hc), (uint32_t)u, (uint32_t)c) : 1.f;
                const float ds = p * (dp * wgt - delta);
                p *= wgt;
#pragma unroll
                for (int x = 0; x < EPL; ++x) acc[x] = fmaf(ds, kk[x], acc[x]);
                if (sub == 0 && head_ok) {
                    const size_t o = (eoff + (size_t)(e0 + j - e_first)) * H + head;  // E edges kept per batch entry, from e_first on
                    ws_p[o] = p;
                    ws_ds[o] = ds;
                }
            }
        }
    }
    if (nw > 1) {
        float* sm_a = smem;  // [nw][EPL][32]
#pragma unroll
        for (int x = 0; x < EPL; ++x) sm_a[(w * EPL + x) * 32 + lane] = acc[x];
        __syncthreads();
        if (w != 0) return;
#pragma unroll
        for (int x = 0; x < EPL; ++x) acc[x] = 0.f;
        for (int j = 0; j < nw; ++j) {
#pragma unroll
            for (int x = 0; x < EPL; ++x) acc[x] += sm_a[(j * EPL + x) * 32 + lane];
        }
    }
#pragma unroll
    for (int x = 0; x < EPL; ++x) acc[x] *= scale;
    if (head_ok) M::store(dq + uoff, sub, acc);
}

// ---------------------------------------------------------------------------------
// B: by source
// ---------------------------------------------------------------------------------
template <typename T, int D, int U>
__global__ void __launch_bounds__(256)
bwd_src_kernel(const int32_t* __restrict__ t_ptr, const int32_t* __restrict__ t_dst, const int32_t* __restrict__ t_eid,
               const T* __restrict__ q, const T* __restrict__ d_out,
               const float* __restrict__ ws_p, const float* __restrict__ ws_ds,
               T* __restrict__ dk, T* __restrict__ dv, int N, int H, int ngroups, int64_t E, float scale) {
    using M = RowMap<T, D>;
    constexpr int EPL = M::EPL;
    extern __shared__ float smem[];
    const int nw = blockDim.x >> 5, w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t bid = blockIdx.x;
    const int vtx = N - 1 - (int)(bid % N);
    const int hg = (int)((bid / N) % ngroups);
    const int b = (int)(bid / ((int64_t)N * ngroups));
    const int head = hg * M::HPW + lane / M::G;
    const bool head_ok = head < H;
    const int hc = head_ok ? head : H - 1;
    const int sub = lane % M::G;
    const size_t rs = (size_t)H * D;
    const size_t boff = (size_t)b * N * rs + (size_t)hc * D;
    const size_t eoff = (size_t)b * E;

    float ak[EPL], av[EPL];
#pragma unroll
    for (int x = 0; x < EPL; ++x) { ak[x] = 0.f; av[x] = 0.f; }

    const int a = t_ptr[vtx], z = t_ptr[vtx + 1];
    for (int e0 = a + w * U; e0 < z; e0 += nw * U) {
        const int cnt = min(U, z - e0);
        int my_u = 0, my_e = 0;
        if (lane < cnt && BPT_IDX_OK(e0 + lane, E, BPT_SITE_CSR_OFFSET)) { my_u = t_dst[e0 + lane]; my_e = t_eid[e0 + lane]; }
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const int u = __shfl_sync(0xffffffffu, my_u, j), e = __shfl_sync(0xffffffffu, my_e, j);
            if (j < cnt && BPT_IDX_OK(u, N, BPT_SITE_NODE) && BPT_IDX_OK(e, E, BPT_SITE_EDGE_ID)) {
                float qv[EPL], gv[EPL];
                M::load(q + boff + (size_t)u * rs, sub, qv);
                M::load(d_out + boff + (size_t)u * rs, sub, gv);
                const size_t o = (eoff + (size_t)e) * H + hc;
                const float p = __ldg(ws_p + o), ds = __ldg(ws_ds + o);
#pragma unroll
                for (int x = 0; x < EPL; ++x) {
                    ak[x] = fmaf(ds, qv[x], ak[x]);
                    av[x] = fmaf(p, gv[x], av[x]);
                }
            }
        }
    }
    if (nw > 1) {
        float* sm_k = smem;
        float* sm_v = smem + nw * EPL * 32;
#pragma unroll
        for (int x = 0; x < EPL; ++x) {
            sm_k[(w * EPL + x) * 32 + lane] = ak[x];
            sm_v[(w * EPL + x) * 32 + lane] = av[x];
        }
        __syncthreads();
        if (w != 0) return;
#pragma unroll
        for (int x = 0; x < EPL; ++x) { ak[x] = 0.f; av[x] = 0.f; }
        for (int j = 0; j < nw; ++j) {
#pragma unroll
            for (int x = 0; x < EPL; ++x) {
                ak[x] += sm_k[(j * EPL + x) * 32 + lane];
                av[x] += sm_v[(j * EPL + x) * 32 + lane];
            }
        }
    }
#pragma unroll
    for (int x = 0; x < EPL; ++x) ak[x] *= scale;
    if (head_ok) {
        M::store(dk + boff + (size_t)vtx * rs, sub, ak);
        M::store(dv + boff + (size_t)vtx * rs, sub, av);
    }
}

// ---------------------------------------------------------------------------------
// C: partial d_rel.  blockIdx.y picks a block of the relation table: left level j
// (0..L-1), right level j (L..2L-1), self (2L); blockIdx.x picks a chunk of tokens.
// Items (token, batch entry, block of up to 8 heads) are staged four at a time in shared
// memory: the q rows as fp32 and the dS values of the block's edges, which are contiguous
// in the token's row.  Thread (og, cg) owns relation rows og, og+NOG, ... of the current
// tile of offsets and channels 4*cg .. 4*cg+3.
// ---------------------------------------------------------------------------------
constexpr int kRelHB = 8;   // heads per item
constexpr int kRelTB = 4;   // items staged together

template <typename T, int D>
__global__ void __launch_bounds__(256)
drel_partial_kernel(TreeParams t, const int32_t* __restrict__ row_ptr, const T* __restrict__ q,
                    const float* __restrict__ ws_ds, float* __restrict__ part,
                    int B, int H, int64_t E, int n_rel, int n_chunks) {
    constexpr int CG = D / 4, NOG = 256 / CG, NJ = D == 64 ? 5 : 3, OT = NOG * NJ;
    __shared__ float q_s[kRelTB][kRelHB][D];
    __shared__ float ds_s[kRelTB][OT][kRelHB];
    __shared__ int it_e0[kRelTB], it_cnt[kRelTB];
    const int tid = threadIdx.x, cg = tid % CG, og = tid / CG;
    const int chunk = blockIdx.x, blk = blockIdx.y;
    const int N = 2 * t.n - 1;
    int side, level, width, rel_base;
    if (blk < t.L) { side = 0; level = blk; width = t.k + 1; rel_base = rel_left(t, level, 0); }
    else if (blk < 2 * t.L) { side = 1; level = blk - t.L; width = t.k + 1; rel_base = rel_right(t, level, 0); }
    else { side = 2; level = 0; width = 1; rel_base = 0; }
    // no token has more than min(k, n) + 1 nodes in one block
    const int wmax = min(width, t.kc + 1);

    const int per = (t.n + n_chunks - 1) / n_chunks;
    const int x0 = min(chunk * per, t.n), x1 = min(x0 + per, t.n);
    const int nhb = (H + kRelHB - 1) / kRelHB;
    const int n_items = (x1 - x0) * B * nhb;  // item = (token, b, head block), token-major
    const size_t rs = (size_t)H * D;

    // A level exists on the left for a suffix of the tokens and on the right for a prefix,
    // so one probe tells whether any token of the chunk has edges in this block.
    bool any = x1 > x0;
    if (any && side != 2) {
        int pos, c, first;
        any = token_block(t, side == 0 ? x1 - 1 : x0, side, level, &pos, &c, &first);
    }

    for (int o0 = 0; o0 < width; o0 += OT) {
        float4 acc[NJ];
#pragma unroll
        for (int j = 0; j < NJ; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (any && o0 < wmax) {
            for (int it0 = 0; it0 < n_items; it0 += kRelTB) {
                __syncthreads();  // previous items consumed
                if (tid < kRelTB) {
                    int e0 = 0, cnt = 0;
                    const int it = it0 + tid;
                    if (it < n_items) {
                        const int x = x0 + it / (B * nhb);
                        int pos, c, first;
                        if (token_block(t, x, side, level, &pos, &c, &first)) {
                            // offset o sits at edge pos + o (right, self) or pos + c - 1 - o (left)
                            cnt = max(0, min(c - o0, OT));
                            e0 = row_ptr[x] + (side == 0 ? pos + c - 1 - o0 : pos + o0);
                        }
                    }
                    it_e0[tid] = e0; it_cnt[tid] = cnt;
                }
                __syncthreads();
                {
                    int tot = 0;
#pragma unroll
                    for (int j = 0; j < kRelTB; ++j) tot += it_cnt[j];
                    if (tot == 0) continue;  // uniform over the block
                }
                // stage q rows (as fp32) and dS values
                for (int idx = tid; idx < kRelTB * kRelHB * D; idx += 256) {
                    const int c = idx % D, h = (idx / D) % kRelHB, j = idx / (D * kRelHB);
                    const int it = it0 + j;
                    float val = 0.f;
                    if (it < n_items && it_cnt[j] > 0) {
                        const int x = x0 + it / (B * nhb), b = (it / nhb) % B, hh = (it % nhb) * kRelHB + h;
                        if (hh < H) val = (float)q[((size_t)b * N + x) * rs + (size_t)hh * D + c];
                    }
                    q_s[j][h][c] = val;
                }
                for (int idx = tid; idx < kRelTB * OT * kRelHB; idx += 256) {
                    const int h = idx % kRelHB, o = (idx / kRelHB) % OT, j = idx / (kRelHB * OT);
                    const int it = it0 + j;
                    float val = 0.f;
                    if (it < n_items && o < it_cnt[j]) {
                        const int b = (it / nhb) % B, hh = (it % nhb) * kRelHB + h;
                        const int e = side == 0 ? it_e0[j] - o : it_e0[j] + o;
                        if (hh < H) val = ws_ds[((size_t)b * E + e) * H + hh];
                    }
                    ds_s[j][o][h] = val;
                }
                __syncthreads();
#pragma unroll
                for (int j = 0; j < kRelTB; ++j) {
#pragma unroll
                    for (int h = 0; h < kRelHB; ++h) {
                        const float4 qq = *reinterpret_cast<const float4*>(&q_s[j][h][cg * 4]);
#pragma unroll
                        for (int jj = 0; jj < NJ; ++jj) {
                            const float a = ds_s[j][og + jj * NOG][h];
                            acc[jj].x = fmaf(a, qq.x, acc[jj].x);
                            acc[jj].y = fmaf(a, qq.y, acc[jj].y);
                            acc[jj].z = fmaf(a, qq.z, acc[jj].z);
                            acc[jj].w = fmaf(a, qq.w, acc[jj].w);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int jj = 0; jj < NJ; ++jj) {
            const int o = o0 + og + jj * NOG;
            if (o < width)
                *reinterpret_cast<float4*>(part + ((size_t)chunk * n_rel + rel_base + o) * D + cg * 4) = acc[jj];
        }
    }
}

// D: d_rel[r, c] = scale * sum over chunks, in chunk order; ancestor rows are zero
__global__ void drel_reduce_kernel(const float* __restrict__ part, float* __restrict__ d_rel, int n_chunks,
                                   size_t per_chunk, size_t first_zero, float scale) {
    const size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= per_chunk) return;
    float acc = 0.f;
    if (x < first_zero)
        for (int c = 0; c < n_chunks; ++c) acc += part[(size_t)c * per_chunk + x];
    d_rel[x] = acc * scale;
}

template <typename T, int D>
static bpt_status launch_bwd_rows(const AttnProblem& p) {
    using M = RowMap<T, D>;
    constexpr int U = 4;
    const bpt_graph& g = *p.g;
    const int N = g.dims.n_nodes, n = g.dims.n;
    const int64_t E = g.dims.n_edges;
    const int ngroups = (p.H + M::HPW - 1) / M::HPW;
    const int nw = rows_kernel_warps(g);
    const int64_t blocks = (int64_t)p.B * N * ngroups;
    if (blocks > 0x7fffffffll) return BPT_ERR_UNSUPPORTED;
    const BwdWorkspace ws = carve(g, p.B, p.H, p.d, p.workspace);

    const size_t smem_a = nw > 1 ? (size_t)nw * 32 * M::EPL * sizeof(float) : 0;
    bwd_dst_kernel<T, D, U><<<(unsigned)blocks, nw * 32, smem_a, p.stream>>>(
        g.row_ptr, g.col, g.rel, (const T*)p.q, (const T*)p.k, (const T*)p.v, (const T*)p.rel_emb,
        (const T*)p.out, p.lse, (const T*)p.d_out, (T*)p.dq, ws.p, ws.ds, N, 0, N, p.H, ngroups, 0, E, p.scale, p.lengths, p.drop, g.dims.n_rel);
    trace_mark(p.stream, "bwd_dst");

    const size_t smem_b = nw > 1 ? (size_t)nw * 32 * (2 * M::EPL) * sizeof(float) : 0;
    bwd_src_kernel<T, D, U><<<(unsigned)blocks, nw * 32, smem_b, p.stream>>>(
        g.t_ptr, g.t_dst, g.t_eid, (const T*)p.q, (const T*)p.d_out, ws.p, ws.ds,
        (T*)p.dk, (T*)p.dv, N, p.H, ngroups, E, p.scale);
    trace_mark(p.stream, "bwd_src");

    const int chunks = rel_chunks(n);
    const dim3 grid_c(chunks, 2 * p.tree.L + 1);
    drel_partial_kernel<T, D><<<grid_c, 256, 0, p.stream>>>(p.tree, g.row_ptr, (const T*)p.q, ws.ds, ws.part,
                                                           p.B, p.H, E, g.dims.n_rel, chunks);
    trace_mark(p.stream, "drel_partial");
    const size_t per_chunk = (size_t)g.dims.n_rel * D;
    drel_reduce_kernel<<<(unsigned)((per_chunk + 255) / 256), 256, 0, p.stream>>>(ws.part, p.d_rel, chunks, per_chunk,
                                                                                      (size_t)rel_anc(p.tree, 1) * D, p.scale);
    trace_mark(p.stream, "drel_reduce");
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

bool bwd_tile_eligible(const bpt_graph& g, int d, bpt_dtype dtype);
size_t bwd_tile_workspace_bytes(const bpt_graph& g, int B, int H, bool minimal);
bpt_status launch_bwd_tile(const AttnProblem& p);

size_t bwd_workspace_bytes(const bpt_graph& g, int B, int H, int d, bpt_dtype dtype, bool minimal) {
    if (bwd_tile_eligible(g, d, dtype)) return bwd_tile_workspace_bytes(g, B, H, minimal);
    return carve(g, B, H, d, nullptr).bytes;
}

bpt_status launch_bwd(const AttnProblem& p) {
    if (bwd_tile_eligible(*p.g, p.d, p.dtype)) return launch_bwd_tile(p);
    if (p.dtype == BPT_F32) return p.d == 64 ? launch_bwd_rows<float, 64>(p) : launch_bwd_rows<float, 32>(p);
    return p.d == 64 ? launch_bwd_rows<__nv_bfloat16, 64>(p) : launch_bwd_rows<__nv_bfloat16, 32>(p);
}

}  // namespace bpt
