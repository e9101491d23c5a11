// Backward of graph self-attention with relative positions (arXiv 1911.04070, Sec. 3.4
// equation; the relation embeddings are trainable and shared across heads).
//
// General path, four launches, no atomics, every sum in a fixed order:
//   A  by destination: dq, and per edge P and dS into the workspace
//   B  by source (transposed lists): dk, dv from the stored P / dS
//   C  per (side, level) block of the relation table: partial d_rel over token chunks
//   D  sum of the partials
#include "bpt_internal.cuh"
#include "row_map.cuh"

namespace bpt {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kRelChunks = 64;  // token chunks of stage C (upper bound)

int rows_kernel_warps(const bpt_graph& g);

struct BwdWorkspace {
    float* p;        // [B, E, H]
    float* ds;       // [B, E, H]
    float* rowsum;   // [B, n-1, H]  sum_e dS_e of every span row
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
    w.rowsum = (float*)(c + off); off += align256(sizeof(float) * B * (n - 1) * H);
    w.part = (float*)(c + off); off += align256(sizeof(float) * rel_chunks((int)n) * (size_t)g.dims.n_rel * d);
    w.bytes = off;
    return w;
}

size_t bwd_workspace_bytes(const bpt_graph& g, int B, int H, int d, bpt_dtype) { return carve(g, B, H, d, nullptr).bytes; }

// ---------------------------------------------------------------------------------
// A: by destination
// ---------------------------------------------------------------------------------
template <typename T, int D, int U>
__global__ void __launch_bounds__(256)
bwd_dst_kernel(const int32_t* __restrict__ row_ptr, const int32_t* __restrict__ col, const int32_t* __restrict__ rel,
               const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, const T* __restrict__ r,
               const T* __restrict__ out, const float* __restrict__ lse, const T* __restrict__ d_out,
               T* __restrict__ dq, float* __restrict__ ws_p, float* __restrict__ ws_ds, float* __restrict__ ws_rowsum,
               int N, int n_tok, int H, int ngroups, int64_t E, float scale) {
    using M = RowMap<T, D>;
    constexpr int EPL = M::EPL;
    extern __shared__ float smem[];
    const int nw = blockDim.x >> 5, w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t bid = blockIdx.x;
    const int u = N - 1 - (int)(bid % N);
    const int hg = (int)((bid / N) % ngroups);
    const int b = (int)(bid / ((int64_t)N * ngroups));
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
    float ds_sum = 0.f;

    const int a = row_ptr[u], z = row_ptr[u + 1];
    const size_t eoff = (size_t)b * E;
    for (int e0 = a + w * U; e0 < z; e0 += nw * U) {
        const int cnt = min(U, z - e0);
        int my_c = 0, my_r = 0;
        if (lane < cnt) { my_c = col[e0 + lane]; my_r = rel[e0 + lane]; }
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const int c = __shfl_sync(0xffffffffu, my_c, j), rr = __shfl_sync(0xffffffffu, my_r, j);
            if (j < cnt) {  // uniform over the warp
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
                const float p = fast_exp2(fmaf(s, sc2, -lse2));
                const float ds = p * (dp - delta);
                ds_sum += ds;
#pragma unroll
                for (int x = 0; x < EPL; ++x) acc[x] = fmaf(ds, kk[x], acc[x]);
                if (sub == 0 && head_ok) {
                    const size_t o = (eoff + (size_t)(e0 + j)) * H + head;
                    ws_p[o] = p;
                    ws_ds[o] = ds;
                }
            }
        }
    }
    if (nw > 1) {
        float* sm_a = smem;               // [nw][EPL][32]
        float* sm_s = smem + nw * EPL * 32;  // [nw][32]
#pragma unroll
        for (int x = 0; x < EPL; ++x) sm_a[(w * EPL + x) * 32 + lane] = acc[x];
        sm_s[w * 32 + lane] = ds_sum;
        __syncthreads();
        if (w != 0) return;
        ds_sum = 0.f;
#pragma unroll
        for (int x = 0; x < EPL; ++x) acc[x] = 0.f;
        for (int j = 0; j < nw; ++j) {
            ds_sum += sm_s[j * 32 + lane];
#pragma unroll
            for (int x = 0; x < EPL; ++x) acc[x] += sm_a[(j * EPL + x) * 32 + lane];
        }
    }
#pragma unroll
    for (int x = 0; x < EPL; ++x) acc[x] *= scale;
    if (head_ok) {
        M::store(dq + uoff, sub, acc);
        if (sub == 0 && u >= n_tok) ws_rowsum[((size_t)b * (N - n_tok) + (u - n_tok)) * H + head] = ds_sum;
    }
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
        if (lane < cnt) { my_u = t_dst[e0 + lane]; my_e = t_eid[e0 + lane]; }
#pragma unroll
        for (int j = 0; j < U; ++j) {
            const int u = __shfl_sync(0xffffffffu, my_u, j), e = __shfl_sync(0xffffffffu, my_e, j);
            if (j < cnt) {
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
// (0..L-1), right level j (L..2L-1), self (2L), ancestor level j (2L+1 .. 3L);
// blockIdx.x picks a chunk of tokens (or of spans for the ancestor rows).
// Thread (og, cg): relation row o0+og of the block, channels 4*cg .. 4*cg+3.
// ---------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float4 load4(const T* p);
template <> __device__ __forceinline__ float4 load4<float>(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
template <> __device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16* p) {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(p));
    return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u),
                       __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
}

template <typename T, int D>
__global__ void __launch_bounds__(256)
drel_partial_kernel(TreeParams t, const int32_t* __restrict__ row_ptr, const T* __restrict__ q,
                    const float* __restrict__ ws_ds, const float* __restrict__ ws_rowsum, float* __restrict__ part,
                    int B, int H, int64_t E, int n_rel, int n_chunks) {
    constexpr int CG = D / 4, NOG = 256 / CG;
    const int cg = threadIdx.x % CG, og = threadIdx.x / CG;
    const int chunk = blockIdx.x, blk = blockIdx.y;
    const int N = 2 * t.n - 1;
    int side, level, width, rel_base;
    if (blk < t.L) { side = 0; level = blk; width = t.k + 1; rel_base = rel_left(t, level, 0); }
    else if (blk < 2 * t.L) { side = 1; level = blk - t.L; width = t.k + 1; rel_base = rel_right(t, level, 0); }
    else if (blk == 2 * t.L) { side = 2; level = 0; width = 1; rel_base = 0; }
    else { side = 3; level = blk - 2 * t.L; width = 1; rel_base = rel_anc(t, level); }

    const int items = side == 3 ? (t.n >> level) : t.n;  // spans of the level, or tokens
    const int per = (items + n_chunks - 1) / n_chunks;
    const int x0 = min(chunk * per, items), x1 = min(x0 + per, items);
    const size_t rs = (size_t)H * D;

    for (int o0 = 0; o0 < width; o0 += NOG) {
        const int o = o0 + og;
        if (o >= width) continue;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int x = x0; x < x1; ++x) {
            int node;
            size_t soff, sstride;  // address of the dS (or row sum) value for b = 0, h = 0 and the stride over b
            if (side == 3) {
                node = node_id(t.n, level, x);
                soff = (size_t)(node - t.n) * H;
                sstride = (size_t)(t.n - 1) * H;
            } else {
                int pos, cnt, first;
                if (!token_block(t, x, side, level, &pos, &cnt, &first) || o >= cnt) continue;
                node = x;
                const int e = row_ptr[x] + (side == 0 ? pos + cnt - 1 - o : pos + o);
                soff = (size_t)e * H;
                sstride = (size_t)E * H;
            }
            const float* sp = (side == 3 ? ws_rowsum : ws_ds) + soff;
            const T* qp = q + (size_t)node * rs + cg * 4;
            for (int b = 0; b < B; ++b) {
                for (int h = 0; h < H; ++h) {
                    const float a = __ldg(sp + (size_t)b * sstride + h);
                    const float4 qq = load4<T>(qp + (size_t)b * N * rs + (size_t)h * D);
                    acc.x = fmaf(a, qq.x, acc.x);
                    acc.y = fmaf(a, qq.y, acc.y);
                    acc.z = fmaf(a, qq.z, acc.z);
                    acc.w = fmaf(a, qq.w, acc.w);
                }
            }
        }
        *reinterpret_cast<float4*>(part + ((size_t)chunk * n_rel + rel_base + o) * D + cg * 4) = acc;
    }
}

// D: d_rel[r, c] = scale * sum over chunks, in chunk order
__global__ void drel_reduce_kernel(const float* __restrict__ part, float* __restrict__ d_rel, int n_chunks, size_t per_chunk, float scale) {
    const size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= per_chunk) return;
    float acc = 0.f;
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

    const size_t smem_a = nw > 1 ? (size_t)nw * 32 * (M::EPL + 1) * sizeof(float) : 0;
    bwd_dst_kernel<T, D, U><<<(unsigned)blocks, nw * 32, smem_a, p.stream>>>(
        g.row_ptr, g.col, g.rel, (const T*)p.q, (const T*)p.k, (const T*)p.v, (const T*)p.rel_emb,
        (const T*)p.out, p.lse, (const T*)p.d_out, (T*)p.dq, ws.p, ws.ds, ws.rowsum, N, n, p.H, ngroups, E, p.scale);
    trace_mark(p.stream, "bwd_dst");

    const size_t smem_b = nw > 1 ? (size_t)nw * 32 * (2 * M::EPL) * sizeof(float) : 0;
    bwd_src_kernel<T, D, U><<<(unsigned)blocks, nw * 32, smem_b, p.stream>>>(
        g.t_ptr, g.t_dst, g.t_eid, (const T*)p.q, (const T*)p.d_out, ws.p, ws.ds,
        (T*)p.dk, (T*)p.dv, N, p.H, ngroups, E, p.scale);
    trace_mark(p.stream, "bwd_src");

    const int chunks = rel_chunks(n);
    const dim3 grid_c(chunks, 3 * p.tree.L + 1);
    drel_partial_kernel<T, D><<<grid_c, 256, 0, p.stream>>>(p.tree, g.row_ptr, (const T*)p.q, ws.ds, ws.rowsum, ws.part,
                                                           p.B, p.H, E, g.dims.n_rel, chunks);
    trace_mark(p.stream, "drel_partial");
    const size_t per_chunk = (size_t)g.dims.n_rel * D;
    drel_reduce_kernel<<<(unsigned)((per_chunk + 255) / 256), 256, 0, p.stream>>>(ws.part, p.d_rel, chunks, per_chunk, p.scale);
    trace_mark(p.stream, "drel_reduce");
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

bpt_status launch_bwd(const AttnProblem& p) {
    if (p.dtype == BPT_F32) return p.d == 64 ? launch_bwd_rows<float, 64>(p) : launch_bwd_rows<float, 32>(p);
    return p.d == 64 ? launch_bwd_rows<__nv_bfloat16, 64>(p) : launch_bwd_rows<__nv_bfloat16, 32>(p);
}

}  // namespace bpt
