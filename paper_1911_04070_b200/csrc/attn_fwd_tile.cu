// Tiled forward for the token rows (arXiv 1911.04070, Sec. 3.4 equation over the contextual
// edges of Sec. 3.2.2), bf16, head size 64.
//
// One CTA = 64 consecutive tokens of one (batch entry, head); each of its 4 warps owns 16
// query rows.  The nodes a token attends at one level and side are one contiguous range,
// and neighbouring tokens' ranges overlap almost completely, so per (side, level) chunk the
// CTA stages the union range of K and V rows once in shared memory and every warp runs
// S = Q K^T and O += P V on the tensor cores over the part of the range its own rows touch
// (flash-style online softmax, 32 keys per step).  The relative-position term
// q_i . r[rel(i, m)] depends on the offset of node m inside token i's range: the warp
// computes Q R_chunk^T once per chunk (a dense 16 x (k+1) product), parks it in shared
// memory and every score picks its entry by offset.
#include "bounds_check.cuh"
#include "bpt_internal.cuh"
#include "mma_tools.cuh"
#include "tile_geom.cuh"

namespace bpt {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kMaxKvRows = 208;  // staged K / V rows per chunk at k = 64 (union range + alignment slack)
constexpr int kMaxRelRows = 80;  // staged relation rows per chunk (k + 1 <= 65, padded to 16)

// Buffer sizes follow k, so that small k leaves room for more CTAs per SM.  (A second set of K / V / R
// buffers, with the next chunk fetched while this one is computed, was measured at k = 4 and 8: 0.178 /
// 0.377 ms against 0.151 / 0.306 ms for one set and the higher occupancy it allows.)
struct FwdTileCfg {
    int kv_rows;    // K / V rows per buffer (multiple of 16)
    int rel_rows;   // relation rows per buffer (multiple of 16)
    int qr_stride;  // floats per row of the per-warp Q R^T scratch
    int q_off, k_off, v_off, r_off, qr_off, bnd_off;  // byte offsets in shared memory
    size_t bytes;
};

FwdTileCfg make_fwd_tile_cfg(const TreeParams& t, int chunks) {
    FwdTileCfg c;
    c.kv_rows = min(kMaxKvRows, (t.kc + 143) & ~15);  // 15 alignment + 64 + k + 2 nodes + 31 block overrun, rounded
    c.rel_rows = min(kMaxRelRows, (t.k + 1 + 15) & ~15);
    c.qr_stride = c.rel_rows - 4;                      // even, >= k + 1, not a multiple of 32 floats (bank spread)
    if (c.qr_stride < t.k + 1) c.qr_stride = c.rel_rows + 4;
    c.q_off = 0;
    c.k_off = kTileTokens * 128;
    c.v_off = c.k_off + c.kv_rows * 128;
    c.r_off = c.v_off + c.kv_rows * 128;
    c.qr_off = c.r_off + c.rel_rows * 128;
    c.bnd_off = c.qr_off + 4 * 16 * c.qr_stride * 4;
    c.bytes = (size_t)c.bnd_off + (size_t)chunks * (kTileTokens * 8 + 8);
    return c;
}

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// kDrop: attention dropout compiled in or out (the plain kernel carries none of it).  NG: 16-key groups per
// step of the key loop (2 = 32 keys; 1 = 16 keys, which skips more of the masked columns when k is small).
template <bool kDrop, int NG>
__global__ void __launch_bounds__(128)
fwd_tile_kernel(TreeParams t, FwdTileCfg cfg, int n_left, int n_right,
                const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ r,
                __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int H, float scale_log2e,
                const int32_t* __restrict__ lengths, DropoutParams drop) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* q_s = smem + cfg.q_off;
    unsigned char* k_s = smem + cfg.k_off;
    unsigned char* v_s = smem + cfg.v_off;
    unsigned char* r_s = smem + cfg.r_off;
    float* qr_s = reinterpret_cast<float*>(smem + cfg.qr_off);
    int2* bnd = reinterpret_cast<int2*>(smem + cfg.bnd_off);
    const int chunks = n_left + n_right;
    int2* crange = bnd + chunks * kTileTokens;

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int g = lane >> 2, c2 = (lane & 3) * 2;
    const int t0 = blockIdx.x * kTileTokens, h = blockIdx.y, b = blockIdx.z;
    const int N = 2 * t.n - 1;
    const size_t rs = (size_t)H * 64;
    const size_t boff = (size_t)b * N * rs + (size_t)h * 64;
    const uint32_t q_u = smem_u32(q_s), k_u = smem_u32(k_s), v_u = smem_u32(v_s), r_u = smem_u32(r_s);

    // ---- prologue: Q tile, the tokens' own K / V rows and r^self; per-row ranges -------
    for (int idx = tid; idx < kTileTokens * 8; idx += 128) {
        const int row = idx >> 3, ch = idx & 7;
        const size_t src = boff + (size_t)(t0 + row) * rs + ch * 8;
        cp_async16(q_u + tile_off(row, ch), q + src);
        cp_async16(k_u + tile_off(row, ch), k + src);
        cp_async16(v_u + tile_off(row, ch), v + src);
    }
    if (tid < 8) cp_async16(r_u + tile_off(0, tid), r + tid * 8);
    cp_async_commit();
    if (tid < kTileTokens) fill_row_bounds(t, t0, tid, n_left, n_right, bnd);
    cp_async_wait<0>();
    __syncthreads();
    for (int c = w; c < chunks; c += 4) {
        const int2 a = rows_union(bnd + c * kTileTokens, 0, 32, lane);
        const int2 bb = rows_union(bnd + c * kTileTokens, 32, 32, lane);
        if (lane == 0) crange[c] = make_int2(min(a.x, bb.x), max(a.y, bb.y));
    }
    const int len = seq_len(lengths, b, t.n);
    if (len < t.n) {  // short sequence: the staged ranges stay those of the full graph, the rows' ranges shrink
        __syncthreads();
        if (tid < kTileTokens) mask_row_bounds(t, t0, tid, n_left, n_right, bnd, len);
    }

    const int r0 = w * 16;
    uint32_t qa[4][4];
    load_a_frags(q_u, r0, lane, qa);

    // running softmax state of rows r0+g (index 0) and r0+g+8 (index 1); the self loop starts it
    float m_run[2], l_run[2], o[8][4];
    {
        float dot[2] = {0.f, 0.f};
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const uint32_t rr = *reinterpret_cast<const uint32_t*>(r_s + tile_off(0, nt) + c2 * 2);
            const float r_lo = __uint_as_float(rr << 16), r_hi = __uint_as_float(rr & 0xffff0000u);
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int row = r0 + g + hh * 8;
                const uint32_t off = tile_off(row, nt) + c2 * 2;
                const uint32_t qq = *reinterpret_cast<const uint32_t*>(q_s + off);
                const uint32_t kk = *reinterpret_cast<const uint32_t*>(k_s + off);
                const uint32_t vv = *reinterpret_cast<const uint32_t*>(v_s + off);
                dot[hh] = fmaf(__uint_as_float(qq << 16), __uint_as_float(kk << 16) + r_lo, dot[hh]);
                dot[hh] = fmaf(__uint_as_float(qq & 0xffff0000u), __uint_as_float(kk & 0xffff0000u) + r_hi, dot[hh]);
                o[nt][hh * 2] = __uint_as_float(vv << 16);
                o[nt][hh * 2 + 1] = __uint_as_float(vv & 0xffff0000u);
            }
        }
        if constexpr (kDrop) {  // dropout on the self loop's weight (the softmax sum keeps the undropped weight)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const uint32_t tok = (uint32_t)(t0 + r0 + g + hh * 8);
                const float wgt = dropout_weight(drop, (uint32_t)(b * H + h), tok, tok);
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) { o[nt][hh * 2] *= wgt; o[nt][hh * 2 + 1] *= wgt; }
            }
        }
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            dot[hh] += __shfl_xor_sync(0xffffffffu, dot[hh], 1);
            dot[hh] += __shfl_xor_sync(0xffffffffu, dot[hh], 2);
            m_run[hh] = dot[hh] * scale_log2e;
            l_run[hh] = (lane & 3) == 0 ? 1.f : 0.f;  // per-thread partial; summed over the quad at the end
        }
    }

    const int kQrStride = cfg.qr_stride;
    float* qr_w = qr_s + w * 16 * kQrStride;
    const int W = t.k + 1;

    auto next_chunk = [&](int c) {  // next chunk this tile reaches
        int cn = c + 1;
        while (cn < chunks && crange[cn].x > crange[cn].y) ++cn;
        return cn;
    };
    // K / V rows of the chunk's node range and its relation rows -> shared memory (async)
    auto stage = [&](int c) {
        const int2 cr = crange[c];
        const int side = c >= n_left, level = side ? c - n_left : c;
        const int n_l = t.n >> level, id_base = node_id(t.n, level, 0);
        const int rel_base = side ? rel_right(t, level, 0) : rel_left(t, level, 0);
        const int base = cr.x & ~15;
        const int nr = min(cfg.kv_rows, (cr.y - base + 1 + 31 + 15) & ~15);
        for (int idx = tid; idx < nr * 8; idx += 128) {
            const int row = idx >> 3, ch = idx & 7;
            const int node = min(base + row, n_l - 1);
            const size_t src = boff + (size_t)(id_base + node) * rs + ch * 8;
            if (!BPT_IDX_OK(id_base + node, 2 * t.n - 1, BPT_SITE_NODE)) continue;
            cp_async16(k_u + tile_off(row, ch), k + src);
            cp_async16(v_u + tile_off(row, ch), v + src);
        }
        for (int idx = tid; idx < cfg.rel_rows * 8; idx += 128) {
            const int row = idx >> 3, ch = idx & 7;
            if (row < W && BPT_IDX_OK(rel_base + row, 1 + 2 * t.L * (t.k + 1) + t.L, BPT_SITE_RELATION)) cp_async16(r_u + tile_off(row, ch), r + (size_t)(rel_base + row) * 64 + ch * 8);
            else *reinterpret_cast<uint4*>(r_s + tile_off(row, ch)) = make_uint4(0, 0, 0, 0);
        }
        cp_async_commit();
    };

    __syncthreads();  // the prologue's reads of the K / V / R buffers are done; crange (and the masked ranges) are visible
    int c = next_chunk(-1);
    if (c < chunks) stage(c);
    while (c < chunks) {
        const int cn = next_chunk(c);
        cp_async_wait<0>();
        __syncthreads();  // this chunk's rows are in place
        const int2 cr = crange[c];
        const int side = c >= n_left;
        const int level = side ? c - n_left : c;
        const int id_base = node_id(t.n, level, 0);
        const int base = cr.x & ~15;

        const int2* bc = bnd + c * kTileTokens;
        const int2 wr = rows_union(bc, r0, 16, lane);
        if (wr.x <= wr.y) {  // uniform over the warp

        // Q R^T for this chunk's relation rows -> per-warp scratch
#pragma unroll
        for (int np = 0; np < kMaxRelRows / 16; ++np) {
            if (np * 16 < W) {
                float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    uint32_t bf[4];
                    load_b_rows(r_u, np * 16, ks, lane, bf);
                    mma_bf16(acc[0], qa[ks], bf[0], bf[1]);
                    mma_bf16(acc[1], qa[ks], bf[2], bf[3]);
                }
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    const int col = np * 16 + j * 8 + c2;
                    if (col < kQrStride) {
                        *reinterpret_cast<float2*>(qr_w + g * kQrStride + col) = make_float2(acc[j][0], acc[j][1]);
                        *reinterpret_cast<float2*>(qr_w + (g + 8) * kQrStride + col) = make_float2(acc[j][2], acc[j][3]);
                    }
                }
            }
        }
        __syncwarp();

        const int2 ba = bc[r0 + g], bb = bc[r0 + g + 8];
        const int lo_r[2] = {ba.x, bb.x}, hi_r[2] = {ba.y, bb.y};
        const int kstart = (wr.x - base) & ~15, kend = wr.y - base;
        for (int kb = kstart; kb <= kend; kb += 16 * NG) {
            float s[2 * NG][4];
#pragma unroll
            for (int j = 0; j < 2 * NG; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
                for (int np = 0; np < NG; ++np) {
                    uint32_t bf[4];
                    load_b_rows(k_u, kb + np * 16, ks, lane, bf);
                    mma_bf16(s[np * 2], qa[ks], bf[0], bf[1]);
                    mma_bf16(s[np * 2 + 1], qa[ks], bf[2], bf[3]);
                }
            }
            // relative-position term, mask, running max
            float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
            for (int j = 0; j < 2 * NG; ++j) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int hh = e >> 1;
                    const int m = base + kb + j * 8 + c2 + (e & 1);
                    const bool ok = m >= lo_r[hh] && m <= hi_r[hh];
                    float val = -INFINITY;
                    if (ok) {
                        const int off = side ? m - lo_r[hh] : hi_r[hh] - m;
                        val = (s[j][e] + qr_w[(g + hh * 8) * kQrStride + off]) * scale_log2e;
                    }
                    s[j][e] = val;
                    mx[hh] = fmaxf(mx[hh], val);
                }
            }
            float corr[2];
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 1));
                mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 2));
                const float m_new = fmaxf(m_run[hh], mx[hh]);  // finite: the self loop seeded m_run
                corr[hh] = ex2(m_run[hh] - m_new);
                m_run[hh] = m_new;
                l_run[hh] *= corr[hh];
            }
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                o[nt][0] *= corr[0]; o[nt][1] *= corr[0];
                o[nt][2] *= corr[1]; o[nt][3] *= corr[1];
            }
            uint32_t pa[NG][4];
#pragma unroll
            for (int j = 0; j < 2 * NG; ++j) {
                float p0 = ex2(s[j][0] - m_run[0]), p1 = ex2(s[j][1] - m_run[0]);
                float p2 = ex2(s[j][2] - m_run[1]), p3 = ex2(s[j][3] - m_run[1]);
                l_run[0] += p0 + p1;
                l_run[1] += p2 + p3;
                if constexpr (kDrop) {  // the weights that reach V are dropped, the softmax sum is not
                    const uint32_t bh = (uint32_t)(b * H + h), src = (uint32_t)(id_base + base + kb + j * 8 + c2);
                    const uint32_t d0 = (uint32_t)(t0 + r0 + g), d1 = d0 + 8;
                    p0 *= dropout_weight(drop, bh, d0, src); p1 *= dropout_weight(drop, bh, d0, src + 1);
                    p2 *= dropout_weight(drop, bh, d1, src); p3 *= dropout_weight(drop, bh, d1, src + 1);
                }
                pa[j >> 1][(j & 1) * 2] = pack_bf16(p0, p1);
                pa[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
            }
#pragma unroll
            for (int kk = 0; kk < NG; ++kk) {
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    uint32_t bf[4];
                    load_b_cols(v_u, kb + kk * 16, np, lane, bf);
                    mma_bf16(o[np * 2], pa[kk], bf[0], bf[1]);
                    mma_bf16(o[np * 2 + 1], pa[kk], bf[2], bf[3]);
                }
            }
        }
        }
        __syncthreads();  // everyone is done with the buffers
        if (cn < chunks) stage(cn);
        c = cn;
    }

    // ---- epilogue: normalise, round once to bf16, coalesced stores through the Q tile -----
    float inv[2];
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 1);
        l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 2);
        inv[hh] = t0 + r0 + g + hh * 8 < len ? 1.f / l_run[hh] : 0.f;  // a placeholder token's row is zero
    }
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        *reinterpret_cast<uint32_t*>(q_s + tile_off(r0 + g, nt) + c2 * 2) = pack_bf16(o[nt][0] * inv[0], o[nt][1] * inv[0]);
        *reinterpret_cast<uint32_t*>(q_s + tile_off(r0 + g + 8, nt) + c2 * 2) = pack_bf16(o[nt][2] * inv[1], o[nt][3] * inv[1]);
    }
    if ((lane & 3) == 0) {
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
            lse[((size_t)b * N + t0 + r0 + g + hh * 8) * H + h] = inv[hh] > 0.f ? (m_run[hh] + log2f(l_run[hh])) * kLn2 : 0.f;
    }
    __syncwarp();
    for (int idx = lane; idx < 16 * 8; idx += 32) {
        const int row = r0 + (idx >> 3), ch = idx & 7;
        *reinterpret_cast<uint4*>(out + boff + (size_t)(t0 + row) * rs + ch * 8) =
            *reinterpret_cast<const uint4*>(q_s + tile_off(row, ch));
    }
}

}  // namespace

// Token rows of the forward on the tensor cores; the span rows are left to the caller.
bpt_status launch_fwd_tile(const AttnProblem& p) {
    int n_left, n_right;
    context_levels(p.tree, &n_left, &n_right);
    const FwdTileCfg cfg = make_fwd_tile_cfg(p.tree, n_left + n_right);
    const size_t smem = cfg.bytes;
    const bool narrow = p.tree.k <= 8;  // measured: 16-key steps win a few percent for k <= 8 and lose at k = 16
    auto kernel = p.drop.thr ? (narrow ? fwd_tile_kernel<true, 1> : fwd_tile_kernel<true, 2>)
                             : (narrow ? fwd_tile_kernel<false, 1> : fwd_tile_kernel<false, 2>);
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) != cudaSuccess)
        return BPT_ERR_CUDA;
    if (smem > 200 * 1024 || p.H > 65535 || p.B > 65535) return BPT_ERR_UNSUPPORTED;
    const dim3 grid(p.tree.n / kTileTokens, p.H, p.B);
    kernel<<<grid, 128, smem, p.stream>>>(p.tree, cfg, n_left, n_right, (const __nv_bfloat16*)p.q,
                                          (const __nv_bfloat16*)p.k, (const __nv_bfloat16*)p.v,
                                          (const __nv_bfloat16*)p.rel_emb, (__nv_bfloat16*)p.out, p.lse, p.H,
                                          p.scale * kLog2e, p.lengths, p.drop);
    trace_mark(p.stream, "fwd_tile");
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

}  // namespace bpt
