// Span rows (affiliated edges, arXiv 1911.04070 Sec. 3.2.2: every span attends the tokens it
// contains, all with the relation r^anc of its level, Sec. 3.4), forward and backward, bf16,
// head size 64.
//
// One CTA = 64 consecutive tokens of one (batch entry, head); their K / V rows are staged once.
// Every span that meets the tile is a query row of one small dense product against those 64
// keys: the 63 spans of levels 1..6 that lie inside the tile (rows 0..62, level by level) are
// finished here; the ancestors of levels 7..L cover the whole tile and many others, so for
// them the CTA emits a partial (running max, sum, weighted V sum in the forward; partial dq in
// the backward) that a small merge kernel combines over the tiles in tile order.  In the
// backward the tile also produces, for its 64 tokens, the complete contribution of all spans
// to dk and dv (a [64][128] fp32 block that the source-side gather adds).
#include "bounds_check.cuh"
#include "bpt_internal.cuh"
#include "mma_tools.cuh"
#include "row_map.cuh"
#include "tile_geom.cuh"

namespace bpt {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kSpanRows = 80;      // 63 inner spans, one unused row, up to 16 outer ancestors
constexpr int kInnerLevels = 6;    // log2(kTileTokens)
constexpr int kExtStride = 66;     // floats per forward partial: max, sum, 64 channels
constexpr int kPsStride = 144;     // bytes per span row of the P / dS tiles (64 bf16 + 16)
constexpr int kSpanThreads = 160;  // 5 warps x 16 span rows

struct SpanRow {
    int node;     // node id, -1 for an unused row
    int lo, hi;   // tokens of the tile it covers (local indices)
    int level;
};

// Row r of the tile's span matrix; `len` = real tokens of the sequence (a span attends only those).
__device__ __forceinline__ SpanRow span_row(const TreeParams& t, int t0, int r, int len) {
    SpanRow s;
    s.node = -1; s.lo = 1; s.hi = 0; s.level = 1;
    if (r < kTileTokens - 1) {
        const int rem = kTileTokens - r;                      // 64 .. 2
        const int j = 7 - (32 - __clz(rem - 1));              // level 1 holds rows 0..31, level 2 rows 32..47, ...
        const int x = r - (kTileTokens - (2 * kTileTokens >> j));
        if (j <= t.L) {
            s.level = j;
            s.node = node_id(t.n, j, (t0 >> j) + x);
            s.lo = x << j;
            s.hi = ((x + 1) << j) - 1;
        }
    } else if (r >= kTileTokens) {
        const int j = kInnerLevels + 1 + (r - kTileTokens);
        if (j <= t.L) {
            s.level = j;
            s.node = node_id(t.n, j, t0 >> j);
            s.lo = 0;
            s.hi = kTileTokens - 1;
        }
    }
    s.hi = min(s.hi, len - 1 - t0);
    if (s.lo > s.hi) { s.lo = 1; s.hi = 0; }  // no real token of this tile under the span
    return s;
}

struct SpanMeta {
    int node[kSpanRows], lo[kSpanRows], hi[kSpanRows], level[kSpanRows];
    float bias[kSpanRows];   // q . r^anc(level), scaled to the base-2 exponent
    float lse2[kSpanRows];   // backward: lse * log2(e)
    float delta[kSpanRows];  // backward: d_out . out
};

// ------------------------------------------------------------------------------------------
// forward
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSpanThreads)
fwd_span_kernel(TreeParams t, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ r,
                __nv_bfloat16* __restrict__ out, float* __restrict__ lse, float* __restrict__ ext_part,
                int H, int n_ext, float scale_log2e, const int32_t* __restrict__ lengths, DropoutParams drop) {
    __shared__ __align__(128) unsigned char qs_s[kSpanRows * 128];
    __shared__ __align__(128) unsigned char k_s[kTileTokens * 128];
    __shared__ __align__(128) unsigned char v_s[kTileTokens * 128];
    __shared__ SpanMeta meta;
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int g = lane >> 2, c2 = (lane & 3) * 2;
    const int tile = blockIdx.x, tiles = gridDim.x, t0 = tile * kTileTokens, h = blockIdx.y, b = blockIdx.z;
    const int N = 2 * t.n - 1;
    const size_t rs = (size_t)H * 64;
    const size_t boff = (size_t)b * N * rs + (size_t)h * 64;
    const uint32_t qs_u = smem_u32(qs_s), k_u = smem_u32(k_s), v_u = smem_u32(v_s);

    if (tid < kSpanRows) {
        const SpanRow s = span_row(t, t0, tid, seq_len(lengths, b, t.n));
        meta.node[tid] = s.node; meta.lo[tid] = s.lo; meta.hi[tid] = s.hi; meta.level[tid] = s.level;
    }
    __syncthreads();
    for (int idx = tid; idx < kSpanRows * 8; idx += kSpanThreads) {
        const int row = idx >> 3, ch = idx & 7;
        if (meta.node[row] >= 0 && BPT_IDX_OK(meta.node[row], N, BPT_SITE_NODE)) cp_async16(qs_u + tile_off(row, ch), q + boff + (size_t)meta.node[row] * rs + ch * 8);
        else *reinterpret_cast<uint4*>(qs_s + tile_off(row, ch)) = make_uint4(0, 0, 0, 0);
    }
    for (int idx = tid; idx < kTileTokens * 8; idx += kSpanThreads) {
        const int row = idx >> 3, ch = idx & 7;
        const size_t src = boff + (size_t)(t0 + row) * rs + ch * 8;
        cp_async16(k_u + tile_off(row, ch), k + src);
        cp_async16(v_u + tile_off(row, ch), v + src);
    }
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();
    {   // bias of a row: q . r^anc(level), two threads per row
        const int row = tid >> 1, half = tid & 1;
        const __nv_bfloat16* rr = r + (size_t)rel_anc(t, meta.level[row]) * 64 + half * 32;
        float acc = 0.f;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            const uint4 a = *reinterpret_cast<const uint4*>(qs_s + tile_off(row, half * 4 + ch));
            const uint4 o = __ldg(reinterpret_cast<const uint4*>(rr) + ch);
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, ow[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                acc = fmaf(__uint_as_float(aw[x] << 16), __uint_as_float(ow[x] << 16), acc);
                acc = fmaf(__uint_as_float(aw[x] & 0xffff0000u), __uint_as_float(ow[x] & 0xffff0000u), acc);
            }
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        if (half == 0) meta.bias[row] = acc * scale_log2e;
    }
    __syncthreads();

    const int r0 = w * 16;
    uint32_t qa[4][4];
    load_a_frags(qs_u, r0, lane, qa);
    // keys this warp's rows touch: level-1 rows only reach half of the tile
    const int kb0 = w == 1 ? 32 : 0, kb1 = w == 0 ? 32 : 64;
    float s[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
#pragma unroll
    for (int kb = 0; kb < 64; kb += 16) {
        if (kb >= kb0 && kb < kb1) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                uint32_t bf[4];
                load_b_rows(k_u, kb, ks, lane, bf);
                mma_bf16(s[kb / 8], qa[ks], bf[0], bf[1]);
                mma_bf16(s[kb / 8 + 1], qa[ks], bf[2], bf[3]);
            }
        }
    }
    int lo_r[2], hi_r[2];
    float bias_r[2], mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        lo_r[hh] = meta.lo[r0 + g + hh * 8]; hi_r[hh] = meta.hi[r0 + g + hh * 8]; bias_r[hh] = meta.bias[r0 + g + hh * 8];
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int hh = e >> 1, m = j * 8 + c2 + (e & 1);
            const bool ok = m >= lo_r[hh] && m <= hi_r[hh];
            s[j][e] = ok ? fmaf(s[j][e], scale_log2e, bias_r[hh]) : -INFINITY;
            mx[hh] = fmaxf(mx[hh], s[j][e]);
        }
    }
    float l_run[2] = {0.f, 0.f};
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 1));
        mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 2));
    }
    const float m_use[2] = {mx[0] == -INFINITY ? 0.f : mx[0], mx[1] == -INFINITY ? 0.f : mx[1]};  // unused rows
    uint32_t pa[4][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float p0 = fast_exp2(s[j][0] - m_use[0]), p1 = fast_exp2(s[j][1] - m_use[0]);
        float p2 = fast_exp2(s[j][2] - m_use[1]), p3 = fast_exp2(s[j][3] - m_use[1]);
        l_run[0] += p0 + p1;
        l_run[1] += p2 + p3;
        if (drop.thr) {  // the weights that reach V are dropped, the softmax sum is not
            const uint32_t bh = (uint32_t)(b * H + h), src = (uint32_t)(t0 + j * 8 + c2);
            const uint32_t d0 = (uint32_t)meta.node[r0 + g], d1 = (uint32_t)meta.node[r0 + g + 8];
            p0 *= dropout_weight(drop, bh, d0, src); p1 *= dropout_weight(drop, bh, d0, src + 1);
            p2 *= dropout_weight(drop, bh, d1, src); p3 *= dropout_weight(drop, bh, d1, src + 1);
        }
        pa[j >> 1][(j & 1) * 2] = pack_bf16(p0, p1);
        pa[j >> 1][(j & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    float o[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
        if (kk * 16 >= kb0 && kk * 16 < kb1) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t bf[4];
                load_b_cols(v_u, kk * 16, np, lane, bf);
                mma_bf16(o[np * 2], pa[kk], bf[0], bf[1]);
                mma_bf16(o[np * 2 + 1], pa[kk], bf[2], bf[3]);
            }
        }
    }
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 1);
        l_run[hh] += __shfl_xor_sync(0xffffffffu, l_run[hh], 2);
    }

    if (w < 4) {  // inner spans: finished here; rounded once and stored through the staging tile
        __syncwarp();
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int row = r0 + g + hh * 8;
            const float inv = l_run[hh] > 0.f ? 1.f / l_run[hh] : 0.f;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt)
                *reinterpret_cast<uint32_t*>(qs_s + tile_off(row, nt) + c2 * 2) = pack_bf16(o[nt][hh * 2] * inv, o[nt][hh * 2 + 1] * inv);
            if ((lane & 3) == 0 && meta.node[row] >= 0)  // a span without real tokens: out = 0, lse = 0
                lse[((size_t)b * N + meta.node[row]) * H + h] = l_run[hh] > 0.f ? (mx[hh] + log2f(l_run[hh])) * kLn2 : 0.f;
        }
        __syncwarp();
        for (int idx = lane; idx < 16 * 8; idx += 32) {
            const int row = r0 + (idx >> 3), ch = idx & 7;
            if (meta.node[row] >= 0)
                *reinterpret_cast<uint4*>(out + boff + (size_t)meta.node[row] * rs + ch * 8) =
                    *reinterpret_cast<const uint4*>(qs_s + tile_off(row, ch));
        }
    } else {      // outer ancestors: partial state of this tile
        const int pair = b * H + h;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int e = g + hh * 8;
            if (e < n_ext) {
                float* dst = ext_part + (((size_t)pair * tiles + tile) * n_ext + e) * kExtStride;
                if ((lane & 3) == 0) { dst[0] = mx[hh]; dst[1] = l_run[hh]; }
#pragma unroll
                for (int nt = 0; nt < 8; ++nt)
                    *reinterpret_cast<float2*>(dst + 2 + nt * 8 + c2) = make_float2(o[nt][hh * 2], o[nt][hh * 2 + 1]);
            }
        }
    }
}

// Outer ancestors of the forward: merge the tiles' partial states in tile order.
// One warp per (pair, span), the root first; lane c holds channels 2c, 2c + 1.
__global__ void __launch_bounds__(128)
fwd_span_merge_kernel(TreeParams t, const float* __restrict__ ext_part, __nv_bfloat16* __restrict__ out,
                      float* __restrict__ lse, int H, int n_pairs, int tiles, int n_ext) {
    const int lane = threadIdx.x & 31;
    const int n_outer = (t.n >> kInnerLevels) - 1;  // spans of levels 7..L, in node-id order
    const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= (int64_t)n_pairs * n_outer) return;
    const int pair = (int)(wid / n_outer), b = pair / H, h = pair % H;
    const int node = 2 * t.n - 2 - (int)(wid % n_outer);  // root first
    const int j = node_level(t.n, node), mi = node - node_id(t.n, j, 0), e = j - kInnerLevels - 1;
    const int T0 = mi << (j - kInnerLevels), nT = 1 << (j - kInnerLevels);
    const float* base = ext_part + (((size_t)pair * tiles + T0) * n_ext + e) * kExtStride;
    const size_t stride = (size_t)n_ext * kExtStride;
    // Lane c holds channels 2c, 2c + 1 and adds the tiles' rows in tile order (coalesced row loads); the tiles'
    // rescaling factors are computed 32 at a time, one per lane, and handed round by shuffle.
    float mx = -INFINITY;
    for (int x = lane; x < nT; x += 32) mx = fmaxf(mx, base[(size_t)x * stride]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (mx == -INFINITY) mx = 0.f;  // a span without real tokens: every partial is empty (2^-inf = 0 below)
    float l = 0.f, a0 = 0.f, a1 = 0.f;
    for (int x0 = 0; x0 < nT; x0 += 32) {
        float f = 0.f, lf = 0.f;
        if (x0 + lane < nT) {
            const float* p = base + (size_t)(x0 + lane) * stride;
            f = fast_exp2(p[0] - mx);
            lf = p[1] * f;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lf += __shfl_xor_sync(0xffffffffu, lf, o);
        l += lf;
        const float* row = base + (size_t)x0 * stride + 2 + 2 * lane;
        if (x0 + 32 <= nT) {
            float2 a[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) a[i] = *reinterpret_cast<const float2*>(row + (size_t)i * stride);
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float fi = __shfl_sync(0xffffffffu, f, i);
                a0 = fmaf(a[i].x, fi, a0);
                a1 = fmaf(a[i].y, fi, a1);
            }
        } else {
            for (int i = 0; i < nT - x0; ++i) {
                const float fi = __shfl_sync(0xffffffffu, f, i);
                const float2 a = *reinterpret_cast<const float2*>(row + (size_t)i * stride);
                a0 = fmaf(a.x, fi, a0);
                a1 = fmaf(a.y, fi, a1);
            }
        }
    }
    const float inv = l > 0.f ? 1.f / l : 0.f;  // l = 0: a span without real tokens
    const size_t rs = (size_t)H * 64;
    *reinterpret_cast<uint32_t*>(out + ((size_t)b * (2 * t.n - 1) + node) * rs + (size_t)h * 64 + lane * 2) = pack_bf16(a0 * inv, a1 * inv);
    if (lane == 0) lse[((size_t)b * (2 * t.n - 1) + node) * H + h] = l > 0.f ? (mx + log2f(l)) * kLn2 : 0.f;
}

// ------------------------------------------------------------------------------------------
// backward
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kSpanThreads)
bwd_span_kernel(TreeParams t, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ r,
                const __nv_bfloat16* __restrict__ out, const float* __restrict__ lse,
                const __nv_bfloat16* __restrict__ d_out, __nv_bfloat16* __restrict__ dq,
                float* __restrict__ ext_dq, float* __restrict__ aff_slab,
                int H, int pair0, int n_ext, float scale, const int32_t* __restrict__ lengths, DropoutParams drop) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* qs_s = smem;
    unsigned char* gs_s = qs_s + kSpanRows * 128;
    unsigned char* k_s = gs_s + kSpanRows * 128;
    unsigned char* v_s = k_s + kTileTokens * 128;
    unsigned char* p_s = v_s + kTileTokens * 128;
    unsigned char* ds_s = p_s + kSpanRows * kPsStride;
    SpanMeta& meta = *reinterpret_cast<SpanMeta*>(ds_s + kSpanRows * kPsStride);
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int g = lane >> 2, c2 = (lane & 3) * 2;
    const int tile = blockIdx.x, tiles = gridDim.x, t0 = tile * kTileTokens;
    const int pair = pair0 + blockIdx.y, b = pair / H, h = pair % H;
    const int N = 2 * t.n - 1;
    const size_t rs = (size_t)H * 64;
    const size_t boff = (size_t)b * N * rs + (size_t)h * 64;
    const uint32_t qs_u = smem_u32(qs_s), gs_u = smem_u32(gs_s), k_u = smem_u32(k_s), v_u = smem_u32(v_s),
                   p_u = smem_u32(p_s), ds_u = smem_u32(ds_s);
    const float scale_log2e = scale * kLog2e;
    unsigned char* o_s = p_s;  // the spans' forward outputs, only until the row terms are known (80 x 128 <= 80 x 144)

    if (tid < kSpanRows) {
        const SpanRow s = span_row(t, t0, tid, seq_len(lengths, b, t.n));
        meta.node[tid] = s.node; meta.lo[tid] = s.lo; meta.hi[tid] = s.hi; meta.level[tid] = s.level;
        meta.lse2[tid] = s.node >= 0 ? lse[((size_t)b * N + s.node) * H + h] * kLog2e : 0.f;
    }
    __syncthreads();
    for (int idx = tid; idx < kSpanRows * 8; idx += kSpanThreads) {
        const int row = idx >> 3, ch = idx & 7;
        if (meta.node[row] >= 0 && BPT_IDX_OK(meta.node[row], N, BPT_SITE_NODE)) {
            const size_t src = boff + (size_t)meta.node[row] * rs + ch * 8;
            cp_async16(qs_u + tile_off(row, ch), q + src);
            cp_async16(gs_u + tile_off(row, ch), d_out + src);
            cp_async16(p_u + row * 128 + ch * 16, out + src);
        } else {
            *reinterpret_cast<uint4*>(qs_s + tile_off(row, ch)) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4*>(gs_s + tile_off(row, ch)) = make_uint4(0, 0, 0, 0);
            *reinterpret_cast<uint4*>(o_s + row * 128 + ch * 16) = make_uint4(0, 0, 0, 0);
        }
    }
    for (int idx = tid; idx < kTileTokens * 8; idx += kSpanThreads) {
        const int row = idx >> 3, ch = idx & 7;
        const size_t src = boff + (size_t)(t0 + row) * rs + ch * 8;
        cp_async16(k_u + tile_off(row, ch), k + src);
        cp_async16(v_u + tile_off(row, ch), v + src);
    }
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();
    {   // per row: bias = q . r^anc(level) and delta = d_out . out, two threads per row
        const int row = tid >> 1, half = tid & 1;
        const __nv_bfloat16* rr = r + (size_t)rel_anc(t, meta.level[row]) * 64 + half * 32;
        float acc = 0.f, del = 0.f;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            const uint4 a = *reinterpret_cast<const uint4*>(qs_s + tile_off(row, half * 4 + ch));
            const uint4 o = __ldg(reinterpret_cast<const uint4*>(rr) + ch);
            const uint4 gg = *reinterpret_cast<const uint4*>(gs_s + tile_off(row, half * 4 + ch));
            const uint4 oo = *reinterpret_cast<const uint4*>(o_s + row * 128 + (half * 4 + ch) * 16);
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, ow[4] = {o.x, o.y, o.z, o.w};
            const uint32_t gw[4] = {gg.x, gg.y, gg.z, gg.w}, pw[4] = {oo.x, oo.y, oo.z, oo.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                acc = fmaf(__uint_as_float(aw[x] << 16), __uint_as_float(ow[x] << 16), acc);
                acc = fmaf(__uint_as_float(aw[x] & 0xffff0000u), __uint_as_float(ow[x] & 0xffff0000u), acc);
                del = fmaf(__uint_as_float(gw[x] << 16), __uint_as_float(pw[x] << 16), del);
                del = fmaf(__uint_as_float(gw[x] & 0xffff0000u), __uint_as_float(pw[x] & 0xffff0000u), del);
            }
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        del += __shfl_xor_sync(0xffffffffu, del, 1);
        if (half == 0) { meta.bias[row] = acc * scale_log2e; meta.delta[row] = del; }
    }
    __syncthreads();  // the outputs in p_s are consumed; phase 1 overwrites them

    // ---- phase 1: this warp's 16 span rows ----
    const int r0 = w * 16;
    {
        uint32_t qa[4][4], ga[4][4];
        load_a_frags(qs_u, r0, lane, qa);
        load_a_frags(gs_u, r0, lane, ga);
        float s[8][4], dp[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
            dp[j][0] = dp[j][1] = dp[j][2] = dp[j][3] = 0.f;
        }
#pragma unroll
        for (int kb = 0; kb < 64; kb += 16) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                uint32_t bf[4];
                load_b_rows(k_u, kb, ks, lane, bf);
                mma_bf16(s[kb / 8], qa[ks], bf[0], bf[1]);
                mma_bf16(s[kb / 8 + 1], qa[ks], bf[2], bf[3]);
                load_b_rows(v_u, kb, ks, lane, bf);
                mma_bf16(dp[kb / 8], ga[ks], bf[0], bf[1]);
                mma_bf16(dp[kb / 8 + 1], ga[ks], bf[2], bf[3]);
            }
        }
        int lo_r[2], hi_r[2], lvl_r[2];
        float bias_r[2], lse_r[2], del_r[2], rowsum[2] = {0.f, 0.f};
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int row = r0 + g + hh * 8;
            lo_r[hh] = meta.lo[row]; hi_r[hh] = meta.hi[row]; lvl_r[hh] = meta.level[row];
            bias_r[hh] = meta.bias[row]; lse_r[hh] = meta.lse2[row]; del_r[hh] = meta.delta[row];
        }
        uint32_t da[4][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            float pv[4], dv[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int hh = e >> 1, m = j * 8 + c2 + (e & 1);
                const bool ok = m >= lo_r[hh] && m <= hi_r[hh];
                float p = 0.f, d = 0.f;
                if (ok) {
                    p = fast_exp2(fmaf(s[j][e], scale_log2e, bias_r[hh] - lse_r[hh]));
                    // dropout: dP = W d_out.v and the weight that reaches dv is W P; dS keeps the undropped P
                    const float wgt = drop.thr ? dropout_weight(drop, (uint32_t)(b * H + h), (uint32_t)meta.node[r0 + g + hh * 8], (uint32_t)(t0 + m)) : 1.f;
                    d = p * (dp[j][e] * wgt - del_r[hh]);
                    p *= wgt;
                }
                pv[e] = p; dv[e] = d;
                rowsum[hh] += d;
            }
            const uint32_t p01 = pack_bf16(pv[0], pv[1]), p23 = pack_bf16(pv[2], pv[3]);
            const uint32_t d01 = pack_bf16(dv[0], dv[1]), d23 = pack_bf16(dv[2], dv[3]);
            *reinterpret_cast<uint32_t*>(p_s + (r0 + g) * kPsStride + (j * 8 + c2) * 2) = p01;
            *reinterpret_cast<uint32_t*>(p_s + (r0 + g + 8) * kPsStride + (j * 8 + c2) * 2) = p23;
            *reinterpret_cast<uint32_t*>(ds_s + (r0 + g) * kPsStride + (j * 8 + c2) * 2) = d01;
            *reinterpret_cast<uint32_t*>(ds_s + (r0 + g + 8) * kPsStride + (j * 8 + c2) * 2) = d23;
            da[j >> 1][(j & 1) * 2] = d01;
            da[j >> 1][(j & 1) * 2 + 1] = d23;
        }
        float acc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) { acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t bf[4];
                load_b_cols(k_u, kk * 16, np, lane, bf);
                mma_bf16(acc[np * 2], da[kk], bf[0], bf[1]);
                mma_bf16(acc[np * 2 + 1], da[kk], bf[2], bf[3]);
            }
        }
        // + (sum of the row's dS) r^anc: all edges of the row carry that one relation
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            rowsum[hh] += __shfl_xor_sync(0xffffffffu, rowsum[hh], 1);
            rowsum[hh] += __shfl_xor_sync(0xffffffffu, rowsum[hh], 2);
            const __nv_bfloat16* rr = r + (size_t)rel_anc(t, lvl_r[hh]) * 64;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                const uint32_t rw = __ldg(reinterpret_cast<const uint32_t*>(rr + nt * 8 + c2));
                acc[nt][hh * 2] = fmaf(rowsum[hh], __uint_as_float(rw << 16), acc[nt][hh * 2]);
                acc[nt][hh * 2 + 1] = fmaf(rowsum[hh], __uint_as_float(rw & 0xffff0000u), acc[nt][hh * 2 + 1]);
            }
        }
        if (w == 4) {  // outer ancestors: partial dq of this tile
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int e = g + hh * 8;
                if (e < n_ext) {
                    float* dst = ext_dq + (((size_t)blockIdx.y * tiles + tile) * n_ext + e) * 64 + c2;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt)
                        *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(acc[nt][hh * 2], acc[nt][hh * 2 + 1]);
                }
            }
        }
        __syncthreads();  // P and dS are complete, and nobody reads the K / V tiles any more
        if (w < 4) {
            // inner spans: dq = scale * acc, rounded once; staged in this warp's rows of v_s (free after phase 1)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int row = r0 + g + hh * 8;
#pragma unroll
                for (int nt = 0; nt < 8; ++nt)
                    *reinterpret_cast<uint32_t*>(v_s + tile_off(row, nt) + c2 * 2) =
                        pack_bf16(acc[nt][hh * 2] * scale, acc[nt][hh * 2 + 1] * scale);
            }
            __syncwarp();
            for (int idx = lane; idx < 16 * 8; idx += 32) {
                const int row = r0 + (idx >> 3), ch = idx & 7;
                if (meta.node[row] >= 0)
                    *reinterpret_cast<uint4*>(dq + boff + (size_t)meta.node[row] * rs + ch * 8) =
                        *reinterpret_cast<const uint4*>(v_s + tile_off(row, ch));
            }
        }
    }

    // ---- phase 2: this warp's 16 tokens: dk_part = dS^T Q_span, dv_part = P^T dO_span ----
    if (w < 4) {
        float ak[8][4], av[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            ak[nt][0] = ak[nt][1] = ak[nt][2] = ak[nt][3] = 0.f;
            av[nt][0] = av[nt][1] = av[nt][2] = av[nt][3] = 0.f;
        }
#pragma unroll
        for (int ks = 0; ks < kSpanRows / 16; ++ks) {
            uint32_t a_ds[4], a_p[4];
            load_a_trans(ds_u, kPsStride, ks * 16, w * 16, lane, a_ds);
            load_a_trans(p_u, kPsStride, ks * 16, w * 16, lane, a_p);
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t bf[4];
                load_b_cols(qs_u, ks * 16, np, lane, bf);
                mma_bf16(ak[np * 2], a_ds, bf[0], bf[1]);
                mma_bf16(ak[np * 2 + 1], a_ds, bf[2], bf[3]);
                load_b_cols(gs_u, ks * 16, np, lane, bf);
                mma_bf16(av[np * 2], a_p, bf[0], bf[1]);
                mma_bf16(av[np * 2 + 1], a_p, bf[2], bf[3]);
            }
        }
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            float* dst = aff_slab + (((size_t)blockIdx.y * tiles + tile) * kTileTokens + w * 16 + g + hh * 8) * 128 + c2;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(ak[nt][hh * 2], ak[nt][hh * 2 + 1]);
                *reinterpret_cast<float2*>(dst + 64 + nt * 8) = make_float2(av[nt][hh * 2], av[nt][hh * 2 + 1]);
            }
        }
    }
}

// Outer ancestors of the backward: dq = scale * sum of the tiles' partials, in tile order.
__global__ void __launch_bounds__(128)
bwd_span_merge_kernel(TreeParams t, const float* __restrict__ ext_dq, __nv_bfloat16* __restrict__ dq,
                      int H, int pair0, int n_pairs, int tiles, int n_ext, float scale) {
    const int lane = threadIdx.x & 31;
    const int n_outer = (t.n >> kInnerLevels) - 1;
    const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= (int64_t)n_pairs * n_outer) return;
    const int pl = (int)(wid / n_outer), pair = pair0 + pl, b = pair / H, h = pair % H;
    const int node = 2 * t.n - 2 - (int)(wid % n_outer);
    const int j = node_level(t.n, node), mi = node - node_id(t.n, j, 0), e = j - kInnerLevels - 1;
    const int T0 = mi << (j - kInnerLevels), nT = 1 << (j - kInnerLevels);
    const float* base = ext_dq + (((size_t)pl * tiles + T0) * n_ext + e) * 64;
    const size_t stride = (size_t)n_ext * 64;
    // lane t takes tiles t, t + 32, ...; the lanes' sums are then added in a fixed butterfly order
    float acc[64];
#pragma unroll
    for (int c = 0; c < 64; ++c) acc[c] = 0.f;
    for (int x = lane; x < nT; x += 32) {
        const float4* p = reinterpret_cast<const float4*>(base + (size_t)x * stride);
#pragma unroll
        for (int c = 0; c < 16; ++c) {
            const float4 a = p[c];
            acc[4 * c] += a.x; acc[4 * c + 1] += a.y; acc[4 * c + 2] += a.z; acc[4 * c + 3] += a.w;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
        for (int c = 0; c < 64; ++c) acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], o);
    }
    float a0 = 0.f, a1 = 0.f;  // this lane's two channels (static register indices only)
#pragma unroll
    for (int c = 0; c < 32; ++c)
        if (c == lane) { a0 = acc[2 * c]; a1 = acc[2 * c + 1]; }
    const size_t rs = (size_t)H * 64;
    *reinterpret_cast<uint32_t*>(dq + ((size_t)b * (2 * t.n - 1) + node) * rs + (size_t)h * 64 + lane * 2) = pack_bf16(a0 * scale, a1 * scale);
}

int outer_levels(const TreeParams& t) { return t.L > kInnerLevels ? t.L - kInnerLevels : 0; }

constexpr size_t kBwdSpanSmem = 2 * kSpanRows * 128 + 2 * kTileTokens * 128 + 2 * kSpanRows * kPsStride + sizeof(SpanMeta);

}  // namespace

// ---- forward launcher ----
size_t fwd_span_workspace_bytes(const TreeParams& t, int B, int H) {
    return (size_t)B * H * (t.n / kTileTokens) * outer_levels(t) * kExtStride * sizeof(float);
}

bpt_status launch_fwd_span(const AttnProblem& p) {
    const TreeParams& t = p.tree;
    const int tiles = t.n / kTileTokens, n_ext = outer_levels(t);
    if (p.H > 65535 || p.B > 65535) return BPT_ERR_UNSUPPORTED;
    float* ext = (float*)p.workspace;
    fwd_span_kernel<<<dim3(tiles, p.H, p.B), kSpanThreads, 0, p.stream>>>(
        t, (const __nv_bfloat16*)p.q, (const __nv_bfloat16*)p.k, (const __nv_bfloat16*)p.v, (const __nv_bfloat16*)p.rel_emb,
        (__nv_bfloat16*)p.out, p.lse, ext, p.H, n_ext, p.scale * kLog2e, p.lengths, p.drop);
    trace_mark(p.stream, "fwd_span");
    if (n_ext > 0) {
        const int64_t warps = (int64_t)p.B * p.H * (tiles - 1);
        fwd_span_merge_kernel<<<(unsigned)((warps + 3) / 4), 128, 0, p.stream>>>(
            t, ext, (__nv_bfloat16*)p.out, p.lse, p.H, p.B * p.H, tiles, n_ext);
        trace_mark(p.stream, "fwd_span_merge");
    }
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

// ---- backward launcher (one pass over pairs [pair0, pair0 + n_pairs)) ----
size_t bwd_span_ext_floats(const TreeParams& t, int n_pairs) {
    return (size_t)n_pairs * (t.n / kTileTokens) * outer_levels(t) * 64;
}
size_t bwd_span_slab_floats(const TreeParams& t, int n_pairs) { return (size_t)n_pairs * t.n * 128; }

bpt_status launch_bwd_span(const AttnProblem& p, int pair0, int n_pairs, float* ext_dq, float* aff_slab) {
    const TreeParams& t = p.tree;
    const int tiles = t.n / kTileTokens, n_ext = outer_levels(t);
    if (cudaFuncSetAttribute(bwd_span_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBwdSpanSmem) != cudaSuccess)
        return BPT_ERR_CUDA;
    bwd_span_kernel<<<dim3(tiles, n_pairs), kSpanThreads, kBwdSpanSmem, p.stream>>>(
        t, (const __nv_bfloat16*)p.q, (const __nv_bfloat16*)p.k, (const __nv_bfloat16*)p.v, (const __nv_bfloat16*)p.rel_emb,
        (const __nv_bfloat16*)p.out, p.lse, (const __nv_bfloat16*)p.d_out, (__nv_bfloat16*)p.dq, ext_dq, aff_slab,
        p.H, pair0, n_ext, p.scale, p.lengths, p.drop);
    trace_mark(p.stream, "bwd_span");
    if (n_ext > 0) {
        const int64_t warps = (int64_t)n_pairs * (tiles - 1);
        bwd_span_merge_kernel<<<(unsigned)((warps + 3) / 4), 128, 0, p.stream>>>(
            t, ext_dq, (__nv_bfloat16*)p.dq, p.H, pair0, n_pairs, tiles, n_ext, p.scale);
        trace_mark(p.stream, "bwd_span_merge");
    }
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

}  // namespace bpt
