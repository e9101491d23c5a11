// Tiled backward for the token rows (arXiv 1911.04070: gradient of the Sec. 3.4 equation over
// the contextual edges of Sec. 3.2.2), bf16, head size 64.
//
// One CTA = 64 consecutive tokens of one (batch entry, head), 4 warps (16 query rows each); the buffers
// are sized so that two CTAs share an SM (see BwdTileCfg).  As in the tiled forward
// the nodes a token attends at one (side, level) are one contiguous range, so per chunk the CTA
// stages the union range of K and V rows once.  The token's self loop is folded into the
// level-0 left chunk: node i follows its left neighbours directly, and the relation ids
// self = 0, left(0, o) = 1 + o are consecutive, so the self loop is simply offset 0 of a range
// that ends at the token itself.
//
//   phase 1 (16 query rows per warp):  S = Q K^T + skewed Q R^T,  P = exp(S - lse),
//            dP = dO V^T,  dS = P (dP - dO.O);  dQ += dS K + skew(dS) R;
//            P, dS and the skewed dS (indexed by relation offset) go to shared memory as bf16
//   phase 2 (a warp owns 16 staged key rows):  dK_part = dS^T Q,  dV_part = P^T dO for the
//            chunk's node range and dR_part = skew(dS)^T Q, written to the workspace.
//
// Nothing is accumulated across CTAs here: bwd_gather_kernel sums, for every source node, the
// partial rows of the tiles whose range covers it, in tile order (no atomics, fixed order), and
// drel_sum kernels do the same for the relation table.
#include "bounds_check.cuh"
#include "bpt_internal.cuh"
#include "mma_tools.cuh"
#include "row_map.cuh"
#include "tile_geom.cuh"

namespace bpt {

size_t bwd_span_ext_floats(const TreeParams& t, int n_pairs);
size_t bwd_span_slab_floats(const TreeParams& t, int n_pairs);
bpt_status launch_bwd_span(const AttnProblem& p, int pair0, int n_pairs, float* ext_dq, float* aff_slab);

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kMaxKvRows = 208;   // staged K / V rows per chunk at k = 64
constexpr int kMaxRelRows = 80;   // staged relation rows per chunk (k + 2 <= 66, padded to 16)
constexpr int kMaxChunks = 2 * kMaxLevels;
constexpr int kDrelGroups = 32;   // first stage of the d_rel sum

struct ChunkPlan {
    int n_left, n_right;
    int slab_row0[kMaxChunks + 1];  // first reserved partial row of each chunk; [chunks] = rows per tile
    int rel_rows;                   // relation offsets a chunk's products cover (multiple of 16)
    int rel_store;                  // rows kept per chunk in the d_rel partials: k + 2, the most a chunk uses
    int group;                      // consecutive 64-token tiles one CTA works through (their partial rows are merged)
};

// Shared-memory layout.  The buffer sizes follow k and are capped so that two CTAs fit an SM (two
// independent CTAs of four warps measured 10 to 30 % faster than one CTA of eight warps that share
// barriers); a chunk whose node range is wider than the K / V buffers is worked through in sub-blocks.
struct BwdTileCfg {
    int kv_rows;      // staged K / V rows (multiple of 16)
    int rel_rows;     // staged relation rows (multiple of 16)
    int qr_stride;    // floats per row of the Q R^T scratch
    int p_stride;     // bytes per token row of the P / dS tiles (an odd number of 16-byte chunks)
    int skew_stride;  // bytes per token row of the skewed dS tile (an odd number of 16-byte chunks)
    int g_off, k_off, v_off, r_off, qr_off, p_off, ds_off, sk_off, row_off, bnd_off;  // byte offsets (Q tile at 0)
    size_t bytes;
};

constexpr BwdTileCfg layout_of(int kv_rows, int rel_rows, int qr_stride) {
    BwdTileCfg c{};
    c.kv_rows = kv_rows;
    c.rel_rows = rel_rows;
    c.qr_stride = qr_stride;
    c.p_stride = kv_rows * 2 + 16;
    c.skew_stride = rel_rows * 2 + 16;
    c.g_off = kTileTokens * 128;
    c.k_off = c.g_off + kTileTokens * 128;
    c.v_off = c.k_off + kv_rows * 128;
    c.r_off = c.v_off + kv_rows * 128;
    c.qr_off = c.r_off + rel_rows * 128;
    c.p_off = c.qr_off + 4 * 16 * qr_stride * 4;
    c.ds_off = c.p_off + kTileTokens * c.p_stride;
    c.sk_off = c.ds_off + kTileTokens * c.p_stride;
    c.row_off = c.sk_off + kTileTokens * c.skew_stride;
    c.bnd_off = c.row_off + 2 * kTileTokens * 4;
    return c;
}
constexpr size_t kTwoCtaBytes = 112 * 1024;  // shared memory per CTA up to which two CTAs fit an SM

BwdTileCfg make_bwd_tile_cfg(const TreeParams& t, int chunks) {
    const size_t tail = (size_t)chunks * (kTileTokens * 8 + 8 + 5 * 4);  // row ranges, chunk range, group bookkeeping
    const int rel_rows = min(kMaxRelRows, (t.k + 2 + 15) & ~15);
    const int qr_stride = rel_rows - 4 >= t.k + 2 ? rel_rows - 4 : rel_rows + 4;
    int kv_rows = min(kMaxKvRows, (t.kc + 97) & ~15);  // 15 (alignment) + 64 + k + 3 columns at most, rounded up to 16
    while (kv_rows > 64 && layout_of(kv_rows, rel_rows, qr_stride).bnd_off + tail > kTwoCtaBytes) kv_rows -= 16;
    BwdTileCfg c = layout_of(kv_rows, rel_rows, qr_stride);
    c.bytes = (size_t)c.bnd_off + tail;
    return c;
}

struct ChunkGeom {
    int side, level, n_l, id_base, rel_base, n_rel_c, base, kend;
};

__device__ __forceinline__ ChunkGeom chunk_geom(const TreeParams& t, int n_left, int c, int2 cr) {
    ChunkGeom gm;
    gm.side = c >= n_left;
    gm.level = gm.side ? c - n_left : c;
    gm.n_l = t.n >> gm.level;
    gm.id_base = node_id(t.n, gm.level, 0);
    gm.rel_base = c == 0 ? 0 : (gm.side ? rel_right(t, gm.level, 0) : rel_left(t, gm.level, 0));
    gm.n_rel_c = c == 0 ? t.k + 2 : t.k + 1;  // chunk 0 also holds r^self
    gm.base = cr.x & ~15;
    gm.kend = cr.y - gm.base;
    return gm;
}

constexpr int kBwdThreads = 128;  // 4 warps, one per group of 16 query rows

__global__ void __launch_bounds__(kBwdThreads)
bwd_tile_kernel(TreeParams t, ChunkPlan plan, BwdTileCfg cfg,
                const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ r,
                const __nv_bfloat16* __restrict__ out, const float* __restrict__ lse,
                const __nv_bfloat16* __restrict__ d_out, __nv_bfloat16* __restrict__ dq,
                int2* __restrict__ tile_range, float* __restrict__ slabs, float* __restrict__ drel_part,
                int H, int pair0, float scale, const int32_t* __restrict__ lengths, DropoutParams drop) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* q_s = smem;
    unsigned char* g_s = smem + cfg.g_off;   // d_out tile
    unsigned char* k_s = smem + cfg.k_off;
    unsigned char* v_s = smem + cfg.v_off;
    unsigned char* r_s = smem + cfg.r_off;
    float* qr_s = reinterpret_cast<float*>(smem + cfg.qr_off);
    unsigned char* p_s = smem + cfg.p_off;
    unsigned char* ds_s = smem + cfg.ds_off;
    unsigned char* sk_s = smem + cfg.sk_off;
    float* lse_s = reinterpret_cast<float*>(smem + cfg.row_off);
    float* delta_s = lse_s + kTileTokens;
    int2* bnd = reinterpret_cast<int2*>(delta_s + kTileTokens);
    const int n_left = plan.n_left, n_right = plan.n_right, chunks = n_left + n_right;
    int2* crange = bnd + chunks * kTileTokens;
    // per chunk, over the tiles of the group done so far: first node of the merged partial rows, last node written,
    // whether the d_rel partial has been written; and the last two as they were before the current tile
    int* st_origin = reinterpret_cast<int*>(crange + chunks);
    int* st_hi = st_origin + chunks;
    int* st_rel = st_hi + chunks;
    int* st_old_hi = st_rel + chunks;
    int* st_rel_old = st_old_hi + chunks;

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int kQrStride = cfg.qr_stride, kPStride = cfg.p_stride, kSkewStride = cfg.skew_stride;
    const int rg = w;  // row group: this warp's 16 query rows
    const int g = lane >> 2, c2 = (lane & 3) * 2;
    const int st = blockIdx.x, n_st = gridDim.x;  // group of plan.group consecutive tiles, and how many groups
    const int pair = pair0 + blockIdx.y, b = pair / H, h = pair % H;
    const int N = 2 * t.n - 1;
    const size_t rs = (size_t)H * 64;
    const size_t boff = (size_t)b * N * rs + (size_t)h * 64;
    const uint32_t q_u = smem_u32(q_s), g_u = smem_u32(g_s), k_u = smem_u32(k_s), v_u = smem_u32(v_s),
                   r_u = smem_u32(r_s), p_u = smem_u32(p_s), ds_u = smem_u32(ds_s), sk_u = smem_u32(sk_s);
    const float scale_log2e = scale * kLog2e;
    float* slab_cta = slabs + ((size_t)blockIdx.y * n_st + st) * plan.slab_row0[chunks] * 128;
    float* drel_cta = drel_part + ((size_t)blockIdx.y * n_st + st) * chunks * plan.rel_store * 64;
    if (tid < chunks) { st_origin[tid] = 0; st_hi[tid] = -1; st_rel[tid] = 0; }

    // The tiles of the group one after the other.  A later tile adds its partial rows to those an earlier tile
    // of the same CTA already wrote (read back from L2, same thread order every run), so that the gather finds
    // one row per node and group instead of one per node and tile.
    for (int hidx = 0; hidx < plan.group; ++hidx) {
    const int tile = st * plan.group + hidx, t0 = tile * kTileTokens;

    // ---- prologue: Q and dO tiles, out tile (into the K buffer) for the row term, row ranges ----
    for (int idx = tid; idx < kTileTokens * 8; idx += kBwdThreads) {
        const int row = idx >> 3, ch = idx & 7;
        const size_t src = boff + (size_t)(t0 + row) * rs + ch * 8;
        cp_async16(q_u + tile_off(row, ch), q + src);
        cp_async16(g_u + tile_off(row, ch), d_out + src);
        cp_async16(k_u + tile_off(row, ch), out + src);
    }
    cp_async_commit();
    if (tid < kTileTokens) {
        fill_row_bounds(t, t0, tid, n_left, n_right, bnd);
        // the self loop joins the level-0 left range: it ends at the token itself
        const int i = t0 + tid;
        const int2 v0 = bnd[tid];
        bnd[tid] = v0.x > v0.y ? make_int2(i, i) : make_int2(v0.x, i);
        lse_s[tid] = lse[((size_t)b * N + i) * H + h] * kLog2e;
    }
    cp_async_wait<0>();
    __syncthreads();
    if (tid < 2 * kTileTokens) {   // delta_i = d_out_i . out_i: two threads per row
        const int row = tid >> 1, hf = tid & 1;
        float acc = 0.f;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            const uint4 a = *reinterpret_cast<const uint4*>(g_s + tile_off(row, hf * 4 + ch));
            const uint4 o = *reinterpret_cast<const uint4*>(k_s + tile_off(row, hf * 4 + ch));
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, ow[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                acc = fmaf(__uint_as_float(aw[x] << 16), __uint_as_float(ow[x] << 16), acc);
                acc = fmaf(__uint_as_float(aw[x] & 0xffff0000u), __uint_as_float(ow[x] & 0xffff0000u), acc);
            }
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        if (hf == 0) delta_s[row] = acc;
    }
    for (int c = w; c < chunks; c += kBwdThreads / 32) {
        const int2 a = rows_union(bnd + c * kTileTokens, 0, 32, lane);
        const int2 bb = rows_union(bnd + c * kTileTokens, 32, 32, lane);
        if (lane == 0) {
            const int2 u = make_int2(min(a.x, bb.x), max(a.y, bb.y));
            crange[c] = u;
        }
    }

    const int r0 = rg * 16;
    uint32_t qa[4][4], ga[4][4];
    load_a_frags(q_u, r0, lane, qa);
    load_a_frags(g_u, r0, lane, ga);
    float acc_q[8][4];
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) { acc_q[nt][0] = acc_q[nt][1] = acc_q[nt][2] = acc_q[nt][3] = 0.f; }

    float* qr_w = qr_s + rg * 16 * kQrStride;

    // A chunk whose node range is wider than the K / V buffers is worked through in sub-blocks of
    // cfg.kv_rows columns; (c, s0) = chunk and first column of the sub-block.  Its length:
    auto sub_len = [&](const ChunkGeom& gm, int s0) { return min(cfg.kv_rows, (gm.kend + 1 - s0 + 15) & ~15); };
    // K / V rows of the sub-block and, with its first sub-block, the chunk's relation rows -> shared memory (async)
    auto stage = [&](int c, int s0) {
        const ChunkGeom gm = chunk_geom(t, n_left, c, crange[c]);
        const int nr = sub_len(gm, s0);
        for (int idx = tid; idx < nr * 8; idx += kBwdThreads) {
            const int row = idx >> 3, ch = idx & 7;
            const int node = min(gm.base + s0 + row, gm.n_l - 1);  // rows past the range repeat a real row: finite values
            const size_t src = boff + (size_t)(gm.id_base + node) * rs + ch * 8;
            if (!BPT_IDX_OK(gm.id_base + node, N, BPT_SITE_NODE)) continue;
            cp_async16(k_u + tile_off(row, ch), k + src);
            cp_async16(v_u + tile_off(row, ch), v + src);
        }
        if (s0 == 0) {
            for (int idx = tid; idx < cfg.rel_rows * 8; idx += kBwdThreads) {
                const int row = idx >> 3, ch = idx & 7;
                if (row < gm.n_rel_c && BPT_IDX_OK(gm.rel_base + row, 1 + 2 * t.L * (t.k + 1) + t.L, BPT_SITE_RELATION))
                    cp_async16(r_u + tile_off(row, ch), r + (size_t)(gm.rel_base + row) * 64 + ch * 8);
                else *reinterpret_cast<uint4*>(r_s + tile_off(row, ch)) = make_uint4(0, 0, 0, 0);
            }
        }
    };

    const int len = seq_len(lengths, b, t.n);
    if (len < t.n) {  // short sequence: staged ranges and partial-row layout stay those of the full graph, the rows' ranges shrink
        __syncthreads();
        if (tid < kTileTokens) mask_row_bounds(t, t0, tid, n_left, n_right, bnd, len);
    }
    __syncthreads();  // delta and crange are visible; the out tile in the K buffer is consumed
    if (tid < chunks) {  // group bookkeeping (first read in phase 2, several barriers from here)
        const int2 u = crange[tid];
        st_old_hi[tid] = st_hi[tid];
        st_rel_old[tid] = st_rel[tid];
        if (u.x <= u.y) {
            if (st_hi[tid] < 0) st_origin[tid] = u.x;
            st_hi[tid] = u.y;
            st_rel[tid] = 1;
        }
    }
    stage(0, 0);      // chunk 0 (left level 0 with the self loop) is never empty
    cp_async_commit();

    int c = 0, s0 = 0;
    while (c < chunks) {
        const int2 cr = crange[c];
        const ChunkGeom gm = chunk_geom(t, n_left, c, cr);
        const int side = gm.side, n_rel_c = gm.n_rel_c;
        const int sb_len = sub_len(gm, s0);                      // columns of this sub-block (a multiple of 16)
        const bool first = s0 == 0, last = s0 + sb_len > gm.kend;  // first / last sub-block of the chunk
        const int base = gm.base + s0;                           // node index of the sub-block's column 0
        if (first)
            for (int idx = tid; idx < kTileTokens * (kSkewStride / 16); idx += kBwdThreads)
                *reinterpret_cast<uint4*>(sk_s + idx * 16) = make_uint4(0, 0, 0, 0);
        cp_async_wait<0>();
        __syncthreads();

        // ================= phase 1: 16 query rows per pair of warps, key blocks alternate =================
        const int2* bc = bnd + c * kTileTokens;
        const int2 wr = rows_union(bc, r0, 16, lane);
        const bool w_any = wr.x <= wr.y;
        if (w_any && first) {  // Q R^T for the chunk's relation rows -> the row group's scratch (kept for all sub-blocks)
#pragma unroll
            for (int np = 0; np < kMaxRelRows / 16; ++np) {
                if (np * 16 < n_rel_c) {
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
        }
        __syncwarp();

        const int2 ba = bc[r0 + g], bb = bc[r0 + g + 8];
        const int lo_r[2] = {ba.x, bb.x}, hi_r[2] = {ba.y, bb.y};
        const float lse_r[2] = {lse_s[r0 + g], lse_s[r0 + g + 8]};
        const float del_r[2] = {delta_s[r0 + g], delta_s[r0 + g + 8]};
        const int w_lo = w_any ? wr.x - base : 1 << 30, w_hi = w_any ? wr.y - base : -1;
        // 16 keys at a time: S, dP, the element-wise part, P / dS / skew to shared memory, dQ += dS K.  (16-key
        // granularity skips more of the masked columns than 32 would: measured 0.77 against 0.83 ms at k = 8.)
        constexpr int NG = 1;
        auto keys = [&](int kb) {
            unsigned char* p_row0 = p_s + (r0 + g) * kPStride + (kb + c2) * 2;
            unsigned char* d_row0 = ds_s + (r0 + g) * kPStride + (kb + c2) * 2;
            if (kb + 16 * NG - 1 < w_lo || kb > w_hi) {  // nothing of these rows here: zeros for phase 2
#pragma unroll
                for (int j = 0; j < 2 * NG; ++j) {
                    *reinterpret_cast<uint32_t*>(p_row0 + j * 16) = 0u;
                    *reinterpret_cast<uint32_t*>(p_row0 + 8 * kPStride + j * 16) = 0u;
                    *reinterpret_cast<uint32_t*>(d_row0 + j * 16) = 0u;
                    *reinterpret_cast<uint32_t*>(d_row0 + 8 * kPStride + j * 16) = 0u;
                }
                return;
            }
            float s[2 * NG][4], dp[2 * NG][4];
#pragma unroll
            for (int j = 0; j < 2 * NG; ++j) {
                s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
                dp[j][0] = dp[j][1] = dp[j][2] = dp[j][3] = 0.f;
            }
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
                for (int np = 0; np < NG; ++np) {
                    uint32_t bf[4];
                    load_b_rows(k_u, kb + np * 16, ks, lane, bf);
                    mma_bf16(s[np * 2], qa[ks], bf[0], bf[1]);
                    mma_bf16(s[np * 2 + 1], qa[ks], bf[2], bf[3]);
                    load_b_rows(v_u, kb + np * 16, ks, lane, bf);
                    mma_bf16(dp[np * 2], ga[ks], bf[0], bf[1]);
                    mma_bf16(dp[np * 2 + 1], ga[ks], bf[2], bf[3]);
                }
            }
            uint32_t da[NG][4];
#pragma unroll
            for (int j = 0; j < 2 * NG; ++j) {
                float pv[4], dv[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int hh = e >> 1;
                    const int m = base + kb + j * 8 + c2 + (e & 1);
                    const bool ok = m >= lo_r[hh] && m <= hi_r[hh];
                    float p = 0.f, d = 0.f;
                    if (ok) {
                        const int off = side ? m - lo_r[hh] : hi_r[hh] - m;
                        const float bias = qr_w[(g + hh * 8) * kQrStride + off];
                        p = fast_exp2(fmaf(s[j][e] + bias, scale_log2e, -lse_r[hh]));
                        // dropout: dP = W d_out.v and the weight that reaches dv is W P; dS keeps the undropped P
                        const float wgt = drop.thr ? dropout_weight(drop, (uint32_t)pair, (uint32_t)(t0 + r0 + g + hh * 8), (uint32_t)(gm.id_base + m)) : 1.f;
                        d = p * (dp[j][e] * wgt - del_r[hh]);
                        p *= wgt;
                        *reinterpret_cast<__nv_bfloat16*>(sk_s + (r0 + g + hh * 8) * kSkewStride + off * 2) = __float2bfloat16_rn(d);
                    }
                    pv[e] = p; dv[e] = d;
                }
                const uint32_t p01 = pack_bf16(pv[0], pv[1]), p23 = pack_bf16(pv[2], pv[3]);
                const uint32_t d01 = pack_bf16(dv[0], dv[1]), d23 = pack_bf16(dv[2], dv[3]);
                *reinterpret_cast<uint32_t*>(p_row0 + j * 16) = p01;
                *reinterpret_cast<uint32_t*>(p_row0 + 8 * kPStride + j * 16) = p23;
                *reinterpret_cast<uint32_t*>(d_row0 + j * 16) = d01;
                *reinterpret_cast<uint32_t*>(d_row0 + 8 * kPStride + j * 16) = d23;
                da[j >> 1][(j & 1) * 2] = d01;
                da[j >> 1][(j & 1) * 2 + 1] = d23;
            }
            // dQ += dS K over these keys
#pragma unroll
            for (int kk = 0; kk < NG; ++kk) {
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    uint32_t bf[4];
                    load_b_cols(k_u, kb + kk * 16, np, lane, bf);
                    mma_bf16(acc_q[np * 2], da[kk], bf[0], bf[1]);
                    mma_bf16(acc_q[np * 2 + 1], da[kk], bf[2], bf[3]);
                }
            }
        };
        for (int kb0 = 0; kb0 < sb_len; kb0 += 32) {
            keys(kb0);
            if (kb0 + 16 < sb_len) keys(kb0 + 16);
        }
        __syncwarp();  // this warp's rows of the skew tile are complete
        if (w_any && last) {  // dQ += skew(dS) R_chunk once the chunk's skew tile is complete, the k-steps shared out between the two warps
#pragma unroll
            for (int kk = 0; kk < kMaxRelRows / 16; ++kk) {
                if (kk * 16 < n_rel_c) {
                    uint32_t a[4];
                    load_a_plain(sk_u, kSkewStride, r0, kk * 16, lane, a);
#pragma unroll
                    for (int np = 0; np < 4; ++np) {
                        uint32_t bf[4];
                        load_b_cols(r_u, kk * 16, np, lane, bf);
                        mma_bf16(acc_q[np * 2], a, bf[0], bf[1]);
                        mma_bf16(acc_q[np * 2 + 1], a, bf[2], bf[3]);
                    }
                }
            }
        }
        __syncthreads();  // P, dS and the skew tile are complete; K, V and R tiles are free

        // next sub-block, or the next chunk that this tile reaches: its rows arrive while phase 2 runs
        int cn = c, sn = s0 + sb_len;
        if (last) {
            cn = c + 1;
            sn = 0;
            while (cn < chunks && crange[cn].x > crange[cn].y) ++cn;  // a level no token of the tile reaches
        }
        if (cn < chunks) stage(cn, sn);
        cp_async_commit();

        // ================= phase 2: key tiles (dk, dv partial rows) and offset tiles (d_rel partial) =================
        // jobs: (key tile | offset tile) x (channels 0..31 | 32..63); key-tile jobs are twice as heavy, so they go first
        const int n_jt = sb_len >> 4, n_ot = last ? plan.rel_rows >> 4 : 0;  // the d_rel tiles once per chunk
        for (int job = w; job < 2 * (n_jt + n_ot); job += kBwdThreads / 32) {
            const int hc = job & 1, tile16 = job >> 1;  // channel half, tile
            if (tile16 < n_jt) {
                const int jt = tile16;
                // the accumulators start from what an earlier tile of the group left in the partial rows (the loads
                // fly while the products below run), from zero otherwise
                float ak[4][4], av[4][4];
                float* dst_row[2];
                bool row_ok[2];
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int m = base + jt * 16 + g + hh * 8;
                    row_ok[hh] = m >= cr.x && m <= cr.y;
                    dst_row[hh] = slab_cta + (size_t)(plan.slab_row0[c] + m - st_origin[c]) * 128 + hc * 32 + c2;
                    const bool add = row_ok[hh] && m <= st_old_hi[c];
#pragma unroll
                    for (int nt = 0; nt < 4; ++nt) {
                        float2 xk = make_float2(0.f, 0.f), xv = xk;
                        if (add) {
                            xk = *reinterpret_cast<const float2*>(dst_row[hh] + nt * 8);
                            xv = *reinterpret_cast<const float2*>(dst_row[hh] + 64 + nt * 8);
                        }
                        ak[nt][hh * 2] = xk.x; ak[nt][hh * 2 + 1] = xk.y;
                        av[nt][hh * 2] = xv.x; av[nt][hh * 2 + 1] = xv.y;
                    }
                }
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    uint32_t a_ds[4], a_p[4];
                    load_a_trans(ds_u, kPStride, ks * 16, jt * 16, lane, a_ds);
                    load_a_trans(p_u, kPStride, ks * 16, jt * 16, lane, a_p);
#pragma unroll
                    for (int np = 0; np < 2; ++np) {
                        uint32_t bf[4];
                        load_b_cols(q_u, ks * 16, hc * 2 + np, lane, bf);
                        mma_bf16(ak[np * 2], a_ds, bf[0], bf[1]);
                        mma_bf16(ak[np * 2 + 1], a_ds, bf[2], bf[3]);
                        load_b_cols(g_u, ks * 16, hc * 2 + np, lane, bf);
                        mma_bf16(av[np * 2], a_p, bf[0], bf[1]);
                        mma_bf16(av[np * 2 + 1], a_p, bf[2], bf[3]);
                    }
                }
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    if (row_ok[hh]) {
#pragma unroll
                        for (int nt = 0; nt < 4; ++nt) {
                            *reinterpret_cast<float2*>(dst_row[hh] + nt * 8) = make_float2(ak[nt][hh * 2], ak[nt][hh * 2 + 1]);
                            *reinterpret_cast<float2*>(dst_row[hh] + 64 + nt * 8) = make_float2(av[nt][hh * 2], av[nt][hh * 2 + 1]);
                        }
                    }
                }
            } else {
                const int ot = tile16 - n_jt;
                float ar[4][4];
                const bool add = st_rel_old[c] != 0;  // an earlier tile of the group wrote this chunk's partial: start from it
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int o = ot * 16 + g + hh * 8;
                    const float* src = drel_cta + ((size_t)c * plan.rel_store + o) * 64 + hc * 32 + c2;
#pragma unroll
                    for (int nt = 0; nt < 4; ++nt) {
                        float2 x = make_float2(0.f, 0.f);
                        if (add && o < plan.rel_store) x = *reinterpret_cast<const float2*>(src + nt * 8);
                        ar[nt][hh * 2] = x.x; ar[nt][hh * 2 + 1] = x.y;
                    }
                }
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    uint32_t a[4];
                    load_a_trans(sk_u, kSkewStride, ks * 16, ot * 16, lane, a);
#pragma unroll
                    for (int np = 0; np < 2; ++np) {
                        uint32_t bf[4];
                        load_b_cols(q_u, ks * 16, hc * 2 + np, lane, bf);
                        mma_bf16(ar[np * 2], a, bf[0], bf[1]);
                        mma_bf16(ar[np * 2 + 1], a, bf[2], bf[3]);
                    }
                }
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int o = ot * 16 + g + hh * 8;
                    if (o < plan.rel_store) {
                        float* dst = drel_cta + ((size_t)c * plan.rel_store + o) * 64 + hc * 32 + c2;
#pragma unroll
                        for (int nt = 0; nt < 4; ++nt)
                            *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(ar[nt][hh * 2], ar[nt][hh * 2 + 1]);
                    }
                }
            }
        }
        __syncthreads();  // P, dS and skew tiles are free again
        c = cn;
        s0 = sn;
    }

    // ---- epilogue: dq = scale * acc, rounded once to bf16, coalesced stores through the Q tile ----
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        *reinterpret_cast<uint32_t*>(q_s + tile_off(r0 + g, nt) + c2 * 2) = pack_bf16(acc_q[nt][0] * scale, acc_q[nt][1] * scale);
        *reinterpret_cast<uint32_t*>(q_s + tile_off(r0 + g + 8, nt) + c2 * 2) = pack_bf16(acc_q[nt][2] * scale, acc_q[nt][3] * scale);
    }
    __syncwarp();
    for (int idx = lane; idx < 16 * 8; idx += 32) {
        const int row = r0 + (idx >> 3), ch = idx & 7;
        *reinterpret_cast<uint4*>(dq + boff + (size_t)(t0 + row) * rs + ch * 8) =
            *reinterpret_cast<const uint4*>(q_s + tile_off(row, ch));
    }
    __syncthreads();  // the Q tile is free for the next tile of the group
    }  // tiles of the group

    // chunks no tile of the group reached: zero d_rel partial; the group's ranges for the gather
    for (int c = 0; c < chunks; ++c) {
        if (st_rel[c]) continue;
        float4* z = reinterpret_cast<float4*>(drel_cta + (size_t)c * plan.rel_store * 64);
        for (int idx = tid; idx < plan.rel_store * 16; idx += kBwdThreads) z[idx] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (blockIdx.y == 0 && pair0 == 0 && tid < chunks) {
        // empty ranges keep the table monotone over the groups: left levels are missing for a prefix of the
        // groups, right levels for a suffix
        const int n_l = t.n >> (tid >= n_left ? tid - n_left : tid);
        tile_range[(size_t)tid * n_st + st] = st_hi[tid] >= 0 ? make_int2(st_origin[tid], st_hi[tid])
                                                              : (tid >= n_left ? make_int2(n_l, n_l - 1) : make_int2(0, -1));
    }
}

// For every node and side the groups of tiles [first, last) whose chunk range covers the node: the same for every
// (batch entry, head) pair, so it is found once per call (two bisections over the monotone table of group ranges)
// and the gather reads it.
__global__ void gather_plan_kernel(TreeParams t, ChunkPlan plan, const int2* __restrict__ tile_range, int tiles,
                                   int2* __restrict__ node_tiles) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    const int N = 2 * t.n - 1;
    if (idx >= 2 * N) return;
    const int vtx = idx >> 1, side = idx & 1;
    const int l = node_level(t.n, vtx), m = vtx - node_id(t.n, l, 0);
    int2 r = make_int2(0, 0);
    if (l < (side ? plan.n_right : plan.n_left)) {
        const int c = side ? plan.n_left + l : l;
        const int2* tr = tile_range + (size_t)c * tiles;
        int lo = 0, hi = tiles;  // first group whose range ends at or beyond m
        while (lo < hi) { const int mid = (lo + hi) >> 1; if (tr[mid].y >= m) hi = mid; else lo = mid + 1; }
        r.x = lo;
        hi = tiles;              // first group whose range starts beyond m
        while (lo < hi) { const int mid = (lo + hi) >> 1; if (tr[mid].x > m) hi = mid; else lo = mid + 1; }
        r.y = lo;
    }
    node_tiles[idx] = r;
}

// dk, dv of every node: the partial rows of the tiles whose chunk range covers the node (both
// sides), in tile order, plus for a token the row the span pass left for it (the affiliated
// edges into its L ancestors).  One warp per (pair, node); lanes 0..15 hold four channels of dk
// each, lanes 16..31 four channels of dv.
__global__ void __launch_bounds__(256)
bwd_gather_kernel(TreeParams t, ChunkPlan plan, const int2* __restrict__ tile_range, const int2* __restrict__ node_tiles,
                  const float* __restrict__ slabs, const float* __restrict__ aff_slab,
                  __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                  int H, int pair0, int n_pairs, int tiles, float scale) {
    const int lane = threadIdx.x & 31;
    const int N = 2 * t.n - 1;
    const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= (int64_t)n_pairs * N) return;
    const int pl = (int)(wid / N);              // pair inside this pass
    const int vtx = N - 1 - (int)(wid % N);     // coarse nodes (many tiles each) first
    const int pair = pair0 + pl, b = pair / H, h = pair % H;
    const int l = node_level(t.n, vtx), m = vtx - node_id(t.n, l, 0);
    const int chunks = plan.n_left + plan.n_right;
    const size_t tile_rows = (size_t)plan.slab_row0[chunks];
    const float* slab_pair = slabs + (size_t)pl * tiles * tile_rows * 128;

    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const int4 nt = __ldg(reinterpret_cast<const int4*>(node_tiles) + vtx);  // (first, last) group of the left side, of the right side
#pragma unroll
    for (int side = 0; side < 2; ++side) {
        const int ta = side ? nt.z : nt.x, tb = side ? nt.w : nt.y;
        if (ta >= tb) continue;
        const int c = side ? plan.n_left + l : l;
        const int2* tr = tile_range + (size_t)c * tiles;
        for (int T = ta; T < tb; ++T) {
            const int row = plan.slab_row0[c] + m - tr[T].x;
            const float4 x = __ldg(reinterpret_cast<const float4*>(slab_pair + ((size_t)T * tile_rows + row) * 128) + lane);
            acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
        }
    }
    const size_t rs = (size_t)H * 64;
    const size_t boff = (size_t)b * N * rs + (size_t)h * 64;
    const int ch4 = (lane & 15) * 4;
    if (l == 0) {
        const float4 x = __ldg(reinterpret_cast<const float4*>(aff_slab + ((size_t)pl * t.n + m) * 128) + lane);
        acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
    }
    const float f = lane < 16 ? scale : 1.f;
    __nv_bfloat16* dst = (lane < 16 ? dk : dv) + boff + (size_t)vtx * rs + ch4;
    *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16(acc.x * f, acc.y * f), pack_bf16(acc.z * f, acc.w * f));
}

// d_rel, first stage: the CTAs of one pass in kDrelGroups groups, each summed in CTA order.
// x indexes (chunk, offset, channel) of the per-CTA partial tables.
__global__ void drel_group_kernel(const float* __restrict__ part, float* __restrict__ grp, int n_ctas, size_t per_cta) {
    const size_t x = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= per_cta) return;
    const int gi = blockIdx.y;
    const int per = (n_ctas + kDrelGroups - 1) / kDrelGroups;
    const int c0 = min(gi * per, n_ctas), c1 = min(c0 + per, n_ctas);
    float acc = 0.f;
    for (int c = c0; c < c1; ++c) acc += part[(size_t)c * per_cta + x];
    grp[(size_t)gi * per_cta + x] = acc;
}

// d_rel, second stage: one thread per (relation row, channel).  Rows that no chunk covers (and
// the ancestor rows) are zero.  With `accumulate` the pass adds to what earlier passes wrote.
__global__ void drel_final_kernel(TreeParams t, ChunkPlan plan, const float* __restrict__ grp, float* __restrict__ d_rel,
                                  int n_rel, size_t per_cta, float scale, int accumulate) {
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= n_rel * 64) return;
    const int rid = x >> 6, ch = x & 63;
    const int W = t.k + 1;
    int c = -1, off = 0;
    if (rid <= W) { c = 0; off = rid; }               // self and left level 0 live in chunk 0
    else if (rid < 1 + t.L * W) { const int j = (rid - 1) / W; if (j < plan.n_left) { c = j; off = (rid - 1) % W; } }
    else if (rid < 1 + 2 * t.L * W) { const int j = (rid - 1 - t.L * W) / W; if (j < plan.n_right) { c = plan.n_left + j; off = (rid - 1 - t.L * W) % W; } }
    float acc = 0.f;
    if (c >= 0) {
        const size_t at = ((size_t)c * plan.rel_store + off) * 64 + ch;
        for (int gi = 0; gi < kDrelGroups; ++gi) acc += grp[(size_t)gi * per_cta + at];
    }
    d_rel[x] = accumulate ? d_rel[x] + acc * scale : acc * scale;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct TileWorkspace {
    int2* tile_range;
    int2* node_tiles;   // per node and side the groups whose range covers it
    float *aff_slab, *ext_dq, *slabs, *drel_part, *drel_grp;
    int pairs_per_pass;
    size_t bytes;
};

// Partial rows the size query plans per pass over the (batch entry, head) pairs.  A caller that brings a
// smaller workspace gets more passes: the launcher fits as many pairs as the given bytes hold.
constexpr size_t kPassBytes = (size_t)10 << 30;

ChunkPlan make_plan(const TreeParams& t) {
    ChunkPlan p{};
    context_levels(t, &p.n_left, &p.n_right);
    p.group = t.n >= 2 * kTileTokens ? 2 : 1;
    const int span = p.group * kTileTokens;  // tokens whose partial rows are merged
    int at = 0;
    for (int c = 0; c < p.n_left + p.n_right; ++c) {
        const int level = c >= p.n_left ? c - p.n_left : c;
        p.slab_row0[c] = at;
        at += (span >> level) + t.kc + 3;  // upper bound of the group's union range at this level
    }
    p.slab_row0[p.n_left + p.n_right] = at;
    p.rel_rows = (t.k + 2 + 15) & ~15;
    p.rel_store = t.k + 2;
    return p;
}

// Carves the workspace for `pairs` (batch entry, head) pairs per pass.
TileWorkspace carve_tile(const TreeParams& t, const ChunkPlan& plan, size_t pairs, void* base) {
    const int chunks = plan.n_left + plan.n_right, tiles = t.n / (kTileTokens * plan.group);  // groups of tiles
    TileWorkspace w;
    w.pairs_per_pass = (int)pairs;
    char* c = (char*)base;
    size_t off = 0;
    w.tile_range = (int2*)(c + off); off += align256(sizeof(int2) * chunks * tiles);
    w.node_tiles = (int2*)(c + off); off += align256(sizeof(int2) * 2 * (size_t)(2 * t.n - 1));
    w.aff_slab = (float*)(c + off); off += align256(sizeof(float) * bwd_span_slab_floats(t, (int)pairs));
    w.ext_dq = (float*)(c + off); off += align256(sizeof(float) * bwd_span_ext_floats(t, (int)pairs));
    w.slabs = (float*)(c + off); off += align256(sizeof(float) * pairs * tiles * plan.slab_row0[chunks] * 128);
    w.drel_part = (float*)(c + off); off += align256(sizeof(float) * pairs * tiles * chunks * plan.rel_store * 64);
    w.drel_grp = (float*)(c + off); off += align256(sizeof(float) * kDrelGroups * chunks * plan.rel_store * 64);
    w.bytes = off;
    return w;
}

// Pairs per pass: as many as `budget` bytes hold (at least one, at most all).
size_t pairs_for_budget(const TreeParams& t, const ChunkPlan& plan, int B, int H, size_t budget) {
    const size_t all = (size_t)B * H;
    const size_t fixed = carve_tile(t, plan, 0, nullptr).bytes;
    const size_t per_pair = carve_tile(t, plan, 1, nullptr).bytes - fixed;  // an upper bound: it includes the rounding of one pair
    size_t pairs = budget > fixed ? (budget - fixed) / per_pair : 0;
    if (pairs > all) pairs = all;
    while (pairs < all && carve_tile(t, plan, pairs + 1, nullptr).bytes <= budget) ++pairs;
    return pairs < 1 ? 1 : pairs;
}

}  // namespace

// ---- tensor-memory path (attn_bwd_q_tc5.cu, attn_bwd_kv_tc5.cu): no partial rows; its workspace holds the row
// terms of all pairs and, per pass, the span pass's blocks and the d_rel partials ----
bool bwd_q_tc5_fits(const TreeParams& t);
bpt_status launch_bwd_q_tc5(const AttnProblem& p, float* delta, int2* ranges);
size_t bwd_kv_tc5_drel_floats(const TreeParams& t, int n_pairs);
int bwd_kv_tc5_tiles(const TreeParams& t);
bpt_status launch_bwd_kv_tc5(const AttnProblem& p, int pair0, int n_pairs, const float* delta, const int2* ranges, int2* plan,
                             const float* aff_slab, float* drel_part);

namespace {

struct Tc5Workspace {
    float *delta, *aff_slab, *ext_dq, *drel_part;
    int2 *ranges, *plan;   // per token and chunk the node range; per key tile and side the query blocks
    int pairs_per_pass;
    size_t bytes;
};

Tc5Workspace carve_tc5(const TreeParams& t, int B, int H, size_t pairs, void* base) {
    Tc5Workspace w;
    w.pairs_per_pass = (int)pairs;
    char* c = (char*)base;
    size_t off = 0;
    w.delta = (float*)(c + off); off += align256(sizeof(float) * (size_t)B * H * t.n);
    int n_left, n_right;
    context_levels(t, &n_left, &n_right);
    w.ranges = (int2*)(c + off); off += align256(sizeof(int2) * (size_t)(n_left + n_right) * t.n);
    w.plan = (int2*)(c + off); off += align256(sizeof(int2) * (size_t)bwd_kv_tc5_tiles(t) * 2);
    w.aff_slab = (float*)(c + off); off += align256(sizeof(float) * bwd_span_slab_floats(t, (int)pairs));
    w.ext_dq = (float*)(c + off); off += align256(sizeof(float) * bwd_span_ext_floats(t, (int)pairs));
    w.drel_part = (float*)(c + off); off += align256(sizeof(float) * bwd_kv_tc5_drel_floats(t, (int)pairs));
    w.bytes = off;
    return w;
}

size_t tc5_pairs_for_budget(const TreeParams& t, int B, int H, size_t budget) {
    const size_t all = (size_t)B * H;
    const size_t fixed = carve_tc5(t, B, H, 0, nullptr).bytes, per_pair = carve_tc5(t, B, H, 1, nullptr).bytes - fixed;
    size_t pairs = budget > fixed ? (budget - fixed) / per_pair : 0;
    if (pairs > all) pairs = all;
    while (pairs < all && carve_tc5(t, B, H, pairs + 1, nullptr).bytes <= budget) ++pairs;
    return pairs < 1 ? 1 : pairs;
}

// The tensor-memory kernels take whole tiles of 128 tokens and pay for their hand-offs where a level holds
// enough nodes per token; bpt_attn_options.path forces either family.
bool want_bwd_tc5(const TreeParams& t, uint32_t path) {
    if (path == BPT_PATH_MMA || !bwd_q_tc5_fits(t)) return false;
    // measured (ms, warp-level / tensor-memory): k = 48: n = 8192 left-only 1.40 / 1.36, n = 4096 2.17 / 1.97, n = 16384 2.78 / 2.42,
    // n = 1024 1.57 / 1.58; k = 40: n = 8192 left-only 1.31 / 1.36, n = 4096 2.00 / 1.97; k = 64: ahead at every n
    return path == BPT_PATH_TC5 || t.k >= 48;
}

bpt_status launch_bwd_tc5(const AttnProblem& p) {
    const TreeParams& t = p.tree;
    const Tc5Workspace ws = carve_tc5(t, p.B, p.H, tc5_pairs_for_budget(t, p.B, p.H, p.workspace_bytes), p.workspace);
    if (ws.bytes > p.workspace_bytes) return BPT_ERR_WORKSPACE;
    bpt_status s = launch_bwd_q_tc5(p, ws.delta, ws.ranges);  // token dq, the row terms of every pair, the table of ranges
    const int total = p.B * p.H;
    for (int pair0 = 0; pair0 < total && s == BPT_OK; pair0 += ws.pairs_per_pass) {
        const int np = min(ws.pairs_per_pass, total - pair0);
        s = launch_bwd_span(p, pair0, np, ws.ext_dq, ws.aff_slab);  // span dq; per token the affiliated edges' share of dk / dv
        if (s == BPT_OK) s = launch_bwd_kv_tc5(p, pair0, np, ws.delta, ws.ranges, ws.plan, ws.aff_slab, ws.drel_part);
    }
    return s;
}

}  // namespace

bool bwd_tile_eligible(const bpt_graph& g, int d, bpt_dtype dtype) {
    return tile_path(g.dims.n, g.dims.k, d, dtype == BPT_BF16);
}

// minimal: the smallest workspace the backward runs with (one pair per pass); otherwise the planned size.
// Either kernel family may be asked for through the options, so the sizes cover both.
size_t bwd_tile_workspace_bytes(const bpt_graph& g, int B, int H, bool minimal) {
    TreeParams t;
    tree_params_from_dims(g.dims, &t);
    const ChunkPlan plan = make_plan(t);
    const size_t pairs = minimal ? 1 : pairs_for_budget(t, plan, B, H, kPassBytes);
    size_t bytes = carve_tile(t, plan, pairs, nullptr).bytes;
    if (bwd_q_tc5_fits(t)) {
        const size_t tp = minimal ? 1 : tc5_pairs_for_budget(t, B, H, kPassBytes);
        bytes = max(bytes, carve_tc5(t, B, H, tp, nullptr).bytes);
    }
    return bytes;
}


bpt_status launch_bwd_tile(const AttnProblem& p) {
    const TreeParams& t = p.tree;
    if (want_bwd_tc5(t, p.path)) return launch_bwd_tc5(p);
    const ChunkPlan plan = make_plan(t);
    const int chunks = plan.n_left + plan.n_right, tiles = t.n / (kTileTokens * plan.group), N = 2 * t.n - 1;  // tiles: groups
    const TileWorkspace ws = carve_tile(t, plan, pairs_for_budget(t, plan, p.B, p.H, p.workspace_bytes), p.workspace);
    if (ws.bytes > p.workspace_bytes) return BPT_ERR_WORKSPACE;
    const BwdTileCfg cfg = make_bwd_tile_cfg(t, chunks);
    const size_t smem = cfg.bytes;
    if (smem > 227 * 1024) return BPT_ERR_UNSUPPORTED;
    auto kernel = bwd_tile_kernel;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return BPT_ERR_CUDA;

    const int total = p.B * p.H;
    const size_t per_cta = (size_t)chunks * plan.rel_store * 64;
    for (int pair0 = 0; pair0 < total; pair0 += ws.pairs_per_pass) {
        const int np = min(ws.pairs_per_pass, total - pair0);
        if (np > 65535) return BPT_ERR_UNSUPPORTED;
        // span rows: dq of the spans and, per token, the affiliated edges' share of dk / dv
        const bpt_status s = launch_bwd_span(p, pair0, np, ws.ext_dq, ws.aff_slab);
        if (s != BPT_OK) return s;
        kernel<<<dim3(tiles, np), kBwdThreads, smem, p.stream>>>(
            t, plan, cfg, (const __nv_bfloat16*)p.q, (const __nv_bfloat16*)p.k, (const __nv_bfloat16*)p.v,
            (const __nv_bfloat16*)p.rel_emb, (const __nv_bfloat16*)p.out, p.lse, (const __nv_bfloat16*)p.d_out,
            (__nv_bfloat16*)p.dq, ws.tile_range, ws.slabs, ws.drel_part, p.H, pair0, p.scale, p.lengths, p.drop);
        trace_mark(p.stream, "bwd_tile");
        if (pair0 == 0) {  // the groups that cover every node: the same for all pairs
            gather_plan_kernel<<<(2 * N + 255) / 256, 256, 0, p.stream>>>(t, plan, ws.tile_range, tiles, ws.node_tiles);
            trace_mark(p.stream, "gather_plan");
        }
        const int64_t warps = (int64_t)np * N;
        bwd_gather_kernel<<<(unsigned)((warps + 7) / 8), 256, 0, p.stream>>>(
            t, plan, ws.tile_range, ws.node_tiles, ws.slabs, ws.aff_slab, (__nv_bfloat16*)p.dk, (__nv_bfloat16*)p.dv,
            p.H, pair0, np, tiles, p.scale);
        trace_mark(p.stream, "bwd_gather");
        drel_group_kernel<<<dim3((unsigned)((per_cta + 255) / 256), kDrelGroups), 256, 0, p.stream>>>(
            ws.drel_part, ws.drel_grp, np * tiles, per_cta);
        trace_mark(p.stream, "drel_group");
        drel_final_kernel<<<(p.g->dims.n_rel * 64 + 255) / 256, 256, 0, p.stream>>>(
            t, plan, ws.drel_grp, p.d_rel, p.g->dims.n_rel, per_cta, p.scale, pair0 > 0);
        trace_mark(p.stream, "drel_final");
    }
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

}  // namespace bpt
