// Backward for the token rows on the 5th-generation tensor cores, key side: dk and dv of every node
// and the per-CTA partial sums of d_rel (arXiv 1911.04070, gradient of the Sec. 3.4 equation over the
// contextual edges of Sec. 3.2.2; relation embeddings of Sec. 3.4 are trainable), bf16, head size 64.
// Companion of attn_bwd_q_tc5.cu, which runs first and leaves the row terms d_out . out.
//
// One CTA = 128 consecutive nodes of one tree level (the keys) of one (batch entry, head) = the 128
// lanes of tensor memory.  The tokens that attend a node at its level from one side form one interval
// (the first and last node of a token's range grow with the token index), so the CTA walks the interval
// of its 128 keys in blocks of 64 query tokens ("items"), first the tokens to the right of the keys
// (for which the keys are left context, or the token itself), then the tokens to their left.  Per item
// one elected thread issues the transposed products
//     S^T = K_tile Q_blk^T,   dP^T = V_tile dO_blk^T,   QR^T = R_side Q_blk^T          (128 x 64 each)
// into tensor memory; four threads per key row rebuild P and dS for their row (the relative-position
// term of (query i, key m) is QR^T[offset(i, m)][i], passed through a shared table), and write P^T and
// dS^T as K-major A operands, plus dS again indexed [offset][query]; then
//     dK += dS^T Q_blk,   dV += P^T dO_blk,   dR_side += skew(dS)^T Q_blk
// accumulate in tensor memory over all items.  Every node's dk / dv row is thus complete inside one
// CTA and is written once, rounded once; there are no partial rows and no atomics.  The per-CTA d_rel
// partials ((k + 2) x 64 floats per side) are summed in a fixed order by drel_kv_reduce_kernel.
//
// A load warp keeps a ring of three (Q_blk, dO_blk) buffers full with TMA (each CTA its own copies) and computes
// each block's per-query facts (node range at this level, lse, row term); an MMA warp issues the
// products; mbarriers carry the hand-offs; every wait is bounded and a give-up is reported through the
// status word while the kernel runs to its end without waiting again.
#include "bpt_internal.cuh"
#include "mma_tools.cuh"
#include "tc5_host.cuh"
#include "tc5_tools.cuh"
#include "tile_geom.cuh"

namespace bpt {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kKvKeys = 128;                     // nodes per CTA
constexpr int kKvQB = 64;                        // query tokens per item
constexpr int kKvTpr = 4;                        // threads per key row
constexpr int kKvRowThreads = kKvKeys * kKvTpr;  // 16 warps
constexpr int kKvThreads = kKvRowThreads + 96;   // + load warp + two MMA warps
constexpr int kKvCols = kKvQB / kKvTpr;          // query columns per thread and item
constexpr int kKvGrp = 16;                       // ... worked through in groups of 16 (one 16-column tensor-memory load)
constexpr int kKvGroups = kKvCols / kKvGrp;
constexpr int kKvChan = 64 / kKvTpr;             // output channels per thread in the read-out
static_assert(kKvCols % kKvGrp == 0 && kKvChan % 16 == 0, "threads per key row: 1, 2 or 4");
constexpr int kKvRing = 3;
constexpr int kKvRelRows = 80;                   // relation rows per side (k + 2 <= 66), in 16-row boxes
constexpr int kKvBiasStride = 66;
constexpr uint32_t kKvColS = 0, kKvColDP = 64, kKvColQR = 128, kKvColDK = 192, kKvColDV = 256, kKvColDR = 320, kKvTmemCols = 512;

struct BwdKvSmem {
    static constexpr int k_off = 0;                                        // [128][64] keys
    static constexpr int v_off = k_off + kKvKeys * 128;
    static constexpr int r_off = v_off + kKvKeys * 128;                    // two sides x [128][64] (80 rows loaded)
    static constexpr int q_off = r_off + 2 * kKvKeys * 128;                // ring of [64][64] Q blocks
    static constexpr int g_off = q_off + kKvRing * kKvQB * 128;            // ring of [64][64] d_out blocks
    static constexpr int p_off = g_off + kKvRing * kKvQB * 128;            // P^T  [128 keys][64 queries]
    static constexpr int ds_off = p_off + kKvKeys * 128;                   // dS^T [128 keys][64 queries]
    static constexpr int sk_off = ds_off + kKvKeys * 128;                  // two x [128 offsets][64 queries]
    static constexpr int bias_off = sk_off + 2 * kKvKeys * 128;            // two x [64 queries][66 offsets] fp32
    static constexpr int meta_off = bias_off + 2 * kKvQB * kKvBiasStride * 4;  // ring of [64] (lo, hi, lse, delta)
    static constexpr int bar_off = meta_off + kKvRing * kKvQB * 16;
    static constexpr size_t bytes = bar_off + 256 + 1024;
};
static_assert(BwdKvSmem::q_off % 1024 == 0 && BwdKvSmem::g_off % 1024 == 0 && BwdKvSmem::p_off % 1024 == 0 &&
              BwdKvSmem::ds_off % 1024 == 0 && BwdKvSmem::sk_off % 1024 == 0 && BwdKvSmem::bias_off % 16 == 0 &&
              BwdKvSmem::meta_off % 16 == 0 && BwdKvSmem::bar_off % 8 == 0, "tile alignment");
static_assert(BwdKvSmem::bytes <= 227 * 1024, "shared memory of the key-side backward");

enum { kvSFull = 0, kvSFree, kvDsFull, kvDsFree, kvTiles, kvQFull, kvQFree = kvQFull + kKvRing, kvBarCount = kvQFree + kKvRing };

struct QMeta { int lo, hi; float lse2, delta; };

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// (level, first node) of key tile `x` when the tiles are numbered from the coarsest level down
__device__ __forceinline__ void tile_of(int n, int L, int x, int* level, int* m0) {
    for (int l = L; l >= 0; --l) {
        const int tiles = ((n >> l) + kKvKeys - 1) / kKvKeys;
        if (x < tiles) { *level = l; *m0 = x * kKvKeys; return; }
        x -= tiles;
    }
    *level = 0; *m0 = 0;
}

// First index in [lo, hi) at which a monotone predicate over the table turns true (hi if it never does), found by
// a whole warp: every round probes 32 evenly spaced entries, so a table of n entries takes log32(n) dependent loads.
template <class Pred>
__device__ __forceinline__ int warp_first_true(int lo, int hi, int lane, Pred pred) {
    while (lo < hi) {
        const int step = (hi - lo + 31) / 32;
        const int i = lo + lane * step;
        const bool p = i < hi ? pred(i) : true;
        const int f = __ffs(__ballot_sync(0xffffffffu, p)) - 1;   // first probe that is true, or -1
        if (f < 0) { lo = lo + 31 * step + 1; continue; }         // all 32 probes lie below hi and are false
        const int new_hi = min(lo + f * step, hi);
        lo = f > 0 ? lo + (f - 1) * step + 1 : new_hi;
        hi = new_hi;
    }
    return hi;
}

// plan[x * 2 + side] = (first query token rounded down to a block, number of 64-token blocks) of key tile x: the
// tokens that reach keys m0 .. m0 + 127 of the tile's level from that side form one interval, because the first
// and the last node of a token's range grow with the token index (two searches on the table of ranges, one warp per
// tile and side).
__global__ void key_tile_plan_kernel(TreeParams t, int n_left, int n_right, const int2* __restrict__ ranges,
                                     int2* __restrict__ plan, int tiles_total) {
    const int id = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (id >= tiles_total * 2) return;
    const int side = id & 1;
    int level, m0;
    tile_of(t.n, t.L, id >> 1, &level, &m0);
    int2 out = make_int2(0, 0);
    if (level < (side ? n_right : n_left)) {
        const int2* rg = ranges + (size_t)(side ? n_left + level : level) * t.n;
        const int m1 = m0 + kKvKeys - 1;
        const int first = warp_first_true(0, t.n, lane, [&](int i) { return __ldg(rg + i).y >= m0; });   // first token whose range ends at or beyond m0
        const int last = warp_first_true(first, t.n, lane, [&](int i) { return __ldg(rg + i).x > m1; }); // first token whose range starts beyond m1
        if (first < last) { out.x = first & ~(kKvQB - 1); out.y = (last - out.x + kKvQB - 1) / kKvQB; }
    }
    if (lane == 0) plan[id] = out;
}

// One group of an item's share of a row thread: its key node m against kKvGrp query columns (col0 .. col0 + 15 of the
// block).  Predicated, no branch per element.
// kSide: 1 = the keys are right context of the queries (offset m - lo), 0 = left context (offset hi - m).
// Two phases, so that no shared-memory store stands between the loads of different elements (the compiler must
// assume the by-offset stores alias the tables): first every weight, then every store.  The by-offset store of a
// missing edge goes, with value zero, to row 127 of the tile, which is no relation offset.
template <int kSide, bool kDrop>
__device__ __forceinline__ void kv_rows_item(const uint32_t* __restrict__ sv, const uint32_t* __restrict__ dv, const QMeta* __restrict__ mq,
                                             const float* __restrict__ bias_col, unsigned char* __restrict__ skw, int m, int col0,
                                             float scale_log2e, const DropoutParams& drop, uint32_t pair, uint32_t dst0, uint32_t src,
                                             uint32_t* __restrict__ pp, uint32_t* __restrict__ dd) {
    uint32_t at[kKvGrp];  // byte offset of each element's by-offset store
#pragma unroll
    for (int x = 0; x < kKvGrp; x += 2) {
        float pv[2], dsv[2];
#pragma unroll
        for (int y = 0; y < 2; ++y) {
            const QMeta a = mq[x + y];
            const bool in = m >= a.lo && m <= a.hi;
            const int off = kSide ? m - a.lo : a.hi - m;
            const int col = col0 + x + y;
            const float bias = in ? bias_col[(x + y) * kKvBiasStride + off] : 0.f;
            float pr = ex2f(fmaf(__uint_as_float(sv[x + y]), scale_log2e, bias));
            float dp = __uint_as_float(dv[x + y]), d;
            if constexpr (kDrop) {  // dP = W d_out.v, the weight that reaches dv is W P, dS keeps the undropped P
                const float wgt = dropout_weight(drop, pair, dst0 + (uint32_t)(x + y), src);
                d = pr * (dp * wgt - a.delta);
                pr *= wgt;
            } else {
                d = pr * (dp - a.delta);
            }
            pv[y] = in ? pr : 0.f;
            dsv[y] = in ? d : 0.f;
            const int so = in ? off : kKvKeys - 1;
            at[x + y] = (uint32_t)(so * 128 + ((((col >> 3) ^ so) & 7) << 4) + (col & 7) * 2);
        }
        pp[x >> 1] = pack_bf16(pv[0], pv[1]);
        dd[x >> 1] = pack_bf16(dsv[0], dsv[1]);
    }
#pragma unroll
    for (int x = 0; x < kKvGrp; ++x)
        *reinterpret_cast<uint16_t*>(skw + at[x]) = (uint16_t)((x & 1) ? dd[x >> 1] >> 16 : dd[x >> 1] & 0xffffu);
}

template <bool kDrop>
__global__ void __launch_bounds__(kKvThreads, 1)
bwd_kv_tc5_kernel(TreeParams t, int n_left, int n_right, const int2* __restrict__ ranges, const int2* __restrict__ plan,
                  const float* __restrict__ lse, const float* __restrict__ delta_in, const float* __restrict__ aff_slab,
                  __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv, float* __restrict__ drel_part,
                  int* __restrict__ status, int H, int pair0, float scale, const int32_t* __restrict__ lengths, DropoutParams drop,
                  const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_g,
                  const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                  const __grid_constant__ CUtensorMap tm_r) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* k_s = smem + BwdKvSmem::k_off;
    unsigned char* v_s = smem + BwdKvSmem::v_off;
    unsigned char* p_s = smem + BwdKvSmem::p_off;
    unsigned char* ds_s = smem + BwdKvSmem::ds_off;
    unsigned char* sk_s = smem + BwdKvSmem::sk_off;
    float* bias_s = reinterpret_cast<float*>(smem + BwdKvSmem::bias_off);
    QMeta* meta_s = reinterpret_cast<QMeta*>(smem + BwdKvSmem::meta_off);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + BwdKvSmem::bar_off);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kvBarCount);
    volatile int* abort_s = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* plan_s = const_cast<int*>(abort_s) + 1;  // qa0, blocks0, qa1, blocks1

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int pl = blockIdx.x, pair = pair0 + pl, b = pair / H, h = pair % H;  // x = pair: all pairs of the coarsest (longest) tiles start first
    const int N_nodes = 2 * t.n - 1;
    int level, m0;
    tile_of(t.n, t.L, blockIdx.y, &level, &m0);
    const int n_l = t.n >> level, id0 = node_id(t.n, level, 0);
    const size_t rs = (size_t)H * 64;
    const size_t boff = (size_t)b * N_nodes * rs + (size_t)h * 64;
    const uint32_t k_u = smem_u32(k_s), v_u = smem_u32(v_s), r_u = smem_u32(smem + BwdKvSmem::r_off),
                   q_u = smem_u32(smem + BwdKvSmem::q_off), g_u = smem_u32(smem + BwdKvSmem::g_off),
                   p_u = smem_u32(p_s), ds_u = smem_u32(ds_s), sk_u = smem_u32(sk_s), bar_u = smem_u32(bars);
    auto bar = [&](int i) { return bar_u + 8u * (uint32_t)i; };
    auto wait = [&](int i, uint32_t parity) {
        if (*abort_s) return;
        if (!tc5::mbar_wait_fast(bar(i), parity)) *abort_s = 1;
    };
    auto wait_idle = [&](int i, uint32_t parity) {  // for the load and MMA threads: suspends instead of spinning
        if (*abort_s) return;
        if (!tc5::mbar_wait_idle(bar(i), parity)) *abort_s = 1;
    };
    const int len = seq_len(lengths, b, t.n);
    const bool side_on[2] = {level < n_left, level < n_right};

    // ---- prologue: barriers, tensor memory, the query intervals of the two sides, cleared tiles ----
    if (tid == 0) {
        tc5::mbar_init(bar(kvSFull), 1);
        tc5::mbar_init(bar(kvSFree), kKvRowThreads);
        tc5::mbar_init(bar(kvDsFull), kKvRowThreads);
        tc5::mbar_init(bar(kvDsFree), 1);
        tc5::mbar_init(bar(kvTiles), 1);
        for (int i = 0; i < kKvRing; ++i) { tc5::mbar_init(bar(kvQFull + i), 33); tc5::mbar_init(bar(kvQFree + i), 1); }
        tc5::mbar_init_fence();
        *abort_s = 0;
    }
    if (w == 0) tc5::tmem_alloc(smem_u32(tmem_slot), kKvTmemCols);
    if (tid < 2) {  // the query blocks of the two sides
        const int2 pq = __ldg(plan + (size_t)blockIdx.y * 2 + tid);
        plan_s[2 * tid] = pq.x; plan_s[2 * tid + 1] = pq.y;
    }
    for (int idx = tid; idx < 2 * kKvKeys * 8; idx += kKvThreads)  // both by-offset tiles start from zero
        *reinterpret_cast<uint4*>(sk_s + idx * 16) = make_uint4(0, 0, 0, 0);
    tc5::fence_async_smem();
    tc5::fence_before_sync();
    __syncthreads();
    tc5::fence_after_sync();
    const uint32_t tbase = *tmem_slot;
    const int qa_side[2] = {plan_s[0], plan_s[2]}, nb_side[2] = {plan_s[1], plan_s[3]};
    const int J = nb_side[0] + nb_side[1];
    auto item_of = [&](int j, int& side, int& q0) {
        side = j >= nb_side[0];
        q0 = side ? qa_side[1] + (j - nb_side[0]) * kKvQB : qa_side[0] + j * kKvQB;
    };
    const int rel_cols = (t.k + 2 + 15) & ~15;

    if (w == kKvRowThreads / 32) {
        // =============== load warp: key / value / relation tiles once, then the ring of query blocks ===============
        if (J > 0) {
            if (lane == 0) {
                int boxes = 2 * (kKvKeys / 16);
                for (int s = 0; s < 2; ++s) if (nb_side[s] > 0) boxes += rel_cols / 16;
                tc5::mbar_expect_tx(bar(kvTiles), (uint32_t)boxes * 2048u);
                for (int x = 0; x < kKvKeys / 16; ++x) {
                    tc5::tma_load_4d(k_u + x * 2048, &tm_k, 0, h, id0 + m0 + 16 * x, b, bar(kvTiles));
                    tc5::tma_load_4d(v_u + x * 2048, &tm_v, 0, h, id0 + m0 + 16 * x, b, bar(kvTiles));
                }
                for (int s = 0; s < 2; ++s) {
                    if (nb_side[s] == 0) continue;
                    const int rel_base = s ? rel_right(t, level, 0) : (level == 0 ? 0 : rel_left(t, level, 0));
                    for (int x = 0; x < rel_cols / 16; ++x)
                        tc5::tma_load_2d(r_u + s * (kKvKeys * 128) + x * 2048, &tm_r, 0, rel_base + 16 * x, bar(kvTiles));
                }
            }
            for (int j = 0; j < J && !*abort_s; ++j) {
                int side, q0;
                item_of(j, side, q0);
                const int rb = j % kKvRing, ru = j / kKvRing;
                if (ru > 0) wait_idle(kvQFree + rb, (ru - 1) & 1);
                if (lane == 0) {
                    tc5::mbar_expect_tx(bar(kvQFull + rb), 2u * (kKvQB / 16) * 2048u);
                    for (int x = 0; x < kKvQB / 16; ++x) {
                        tc5::tma_load_4d(q_u + rb * (kKvQB * 128) + x * 2048, &tm_q, 0, h, q0 + 16 * x, b, bar(kvQFull + rb));
                        tc5::tma_load_4d(g_u + rb * (kKvQB * 128) + x * 2048, &tm_g, 0, h, q0 + 16 * x, b, bar(kvQFull + rb));
                    }
                }
                // per query: node range at this level (from the table), lse and row term
                float lv[kKvQB / 32], dl[kKvQB / 32];
                int2 rgv[kKvQB / 32];
#pragma unroll
                for (int x = 0; x < kKvQB / 32; ++x) {
                    const int i = q0 + lane + 32 * x;
                    rgv[x] = __ldg(ranges + (size_t)(side ? n_left + level : level) * t.n + i);
                    lv[x] = __ldg(lse + ((size_t)b * N_nodes + i) * H + h);
                    dl[x] = __ldg(delta_in + (size_t)pair * t.n + i);
                }
#pragma unroll
                for (int x = 0; x < kKvQB / 32; ++x) {
                    const int i = q0 + lane + 32 * x;
                    int2 rg = rgv[x];
                    if (len < t.n) {  // short sequence: a placeholder token attends nothing, right ranges end at the last real node
                        if (i >= len) rg = make_int2(1, 0);
                        else if (side == 1) rg.y = min(rg.y, (len - 1) >> level);
                    }
                    QMeta qm;
                    qm.lo = rg.x; qm.hi = rg.y;
                    qm.lse2 = lv[x] * kLog2e;
                    qm.delta = dl[x];
                    meta_s[rb * kKvQB + lane + 32 * x] = qm;
                }
                tc5::mbar_arrive(bar(kvQFull + rb));
            }
        }
    } else if (w == kKvRowThreads / 32 + 1) {
        // =============== first MMA warp: one thread issues S^T, dP^T and QR^T of every item ===============
        if (lane == 0 && J > 0) {
            const uint32_t id_t = tc5::instr_desc(kKvKeys, kKvQB, 0, 0);
            const uint32_t k_lo = tc5::desc_lo_k_major(k_u), v_lo = tc5::desc_lo_k_major(v_u);
            for (int j = 0; j < J && !*abort_s; ++j) {
                int side, q0;
                item_of(j, side, q0);
                const int rb = j % kKvRing, ru = j / kKvRing;
                if (j == 0) wait_idle(kvTiles, 0);
                wait_idle(kvQFull + rb, ru & 1);
                if (j > 0) wait_idle(kvSFree, (j - 1) & 1);
                if (*abort_s) break;
                tc5::fence_after_sync();
                const uint32_t q_lo = tc5::desc_lo_k_major(q_u + rb * (kKvQB * 128)), g_lo = tc5::desc_lo_k_major(g_u + rb * (kKvQB * 128)),
                               r_lo = tc5::desc_lo_k_major(r_u + side * (kKvKeys * 128));
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) tc5::mma_lo(tbase + kKvColS, k_lo + ks * 2, q_lo + ks * 2, id_t, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) tc5::mma_lo(tbase + kKvColDP, v_lo + ks * 2, g_lo + ks * 2, id_t, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) tc5::mma_lo(tbase + kKvColQR, r_lo + ks * 2, q_lo + ks * 2, id_t, ks > 0);
                tc5::commit(bar(kvSFull));
            }
        }
    } else if (w == kKvRowThreads / 32 + 2) {
        // =============== second MMA warp: one thread issues dK += dS^T Q_blk, dV += P^T dO_blk, dR_side += skew(dS)^T Q_blk ===============
        if (lane == 0 && J > 0) {
            const uint32_t id_o = tc5::instr_desc(kKvKeys, 64, 0, 1);
            const uint32_t ds_lo = tc5::desc_lo_k_major(ds_u), p_lo = tc5::desc_lo_k_major(p_u);
            for (int j = 0; j < J && !*abort_s; ++j) {
                int side, q0;
                item_of(j, side, q0);
                const int rb = j % kKvRing;
                wait_idle(kvDsFull, j & 1);
                if (*abort_s) break;
                tc5::fence_after_sync();
                const uint32_t q_lo = tc5::desc_lo_mn_major(q_u + rb * (kKvQB * 128)), g_lo = tc5::desc_lo_mn_major(g_u + rb * (kKvQB * 128));
                const uint32_t sk_lo = tc5::desc_lo_k_major(sk_u + (j & 1) * (kKvKeys * 128));
                const uint32_t first_all = j > 0, first_side = (side ? j > nb_side[0] : j > 0);
#pragma unroll
                for (int kk = 0; kk < kKvQB / 16; ++kk)
                    tc5::mma_lo(tbase + kKvColDK, ds_lo + kk * 2, q_lo + kk * (2048 / 16), id_o, (first_all || kk > 0) ? 1u : 0u);
#pragma unroll
                for (int kk = 0; kk < kKvQB / 16; ++kk)
                    tc5::mma_lo(tbase + kKvColDV, p_lo + kk * 2, g_lo + kk * (2048 / 16), id_o, (first_all || kk > 0) ? 1u : 0u);
#pragma unroll
                for (int kk = 0; kk < kKvQB / 16; ++kk)
                    tc5::mma_lo(tbase + kKvColDR + side * 64, sk_lo + kk * 2, q_lo + kk * (2048 / 16), id_o, (first_side || kk > 0) ? 1u : 0u);
                tc5::commit(bar(kvQFree + rb));
                tc5::commit(bar(kvDsFree));
            }
        }
    } else {
        // =============== row threads: four per key row, sixteen query columns each ===============
        const int quad = w & 3, part = w >> 2, row = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const float scale_log2e = scale * kLog2e;
        const int m = m0 + row;            // this thread's key node
        const int mw0 = m0 + quad * 32;    // first key of the warp
        for (int j = 0; j < J; ++j) {
            int side, q0;
            item_of(j, side, q0);
            const int rb = j % kKvRing;
            float* bias = bias_s + (j & 1) * (kKvQB * kKvBiasStride);
            unsigned char* skw = sk_s + (j & 1) * (kKvKeys * 128);
            wait(kvSFull, j & 1);
            tc5::fence_after_sync();
            uint32_t sv[kKvCols], dv[kKvCols], qr[kKvCols];
#pragma unroll
            for (int gq = 0; gq < kKvGroups; ++gq) {
                tc5::tmem_ld16(tbase + lane_base + kKvColS + part * kKvCols + gq * kKvGrp, *reinterpret_cast<uint32_t (*)[16]>(sv + gq * kKvGrp));
                tc5::tmem_ld16(tbase + lane_base + kKvColDP + part * kKvCols + gq * kKvGrp, *reinterpret_cast<uint32_t (*)[16]>(dv + gq * kKvGrp));
                if (quad < 3)   // lanes = relation offsets here
                    tc5::tmem_ld16(tbase + lane_base + kKvColQR + part * kKvCols + gq * kKvGrp, *reinterpret_cast<uint32_t (*)[16]>(qr + gq * kKvGrp));
            }
            tc5::tmem_ld_wait();
            tc5::fence_before_sync();
            tc5::mbar_arrive(bar(kvSFree));
            const QMeta* mq = meta_s + rb * kKvQB + part * kKvCols;
            if (quad < 3 && row < kKvBiasStride) {  // table entry = scale * log2(e) * q.r - lse * log2(e) of the query
                float nl[kKvCols];
#pragma unroll
                for (int x = 0; x < kKvCols; ++x) nl[x] = -mq[x].lse2;   // all loads before the first store
#pragma unroll
                for (int x = 0; x < kKvCols; ++x)
                    bias[(part * kKvCols + x) * kKvBiasStride + row] = fmaf(__uint_as_float(qr[x]), scale_log2e, nl[x]);
            }
            asm volatile("bar.sync 1, %0;" ::"n"(kKvRowThreads) : "memory");  // the table of this item is complete (and the other by-offset tile is cleared)

            // does any of the warp's 32 keys meet any of this thread group's 16 queries?
            bool hit = false;
            if (lane < kKvCols) { const QMeta a = mq[lane]; hit = a.lo <= a.hi && a.hi >= mw0 && a.lo <= mw0 + 31; }
            const unsigned hits = __ballot_sync(0xffffffffu, hit);
            uint32_t pp[kKvCols / 2], dd[kKvCols / 2];
#pragma unroll
            for (int x = 0; x < kKvCols / 2; ++x) pp[x] = dd[x] = 0u;
#pragma unroll
            for (int gq = 0; gq < kKvGroups; ++gq) {
                if ((hits >> (gq * kKvGrp)) & 0xffffu) {   // some of the warp's keys meet some of the group's queries
                    const int col0 = part * kKvCols + gq * kKvGrp;
                    const float* bias_col = bias + col0 * kKvBiasStride;
                    const uint32_t src = (uint32_t)(id0 + m), dst0 = (uint32_t)(q0 + col0);
                    if (side) kv_rows_item<1, kDrop>(sv + gq * kKvGrp, dv + gq * kKvGrp, mq + gq * kKvGrp, bias_col, skw, m, col0, scale_log2e, drop,
                                                     (uint32_t)pair, dst0, src, pp + gq * (kKvGrp / 2), dd + gq * (kKvGrp / 2));
                    else kv_rows_item<0, kDrop>(sv + gq * kKvGrp, dv + gq * kKvGrp, mq + gq * kKvGrp, bias_col, skw, m, col0, scale_log2e, drop,
                                                (uint32_t)pair, dst0, src, pp + gq * (kKvGrp / 2), dd + gq * (kKvGrp / 2));
                }
            }
            if (j > 0) wait(kvDsFree, (j - 1) & 1);   // the products that read P^T, dS^T of the item before are done (hidden behind the weights above)
#pragma unroll
            for (int c = 0; c < kKvCols / 8; ++c) {
                *reinterpret_cast<uint4*>(p_s + tile_off(row, part * (kKvCols / 8) + c)) = make_uint4(pp[4 * c], pp[4 * c + 1], pp[4 * c + 2], pp[4 * c + 3]);
                *reinterpret_cast<uint4*>(ds_s + tile_off(row, part * (kKvCols / 8) + c)) = make_uint4(dd[4 * c], dd[4 * c + 1], dd[4 * c + 2], dd[4 * c + 3]);
            }
            {   // clear the other by-offset tile for the next item (its products finished before this item's P^T was written)
                unsigned char* other = sk_s + ((j + 1) & 1) * (kKvKeys * 128);
                for (int idx = tid; idx < kKvRelRows * 8; idx += kKvRowThreads)
                    *reinterpret_cast<uint4*>(other + idx * 16) = make_uint4(0, 0, 0, 0);
            }
            tc5::fence_async_smem();
            tc5::fence_before_sync();
            tc5::mbar_arrive(bar(kvDsFull));
        }

        // ---- results: dk, dv rows (plus, for tokens, what the span rows left for them), d_rel partials ----
        if (J > 0) wait(kvDsFree, (J - 1) & 1);
        tc5::fence_after_sync();
#pragma unroll
        for (int cg = 0; cg < kKvChan / 16; ++cg) {   // this thread's output channels, sixteen at a time
            const int ch0 = part * kKvChan + cg * 16;
            uint32_t xk[16], xv[16];
            if (J > 0) {
                tc5::tmem_ld16(tbase + lane_base + kKvColDK + ch0, xk);
                tc5::tmem_ld16(tbase + lane_base + kKvColDV + ch0, xv);
                tc5::tmem_ld_wait();
            } else {
#pragma unroll
                for (int x = 0; x < 16; ++x) xk[x] = xv[x] = 0u;
            }
            if (level == 0 && m < t.n) {  // affiliated edges: the span pass's share of this token's dk / dv
                const float4* a = reinterpret_cast<const float4*>(aff_slab + ((size_t)pl * t.n + m) * 128 + ch0);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float4 ak = __ldg(a + c), av = __ldg(a + 16 + c);
                    xk[4 * c] = __float_as_uint(__uint_as_float(xk[4 * c]) + ak.x); xk[4 * c + 1] = __float_as_uint(__uint_as_float(xk[4 * c + 1]) + ak.y);
                    xk[4 * c + 2] = __float_as_uint(__uint_as_float(xk[4 * c + 2]) + ak.z); xk[4 * c + 3] = __float_as_uint(__uint_as_float(xk[4 * c + 3]) + ak.w);
                    xv[4 * c] = __float_as_uint(__uint_as_float(xv[4 * c]) + av.x); xv[4 * c + 1] = __float_as_uint(__uint_as_float(xv[4 * c + 1]) + av.y);
                    xv[4 * c + 2] = __float_as_uint(__uint_as_float(xv[4 * c + 2]) + av.z); xv[4 * c + 3] = __float_as_uint(__uint_as_float(xv[4 * c + 3]) + av.w);
                }
            }
#pragma unroll
            for (int c = 0; c < 2; ++c) {  // rounded once; staged in the K / V tiles for coalesced stores
                uint32_t a[4], bq[4];
#pragma unroll
                for (int y = 0; y < 4; ++y) {
                    a[y] = pack_bf16(__uint_as_float(xk[c * 8 + 2 * y]) * scale, __uint_as_float(xk[c * 8 + 2 * y + 1]) * scale);
                    bq[y] = pack_bf16(__uint_as_float(xv[c * 8 + 2 * y]), __uint_as_float(xv[c * 8 + 2 * y + 1]));
                }
                *reinterpret_cast<uint4*>(k_s + tile_off(row, (ch0 >> 3) + c)) = make_uint4(a[0], a[1], a[2], a[3]);
                *reinterpret_cast<uint4*>(v_s + tile_off(row, (ch0 >> 3) + c)) = make_uint4(bq[0], bq[1], bq[2], bq[3]);
            }
        }
        // d_rel partials of this CTA: [side][offset][channel], zero where the side brought nothing
        if (quad < 3) {  // lanes = relation offsets; the loads are warp-wide, the stores take the offsets in use
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                if (!side_on[s]) continue;
#pragma unroll
                for (int cg = 0; cg < kKvChan / 16; ++cg) {
                    const int ch0 = part * kKvChan + cg * 16;
                    uint32_t xr[16];
                    if (nb_side[s] > 0) {
                        tc5::tmem_ld16(tbase + lane_base + kKvColDR + s * 64 + ch0, xr);
                        tc5::tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int x = 0; x < 16; ++x) xr[x] = 0u;
                    }
                    if (row >= kKvBiasStride) continue;
                    float4* dst = reinterpret_cast<float4*>(drel_part + ((((size_t)pl * gridDim.y + blockIdx.y) * 2 + s) * kKvBiasStride + row) * 64 + ch0);
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        dst[c] = make_float4(__uint_as_float(xr[4 * c]), __uint_as_float(xr[4 * c + 1]), __uint_as_float(xr[4 * c + 2]), __uint_as_float(xr[4 * c + 3]));
                }
            }
        }
    }

    tc5::fence_before_sync();
    __syncthreads();
    for (int idx = tid; idx < kKvKeys * 8; idx += kKvThreads) {
        const int rr = idx >> 3, ch = idx & 7;
        if (m0 + rr < n_l) {
            const size_t at = boff + (size_t)(id0 + m0 + rr) * rs + ch * 8;
            *reinterpret_cast<uint4*>(dk + at) = *reinterpret_cast<const uint4*>(k_s + tile_off(rr, ch));
            *reinterpret_cast<uint4*>(dv + at) = *reinterpret_cast<const uint4*>(v_s + tile_off(rr, ch));
        }
    }
    if (tid == 0 && *abort_s && status) status[0] = (int)BPT_ERR_TIMEOUT;
    if (w == 0) tc5::tmem_free(tbase, kKvTmemCols);
}

constexpr int kKvDrelGroups = 32;
constexpr int kKvDrelVec = kKvBiasStride * 64 / 4;  // float4 per (CTA, side) partial

// d_rel, first stage: the (pair, tile) partials of one (level, side) in kKvDrelGroups groups, each summed in order.
// grid: (float4 blocks, level * 2 + side, group)
__global__ void __launch_bounds__(256)
drel_kv_group_kernel(TreeParams t, int n_left, int n_right, const float4* __restrict__ part, float4* __restrict__ grp,
                     int n_pairs, int tiles_total) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    const int level = blockIdx.y >> 1, side = blockIdx.y & 1, g = blockIdx.z;
    if (e >= kKvDrelVec || level >= (side ? n_right : n_left)) return;
    int x0 = 0;  // first tile of the level in the coarse-to-fine numbering
    for (int l = t.L; l > level; --l) x0 += ((t.n >> l) + kKvKeys - 1) / kKvKeys;
    const int tl = ((t.n >> level) + kKvKeys - 1) / kKvKeys, total = n_pairs * tl;
    const int per = (total + kKvDrelGroups - 1) / kKvDrelGroups;
    const int i0 = min(g * per, total), i1 = min(i0 + per, total);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i = i0; i < i1; ++i) {
        const int pl = i / tl, x = x0 + i % tl;
        const float4 v = part[(((size_t)pl * tiles_total + x) * 2 + side) * kKvDrelVec + e];
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    grp[((size_t)blockIdx.y * kKvDrelGroups + g) * kKvDrelVec + e] = acc;
}

// d_rel, second stage: one thread per (relation row, channel) adds the groups in order.  Rows no token edge carries
// (levels without contextual edges, the ancestor relations) are exact zeros.  With `accumulate` the pass adds to
// what earlier passes wrote.
__global__ void __launch_bounds__(256)
drel_kv_final_kernel(TreeParams t, int n_left, int n_right, const float* __restrict__ grp, float* __restrict__ d_rel,
                     int n_rel, float scale, int accumulate) {
    const int x = blockIdx.x * blockDim.x + threadIdx.x;
    if (x >= n_rel * 64) return;
    const int rid = x >> 6, ch = x & 63;
    const int W = t.k + 1;
    int level = -1, side = 0, off = 0;
    if (rid <= W) { level = 0; off = rid; }  // self and the left relations of level 0
    else if (rid < 1 + t.L * W) { level = (rid - 1) / W; off = (rid - 1) % W; if (level >= n_left) level = -1; }
    else if (rid < 1 + 2 * t.L * W) { side = 1; level = (rid - 1 - t.L * W) / W; off = (rid - 1 - t.L * W) % W; if (level >= n_right) level = -1; }
    float acc = 0.f;
    if (level >= 0) {
        const float* src = grp + ((size_t)(level * 2 + side) * kKvDrelGroups * kKvDrelVec) * 4 + off * 64 + ch;
        for (int g = 0; g < kKvDrelGroups; ++g) acc += src[(size_t)g * kKvDrelVec * 4];
    }
    d_rel[x] = accumulate ? d_rel[x] + acc * scale : acc * scale;
}

}  // namespace

int bwd_kv_tc5_tiles(const TreeParams& t) {
    int x = 0;
    for (int l = 0; l <= t.L; ++l) x += ((t.n >> l) + kKvKeys - 1) / kKvKeys;
    return x;
}

// per-CTA d_rel partials of n_pairs pairs, followed by the group sums of the first reduction stage
size_t bwd_kv_tc5_drel_floats(const TreeParams& t, int n_pairs) {
    return ((size_t)n_pairs * bwd_kv_tc5_tiles(t) * 2 + (size_t)2 * (t.L + 1) * kKvDrelGroups) * kKvBiasStride * 64;
}

// dk, dv of all nodes of pairs [pair0, pair0 + n_pairs) and d_rel (added to with pair0 > 0).
bpt_status launch_bwd_kv_tc5(const AttnProblem& p, int pair0, int n_pairs, const float* delta, const int2* ranges, int2* plan,
                             const float* aff_slab, float* drel_part) {
    const TreeParams& t = p.tree;
    int n_left, n_right;
    context_levels(t, &n_left, &n_right);
    auto kernel = p.drop.thr ? bwd_kv_tc5_kernel<true> : bwd_kv_tc5_kernel<false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BwdKvSmem::bytes) != cudaSuccess) return BPT_ERR_CUDA;
    alignas(64) CUtensorMap tm_q, tm_g, tm_k, tm_v, tm_r;
    const int N = 2 * t.n - 1;
    if (!tc5::encode_tiled() || !tc5::node_rows_map(&tm_q, p.q, p.B, N, p.H) || !tc5::node_rows_map(&tm_g, p.d_out, p.B, N, p.H) ||
        !tc5::node_rows_map(&tm_k, p.k, p.B, N, p.H) || !tc5::node_rows_map(&tm_v, p.v, p.B, N, p.H) ||
        !tc5::rel_rows_map(&tm_r, p.rel_emb, p.g->dims.n_rel))
        return BPT_ERR_CUDA;
    const int tiles = bwd_kv_tc5_tiles(t);
    if (pair0 == 0) {
        key_tile_plan_kernel<<<(tiles * 2 * 32 + 127) / 128, 128, 0, p.stream>>>(t, n_left, n_right, ranges, plan, tiles);
        trace_mark(p.stream, "key_tile_plan");
    }
    kernel<<<dim3(n_pairs, tiles), kKvThreads, BwdKvSmem::bytes, p.stream>>>(
        t, n_left, n_right, ranges, plan, p.lse, delta, aff_slab, (__nv_bfloat16*)p.dk, (__nv_bfloat16*)p.dv, drel_part, p.status,
        p.H, pair0, p.scale, p.lengths, p.drop, tm_q, tm_g, tm_k, tm_v, tm_r);
    trace_mark(p.stream, "bwd_kv_tc5");
    const int n_rel = p.g->dims.n_rel, n_lv = max(n_left, n_right);
    float* grp = drel_part + (size_t)n_pairs * tiles * 2 * kKvBiasStride * 64;
    drel_kv_group_kernel<<<dim3((kKvDrelVec + 255) / 256, 2 * n_lv, kKvDrelGroups), 256, 0, p.stream>>>(
        t, n_left, n_right, (const float4*)drel_part, (float4*)grp, n_pairs, tiles);
    trace_mark(p.stream, "drel_kv_group");
    drel_kv_final_kernel<<<(n_rel * 64 + 255) / 256, 256, 0, p.stream>>>(t, n_left, n_right, grp, p.d_rel, n_rel, p.scale, pair0 > 0);
    trace_mark(p.stream, "drel_kv_final");
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

}  // namespace bpt
