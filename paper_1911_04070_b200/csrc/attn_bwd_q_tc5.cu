// Backward for the token rows on the 5th-generation tensor cores, query side: dq of the tokens
// (arXiv 1911.04070, gradient of the Sec. 3.4 equation over the contextual edges of Sec. 3.2.2),
// bf16, head size 64.  Its companion, the key side (dk, dv, d_rel), is attn_bwd_kv_tc5.cu; the two
// kernels each recompute the edge weights from q, k and the stored log-sum-exp, so nothing but the
// row terms d_out . out travels between them and no partial gradient row ever leaves the chip.
//
// One CTA = 128 consecutive tokens of one (batch entry, head) = the 128 lanes of tensor memory, four
// threads per token row, plus a load warp and an MMA warp.  As in the tensor-memory forward the nodes
// a tile attends at one (side, level) are one contiguous range; a range wider than 96 nodes is worked
// through in "items" of at most 96 key columns.  Per item one elected thread issues
//     QR = Q R_chunk^T (first item of a chunk),  S = Q K_item^T,  dP = dO V_item^T
// into tensor memory; the row threads read their part, form P = exp2(S + bias - lse) and
// dS = P (dP - d_out . out) in registers and write dS to shared memory twice: by key column (the
// K-major A operand of dQ += dS K_item) and by relation offset (the A operand of dQ += skew(dS) R_chunk,
// issued with the chunk's last item).  dQ stays in tensor memory for the whole tile.
//
// Pipeline: the load thread keeps three K buffers, one V buffer and two R buffers full with TMA
// (cp.async.bulk.tensor, each CTA its own copies); every hand-off is an mbarrier; every wait is bounded and a
// give-up is reported through the status word while the kernel runs to its end without waiting again.
#include "bpt_internal.cuh"
#include "mma_tools.cuh"
#include "tc5_host.cuh"
#include "tc5_tools.cuh"
#include "tile_geom.cuh"

namespace bpt {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kQTok = 128;                      // tokens per CTA
constexpr int kQTpr = 4;                        // threads per token row
constexpr int kQRowThreads = kQTok * kQTpr;     // 16 warps
constexpr int kQThreads = kQRowThreads + 96;    // + load warp + two MMA warps
constexpr int kQItemCols = 96;                  // key columns per item (three 32-column pieces per warp)
constexpr int kQPieces = kQItemCols / 32;
constexpr int kQRelRows = 80;                   // relation rows per chunk (k + 2 <= 66), in 16-row boxes
constexpr int kQBiasRows = 66;
constexpr int kQKBufs = 3;
constexpr uint32_t kQColS = 0, kQColDP = 160, kQColQR = 320, kQColDQ = 400, kQTmemCols = 512;  // reads of S / dP may run 63 columns past the item
constexpr int kQMaxItems = 96;

struct BwdQSmem {
    static constexpr int q_off = 0;
    static constexpr int g_off = q_off + kQTok * 128;                     // d_out tile
    static constexpr int k_off = g_off + kQTok * 128;                     // three buffers of 96 rows
    static constexpr int v_off = k_off + kQKBufs * kQItemCols * 128;
    static constexpr int r_off = v_off + kQItemCols * 128;                // two buffers of 80 rows
    static constexpr int ds_off = r_off + 2 * kQRelRows * 128;            // dS by key column: 2 blocks of [128][64]
    static constexpr int sk_off = ds_off + 2 * kQTok * 128;               // dS by relation offset: 2 blocks of [128][64]
    static constexpr int bias_off = sk_off + 2 * kQTok * 128;             // [66 offsets][128 rows] fp32
    static constexpr int bar_off = bias_off + kQBiasRows * kQTok * 4;     // mbarriers, tensor-memory slot, abort flag
    static constexpr int row_off = bar_off + 256;                         // lse * log2(e), d_out . out per row
    static constexpr int bnd_off = row_off + 2 * kQTok * 4;               // [chunks][128] short2, [chunks] int2, items
    static size_t bytes(int chunks) {
        return (size_t)bnd_off + (size_t)chunks * (kQTok * 4 + 8 + 16) + (size_t)kQMaxItems * 16 + 16 + 1024;
    }
};
static_assert(BwdQSmem::k_off % 1024 == 0 && BwdQSmem::v_off % 1024 == 0 && BwdQSmem::r_off % 1024 == 0 &&
              BwdQSmem::ds_off % 1024 == 0 && BwdQSmem::sk_off % 1024 == 0 && (kQItemCols * 128) % 1024 == 0 &&
              (kQRelRows * 128) % 1024 == 0, "swizzled tiles start on 1024-byte boundaries");

enum { kBarSFull = 0, kBarSFree, kBarDsFull, kBarDsFree, kBarVFull, kBarVFree, kBarKFull, kBarKFree = kBarKFull + kQKBufs,
       kBarRFull = kBarKFree + kQKBufs, kBarRFree = kBarRFull + 2, kBarCount = kBarRFree + 2 };

struct Item { int c, col0, ncols, flags; };  // flags: 1 = first item of its chunk, 2 = last

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void quad_bar(int quad) {  // the kQTpr warps that share a lane quadrant
    switch (quad) {
        case 0: asm volatile("bar.sync 1, %0;" ::"n"(32 * kQTpr) : "memory"); break;
        case 1: asm volatile("bar.sync 2, %0;" ::"n"(32 * kQTpr) : "memory"); break;
        case 2: asm volatile("bar.sync 3, %0;" ::"n"(32 * kQTpr) : "memory"); break;
        default: asm volatile("bar.sync 4, %0;" ::"n"(32 * kQTpr) : "memory"); break;
    }
}

constexpr int kQCols = 32 / kQTpr;  // columns of one 32-column piece a thread takes

struct RowCtx {
    int row, part;
    float lse, delta, scale_log2e;
    const float* bias_row;   // bias table entry of offset 0 of this row
    unsigned char* sk_row;   // this row inside a [128][64] block of the by-offset tile
    unsigned char* ds_s;
    uint32_t pair, dst;      // dropout: (batch entry, head) pair and destination node
};

// One item's share of a row thread: kQCols columns of each of `npieces` 32-column pieces.  kDir = +1: offsets grow
// with the column (right side), -1: they fall (left side), so that the bias loads and the by-offset stores of
// consecutive columns are a compile-time stride apart.  Everything is predicated, nothing branches per element.
template <int kDir, bool kDrop>
__device__ __forceinline__ void q_rows_item(const RowCtx& rc, const uint32_t (&sv)[kQPieces][kQCols], const uint32_t (&dv)[kQPieces][kQCols],
                                            int npieces, int ob, int omin, int orange, int ch0, int n_ch,
                                            const DropoutParams& drop, uint32_t src0,
                                            uint32_t tiles_free_bar, uint32_t tiles_free_parity, bool must_wait, volatile int* abort_s) {
    const int r7 = rc.row & 7;
    const float* bp = rc.bias_row + ob * kQTok;
    // Per piece two phases, so that no shared-memory store stands between the table loads of its elements (the
    // compiler must assume that the tile stores alias the table): first the piece's dS values, then its stores.
#pragma unroll
    for (int p = 0; p < kQPieces; ++p) {
        if (p < npieces) {
            float dsv[kQCols];
            uint32_t inm = 0;  // bit x: the element is an edge
#pragma unroll
            for (int x = 0; x < kQCols; ++x) {
                const int u = p * 32 + x;
                const bool in = (unsigned)(ob - omin + kDir * u) < (unsigned)orange;
                const float bias = in ? bp[kDir * u * kQTok] : 0.f;
                const float pr = ex2f(fmaf(__uint_as_float(sv[p][x]), rc.scale_log2e, bias));
                float dp = __uint_as_float(dv[p][x]);
                if constexpr (kDrop) dp *= dropout_weight(drop, rc.pair, rc.dst, src0 + (uint32_t)u);  // dP = W d_out.v; dS keeps the undropped P
                dsv[x] = in ? pr * (dp - rc.delta) : 0.f;
                inm |= in ? 1u << x : 0u;
            }
            if (p == 0 && must_wait && !*abort_s && !tc5::mbar_wait_fast(tiles_free_bar, tiles_free_parity)) *abort_s = 1;  // first store of the item: the dS tiles must be free
            // by-offset stores: the 8 offsets of this piece lie in at most two 16-byte chunks of the row
            const int of = ob + kDir * (p * 32);          // offset of the thread's first column of the piece
            const int a = of & 7, c1 = of >> 3, c2 = c1 + kDir;
            unsigned char* b1 = rc.sk_row + ((c1 >> 3) * (kQTok * 128)) + (((c1 & 7) ^ r7) << 4) + a * 2;
            unsigned char* b2 = rc.sk_row + ((c2 >> 3) * (kQTok * 128)) + (((c2 & 7) ^ r7) << 4) + (a - kDir * 8) * 2;
            uint32_t pk[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) pk[x] = pack_bf16(dsv[2 * x], dsv[2 * x + 1]);
#pragma unroll
            for (int x = 0; x < kQCols; ++x) {
                const bool first_chunk = kDir > 0 ? (x < 8 - a) : (x <= a);
                if (inm & (1u << x))
                    *reinterpret_cast<uint16_t*>((first_chunk ? b1 : b2) + kDir * x * 2) = (uint16_t)((x & 1) ? pk[x >> 1] >> 16 : pk[x >> 1] & 0xffffu);
            }
            const int ci = ch0 + p * 4 + rc.part;  // 16-byte chunk (8 keys) of the dS row
            if (ci < n_ch)
                *reinterpret_cast<uint4*>(rc.ds_s + (ci >> 3) * (kQTok * 128) + tile_off(rc.row, ci & 7)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
    }
}

// ranges[c * n + i] = (first, last) node of chunk c (left levels, then right levels) that token i attends, with the
// conventions of fill_row_bounds and the self loop folded into the left range of level 0.  Both tensor-memory
// backward kernels read the table instead of walking the levels again for every tile they visit.
__global__ void level_ranges_kernel(TreeParams t, int n_left, int n_right, int2* __restrict__ ranges) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= t.n) return;
    {
        LeftWalk w(t, i);
        for (int c = 0; c < n_left; ++c) {
            int2 v = make_int2(0, -1);
            if (w.valid()) { v = make_int2(w.lo, w.hi); w.next(); }
            if (c == 0) v = v.x > v.y ? make_int2(i, i) : make_int2(v.x, i);
            ranges[(size_t)c * t.n + i] = v;
        }
    }
    RightWalk w(t, i);
    for (int c = 0; c < n_right; ++c) {
        const int n_l = t.n >> c;
        int2 v = make_int2(n_l, n_l - 1);
        if (w.valid()) { v = make_int2(w.lo, w.hi); w.next(); }
        ranges[(size_t)(n_left + c) * t.n + i] = v;
    }
}

template <bool kDrop>
__global__ void __launch_bounds__(kQThreads, 1)
bwd_q_tc5_kernel(TreeParams t, int n_left, int n_right, const int2* __restrict__ ranges,
                 const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ out,
                 const float* __restrict__ lse, const __nv_bfloat16* __restrict__ d_out,
                 __nv_bfloat16* __restrict__ dq, float* __restrict__ delta_out, int* __restrict__ status,
                 int H, float scale, const int32_t* __restrict__ lengths, DropoutParams drop,
                 const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                 const __grid_constant__ CUtensorMap tm_r) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* q_s = smem + BwdQSmem::q_off;
    unsigned char* g_s = smem + BwdQSmem::g_off;
    unsigned char* ds_s = smem + BwdQSmem::ds_off;
    unsigned char* sk_s = smem + BwdQSmem::sk_off;
    float* bias_s = reinterpret_cast<float*>(smem + BwdQSmem::bias_off);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + BwdQSmem::bar_off);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kBarCount);
    volatile int* abort_s = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* n_items_s = const_cast<int*>(abort_s) + 1;
    float* lse_s = reinterpret_cast<float*>(smem + BwdQSmem::row_off);
    float* delta_s = lse_s + kQTok;
    short2* bnd = reinterpret_cast<short2*>(smem + BwdQSmem::bnd_off);
    const int chunks = n_left + n_right;
    int2* crange = reinterpret_cast<int2*>(bnd + chunks * kQTok);
    Item* items = reinterpret_cast<Item*>(crange + chunks + (chunks & 1));  // 16-byte aligned
    short2* wrange = reinterpret_cast<short2*>(items + kQMaxItems);           // [chunks][4]: union of the ranges of 32 rows

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int t0 = blockIdx.x * kQTok, h = blockIdx.y, b = blockIdx.z;
    const int N_nodes = 2 * t.n - 1;
    const size_t rs = (size_t)H * 64;
    const size_t boff = (size_t)b * N_nodes * rs + (size_t)h * 64;
    const uint32_t q_u = smem_u32(q_s), g_u = smem_u32(g_s), k_u = smem_u32(smem + BwdQSmem::k_off),
                   v_u = smem_u32(smem + BwdQSmem::v_off), r_u = smem_u32(smem + BwdQSmem::r_off),
                   ds_u = smem_u32(ds_s), sk_u = smem_u32(sk_s), bar_u = smem_u32(bars);
    auto bar = [&](int i) { return bar_u + 8u * (uint32_t)i; };
    // bounded wait; once any wait has given up every later one returns at once, so the kernel winds down
    auto wait = [&](int i, uint32_t parity) {
        if (*abort_s) return;
        if (!tc5::mbar_wait_fast(bar(i), parity)) *abort_s = 1;
    };
    auto wait_idle = [&](int i, uint32_t parity) {  // for the load and MMA threads: suspends instead of spinning
        if (*abort_s) return;
        if (!tc5::mbar_wait_idle(bar(i), parity)) *abort_s = 1;
    };

    // ---- prologue: Q, d_out and out tiles, row terms, row ranges, barriers, tensor memory ----
    unsigned char* o_s = ds_s;  // the forward's output rows, only until the row terms are known
    for (int idx = tid; idx < kQTok * 8; idx += kQThreads) {
        const int rr = idx >> 3, ch = idx & 7;
        const size_t src = boff + (size_t)(t0 + rr) * rs + ch * 8;
        cp_async16(q_u + tile_off(rr, ch), q + src);
        cp_async16(g_u + tile_off(rr, ch), d_out + src);
        cp_async16(ds_u + tile_off(rr, ch), out + src);
    }
    cp_async_commit();
    int2* bnd_abs = reinterpret_cast<int2*>(sk_s);  // absolute ranges, only until the relative table is written
    for (int idx = tid; idx < chunks * kQTok; idx += kQThreads)   // the rows' ranges, self loop included, from the table
        bnd_abs[idx] = __ldg(ranges + (size_t)(idx / kQTok) * t.n + t0 + (idx % kQTok));
    if (tid < kQTok) lse_s[tid] = lse[((size_t)b * N_nodes + t0 + tid) * H + h] * kLog2e;
    if (tid == 0) {
        tc5::mbar_init(bar(kBarSFull), 1);
        tc5::mbar_init(bar(kBarSFree), kQRowThreads);
        tc5::mbar_init(bar(kBarDsFull), kQRowThreads);
        tc5::mbar_init(bar(kBarDsFree), 1);
        tc5::mbar_init(bar(kBarVFull), 1);
        tc5::mbar_init(bar(kBarVFree), 1);
        for (int i = 0; i < kQKBufs; ++i) { tc5::mbar_init(bar(kBarKFull + i), 1); tc5::mbar_init(bar(kBarKFree + i), 1); }
        for (int i = 0; i < 2; ++i) { tc5::mbar_init(bar(kBarRFull + i), 1); tc5::mbar_init(bar(kBarRFree + i), 1); }
        tc5::mbar_init_fence();
        *abort_s = 0;
    }
    if (w == 0) tc5::tmem_alloc(smem_u32(tmem_slot), kQTmemCols);
    cp_async_wait<0>();
    tc5::fence_async_smem();
    tc5::fence_before_sync();
    __syncthreads();
    tc5::fence_after_sync();
    const uint32_t tbase = *tmem_slot;
    if (tid < 2 * kQTok) {   // delta_i = d_out_i . out_i: two threads per row
        const int row = tid >> 1, hf = tid & 1;
        float acc = 0.f;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            const uint4 a = *reinterpret_cast<const uint4*>(g_s + tile_off(row, hf * 4 + ch));
            const uint4 o = *reinterpret_cast<const uint4*>(o_s + tile_off(row, hf * 4 + ch));
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, ow[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                acc = fmaf(__uint_as_float(aw[x] << 16), __uint_as_float(ow[x] << 16), acc);
                acc = fmaf(__uint_as_float(aw[x] & 0xffff0000u), __uint_as_float(ow[x] & 0xffff0000u), acc);
            }
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        if (hf == 0) {
            delta_s[row] = acc;
            delta_out[((size_t)b * H + h) * t.n + t0 + row] = acc;  // the key-side kernel reads the row terms from here
        }
    }
    for (int c = w; c < chunks; c += kQThreads / 32) {
        int2 u = make_int2(0x7fffffff, -1);
#pragma unroll
        for (int part = 0; part < kQTok / 32; ++part) {
            const int2 a = rows_union(bnd_abs + c * kQTok, part * 32, 32, lane);
            u.x = min(u.x, a.x); u.y = max(u.y, a.y);
        }
        if (lane == 0) crange[c] = u;
    }
    __syncthreads();
    {   // short sequence: the staged ranges stay those of the full graph, the rows' ranges shrink
        const int len = seq_len(lengths, b, t.n);
        if (len < t.n) {
            if (tid < kQTok) mask_row_bounds<kQTok>(t, t0, tid, n_left, n_right, bnd_abs, len);
            __syncthreads();
        }
    }
    for (int idx = tid; idx < chunks * kQTok; idx += kQThreads) {
        const int2 a = bnd_abs[idx];
        const int base = crange[idx / kQTok].x;
        bnd[idx] = a.x <= a.y ? make_short2((short)(a.x - base), (short)(a.y - base)) : make_short2(1, 0);
    }
    if (tid == 0) {  // the item list: every non-empty chunk in pieces of at most kQItemCols columns
        int n = 0;
        for (int c = 0; c < chunks; ++c) {
            const int2 cr = crange[c];
            if (cr.x > cr.y) continue;
            const int width = cr.y - cr.x + 1;
            const int nb = (width + kQItemCols - 1) / kQItemCols;
            const int per = (((width + nb - 1) / nb) + 15) & ~15;
            for (int s = 0; s < nb && n < kQMaxItems; ++s) {
                const int col0 = s * per, left = width - col0;
                items[n++] = Item{c, col0, min(per, (left + 15) & ~15), (s == 0 ? 1 : 0) | (s == nb - 1 ? 2 : 0)};
            }
        }
        *n_items_s = n;
    }
    for (int e = w; e < chunks * 4; e += kQThreads / 32) {  // per chunk and group of 32 rows: the union of the rows' ranges
        const int2 a = rows_union(bnd_abs + (e >> 2) * kQTok, (e & 3) * 32, 32, lane);
        const int base = crange[e >> 2].x;
        if (lane == 0) wrange[e] = a.x <= a.y ? make_short2((short)(a.x - base), (short)(a.y - base)) : make_short2(1, 0);
    }
    __syncthreads();  // also: the out tile in the dS buffer and the absolute ranges in the skew buffer are consumed
    const int J = *n_items_s;
    const int rel_cols = (t.k + 2 + 15) & ~15;  // relation rows a chunk can use, in whole 16-row boxes

    auto chunk_of = [&](const Item& it, int& level, int& side, int& base) {
        side = it.c >= n_left;
        level = side ? it.c - n_left : it.c;
        base = crange[it.c].x;
    };

    if (w == kQRowThreads / 32) {
        // =============== load warp: one thread keeps the K, V and R buffers full ===============
        if (lane == 0) {
            int ci = -1;  // chunks started so far - 1
            for (int j = 0; j < J && !*abort_s; ++j) {
                const Item it = items[j];
                int level, side, base;
                chunk_of(it, level, side, base);
                const int node0 = node_id(t.n, level, 0) + base + it.col0;
                const int kb = j % kQKBufs, ku = j / kQKBufs;
                if (it.flags & 1) {
                    ++ci;
                    const int rb = ci & 1, ru = ci >> 1;
                    if (ru > 0) wait_idle(kBarRFree + rb, (ru - 1) & 1);
                    const int rel_base = it.c == 0 ? 0 : (side ? rel_right(t, level, 0) : rel_left(t, level, 0));
                    tc5::mbar_expect_tx(bar(kBarRFull + rb), (uint32_t)(rel_cols / 16) * 2048u);
                    for (int x = 0; x < rel_cols / 16; ++x)
                        tc5::tma_load_2d(r_u + rb * (kQRelRows * 128) + x * 2048, &tm_r, 0, rel_base + 16 * x, bar(kBarRFull + rb));
                }
                if (ku > 0) wait_idle(kBarKFree + kb, (ku - 1) & 1);
                tc5::mbar_expect_tx(bar(kBarKFull + kb), (uint32_t)(it.ncols / 16) * 2048u);
                for (int x = 0; x < it.ncols / 16; ++x)
                    tc5::tma_load_4d(k_u + kb * (kQItemCols * 128) + x * 2048, &tm_k, 0, h, node0 + 16 * x, b, bar(kBarKFull + kb));
                if (j > 0) wait_idle(kBarVFree, (j - 1) & 1);
                tc5::mbar_expect_tx(bar(kBarVFull), (uint32_t)(it.ncols / 16) * 2048u);
                for (int x = 0; x < it.ncols / 16; ++x)
                    tc5::tma_load_4d(v_u + x * 2048, &tm_v, 0, h, node0 + 16 * x, b, bar(kBarVFull));
            }
        }
    } else if (w == kQRowThreads / 32 + 1) {
        // =============== first MMA warp: one thread issues QR (first item of a chunk), S and dP of every item ===============
        if (lane == 0) {
            const uint32_t q_lo = tc5::desc_lo_k_major(q_u), g_lo = tc5::desc_lo_k_major(g_u), v_lo = tc5::desc_lo_k_major(v_u);
            const uint32_t id_qr = tc5::instr_desc(kQTok, rel_cols, 0, 0);
            int ci_a = -1;
            for (int j = 0; j < J && !*abort_s; ++j) {
                const Item it = items[j];
                const int kb = j % kQKBufs, ku = j / kQKBufs;
                if (it.flags & 1) { ++ci_a; wait_idle(kBarRFull + (ci_a & 1), (ci_a >> 1) & 1); }
                wait_idle(kBarKFull + kb, ku & 1);
                wait_idle(kBarVFull, j & 1);
                if (j > 0) wait_idle(kBarSFree, (j - 1) & 1);   // every row thread holds its part of the item before
                if (*abort_s) break;
                tc5::fence_after_sync();
                const uint32_t k_lo = tc5::desc_lo_k_major(k_u + kb * (kQItemCols * 128));
                if (it.flags & 1) {
                    const uint32_t r_lo = tc5::desc_lo_k_major(r_u + (ci_a & 1) * (kQRelRows * 128));
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) tc5::mma_lo(tbase + kQColQR, q_lo + ks * 2, r_lo + ks * 2, id_qr, ks > 0);
                }
                const uint32_t id_s = tc5::instr_desc(kQTok, it.ncols, 0, 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) tc5::mma_lo(tbase + kQColS, q_lo + ks * 2, k_lo + ks * 2, id_s, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) tc5::mma_lo(tbase + kQColDP, g_lo + ks * 2, v_lo + ks * 2, id_s, ks > 0);
                tc5::commit(bar(kBarSFull));
                tc5::commit(bar(kBarVFree));
            }
        }
    } else if (w == kQRowThreads / 32 + 2) {
        // =============== second MMA warp: one thread issues dQ += dS K_item (+ skew(dS) R_chunk with the chunk's last item) ===============
        if (lane == 0) {
            const uint32_t ds_lo = tc5::desc_lo_k_major(ds_u), sk_lo = tc5::desc_lo_k_major(sk_u);
            const uint32_t id_o = tc5::instr_desc(kQTok, 64, 0, 1);
            int ci_b = -1;
            for (int j = 0; j < J && !*abort_s; ++j) {
                const Item it = items[j];
                const int kb = j % kQKBufs;
                if (it.flags & 1) ++ci_b;
                wait_idle(kBarDsFull, j & 1);
                if (*abort_s) break;
                tc5::fence_after_sync();
                const uint32_t k_lo = tc5::desc_lo_mn_major(k_u + kb * (kQItemCols * 128));
                const int nk = it.ncols >> 4;
#pragma unroll
                for (int kk = 0; kk < kQItemCols / 16; ++kk)   // a k-step of 16 keys: 32 bytes along a dS row, 16 rows of K
                    if (kk < nk)
                        tc5::mma_lo(tbase + kQColDQ, ds_lo + (kk >> 2) * (kQTok * 128 / 16) + (kk & 3) * 2, k_lo + kk * (2048 / 16), id_o,
                                    (j > 0 || kk > 0) ? 1u : 0u);
                if (it.flags & 2) {
                    const uint32_t r_lo = tc5::desc_lo_mn_major(r_u + (ci_b & 1) * (kQRelRows * 128));
                    const int nr = rel_cols >> 4;
#pragma unroll
                    for (int kk = 0; kk < kQRelRows / 16; ++kk)
                        if (kk < nr)
                            tc5::mma_lo(tbase + kQColDQ, sk_lo + (kk >> 2) * (kQTok * 128 / 16) + (kk & 3) * 2, r_lo + kk * (2048 / 16), id_o, 1u);
                    tc5::commit(bar(kBarRFree + (ci_b & 1)));
                }
                tc5::commit(bar(kBarKFree + kb));
                tc5::commit(bar(kBarDsFree));
            }
        }
    } else {
        // =============== row threads: four per token row ===============
        const int quad = w & 3, part = w >> 2, row = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const float scale_log2e = scale * kLog2e;
        RowCtx rc;
        rc.row = row; rc.part = part;
        rc.lse = lse_s[row]; rc.delta = delta_s[row]; rc.scale_log2e = scale_log2e;
        rc.bias_row = bias_s + row;
        rc.sk_row = sk_s + row * 128;
        rc.ds_s = ds_s;
        rc.pair = (uint32_t)(b * H + h); rc.dst = (uint32_t)(t0 + row);
        for (int j = 0; j < J; ++j) {
            const Item it = items[j];
            const int side = it.c >= n_left;
            const bool first = it.flags & 1;
            wait(kBarSFull, j & 1);   // QR (first item), S and dP of this item are in tensor memory
            tc5::fence_after_sync();

            uint32_t qr[16], qr2[16];
            const bool have_qr = first && part * 16 < rel_cols, have_qr2 = first && part == 0 && rel_cols > 64;
            if (have_qr) tc5::tmem_ld16(tbase + lane_base + kQColQR + part * 16, qr);
            if (have_qr2) tc5::tmem_ld16(tbase + lane_base + kQColQR + 64, qr2);

            // the columns of the item this warp's rows reach (chunk coordinates), from the table of the prologue
            const short2 my = bnd[it.c * kQTok + row];
            const short2 wu = wrange[it.c * 4 + quad];
            const int col_end = it.col0 + it.ncols;
            const int wlo = max((int)wu.x, it.col0), whi = min((int)wu.y, col_end - 1);
            const bool w_any = wu.x <= wu.y && wlo <= whi;
            const int c0 = w_any ? ((wlo - it.col0) & ~7) : 0;   // item coordinates
            const int npieces = w_any ? min(kQPieces, ((whi - it.col0 - c0) >> 5) + 1) : 0;
            uint32_t sv[kQPieces][kQCols], dv[kQPieces][kQCols];
#pragma unroll
            for (int p = 0; p < kQPieces; ++p)
                if (p < npieces) {
                    tc5::tmem_ld8(tbase + lane_base + kQColS + c0 + p * 32 + part * kQCols, sv[p]);
                    tc5::tmem_ld8(tbase + lane_base + kQColDP + c0 + p * 32 + part * kQCols, dv[p]);
                }
            tc5::tmem_ld_wait();
            tc5::fence_before_sync();
            tc5::mbar_arrive(bar(kBarSFree));  // this thread holds its part: the next item's products may overwrite it

            // The dS tiles are free once the products of the item before are done.  A chunk's first item needs that
            // at once (it clears the by-offset tile; and since those products only started when every row thread had
            // finished that item, nobody still reads the old bias values either); any other item only before its
            // first store, so its wait hides behind the first piece's arithmetic.
            const bool wait_late = j > 0 && !first && npieces > 0;
            if (j > 0 && !wait_late) wait(kBarDsFree, (j - 1) & 1);
            if (first) {
                // table entry = scale * log2(e) * q.r - lse * log2(e): the exponent of an edge is one fused multiply-add away
                if (have_qr) {
#pragma unroll
                    for (int x = 0; x < 16; ++x)
                        if (part * 16 + x < kQBiasRows) bias_s[(part * 16 + x) * kQTok + row] = fmaf(__uint_as_float(qr[x]), scale_log2e, -rc.lse);
                }
                if (have_qr2) {
#pragma unroll
                    for (int x = 0; x < kQBiasRows - 64; ++x) bias_s[(64 + x) * kQTok + row] = fmaf(__uint_as_float(qr2[x]), scale_log2e, -rc.lse);
                }
            }
            if (first) {
                // this row's entries of the by-offset tile start from zero (the row's four threads share the ten chunks)
                for (int ch = part; ch < kQRelRows / 8; ch += kQTpr)
                    *reinterpret_cast<uint4*>(sk_s + (ch >> 3) * (kQTok * 128) + tile_off(row, ch & 7)) = make_uint4(0, 0, 0, 0);
                quad_bar(quad);  // bias values and zeros of the row are in place
            }

            // The row attends chunk columns my.x .. my.y (cnt of them); chunk column e has offset e - my.x on the right
            // side and my.y - e on the left side.  This thread's first column is e0; its columns inside both the row's
            // range and the item are those whose offset lies in [omin, omin + orange).
            const int cnt = my.x <= my.y ? my.y - my.x + 1 : 0;
            const int e0 = it.col0 + c0 + part * kQCols;
            const int n_ch = it.ncols >> 3, ch0 = c0 >> 3;
            int ob, omin, omax1;
            if (side) { ob = e0 - my.x; omin = 0; omax1 = min(cnt, col_end - my.x); }
            else { ob = my.y - e0; omin = max(0, my.y - (col_end - 1)); omax1 = cnt; }
            const int orange = max(omax1 - omin, 0);
            uint32_t src0 = 0;
            if constexpr (kDrop) src0 = (uint32_t)(node_id(t.n, side ? it.c - n_left : it.c, 0) + crange[it.c].x + e0);
            if (side) q_rows_item<1, kDrop>(rc, sv, dv, npieces, ob, omin, orange, ch0, n_ch, drop, src0, bar(kBarDsFree), (j - 1) & 1, wait_late, abort_s);
            else q_rows_item<-1, kDrop>(rc, sv, dv, npieces, ob, omin, orange, ch0, n_ch, drop, src0, bar(kBarDsFree), (j - 1) & 1, wait_late, abort_s);
            for (int ci = part; ci < n_ch; ci += kQTpr)  // the rest of the row is zero
                if (ci < ch0 || ci >= ch0 + npieces * 4)
                    *reinterpret_cast<uint4*>(ds_s + (ci >> 3) * (kQTok * 128) + tile_off(row, ci & 7)) = make_uint4(0, 0, 0, 0);
            tc5::fence_async_smem();   // written with ordinary stores, read by the tensor core
            tc5::fence_before_sync();
            tc5::mbar_arrive(bar(kBarDsFull));
        }
        // ---- dq = scale * dQ, rounded once to bf16 into the Q tile ----
        if (J > 0) wait(kBarDsFree, (J - 1) & 1);
        tc5::fence_after_sync();
        uint32_t x[16];
        tc5::tmem_ld16(tbase + lane_base + kQColDQ + part * 16, x);
        tc5::tmem_ld_wait();
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
            uint32_t pk[4];
#pragma unroll
            for (int y = 0; y < 4; ++y)
                pk[y] = J > 0 ? pack_bf16(__uint_as_float(x[ch * 8 + 2 * y]) * scale, __uint_as_float(x[ch * 8 + 2 * y + 1]) * scale) : 0u;
            *reinterpret_cast<uint4*>(q_s + tile_off(row, part * 2 + ch)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
    }

    // ---- epilogue: coalesced stores of the dq tile; tensor memory back ----
    tc5::fence_before_sync();
    __syncthreads();
    for (int idx = tid; idx < kQTok * 8; idx += kQThreads) {
        const int rr = idx >> 3, ch = idx & 7;
        *reinterpret_cast<uint4*>(dq + boff + (size_t)(t0 + rr) * rs + ch * 8) = *reinterpret_cast<const uint4*>(q_s + tile_off(rr, ch));
    }
    if (tid == 0 && *abort_s && status) status[0] = (int)BPT_ERR_TIMEOUT;
    if (w == 0) tc5::tmem_free(tbase, kQTmemCols);
}

}  // namespace

void launch_level_ranges(const TreeParams& t, int n_left, int n_right, int2* ranges, cudaStream_t stream) {
    level_ranges_kernel<<<(t.n + 127) / 128, 128, 0, stream>>>(t, n_left, n_right, ranges);
}

int bwd_q_tc5_chunks(const TreeParams& t) {
    int n_left, n_right;
    context_levels(t, &n_left, &n_right);
    return n_left + n_right;
}

bool bwd_q_tc5_fits(const TreeParams& t) {
    if (!tc5::encode_tiled() || t.n < kQTok) return false;
    int n_left, n_right;
    context_levels(t, &n_left, &n_right);
    // items: every chunk of a tile is at most 128 / 2^level + k + 2 nodes wide
    int n_items = 0;
    for (int c = 0; c < n_left + n_right; ++c) {
        const int level = c >= n_left ? c - n_left : c;
        n_items += ((kQTok >> level) + t.kc + 2 + kQItemCols - 1) / kQItemCols;
    }
    return n_items <= kQMaxItems && BwdQSmem::bytes(n_left + n_right) <= 227 * 1024;
}

// dq of the token rows, the row terms d_out . out of the tokens into `delta` ([B * H][n] fp32) and the table of the
// tokens' node ranges into `ranges` ([chunks][n] int2), which the key-side kernel reads too.
bpt_status launch_bwd_q_tc5(const AttnProblem& p, float* delta, int2* ranges) {
    int n_left, n_right;
    context_levels(p.tree, &n_left, &n_right);
    const size_t smem = BwdQSmem::bytes(n_left + n_right);
    if (smem > 227 * 1024 || p.H > 65535 || p.B > 65535) return BPT_ERR_UNSUPPORTED;
    auto kernel = p.drop.thr ? bwd_q_tc5_kernel<true> : bwd_q_tc5_kernel<false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return BPT_ERR_CUDA;
    alignas(64) CUtensorMap tm_k, tm_v, tm_r;
    const int N = 2 * p.tree.n - 1;
    if (!tc5::encode_tiled() || !tc5::node_rows_map(&tm_k, p.k, p.B, N, p.H) || !tc5::node_rows_map(&tm_v, p.v, p.B, N, p.H) ||
        !tc5::rel_rows_map(&tm_r, p.rel_emb, p.g->dims.n_rel))
        return BPT_ERR_CUDA;
    launch_level_ranges(p.tree, n_left, n_right, ranges, p.stream);
    trace_mark(p.stream, "level_ranges");
    const dim3 grid(p.tree.n / kQTok, p.H, p.B);
    kernel<<<grid, kQThreads, smem, p.stream>>>(p.tree, n_left, n_right, ranges, (const __nv_bfloat16*)p.q, (const __nv_bfloat16*)p.out,
                                                p.lse, (const __nv_bfloat16*)p.d_out, (__nv_bfloat16*)p.dq, delta, p.status,
                                                p.H, p.scale, p.lengths, p.drop, tm_k, tm_v, tm_r);
    trace_mark(p.stream, "bwd_q_tc5");
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

}  // namespace bpt
