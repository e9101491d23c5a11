// Tiled forward for the token rows on the 5th-generation tensor cores (tcgen05, accumulators in
// tensor memory): arXiv 1911.04070, Sec. 3.4 equation over the contextual edges of Sec. 3.2.2,
// bf16, head size 64.
//
// One CTA = 128 consecutive tokens of one (batch entry, head) = the 128 lanes of tensor memory, two
// threads per token row (warps w and w + 4 read the same lane quadrant and split the columns), plus
// a load warp and two MMA warps.  The nodes a tile attends at one (side, level) are one contiguous
// range ("chunk"); a chunk is worked through in "items" of at most 64 key columns.  Per item one
// elected thread issues
//     QR = Q R_chunk^T (first item of a chunk)   -- the relative-position terms of every offset
//     S  = Q K_item^T  (128 x 16..64)
// into tensor memory.  The row's bias values go to a shared table indexed [offset][row], so that the
// per-row shift between node index and offset is plain address arithmetic.  The row threads read their
// part of S, form the masked scores, and write P = exp2(score - m) to shared memory as the K-major A
// operand of
//     O += P V_item    (128 x 64),
// which stays in tensor memory for the whole tile and is read once at the end.  m is the row's
// reference exponent: the row maximum of the first item that holds an edge of the row, raised later
// (with O and the row sum rescaled in place) only when an item's maximum exceeds it by more than 8
// binary orders of magnitude -- softmax is invariant to the shift, and P stays far inside the range
// of bf16 and fp32 either way.  The self loop is offset 0 of the level-0 left chunk.
//
// The kernel is sized for two CTAs per SM (at most 112 KB of shared memory, 256 tensor-memory columns,
// 80 registers): while one tile waits for a product, a copy or a barrier the other one computes.  A
// load thread keeps two K and two V buffers and one R buffer full with TMA (cp.async.bulk.tensor, 16-row
// boxes straight into the 128-byte-swizzled layout the tensor core reads, each CTA its own copies); every hand-off
// is an mbarrier; the load and MMA threads suspend in their waits instead of spinning; every wait is
// bounded and a give-up is reported through the status word while the kernel runs to its end without
// waiting again.  The per-token node ranges come from a table (one entry per chunk and token) that a small
// kernel writes before this one.
#include "bpt_internal.cuh"
#include "mma_tools.cuh"
#include "tc5_host.cuh"
#include "tc5_tools.cuh"
#include "tile_geom.cuh"

namespace bpt {

void launch_level_ranges(const TreeParams& t, int n_left, int n_right, int2* ranges, cudaStream_t stream);

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kFTok = 128;                      // tokens per CTA
constexpr int kFTpr = 2;                        // threads per token row
constexpr int kFRowThreads = kFTok * kFTpr;     // 8 warps
constexpr int kFThreads = kFRowThreads + 96;    // + load warp + two MMA warps
constexpr int kFItemCols = 64;                  // key columns per item
constexpr int kFPieces = kFItemCols / 32;       // 32-column pieces of an item
constexpr int kFCols = 32 / kFTpr;              // columns of a piece one thread takes
constexpr int kFRelRows = 80;                   // relation rows per chunk (k + 2 <= 66), in 16-row boxes
constexpr int kFBiasRows = 66;
constexpr int kFBufs = 2;                       // K buffers and V buffers
constexpr uint32_t kFColS = 0, kFColQR = 64, kFColO = 160, kFTmemCols = 256;
constexpr int kFMaxItems = 96;
constexpr float kFBump = 8.f;                   // an item's maximum may exceed the reference by this much (base-2 exponent)

struct FwdSmem {
    static constexpr int q_off = 0;
    static constexpr int k_off = q_off + kFTok * 128;
    static constexpr int v_off = k_off + kFBufs * kFItemCols * 128;
    static constexpr int r_off = v_off + kFBufs * kFItemCols * 128;
    static constexpr int p_off = r_off + kFRelRows * 128;                 // [128 rows][64 keys] bf16
    static constexpr int bias_off = p_off + kFTok * 128;                  // [66 offsets][128 rows] fp32
    static constexpr int bar_off = bias_off + kFBiasRows * kFTok * 4;     // mbarriers, tensor-memory slot, abort flag, item count
    static constexpr int xch_off = bar_off + 256;                         // [2 items in flight][kFTpr][128 rows] fp32
    static constexpr int tab_off = xch_off + 2 * kFTpr * kFTok * 4;       // [chunks] int2, then the items
    static size_t bytes(int chunks) { return (size_t)tab_off + (size_t)(chunks + (chunks & 1)) * 8 + (size_t)kFMaxItems * 16 + 1024; }
};
static_assert(FwdSmem::k_off % 1024 == 0 && FwdSmem::v_off % 1024 == 0 && FwdSmem::r_off % 1024 == 0 &&
              FwdSmem::p_off % 1024 == 0 && (kFItemCols * 128) % 1024 == 0, "swizzled tiles start on 1024-byte boundaries");
static_assert(kFColQR + kFRelRows <= kFColO && kFColO + 64 <= kFTmemCols, "tensor-memory regions");

enum { kFBarSFull = 0, kFBarSFree, kFBarPFull, kFBarPFree, kFBarRFull, kFBarRFree, kFBarKFull, kFBarKFree = kFBarKFull + kFBufs,
       kFBarVFull = kFBarKFree + kFBufs, kFBarVFree = kFBarVFull + kFBufs, kFBarCount = kFBarVFree + kFBufs };

struct FItem { int c, col0, ncols, flags; };  // flags: 1 = first item of its chunk

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// barrier of the kFTpr warps that share a lane quadrant (ids 1..4; id 0 is __syncthreads)
__device__ __forceinline__ void quad_barrier(int quad) {
    switch (quad) {
        case 0: asm volatile("bar.sync 1, %0;" ::"n"(32 * kFTpr) : "memory"); break;
        case 1: asm volatile("bar.sync 2, %0;" ::"n"(32 * kFTpr) : "memory"); break;
        case 2: asm volatile("bar.sync 3, %0;" ::"n"(32 * kFTpr) : "memory"); break;
        default: asm volatile("bar.sync 4, %0;" ::"n"(32 * kFTpr) : "memory"); break;
    }
}

// Masked scores of one thread's share of an item (base-2 exponent; -inf where the row has no edge) and their
// maximum.  kDir = +1: offsets grow with the column (right side), -1: they fall (left side), so that the bias
// loads of consecutive columns are a compile-time stride apart.  ob: offset of the thread's first column;
// an element is an edge when its offset lies in [omin, omin + orange).
template <int kDir>
__device__ __forceinline__ float scores_item(uint32_t (&sv)[kFPieces][kFCols], const bool (&pp)[kFPieces], const float* bias_row,
                                             int ob, int omin, int orange, float scale_log2e) {
    const float* bp = bias_row + ob * kFTok;
    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // independent chains
#pragma unroll
    for (int p = 0; p < kFPieces; ++p) {
        if (pp[p]) {
#pragma unroll
            for (int x = 0; x < kFCols; ++x) {
                const int u = p * 32 + x;
                const bool in = (unsigned)(ob - omin + kDir * u) < (unsigned)orange;
                const float bias = in ? bp[kDir * u * kFTok] : 0.f;
                const float val = in ? fmaf(__uint_as_float(sv[p][x]), scale_log2e, bias) : -INFINITY;
                sv[p][x] = __float_as_uint(val);
                mx4[x & 3] = fmaxf(mx4[x & 3], val);
            }
        }
    }
    return fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
}

template <bool kDrop>  // attention dropout compiled in or out
__global__ void __launch_bounds__(kFThreads, 2)
fwd_tc5_kernel(TreeParams t, int n_left, int n_right, const int2* __restrict__ ranges,
               const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
               int* __restrict__ status, int H, float scale_log2e, const int32_t* __restrict__ lengths, DropoutParams drop,
               const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
               const __grid_constant__ CUtensorMap tm_r) {
    extern __shared__ unsigned char smem_raw[];
    // the swizzle pattern is a function of the address bits, so the tiles must start 1024-aligned
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* q_s = smem + FwdSmem::q_off;
    unsigned char* p_s = smem + FwdSmem::p_off;
    float* bias_s = reinterpret_cast<float*>(smem + FwdSmem::bias_off);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + FwdSmem::bar_off);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kFBarCount);
    volatile int* abort_s = reinterpret_cast<volatile int*>(tmem_slot + 1);
    int* n_items_s = const_cast<int*>(abort_s) + 1;
    float* xch_s = reinterpret_cast<float*>(smem + FwdSmem::xch_off);
    const int chunks = n_left + n_right;
    int2* crange = reinterpret_cast<int2*>(smem + FwdSmem::tab_off);
    FItem* items = reinterpret_cast<FItem*>(crange + chunks + (chunks & 1));  // 16-byte aligned

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int t0 = blockIdx.x * kFTok, h = blockIdx.y, b = blockIdx.z;
    const int N_nodes = 2 * t.n - 1;
    const size_t rs = (size_t)H * 64;
    const size_t boff = (size_t)b * N_nodes * rs + (size_t)h * 64;
    const uint32_t q_u = smem_u32(q_s), k_u = smem_u32(smem + FwdSmem::k_off), v_u = smem_u32(smem + FwdSmem::v_off),
                   r_u = smem_u32(smem + FwdSmem::r_off), p_u = smem_u32(p_s), bar_u = smem_u32(bars);
    auto bar = [&](int i) { return bar_u + 8u * (uint32_t)i; };
    // bounded wait; once any wait has given up every later one returns at once, so the kernel winds down
    auto wait = [&](int i, uint32_t parity) {
        if (*abort_s) return;
        if (!tc5::mbar_wait_fast(bar(i), parity)) *abort_s = 1;
    };
    auto wait_idle = [&](int i, uint32_t parity) {  // for the load and MMA threads
        if (*abort_s) return;
        if (!tc5::mbar_wait_idle(bar(i), parity)) *abort_s = 1;
    };

    // ---- prologue: Q tile, the tile's node range per chunk, the item list, barriers, tensor memory ----
    for (int idx = tid; idx < kFTok * 8; idx += kFThreads) {
        const int rr = idx >> 3, ch = idx & 7;
        cp_async16(q_u + tile_off(rr, ch), q + boff + (size_t)(t0 + rr) * rs + ch * 8);
    }
    cp_async_commit();
    if (tid == 0) {
        tc5::mbar_init(bar(kFBarSFull), 1);
        tc5::mbar_init(bar(kFBarSFree), kFRowThreads);
        tc5::mbar_init(bar(kFBarPFull), kFRowThreads);
        tc5::mbar_init(bar(kFBarPFree), 1);
        tc5::mbar_init(bar(kFBarRFull), 1);
        tc5::mbar_init(bar(kFBarRFree), 1);
        for (int i = 0; i < kFBufs; ++i) {
            tc5::mbar_init(bar(kFBarKFull + i), 1); tc5::mbar_init(bar(kFBarKFree + i), 1);
            tc5::mbar_init(bar(kFBarVFull + i), 1); tc5::mbar_init(bar(kFBarVFree + i), 1);
        }
        tc5::mbar_init_fence();
        *abort_s = 0;
    }
    if (w == 0) tc5::tmem_alloc(smem_u32(tmem_slot), kFTmemCols);
    for (int c = w; c < chunks; c += kFThreads / 32) {  // union of the 128 rows' ranges (full graph: a length only shrinks rows)
        int2 u = make_int2(0x7fffffff, -1);
#pragma unroll
        for (int part = 0; part < kFTok / 32; ++part) {
            const int2 a = __ldg(ranges + (size_t)c * t.n + t0 + part * 32 + lane);
            if (a.x <= a.y) { u.x = min(u.x, a.x); u.y = max(u.y, a.y); }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            u.x = min(u.x, __shfl_xor_sync(0xffffffffu, u.x, o));
            u.y = max(u.y, __shfl_xor_sync(0xffffffffu, u.y, o));
        }
        if (lane == 0) crange[c] = u;
    }
    cp_async_wait<0>();
    tc5::fence_async_smem();
    tc5::fence_before_sync();
    __syncthreads();
    tc5::fence_after_sync();
    const uint32_t tbase = *tmem_slot;
    if (tid == 0) {  // the item list: every non-empty chunk in pieces of at most kFItemCols columns
        int n = 0;
        for (int c = 0; c < chunks; ++c) {
            const int2 cr = crange[c];
            if (cr.x > cr.y) continue;
            const int width = cr.y - cr.x + 1;
            const int nb = (width + kFItemCols - 1) / kFItemCols;
            const int per = (((width + nb - 1) / nb) + 15) & ~15;
            for (int s = 0; s < nb && n < kFMaxItems; ++s) {
                const int col0 = s * per, left = width - col0;
                if (left <= 0) break;
                items[n++] = FItem{c, col0, min(per, (left + 15) & ~15), s == 0 ? 1 : 0};
            }
        }
        *n_items_s = n;
    }
    __syncthreads();
    const int J = *n_items_s;
    const int rel_cols = (t.k + 2 + 15) & ~15;  // relation rows a chunk can use, in whole 16-row boxes

    if (w == kFRowThreads / 32) {
        // =============== load warp: one thread keeps the K, V and R buffers full ===============
        if (lane == 0) {
            int ci = -1;  // chunks started so far - 1
            for (int j = 0; j < J && !*abort_s; ++j) {
                const FItem it = items[j];
                const int side = it.c >= n_left, level = side ? it.c - n_left : it.c;
                const int node0 = node_id(t.n, level, 0) + crange[it.c].x + it.col0;
                const int kb = j % kFBufs, ku = j / kFBufs;
                if (ku > 0) wait_idle(kFBarKFree + kb, (ku - 1) & 1);
                tc5::mbar_expect_tx(bar(kFBarKFull + kb), (uint32_t)(it.ncols / 16) * 2048u);
                for (int x = 0; x < it.ncols / 16; ++x)
                    tc5::tma_load_4d(k_u + kb * (kFItemCols * 128) + x * 2048, &tm_k, 0, h, node0 + 16 * x, b, bar(kFBarKFull + kb));
                if (it.flags & 1) {
                    ++ci;
                    if (ci > 0) wait_idle(kFBarRFree, (ci - 1) & 1);
                    const int rel_base = it.c == 0 ? 0 : (side ? rel_right(t, level, 0) : rel_left(t, level, 0));
                    tc5::mbar_expect_tx(bar(kFBarRFull), (uint32_t)(rel_cols / 16) * 2048u);
                    for (int x = 0; x < rel_cols / 16; ++x)
                        tc5::tma_load_2d(r_u + x * 2048, &tm_r, 0, rel_base + 16 * x, bar(kFBarRFull));
                }
                if (ku > 0) wait_idle(kFBarVFree + kb, (ku - 1) & 1);
                tc5::mbar_expect_tx(bar(kFBarVFull + kb), (uint32_t)(it.ncols / 16) * 2048u);
                for (int x = 0; x < it.ncols / 16; ++x)
                    tc5::tma_load_4d(v_u + kb * (kFItemCols * 128) + x * 2048, &tm_v, 0, h, node0 + 16 * x, b, bar(kFBarVFull + kb));
            }
        }
    } else if (w == kFRowThreads / 32 + 1) {
        // =============== first MMA warp: one thread issues QR (first item of a chunk) and S of every item ===============
        if (lane == 0) {
            const uint32_t q_lo = tc5::desc_lo_k_major(q_u), r_lo = tc5::desc_lo_k_major(r_u);
            const uint32_t id_qr = tc5::instr_desc(kFTok, rel_cols, 0, 0);
            int ci = -1;
            for (int j = 0; j < J && !*abort_s; ++j) {
                const FItem it = items[j];
                const int kb = j % kFBufs, ku = j / kFBufs;
                if (it.flags & 1) { ++ci; wait_idle(kFBarRFull, ci & 1); }
                wait_idle(kFBarKFull + kb, ku & 1);
                if (j > 0) wait_idle(kFBarSFree, (j - 1) & 1);   // every row thread holds its part of the item before
                if (*abort_s) break;
                tc5::fence_after_sync();
                if (it.flags & 1) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) tc5::mma_lo(tbase + kFColQR, q_lo + ks * 2, r_lo + ks * 2, id_qr, ks > 0);
                    tc5::commit(bar(kFBarRFree));
                }
                const uint32_t k_lo = tc5::desc_lo_k_major(k_u + kb * (kFItemCols * 128));
                const uint32_t id_s = tc5::instr_desc(kFTok, it.ncols, 0, 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) tc5::mma_lo(tbase + kFColS, q_lo + ks * 2, k_lo + ks * 2, id_s, ks > 0);
                tc5::commit(bar(kFBarSFull));
                tc5::commit(bar(kFBarKFree + kb));
            }
        }
    } else if (w == kFRowThreads / 32 + 2) {
        // =============== second MMA warp: one thread issues O += P V_item ===============
        if (lane == 0) {
            const uint32_t p_lo = tc5::desc_lo_k_major(p_u);
            const uint32_t id_o = tc5::instr_desc(kFTok, 64, 0, 1);
            for (int j = 0; j < J && !*abort_s; ++j) {
                const FItem it = items[j];
                const int kb = j % kFBufs, ku = j / kFBufs;
                wait_idle(kFBarVFull + kb, ku & 1);
                wait_idle(kFBarPFull, j & 1);
                if (*abort_s) break;
                tc5::fence_after_sync();
                const uint32_t v_lo = tc5::desc_lo_mn_major(v_u + kb * (kFItemCols * 128));
                const int nk = it.ncols >> 4;
#pragma unroll
                for (int kk = 0; kk < kFItemCols / 16; ++kk)   // a k-step of 16 keys: 32 bytes along a P row, 16 rows of V
                    if (kk < nk) tc5::mma_lo(tbase + kFColO, p_lo + kk * 2, v_lo + kk * (2048 / 16), id_o, (j > 0 || kk > 0) ? 1u : 0u);
                tc5::commit(bar(kFBarPFree));
                tc5::commit(bar(kFBarVFree + kb));
            }
        }
    } else {
        // =============== row threads: two per token row ===============
        const int quad = w & 3, part = w >> 2, row = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const int len = seq_len(lengths, b, t.n);
        const float* bias_row = bias_s + row;
        float m_ref = -INFINITY, l_run = 0.f;
        int my_lo = 1, my_hi = 0, wlo = 1, whi = 0, id0 = 0;  // the row's and the warp's columns of the current chunk
        for (int j = 0; j < J; ++j) {
            const FItem it = items[j];
            const int side = it.c >= n_left;
            const bool first = it.flags & 1;
            if (first) {  // the row's node range at this chunk, from the table; a length shrinks it
                const int level = side ? it.c - n_left : it.c;
                int2 a = __ldg(ranges + (size_t)it.c * t.n + t0 + row);
                if (len < t.n) {
                    if (side && a.x <= a.y) a.y = min(a.y, (len - 1) >> level);
                    if (t0 + row >= len) a = make_int2(1, 0);
                }
                const int base = crange[it.c].x;
                const bool any = a.x <= a.y;
                my_lo = any ? a.x - base : 1;
                my_hi = any ? a.y - base : 0;
                wlo = __reduce_min_sync(0xffffffffu, any ? my_lo : 0x7fffffff);
                whi = __reduce_max_sync(0xffffffffu, any ? my_hi : -1);
                id0 = node_id(t.n, level, 0) + base;
                if (j > 0) quad_barrier(quad);  // the row's other thread has read the bias values of the chunk before
            }
            wait(kFBarSFull, j & 1);   // QR (first item) and S of this item are in tensor memory
            tc5::fence_after_sync();
            if (first) {  // bias row -> table [offset][row]; the threads of a row share the offsets
#pragma unroll
                for (int gi = 0; gi < (kFRelRows / 16 + kFTpr - 1) / kFTpr; ++gi) {
                    const int g = part + gi * kFTpr;
                    if (g * 16 < rel_cols) {  // the same for the whole warp
                        uint32_t x[16];
                        tc5::tmem_ld16(tbase + lane_base + kFColQR + g * 16, x);
                        tc5::tmem_ld_wait();
#pragma unroll
                        for (int y = 0; y < 16; ++y)
                            if (g * 16 + y < kFBiasRows) bias_s[(g * 16 + y) * kFTok + row] = __uint_as_float(x[y]) * scale_log2e;
                    }
                }
            }
            // the 32-column pieces of the item that this warp's rows reach
            const int col_end = it.col0 + it.ncols;
            bool pp[kFPieces];
            uint32_t sv[kFPieces][kFCols];
#pragma unroll
            for (int p = 0; p < kFPieces; ++p) {
                pp[p] = p * 32 < it.ncols && wlo <= it.col0 + p * 32 + 31 && whi >= it.col0 + p * 32;
                if (pp[p]) tc5::tmem_ld16(tbase + lane_base + kFColS + p * 32 + part * kFCols, sv[p]);
            }
            tc5::tmem_ld_wait();
            tc5::fence_before_sync();
            tc5::mbar_arrive(bar(kFBarSFree));  // this thread holds its part: the next item's product may overwrite it
            if (first) quad_barrier(quad);      // the row's bias values are all in the table

            // The row attends chunk columns my_lo .. my_hi (cnt of them); chunk column e has offset e - my_lo on the right
            // side and my_hi - e on the left side.  This thread's first column is e0; its columns inside both the row's
            // range and the item are those whose offset lies in [omin, omin + orange).
            const int cnt = my_lo <= my_hi ? my_hi - my_lo + 1 : 0;
            const int e0 = it.col0 + part * kFCols;
            int ob, omin, omax1;
            if (side) { ob = e0 - my_lo; omin = 0; omax1 = min(cnt, col_end - my_lo); }
            else { ob = my_hi - e0; omin = max(0, my_hi - (col_end - 1)); omax1 = cnt; }
            const int orange = max(omax1 - omin, 0);
            const float mx = side ? scores_item<1>(sv, pp, bias_row, ob, omin, orange, scale_log2e)
                                  : scores_item<-1>(sv, pp, bias_row, ob, omin, orange, scale_log2e);
            float* xch = xch_s + (j & 1) * (kFTpr * kFTok);
            xch[part * kFTok + row] = mx;
            quad_barrier(quad);
            const float mx_row = fmaxf(xch[row], xch[kFTok + row]);
            const bool bump = m_ref != -INFINITY && mx_row > m_ref + kFBump;
            if (__any_sync(0xffffffffu, bump)) {
                // rare: raise the reference of the rows that need it; O and the row sums follow (the other rows scale by 1)
                if (j > 0) wait(kFBarPFree, (j - 1) & 1);  // every product into O so far is done
                tc5::fence_after_sync();
                const float corr = bump ? ex2(m_ref - mx_row) : 1.f;
#pragma unroll
                for (int hh = 0; hh < 64 / kFTpr / 16; ++hh) {
                    uint32_t x[16];
                    tc5::tmem_ld16(tbase + lane_base + kFColO + part * (64 / kFTpr) + hh * 16, x);
                    tc5::tmem_ld_wait();
#pragma unroll
                    for (int y = 0; y < 16; ++y) x[y] = __float_as_uint(__uint_as_float(x[y]) * corr);
                    tc5::tmem_st16(tbase + lane_base + kFColO + part * (64 / kFTpr) + hh * 16, x);
                }
                tc5::tmem_st_wait();
                tc5::fence_before_sync();
                l_run *= corr;
                if (bump) m_ref = mx_row;
            }
            if (m_ref == -INFINITY) m_ref = mx_row;  // the first item that holds an edge of the row sets the reference
            const float m_use = m_ref == -INFINITY ? 0.f : m_ref;

            if (j > 0) wait(kFBarPFree, (j - 1) & 1);  // the product that read the P tile of the item before is done
            float l4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int p = 0; p < kFPieces; ++p) {
                if (pp[p]) {
                    uint32_t pk[kFCols / 2];
#pragma unroll
                    for (int x = 0; x < kFCols / 2; ++x) {
                        float p0 = ex2(__uint_as_float(sv[p][2 * x]) - m_use);
                        float p1 = ex2(__uint_as_float(sv[p][2 * x + 1]) - m_use);
                        l4[x & 3] += p0 + p1;
                        if constexpr (kDrop) {  // the weights that reach V are dropped, the softmax sum is not
                            const uint32_t src = (uint32_t)(id0 + e0 + p * 32 + 2 * x);
                            p0 *= dropout_weight(drop, (uint32_t)(b * H + h), (uint32_t)(t0 + row), src);
                            p1 *= dropout_weight(drop, (uint32_t)(b * H + h), (uint32_t)(t0 + row), src + 1);
                        }
                        pk[x] = pack_bf16(p0, p1);
                    }
#pragma unroll
                    for (int cc = 0; cc < kFCols / 8; ++cc)  // 16-byte chunks (8 keys) of the P row
                        *reinterpret_cast<uint4*>(p_s + tile_off(row, p * 4 + part * (kFCols / 8) + cc)) =
                            make_uint4(pk[cc * 4], pk[cc * 4 + 1], pk[cc * 4 + 2], pk[cc * 4 + 3]);
                } else if (p * 32 < it.ncols) {
#pragma unroll
                    for (int cc = 0; cc < kFCols / 8; ++cc)
                        *reinterpret_cast<uint4*>(p_s + tile_off(row, p * 4 + part * (kFCols / 8) + cc)) = make_uint4(0, 0, 0, 0);
                }
            }
            l_run += (l4[0] + l4[1]) + (l4[2] + l4[3]);
            tc5::fence_async_smem();   // P was written with ordinary stores and is read by the tensor core
            tc5::mbar_arrive(bar(kFBarPFull));
        }

        // ---- row sums of the row's threads, normalise, round once to bf16 into the Q tile ----
        float* xl = xch_s + (J & 1) * (kFTpr * kFTok);  // the buffer the last item did not use
        xl[part * kFTok + row] = l_run;
        if (J > 0) wait(kFBarPFree, (J - 1) & 1);
        tc5::fence_after_sync();
        quad_barrier(quad);
        float l_all = 0.f;
#pragma unroll
        for (int x = 0; x < kFTpr; ++x) l_all += xl[x * kFTok + row];
        const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
#pragma unroll
        for (int hh = 0; hh < 64 / kFTpr / 16; ++hh) {
            uint32_t x[16];
            tc5::tmem_ld16(tbase + lane_base + kFColO + part * (64 / kFTpr) + hh * 16, x);
            tc5::tmem_ld_wait();
#pragma unroll
            for (int ch = 0; ch < 2; ++ch) {
                uint32_t pk[4];
#pragma unroll
                for (int y = 0; y < 4; ++y)
                    pk[y] = inv > 0.f ? pack_bf16(__uint_as_float(x[ch * 8 + 2 * y]) * inv, __uint_as_float(x[ch * 8 + 2 * y + 1]) * inv) : 0u;
                *reinterpret_cast<uint4*>(q_s + tile_off(row, part * (64 / kFTpr / 8) + hh * 2 + ch)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
        }
        if (part == 0) lse[((size_t)b * N_nodes + t0 + row) * H + h] = l_all > 0.f ? (m_ref + log2f(l_all)) * kLn2 : 0.f;
    }

    // ---- epilogue: coalesced stores of the output tile; tensor memory back ----
    tc5::fence_before_sync();
    __syncthreads();
    for (int idx = tid; idx < kFTok * 8; idx += kFThreads) {
        const int rr = idx >> 3, ch = idx & 7;
        *reinterpret_cast<uint4*>(out + boff + (size_t)(t0 + rr) * rs + ch * 8) =
            *reinterpret_cast<const uint4*>(q_s + tile_off(rr, ch));
    }
    if (tid == 0 && *abort_s && status) status[0] = (int)BPT_ERR_TIMEOUT;
    if (w == 0) tc5::tmem_free(tbase, kFTmemCols);
}

int fwd_tc5_items(const TreeParams& t, int n_left, int n_right) {
    int n_items = 0;
    for (int c = 0; c < n_left + n_right; ++c) {
        const int level = c >= n_left ? c - n_left : c;
        n_items += ((kFTok >> level) + t.kc + 2 + kFItemCols - 1) / kFItemCols;
    }
    return n_items;
}

}  // namespace

// The tensor-memory kernel takes whole tiles of 128 tokens.
bool fwd_tc5_eligible(const AttnProblem& p) {
    if (!tc5::encode_tiled()) return false;
    if (!tile_path(p.tree.n, p.tree.k, p.d, p.dtype == BPT_BF16) || p.tree.n < kFTok) return false;
    int n_left, n_right;
    context_levels(p.tree, &n_left, &n_right);
    return fwd_tc5_items(p.tree, n_left, n_right) <= kFMaxItems && FwdSmem::bytes(n_left + n_right) <= 113 * 1024;
}

// The table of the tokens' node ranges ([chunks][n] int2) the kernel reads, in bytes.
size_t fwd_tc5_ranges_bytes(const TreeParams& t) {
    int n_left, n_right;
    context_levels(t, &n_left, &n_right);
    return ((size_t)(n_left + n_right) * t.n * sizeof(int2) + 255) & ~(size_t)255;
}

// Token rows of the forward; `status` is a device word that receives BPT_ERR_TIMEOUT when a wait gave up, `ranges`
// scratch of fwd_tc5_ranges_bytes().
bpt_status launch_fwd_tc5(const AttnProblem& p, int* status, int2* ranges) {
    int n_left, n_right;
    context_levels(p.tree, &n_left, &n_right);
    const size_t smem = FwdSmem::bytes(n_left + n_right);
    if (smem > 113 * 1024 || p.H > 65535 || p.B > 65535 || !ranges) return BPT_ERR_UNSUPPORTED;
    auto kernel = p.drop.thr ? fwd_tc5_kernel<true> : fwd_tc5_kernel<false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return BPT_ERR_CUDA;
    alignas(64) CUtensorMap tm_k, tm_v, tm_r;
    const int N = 2 * p.tree.n - 1;
    if (!tc5::encode_tiled() || !tc5::node_rows_map(&tm_k, p.k, p.B, N, p.H) || !tc5::node_rows_map(&tm_v, p.v, p.B, N, p.H) ||
        !tc5::rel_rows_map(&tm_r, p.rel_emb, p.g->dims.n_rel))
        return BPT_ERR_CUDA;
    launch_level_ranges(p.tree, n_left, n_right, ranges, p.stream);
    trace_mark(p.stream, "level_ranges");
    const dim3 grid(p.tree.n / kFTok, p.H, p.B);
    kernel<<<grid, kFThreads, smem, p.stream>>>(p.tree, n_left, n_right, ranges, (const __nv_bfloat16*)p.q, (__nv_bfloat16*)p.out, p.lse,
                                                status, p.H, p.scale * kLog2e, p.lengths, p.drop, tm_k, tm_v, tm_r);
    trace_mark(p.stream, "fwd_tc5");
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

}  // namespace bpt
