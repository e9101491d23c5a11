// Tiled forward for the token rows on the 5th-generation tensor cores (tcgen05, accumulators in
// tensor memory): arXiv 1911.04070, Sec. 3.4 equation over the contextual edges of Sec. 3.2.2,
// bf16, head size 64.
//
// One CTA = 128 consecutive tokens of one (batch entry, head) = the 128 lanes of tensor memory,
// four threads per token row (warps w, w + 4, w + 8, w + 12 read the same lane quadrant), each
// taking a quarter of the columns, plus a driver warp.  Per (side, level) chunk the union node range
// of the tile (at most 128 / 2^level + k + 2 nodes) is staged once in shared memory, and one elected
// thread issues
//     QR = Q R_chunk^T   (128 x round16(k + 2)) -- the relative-position terms of every offset
//     S  = Q K_range^T   (128 x N, N <= 208)
// into tensor memory.  The row's bias values go to a shared table indexed [offset][row], so that
// the per-row shift between node index and offset is plain address arithmetic; the part of S that
// covers the warp's rows is read into registers (8 columns of each 32-column piece per thread)
// and the row does its masked softmax update in one sweep -- the softmax code issues no
// tensor-core instruction.  P goes to shared memory as the K-major A operand of
//     O_chunk = P V_range (128 x 64),
// which each thread adds (its 16 channels) to the running output row with the usual rescale.
// The self loop is offset 0 of the level-0 left chunk, as in the tiled backward.
//
// Warp roles: sixteen softmax warps and one driver warp.  The driver's elected thread brings the K, V
// and R rows in with TMA (cp.async.bulk.tensor, 16-row boxes straight into the swizzled layout the
// tensor core reads) and issues every MMA; mbarriers carry all hand-offs (rows landed -> driver,
// S / QR done and O_chunk done -> softmax threads, scores read and P complete -> driver), so the
// softmax code has no block-wide barrier.  QR and S of the next chunk are issued as soon as every
// thread holds its part of this chunk's scores, the next K / R rows are fetched as soon as S is done
// (single buffers) and the next V rows into the other of two buffers; O_chunk is collected just
// before the next chunk's P is written.  Every mbarrier wait gives up after about a second and the
// kernel then winds down.
#include "bpt_internal.cuh"
#include "mma_tools.cuh"
#include "tc5_host.cuh"
#include "tc5_tools.cuh"
#include "tile_geom.cuh"

namespace bpt {

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kTcTokens = 128;
constexpr int kTpr = 4;                             // threads per token row
constexpr int kTcSoftmaxThreads = kTcTokens * kTpr;
constexpr int kTcThreads = kTcSoftmaxThreads + 32;  // + the driver warp (TMA and MMA issue)
constexpr int kTcKvRows = 208;    // staged K / V rows per chunk: 128 + 64 + 2 nodes, rounded up to 16
constexpr int kTcRelRows = 80;    // relation rows per chunk (k + 2 <= 66), rounded up to 16
constexpr int kTcBiasRows = 68;   // offsets kept in the bias table
constexpr int kTcPieces = 4;      // 32-column pieces of S per warp (32 rows reach <= 32 + k + 2 + 7 columns)
constexpr uint32_t kColS = 0, kColQR = 352, kColO = 432, kTmemCols = 512;  // S reads may run 127 columns past N

struct FwdTcSmem {
    static constexpr int q_off = 0;
    static constexpr int k_off = q_off + kTcTokens * 128;
    static constexpr int v_off = k_off + kTcKvRows * 128;                // two buffers
    static constexpr int r_off = v_off + 2 * kTcKvRows * 128;
    static constexpr int p_off = r_off + kTcRelRows * 128;               // 4 key blocks of [128 rows][128 B]
    static constexpr int bias_off = p_off + 4 * kTcTokens * 128;         // [68 offsets][128 rows] fp32
    static constexpr int misc_off = bias_off + kTcBiasRows * kTcTokens * 4;  // 7 mbarriers, tensor-memory slot, abort flag
    static constexpr int xch_off = misc_off + 64;                        // [kTpr][128 rows] fp32 exchange + the same of give-up flags
    static constexpr int bnd_off = xch_off + 2 * kTpr * kTcTokens * 4;          // [chunks][128] short2, then [chunks] int2
    static size_t bytes(int chunks) { return (size_t)bnd_off + (size_t)chunks * (kTcTokens * 4 + 8) + 1024; }
};
static_assert(FwdTcSmem::k_off % 1024 == 0 && FwdTcSmem::v_off % 1024 == 0 && FwdTcSmem::r_off % 1024 == 0 &&
              FwdTcSmem::p_off % 1024 == 0 && (kTcKvRows * 128) % 1024 == 0, "swizzled tiles start on 1024-byte boundaries");

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// barrier of the kTpr warps that share a lane quadrant (ids 1..4; id 0 is __syncthreads)
__device__ __forceinline__ void quad_barrier(int quad) {
    switch (quad) {
        case 0: asm volatile("bar.sync 1, %0;" ::"n"(32 * kTpr) : "memory"); break;
        case 1: asm volatile("bar.sync 2, %0;" ::"n"(32 * kTpr) : "memory"); break;
        case 2: asm volatile("bar.sync 3, %0;" ::"n"(32 * kTpr) : "memory"); break;
        default: asm volatile("bar.sync 4, %0;" ::"n"(32 * kTpr) : "memory"); break;
    }
}

template <bool kDrop>  // attention dropout compiled in or out
__global__ void __launch_bounds__(kTcThreads, 1)
fwd_tc5_kernel(TreeParams t, int n_left, int n_right,
               const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
               const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ r,
               __nv_bfloat16* __restrict__ out, float* __restrict__ lse, int* __restrict__ status,
               int H, float scale_log2e, const int32_t* __restrict__ lengths, DropoutParams drop,
               const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_r) {
    extern __shared__ unsigned char smem_raw[];
    // the swizzle pattern is a function of the address bits, so the tiles must start 1024-aligned
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    unsigned char* q_s = smem + FwdTcSmem::q_off;
    unsigned char* p_s = smem + FwdTcSmem::p_off;
    unsigned char* r_s = smem + FwdTcSmem::r_off;
    float* bias_s = reinterpret_cast<float*>(smem + FwdTcSmem::bias_off);
    uint64_t* mbar = reinterpret_cast<uint64_t*>(smem + FwdTcSmem::misc_off);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(mbar + 7);
    volatile int* abort_s = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* xch_s = reinterpret_cast<float*>(smem + FwdTcSmem::xch_off);
    int* dead_s = reinterpret_cast<int*>(xch_s + kTpr * kTcTokens);
    short2* bnd = reinterpret_cast<short2*>(smem + FwdTcSmem::bnd_off);  // row ranges relative to the chunk's first node
    const int chunks = n_left + n_right;
    int2* crange = reinterpret_cast<int2*>(bnd + chunks * kTcTokens);

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int quad = w & 3, part = w >> 2, row = quad * 32 + lane;  // part: which share of the row's columns / channels
    const int t0 = blockIdx.x * kTcTokens, h = blockIdx.y, b = blockIdx.z;
    const int N_nodes = 2 * t.n - 1;
    const size_t rs = (size_t)H * 64;
    const size_t boff = (size_t)b * N_nodes * rs + (size_t)h * 64;
    const uint32_t q_u = smem_u32(q_s), k_u = smem_u32(smem + FwdTcSmem::k_off), v_u = smem_u32(smem + FwdTcSmem::v_off),
                   r_u = smem_u32(r_s), p_u = smem_u32(p_s);
    // S / QR done, O_chunk done, K + R rows landed, V rows landed (two buffers), P complete, S / QR read
    const uint32_t mbar_s = smem_u32(&mbar[0]), mbar_o = smem_u32(&mbar[1]), mbar_kr = smem_u32(&mbar[2]),
                   mbar_v0 = smem_u32(&mbar[3]), mbar_v1 = smem_u32(&mbar[4]), mbar_p = smem_u32(&mbar[5]),
                   mbar_r = smem_u32(&mbar[6]);

    // ---- prologue: Q tile, row ranges, barriers, tensor memory ----
    for (int idx = tid; idx < kTcTokens * 8; idx += kTcThreads) {
        const int rr = idx >> 3, ch = idx & 7;
        cp_async16(q_u + tile_off(rr, ch), q + boff + (size_t)(t0 + rr) * rs + ch * 8);
    }
    cp_async_commit();
    int2* bnd_abs = reinterpret_cast<int2*>(p_s);  // absolute ranges, only until the relative table is written
    if (tid < kTcTokens) {
        fill_row_bounds<kTcTokens>(t, t0, tid, n_left, n_right, bnd_abs);
        const int i = t0 + tid;  // the self loop joins the level-0 left range: it ends at the token itself
        const int2 v0 = bnd_abs[tid];
        bnd_abs[tid] = v0.x > v0.y ? make_int2(i, i) : make_int2(v0.x, i);
    }
    if (tid == 0) {
        tc5::mbar_init(mbar_s, 1);
        tc5::mbar_init(mbar_o, 1);
        tc5::mbar_init(mbar_kr, 1);
        tc5::mbar_init(mbar_v0, 1);
        tc5::mbar_init(mbar_v1, 1);
        tc5::mbar_init(mbar_p, kTcSoftmaxThreads);
        tc5::mbar_init(mbar_r, kTcSoftmaxThreads);
        tc5::mbar_init_fence();
        *abort_s = 0;
    }
    if (w == 0) tc5::tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    cp_async_wait<0>();
    tc5::fence_async_smem();
    tc5::fence_before_sync();
    __syncthreads();
    tc5::fence_after_sync();
    const uint32_t tbase = *tmem_slot;
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    for (int c = w; c < chunks; c += kTcThreads / 32) {
        int2 u = make_int2(0x7fffffff, -1);
#pragma unroll
        for (int part = 0; part < kTcTokens / 32; ++part) {
            const int2 a = rows_union(bnd_abs + c * kTcTokens, part * 32, 32, lane);
            u.x = min(u.x, a.x); u.y = max(u.y, a.y);
        }
        if (lane == 0) crange[c] = u;
    }
    __syncthreads();
    {   // short sequence: the staged ranges stay those of the full graph, the rows' ranges shrink
        const int len = seq_len(lengths, b, t.n);
        if (len < t.n) {
            if (tid < kTcTokens) mask_row_bounds<kTcTokens>(t, t0, tid, n_left, n_right, bnd_abs, len);
            __syncthreads();
        }
    }
    for (int idx = tid; idx < chunks * kTcTokens; idx += kTcThreads) {
        const int2 a = bnd_abs[idx];
        const int base = crange[idx / kTcTokens].x;
        bnd[idx] = a.x <= a.y ? make_short2((short)(a.x - base), (short)(a.y - base)) : make_short2(1, 0);
    }
    __syncthreads();

    auto geom = [&](int c, int& level, int& side, int& base, int& n_cols) {
        const int2 cr = crange[c];
        side = c >= n_left;
        level = side ? c - n_left : c;
        base = cr.x;
        n_cols = (cr.y - cr.x + 1 + 15) & ~15;
    };
    const int rel_cols = (t.k + 2 + 15) & ~15;  // relation rows (offsets) a chunk can use, in whole 16-row boxes
    auto next_chunk = [&](int c) {  // next chunk this tile reaches
        int cn = c + 1;
        while (cn < chunks && crange[cn].x > crange[cn].y) ++cn;
        return cn;
    };

    if (w == kTcSoftmaxThreads / 32) {
        // =============== driver: one thread moves the tiles (TMA) and issues every MMA ===============
        if (lane == 0) {
            // K and R rows of chunk c (16 rows per copy; rows past the range are real rows of later
            // nodes / relations or, past the end of the tensor, zeros: finite either way)
            auto load_kr = [&](int c) {
                int level, side, base, n_cols;
                geom(c, level, side, base, n_cols);
                const int node0 = node_id(t.n, level, 0) + base;
                const int rel_base = c == 0 ? 0 : (side ? rel_right(t, level, 0) : rel_left(t, level, 0));
                tc5::mbar_expect_tx(mbar_kr, (uint32_t)(n_cols / 16 + rel_cols / 16) * 2048u);
                for (int j = 0; j < n_cols / 16; ++j) tc5::tma_load_4d(k_u + j * 2048, &tm_k, 0, h, node0 + 16 * j, b, mbar_kr);
                for (int j = 0; j < rel_cols / 16; ++j) tc5::tma_load_2d(r_u + j * 2048, &tm_r, 0, rel_base + 16 * j, mbar_kr);
            };
            auto load_v = [&](int c, int buf) {
                int level, side, base, n_cols;
                geom(c, level, side, base, n_cols);
                const int node0 = node_id(t.n, level, 0) + base;
                const uint32_t bar = buf ? mbar_v1 : mbar_v0;
                tc5::mbar_expect_tx(bar, (uint32_t)(n_cols / 16) * 2048u);
                for (int j = 0; j < n_cols / 16; ++j)
                    tc5::tma_load_4d(v_u + buf * (kTcKvRows * 128) + j * 2048, &tm_v, 0, h, node0 + 16 * j, b, bar);
            };
            auto issue_s = [&](int c) {  // QR and S of chunk c
                int level, side, base, n_cols;
                geom(c, level, side, base, n_cols);
                const uint32_t id_qr = tc5::instr_desc(kTcTokens, rel_cols, 0, 0), id_s = tc5::instr_desc(kTcTokens, n_cols, 0, 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    tc5::mma(tbase + kColQR, tc5::desc_k_major(q_u + ks * 32), tc5::desc_k_major(r_u + ks * 32), id_qr, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    tc5::mma(tbase + kColS, tc5::desc_k_major(q_u + ks * 32), tc5::desc_k_major(k_u + ks * 32), id_s, ks > 0);
                tc5::commit(mbar_s);
            };
            uint32_t ph_kr = 0, ph_v[2] = {0, 0}, ph_p = 0, ph_s = 0, ph_o = 0, ph_r = 0;
            bool ok = true;
            load_kr(0);  // chunk 0 (left level 0 with the self loop) is never empty
            load_v(0, 0);
            ok = tc5::mbar_wait(mbar_kr, ph_kr); ph_kr ^= 1;
            tc5::fence_after_sync();
            if (ok) issue_s(0);
            int c = 0, it = 0;
            while (ok && c < chunks && !*abort_s) {
                int level, side, base, n_cols;
                geom(c, level, side, base, n_cols);
                const int cn = next_chunk(c);
                ok = tc5::mbar_wait(mbar_s, ph_s); ph_s ^= 1;         // S, QR done: K and R buffers are free
                if (ok && cn < chunks) load_kr(cn);
                if (ok && cn < chunks) {
                    // S and QR of the next chunk as soon as every thread holds its part of this chunk's S and QR
                    ok = tc5::mbar_wait(mbar_r, ph_r); ph_r ^= 1;
                    if (ok) { ok = tc5::mbar_wait(mbar_kr, ph_kr); ph_kr ^= 1; }
                    if (ok) { tc5::fence_after_sync(); issue_s(cn); }
                }
                if (ok && it > 0) { ok = tc5::mbar_wait(mbar_o, ph_o); ph_o ^= 1; }  // O_chunk of the chunk before: other V buffer free
                if (ok && cn < chunks) load_v(cn, (it + 1) & 1);
                if (ok) { ok = tc5::mbar_wait(mbar_p, ph_p); ph_p ^= 1; }            // P complete, O_chunk has been read
                if (ok) { ok = tc5::mbar_wait((it & 1) ? mbar_v1 : mbar_v0, ph_v[it & 1]); ph_v[it & 1] ^= 1; }
                if (!ok) break;
                tc5::fence_after_sync();
                const uint32_t id_o = tc5::instr_desc(kTcTokens, 64, 0, 1);
                const uint32_t vb_u = v_u + (it & 1) * (kTcKvRows * 128);
                for (int kk = 0; kk < (n_cols >> 4); ++kk)
                    tc5::mma(tbase + kColO, tc5::desc_k_major(p_u + (kk >> 2) * (kTcTokens * 128) + (kk & 3) * 32),
                             tc5::desc_mn_major(vb_u + kk * 2048), id_o, kk > 0);
                tc5::commit(mbar_o);
                c = cn;
                ++it;
            }
            if (!ok) *abort_s = 1;
        }
    } else {
        // =============== softmax: two threads per token row ===============
        constexpr int kCols = 32 / kTpr, kChan = 64 / kTpr;  // columns per 32-column piece and output channels of one thread
        float m_run = -INFINITY, l_run = 0.f, corr_prev = 1.f, o[kChan];
#pragma unroll
        for (int j = 0; j < kChan; ++j) o[j] = 0.f;
        uint32_t ph_s = 0, ph_o = 0;
        bool o_pending = false;
        // O_chunk of the previous chunk -> running output (rescaled by that chunk's correction)
        auto collect_o = [&]() {
            if (!tc5::mbar_wait(mbar_o, ph_o)) *abort_s = 1;
            ph_o ^= 1;
            tc5::fence_after_sync();
            uint32_t x[kChan];
            tc5::tmem_ld16(tbase + lane_base + kColO + part * kChan, x);
            tc5::tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < kChan; ++j) o[j] = fmaf(o[j], corr_prev, __uint_as_float(x[j]));
        };

        int c = 0;
        while (c < chunks) {
            int level, side, base, n_cols;
            geom(c, level, side, base, n_cols);
            if (!tc5::mbar_wait(mbar_s, ph_s)) *abort_s = 1;  // S and QR of this chunk are in tensor memory
            ph_s ^= 1;
            tc5::fence_after_sync();
            const int dead = *abort_s;   // some wait gave up: leave, but together with the row's other thread (below)

            // ---- bias row -> table [offset][row]; the threads of a row share the offsets ----
            {
                uint32_t x[16];
                if (part * 16 < rel_cols) {  // the same for the whole warp
                    tc5::tmem_ld16(tbase + lane_base + kColQR + part * 16, x);
                    tc5::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) bias_s[(part * 16 + j) * kTcTokens + row] = __uint_as_float(x[j]) * scale_log2e;
                }
                if (part == 0 && rel_cols > 64) {  // offsets 64 .. 67 (k + 2 <= 66 are used)
                    tc5::tmem_ld16(tbase + lane_base + kColQR + 64, x);
                    tc5::tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < kTcBiasRows - 64; ++j) bias_s[(64 + j) * kTcTokens + row] = __uint_as_float(x[j]) * scale_log2e;
                }
            }

            // ---- this thread's share of the row's part of S ----
            const short2 my = bnd[c * kTcTokens + row];
            int wlo = my.x <= my.y ? my.x : 0x7fff, whi = my.x <= my.y ? my.y : -1;
#pragma unroll
            for (int sh = 16; sh > 0; sh >>= 1) {
                wlo = min(wlo, __shfl_xor_sync(0xffffffffu, wlo, sh));
                whi = max(whi, __shfl_xor_sync(0xffffffffu, whi, sh));
            }
            const bool w_any = wlo <= whi;
            const int c0 = w_any ? (wlo & ~7) : 0;
            const int npieces = w_any ? min(kTcPieces, ((whi - c0) >> 5) + 1) : 0;
            uint32_t sv[kTcPieces][kCols];
#pragma unroll
            for (int p = 0; p < kTcPieces; ++p)
                if (p < npieces) tc5::tmem_ld8(tbase + lane_base + kColS + c0 + p * 32 + part * kCols, sv[p]);
            tc5::tmem_ld_wait();
            tc5::fence_before_sync();
            tc5::mbar_arrive(mbar_r);  // this thread holds its part of S and QR: the driver may overwrite them
            quad_barrier(quad);        // the row's bias values are all in the table

            const int cnt = max(my.y - my.x + 1, 0);
            const int a = my.x - c0 - part * kCols;  // column, relative to this thread's first one, of the row's first node
            // offset of column e: right side e - a, left side (cnt - 1) - (e - a): one pointer and a signed stride
            const int sgn = side ? kTcTokens : -kTcTokens;
            const float* bptr = bias_s + row + (side ? -a : (cnt - 1 + a)) * kTcTokens;
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};  // independent chains
#pragma unroll
            for (int p = 0; p < kTcPieces; ++p) {
                if (p < npieces) {
#pragma unroll
                    for (int j = 0; j < kCols; ++j) {
                        const int e = p * 32 + j;
                        const bool in = (unsigned)(e - a) < (unsigned)cnt;
                        float val = -INFINITY;
                        if (in) val = fmaf(__uint_as_float(sv[p][j]), scale_log2e, bptr[e * sgn]);
                        sv[p][j] = __float_as_uint(val);
                        mx4[j & 3] = fmaxf(mx4[j & 3], val);
                    }
                }
            }
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            xch_s[part * kTcTokens + row] = mx;
            dead_s[part * kTcTokens + row] = dead;
            quad_barrier(quad);
            // the threads of a lane quadrant share barriers and warp-wide loads: they leave as one
            int dead_row = 0;
            float mx_row = -INFINITY;
#pragma unroll
            for (int x = 0; x < kTpr; ++x) {
                dead_row |= dead_s[x * kTcTokens + row];
                mx_row = fmaxf(mx_row, xch_s[x * kTcTokens + row]);
            }
            if (__any_sync(0xffffffffu, dead_row)) break;
            const float m_new = fmaxf(m_run, mx_row);
            const float m_ref = m_new == -INFINITY ? 0.f : m_new;
            const float corr = ex2(m_run - m_ref);
            m_run = m_new;
            if (o_pending) collect_o();  // O_chunk of the chunk before; the P tile is free after it
            float l4[4] = {0.f, 0.f, 0.f, 0.f};
            const int ch0 = c0 >> 3, n_ch = n_cols >> 3;
#pragma unroll
            for (int p = 0; p < kTcPieces; ++p) {
                if (p < npieces) {
                    uint32_t pk[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        float p0 = ex2(__uint_as_float(sv[p][2 * x]) - m_ref);
                        float p1 = ex2(__uint_as_float(sv[p][2 * x + 1]) - m_ref);
                        l4[x] += p0 + p1;
                        if constexpr (kDrop) {  // the weights that reach V are dropped, the softmax sum is not
                            const uint32_t src = (uint32_t)(node_id(t.n, level, 0) + base + c0 + p * 32 + part * kCols + 2 * x);
                            p0 *= dropout_weight(drop, (uint32_t)(b * H + h), (uint32_t)(t0 + row), src);
                            p1 *= dropout_weight(drop, (uint32_t)(b * H + h), (uint32_t)(t0 + row), src + 1);
                        }
                        pk[x] = pack_bf16(p0, p1);
                    }
                    const int ci = ch0 + p * 4 + part;  // 16-byte chunk (8 keys) of the P row
                    if (ci < n_ch)
                        *reinterpret_cast<uint4*>(p_s + (ci >> 3) * (kTcTokens * 128) + tile_off(row, ci & 7)) =
                            make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            }
            l_run = fmaf(l_run, corr, (l4[0] + l4[1]) + (l4[2] + l4[3]));
            corr_prev = corr;
            for (int ci = part; ci < n_ch; ci += kTpr)  // the rest of the row is zero (the row's threads take chunks in turn)
                if (ci < ch0 || ci >= ch0 + npieces * 4)
                    *reinterpret_cast<uint4*>(p_s + (ci >> 3) * (kTcTokens * 128) + tile_off(row, ci & 7)) = make_uint4(0, 0, 0, 0);

            tc5::fence_async_smem();   // P was written with ordinary stores and is read by the tensor core
            tc5::fence_before_sync();
            tc5::mbar_arrive(mbar_p);  // this thread's part of P is in place and its tensor-memory reads are done
            o_pending = true;
            c = next_chunk(c);
        }
        if (o_pending && !*abort_s) collect_o();

        // ---- row sums of the row's threads, normalise, round once to bf16 into the Q tile ----
        xch_s[part * kTcTokens + row] = l_run;
        quad_barrier(quad);
        float l_all = 0.f;
#pragma unroll
        for (int x = 0; x < kTpr; ++x) l_all += xch_s[x * kTcTokens + row];
        const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
#pragma unroll
        for (int ch = 0; ch < kChan / 8; ++ch) {
            uint32_t pk[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) pk[x] = pack_bf16(o[ch * 8 + 2 * x] * inv, o[ch * 8 + 2 * x + 1] * inv);
            *reinterpret_cast<uint4*>(q_s + tile_off(row, part * (kChan / 8) + ch)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
        if (part == 0) lse[((size_t)b * N_nodes + t0 + row) * H + h] = l_all > 0.f ? (m_run + log2f(l_all)) * kLn2 : 0.f;
    }

    // ---- epilogue: coalesced stores of the output tile; tensor memory back ----
    tc5::fence_before_sync();
    __syncthreads();
    for (int idx = tid; idx < kTcTokens * 8; idx += kTcThreads) {
        const int rr = idx >> 3, ch = idx & 7;
        *reinterpret_cast<uint4*>(out + boff + (size_t)(t0 + rr) * rs + ch * 8) =
            *reinterpret_cast<const uint4*>(q_s + tile_off(rr, ch));
    }
    if (tid == 0 && *abort_s && status) status[0] = (int)BPT_ERR_TIMEOUT;
    if (w == 0) tc5::tmem_free(tbase, kTmemCols);
}

}  // namespace

// The tensor-memory kernel takes whole tiles of 128 tokens.
bool fwd_tc5_eligible(const AttnProblem& p) {
    if (!tc5::encode_tiled()) return false;
    if (!tile_path(p.tree.n, p.tree.k, p.d, p.dtype == BPT_BF16) || p.tree.n < kTcTokens) return false;
    int n_left, n_right;
    context_levels(p.tree, &n_left, &n_right);
    return FwdTcSmem::bytes(n_left + n_right) <= 227 * 1024;
}

// Token rows of the forward; `status` is a device word that receives BPT_ERR_TIMEOUT when a wait gave up.
bpt_status launch_fwd_tc5(const AttnProblem& p, int* status) {
    int n_left, n_right;
    context_levels(p.tree, &n_left, &n_right);
    const size_t smem = FwdTcSmem::bytes(n_left + n_right);
    if (smem > 227 * 1024 || p.H > 65535 || p.B > 65535) return BPT_ERR_UNSUPPORTED;
    auto kernel = p.drop.thr ? fwd_tc5_kernel<true> : fwd_tc5_kernel<false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return BPT_ERR_CUDA;
    alignas(64) CUtensorMap tm_k, tm_v, tm_r;
    const int N = 2 * p.tree.n - 1;
    if (!tc5::encode_tiled() || !tc5::node_rows_map(&tm_k, p.k, p.B, N, p.H) || !tc5::node_rows_map(&tm_v, p.v, p.B, N, p.H) ||
        !tc5::rel_rows_map(&tm_r, p.rel_emb, p.g->dims.n_rel))
        return BPT_ERR_CUDA;
    const dim3 grid(p.tree.n / kTcTokens, p.H, p.B);
    kernel<<<grid, kTcThreads, smem, p.stream>>>(p.tree, n_left, n_right, (const __nv_bfloat16*)p.q,
                                                 (const __nv_bfloat16*)p.k, (const __nv_bfloat16*)p.v,
                                                 (const __nv_bfloat16*)p.rel_emb, (__nv_bfloat16*)p.out, p.lse,
                                                 status, p.H, p.scale * kLog2e, p.lengths, p.drop, tm_k, tm_v, tm_r);
    trace_mark(p.stream, "fwd_tc5");
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

}  // namespace bpt
