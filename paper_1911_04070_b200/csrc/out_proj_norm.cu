// Output projection, residual and layer normalisation of a BP-Transformer layer in one kernel
// (arXiv 1911.04070, Algorithm 2 of Sec. 3.3: Z = norm(H + GSA(H) W^O) with the W^O of Sec. 3.1):
//     z = LayerNorm(h + a w_o^T) * gamma + beta,   row by row,
// a = the attention output with the heads concatenated.  bf16 in and out, fp32 accumulation and statistics.
//
// One CTA = 128 rows = the 128 lanes of tensor memory; the whole output row (D <= 512 channels) stays in
// tensor memory as fp32, so the residual add and both normalisation passes run on it without a trip through
// HBM.  A load thread brings a [128 x 64] and w_o [D x 64] k-blocks in with TMA (two stages, each CTA its own copies), an
// MMA thread issues tcgen05.mma (N = min(D, 256) columns per instruction), sixteen epilogue warps (four threads
// per row, a quarter of the columns each; the row statistics pass between them through shared memory) add the
// residual into tensor memory, take mean and variance in two further sweeps, normalise, and stage the bf16 rows in
// shared memory for coalesced stores.  Every wait is bounded; a give-up is reported through the status word.
#include "bpt_internal.cuh"
#include "mma_tools.cuh"
#include "tc5_host.cuh"
#include "tc5_tools.cuh"

namespace bpt {

namespace {

constexpr int kOpRows = 128;
constexpr int kOpTpr = 4;                              // epilogue threads per row
constexpr int kOpEpiWarps = 4 * kOpTpr;
constexpr int kOpThreads = (kOpEpiWarps + 2) * 32;     // epilogue warps, a load warp, an MMA warp
constexpr int kOpStages = 2;
constexpr int kOpMaxD = 512;

struct OpSmem {   // byte offsets for a given D
    int a_bytes, w_bytes, stage_bytes, bar_off, out_stride;
    size_t bytes;
};
inline OpSmem op_smem(int D) {
    OpSmem s;
    s.a_bytes = kOpRows * 128;
    s.w_bytes = D * 128;
    s.stage_bytes = s.a_bytes + s.w_bytes;
    s.bar_off = kOpStages * s.stage_bytes;      // the output staging ([128][D] bf16, padded rows) reuses the stages
    s.out_stride = D * 2 + 16;
    const int staging = kOpRows * s.out_stride;
    if (s.bar_off < staging) s.bar_off = (staging + 1023) & ~1023;
    s.bytes = (size_t)s.bar_off + 128 + kOpTpr * kOpRows * 4 + 1024;   // barriers, then the exchange of row statistics
    return s;
}

__global__ void __launch_bounds__(kOpThreads, 1)
out_proj_norm_kernel(const __nv_bfloat16* __restrict__ h, const float* __restrict__ gamma, const float* __restrict__ beta,
                     __nv_bfloat16* __restrict__ z, int* __restrict__ status, long long rows, int D, float eps, OpSmem cfg,
                     const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + cfg.bar_off);   // full[2], empty[2], done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
    volatile int* abort_s = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* xch_s = reinterpret_cast<float*>(smem + cfg.bar_off + 128);   // [kOpTpr][128 rows]
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const long long row0 = (long long)blockIdx.x * kOpRows;
    const uint32_t s_u = smem_u32(smem), bar_u = smem_u32(bars);
    auto bar = [&](int i) { return bar_u + 8u * (uint32_t)i; };
    auto wait = [&](int i, uint32_t parity) {
        if (*abort_s) return;
        if (!tc5::mbar_wait_fast(bar(i), parity)) *abort_s = 1;
    };
    const int n_kb = D / 64;
    const uint32_t tmem_cols = D <= 128 ? 128u : (D <= 256 ? 256u : 512u);

    if (tid == 0) {
        for (int i = 0; i < 5; ++i) tc5::mbar_init(bar(i), 1);
        tc5::mbar_init_fence();
        *abort_s = 0;
    }
    if (w == 0) tc5::tmem_alloc(smem_u32(tmem_slot), tmem_cols);
    tc5::fence_before_sync();
    __syncthreads();
    tc5::fence_after_sync();
    const uint32_t tbase = *tmem_slot;

    if (w == kOpEpiWarps) {
        // =============== load warp: k-blocks of a and w_o, two stages ===============
        if (lane == 0) {
            for (int kb = 0; kb < n_kb && !*abort_s; ++kb) {
                const int st = kb % kOpStages, use = kb / kOpStages;
                if (use > 0) wait(2 + st, (use - 1) & 1);
                const uint32_t dst = s_u + st * cfg.stage_bytes;
                tc5::mbar_expect_tx(bar(st), (uint32_t)cfg.stage_bytes);
                tc5::tma_load_2d(dst, &tm_a, kb * 64, (int)row0, bar(st));                       // rows past the end read as zeros
                for (int nb = 0; nb < D; nb += 128)
                    tc5::tma_load_2d(dst + cfg.a_bytes + nb * 128, &tm_w, kb * 64, nb, bar(st));
            }
        }
    } else if (w == kOpEpiWarps + 1) {
        // =============== MMA warp: acc[128 x D] += a_kb w_kb^T ===============
        if (lane == 0) {
            const int n_half = D > 256 ? 2 : 1, n_cols = D > 256 ? 256 : D;
            const uint32_t idesc = tc5::instr_desc(kOpRows, n_cols, 0, 0);
            for (int kb = 0; kb < n_kb && !*abort_s; ++kb) {
                const int st = kb % kOpStages, use = kb / kOpStages;
                wait(st, use & 1);
                if (*abort_s) break;
                tc5::fence_after_sync();
                const uint32_t a_lo = tc5::desc_lo_k_major(s_u + st * cfg.stage_bytes);
                const uint32_t w_lo = tc5::desc_lo_k_major(s_u + st * cfg.stage_bytes + cfg.a_bytes);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    for (int nh = 0; nh < n_half; ++nh)
                        tc5::mma_lo(tbase + nh * 256, a_lo + ks * 2, w_lo + nh * (256 * 128 / 16) + ks * 2, idesc, (kb > 0 || ks > 0) ? 1u : 0u);
                tc5::commit(bar(2 + st));
            }
            tc5::commit(bar(4));
        }
    } else {
        // =============== epilogue warps: four threads per row, D / 4 consecutive columns each ===============
        const int quad = w & 3, part = w >> 2;
        const int r = quad * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const long long row = row0 + r;
        const bool live = row < rows;
        const int c_lo = part * (D / kOpTpr), c_hi = c_lo + D / kOpTpr;
        auto row_sum = [&](float v) {   // sum over the row's threads (the warps that share a lane quadrant)
            xch_s[part * kOpRows + r] = v;
            switch (quad) {
                case 0: asm volatile("bar.sync 1, %0;" ::"n"(32 * kOpTpr) : "memory"); break;
                case 1: asm volatile("bar.sync 2, %0;" ::"n"(32 * kOpTpr) : "memory"); break;
                case 2: asm volatile("bar.sync 3, %0;" ::"n"(32 * kOpTpr) : "memory"); break;
                default: asm volatile("bar.sync 4, %0;" ::"n"(32 * kOpTpr) : "memory"); break;
            }
            float t = 0.f;
#pragma unroll
            for (int x = 0; x < kOpTpr; ++x) t += xch_s[x * kOpRows + r];
            return t;
        };
        auto quad_sync = [&]() {        // before the exchange slots are written again
            switch (quad) {
                case 0: asm volatile("bar.sync 1, %0;" ::"n"(32 * kOpTpr) : "memory"); break;
                case 1: asm volatile("bar.sync 2, %0;" ::"n"(32 * kOpTpr) : "memory"); break;
                case 2: asm volatile("bar.sync 3, %0;" ::"n"(32 * kOpTpr) : "memory"); break;
                default: asm volatile("bar.sync 4, %0;" ::"n"(32 * kOpTpr) : "memory"); break;
            }
        };
        wait(4, 0);
        tc5::fence_after_sync();
        const uint4* hrow = reinterpret_cast<const uint4*>(h + (live ? row : 0) * (long long)D);
        // sweep 1: x = acc + h back into tensor memory, and the row sum
        float sum = 0.f;
        for (int c = c_lo; c < c_hi; c += 32) {
            uint32_t x[32];
            tc5::tmem_ld32(tbase + lane_base + c, x);
            uint4 hv[4];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) hv[q4] = live ? __ldg(hrow + (c >> 3) + q4) : make_uint4(0, 0, 0, 0);
            tc5::tmem_ld_wait();
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                const uint32_t hw[4] = {hv[q4].x, hv[q4].y, hv[q4].z, hv[q4].w};
#pragma unroll
                for (int y = 0; y < 4; ++y) {
                    const float v0 = __uint_as_float(x[q4 * 8 + 2 * y]) + __uint_as_float(hw[y] << 16);
                    const float v1 = __uint_as_float(x[q4 * 8 + 2 * y + 1]) + __uint_as_float(hw[y] & 0xffff0000u);
                    x[q4 * 8 + 2 * y] = __float_as_uint(v0);
                    x[q4 * 8 + 2 * y + 1] = __float_as_uint(v1);
                    sum += v0 + v1;
                }
            }
            tc5::tmem_st32(tbase + lane_base + c, x);
        }
        tc5::tmem_st_wait();
        const float mean = row_sum(sum) / (float)D;
        // sweep 2: the variance about the mean
        float ssq = 0.f;
        for (int c = c_lo; c < c_hi; c += 32) {
            uint32_t x[32];
            tc5::tmem_ld32(tbase + lane_base + c, x);
            tc5::tmem_ld_wait();
#pragma unroll
            for (int y = 0; y < 32; ++y) { const float d = __uint_as_float(x[y]) - mean; ssq = fmaf(d, d, ssq); }
        }
        quad_sync();   // every thread of the row has read the sums
        const float rstd = rsqrtf(row_sum(ssq) / (float)D + eps);
        // the stage buffers are free (every product has completed): stage the normalised rows there
        unsigned char* orow = smem + (size_t)r * cfg.out_stride;
        for (int c = c_lo; c < c_hi; c += 32) {
            uint32_t x[32];
            tc5::tmem_ld32(tbase + lane_base + c, x);
            tc5::tmem_ld_wait();
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                uint32_t pk[4];
#pragma unroll
                for (int y = 0; y < 4; ++y) {
                    const int ch = c + q4 * 8 + 2 * y;
                    const float v0 = (__uint_as_float(x[q4 * 8 + 2 * y]) - mean) * rstd * __ldg(gamma + ch) + __ldg(beta + ch);
                    const float v1 = (__uint_as_float(x[q4 * 8 + 2 * y + 1]) - mean) * rstd * __ldg(gamma + ch + 1) + __ldg(beta + ch + 1);
                    pk[y] = pack_bf16(v0, v1);
                }
                *reinterpret_cast<uint4*>(orow + (c + q4 * 8) * 2) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
        }
    }

    tc5::fence_before_sync();
    __syncthreads();
    // coalesced stores of the staged rows
    const int chunks_per_row = D / 8;
    for (int idx = tid; idx < kOpRows * chunks_per_row; idx += kOpThreads) {
        const int rr = idx / chunks_per_row, ch = idx % chunks_per_row;
        if (row0 + rr < rows)
            *reinterpret_cast<uint4*>(z + (row0 + rr) * (long long)D + ch * 8) =
                *reinterpret_cast<const uint4*>(smem + (size_t)rr * cfg.out_stride + ch * 16);
    }
    if (tid == 0 && *abort_s && status) status[0] = (int)BPT_ERR_TIMEOUT;
    if (w == 0) tc5::tmem_free(tbase, tmem_cols);
}

// 2-D map over a row-major [n_rows, D] bf16 matrix; a box is `box_rows` rows of 64 elements, 128-byte swizzle.
bool matrix_map(CUtensorMap* m, const void* base, long long n_rows, int D, int box_rows) {
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)n_rows};
    const cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows}, estr[2] = {1, 1};
    return tc5::encode_tiled()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace
}  // namespace bpt

using namespace bpt;

extern "C" bpt_status bpt_out_proj_norm(const void* a, const void* w_o, const void* h, const float* gamma, const float* beta,
                                        void* z, int64_t rows, int32_t D, float eps, void* status_word, void* cuda_stream) {
    if (!a || !w_o || !h || !gamma || !beta || !z || rows < 1 || !(eps > 0.f)) return BPT_ERR_INVALID_ARG;
    if (D != 128 && D != 256 && D != 512) return BPT_ERR_UNSUPPORTED;
    if (rows > 0x7fffffffll) return BPT_ERR_UNSUPPORTED;
    if (((uintptr_t)a | (uintptr_t)w_o | (uintptr_t)h | (uintptr_t)z) & 15) return BPT_ERR_INVALID_ARG;
    if (!tc5::encode_tiled()) return BPT_ERR_CUDA;
    const OpSmem cfg = op_smem(D);
    if (cudaFuncSetAttribute(out_proj_norm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cfg.bytes) != cudaSuccess)
        return BPT_ERR_CUDA;
    alignas(64) CUtensorMap tm_a, tm_w;
    if (!matrix_map(&tm_a, a, rows, D, kOpRows) || !matrix_map(&tm_w, w_o, D, D, 128)) return BPT_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (status_word && cudaMemsetAsync(status_word, 0, 256, st) != cudaSuccess) return BPT_ERR_CUDA;
    const unsigned grid = (unsigned)((rows + kOpRows - 1) / kOpRows);
    out_proj_norm_kernel<<<grid, kOpThreads, cfg.bytes, st>>>((const __nv_bfloat16*)h, gamma, beta, (__nv_bfloat16*)z,
                                                              (int*)status_word, (long long)rows, D, eps, cfg, tm_a, tm_w);
    trace_mark(st, "out_proj_norm");
    return cudaGetLastError() == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}
