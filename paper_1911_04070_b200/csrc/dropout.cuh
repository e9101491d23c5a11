// Attention dropout (arXiv 1911.04070, App. A.1 lists an attention dropout rate for every experiment;
// how the masks are drawn is this library's choice): every edge weight of every (batch entry, head)
// is kept with probability 1 - p and divided by 1 - p, after the softmax and before the product
// with V.  The mask is a pure function of (seed, batch entry, head, destination node, source node),
// so the backward pass rebuilds it instead of storing it: Philox4x32 with 10 rounds (Salmon et al.,
// "Parallel random numbers: as easy as 1, 2, 3", SC'11), key = the two halves of the seed, counter =
// (destination, source, batch entry * H + head, tag); the edge is kept iff the first output word
// is >= floor(p * 2^32).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace bpt {

struct DropoutParams {
    uint32_t thr;     // floor(p * 2^32); 0 = no dropout (nothing is drawn)
    float inv_keep;   // 1 / (1 - p)
    uint32_t k0, k1;  // seed halves
};

inline DropoutParams make_dropout(float p, uint64_t seed) {
    DropoutParams d{0u, 1.f, (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
    if (p > 0.f) {
        double t = (double)p * 4294967296.0;
        t = t < 4294967295.0 ? t : 4294967295.0;
        d.thr = (uint32_t)t;
        d.inv_keep = (float)(1.0 / (1.0 - (double)p));
    }
    return d;
}

// keep / (1 - p) of the edge src -> dst for (batch entry, head) pair index bh
__device__ __forceinline__ float dropout_weight(const DropoutParams& d, uint32_t bh, uint32_t dst, uint32_t src) {
    uint32_t c0 = dst, c1 = src, c2 = bh, c3 = 0x42505431u, k0 = d.k0, k1 = d.k1;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0; c1 = lo1;
        c2 = hi0 ^ c3 ^ k1; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return c0 >= d.thr ? d.inv_keep : 0.f;
}

}  // namespace bpt
