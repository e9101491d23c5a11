/*
 * Plain-C twin of oracle/bpt_oracle.py -- TEST INFRASTRUCTURE ONLY.
 *
 * The same definitions (arXiv 1911.04070, Sec. 3.2 graph construction with the
 * parity pad rule / Algorithm 1, Sec. 3.4 relation labels, Sec. 3.1 + 3.4 graph
 * self-attention and its analytic gradient), written edge by edge in fp64 so
 * that sizes too large for the NumPy version can still be checked and timed.
 * OpenMP runs independent (batch, head) pairs on separate threads; nothing is
 * blocked, fused or reordered beyond that.  It shares no code with the CUDA
 * library and is pinned against the NumPy oracle by tests/test_oracle_ctwin.py.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC bpt_oracle_c.c -o libbpt_oracle.so -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_LEFT_ONLY 1u
#define ORC_MODE_ALG1 2u

static int ilog2(int64_t n) { int l = 0; while ((1ll << l) < n) ++l; return l; }
static int64_t nid(int64_t n, int l, int64_t m) { return 2 * n - ((2 * n) >> l) + m; }

int orc_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* One token's row, sources ascending by node id.  With col == NULL it only counts. */
static int64_t token_row(int64_t n, int64_t k, uint32_t flags, int64_t i, int32_t* col, int32_t* rel) {
    const int L = ilog2(n);
    const int pad = !(flags & ORC_MODE_ALG1);
    const int64_t W = k + 1;
    /* first walk both sides to find, per level, the node range on that side */
    int64_t llo[64], lhi[64], rlo[64], rhi[64];
    int nl = 0, nr = 0;
    {   /* left: nodes last..q at each level, nearest (q) joins first */
        int64_t q = i - 1; int l = 0;
        while (q >= 0) {
            int64_t last = q - k + 1;
            if (pad && (last & 1)) last -= 1;
            if (last < 0) last = 0;
            llo[l] = last; lhi[l] = q; nl = l + 1;
            int64_t nxt = last - 1;
            if (nxt < 0) break;
            q = nxt >> 1; ++l;
        }
    }
    if (!(flags & ORC_LEFT_ONLY)) {
        int64_t p = i + 1; int l = 0;
        while (p < (n >> l)) {
            int64_t last = p + k - 1;
            if (pad && !(last & 1)) last += 1;
            if (last > (n >> l) - 1) last = (n >> l) - 1;
            rlo[l] = p; rhi[l] = last; nr = l + 1;
            int64_t nxt = last + 1;
            if (nxt >= (n >> l)) break;
            p = nxt >> 1; ++l;
        }
    }
    int64_t c = 0;
    int top = nl > nr ? nl : nr;
    if (top < 1) top = 1;
    for (int l = 0; l < top; ++l) {
        if (l < nl)
            for (int64_t m = llo[l]; m <= lhi[l]; ++m, ++c)
                if (col) { col[c] = (int32_t)nid(n, l, m); rel[c] = (int32_t)(1 + l * W + (lhi[l] - m)); }
        if (l == 0) { if (col) { col[c] = (int32_t)i; rel[c] = 0; } ++c; }
        if (l < nr)
            for (int64_t m = rlo[l]; m <= rhi[l]; ++m, ++c)
                if (col) { col[c] = (int32_t)nid(n, l, m); rel[c] = (int32_t)(1 + L * W + l * W + (m - rlo[l])); }
    }
    return c;
}

/* Number of edges of the whole graph. */
int64_t orc_count_edges(int64_t n, int64_t k, uint32_t flags) {
    int64_t e = 0;
    for (int64_t i = 0; i < n; ++i) e += token_row(n, k, flags, i, NULL, NULL);
    return e + n * ilog2(n);
}

/* CSR by destination; row_ptr has 2n entries, col/rel have orc_count_edges entries. */
void orc_build_csr(int64_t n, int64_t k, uint32_t flags, int32_t* row_ptr, int32_t* col, int32_t* rel) {
    const int L = ilog2(n);
    const int64_t W = k + 1;
    int64_t e = 0;
    for (int64_t i = 0; i < n; ++i) {
        row_ptr[i] = (int32_t)e;
        e += token_row(n, k, flags, i, col + e, rel + e);
    }
    for (int l = 1; l <= L; ++l)
        for (int64_t m = 0; m < (n >> l); ++m) {
            row_ptr[nid(n, l, m)] = (int32_t)e;
            for (int64_t t = m << l; t < ((m + 1) << l); ++t, ++e) {
                col[e] = (int32_t)t;
                rel[e] = (int32_t)(1 + 2 * L * W + (l - 1));
            }
        }
    row_ptr[2 * n - 1] = (int32_t)e;
}

/* By-source transpose: counting sort of the CSR by source, destinations ascending. */
void orc_transpose(int64_t n_nodes, const int32_t* row_ptr, const int32_t* col,
                   int32_t* t_ptr, int32_t* t_dst, int32_t* t_eid) {
    const int64_t E = row_ptr[n_nodes];
    memset(t_ptr, 0, sizeof(int32_t) * (size_t)(n_nodes + 1));
    for (int64_t e = 0; e < E; ++e) t_ptr[col[e] + 1]++;
    for (int64_t v = 0; v < n_nodes; ++v) t_ptr[v + 1] += t_ptr[v];
    int32_t* fill = (int32_t*)malloc(sizeof(int32_t) * (size_t)n_nodes);
    memcpy(fill, t_ptr, sizeof(int32_t) * (size_t)n_nodes);
    for (int64_t u = 0; u < n_nodes; ++u)
        for (int64_t e = row_ptr[u]; e < row_ptr[u + 1]; ++e) {
            int32_t pos = fill[col[e]]++;
            t_dst[pos] = (int32_t)u;
            t_eid[pos] = (int32_t)e;
        }
    free(fill);
}

/*
 * Attention dropout mask (see oracle/bpt_oracle.py for the definition): Philox4x32 with 10 rounds,
 * key = (seed low word, seed high word), counter = (destination, source, batch * H + head, tag);
 * the edge is kept iff the first output word is >= floor(p * 2^32).  Returns keep / (1 - p).
 */
static double dropout_weight(uint64_t seed, double p, int64_t bh, int64_t dst, int64_t src) {
    if (p <= 0.0) return 1.0;
    uint32_t c0 = (uint32_t)dst, c1 = (uint32_t)src, c2 = (uint32_t)bh, c3 = 0x42505431u;
    uint32_t k0 = (uint32_t)(seed & 0xffffffffu), k1 = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    double thr = floor(p * 4294967296.0);
    if (thr > 4294967295.0) thr = 4294967295.0;
    return (double)c0 >= thr ? 1.0 / (1.0 - p) : 0.0;
}

/*
 * Forward.  q,k,v,out: [B, N, H, d] doubles; r: [n_rel, d]; lse: [B, N, H].
 * Only batch entries [b0, b1) are computed (they are independent).
 */
void orc_attn_fwd(int64_t N, const int32_t* row_ptr, const int32_t* col, const int32_t* rel,
                  int64_t B, int64_t H, int64_t d, int64_t b0, int64_t b1,
                  const double* q, const double* k, const double* v, const double* r, double scale,
                  double* out, double* lse, double p_drop, uint64_t seed) {
    (void)B;
    const int64_t rs = H * d; /* row stride */
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int64_t b = b0; b < b1; ++b)
        for (int64_t h = 0; h < H; ++h) {
            int64_t maxdeg = 0;
            for (int64_t u = 0; u < N; ++u)
                if (row_ptr[u + 1] - row_ptr[u] > maxdeg) maxdeg = row_ptr[u + 1] - row_ptr[u];
            double* s = (double*)malloc(sizeof(double) * (size_t)(maxdeg ? maxdeg : 1));
            for (int64_t u = 0; u < N; ++u) {
                const double* qu = q + (b * N + u) * rs + h * d;
                double* ou = out + (b * N + u) * rs + h * d;
                const int64_t a = row_ptr[u], z = row_ptr[u + 1];
                if (a == z) { /* no predecessors (length-masked graph): out = 0, lse = 0 */
                    for (int64_t c = 0; c < d; ++c) ou[c] = 0.0;
                    lse[(b * N + u) * H + h] = 0.0;
                    continue;
                }
                double mx = -INFINITY;
                for (int64_t e = a; e < z; ++e) {
                    const double* kv = k + (b * N + col[e]) * rs + h * d;
                    const double* re = r + (int64_t)rel[e] * d;
                    double acc = 0.0;
                    for (int64_t c = 0; c < d; ++c) acc += qu[c] * (kv[c] + re[c]);
                    s[e - a] = scale * acc;
                    if (s[e - a] > mx) mx = s[e - a];
                }
                double sum = 0.0;
                for (int64_t e = a; e < z; ++e) { s[e - a] = exp(s[e - a] - mx); sum += s[e - a]; }
                for (int64_t c = 0; c < d; ++c) ou[c] = 0.0;
                for (int64_t e = a; e < z; ++e) {
                    const double* vv = v + (b * N + col[e]) * rs + h * d;
                    const double p = s[e - a] / sum * dropout_weight(seed, p_drop, b * H + h, u, col[e]);
                    for (int64_t c = 0; c < d; ++c) ou[c] += p * vv[c];
                }
                lse[(b * N + u) * H + h] = mx + log(sum);
            }
            free(s);
        }
}

/*
 * Backward of sum(out * d_out).  dq,dk,dv: [B, N, H, d] (entries of batches
 * [b0,b1) are overwritten); dr: [n_rel, d], overwritten with the sum over the
 * computed batches and all heads.  The row term sum_e P_e dP_e equals
 * d_out_u . out_u; when out_opt is not NULL that second form is evaluated with the
 * given (possibly rounded) forward output, otherwise the exact sum is used.
 */
void orc_attn_bwd(int64_t N, int64_t n_rel, const int32_t* row_ptr, const int32_t* col, const int32_t* rel,
                  int64_t B, int64_t H, int64_t d, int64_t b0, int64_t b1,
                  const double* q, const double* k, const double* v, const double* r, double scale,
                  const double* d_out, const double* out_opt, double* dq, double* dk, double* dv, double* dr,
                  double p_drop, uint64_t seed) {
    (void)B;
    const int64_t rs = H * d;
    const int64_t nbh = (b1 - b0) * H;
    double* dr_part = (double*)calloc((size_t)(nbh * n_rel * d), sizeof(double));
    for (int64_t b = b0; b < b1; ++b) {
        memset(dq + b * N * rs, 0, sizeof(double) * (size_t)(N * rs));
        memset(dk + b * N * rs, 0, sizeof(double) * (size_t)(N * rs));
        memset(dv + b * N * rs, 0, sizeof(double) * (size_t)(N * rs));
    }
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int64_t b = b0; b < b1; ++b)
        for (int64_t h = 0; h < H; ++h) {
            double* drp = dr_part + ((b - b0) * H + h) * n_rel * d;
            int64_t maxdeg = 1;
            for (int64_t u = 0; u < N; ++u)
                if (row_ptr[u + 1] - row_ptr[u] > maxdeg) maxdeg = row_ptr[u + 1] - row_ptr[u];
            double* p = (double*)malloc(sizeof(double) * (size_t)maxdeg);
            double* dp = (double*)malloc(sizeof(double) * (size_t)maxdeg);
            for (int64_t u = 0; u < N; ++u) {
                const int64_t off_u = (b * N + u) * rs + h * d;
                const double* qu = q + off_u;
                const double* gu = d_out + off_u;
                const int64_t a = row_ptr[u], z = row_ptr[u + 1];
                if (a == z) continue;
                double mx = -INFINITY;
                for (int64_t e = a; e < z; ++e) {
                    const double* kv = k + (b * N + col[e]) * rs + h * d;
                    const double* re = r + (int64_t)rel[e] * d;
                    double acc = 0.0;
                    for (int64_t c = 0; c < d; ++c) acc += qu[c] * (kv[c] + re[c]);
                    p[e - a] = scale * acc;
                    if (p[e - a] > mx) mx = p[e - a];
                }
                double sum = 0.0;
                for (int64_t e = a; e < z; ++e) { p[e - a] = exp(p[e - a] - mx); sum += p[e - a]; }
                double dot = 0.0; /* sum_e P_e dP_e */
                for (int64_t e = a; e < z; ++e) {
                    const double* vv = v + (b * N + col[e]) * rs + h * d;
                    double acc = 0.0;
                    for (int64_t c = 0; c < d; ++c) acc += gu[c] * vv[c];
                    p[e - a] /= sum;
                    dp[e - a] = acc * dropout_weight(seed, p_drop, b * H + h, u, col[e]); /* dP_e = W_e d_out . v */
                    dot += p[e - a] * dp[e - a];
                }
                if (out_opt) {
                    dot = 0.0;
                    for (int64_t c = 0; c < d; ++c) dot += gu[c] * out_opt[off_u + c];
                }
                for (int64_t e = a; e < z; ++e) {
                    const int64_t off_v = (b * N + col[e]) * rs + h * d;
                    const double* re = r + (int64_t)rel[e] * d;
                    const double ds = p[e - a] * (dp[e - a] - dot);
                    for (int64_t c = 0; c < d; ++c) {
                        dq[off_u + c] += scale * ds * (k[off_v + c] + re[c]);
                        dk[off_v + c] += scale * ds * qu[c];
                        dv[off_v + c] += p[e - a] * dropout_weight(seed, p_drop, b * H + h, u, col[e]) * gu[c];
                        drp[(int64_t)rel[e] * d + c] += scale * ds * qu[c];
                    }
                }
            }
            free(p); free(dp);
        }
    for (int64_t x = 0; x < n_rel * d; ++x) {
        double acc = 0.0;
        for (int64_t j = 0; j < nbh; ++j) acc += dr_part[j * n_rel * d + x];
        dr[x] = acc;
    }
    free(dr_part);
}
