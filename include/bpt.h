/*
 * bpt.h -- C ABI of the B200 (sm_100a) implementation of BP-Transformer's graph
 * self-attention (arXiv 1911.04070).
 *
 * The library builds the binary-partition attention graph of Sec. 3.2 on the
 * device and evaluates graph self-attention with tree relative positions
 * (Sec. 3.1 and 3.4) forward and backward over it.
 *
 * Conventions (0-indexed): n tokens (a power of two), L = log2 n, node (l, m)
 * is the m-th node of level l and covers tokens [m*2^l, (m+1)*2^l); level 0 are
 * the tokens, level L is the root.  Node ids are level-major:
 *     id(l, m) = 2n - (2n >> l) + m        (tokens 0..n-1, root 2n-2).
 * An edge v -> u means "u attends to v".
 *
 * Ownership: the caller owns every buffer.  Unless a comment says "host", every
 * pointer is a DEVICE pointer valid on the current device.  Calls enqueue work on
 * `cuda_stream` (a cudaStream_t passed as void*, NULL = legacy default stream) and
 * return without synchronising.  Nothing is allocated or kept between calls, so the attention calls
 * (bpt_attn_fwd / bpt_attn_bwd and their _varlen, _ex, _rows forms) can be captured in a CUDA graph.
 * The library reads no environment variable and keeps no process-wide setting (the one exception,
 * the benchmark trace, is described at bpt_trace_begin).
 * Argument errors are detected on the host before anything is launched.
 *
 * Device-side failure report.  A non-empty attention workspace begins with a 256-byte status block
 * that every attention call clears on its stream before its kernels run.  Kernels that wait on
 * hardware barriers (the tensor-memory kernels) bound every wait to about a second; if one expires
 * the kernel winds down, the results of the call are invalid and BPT_ERR_TIMEOUT is stored in the
 * block.  bpt_check reads it.
 */
#ifndef BPT_H
#define BPT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BPT_OK = 0,
    BPT_ERR_INVALID_ARG = 1,  /* null pointer, non-positive size, unknown flag, ...          */
    BPT_ERR_UNSUPPORTED = 2,  /* head size / dtype / range the kernels do not cover; n not  */
                              /* a power of two                                             */
    BPT_ERR_WORKSPACE = 3,    /* workspace missing or smaller than the size query says      */
    BPT_ERR_CUDA = 4,         /* a CUDA runtime call or launch failed                       */
    BPT_ERR_TIMEOUT = 5,      /* a bounded device-side wait expired (see bpt_attn_fwd)      */
    BPT_ERR_OVERFLOW = 6,     /* edge count does not fit the 32-bit index arrays            */
    BPT_ERR_SCRATCH_LIMIT = 7 /* problem needs more scratch than the built-in static array  */
} bpt_status;

/* flags of a graph */
enum {
    BPT_BIDIR = 0,      /* contextual edges from both sides (Sec. 3.2.2)                          */
    BPT_LEFT_ONLY = 1,  /* only the left context, for autoregressive use (Sec. 4.2); self and      */
                        /* affiliated edges are kept                                               */
    BPT_MODE_PAD = 0,   /* default: k nodes per level plus the alignment node of Sec. 3.2.2 -- one  */
                        /* more when the level's last node is a left child, so that the next level  */
                        /* starts on a whole parent                                                 */
    BPT_MODE_ALG1 = 2   /* Algorithm 1 taken literally: exactly k nodes per level, no extra node   */
};

typedef enum { BPT_F32 = 0, BPT_BF16 = 1 } bpt_dtype;

typedef struct {
    int32_t n, k;
    uint32_t flags;
    int32_t n_levels;             /* L = log2 n                                     */
    int32_t n_nodes;              /* 2n - 1 (Sec. 3.2.1)                            */
    int32_t n_rel;                /* rows of the relation table, see bpt_build_graph */
    int64_t n_edges;              /* E                                              */
    size_t build_workspace_bytes; /* workspace bpt_build_graph needs                */
} bpt_graph_dims;

typedef struct {
    const int32_t* row_ptr; /* [n_nodes + 1] CSR by destination                              */
    const int32_t* col;     /* [E] source node of each edge, ascending inside a row          */
    const int32_t* rel;     /* [E] relation id of each edge                                  */
    const int32_t* t_ptr;   /* [n_nodes + 1] by-source lists (needed by the backward), or NULL */
    const int32_t* t_dst;   /* [E] destination node, ascending inside a source's list        */
    const int32_t* t_eid;   /* [E] position of that edge in col/rel                          */
    bpt_graph_dims dims;
} bpt_graph;

/*
 * Sizes of the graph for (n, k, flags) -- host only, no device work.
 * Sec. 3.2: 2n-1 nodes; per token a self loop (Algorithm 1, N <- {u}), k (or k+1
 * with the pad rule) contextual nodes per level and side, fine to coarse; per span
 * one affiliated edge from every token it contains.
 * Requires n a power of two (Sec. 3.2.1 builds a perfect binary tree; shorter sequences are served
 * by the length arguments of the attention calls), 2 <= n <= 2^20, 1 <= k <= 2^20.  `out` is a host pointer.
 * Errors: INVALID_ARG, UNSUPPORTED (range, n not a power of two), OVERFLOW (E >= 2^31).
 */
bpt_status bpt_graph_dims_query(int32_t n, int32_t k, uint32_t flags, bpt_graph_dims* out);

/*
 * Build the graph on the device (Sec. 3.2.2 edge construction, Sec. 3.4 labels).
 *
 * Outputs (device, caller-allocated): row_ptr[n_nodes+1], col[E], rel[E] and, unless
 * all three are NULL, the by-source lists t_ptr[n_nodes+1], t_dst[E], t_eid[E].
 * Rows are destinations in node-id order, sources ascending by node id.
 * Relation ids, with W = k+1:  self = 0;  o-th node (nearest first) joining on the
 * left at level j: 1 + j*W + o;  on the right: 1 + L*W + j*W + o;  token -> its
 * ancestor at level j (1..L): 1 + 2*L*W + (j-1);  n_rel = 1 + 2*L*W + L.
 * `dims` (host) must come from bpt_graph_dims_query.  `workspace` (device) must hold
 * dims->build_workspace_bytes.  `out` (host) receives the pointers and dims.
 * Errors: INVALID_ARG, WORKSPACE, CUDA.
 */
bpt_status bpt_build_graph(const bpt_graph_dims* dims, int32_t* row_ptr, int32_t* col, int32_t* rel,
                           int32_t* t_ptr, int32_t* t_dst, int32_t* t_eid,
                           void* workspace, void* cuda_stream, bpt_graph* out);

/*
 * Bytes of device workspace bpt_attn_fwd (backward == 0) or bpt_attn_bwd
 * (backward != 0) should be given for this problem; 0 on invalid arguments.  Host only.
 * The same sizes serve the _varlen and _ex forms.
 *
 * The backward accepts any workspace of at least bpt_attn_bwd_min_workspace_bytes: where its
 * kernels keep per-(batch entry, head) scratch they work through the pairs in passes, as many pairs
 * per pass as the given bytes hold (the size returned here plans at most 10 GiB per pass).  dq, dk
 * and dv do not depend on the number of passes; d_rel is summed pass by pass, in a fixed order
 * for a given workspace size.
 */
size_t bpt_attn_workspace_bytes(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype, int backward);
size_t bpt_attn_bwd_min_workspace_bytes(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype);

/*
 * Waits for `cuda_stream` and reports what the last attention call that used `workspace` (device
 * pointer, the one passed to that call; NULL is allowed and reports BPT_OK) left in the status
 * block: BPT_OK, or BPT_ERR_TIMEOUT when a bounded device-side wait expired and the call's results
 * are invalid.  BPT_ERR_CUDA when the synchronisation or the copy fails.  Host-synchronous: not for
 * use inside a stream capture.
 */
bpt_status bpt_check(const void* workspace, void* cuda_stream);

/*
 * Forward graph self-attention with relative positions (Sec. 3.4 equation, built on
 * the GSA equations of Sec. 3.1).  For every batch entry b, node u, head h:
 *     s_e = scale * q[b,u,h,:] . (k[b,v,h,:] + rel_emb[rel_e,:])   over edges e = (v -> u)
 *     P   = softmax_e(s),   out[b,u,h,:] = sum_e P_e v[b,v,h,:],   lse[b,u,h] = log sum_e exp(s_e)
 * q, k, v, out: [B, n_nodes, H, d] contiguous, element type `dtype`; rel_emb: [n_rel, d],
 * same type, shared by all heads; lse: [B, n_nodes, H] fp32.  Accumulation is fp32.
 * `scale` is explicit (the paper divides by sqrt(d); callers pass 1/sqrt(d)).
 * d must be 32 or 64.  `g` is a host pointer to a struct of device pointers.
 * `workspace` may be NULL when the size query returns 0.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA; device-side: see bpt_check.
 */
bpt_status bpt_attn_fwd(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                        const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                        void* out, float* lse, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Backward of the same equation: given d_out = dLoss/d out, with P_e = exp(s_e - lse_u),
 *     dP_e = d_out_u . v_v,   dS_e = P_e (dP_e - d_out_u . out_u),
 *     dq_u = scale * sum_{e into u} dS_e (k_v + rel_emb[rel_e]),
 *     dk_v = scale * sum_{e out of v} dS_e q_u,      dv_v = sum_{e out of v} P_e d_out_u,
 *     d_rel[r] = scale * sum_{b,h} sum_{e: rel_e = r} dS_e q_u     (the table is shared, Sec. 3.4).
 * out and lse are the forward's results.  dq, dk, dv: [B, n_nodes, H, d] in `dtype`;
 * d_rel: [n_rel, d] fp32.  All four are overwritten, not accumulated into.  The sums are
 * taken in a fixed order without atomics, so results are bit-reproducible.
 * The d_rel rows of the ancestor relations are written as exact zeros: all edges into a
 * span share one relation, so that embedding shifts every score of the row alike and
 * the softmax (hence the loss) does not depend on it.
 * d_out_u . out_u is evaluated with the stored `out`, so for bf16 the gradients carry the
 * rounding of `out` (relative 2^-9 per element) on top of the fp32 arithmetic.
 * The graph must carry the by-source lists.  Errors as for the forward.
 */
bpt_status bpt_attn_bwd(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                        const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                        const void* out, const float* lse, const void* d_out,
                        void* dq, void* dk, void* dv, float* d_rel,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same two operations for sequences shorter than n (Sec. 3.2.1 defines the tree over a
 * power-of-two number of tokens and is silent about other lengths; this is the library's reading).
 * lengths: device array [B], 1 <= lengths[b] <= n (values outside are clamped).  Batch entry b has
 * its real tokens in the first lengths[b] leaves; a node is real when it covers at least one real
 * token.  Every edge whose source or destination is not real is dropped; node ids, relation ids and
 * offsets stay those of the full graph, so the same bpt_graph and relation table serve all lengths.
 * Rows of nodes that are not real: out = 0, lse = 0, dq = dk = dv = 0.
 * The q, k, v, d_out rows of nodes that are not real never influence a result, but they must hold
 * finite values (they may be multiplied by an exact zero weight): initialise the padding.
 * Everything else is as for bpt_attn_fwd / bpt_attn_bwd; the forward of the backward's `out`, `lse`
 * must have been computed with the same lengths.
 */
bpt_status bpt_attn_fwd_varlen(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                               const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                               const int32_t* lengths, void* out, float* lse,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);
bpt_status bpt_attn_bwd_varlen(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                               const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                               const int32_t* lengths, const void* out, const float* lse, const void* d_out,
                               void* dq, void* dk, void* dv, float* d_rel,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The general form of the two operations: optional sequence lengths (as for the _varlen entry points,
 * NULL = all n) and attention dropout (App. A.1 of the paper lists an attention dropout rate for
 * every experiment; the way the masks are drawn is the library's).  With 0 < dropout_p < 1 every edge
 * weight of every (batch entry, head) is kept with probability 1 - dropout_p and divided by
 * 1 - dropout_p, after the softmax and before the product with v; lse is that of the softmax.
 * The mask is a pure function of (dropout_seed, batch entry, head, destination node, source node):
 * Philox4x32 with 10 rounds, key = (low, high) word of the seed, counter = (destination, source,
 * batch entry * H + head, 0x42505431), edge kept iff the first output word >= floor(dropout_p * 2^32).
 * The backward rebuilds it from the same options (nothing is stored); pass the options the forward had.
 * `path` picks the kernels of the token rows where the tiled tensor-core path applies (bf16, head
 * size 64, n >= 64, k <= 64): BPT_PATH_AUTO lets the library choose by k; BPT_PATH_MMA forces the
 * warp-level (mma.sync) kernels, BPT_PATH_TC5 the tensor-memory (tcgen05) kernels wherever they cover
 * the shape -- for comparison runs and tests.  Other values: INVALID_ARG.
 * `opt` is a host pointer; NULL means no lengths, no dropout, automatic path.  dropout_p outside
 * [0, 1): INVALID_ARG.
 */
enum { BPT_PATH_AUTO = 0, BPT_PATH_MMA = 1, BPT_PATH_TC5 = 2 };
typedef struct {
    const int32_t* lengths; /* device [B] or NULL */
    float dropout_p;
    uint64_t dropout_seed;
    uint32_t path;          /* BPT_PATH_* */
} bpt_attn_options;

bpt_status bpt_attn_fwd_ex(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                           const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                           const bpt_attn_options* opt, void* out, float* lse,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);
bpt_status bpt_attn_bwd_ex(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                           const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                           const bpt_attn_options* opt, const void* out, const float* lse, const void* d_out,
                           void* dq, void* dk, void* dv, float* d_rel,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Forward for a few destination rows only -- the building block of step-by-step decoding with the
 * left-only graph (Sec. 4.2 uses BPT autoregressively): when token i arrives, the rows that change in
 * a layer are token i and its L ancestors, and with lengths[b] = i + 1 the ancestors attend exactly
 * the tokens seen so far.  rows: device array [B][n_rows] of node ids (one list per batch entry;
 * ids outside [0, n_nodes) are skipped); only those rows of out and lse are written.  Same equation,
 * options and layouts as bpt_attn_fwd_ex; runs on the general row kernel, needs no workspace.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 */
bpt_status bpt_attn_fwd_rows(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                             const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                             const bpt_attn_options* opt, const int32_t* rows, int32_t n_rows,
                             void* out, float* lse, void* cuda_stream);

/*
 * Output projection, residual and layer normalisation of a layer in one kernel (Algorithm 2 of Sec. 3.3:
 * Z = norm(H + GSA(H) W^O), with the output projection W^O of Sec. 3.1):
 *     z[r, :] = LayerNorm(h[r, :] + a[r, :] w_o^T) * gamma + beta        for every row r,
 * where a is the attention output with the heads concatenated ([B, n_nodes, H, d] seen as [rows, D], D = H * d),
 * w_o is [D, D] with row o holding the weights of output channel o (the layout of a linear layer's weight),
 * h the layer's input states [rows, D], gamma / beta the normalisation's scale and shift [D] (fp32), z the
 * result [rows, D].  a, w_o, h, z are bf16, contiguous and 16-byte aligned; the product accumulates in fp32 and
 * mean / variance (biased, about the mean) are taken in fp32 over the D channels; one rounding to bf16.
 * D must be 128, 256 or 512; rows >= 1.  `workspace` is NULL or a device buffer of at least 256 bytes that
 * receives the status block (see bpt_check).  Forward only: training goes through the separate operators.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 */
bpt_status bpt_out_proj_norm(const void* a, const void* w_o, const void* h, const float* gamma, const float* beta,
                             void* z, int64_t rows, int32_t D, float eps, void* workspace, void* cuda_stream);

/*
 * Backward pass for callers that must not allocate device memory (the paper has no
 * counterpart; this is a deployment convenience).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin inside a host
 * application that hands out tensors but no raw allocator, a real-time or safety-reviewed
 * loop whose rules forbid allocation after start-up, a process whose memory pool already
 * owns the whole device.  Such callers can provide the inputs and outputs of the
 * backward, but have nowhere to get its workspace from.
 *
 * Same arguments, results and errors as bpt_attn_bwd, minus the workspace: the scratch
 * is a 32 MiB array that lives inside the library's device image (every GPU that loads
 * the library carries it until the process exits).  bpt_static_scratch_bytes() returns
 * that limit.  The backward fits its passes to the array (fewer (batch entry, head) pairs
 * per pass than with a large workspace, same results for dq, dk, dv); only a problem whose
 * bpt_attn_bwd_min_workspace_bytes exceeds the limit -- one pair alone does not fit -- is
 * refused with BPT_ERR_SCRATCH_LIMIT before anything is launched (use bpt_attn_bwd with
 * your own workspace then).  The call itself performs no cudaMalloc / cudaFree and calls
 * no allocating library routine.
 *
 * The first call on each device looks up the array's device address (with that device
 * current); make that first call outside of any stream capture.  The CUDA runtime loads the
 * part of the library that holds the array at that first look-up, and that is when the
 * driver sets the 32 MiB aside: a process that hands the rest of the device to a pool of its
 * own should make one call (any small problem) during start-up, before the pool takes the
 * memory.  All calls on a device
 * share the one array, and it keeps whatever the previous call left in it: the backward
 * overwrites every part before reading it, so nothing needs clearing, but two calls whose
 * GPU work overlaps (different streams, or different threads) would race on it -- keep
 * them ordered on one stream.
 */
size_t bpt_static_scratch_bytes(void);
bpt_status bpt_attn_bwd_static_scratch(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                                       const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                                       const void* out, const float* lse, const void* d_out,
                                       void* dq, void* dk, void* dv, float* d_rel, void* cuda_stream);

/*
 * Per-launch timing for benchmarks (no counterpart in the paper).  Between
 * bpt_trace_begin and bpt_trace_end every kernel the library launches is followed by
 * a CUDA event on its stream; bpt_trace_end waits for the last one and returns, for
 * the first min(*n_marks, capacity) launches, the milliseconds since the previous
 * mark (ms, host array, may be NULL) and a static name (names, host array, may be
 * NULL).  `capacity` of bpt_trace_begin bounds the number of launches recorded
 * (< 4096); later launches go unrecorded.  This is the one piece of process-global
 * state in the library: not thread-safe, off by default, one trace at a time.
 * Errors: INVALID_ARG (nesting, capacity), CUDA.
 */
bpt_status bpt_trace_begin(int32_t capacity, void* cuda_stream);
bpt_status bpt_trace_end(int32_t* n_marks, float* ms, const char** names, int32_t capacity);

/*
 * Test hook for the failure report (no counterpart in the paper): launches one tiny kernel in which
 * one thread waits, for at most `limit_cycles` clock cycles (1 .. 2^31), on a hardware barrier that
 * expects one arrival.  With arrive == 0 nobody arrives: the wait runs out, the kernel stores
 * BPT_ERR_TIMEOUT in the status block at `workspace` (device, >= 256 bytes, cleared first) and ends --
 * exactly the give-up path of the tensor-memory kernels; with arrive != 0 the thread arrives itself
 * and the block stays clear.  Nothing faults or hangs either way.  Read the outcome with bpt_check.
 * Errors: INVALID_ARG, CUDA.
 */
bpt_status bpt_selftest_wait_timeout(void* workspace, int64_t limit_cycles, int32_t arrive, void* cuda_stream);

/*
 * Index checks (no counterpart in the paper).  The package builds the library twice: libbpt.so, and
 * libbpt_check.so compiled with -DBPT_BOUNDS_CHECK, in which every index a gather or an index-array
 * write uses (an offset into col / rel / t_dst / t_eid against E, a gathered or staged node row against
 * n_nodes, a relation row against n_rel, an edge id against E) is tested before the access.  A
 * violation is counted, the first one recorded, and the access skipped; nothing traps.
 * bpt_debug_bounds waits for `cuda_stream`, copies the record to `record` (host, four words:
 * number of violations, site code of the first one, its index, its limit) and clears it.
 * In libbpt.so the checks are compiled out and the call returns BPT_ERR_UNSUPPORTED.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 */
bpt_status bpt_debug_bounds(uint32_t* record, void* cuda_stream);

/* Static description of a status code (host). */
const char* bpt_status_str(bpt_status s);

#ifdef __cplusplus
}
#endif
#endif /* BPT_H */
