// C-ABI entry points: argument validation and dispatch.  See include/bpt.h.
#include "bounds_check.cuh"
#include "bpt_internal.cuh"

#ifdef BPT_BOUNDS_CHECK
namespace bpt {
__device__ unsigned int g_bounds_record[4];
}
#endif

using namespace bpt;

static bpt_status check_problem(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype, bool backward) {
    if (!g || !g->row_ptr || !g->col || !g->rel) return BPT_ERR_INVALID_ARG;
    if (B < 1 || H < 1) return BPT_ERR_INVALID_ARG;
    if (dtype != BPT_F32 && dtype != BPT_BF16) return BPT_ERR_INVALID_ARG;
    if (d != 32 && d != 64) return BPT_ERR_UNSUPPORTED;
    TreeParams t;
    if (g->dims.n >= 2 && (g->dims.n & (g->dims.n - 1)) != 0) return BPT_ERR_UNSUPPORTED;
    if (!tree_params_from_dims(g->dims, &t)) return BPT_ERR_INVALID_ARG;
    if (g->dims.n_nodes != 2 * g->dims.n - 1 || g->dims.n_edges < g->dims.n_nodes || g->dims.n_edges >= INT32_MAX)
        return BPT_ERR_INVALID_ARG;
    if (backward && !(g->t_ptr && g->t_dst && g->t_eid)) return BPT_ERR_INVALID_ARG;
    return BPT_OK;
}

// Every non-empty workspace starts with a 256-byte status block (first word: 0, or the bpt_status a
// kernel reported); the launchers get what follows it.
constexpr size_t kStatusBytes = 256;
static size_t with_status(size_t inner) { return inner ? inner + kStatusBytes : 0; }

extern "C" size_t bpt_attn_workspace_bytes(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype, int backward) {
    if (check_problem(g, B, H, d, dtype, false) != BPT_OK) return 0;
    return with_status(backward ? bwd_workspace_bytes(*g, B, H, d, dtype) : fwd_workspace_bytes(*g, B, H, d, dtype));
}

extern "C" size_t bpt_attn_bwd_min_workspace_bytes(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype) {
    if (check_problem(g, B, H, d, dtype, false) != BPT_OK) return 0;
    return with_status(bwd_workspace_bytes(*g, B, H, d, dtype, true));
}

extern "C" bpt_status bpt_check(const void* workspace, void* cuda_stream) {
    if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return BPT_ERR_CUDA;
    if (!workspace) return BPT_OK;
    int32_t word = 0;
    if (cudaMemcpy(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return BPT_ERR_CUDA;
    return word == 0 ? BPT_OK : (word == (int32_t)BPT_ERR_TIMEOUT ? BPT_ERR_TIMEOUT : BPT_ERR_CUDA);
}

static bool options_ok(const bpt_attn_options* opt) {
    return !opt || (opt->dropout_p >= 0.f && opt->dropout_p < 1.f && opt->path <= BPT_PATH_TC5);
}

// Splits the caller's workspace into the status block (cleared on the stream) and the launcher's part.
static bpt_status take_workspace(AttnProblem& p, void* workspace, size_t workspace_bytes, size_t inner_need) {
    p.status = nullptr; p.workspace = nullptr; p.workspace_bytes = 0;
    if (inner_need == 0) return BPT_OK;
    if (!workspace || workspace_bytes < inner_need + kStatusBytes) return BPT_ERR_WORKSPACE;
    p.status = static_cast<int*>(workspace);
    p.workspace = static_cast<char*>(workspace) + kStatusBytes;
    p.workspace_bytes = workspace_bytes - kStatusBytes;
    return cudaMemsetAsync(workspace, 0, kStatusBytes, p.stream) == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
}

static bpt_status attn_fwd_impl(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                                const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                                const int32_t* lengths, DropoutParams drop, uint32_t path, void* out, float* lse, void* workspace,
                                size_t workspace_bytes, void* cuda_stream) {
    const bpt_status s = check_problem(g, B, H, d, dtype, false);
    if (s != BPT_OK) return s;
    if (!q || !k || !v || !rel_emb || !out || !lse) return BPT_ERR_INVALID_ARG;
    AttnProblem p{};
    p.g = g;
    tree_params_from_dims(g->dims, &p.tree);
    p.B = B; p.H = H; p.d = d; p.dtype = dtype;
    p.q = q; p.k = k; p.v = v; p.rel_emb = rel_emb; p.scale = scale; p.lengths = lengths; p.drop = drop; p.path = path;
    p.out = out; p.lse = lse;
    p.stream = (cudaStream_t)cuda_stream;
    const bpt_status w = take_workspace(p, workspace, workspace_bytes, fwd_workspace_bytes(*g, B, H, d, dtype));
    return w != BPT_OK ? w : launch_fwd(p);
}

extern "C" bpt_status bpt_attn_fwd(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                                   const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                                   void* out, float* lse, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return attn_fwd_impl(g, B, H, d, dtype, q, k, v, rel_emb, scale, nullptr, make_dropout(0.f, 0), BPT_PATH_AUTO, out, lse, workspace, workspace_bytes, cuda_stream);
}

extern "C" bpt_status bpt_attn_fwd_varlen(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                                          const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                                          const int32_t* lengths, void* out, float* lse, void* workspace,
                                          size_t workspace_bytes, void* cuda_stream) {
    if (!lengths) return BPT_ERR_INVALID_ARG;
    return attn_fwd_impl(g, B, H, d, dtype, q, k, v, rel_emb, scale, lengths, make_dropout(0.f, 0), BPT_PATH_AUTO, out, lse, workspace, workspace_bytes, cuda_stream);
}

extern "C" bpt_status bpt_attn_fwd_ex(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                                      const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                                      const bpt_attn_options* opt, void* out, float* lse, void* workspace,
                                      size_t workspace_bytes, void* cuda_stream) {
    if (!options_ok(opt)) return BPT_ERR_INVALID_ARG;
    return attn_fwd_impl(g, B, H, d, dtype, q, k, v, rel_emb, scale, opt ? opt->lengths : nullptr,
                         opt ? make_dropout(opt->dropout_p, opt->dropout_seed) : make_dropout(0.f, 0), opt ? opt->path : BPT_PATH_AUTO,
                         out, lse, workspace, workspace_bytes, cuda_stream);
}

static bpt_status attn_bwd_impl(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                                const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                                const int32_t* lengths, DropoutParams drop, uint32_t path, const void* out, const float* lse, const void* d_out,
                                void* dq, void* dk, void* dv, float* d_rel,
                                void* workspace, size_t workspace_bytes, void* cuda_stream) {
    const bpt_status s = check_problem(g, B, H, d, dtype, true);
    if (s != BPT_OK) return s;
    if (!q || !k || !v || !rel_emb || !out || !lse || !d_out || !dq || !dk || !dv || !d_rel) return BPT_ERR_INVALID_ARG;
    AttnProblem p{};
    p.g = g;
    tree_params_from_dims(g->dims, &p.tree);
    p.B = B; p.H = H; p.d = d; p.dtype = dtype;
    p.q = q; p.k = k; p.v = v; p.rel_emb = rel_emb; p.scale = scale; p.lengths = lengths; p.drop = drop; p.path = path;
    p.out = const_cast<void*>(out); p.lse = const_cast<float*>(lse);
    p.d_out = d_out; p.dq = dq; p.dk = dk; p.dv = dv; p.d_rel = d_rel;
    p.stream = (cudaStream_t)cuda_stream;
    // the tiled backward runs with any workspace from the minimum up: fewer pairs per pass with a smaller one
    const bpt_status w = take_workspace(p, workspace, workspace_bytes, bwd_workspace_bytes(*g, B, H, d, dtype, true));
    return w != BPT_OK ? w : launch_bwd(p);
}

extern "C" bpt_status bpt_attn_fwd_rows(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                                        const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                                        const bpt_attn_options* opt, const int32_t* rows, int32_t n_rows,
                                        void* out, float* lse, void* cuda_stream) {
    const bpt_status s = check_problem(g, B, H, d, dtype, false);
    if (s != BPT_OK) return s;
    if (!q || !k || !v || !rel_emb || !out || !lse || !rows || n_rows < 1 || !options_ok(opt)) return BPT_ERR_INVALID_ARG;
    AttnProblem p{};
    p.g = g;
    tree_params_from_dims(g->dims, &p.tree);
    p.B = B; p.H = H; p.d = d; p.dtype = dtype;
    p.q = q; p.k = k; p.v = v; p.rel_emb = rel_emb; p.scale = scale;
    p.lengths = opt ? opt->lengths : nullptr;
    p.drop = opt ? make_dropout(opt->dropout_p, opt->dropout_seed) : make_dropout(0.f, 0);
    p.out = out; p.lse = lse;
    p.stream = (cudaStream_t)cuda_stream;
    return launch_fwd_row_list(p, rows, n_rows);
}

extern "C" bpt_status bpt_attn_bwd(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                                   const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                                   const void* out, const float* lse, const void* d_out,
                                   void* dq, void* dk, void* dv, float* d_rel,
                                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return attn_bwd_impl(g, B, H, d, dtype, q, k, v, rel_emb, scale, nullptr, make_dropout(0.f, 0), BPT_PATH_AUTO, out, lse, d_out, dq, dk, dv, d_rel,
                         workspace, workspace_bytes, cuda_stream);
}

extern "C" bpt_status bpt_attn_bwd_varlen(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                                          const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                                          const int32_t* lengths, const void* out, const float* lse, const void* d_out,
                                          void* dq, void* dk, void* dv, float* d_rel,
                                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!lengths) return BPT_ERR_INVALID_ARG;
    return attn_bwd_impl(g, B, H, d, dtype, q, k, v, rel_emb, scale, lengths, make_dropout(0.f, 0), BPT_PATH_AUTO, out, lse, d_out, dq, dk, dv, d_rel,
                         workspace, workspace_bytes, cuda_stream);
}

extern "C" bpt_status bpt_attn_bwd_ex(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                                      const void* q, const void* k, const void* v, const void* rel_emb, float scale,
                                      const bpt_attn_options* opt, const void* out, const float* lse, const void* d_out,
                                      void* dq, void* dk, void* dv, float* d_rel,
                                      void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!options_ok(opt)) return BPT_ERR_INVALID_ARG;
    return attn_bwd_impl(g, B, H, d, dtype, q, k, v, rel_emb, scale, opt ? opt->lengths : nullptr,
                         opt ? make_dropout(opt->dropout_p, opt->dropout_seed) : make_dropout(0.f, 0), opt ? opt->path : BPT_PATH_AUTO,
                         out, lse, d_out, dq, dk, dv, d_rel, workspace, workspace_bytes, cuda_stream);
}

// ---------------------------------------------------------------------------------
// tracing
// ---------------------------------------------------------------------------------
namespace {
constexpr int kTraceMax = 4096;
struct TraceState {
    bool on = false;
    int n = 0, cap = 0;
    cudaEvent_t ev[kTraceMax];
    const char* name[kTraceMax];
} g_trace;
}  // namespace

void bpt::trace_mark(cudaStream_t st, const char* name) {
    if (!g_trace.on || g_trace.n >= g_trace.cap) return;
    cudaEventRecord(g_trace.ev[g_trace.n], st);
    g_trace.name[g_trace.n] = name;
    ++g_trace.n;
}

extern "C" bpt_status bpt_trace_begin(int32_t capacity, void* cuda_stream) {
    if (g_trace.on || capacity < 1 || capacity >= kTraceMax) return BPT_ERR_INVALID_ARG;
    for (int i = 0; i <= capacity; ++i)
        if (cudaEventCreate(&g_trace.ev[i]) != cudaSuccess) return BPT_ERR_CUDA;
    g_trace.cap = capacity + 1;
    g_trace.n = 0;
    g_trace.on = true;
    bpt::trace_mark((cudaStream_t)cuda_stream, "begin");
    return BPT_OK;
}

extern "C" bpt_status bpt_trace_end(int32_t* n_marks, float* ms, const char** names, int32_t capacity) {
    if (!g_trace.on || !n_marks) return BPT_ERR_INVALID_ARG;
    g_trace.on = false;
    bpt_status st = BPT_OK;
    const int n = g_trace.n - 1;  // intervals
    if (n >= 1 && cudaEventSynchronize(g_trace.ev[n]) != cudaSuccess) st = BPT_ERR_CUDA;
    for (int i = 0; i < n && i < capacity && st == BPT_OK; ++i) {
        if (ms && cudaEventElapsedTime(&ms[i], g_trace.ev[i], g_trace.ev[i + 1]) != cudaSuccess) st = BPT_ERR_CUDA;
        if (names) names[i] = g_trace.name[i + 1];
    }
    for (int i = 0; i < g_trace.cap; ++i) cudaEventDestroy(g_trace.ev[i]);
    *n_marks = n < 0 ? 0 : n;
    g_trace.n = g_trace.cap = 0;
    return st;
}

extern "C" bpt_status bpt_debug_bounds(uint32_t* record, void* cuda_stream) {
#ifdef BPT_BOUNDS_CHECK
    if (!record) return BPT_ERR_INVALID_ARG;
    if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return BPT_ERR_CUDA;
    if (cudaMemcpyFromSymbol(record, g_bounds_record, sizeof(g_bounds_record)) != cudaSuccess) return BPT_ERR_CUDA;
    const unsigned int zero[4] = {0, 0, 0, 0};
    return cudaMemcpyToSymbol(g_bounds_record, zero, sizeof(zero)) == cudaSuccess ? BPT_OK : BPT_ERR_CUDA;
#else
    (void)record; (void)cuda_stream;
    return BPT_ERR_UNSUPPORTED;   // this build carries no index checks
#endif
}

extern "C" const char* bpt_status_str(bpt_status s) {
    switch (s) {
        case BPT_OK: return "ok";
        case BPT_ERR_INVALID_ARG: return "invalid argument";
        case BPT_ERR_UNSUPPORTED: return "unsupported size or type";
        case BPT_ERR_WORKSPACE: return "workspace missing or too small";
        case BPT_ERR_CUDA: return "CUDA error";
        case BPT_ERR_TIMEOUT: return "device-side wait timed out";
        case BPT_ERR_OVERFLOW: return "edge count exceeds 32-bit indices";
        case BPT_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the built-in static array holds";
    }
    return "unknown status";
}
