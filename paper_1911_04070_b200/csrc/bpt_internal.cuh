// Declarations shared by the translation units of libbpt (not part of the C ABI).
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/bpt.h"
#include "bpt_tree.cuh"
#include "dropout.cuh"

namespace bpt {

bool tree_params_from_dims(const bpt_graph_dims& d, TreeParams* t);

// Problem description handed to the attention launchers (all pointers device).
struct AttnProblem {
    const bpt_graph* g;
    TreeParams tree;
    int B, H, d;
    bpt_dtype dtype;
    const void *q, *k, *v, *rel_emb;
    const int32_t* lengths;  // [B] real tokens per batch entry, or nullptr: all n (see bpt_attn_fwd_varlen)
    DropoutParams drop;      // attention dropout (thr = 0: none)
    float scale;
    // forward outputs / backward inputs
    void* out;
    float* lse;
    // backward only
    const void* d_out;
    void *dq, *dk, *dv;
    float* d_rel;
    void* workspace;         // past the status block
    size_t workspace_bytes;
    int* status;             // device status word (first word of the caller's workspace), or nullptr without a workspace
    uint32_t path;           // BPT_PATH_*: which token-row kernels the tiled path takes
    cudaStream_t stream;
};

// Optional per-launch timing (see bpt_trace_begin): a mark after every kernel launch.
void trace_mark(cudaStream_t st, const char* name);

size_t fwd_workspace_bytes(const bpt_graph& g, int B, int H, int d, bpt_dtype dtype);
// minimal: the least the backward accepts (the tiled path then takes one (batch entry, head) pair per pass)
size_t bwd_workspace_bytes(const bpt_graph& g, int B, int H, int d, bpt_dtype dtype, bool minimal = false);
bpt_status launch_fwd(const AttnProblem& p);
bpt_status launch_fwd_row_list(const AttnProblem& p, const int32_t* rows, int n_rows);
bpt_status launch_bwd(const AttnProblem& p);

}  // namespace bpt
