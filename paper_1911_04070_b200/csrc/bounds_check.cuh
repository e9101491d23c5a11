// Index checks of the debug build.  Compiled with -DBPT_BOUNDS_CHECK (a second shared object, libbpt_check.so),
// every index a gather or an index-array write uses -- an offset into the CSR arrays against E, a gathered node
// against the node count, a relation against n_rel -- is tested before the access.  A violation is counted, its
// first occurrence is recorded (site code, index, limit) in a device word block, and the access is skipped:
// nothing traps, the kernel runs to its end and bpt_debug_bounds hands the record to the host.  In the normal
// build BPT_IDX_OK(...) is the constant true and the checks cost nothing.
#pragma once

#ifdef BPT_BOUNDS_CHECK
namespace bpt {
extern __device__ unsigned int g_bounds_record[4];  // violations, site code, index, limit (defined in api.cu)
__device__ __forceinline__ bool idx_ok(long long i, long long n, int site) {
    if (i >= 0 && i < n) return true;
    if (atomicAdd(&g_bounds_record[0], 1u) == 0u) {
        g_bounds_record[1] = (unsigned int)site;
        g_bounds_record[2] = (unsigned int)i;
        g_bounds_record[3] = (unsigned int)n;
    }
    return false;
}
}  // namespace bpt
#define BPT_IDX_OK(i, n, site) ::bpt::idx_ok((long long)(i), (long long)(n), (site))
#else
#define BPT_IDX_OK(i, n, site) true
#endif

// site codes
#define BPT_SITE_CSR_OFFSET 1     // position in col / rel / t_dst / t_eid
#define BPT_SITE_NODE 2           // a gathered or staged node row
#define BPT_SITE_RELATION 3       // a relation-table row
#define BPT_SITE_EDGE_ID 4        // an edge id read from the by-source lists
#define BPT_SITE_GRAPH_WRITE 5    // a position the graph builder writes
