// Range guards for everything the edge kernels read out of the caller's graph arrays before they use it
// as an index.  sobek_graph_prepare validates a graph once, but the arrays are the caller's: a buffer that
// was freed, reused or overwritten since must end in SOBEK_ERR_GRAPH in the status word, never in a wild
// address.  A value that fails its guard is replaced by a harmless one (index 0, an empty segment) and the
// copy it would have driven is turned into its zero-fill form, so the bad address is never formed.
#pragma once
#include <stdint.h>

#include "sobek.h"

namespace sobek {

// true if 0 <= v < n; else records SOBEK_ERR_GRAPH (status may be NULL) and returns false
__device__ __forceinline__ bool id_ok(int64_t v, int64_t n, int* status) {
    if ((uint64_t)v < (uint64_t)n) return true;
    if (status) atomicExch(status, (int)SOBEK_ERR_GRAPH);
    return false;
}

// segment [s0, s1) of `node` in a CSR pointer array over E edges, forced into 0 <= s0 <= s1 <= E
__device__ __forceinline__ void seg_bounds(const int64_t* __restrict__ ptr, int64_t node, int64_t E, int* status,
                                           int64_t& s0, int64_t& s1) {
    const int64_t a = ptr[node], b = ptr[node + 1];
    s0 = a < 0 ? 0 : (a > E ? E : a);
    s1 = b < s0 ? s0 : (b > E ? E : b);
    if ((s0 != a || s1 != b) && status) atomicExch(status, (int)SOBEK_ERR_GRAPH);
}

}  // namespace sobek
