// Kernel arguments of the edge stream (shared by the host launcher and the kernel translation units).
#pragma once
#include "internal.h"

namespace sobek {

struct StreamArgs {
    const STask* tasks;
    const SComp* comps;
    const int64_t* zb_off;     // per group: bf16 state offset per node (elements)
    const int32_t* zb_ld;      // per group: row pitch of the bf16 state (elements)
    const int32_t* tab_ptr;
    const int32_t* tab_idx;
    const float* tab_coef;
    EdgeView ev;
    int64_t node0, n_nodes;
    const float* src;
    const float* vsrc;         // DUAL only; may be NULL
    const float* Y;
    const float* vY;           // DUAL only; may be NULL
    const float* phi;
    const float* vphi;         // DUAL only; may be NULL
    void* zh;
    void* zl;
    int32_t K, dsh, C_src;
    int32_t warp_floats;       // shared floats per warp
    int* status;               // device status word (range guards report SOBEK_ERR_GRAPH there); may be NULL
};


typedef StreamArgs StreamArgsHost;

}  // namespace sobek
