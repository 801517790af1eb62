// Instantiation of the edge-stream kernels for K-chunk 8.
#include "edge_stream_impl.cuh"

namespace sobek {

cudaError_t stream_launch_k8(const sobek_plan* p, const Direction& dir, const EdgeView& ev, int64_t node0, int64_t n_nodes,
                     const float* src, const float* Y, const float* phi, void* zh, void* zl,
                     int cls, int t_begin, int t_count, cudaStream_t s) {
    StreamArgs a{};
    a.paths = dir.d_paths; a.tasks = dir.d_stasks; a.groups = dir.d_groups;
    a.zb_off = dir.d_zb_off; a.zb_ld = dir.d_nk_ld;
    a.tab_ptr = p->d_tab_ptr; a.tab_idx = p->d_tab_idx; a.tab_coef = p->d_tab_coef;
    a.ev = ev; a.node0 = node0; a.n_nodes = n_nodes; a.n_tasks = t_count;
    a.src = src; a.vsrc = nullptr; a.Y = Y; a.vY = nullptr; a.phi = phi; a.vphi = nullptr;
    a.zh = (__nv_bfloat16*)zh; a.zl = (__nv_bfloat16*)zl;
    a.K = p->K; a.dsh = p->dim_sh; a.C_src = dir.C_src; a.ms_max = dir.ms_max;
    int wf = 32 * dir.ms_max + 32 * 8 + 32 * (a.dsh + 1) + 64;
    if (false) wf += 32 * dir.ms_max + 32 * 8 + 32 * (a.dsh + 1);
    a.warp_floats = wf;
    const size_t sh = (size_t)wf * SW * sizeof(float);
    return launch_class<8, false>(cls, a, t_begin, t_count, sh, s);
}

}  // namespace sobek
