// Host side of the edge stream: task lists and launches (kernels in edge_stream_impl.cuh,
// instantiated in edge_stream_k*.cu).
#include <algorithm>

#include "edge_stream_args.h"
#include "internal.h"

namespace sobek {

// Source-major task list of one direction, sorted by kernel class (= padded d_src).  For every source
// irrep block and every block of 32 multiplicities, the output components (path, o) of all paths that
// read this block are packed into tasks of at most CAP components, split evenly.
void build_stream_tasks(const sobek_plan* p, Direction& dir) {
    const int KC = p->K <= 8 ? 8 : 16;
    const int CAP = KC == 8 ? 4 : 3;
    dir.stasks.clear();
    dir.scomps.clear();
    dir.sclasses.clear();
    // distinct source blocks, in order of appearance
    std::vector<int> src_offs;
    for (const DPath& P : dir.paths)
        if (std::find(src_offs.begin(), src_offs.end(), P.src_off) == src_offs.end()) src_offs.push_back(P.src_off);
    for (int so : src_offs) {
        std::vector<SComp> all;
        int c_src = 0, d_src = 0;
        for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
            const DGroup& G = dir.groups[gi];
            for (int k = G.path_begin; k < G.path_end; ++k) {
                const DPath& P = dir.paths[k];
                if (P.src_off != so) continue;
                c_src = P.c_src; d_src = P.d_src;
                for (int o = 0; o < G.d_dst; ++o)
                    all.push_back(SComp{P.tabM + o, G.d_dst, P.sh_off, (int)gi, o, P.koff, G.d_dst, 0});
            }
        }
        if (all.empty()) continue;
        const int ntask = ((int)all.size() + CAP - 1) / CAP;
        const int per = ((int)all.size() + ntask - 1) / ntask;
        const int cls = d_src <= 3 ? 0 : (d_src <= 5 ? 1 : 2);
        for (int u0 = 0; u0 < c_src; u0 += 32)
            for (int t = 0; t < ntask; ++t) {
                const int c0 = t * per, c1 = std::min((int)all.size(), c0 + per);
                STask T{};
                T.src_off = so; T.c_src = c_src; T.d_src = d_src; T.u0 = u0;
                T.ncomp = c1 - c0; T.comp_begin = (int)dir.scomps.size(); T.cls = cls;
                dir.scomps.insert(dir.scomps.end(), all.begin() + c0, all.begin() + c1);
                dir.stasks.push_back(T);
            }
    }
    std::stable_sort(dir.stasks.begin(), dir.stasks.end(), [](const STask& x, const STask& y) { return x.cls < y.cls; });
    for (size_t i = 0; i < dir.stasks.size();) {
        size_t j = i;
        while (j < dir.stasks.size() && dir.stasks[j].cls == dir.stasks[i].cls) ++j;
        dir.sclasses.push_back({dir.stasks[i].cls, (int)i, (int)(j - i)});
        i = j;
    }
}

cudaError_t launch_stream(const sobek_plan* p, const Direction& dir, const EdgeView& ev, int64_t node0,
                          int64_t n_nodes, const float* src, const float* vsrc, const SplitSrc& ss, const float* Y,
                          const float* vY, const float* phi, const float* vphi, int dual, void* zh, void* zl,
                          int* status, cudaStream_t s) {
    if (n_nodes <= 0 || dir.stasks.empty()) return cudaSuccess;
    // tensor-core stream when the profile allows it and the caller made the bf16 copies of the sources
    if (p->use_tc_stream && dir.tc[dual ? 1 : 0].ok && status && ss.h && ss.l && (!vsrc || (ss.vh && ss.vl)))
        return launch_stream_tc(p, dir, ev, node0, n_nodes, ss, Y, vY, phi, vphi, dual, zh, zl, status, s);
    if (ss.rvec) return cudaErrorNotSupported;      // the geometry mode exists in the tensor-core kernels only
    const int KC = p->K <= 8 ? 8 : 16;
    StreamArgsHost a{};
    a.tasks = dir.d_stasks; a.comps = dir.d_scomps;
    a.zb_off = dir.d_zb_off; a.zb_ld = dir.d_nk_ld;
    a.tab_ptr = p->d_tab_ptr; a.tab_idx = p->d_tab_idx; a.tab_coef = p->d_tab_coef;
    a.ev = ev; a.node0 = node0; a.n_nodes = n_nodes;
    a.src = src; a.vsrc = vsrc; a.Y = Y; a.vY = vY; a.phi = phi; a.vphi = vphi;
    a.zh = zh; a.zl = zl;
    a.K = p->K; a.dsh = p->dim_sh; a.C_src = dir.C_src; a.warp_floats = 0; a.status = status;
    Fork fork(p, s);   // the kernel classes touch disjoint parts of the state: run them concurrently
    for (const auto& c : dir.sclasses) {
        cudaStream_t cs = fork.pick();
        KernelTimer kt(K_STATE, cs);
        cudaError_t e;
        if (KC == 8) e = dual ? stream_launch_k8_dual(&a, c.cls, c.begin, c.count, cs) : stream_launch_k8(&a, c.cls, c.begin, c.count, cs);
        else e = dual ? stream_launch_k16_dual(&a, c.cls, c.begin, c.count, cs) : stream_launch_k16(&a, c.cls, c.begin, c.count, cs);
        count_launch();
        if (e != cudaSuccess) return e;
    }
    return fork.join();
}

}  // namespace sobek
