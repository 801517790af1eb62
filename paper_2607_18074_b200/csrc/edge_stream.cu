// Host side of the edge stream: task lists and launches (kernels in edge_stream_impl.cuh,
// instantiated in edge_stream_k*.cu).
#include <algorithm>

#include "internal.h"

namespace sobek {

// Task list of one direction, sorted by kernel class.  Output components are cut into chunks of at
// most 5, and the multiplicity block per lane (UB) is the largest of {4,2,1} that keeps OC*KC*UB
// accumulators within the register budget and does not exceed what the path's multiplicity can use.
void build_stream_tasks(const sobek_plan* p, Direction& dir) {
    const int KC = p->K <= 8 ? 8 : 16;
    dir.stasks.clear();
    dir.sclasses.clear();
    dir.ms_max = 4;
    for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
        const DGroup& G = dir.groups[gi];
        for (int k = G.path_begin; k < G.path_end; ++k) {
            const DPath& P = dir.paths[k];
            int chunks[2][2];
            int nch = 0;
            const int D = G.d_dst;
            if (D <= 5) { chunks[0][0] = 0; chunks[0][1] = D; nch = 1; }
            else if (D == 7) { chunks[0][0] = 0; chunks[0][1] = 4; chunks[1][0] = 4; chunks[1][1] = 3; nch = 2; }
            else { chunks[0][0] = 0; chunks[0][1] = 5; chunks[1][0] = 5; chunks[1][1] = 4; nch = 2; }
            for (int c = 0; c < nch; ++c) {
                const int oc = chunks[c][1];
                const int ub_budget = 96 / (oc * KC);
                int ub = ub_budget >= 4 ? 4 : (ub_budget >= 2 ? 2 : 1);
                const int need = P.c_src <= 32 ? 1 : (P.c_src <= 64 ? 2 : 4);
                ub = std::min(ub, need);
                const int oci = oc == 1 ? 0 : (oc == 3 ? 1 : (oc == 4 ? 2 : 3));
                const int ubi = ub == 1 ? 0 : (ub == 2 ? 1 : 2);
                const int dsi = P.d_src <= 3 ? 0 : (P.d_src <= 5 ? 1 : 2);
                for (int u0 = 0; u0 < P.c_src; u0 += 32 * ub) {
                    STask t{};
                    t.path = k; t.u0 = u0; t.o0 = chunks[c][0]; t.oc = oc; t.ub = ub;
                    t.cls = (3 * oci + ubi) * 3 + dsi; t.group = (int)gi;
                    dir.stasks.push_back(t);
                }
                int ms = P.d_src * oc;
                ms = (ms + 3) & ~3;
                if ((ms & 31) == 0) ms += 4;
                dir.ms_max = std::max(dir.ms_max, ms);
            }
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
                          int64_t n_nodes, const float* src, const float* vsrc, const float* Y, const float* vY,
                          const float* phi, const float* vphi, int dual, void* zh, void* zl, cudaStream_t s) {
    if (n_nodes <= 0 || dir.stasks.empty()) return cudaSuccess;
    const int KC = p->K <= 8 ? 8 : 16;
    Fork fork(p, s);   // the kernel classes touch disjoint parts of the state: run them concurrently
    const cudaStream_t main = s;
    for (const auto& c : dir.sclasses) {
        s = fork.pick();
        KernelTimer kt(K_STATE, s);
        cudaError_t e;
        if (KC == 8) e = dual ? stream_launch_k8_dual(p, dir, ev, node0, n_nodes, src, vsrc, Y, vY, phi, vphi, zh, zl, c.cls, c.begin, c.count, s)
                              : stream_launch_k8(p, dir, ev, node0, n_nodes, src, Y, phi, zh, zl, c.cls, c.begin, c.count, s);
        else e = dual ? stream_launch_k16_dual(p, dir, ev, node0, n_nodes, src, vsrc, Y, vY, phi, vphi, zh, zl, c.cls, c.begin, c.count, s)
                      : stream_launch_k16(p, dir, ev, node0, n_nodes, src, Y, phi, zh, zl, c.cls, c.begin, c.count, s);
        count_launch();
        if (e != cudaSuccess) return e;
    }
    (void)main;
    return fork.join();
}

}  // namespace sobek
