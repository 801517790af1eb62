// Receiver-owned edge pass (sm_100a), SOURCE-MAJOR: the two edge outputs of the backward program
// (Section "Receiver-factorized backward"; Eqs. streamed_radial_adjoints,
// streamed_operand_adjoints written against the receiver state):
//     gphi_e[q] = sum_{pi,u,o} Zbar_i[pi,u,q,o] * C_e[pi,u,o]
//     gY_e[b]   = sum_{pi} sum_{s,o} c[s,b,o] * G_e[pi][s][o],   G_e[s][o] = sum_u xs_e[u,s] * Cbar_e[u,o]
//     Cbar_e[u,o] = sum_q phi_e[q] * Zbar_i[pi,u,q,o],   C_e[u,o] = sum_s xs_e[u,s] * M_e[s,o]
// with i the receiver of edge e and Zbar = gy R^T the adjoint of the receiver state.
//
// One WARP per receiver, LANES <-> EDGES of its segment (32 at a time): both outputs are per edge,
// so nothing is reduced across lanes and every output element has exactly one writer.  A task is
// (source irrep block, up to CAP output components (path, o) of the paths reading that block): each
// lane reads its own sender row once per task with 128-bit loads (next block prefetched), keeps the
// M_e entries, the G_e accumulators and gphi_e in registers, and the Zbar rows of the task's
// components - shared by all lanes - are staged per warp in shared memory with cp.async (double
// buffered) and read with broadcast 128-bit loads.  One launch per kernel class (padded d_src); the
// first class overwrites gphi / gY, later classes accumulate (same owner lane).
//
// With DUAL the pass evaluates the second-order terms that share Zbar in one go
// (Eq. streamed_operand_second_adjoints):
//     hphi_e += <Zbar, C(vx,Y) + C(x,vY)>,   hY_e += CG^T_Y(vx, phi Zbar) + CG^T_Y(x, vphi Zbar).
#include <algorithm>

#include "guard.cuh"
#include "internal.h"

namespace sobek {
namespace {

constexpr int EW = 8;    // warps per CTA
constexpr int XB = 4;    // multiplicities per sender-row block

struct EdgeArgs {
    const STask* tasks;      // source-major tasks (u0 unused: a task covers all multiplicities)
    const SComp* comps;
    const DGroup* groups;
    const int32_t* tab_ptr;
    const int32_t* tab_idx;
    const float* tab_coef;
    EdgeView ev;
    int64_t node0, n_nodes;
    const float* src;
    const float* vsrc;   // DUAL only; may be NULL
    const float* Y;
    const float* vY;     // DUAL only; may be NULL
    const float* phi;
    const float* vphi;   // DUAL only; may be NULL
    const float* Zbar;
    float* gphi;
    float* gY;
    int K, dsh, C_src, phi_mode, Y_mode;
    int warp_floats;     // shared floats per warp
    int zslab;           // floats of one Zbar slab buffer
    int* status;         // device status word (range guards report SOBEK_ERR_GRAPH there)
    int zvec;            // 1: every row pitch and offset of Zbar is a multiple of 4 floats (16-byte pieces may be copied)
};

__device__ __forceinline__ void cp_async4(float* dst, const float* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void cp_async16(float* dst, const float* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}

// Stage the Zbar rows of the task's components for multiplicities [u0, u0+XB) and K-chunk [q0, q0+KC):
// sZ[(c*KC + q)*XB + uu]   (the contraction index of the state is k = koff + q*c_src + u, so the XB
// multiplicities of one (component, q) are 16 contiguous bytes)
template <int CAP, int KC>
__device__ __forceinline__ void stage_zbar(const EdgeArgs& a, const STask& T, const SComp* comps, const int64_t nl,
                                           int u0, int q0, float* sZ, int lane) {
    // 16-byte pieces need the group's row pitch D, the path offset koff and the task's own stride to be multiples of
    // 4 floats: true when every multiplicity of the direction is (a.zvec), not when only this task's is
    const bool vec = a.zvec && (T.c_src & 3) == 0;
    if (vec) {
        for (int i = lane; i < T.ncomp * KC; i += 32) {
            const int c = i / KC, q = i - c * KC;
            const SComp cp = comps[c];
            const DGroup G = a.groups[cp.group];
            float* dst = sZ + i * XB;
            if (u0 + XB <= T.c_src && q0 + q < a.K)
                cp_async16(dst, a.Zbar + a.n_nodes * G.z_off + (nl * G.d_dst + cp.o) * (int64_t)G.D + cp.koff +
                                    (int64_t)(q0 + q) * T.c_src + u0);
            else
                *reinterpret_cast<float4*>(dst) = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    } else {
        for (int i = lane; i < T.ncomp * KC * XB; i += 32) {
            const int uu = i % XB, cq = i / XB;
            const int c = cq / KC, q = cq - c * KC;
            const SComp cp = comps[c];
            const DGroup G = a.groups[cp.group];
            float* dst = sZ + i;
            if (u0 + uu < T.c_src && q0 + q < a.K)
                cp_async4(dst, a.Zbar + a.n_nodes * G.z_off + (nl * G.d_dst + cp.o) * (int64_t)G.D + cp.koff +
                                   (int64_t)(q0 + q) * T.c_src + u0 + uu);
            else
                *dst = 0.f;
        }
    }
    cp_async_commit();
}

template <int DS>
__device__ __forceinline__ void load_rows(const float* xrow, int c_src, int d_src, bool vec_ok, int u0, bool on,
                                          float (&xs)[DS][XB]) {
#pragma unroll
    for (int s = 0; s < DS; ++s) {
        if (on && s < d_src) {
            const float* p = xrow + s * c_src + u0;
            if (vec_ok && u0 + XB <= c_src) {
                const float4 t = __ldg(reinterpret_cast<const float4*>(p));
                xs[s][0] = t.x; xs[s][1] = t.y; xs[s][2] = t.z; xs[s][3] = t.w;
            } else {
#pragma unroll
                for (int v = 0; v < XB; ++v) xs[s][v] = (u0 + v < c_src) ? __ldg(p + v) : 0.f;
            }
        } else {
#pragma unroll
            for (int v = 0; v < XB; ++v) xs[s][v] = 0.f;
        }
    }
}

// One task for this lane's edge.
template <int CAP, int KC, int DS, bool DUAL>
__device__ __forceinline__ void run_task(const EdgeArgs& a, const STask T, const int64_t nl, const int64_t sn,
                                         const float* sY, const float* sVY, float* sGY, float* sZ0, float* sZ1,
                                         const float* sPhi, const float* sVphi, float* sGphi, const int lane) {
    const SComp* comps = a.comps + T.comp_begin;
    const int ncomp = T.ncomp;
    const bool has_vx = DUAL && a.vsrc != nullptr, has_vY = DUAL && a.vY != nullptr, has_vphi = DUAL && a.vphi != nullptr;
    const bool vec_ok = ((T.src_off | T.c_src | a.C_src) & 3) == 0;
    // M (and dM) entries of the task's components for this lane's edge, straight into registers
    float m[CAP][DS], dm[CAP][DS], G[CAP][DS];
#pragma unroll
    for (int c = 0; c < CAP; ++c) {
        SComp cp{};
        if (c < ncomp) cp = comps[c];
#pragma unroll
        for (int s = 0; s < DS; ++s) {
            float v = 0.f, dv = 0.f;
            if (c < ncomp && s < T.d_src) {
                const int t = cp.tab0 + s * cp.tstride;
                const int t0 = __ldg(a.tab_ptr + t), t1 = __ldg(a.tab_ptr + t + 1);
                for (int k = t0; k < t1; ++k) {
                    const float cf = __ldg(a.tab_coef + k);
                    const int bb = (cp.sh_off + __ldg(a.tab_idx + k)) * 32 + lane;
                    v = fmaf(cf, sY[bb], v);
                    if (has_vY) dv = fmaf(cf, sVY[bb], dv);
                }
            }
            m[c][s] = v; dm[c][s] = dv; G[c][s] = 0.f;
        }
    }
    const float* xrow = a.src + sn * a.C_src + T.src_off;
    const float* vxrow = has_vx ? a.vsrc + sn * a.C_src + T.src_off : xrow;
    const int nblk = (T.c_src + XB - 1) / XB;

    for (int q0 = 0; q0 < a.K; q0 += KC) {
        float ph[KC], vph[KC], gp[KC];
#pragma unroll
        for (int q = 0; q < KC; ++q) {
            ph[q] = sPhi[(q0 + q) * 32 + lane];
            vph[q] = has_vphi ? sVphi[(q0 + q) * 32 + lane] : 0.f;
            gp[q] = 0.f;
        }
        stage_zbar<CAP, KC>(a, T, comps, nl, 0, q0, sZ0, lane);
        float xn[DS][XB], vxn[DS][XB];
        load_rows<DS>(xrow, T.c_src, T.d_src, vec_ok, 0, true, xn);
        load_rows<DS>(vxrow, T.c_src, T.d_src, vec_ok, 0, has_vx, vxn);
        for (int blk = 0; blk < nblk; ++blk) {
            const int u0 = blk * XB;
            float* sZ = (blk & 1) ? sZ1 : sZ0;
            float xs[DS][XB], vxs[DS][XB];
#pragma unroll
            for (int s = 0; s < DS; ++s)
#pragma unroll
                for (int v = 0; v < XB; ++v) { xs[s][v] = xn[s][v]; vxs[s][v] = vxn[s][v]; }
            if (blk + 1 < nblk) {     // sender rows of the next block are requested before this one is consumed
                load_rows<DS>(xrow, T.c_src, T.d_src, vec_ok, u0 + XB, true, xn);
                if (DUAL) load_rows<DS>(vxrow, T.c_src, T.d_src, vec_ok, u0 + XB, has_vx, vxn);
            }
            cp_async_wait_all();
            __syncwarp();
            if (blk + 1 < nblk) stage_zbar<CAP, KC>(a, T, comps, nl, u0 + XB, q0, (blk & 1) ? sZ0 : sZ1, lane);
#pragma unroll
            for (int c = 0; c < CAP; ++c) {
                if (c < ncomp) {
                    float Co[XB], Cb[XB], Cbv[XB];
#pragma unroll
                    for (int uu = 0; uu < XB; ++uu) {
                        float v = 0.f;
#pragma unroll
                        for (int s = 0; s < DS; ++s) {
                            if (!DUAL) v = fmaf(xs[s][uu], m[c][s], v);
                            else {
                                if (has_vx) v = fmaf(vxs[s][uu], m[c][s], v);
                                if (has_vY) v = fmaf(xs[s][uu], dm[c][s], v);
                            }
                        }
                        Co[uu] = v; Cb[uu] = 0.f; Cbv[uu] = 0.f;
                    }
                    const float4* z4 = reinterpret_cast<const float4*>(sZ + c * KC * XB);
#pragma unroll
                    for (int q = 0; q < KC; ++q) {
                        const float4 z = z4[q];       // the XB multiplicities of (component c, q)
                        const float zz[XB] = {z.x, z.y, z.z, z.w};
#pragma unroll
                        for (int uu = 0; uu < XB; ++uu) {
                            gp[q] = fmaf(zz[uu], Co[uu], gp[q]);
                            Cb[uu] = fmaf(ph[q], zz[uu], Cb[uu]);
                            if (has_vphi) Cbv[uu] = fmaf(vph[q], zz[uu], Cbv[uu]);
                        }
                    }
#pragma unroll
                    for (int uu = 0; uu < XB; ++uu) {
#pragma unroll
                        for (int s = 0; s < DS; ++s) {
                            if (!DUAL) G[c][s] = fmaf(xs[s][uu], Cb[uu], G[c][s]);
                            else {
                                if (has_vx) G[c][s] = fmaf(vxs[s][uu], Cb[uu], G[c][s]);
                                if (has_vphi) G[c][s] = fmaf(xs[s][uu], Cbv[uu], G[c][s]);
                            }
                        }
                    }
                }
            }
            __syncwarp();   // everyone is done with sZ before it is overwritten two blocks later
        }
#pragma unroll
        for (int q = 0; q < KC; ++q) sGphi[(q0 + q) * 32 + lane] += gp[q];
    }
    // gY_e[b] += c[s,b,o] * G[(path,o)][s]: the same sparse entries that built M, used transposed
    if (a.Y_mode) {
#pragma unroll
        for (int c = 0; c < CAP; ++c) {
            if (c < ncomp) {
                const SComp cp = comps[c];
#pragma unroll
                for (int s = 0; s < DS; ++s) {
                    if (s < T.d_src) {
                        const int t = cp.tab0 + s * cp.tstride;
                        const int t0 = __ldg(a.tab_ptr + t), t1 = __ldg(a.tab_ptr + t + 1);
                        for (int k = t0; k < t1; ++k)
                            sGY[(cp.sh_off + __ldg(a.tab_idx + k)) * 32 + lane] += __ldg(a.tab_coef + k) * G[c][s];
                    }
                }
            }
        }
    }
}

template <int CAP, int KC, int DS, bool DUAL>
__global__ void __launch_bounds__(EW * 32, (DUAL || KC == 16) ? 1 : 2)
k_edge_pass(const EdgeArgs a, const int t_begin, const int t_count) {
    extern __shared__ float smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int Kp = (a.K + KC - 1) / KC * KC;
    float* base = smem + (size_t)warp * a.warp_floats;
    float* sY = base;                       // [dsh][32]
    float* sGY = sY + a.dsh * 32;           // [dsh][32]
    float* sPhi = sGY + a.dsh * 32;         // [Kp][32]
    float* sGphi = sPhi + Kp * 32;          // [Kp][32]
    float* sZ0 = sGphi + Kp * 32;           // Zbar slab, two buffers
    float* sZ1 = sZ0 + a.zslab;
    float* sVY = sZ1 + a.zslab;             // DUAL: [dsh][32]
    float* sVphi = sVY + a.dsh * 32;        // DUAL: [Kp][32]
    const bool has_vY = DUAL && a.vY != nullptr, has_vphi = DUAL && a.vphi != nullptr;

    // One CTA per receiver; its warps share the receiver's tasks (warp w takes tasks w, w+nw, ...), each
    // accumulating partial gphi / gY of the same 32 edges in its own stage; the partials are then summed
    // across warps in a fixed order by the owner thread of each output element.
    const int nw = blockDim.x >> 5;
    for (int64_t nl = blockIdx.x; nl < a.n_nodes; nl += gridDim.x) {
        const int64_t node = a.node0 + nl;
        int64_t seg0, seg1;
        seg_bounds(a.ev.ptr, node, a.ev.E, a.status, seg0, seg1);
        for (int64_t b0 = seg0; b0 < seg1; b0 += 32) {
            const int64_t e = b0 + lane;
            const bool valid = e < seg1;
            int64_t sn = (int64_t)a.ev.col[valid ? e : seg0];   // e < seg1 <= E, or seg0 < seg1
            if (!id_ok(sn, a.ev.N, a.status)) sn = 0;          // reported; the edge then reads node 0
            for (int b = 0; b < a.dsh; ++b) {
                sY[b * 32 + lane] = valid ? a.Y[e * a.dsh + b] : 0.f;
                if (has_vY) sVY[b * 32 + lane] = valid ? a.vY[e * a.dsh + b] : 0.f;
                sGY[b * 32 + lane] = 0.f;
            }
            for (int q = 0; q < Kp; ++q) {
                sPhi[q * 32 + lane] = (valid && q < a.K) ? a.phi[e * a.K + q] : 0.f;
                if (has_vphi) sVphi[q * 32 + lane] = (valid && q < a.K) ? a.vphi[e * a.K + q] : 0.f;
                sGphi[q * 32 + lane] = 0.f;
            }
            __syncwarp();
            for (int t = warp; t < t_count; t += nw)
                run_task<CAP, KC, DS, DUAL>(a, a.tasks[t_begin + t], nl, sn, sY, sVY, sGY, sZ0, sZ1, sPhi, sVphi,
                                            sGphi, lane);
            __syncthreads();
            // fixed-order sum over the warps' partials; thread (warp, lane) owns the outputs of edge b0+lane
            // with index == warp (mod nw)
            if (valid) {
                if (a.phi_mode)
                    for (int q = warp; q < a.K; q += nw) {
                        float v = 0.f;
                        for (int w = 0; w < nw; ++w) v += smem[(size_t)w * a.warp_floats + (2 * a.dsh + Kp + q) * 32 + lane];
                        float* p = a.gphi + e * a.K + q;
                        *p = (a.phi_mode == 2 ? *p : 0.f) + v;
                    }
                if (a.Y_mode)
                    for (int b = warp; b < a.dsh; b += nw) {
                        float v = 0.f;
                        for (int w = 0; w < nw; ++w) v += smem[(size_t)w * a.warp_floats + (a.dsh + b) * 32 + lane];
                        float* p = a.gY + e * a.dsh + b;
                        *p = (a.Y_mode == 2 ? *p : 0.f) + v;
                    }
            }
            __syncthreads();
        }
    }
}

template <int CAP, int KC, int DS, bool DUAL>
cudaError_t launch_one(EdgeArgs a, int t_begin, int t_count, cudaStream_t s) {
    const int Kp = (a.K + KC - 1) / KC * KC;
    a.zslab = CAP * XB * KC;
    a.warp_floats = 2 * a.dsh * 32 + 2 * Kp * 32 + 2 * a.zslab + (DUAL ? a.dsh * 32 + Kp * 32 : 0);
    const int nw = std::max(1, std::min(EW, t_count));
    const size_t sh = (size_t)a.warp_floats * nw * sizeof(float);
    auto kern = k_edge_pass<CAP, KC, DS, DUAL>;
    if (sh > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
        if (e != cudaSuccess) return e;
    }
    const int grid = (int)std::min<int64_t>(a.n_nodes, 148 * 32);
    kern<<<grid, nw * 32, sh, s>>>(a, t_begin, t_count);
    return cudaGetLastError();
}

template <int KC, bool DUAL>
cudaError_t launch_class(int cls, const EdgeArgs& a, int t_begin, int t_count, cudaStream_t s) {
    constexpr int CAP = 4;
    switch (cls) {
        case 0: return launch_one<CAP, KC, 3, DUAL>(a, t_begin, t_count, s);
        case 1: return launch_one<CAP, KC, 5, DUAL>(a, t_begin, t_count, s);
        default: return launch_one<CAP, KC, 9, DUAL>(a, t_begin, t_count, s);
    }
}

}  // namespace

// Source-major task list of the edge pass (forward direction only): for every source irrep block the
// output components of all paths reading it, in tasks of at most 4, split evenly; sorted by class.
void build_edge_tasks(const sobek_plan* p, Direction& dir) {
    (void)p;
    const int CAP = 4;
    dir.etasks.clear();
    dir.ecomps.clear();
    dir.eclasses.clear();
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
        for (int t = 0; t < ntask; ++t) {
            const int c0 = t * per, c1 = std::min((int)all.size(), c0 + per);
            if (c1 <= c0) continue;
            STask T{};
            T.src_off = so; T.c_src = c_src; T.d_src = d_src; T.u0 = 0;
            T.ncomp = c1 - c0; T.comp_begin = (int)dir.ecomps.size(); T.cls = cls;
            dir.ecomps.insert(dir.ecomps.end(), all.begin() + c0, all.begin() + c1);
            dir.etasks.push_back(T);
        }
    }
    std::stable_sort(dir.etasks.begin(), dir.etasks.end(), [](const STask& x, const STask& y) { return x.cls < y.cls; });
    for (size_t i = 0; i < dir.etasks.size();) {
        size_t j = i;
        while (j < dir.etasks.size() && dir.etasks[j].cls == dir.etasks[i].cls) ++j;
        dir.eclasses.push_back({dir.etasks[i].cls, (int)i, (int)(j - i)});
        i = j;
    }
}

cudaError_t launch_edge_pass(const sobek_plan* p, const Direction& dir, const EdgeView& ev, int64_t node0,
                             int64_t n_nodes, const float* src, const float* vsrc, const float* Y, const float* vY,
                             const float* phi, const float* vphi, int dual, const float* Zbar, float* gphi,
                             float* gY, int phi_mode, int Y_mode, int* status, cudaStream_t s) {
    if (n_nodes <= 0 || dir.etasks.empty()) return cudaSuccess;
    EdgeArgs a{};
    a.status = status;
    a.tasks = dir.d_etasks; a.comps = dir.d_ecomps; a.groups = dir.d_groups;
    a.tab_ptr = p->d_tab_ptr; a.tab_idx = p->d_tab_idx; a.tab_coef = p->d_tab_coef;
    a.ev = ev; a.node0 = node0; a.n_nodes = n_nodes;
    a.src = src; a.vsrc = vsrc; a.Y = Y; a.vY = vY; a.phi = phi; a.vphi = vphi;
    a.Zbar = Zbar; a.gphi = gphi; a.gY = gY;
    a.K = p->K; a.dsh = p->dim_sh; a.C_src = dir.C_src;
    a.zvec = 1;      // koff = K * (sum of earlier multiplicities) and D = K * (sum of all): multiples of 4 iff every one is
    for (const DPath& P : dir.paths) if (P.c_src & 3) a.zvec = 0;
    const bool k16 = p->K > 8;
    bool first = true;
    for (const auto& c : dir.eclasses) {
        // the first class writes in the caller's mode, later classes accumulate
        a.phi_mode = phi_mode ? (first ? phi_mode : 2) : 0;
        a.Y_mode = Y_mode ? (first ? Y_mode : 2) : 0;
        first = false;
        KernelTimer kt(K_EDGE, s);
        cudaError_t e;
        if (k16) e = dual ? launch_class<16, true>(c.cls, a, c.begin, c.count, s) : launch_class<16, false>(c.cls, a, c.begin, c.count, s);
        else e = dual ? launch_class<8, true>(c.cls, a, c.begin, c.count, s) : launch_class<8, false>(c.cls, a, c.begin, c.count, s);
        count_launch();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace sobek
