// Receiver-owned edge pass (sm_100a): the two edge outputs of the backward program
// (Section "Receiver-factorized backward"; Eqs. streamed_radial_adjoints,
// streamed_operand_adjoints written against the receiver state):
//     gphi_e[q] = sum_{pi,u,o} Zbar_i[pi,u,q,o] * C_e[pi,u,o]
//     gY_e[b]   = sum_{pi} sum_{s,o} c[s,b,o] * G_e[pi][s][o],   G_e[s][o] = sum_u xs_e[u,s] * Cbar_e[u,o]
//     Cbar_e[u,o] = sum_q phi_e[q] * Zbar_i[pi,u,q,o],   C_e[u,o] = sum_s xs_e[u,s] * M_e[s,o]
// with i the receiver of edge e and Zbar = gy R^T the adjoint of the receiver state.
//
// One WARP per receiver, LANES <-> EDGES of its segment (32 at a time): both outputs are per
// edge, so nothing is reduced across lanes and every output element has exactly one writer.
// Each lane reads its own sender row with 128-bit loads in blocks of XB multiplicities; the
// Zbar slab of the same multiplicities is shared by all lanes and staged once per warp in shared
// memory (cp.async, double buffered) and read with broadcast 128-bit loads.  One launch per
// output group; the first group overwrites gphi / gY, later groups accumulate (same owner lane).
#include <type_traits>

#include "internal.h"

namespace sobek {
namespace {

constexpr int EW = 8;   // warps per CTA (upper bound; fewer when the per-warp stage is large)

struct EdgeArgs {
    const DPath* paths;
    const int32_t* tab_ptr;
    const int32_t* tab_idx;
    const float* tab_coef;
    DGroup G;
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
    int K, Kpad, dsh, C_src, phi_mode, Y_mode;
    int max_ent;       // max over the group's paths of d_src*d_dst
    int warp_floats;   // shared floats per warp
    int zslab;         // floats of one Zbar slab buffer
};

__device__ __forceinline__ void cp_async4(float* dst, const float* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async16(float* dst, const float* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// Stage the Zbar slab of multiplicities [u0, u0+XB) and K-chunk [q0, q0+KC) of one path:
// sZ[(o*XB + uu)*KC + q]
template <int D, int KC, int XB>
__device__ __forceinline__ void stage_zbar(const EdgeArgs& a, const DPath& P, const float* Zg, int u0, int q0,
                                           float* sZ, int lane) {
    const bool vec = ((a.K & 3) == 0) && ((a.G.D & 3) == 0) && ((P.koff & 3) == 0);
    if (vec) {
        constexpr int per_row = XB * KC / 4;     // 16-byte pieces per (o) row
        for (int i = lane; i < D * per_row; i += 32) {
            const int o = i / per_row, r = i - o * per_row;
            const int uu = r / (KC / 4), q = (r - uu * (KC / 4)) * 4;
            float* dst = sZ + (o * XB + uu) * KC + q;
            if (u0 + uu < P.c_src && q0 + q < a.K)
                cp_async16(dst, Zg + (int64_t)o * a.G.D + P.koff + (int64_t)(u0 + uu) * a.K + q0 + q);
            else
                *reinterpret_cast<float4*>(dst) = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    } else {
        for (int i = lane; i < D * XB * KC; i += 32) {
            const int o = i / (XB * KC), r = i - o * (XB * KC);
            const int uu = r / KC, q = r - uu * KC;
            float* dst = sZ + i;
            if (u0 + uu < P.c_src && q0 + q < a.K)
                cp_async4(dst, Zg + (int64_t)o * a.G.D + P.koff + (int64_t)(u0 + uu) * a.K + q0 + q);
            else
                *dst = 0.f;
        }
    }
    cp_async_commit();
}

// Loads this lane's sender-row block xs[s][0..XB) for multiplicities [u0, u0+XB).
template <int DS, int XB>
__device__ __forceinline__ void load_rows(const float* xrow, const DPath& P, bool vec_ok, int u0, bool on,
                                          float (&xs)[DS][XB]) {
#pragma unroll
    for (int s = 0; s < DS; ++s) {
        if (on && s < P.d_src) {
            const float* p = xrow + s * P.c_src + u0;
            if (vec_ok && u0 + XB <= P.c_src) {
#pragma unroll
                for (int v = 0; v < XB / 4; ++v) {
                    const float4 t = __ldg(reinterpret_cast<const float4*>(p) + v);
                    xs[s][4 * v] = t.x; xs[s][4 * v + 1] = t.y; xs[s][4 * v + 2] = t.z; xs[s][4 * v + 3] = t.w;
                }
            } else {
#pragma unroll
                for (int v = 0; v < XB; ++v) xs[s][v] = (u0 + v < P.c_src) ? __ldg(p + v) : 0.f;
            }
        } else {
#pragma unroll
            for (int v = 0; v < XB; ++v) xs[s][v] = 0.f;
        }
    }
}

// One path, one output-component chunk [o0, o0+oc), all multiplicities, one K-chunk.
// Plain:  gp[q] += Zbar*C(x,Y);            G[s][o] += xs[s] * <phi, Zbar>
// DUAL :  gp[q] += Zbar*(C(vx,Y)+C(x,vY)); G[s][o] += vxs[s] * <phi, Zbar> + xs[s] * <vphi, Zbar>
// (the edge-local second-order terms that share Zbar, Eq. streamed_operand_second_adjoints).
template <int D, int DS, int OC, int KC, int XB, bool DUAL>
__device__ __forceinline__ void path_chunk(const EdgeArgs& a, const DPath& P, const float* Zg, const float* xrow,
                                           const float* vxrow, const int o0, const int oc, const int q0,
                                           const float* sMl, const float* sdMl, float* sZ0, float* sZ1,
                                           const float (&ph)[KC], const float (&vph)[KC], float (&gp)[KC],
                                           float (&G)[DS][OC], const int lane) {
    const bool vec_ok = ((P.src_off | P.c_src | a.C_src) & 3) == 0;
    const bool has_vx = DUAL && a.vsrc != nullptr, has_vY = DUAL && a.vY != nullptr, has_vphi = DUAL && a.vphi != nullptr;
    // M (and dM) columns of this chunk, for this lane's edge
    float m[DS][OC], dm[DS][OC];
#pragma unroll
    for (int s = 0; s < DS; ++s)
#pragma unroll
        for (int o = 0; o < OC; ++o) {
            const bool in = s < P.d_src && o < oc;
            m[s][o] = in ? sMl[(s * D + o0 + o) * 32] : 0.f;
            dm[s][o] = (in && has_vY) ? sdMl[(s * D + o0 + o) * 32] : 0.f;
        }

    const int nblk = (P.c_src + XB - 1) / XB;
    stage_zbar<D, KC, XB>(a, P, Zg, 0, q0, sZ0, lane);
    float xn[DS][XB], vxn[DS][XB];
    load_rows<DS, XB>(xrow, P, vec_ok, 0, true, xn);
    load_rows<DS, XB>(vxrow, P, vec_ok, 0, has_vx, vxn);
    for (int blk = 0; blk < nblk; ++blk) {
        const int u0 = blk * XB;
        float* sZ = (blk & 1) ? sZ1 : sZ0;
        float xs[DS][XB], vxs[DS][XB];
#pragma unroll
        for (int s = 0; s < DS; ++s)
#pragma unroll
            for (int v = 0; v < XB; ++v) { xs[s][v] = xn[s][v]; vxs[s][v] = vxn[s][v]; }
        // sender rows of the next block are requested before this block is consumed
        if (blk + 1 < nblk) {
            load_rows<DS, XB>(xrow, P, vec_ok, u0 + XB, true, xn);
            if (DUAL) load_rows<DS, XB>(vxrow, P, vec_ok, u0 + XB, has_vx, vxn);
        }
        cp_async_wait_all();
        __syncwarp();
        if (blk + 1 < nblk) stage_zbar<D, KC, XB>(a, P, Zg, u0 + XB, q0, (blk & 1) ? sZ0 : sZ1, lane);
#pragma unroll
        for (int o = 0; o < OC; ++o) {
            if (o < oc) {
#pragma unroll
                for (int uu = 0; uu < XB; ++uu) {
                    float Co = 0.f;
                    if (!DUAL) {
#pragma unroll
                        for (int s = 0; s < DS; ++s) Co = fmaf(xs[s][uu], m[s][o], Co);
                    } else {
#pragma unroll
                        for (int s = 0; s < DS; ++s) {
                            if (has_vx) Co = fmaf(vxs[s][uu], m[s][o], Co);
                            if (has_vY) Co = fmaf(xs[s][uu], dm[s][o], Co);
                        }
                    }
                    const float4* z4 = reinterpret_cast<const float4*>(sZ + ((o0 + o) * XB + uu) * KC);
                    float Cb = 0.f, Cbv = 0.f;
#pragma unroll
                    for (int q4 = 0; q4 < KC / 4; ++q4) {
                        const float4 z = z4[q4];
                        gp[4 * q4] = fmaf(z.x, Co, gp[4 * q4]);
                        gp[4 * q4 + 1] = fmaf(z.y, Co, gp[4 * q4 + 1]);
                        gp[4 * q4 + 2] = fmaf(z.z, Co, gp[4 * q4 + 2]);
                        gp[4 * q4 + 3] = fmaf(z.w, Co, gp[4 * q4 + 3]);
                        Cb = fmaf(ph[4 * q4], z.x, Cb);
                        Cb = fmaf(ph[4 * q4 + 1], z.y, Cb);
                        Cb = fmaf(ph[4 * q4 + 2], z.z, Cb);
                        Cb = fmaf(ph[4 * q4 + 3], z.w, Cb);
                        if (has_vphi) {
                            Cbv = fmaf(vph[4 * q4], z.x, Cbv);
                            Cbv = fmaf(vph[4 * q4 + 1], z.y, Cbv);
                            Cbv = fmaf(vph[4 * q4 + 2], z.z, Cbv);
                            Cbv = fmaf(vph[4 * q4 + 3], z.w, Cbv);
                        }
                    }
                    if (!DUAL) {
#pragma unroll
                        for (int s = 0; s < DS; ++s) G[s][o] = fmaf(xs[s][uu], Cb, G[s][o]);
                    } else {
#pragma unroll
                        for (int s = 0; s < DS; ++s) {
                            if (has_vx) G[s][o] = fmaf(vxs[s][uu], Cb, G[s][o]);
                            if (has_vphi) G[s][o] = fmaf(xs[s][uu], Cbv, G[s][o]);
                        }
                    }
                }
            }
        }
        __syncwarp();   // everyone is done with sZ before it is overwritten two blocks later
    }
}

template <int D, int DS, int OC, int KC, int XB, bool DUAL>
__device__ __forceinline__ void run_path(const EdgeArgs& a, const DPath& P, const float* Zg, const float* xrow,
                                         const float* vxrow, float* sM, float* sdM, float* sPhi, float* sVphi,
                                         float* sGphi, float* sGY, float* sZ0, float* sZ1, const int lane) {
    // output components in chunks of OC (one chunk when D <= 5)
    for (int o0 = 0; o0 < D; o0 += OC) {
        const int oc = min(OC, D - o0);
        float G[DS][OC];
#pragma unroll
        for (int s = 0; s < DS; ++s)
#pragma unroll
            for (int o = 0; o < OC; ++o) G[s][o] = 0.f;
        for (int q0 = 0; q0 < a.K; q0 += KC) {
            float ph[KC], vph[KC], gp[KC];
#pragma unroll
            for (int q = 0; q < KC; ++q) {
                ph[q] = sPhi[(q0 + q) * 32 + lane];
                vph[q] = (DUAL && a.vphi) ? sVphi[(q0 + q) * 32 + lane] : 0.f;
                gp[q] = 0.f;
            }
            path_chunk<D, DS, OC, KC, XB, DUAL>(a, P, Zg, xrow, vxrow, o0, oc, q0, sM + lane, sdM + lane, sZ0, sZ1,
                                                ph, vph, gp, G, lane);
#pragma unroll
            for (int q = 0; q < KC; ++q) sGphi[(q0 + q) * 32 + lane] += gp[q];
        }
        // park G behind the M area
        if (a.Y_mode) {
#pragma unroll
            for (int s = 0; s < DS; ++s)
#pragma unroll
                for (int o = 0; o < OC; ++o)
                    if (s < P.d_src && o < oc) sM[(a.max_ent + s * D + o0 + o) * 32 + lane] = G[s][o];
        }
    }
    if (a.Y_mode) {
        // gY_e[b] += sum_{(s,o)} c[s,b,o] * G[s][o]   (sparse adjoint table of the path)
        for (int b = 0; b < P.d_sh; ++b) {
            const int t0 = __ldg(a.tab_ptr + P.tabY + b), t1 = __ldg(a.tab_ptr + P.tabY + b + 1);
            float s = 0.f;
            for (int k = t0; k < t1; ++k)
                s = fmaf(__ldg(a.tab_coef + k), sM[(a.max_ent + __ldg(a.tab_idx + k)) * 32 + lane], s);
            sGY[(P.sh_off + b) * 32 + lane] += s;
        }
    }
}

template <int D, int KC, bool DUAL>
__global__ void __launch_bounds__(EW * 32) k_edge_pass(const EdgeArgs a) {
    extern __shared__ float smem[];
    constexpr int OC = D <= 5 ? D : (D == 7 ? 4 : 5);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nw = blockDim.x >> 5;
    float* base = smem + (size_t)warp * a.warp_floats;
    float* sM = base;                                  // [2*max_ent][32]  M, then G
    float* sY = sM + 2 * a.max_ent * 32;               // [dsh][32]
    float* sGY = sY + a.dsh * 32;                      // [dsh][32]
    float* sPhi = sGY + a.dsh * 32;                    // [Kpad][32]
    float* sGphi = sPhi + a.Kpad * 32;                 // [Kpad][32]
    float* sZ0 = sGphi + a.Kpad * 32;                  // Zbar slab, two buffers
    float* sZ1 = sZ0 + a.zslab;
    float* sdM = sZ1 + a.zslab;                        // DUAL: [max_ent][32]
    float* sVY = sdM + a.max_ent * 32;                 // DUAL: [dsh][32]
    float* sVphi = sVY + a.dsh * 32;                   // DUAL: [Kpad][32]
    const bool has_vY = DUAL && a.vY != nullptr, has_vphi = DUAL && a.vphi != nullptr;

    for (int64_t nl = (int64_t)blockIdx.x * nw + warp; nl < a.n_nodes; nl += (int64_t)gridDim.x * nw) {
        const int64_t node = a.node0 + nl;
        const int64_t seg0 = a.ev.ptr[node], seg1 = a.ev.ptr[node + 1];
        const float* Zg = a.Zbar + a.n_nodes * a.G.z_off + nl * D * (int64_t)a.G.D;
        for (int64_t b0 = seg0; b0 < seg1; b0 += 32) {
            const int64_t e = b0 + lane;
            const bool valid = e < seg1;
            const int64_t sn = (int64_t)a.ev.col[valid ? e : seg0];
            __syncwarp();
            for (int b = 0; b < a.dsh; ++b) {
                sY[b * 32 + lane] = valid ? a.Y[e * a.dsh + b] : 0.f;
                if (has_vY) sVY[b * 32 + lane] = valid ? a.vY[e * a.dsh + b] : 0.f;
                sGY[b * 32 + lane] = 0.f;
            }
            for (int q = 0; q < a.Kpad; ++q) {
                sPhi[q * 32 + lane] = (valid && q < a.K) ? a.phi[e * a.K + q] : 0.f;
                if (has_vphi) sVphi[q * 32 + lane] = (valid && q < a.K) ? a.vphi[e * a.K + q] : 0.f;
                sGphi[q * 32 + lane] = 0.f;
            }
            for (int pp = a.G.path_begin; pp < a.G.path_end; ++pp) {
                const DPath P = a.paths[pp];
                const int ne = P.d_src * D;
                // M (and dM) of this lane's edge: sM[(s*D+o)*32 + lane]
                for (int t = 0; t < ne; ++t) {
                    const int t0 = __ldg(a.tab_ptr + P.tabM + t), t1 = __ldg(a.tab_ptr + P.tabM + t + 1);
                    float s = 0.f, ds = 0.f;
                    for (int k = t0; k < t1; ++k) {
                        const float c = __ldg(a.tab_coef + k);
                        const int bb = (P.sh_off + __ldg(a.tab_idx + k)) * 32 + lane;
                        s = fmaf(c, sY[bb], s);
                        if (has_vY) ds = fmaf(c, sVY[bb], ds);
                    }
                    sM[t * 32 + lane] = s;
                    if (has_vY) sdM[t * 32 + lane] = ds;
                }
                const float* xrow = a.src + sn * a.C_src + P.src_off;
                const float* vxrow = (DUAL && a.vsrc) ? a.vsrc + sn * a.C_src + P.src_off : xrow;
                if (P.d_src <= 3) run_path<D, 3, OC, KC, 4, DUAL>(a, P, Zg, xrow, vxrow, sM, sdM, sPhi, sVphi, sGphi, sGY, sZ0, sZ1, lane);
                else if (P.d_src <= 5) run_path<D, 5, OC, KC, 4, DUAL>(a, P, Zg, xrow, vxrow, sM, sdM, sPhi, sVphi, sGphi, sGY, sZ0, sZ1, lane);
                else run_path<D, 9, OC, KC, 4, DUAL>(a, P, Zg, xrow, vxrow, sM, sdM, sPhi, sVphi, sGphi, sGY, sZ0, sZ1, lane);
            }
            if (valid) {
                if (a.phi_mode)
                    for (int q = 0; q < a.K; ++q) {
                        float* p = a.gphi + e * a.K + q;
                        *p = (a.phi_mode == 2 ? *p : 0.f) + sGphi[q * 32 + lane];
                    }
                if (a.Y_mode)
                    for (int b = 0; b < a.dsh; ++b) {
                        float* p = a.gY + e * a.dsh + b;
                        *p = (a.Y_mode == 2 ? *p : 0.f) + sGY[b * 32 + lane];
                    }
            }
        }
    }
}

template <typename F>
cudaError_t dispatch_d(int d, F&& f) {
    switch (d) {
        case 1: return f(std::integral_constant<int, 1>());
        case 3: return f(std::integral_constant<int, 3>());
        case 5: return f(std::integral_constant<int, 5>());
        case 7: return f(std::integral_constant<int, 7>());
        case 9: return f(std::integral_constant<int, 9>());
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

cudaError_t launch_edge_pass(const sobek_plan* p, const Direction& dir, const EdgeView& ev, int64_t node0,
                             int64_t n_nodes, const float* src, const float* vsrc, const float* Y, const float* vY,
                             const float* phi, const float* vphi, int dual, const float* Zbar, float* gphi,
                             float* gY, int phi_mode, int Y_mode, cudaStream_t s) {
    bool first = true;
    for (const DGroup& G : dir.groups) {
        if (G.path_end == G.path_begin) continue;
        EdgeArgs a{};
        a.paths = dir.d_paths;
        a.tab_ptr = p->d_tab_ptr; a.tab_idx = p->d_tab_idx; a.tab_coef = p->d_tab_coef;
        a.G = G; a.ev = ev; a.node0 = node0; a.n_nodes = n_nodes;
        a.src = src; a.vsrc = vsrc; a.Y = Y; a.vY = vY; a.phi = phi; a.vphi = vphi;
        a.Zbar = Zbar; a.gphi = gphi; a.gY = gY;
        a.K = p->K; a.dsh = p->dim_sh; a.C_src = dir.C_src;
        // the first group writes in the caller's mode, later groups accumulate
        a.phi_mode = phi_mode ? (first ? phi_mode : 2) : 0;
        a.Y_mode = Y_mode ? (first ? Y_mode : 2) : 0;
        first = false;
        const bool k16 = (p->K > 8);
        const int KC = k16 ? 16 : 8;
        a.Kpad = ((p->K + KC - 1) / KC) * KC;
        a.max_ent = 1;
        for (int k = G.path_begin; k < G.path_end; ++k) a.max_ent = std::max(a.max_ent, dir.paths[k].d_src * G.d_dst);
        a.zslab = G.d_dst * 4 * KC;    // XB = 4
        a.warp_floats = 2 * a.max_ent * 32 + 2 * a.dsh * 32 + 2 * a.Kpad * 32 + 2 * a.zslab;
        if (dual) a.warp_floats += a.max_ent * 32 + a.dsh * 32 + a.Kpad * 32;
        const int nw = (int)std::max<size_t>(1, std::min<size_t>(EW, (size_t)(100 * 1024) / ((size_t)a.warp_floats * 4)));
        const size_t sh = (size_t)a.warp_floats * nw * sizeof(float);
        const int grid = (int)std::min<int64_t>((n_nodes + nw - 1) / nw, 148 * 8);
        KernelTimer kt(K_EDGE, s);
        cudaError_t e = dispatch_d(G.d_dst, [&](auto dtag) -> cudaError_t {
            constexpr int D = decltype(dtag)::value;
#define SOBEK_EP_LAUNCH(KC_, DUAL_)                                                                           \
    do {                                                                                                      \
        auto kern = k_edge_pass<D, KC_, DUAL_>;                                                               \
        if (sh > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh); \
        kern<<<grid, nw * 32, sh, s>>>(a);                                                                    \
    } while (0)
            if (k16) { if (dual) SOBEK_EP_LAUNCH(16, true); else SOBEK_EP_LAUNCH(16, false); }
            else { if (dual) SOBEK_EP_LAUNCH(8, true); else SOBEK_EP_LAUNCH(8, false); }
#undef SOBEK_EP_LAUNCH
            return cudaGetLastError();
        });
        count_launch();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace sobek
