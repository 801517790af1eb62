// Edge-stream kernel (sm_100a): the per-edge work of the convolution, SOURCE-MAJOR.
//
// k_stream<CAP, KC, DS, DUAL> folds the edges of every node of a chunk into the bounded node state
//     Z[pi,u,q,o] = sum_e phi_e[q] * C_e[pi,u,o],   C_e[pi,u,o] = sum_s xs_e[u,s] * M_e[pi][s,o]
// (Eqs. angular_path_contraction, receiver_state) and writes it as the split-bf16 (hi, lo) A operand of
// the tensor-core contraction with R.  M_e[pi][s,o] = sum_b c[s,b,o] * Y_e[b] depends on the edge and
// the path only and is expanded from the sparse table once per (edge, task).
//
// A task is (source irrep block, 32 multiplicities, up to CAP output components taken from ALL paths
// that read this source block).  The gathered sender row xs_e[u, 0..d_src) is therefore loaded once per
// edge and reused by every path that consumes it, and each lane keeps acc[CAP][KC] in registers.
// One WARP per (node, task); lanes own multiplicities, so the sum over a node's edges needs no
// cross-lane reduction and no atomics; the operands that are uniform across lanes (M_e, phi_e) come from
// the warp's private shared-memory stage as 128-bit broadcast loads.  Warps never synchronise with
// each other.  With DUAL the kernel produces the directional state of the double backward in one pass,
//     dZ = sum_e ( vphi_e (x) C(x,Y) + phi_e (x) [ C(vx,Y) + C(x,vY) ] )       (Eq. receiver_double_adjoint).
// The same kernel runs the sender-owned transposed traversal.
#pragma once
#include <cuda_bf16.h>

#include "edge_stream_args.h"
#include "guard.cuh"
#include "internal.h"

namespace sobek {
namespace {

__device__ __forceinline__ int64_t owner_of(const int64_t* __restrict__ row_ptr, int64_t N, int64_t e) {
    int64_t lo = 0, hi = N;   // row_ptr[lo] <= e < row_ptr[hi]
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (__ldg(row_ptr + mid) <= e) lo = mid; else hi = mid;
    }
    return lo;
}

constexpr int S_EB = 16;       // edges staged per batch

template <int CAP, int KC, int DS, bool DUAL>
__device__ __forceinline__ void run_task(const StreamArgs& a, const STask T, const int64_t nl, float* sm,
                                         const int lane) {
    constexpr int DSP = DS <= 3 ? 4 : (DS <= 5 ? 8 : 12);   // padded d_src: M rows as float4s
    constexpr int MS = CAP * DSP;                           // floats of M per edge
    const int YS = a.dsh + 1;
    float* sM = sm;                                // [EB][MS]
    float* sPhi = sM + S_EB * MS;                  // [EB][KC]
    float* sY = sPhi + S_EB * KC;                  // [EB][YS]
    int32_t* sSrc = (int32_t*)(sY + S_EB * YS);    // [EB] source node
    int32_t* sE = sSrc + S_EB;                     // [EB] edge id
    float* sdM = (float*)(sE + S_EB);              // DUAL: [EB][MS]
    float* sVphi = sdM + S_EB * MS;                // DUAL: [EB][KC]
    float* sVY = sVphi + S_EB * KC;                // DUAL: [EB][YS]

    const int64_t node = a.node0 + nl;
    int64_t seg0, seg1;
    seg_bounds(a.ev.ptr, node, a.ev.E, a.status, seg0, seg1);
    const int u = T.u0 + lane;
    const bool act = u < T.c_src;
    const bool has_vx = DUAL && a.vsrc != nullptr, has_vY = DUAL && a.vY != nullptr,
               has_vphi = DUAL && a.vphi != nullptr;
    const SComp* comps = a.comps + T.comp_begin;
    const int ncomp = T.ncomp;

    for (int q0 = 0; q0 < a.K; q0 += KC) {
        float acc[CAP][KC];
#pragma unroll
        for (int c = 0; c < CAP; ++c)
#pragma unroll
            for (int q = 0; q < KC; ++q) acc[c][q] = 0.f;

        for (int64_t b0 = seg0; b0 < seg1; b0 += S_EB) {
            const int nb = (int)min((int64_t)S_EB, seg1 - b0);
            __syncwarp();
            if (lane < nb) {
                const int64_t pos = b0 + lane;
                // an id out of range is reported; the edge then reads edge 0 / node 0 (valid memory, wrong data)
                int64_t eid = a.ev.perm ? (int64_t)a.ev.perm[pos] : pos;
                if (!id_ok(eid, a.ev.E, a.status)) eid = 0;
                sE[lane] = (int32_t)eid;
                int64_t sn = a.ev.transposed ? owner_of(a.ev.row_ptr, a.ev.N, eid) : (int64_t)a.ev.col[eid];
                if (!id_ok(sn, a.ev.N, a.status)) sn = 0;
                sSrc[lane] = (int32_t)sn;
            }
            __syncwarp();
            for (int i = lane; i < nb * a.dsh; i += 32) {
                const int el = i / a.dsh, b = i - el * a.dsh;
                const int64_t g = (int64_t)sE[el] * a.dsh + b;
                sY[el * YS + b] = a.Y[g];
                if (has_vY) sVY[el * YS + b] = a.vY[g];
            }
            for (int i = lane; i < nb * KC; i += 32) {
                const int el = i / KC, q = i - el * KC;
                const bool in = q0 + q < a.K;
                const int64_t g = (int64_t)sE[el] * a.K + q0 + q;
                sPhi[i] = in ? a.phi[g] : 0.f;
                if (has_vphi) sVphi[i] = in ? a.vphi[g] : 0.f;
            }
            __syncwarp();
            // ---- expand M (and dM): lane <-> (edge = lane % 16, components of parity lane / 16)
            {
                const int el = lane & 15;
                if (el < nb) {
                    const float* y = sY + el * YS;
                    const float* vy = sVY + el * YS;
                    for (int c = lane >> 4; c < ncomp; c += 2) {
                        const SComp cp = comps[c];
                        for (int s = 0; s < DSP; ++s) {     // padded rows are written as zeros
                            const int t = cp.tab0 + s * cp.tstride;
                            int t0 = 0, t1 = 0;
                            if (s < T.d_src) { t0 = __ldg(a.tab_ptr + t); t1 = __ldg(a.tab_ptr + t + 1); }
                            float m = 0.f, dm = 0.f;
                            for (int k = t0; k < t1; ++k) {
                                const float cf = __ldg(a.tab_coef + k);
                                const int b = cp.sh_off + __ldg(a.tab_idx + k);
                                m = fmaf(cf, y[b], m);
                                if (has_vY) dm = fmaf(cf, vy[b], dm);
                            }
                            sM[el * MS + c * DSP + s] = m;
                            if (has_vY) sdM[el * MS + c * DSP + s] = dm;
                        }
                    }
                }
            }
            __syncwarp();
            // ---- fold the batch's edges; the sender rows of PB edges are requested together
            constexpr int PB = (24 / (DS * (DUAL ? 2 : 1))) >= 8 ? 8 : ((24 / (DS * (DUAL ? 2 : 1))) >= 4 ? 4 :
                               ((24 / (DS * (DUAL ? 2 : 1))) >= 2 ? 2 : 1));
            for (int el0 = 0; el0 < nb; el0 += PB) {
                float xb[PB][DS], vxb[PB][DS];
#pragma unroll
                for (int pe = 0; pe < PB; ++pe) {
                    const int el = min(el0 + pe, nb - 1);
                    const float* xr = a.src + (int64_t)sSrc[el] * a.C_src + T.src_off + u;
#pragma unroll
                    for (int s = 0; s < DS; ++s) xb[pe][s] = (act && s < T.d_src) ? __ldg(xr + s * T.c_src) : 0.f;
                    if (DUAL) {
                        const float* vr = a.vsrc + (int64_t)sSrc[el] * a.C_src + T.src_off + u;
#pragma unroll
                        for (int s = 0; s < DS; ++s) vxb[pe][s] = (has_vx && act && s < T.d_src) ? __ldg(vr + s * T.c_src) : 0.f;
                    }
                }
#pragma unroll
                for (int pe = 0; pe < PB; ++pe) {
                    const int el = el0 + pe;
                    if (el < nb) {
                        const float4* Me = reinterpret_cast<const float4*>(sM + el * MS);
                        const float4* dMe = reinterpret_cast<const float4*>(sdM + el * MS);
                        const float4* ph4 = reinterpret_cast<const float4*>(sPhi + el * KC);
                        const float4* vph4 = reinterpret_cast<const float4*>(sVphi + el * KC);
                        float ph[KC], vph[KC];
#pragma unroll
                        for (int q4 = 0; q4 < KC / 4; ++q4) {
                            const float4 t = ph4[q4];
                            ph[4 * q4] = t.x; ph[4 * q4 + 1] = t.y; ph[4 * q4 + 2] = t.z; ph[4 * q4 + 3] = t.w;
                            if (has_vphi) {
                                const float4 v = vph4[q4];
                                vph[4 * q4] = v.x; vph[4 * q4 + 1] = v.y; vph[4 * q4 + 2] = v.z; vph[4 * q4 + 3] = v.w;
                            }
                        }
#pragma unroll
                        for (int c = 0; c < CAP; ++c) {
                            if (c < ncomp) {
                                float C = 0.f, dC = 0.f;
#pragma unroll
                                for (int s4 = 0; s4 < DSP / 4; ++s4) {
                                    const float4 m = Me[c * (DSP / 4) + s4];
                                    const float mm[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
                                    for (int j = 0; j < 4; ++j)
                                        if (4 * s4 + j < DS) {
                                            C = fmaf(xb[pe][4 * s4 + j], mm[j], C);
                                            if (has_vx) dC = fmaf(vxb[pe][4 * s4 + j], mm[j], dC);
                                        }
                                    if (has_vY) {
                                        const float4 d = dMe[c * (DSP / 4) + s4];
                                        const float dd[4] = {d.x, d.y, d.z, d.w};
#pragma unroll
                                        for (int j = 0; j < 4; ++j)
                                            if (4 * s4 + j < DS) dC = fmaf(xb[pe][4 * s4 + j], dd[j], dC);
                                    }
                                }
                                const float Cm = DUAL ? dC : C;
#pragma unroll
                                for (int q = 0; q < KC; ++q) acc[c][q] = fmaf(ph[q], Cm, acc[c][q]);
                                if (has_vphi) {
#pragma unroll
                                    for (int q = 0; q < KC; ++q) acc[c][q] = fmaf(vph[q], C, acc[c][q]);
                                }
                            }
                        }
                    }
                }
            }
        }
        // ---- write the state slice as bf16 (hi, lo); contraction index k = koff + q*c_src + u
        if (act) {
#pragma unroll
            for (int c = 0; c < CAP; ++c) {
                if (c < ncomp) {
                    const SComp cp = comps[c];
                    const int64_t ld = a.zb_ld[cp.group];
                    const int64_t off = a.n_nodes * a.zb_off[cp.group] + (nl * cp.d_dst + cp.o) * ld + cp.koff + u;
#pragma unroll
                    for (int q = 0; q < KC; ++q) {
                        if (q0 + q < a.K) {
                            const float v = acc[c][q];
                            const __nv_bfloat16 h = __float2bfloat16_rn(v);
                            const int64_t o = off + (int64_t)(q0 + q) * T.c_src;
                            ((__nv_bfloat16*)a.zh)[o] = h;
                            ((__nv_bfloat16*)a.zl)[o] = __float2bfloat16_rn(v - __bfloat162float(h));
                        }
                    }
                }
            }
        }
    }
}

constexpr int SW = 8;   // warps per CTA

template <int CAP, int KC, int DS, bool DUAL>
__global__ void __launch_bounds__(SW * 32, (DUAL ? 2 : 3) - (KC == 16 ? 1 : 0))
k_stream(const StreamArgs a, const int t_begin, const int t_count) {
    extern __shared__ float smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* sm = smem + (size_t)warp * a.warp_floats;
    const int64_t total = a.n_nodes * t_count;
    for (int64_t item = (int64_t)blockIdx.x * SW + warp; item < total; item += (int64_t)gridDim.x * SW) {
        const int64_t nl = item / t_count;
        const STask T = a.tasks[t_begin + (int)(item - nl * t_count)];
        run_task<CAP, KC, DS, DUAL>(a, T, nl, sm, lane);
    }
}

template <int CAP, int KC, int DS, bool DUAL>
cudaError_t launch_one(StreamArgs a, int t_begin, int t_count, cudaStream_t s) {
    constexpr int DSP = DS <= 3 ? 4 : (DS <= 5 ? 8 : 12);
    int wf = S_EB * CAP * DSP + S_EB * KC + S_EB * (a.dsh + 1) + 2 * S_EB;
    if (DUAL) wf += S_EB * CAP * DSP + S_EB * KC + S_EB * (a.dsh + 1);
    wf = (wf + 3) & ~3;
    a.warp_floats = wf;
    const size_t sh = (size_t)wf * SW * sizeof(float);
    auto kern = k_stream<CAP, KC, DS, DUAL>;
    if (sh > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
        if (e != cudaSuccess) return e;
    }
    const int64_t total = a.n_nodes * t_count;
    const int grid = (int)std::min<int64_t>((total + SW - 1) / SW, (int64_t)148 * 8);
    kern<<<grid, SW * 32, sh, s>>>(a, t_begin, t_count);
    return cudaGetLastError();
}

// class = index(DS in {3,5,9})
template <int KC, bool DUAL>
cudaError_t launch_class(int cls, const StreamArgs& a, int t_begin, int t_count, cudaStream_t s) {
    constexpr int CAP = KC == 8 ? 4 : 3;
    switch (cls) {
        case 0: return launch_one<CAP, KC, 3, DUAL>(a, t_begin, t_count, s);
        case 1: return launch_one<CAP, KC, 5, DUAL>(a, t_begin, t_count, s);
        default: return launch_one<CAP, KC, 9, DUAL>(a, t_begin, t_count, s);
    }
}

}  // namespace
}  // namespace sobek
