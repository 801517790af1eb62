// Edge-stream kernels (sm_100a): the per-edge work of the convolution.
//
// k_stream<KC, DUAL> folds the edges of every node of a chunk into the bounded node state
//     Z[pi,u,q,o] = sum_e phi_e[q] * C_e[pi,u,o],   C_e[pi,u,o] = sum_s xs_e[u,s] * M_e[s,o]
// (Eqs. angular_path_contraction, receiver_state) and writes it as the split-bf16 (hi, lo)
// A operand of the tensor-core contraction with R.  M_e[s,o] = sum_b c[s,b,o] * Y_e[b] depends on
// the edge and the path only; it is expanded from the sparse table once per (edge, task).
// With DUAL it produces the directional state of the double backward in one pass,
//     dZ = sum_e ( vphi_e (x) C(x,Y) + phi_e (x) [ C(vx,Y) + C(x,vY) ] )
// (Eq. receiver_double_adjoint: dS).  The same kernel runs the sender-owned transposed traversal
// (source rows = output adjoints of the receivers, edges through the sender view).
//
// Work decomposition: one WARP per (node, task); a task is (path, block of 32*UB multiplicities,
// chunk of OC output components).  Lanes own multiplicities, so the sum over a node's edges needs
// no cross-lane reduction and no atomics, and sender rows are read with coalesced (vector) loads.
// Each lane keeps acc[UB][OC][KC] in registers; per edge the operands that are uniform across lanes
// (M_e, phi_e) come from the warp's private shared-memory stage as 128-bit broadcast loads.
// Warps never synchronise with each other.
#pragma once
#include <cuda_bf16.h>

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

struct StreamArgs {
    const DPath* paths;
    const STask* tasks;
    const DGroup* groups;
    const int64_t* zb_off;     // per group: bf16 state offset per node (elements)
    const int32_t* zb_ld;      // per group: row pitch of the bf16 state (elements)
    const int32_t* tab_ptr;
    const int32_t* tab_idx;
    const float* tab_coef;
    EdgeView ev;
    int64_t node0, n_nodes;
    int32_t n_tasks;
    const float* src;
    const float* vsrc;         // DUAL only; may be NULL
    const float* Y;
    const float* vY;           // DUAL only; may be NULL
    const float* phi;
    const float* vphi;         // DUAL only; may be NULL
    __nv_bfloat16* zh;
    __nv_bfloat16* zl;
    int32_t K, dsh, C_src;
    int32_t warp_floats;       // shared floats per warp
    int32_t ms_max;            // row pitch of the M stage
};

template <int UB>
__device__ __forceinline__ void load_x(const float* __restrict__ p, bool vec_ok, int u, int c_src, float (&v)[UB]) {
    if (UB == 4 && vec_ok) {
        if (u < c_src) {
            const float4 t = __ldg(reinterpret_cast<const float4*>(p));
            v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3 % UB] = t.w;
        } else {
#pragma unroll
            for (int i = 0; i < UB; ++i) v[i] = 0.f;
        }
    } else if (UB == 2 && vec_ok) {
        if (u < c_src) {
            const float2 t = __ldg(reinterpret_cast<const float2*>(p));
            v[0] = t.x; v[1 % UB] = t.y;
        } else {
#pragma unroll
            for (int i = 0; i < UB; ++i) v[i] = 0.f;
        }
    } else {
#pragma unroll
        for (int i = 0; i < UB; ++i) v[i] = (u + i < c_src) ? __ldg(p + i) : 0.f;
    }
}

template <int OC, int KC, int UB, int DS, bool DUAL>
__device__ __forceinline__ void run_task(const StreamArgs& a, const STask T, const int64_t nl, float* sm,
                                         const int lane) {
    const DPath P = a.paths[T.path];
    const int D = P.d_dst;
    const int MS = a.ms_max;
    const int YS = a.dsh + 1;
    // warp-private stage
    float* sM = sm;                               // [32][MS]
    float* sPhi = sM + 32 * MS;                   // [32][KC]
    float* sY = sPhi + 32 * KC;                   // [32][YS]
    int32_t* sSrc = (int32_t*)(sY + 32 * YS);     // [32] source node
    int32_t* sE = sSrc + 32;                      // [32] edge id
    float* sdM = (float*)(sE + 32);               // DUAL: [32][MS]
    float* sVphi = sdM + 32 * MS;                 // DUAL: [32][KC]
    float* sVY = sVphi + 32 * KC;                 // DUAL: [32][YS]

    const int64_t node = a.node0 + nl;
    const int64_t seg0 = a.ev.ptr[node], seg1 = a.ev.ptr[node + 1];
    const int u = T.u0 + lane * UB;
    const bool vec_ok = (UB == 1) || (((P.src_off | P.c_src | a.C_src) & (UB - 1)) == 0);
    const bool has_vx = DUAL && a.vsrc != nullptr, has_vY = DUAL && a.vY != nullptr,
               has_vphi = DUAL && a.vphi != nullptr;
    const int oc = T.oc;   // <= OC

    for (int q0 = 0; q0 < a.K; q0 += KC) {
        float acc[UB][OC][KC];
#pragma unroll
        for (int i = 0; i < UB; ++i)
#pragma unroll
            for (int o = 0; o < OC; ++o)
#pragma unroll
                for (int q = 0; q < KC; ++q) acc[i][o][q] = 0.f;

        for (int64_t b0 = seg0; b0 < seg1; b0 += 32) {
            const int nb = (int)min((int64_t)32, seg1 - b0);
            __syncwarp();
            // ---- stage the batch: lane <-> edge for ids, then flat copies of the Y and phi rows
            {
                int32_t e = 0, sn = 0;
                if (lane < nb) {
                    const int64_t pos = b0 + lane;
                    const int64_t eid = a.ev.perm ? (int64_t)a.ev.perm[pos] : pos;
                    e = (int32_t)eid;
                    sn = a.ev.transposed ? (int32_t)owner_of(a.ev.row_ptr, a.ev.N, eid) : a.ev.col[eid];
                }
                sE[lane] = e;
                sSrc[lane] = sn;
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
            // ---- expand M (and dM) for this lane's edge, own output components only
            if (lane < nb) {
                const float* y = sY + lane * YS + P.sh_off;
                const float* vy = sVY + lane * YS + P.sh_off;
                for (int s = 0; s < P.d_src; ++s)
                    for (int o = 0; o < oc; ++o) {
                        const int t = P.tabM + s * D + T.o0 + o;
                        const int t0 = __ldg(a.tab_ptr + t), t1 = __ldg(a.tab_ptr + t + 1);
                        float m = 0.f, dm = 0.f;
                        for (int k = t0; k < t1; ++k) {
                            const float c = __ldg(a.tab_coef + k);
                            const int b = __ldg(a.tab_idx + k);
                            m = fmaf(c, y[b], m);
                            if (has_vY) dm = fmaf(c, vy[b], dm);
                        }
                        sM[lane * MS + s * OC + o] = m;
                        if (has_vY) sdM[lane * MS + s * OC + o] = dm;
                    }
                if (oc < OC)
                    for (int s = 0; s < P.d_src; ++s)
                        for (int o = oc; o < OC; ++o) {
                            sM[lane * MS + s * OC + o] = 0.f;
                            if (has_vY) sdM[lane * MS + s * OC + o] = 0.f;
                        }
            }
            __syncwarp();
            // ---- fold the batch's edges.  The sender rows of PB edges are requested together so
            //      that PB gathers are in flight per warp, then the PB edges are folded one by one.
            constexpr int PB = (40 / (DS * UB * (DUAL ? 2 : 1))) >= 8 ? 8 : ((40 / (DS * UB * (DUAL ? 2 : 1))) >= 4 ? 4 :
                               ((40 / (DS * UB * (DUAL ? 2 : 1))) >= 2 ? 2 : 1));
            for (int el0 = 0; el0 < nb; el0 += PB) {
                float xb[PB][DS][UB], vxb[PB][DS][UB];
#pragma unroll
                for (int pe = 0; pe < PB; ++pe) {
                    const int el = min(el0 + pe, nb - 1);
                    const float* xr = a.src + (int64_t)sSrc[el] * a.C_src + P.src_off + u;
#pragma unroll
                    for (int s = 0; s < DS; ++s) {
                        if (s < P.d_src) load_x<UB>(xr + s * P.c_src, vec_ok, u, P.c_src, xb[pe][s]);
                        else {
#pragma unroll
                            for (int i = 0; i < UB; ++i) xb[pe][s][i] = 0.f;
                        }
                    }
                    if (DUAL) {
                        const float* vr = a.vsrc + (int64_t)sSrc[el] * a.C_src + P.src_off + u;
#pragma unroll
                        for (int s = 0; s < DS; ++s) {
                            if (has_vx && s < P.d_src) load_x<UB>(vr + s * P.c_src, vec_ok, u, P.c_src, vxb[pe][s]);
                            else {
#pragma unroll
                                for (int i = 0; i < UB; ++i) vxb[pe][s][i] = 0.f;
                            }
                        }
                    }
                }
#pragma unroll
                for (int pe = 0; pe < PB; ++pe) {
                const int el = el0 + pe;
                if (el < nb) {
                const float (&xs)[DS][UB] = xb[pe];
                const float (&vxs)[DS][UB] = vxb[pe];
                const float4* Me = reinterpret_cast<const float4*>(sM + el * MS);
                const float4* dMe = reinterpret_cast<const float4*>(sdM + el * MS);
                float C[UB][OC], dC[UB][OC];
#pragma unroll
                for (int i = 0; i < UB; ++i)
#pragma unroll
                    for (int o = 0; o < OC; ++o) { C[i][o] = 0.f; dC[i][o] = 0.f; }
                float4 mv = make_float4(0.f, 0.f, 0.f, 0.f), dmv = mv;
#pragma unroll
                for (int s = 0; s < DS; ++s) {
                    if (s < P.d_src) {
#pragma unroll
                        for (int o = 0; o < OC; ++o) {
                            const int t = s * OC + o;     // static after unrolling
                            if ((t & 3) == 0) { mv = Me[t >> 2]; if (has_vY) dmv = dMe[t >> 2]; }
                            const float m = (t & 3) == 0 ? mv.x : ((t & 3) == 1 ? mv.y : ((t & 3) == 2 ? mv.z : mv.w));
#pragma unroll
                            for (int i = 0; i < UB; ++i) C[i][o] = fmaf(xs[s][i], m, C[i][o]);
                            if (has_vx) {
#pragma unroll
                                for (int i = 0; i < UB; ++i) dC[i][o] = fmaf(vxs[s][i], m, dC[i][o]);
                            }
                            if (has_vY) {
                                const float dm = (t & 3) == 0 ? dmv.x : ((t & 3) == 1 ? dmv.y : ((t & 3) == 2 ? dmv.z : dmv.w));
#pragma unroll
                                for (int i = 0; i < UB; ++i) dC[i][o] = fmaf(xs[s][i], dm, dC[i][o]);
                            }
                        }
                    }
                }
                const float4* ph4 = reinterpret_cast<const float4*>(sPhi + el * KC);
                const float4* vph4 = reinterpret_cast<const float4*>(sVphi + el * KC);
#pragma unroll
                for (int q4 = 0; q4 < KC / 4; ++q4) {
                    const float4 pv = ph4[q4];
                    const float pq[4] = {pv.x, pv.y, pv.z, pv.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int i = 0; i < UB; ++i)
#pragma unroll
                            for (int o = 0; o < OC; ++o)
                                acc[i][o][4 * q4 + j] = fmaf(pq[j], DUAL ? dC[i][o] : C[i][o], acc[i][o][4 * q4 + j]);
                    if (has_vphi) {
                        const float4 vv = vph4[q4];
                        const float vq[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j)
#pragma unroll
                            for (int i = 0; i < UB; ++i)
#pragma unroll
                                for (int o = 0; o < OC; ++o)
                                    acc[i][o][4 * q4 + j] = fmaf(vq[j], C[i][o], acc[i][o][4 * q4 + j]);
                    }
                }
                }
                }
            }
        }
        // ---- write the state slice as bf16 (hi, lo)
        const int gi = T.group;
        const int64_t ld = a.zb_ld[gi];
        const int64_t gbase = a.n_nodes * a.zb_off[gi];
#pragma unroll
        for (int i = 0; i < UB; ++i) {
            if (u + i >= P.c_src) continue;
#pragma unroll
            for (int o = 0; o < OC; ++o) {
                if (o >= oc) continue;
                const int64_t off = gbase + (nl * D + T.o0 + o) * ld + P.koff + (int64_t)(u + i) * a.K + q0;
                if ((a.K & 7) == 0) {
#pragma unroll
                    for (int q = 0; q < KC; q += 8) {
                        if (q0 + q >= a.K) break;
                        __align__(16) __nv_bfloat16 h[8], l[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float v = acc[i][o][q + j];
                            h[j] = __float2bfloat16_rn(v);
                            l[j] = __float2bfloat16_rn(v - __bfloat162float(h[j]));
                        }
                        *reinterpret_cast<uint4*>(a.zh + off + q) = *reinterpret_cast<const uint4*>(h);
                        *reinterpret_cast<uint4*>(a.zl + off + q) = *reinterpret_cast<const uint4*>(l);
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < KC; ++q) {
                        if (q0 + q < a.K) {
                            const float v = acc[i][o][q];
                            const __nv_bfloat16 h = __float2bfloat16_rn(v);
                            a.zh[off + q] = h;
                            a.zl[off + q] = __float2bfloat16_rn(v - __bfloat162float(h));
                        }
                    }
                }
            }
        }
    }
}

constexpr int SW = 8;   // warps per CTA

constexpr int min_blocks(int OC, int KC, int UB, int DS, bool DUAL) {
    const int est = UB * OC * KC + 2 * DS * UB * (DUAL ? 2 : 1) + 2 * UB * OC + 40;
    return est <= 80 ? 3 : (est <= 124 ? 2 : 1);
}

template <int OC, int KC, int UB, int DS, bool DUAL>
__global__ void __launch_bounds__(SW * 32, min_blocks(OC, KC, UB, DS, DUAL))
k_stream(const StreamArgs a, const int t_begin, const int t_count) {
    extern __shared__ float smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* sm = smem + (size_t)warp * a.warp_floats;
    const int64_t total = a.n_nodes * t_count;
    for (int64_t item = (int64_t)blockIdx.x * SW + warp; item < total; item += (int64_t)gridDim.x * SW) {
        const int64_t nl = item / t_count;
        const STask T = a.tasks[t_begin + (int)(item - nl * t_count)];
        run_task<OC, KC, UB, DS, DUAL>(a, T, nl, sm, lane);
    }
}

template <int OC, int KC, int UB, int DS, bool DUAL>
cudaError_t launch_one(const StreamArgs& a, int t_begin, int t_count, size_t sh, cudaStream_t s) {
    auto kern = k_stream<OC, KC, UB, DS, DUAL>;
    if (sh > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
        if (e != cudaSuccess) return e;
    }
    const int64_t total = a.n_nodes * t_count;
    const int per_sm = min_blocks(OC, KC, UB, DS, DUAL);
    const int grid = (int)std::min<int64_t>((total + SW - 1) / SW, (int64_t)148 * per_sm * 2);
    kern<<<grid, SW * 32, sh, s>>>(a, t_begin, t_count);
    return cudaGetLastError();
}

template <int OC, int KC, int UB, bool DUAL>
cudaError_t launch_ds(int ds, const StreamArgs& a, int t_begin, int t_count, size_t sh, cudaStream_t s) {
    switch (ds) {
        case 3: return launch_one<OC, KC, UB, 3, DUAL>(a, t_begin, t_count, sh, s);
        case 5: return launch_one<OC, KC, UB, 5, DUAL>(a, t_begin, t_count, sh, s);
        default: return launch_one<OC, KC, UB, 9, DUAL>(a, t_begin, t_count, sh, s);
    }
}

// class key = (index(OC in {1,3,4,5}) * 3 + index(UB in {1,2,4})) * 3 + index(DS in {3,5,9})
template <int KC, bool DUAL>
cudaError_t launch_class(int cls, const StreamArgs& a, int t_begin, int t_count, size_t sh, cudaStream_t s) {
    const int ds = (cls % 3 == 0) ? 3 : (cls % 3 == 1 ? 5 : 9);
    switch (cls / 3) {
        case 0: return launch_ds<1, KC, 1, DUAL>(ds, a, t_begin, t_count, sh, s);
        case 1: return launch_ds<1, KC, 2, DUAL>(ds, a, t_begin, t_count, sh, s);
        case 2: return launch_ds<1, KC, 4, DUAL>(ds, a, t_begin, t_count, sh, s);
        case 3: return launch_ds<3, KC, 1, DUAL>(ds, a, t_begin, t_count, sh, s);
        case 4: return launch_ds<3, KC, 2, DUAL>(ds, a, t_begin, t_count, sh, s);
        case 5: return launch_ds<3, KC, (KC == 8 ? 4 : 1), DUAL>(ds, a, t_begin, t_count, sh, s);
        case 6: return launch_ds<4, KC, 1, DUAL>(ds, a, t_begin, t_count, sh, s);
        case 7: return launch_ds<4, KC, (KC == 8 ? 2 : 1), DUAL>(ds, a, t_begin, t_count, sh, s);
        case 9: return launch_ds<5, KC, 1, DUAL>(ds, a, t_begin, t_count, sh, s);
        case 10: return launch_ds<5, KC, (KC == 8 ? 2 : 1), DUAL>(ds, a, t_begin, t_count, sh, s);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace
}  // namespace sobek
