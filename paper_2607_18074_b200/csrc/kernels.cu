// Device kernels of the streaming convolution (sm_100a).
//
//   k_pack_R<UNPACK>      : the accumulated R adjoint, kept per group as gRp_g[(pi,u,q), w],
//                           back into the layout of R[K, N_w]
//   k_edge_pass           : receiver-owned edge derivatives gphi_e, gY_e
//                           (Section "Receiver-factorized backward")
// (the edge stream lives in edge_stream*.cu, the node-side contractions in gemm_tc.cu)
#include <stdio.h>

#include <atomic>
#include <type_traits>
#include <vector>

#include "internal.h"

namespace sobek {

static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// Optional per-kernel-class timing (off by default): every launch is bracketed by two CUDA
// events on the launching stream; sobek_timing_collect sums the elapsed times per class.
static bool g_timing = false;
struct TimedLaunch { cudaEvent_t a, b; int cls; };
static std::vector<TimedLaunch> g_timed;
static const char* kClassNames[K_NCLASS] = {"pack_R", "edge_stream_state", "node_gemm", "edge_pass", "fill"};

KernelTimer::KernelTimer(int cls, cudaStream_t s) : cls_(cls), s_(s), on_(g_timing) {
    if (!on_) return;
    if (cudaEventCreate(&a_) != cudaSuccess || cudaEventCreate(&b_) != cudaSuccess) { on_ = false; return; }
    cudaEventRecord(a_, s_);
}
KernelTimer::~KernelTimer() {
    if (!on_) return;
    cudaEventRecord(b_, s_);
    g_timed.push_back(TimedLaunch{a_, b_, cls_});
}

}  // namespace sobek

extern "C" int64_t sobek_launch_count(void) { return sobek::g_launches.load(); }

extern "C" int sobek_timing_enable(int on) {
    sobek::g_timing = on != 0;
    return SOBEK_OK;
}

extern "C" int sobek_timing_classes(void) { return sobek::K_NCLASS; }

extern "C" const char* sobek_timing_class_name(int cls) {
    return (cls >= 0 && cls < sobek::K_NCLASS) ? sobek::kClassNames[cls] : "";
}

extern "C" int sobek_timing_collect(double* total_ms, int64_t* launches) {
    if (!total_ms || !launches) return SOBEK_ERR_INVALID_ARG;
    for (int c = 0; c < sobek::K_NCLASS; ++c) { total_ms[c] = 0.0; launches[c] = 0; }
    int rc = SOBEK_OK;
    for (auto& t : sobek::g_timed) {
        float ms = 0.f;
        if (cudaEventSynchronize(t.b) != cudaSuccess || cudaEventElapsedTime(&ms, t.a, t.b) != cudaSuccess) {
            (void)cudaGetLastError();
            rc = SOBEK_ERR_CUDA;
        }
        total_ms[t.cls] += ms;
        launches[t.cls] += 1;
        cudaEventDestroy(t.a);
        cudaEventDestroy(t.b);
    }
    sobek::g_timed.clear();
    return rc;
}

namespace sobek {
namespace {

// ------------------------------------------------------------------------------------
// small helpers
// ------------------------------------------------------------------------------------
__device__ __forceinline__ int64_t owner_of_edge(const int64_t* __restrict__ row_ptr, int64_t N,
                                                 int64_t e) {
    // largest i with row_ptr[i] <= e   (rows may be empty)
    int64_t lo = 0, hi = N;   // invariant: row_ptr[lo] <= e < row_ptr[hi]
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (__ldg(row_ptr + mid) <= e) lo = mid; else hi = mid;
    }
    return lo;
}

__global__ void k_fill_zero(float* __restrict__ p, int64_t n) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t st = (int64_t)gridDim.x * blockDim.x;
    for (; i < n; i += st) p[i] = 0.f;
}

// ------------------------------------------------------------------------------------
// R re-layout.  One blockIdx.y per path; element (us, q, n) of the path's slab:
//   forward    : us = u (input mult.), n = w      Rp[rp_off + (koff + u*K + q)*c_out + w]
//   transposed : us = w (output mult.), n = u     Rt[rp_off + (koff + w*K + q)*c_in  + u]
// both read/write R[q*N_w + w_off + u*c_out + w].
// ------------------------------------------------------------------------------------
template <bool UNPACK>
__global__ void k_pack_R(const DPath* __restrict__ paths, int transposed, int K, int64_t N_w,
                         const float* __restrict__ src, float* __restrict__ dst) {
    const DPath P = paths[blockIdx.y];
    const int64_t total = (int64_t)K * P.c_src * P.c_dst;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(i % P.c_dst);
        const int64_t r = i / P.c_dst;
        const int q = (int)(r % K);
        const int us = (int)(r / K);
        const int u = transposed ? n : us, w = transposed ? us : n;
        const int64_t ri = (int64_t)q * N_w + P.w_off + (int64_t)u * P.c_out + w;
        const int64_t pi = P.rp_off + ((int64_t)P.koff + (int64_t)us * K + q) * P.c_dst + n;
        if (UNPACK) dst[ri] = src[pi]; else dst[pi] = src[ri];
    }
}

// ------------------------------------------------------------------------------------
// Receiver-owned edge pass (one launch per group).
// One warp per receiver; lanes <-> edges of its segment, 32 at a time, so that the two edge
// outputs need no cross-lane reduction:
//   gphi_e[q] = sum_{pi,u,o} Zbar[pi,u,q,o] * C_e[pi,u,o]
//   gY_e[b]   = sum_{pi} sum_{s,o} c[s,b,o] * G_e[pi][s][o],  G_e[s][o] = sum_u xs[u,s] * Cbar_e[u,o],
//   Cbar_e[u,o] = sum_q phi_e[q] * Zbar[pi,u,q,o]
// Sender rows and the Zbar slab of UCH multiplicities are staged in shared memory per warp.
// ------------------------------------------------------------------------------------
constexpr int EP_WARPS = 4;
constexpr int EP_UCH = 8;

struct EdgeArgs {
    const DPath* paths;
    const int32_t* tab_ptr;
    const int32_t* tab_idx;
    const float* tab_coef;
    DGroup G;
    EdgeView ev;
    int64_t node0, n_nodes;
    const float* src;
    const float* Y;
    const float* phi;
    const float* Zbar;
    float* gphi;
    float* gY;
    int K, Kpad, dsh, C_src, phi_mode, Y_mode;
    int max_dsrc, max_ent;     // over the group's paths
    int warp_floats;           // shared floats per warp
};

template <int D_DST, int KC>
__global__ void __launch_bounds__(EP_WARPS * 32) k_edge_pass(const EdgeArgs a) {
    extern __shared__ float smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t nl = (int64_t)blockIdx.x * EP_WARPS + warp;   // node index inside the chunk
    if (nl >= a.n_nodes) return;                                 // whole warp leaves; no CTA barriers used
    float* base = smem + (size_t)warp * a.warp_floats;
    float* sX = base;                                            // [max_dsrc*UCH][33]
    float* sZ = sX + a.max_dsrc * EP_UCH * 33;                   // [UCH][D_DST][KC]
    float* sM = sZ + EP_UCH * D_DST * KC;                        // [max_ent][32]   (also G)
    float* sY = sM + a.max_ent * 32;                             // [dsh][32]
    float* sGY = sY + a.dsh * 32;                                // [dsh][32]
    float* sPhi = sGY + a.dsh * 32;                              // [Kpad][32]
    float* sGphi = sPhi + a.Kpad * 32;                           // [Kpad][32]
    int64_t* sSrc = (int64_t*)(sGphi + a.Kpad * 32);             // [32]

    const int64_t node = a.node0 + nl;
    const int64_t seg0 = a.ev.ptr[node], seg1 = a.ev.ptr[node + 1];
    const float* Zg = a.Zbar + a.n_nodes * a.G.z_off + nl * D_DST * (int64_t)a.G.D;

    for (int64_t b0 = seg0; b0 < seg1; b0 += 32) {
        const int64_t e = b0 + lane;            // fwd direction only: position == edge id
        const bool valid = e < seg1;
        __syncwarp();
        sSrc[lane] = valid ? (int64_t)a.ev.col[e] : (int64_t)a.ev.col[seg0];
        for (int b = 0; b < a.dsh; ++b) {
            sY[b * 32 + lane] = valid ? a.Y[e * a.dsh + b] : 0.f;
            sGY[b * 32 + lane] = 0.f;
        }
        for (int q = 0; q < a.Kpad; ++q) {
            sPhi[q * 32 + lane] = (valid && q < a.K) ? a.phi[e * a.K + q] : 0.f;
            sGphi[q * 32 + lane] = 0.f;
        }
        __syncwarp();
        for (int pp = a.G.path_begin; pp < a.G.path_end; ++pp) {
            const DPath P = a.paths[pp];
            const int ne = P.d_src * D_DST;
            // M for this lane's edge
            for (int t = 0; t < ne; ++t) {
                const int t0 = a.tab_ptr[P.tabM + t], t1 = a.tab_ptr[P.tabM + t + 1];
                float s = 0.f;
                for (int k = t0; k < t1; ++k)
                    s = fmaf(a.tab_coef[k], sY[(P.sh_off + a.tab_idx[k]) * 32 + lane], s);
                sM[t * 32 + lane] = s;
            }
            float G[9][D_DST];
#pragma unroll
            for (int s = 0; s < 9; ++s)
#pragma unroll
                for (int o = 0; o < D_DST; ++o) G[s][o] = 0.f;

            for (int q0 = 0; q0 < a.K; q0 += KC) {
                float ph[KC], gp[KC];
#pragma unroll
                for (int q = 0; q < KC; ++q) { ph[q] = sPhi[(q0 + q) * 32 + lane]; gp[q] = 0.f; }
                for (int u0 = 0; u0 < P.c_src; u0 += EP_UCH) {
                    const int nu = min(EP_UCH, P.c_src - u0);
                    __syncwarp();
                    // stage sender rows: sX[(s*UCH+uu)*33 + edge]
                    for (int i = lane; i < 32 * P.d_src * EP_UCH; i += 32) {
                        const int uu = i % EP_UCH;
                        const int r = i / EP_UCH;
                        const int s = r % P.d_src;
                        const int el = r / P.d_src;
                        float v = 0.f;
                        if (uu < nu) v = __ldg(a.src + sSrc[el] * a.C_src + P.src_off + s * P.c_src + u0 + uu);
                        sX[(s * EP_UCH + uu) * 33 + el] = v;
                    }
                    // stage Zbar slab: sZ[(uu*D_DST+o)*KC + q]
                    for (int i = lane; i < EP_UCH * D_DST * KC; i += 32) {
                        const int q = i % KC;
                        const int r = i / KC;
                        const int uu = r % EP_UCH;
                        const int o = r / EP_UCH;
                        float v = 0.f;
                        if (uu < nu && q0 + q < a.K)
                            v = Zg[(int64_t)o * a.G.D + P.koff + (int64_t)(u0 + uu) * a.K + q0 + q];
                        sZ[(uu * D_DST + o) * KC + q] = v;
                    }
                    __syncwarp();
                    for (int uu = 0; uu < nu; ++uu) {
                        float xs[9];
#pragma unroll
                        for (int s = 0; s < 9; ++s) xs[s] = (s < P.d_src) ? sX[(s * EP_UCH + uu) * 33 + lane] : 0.f;
#pragma unroll
                        for (int o = 0; o < D_DST; ++o) {
                            float Co = 0.f;
#pragma unroll
                            for (int s = 0; s < 9; ++s)
                                if (s < P.d_src) Co = fmaf(xs[s], sM[(s * D_DST + o) * 32 + lane], Co);
                            const float* z = sZ + (uu * D_DST + o) * KC;
                            float Cb = 0.f;
#pragma unroll
                            for (int q = 0; q < KC; ++q) {
                                const float zq = z[q];
                                gp[q] = fmaf(zq, Co, gp[q]);
                                Cb = fmaf(ph[q], zq, Cb);
                            }
#pragma unroll
                            for (int s = 0; s < 9; ++s)
                                if (s < P.d_src) G[s][o] = fmaf(xs[s], Cb, G[s][o]);
                        }
                    }
                }
#pragma unroll
                for (int q = 0; q < KC; ++q)
                    if (q0 + q < a.Kpad) sGphi[(q0 + q) * 32 + lane] += gp[q];
            }
            // G -> gY through the adjoint table (G parked in the M area)
            if (a.Y_mode) {
                __syncwarp();
#pragma unroll
                for (int s = 0; s < 9; ++s)
#pragma unroll
                    for (int o = 0; o < D_DST; ++o)
                        if (s < P.d_src) sM[(s * D_DST + o) * 32 + lane] = G[s][o];
                for (int b = 0; b < P.d_sh; ++b) {
                    const int t0 = a.tab_ptr[P.tabY + b], t1 = a.tab_ptr[P.tabY + b + 1];
                    float s = 0.f;
                    for (int k = t0; k < t1; ++k) s = fmaf(a.tab_coef[k], sM[a.tab_idx[k] * 32 + lane], s);
                    sGY[(P.sh_off + b) * 32 + lane] += s;
                }
            }
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

// ======================================================================================
// host launchers
// ======================================================================================
cudaError_t launch_fill_zero(float* p, int64_t n, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    const int blocks = (int)std::min<int64_t>((n + 255) / 256, 148 * 8);
    KernelTimer kt(K_FILL, s);
    k_fill_zero<<<blocks, 256, 0, s>>>(p, n);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_unpack_R(const sobek_plan* p, const Direction& dir, const float* Rp, float* R,
                            cudaStream_t s) {
    dim3 grid(32, (unsigned)dir.paths.size());
    KernelTimer kt(K_PACK, s);
    k_pack_R<true><<<grid, 256, 0, s>>>(dir.d_paths, 0, p->K, p->N_w, Rp, R);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_edge_pass(const sobek_plan* p, const Direction& dir, const EdgeView& ev,
                             int64_t node0, int64_t n_nodes, const float* src, const float* Y,
                             const float* phi, const float* Zbar, float* gphi, float* gY,
                             int phi_mode, int Y_mode, cudaStream_t s) {
    bool first = true;
    for (const DGroup& G : dir.groups) {
        if (G.path_end == G.path_begin) continue;
        EdgeArgs a;
        a.paths = dir.d_paths;
        a.tab_ptr = p->d_tab_ptr; a.tab_idx = p->d_tab_idx; a.tab_coef = p->d_tab_coef;
        a.G = G; a.ev = ev; a.node0 = node0; a.n_nodes = n_nodes;
        a.src = src; a.Y = Y; a.phi = phi; a.Zbar = Zbar; a.gphi = gphi; a.gY = gY;
        a.K = p->K; a.dsh = p->dim_sh; a.C_src = dir.C_src;
        // the first group writes in the caller's mode, later groups accumulate
        a.phi_mode = phi_mode ? (first ? phi_mode : 2) : 0;
        a.Y_mode = Y_mode ? (first ? Y_mode : 2) : 0;
        first = false;
        const bool k16 = (p->K > 8);
        const int KC = k16 ? 16 : 8;
        a.Kpad = ((p->K + KC - 1) / KC) * KC;
        a.max_dsrc = 1; a.max_ent = 1;
        for (int k = G.path_begin; k < G.path_end; ++k) {
            a.max_dsrc = std::max(a.max_dsrc, dir.paths[k].d_src);
            a.max_ent = std::max(a.max_ent, dir.paths[k].d_src * G.d_dst);
        }
        int wf = a.max_dsrc * EP_UCH * 33 + EP_UCH * G.d_dst * KC + a.max_ent * 32 + 2 * a.dsh * 32 +
                 2 * a.Kpad * 32;
        wf = (wf + 1) & ~1;        // int64 alignment of the index array that follows
        a.warp_floats = wf + 64;   // + 32 int64
        const size_t sh = (size_t)a.warp_floats * EP_WARPS * sizeof(float);
        dim3 grid((unsigned)((n_nodes + EP_WARPS - 1) / EP_WARPS));
        KernelTimer kt(K_EDGE, s);
        cudaError_t e = dispatch_d(G.d_dst, [&](auto dtag) -> cudaError_t {
            constexpr int D = decltype(dtag)::value;
            if (k16) {
                auto kern = k_edge_pass<D, 16>;
                if (sh > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
                kern<<<grid, EP_WARPS * 32, sh, s>>>(a);
            } else {
                auto kern = k_edge_pass<D, 8>;
                if (sh > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
                kern<<<grid, EP_WARPS * 32, sh, s>>>(a);
            }
            return cudaGetLastError();
        });
        count_launch();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace sobek
