// Direct kernel of the channelwise (uvu) mode (Eq. uvu_connection): y and gx, for profiles  C x 0e + C x 1o + ... + C x L  on
// both sides with l_max = L:
//   y_i[l_out, u, o] = sum_{e into i} sum_{paths (l_in, l_sh, l_out)} w_e[pi, u] * sum_a M_e^pi[a, o] x_{j(e)}[l_in, u, a],
//   w_e[pi, u] = sum_q phi_e[q] R[q, w_off(pi) + u],        M_e^pi[a, o] = sum_b c^pi[a, b, o] Y_e[b].
// No receiver state and no node-side pass: a multiplicity channel u never mixes with another one, so a thread owns a
// channel for the whole launch and keeps in REGISTERS both the K weights of its channel for every path it walks and
// the output components of the receiver at hand.  K + d_in d_out multiply-adds per channel, edge and path instead of
// the K d_out of the route through the K-expanded state, and a gathered sender row is read exactly once.
//
// CTA = C x NG threads, persistent over receivers (receiver = blockIdx.x, + gridDim.x, ...).  Thread (u, g) owns channel
// u and the g-th contiguous share of the paths (NG > 1 where K x paths would not fit the register file; the shares'
// partial outputs meet in shared memory when a receiver ends).  The paths are a compile-time walk over the
// (l_in, l_sh, l_out) triples, so every register array has constant indices.
//
// Edges run in batches of TB through a software pipeline with one CTA barrier per batch:
//   thread 0 walks the CSR three batches ahead and leaves batch descriptors in a ring of four;
//   two batches ahead:  phi, Y rows and sender ids by 4-byte asynchronous copies (ring of three);
//   one batch ahead:    the senders' feature rows (one contiguous row each) by 16-byte asynchronous copies, and the
//                       coupling matrices M_e of all paths from the sparse CG terms (shared by all channels);
//   now:                per edge, w_e for the share's paths from the broadcast phi row, then path by path the
//                       contraction, with rows of M_e as broadcast 16-byte shared loads.
// M_e per path is stored row-padded to four floats in the orientation with fewer rows to load; a path with
// l_sh = 0 is a multiple of the identity and keeps one number.
//
// The input adjoint of the same operator, gx_j[l_in, u, a] = sum_{e out of j} sum_paths w_e[pi, u] sum_o M_e^pi[a, o]
// gy_{i(e)}[l_out, u, o] (Eq. adjoints, channelwise), is the same kernel on the sender view of the graph: segments of
// the senders, the receivers' gy rows gathered, phi and Y rows through the view's edge permutation, and host-built
// tables in which the walk position (l_a, l_sh, l_b) stands for the path (l_in = l_b, l_out = l_a) with M_e transposed.
#include <cuda_runtime.h>

#include <string.h>

#include <algorithm>
#include <cmath>
#include <vector>

#include "guard.cuh"
#include "internal.h"

namespace sobek {
namespace {

constexpr int TB = 8;           // edges per batch
constexpr int KMAX = 16;
constexpr int R_REG_BUDGET = 176;   // weights a thread may hold in registers

struct UdArgs {
    const int64_t* row_ptr;     // segments of the owning node (receivers; senders on the sender view)
    const int32_t* ids;         // per position: the node whose row is gathered
    const int32_t* perm;        // per position: the edge id (NULL: the position itself)
    int64_t N, E;
    const float* x;             // gathered rows (x; gy on the sender view)
    const float* Y;
    const float* phi;
    const float* R;
    float* y;                   // rows of the owning nodes (y; gx on the sender view)
    const float* own;           // weight adjoint: rows of the owning nodes that are read (gy), else NULL
    float* part;                // weight adjoint: [gridDim.x][K * N_w] partial sums
    const int32_t* woff;        // per path (static order): first weight column
    const int2* ent;            // per stored M entry: {offset in the padded M_e | number of terms << 16, first term}
    const int2* nz;             // terms: {index b into a Y row, coefficient bits}
    int32_t C;                  // channels of a CTA: slice blockIdx.x % H of the profile's Cf = C * H channels
    int32_t Cf, H;
    int32_t K, nM, N_w, C_x, C_y, n_nz;
    int* status;
};

__host__ __device__ constexpr bool path_ok(int li, int ls, int lo, int L) {
    return lo <= L && ((li + ls + lo) & 1) == 0 && lo >= (li > ls ? li - ls : ls - li) && lo <= li + ls;
}
__host__ __device__ constexpr int n_paths_c(int L) {
    int n = 0;
    for (int li = 0; li <= L; ++li)
        for (int ls = 0; ls <= L; ++ls)
            for (int lo = 0; lo <= L; ++lo) n += path_ok(li, ls, lo, L) ? 1 : 0;
    return n;
}
__host__ __device__ constexpr int pad4(int n) { return (n + 3) & ~3; }
// stored transposed ([o][a] rows) when that takes fewer 16-byte row loads
__host__ __device__ constexpr bool m_transposed(int di, int dO) { return dO * (pad4(di) / 4) < di * (pad4(dO) / 4); }
__host__ __device__ constexpr int m_block(int li, int ls, int lo) {
    const int di = 2 * li + 1, dO = 2 * lo + 1;
    return ls == 0 ? 4 : (m_transposed(di, dO) ? dO * pad4(di) : di * pad4(dO));
}
__host__ __device__ constexpr int m_floats_c(int L) {       // padded floats of M_e, all paths
    int n = 0;
    for (int li = 0; li <= L; ++li)
        for (int ls = 0; ls <= L; ++ls)
            for (int lo = 0; lo <= L; ++lo) n += path_ok(li, ls, lo, L) ? m_block(li, ls, lo) : 0;
    return n;
}
__host__ __device__ constexpr int n_groups_c(int L, int KP) { return (n_paths_c(L) * KP + R_REG_BUDGET - 1) / R_REG_BUDGET; }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async4(void* dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

struct UdSmem {           // carved from dynamic shared memory; every part a multiple of 16 bytes
    int4* desc;           // [4] {edge offset lo, hi, nb | last << 8, receiver (-1: end)}
    float* phi;           // [3][TB][KP]
    float* Y;             // [3][TB][DT]
    int32_t* sid;         // [3][TB]
    int32_t* eid;         // [4][TB] edge ids of a batch (sender view), in step with desc
    float* M;             // [2][TB][MF]
    float* X;             // [2][TB][DT * C]
    float* out;           // [NG - 1][DT * C]
    float* own;           // [2][DT * C] (weight adjoint)
    int2* ent;            // [nM]
    int2* nz;             // [n_nz]
};

// The software pipeline both kernels share (see the header): prefetch(it) waits for the copies in flight, meets the
// CTA barrier, and issues the work that runs ahead of batch `it`; the caller then consumes batch `it` and calls rotate().
// SP: the channels are split into slices, one CTA each (else H = 1 is known at compile time)
template <int L, int KP, bool SP>
struct UdPipe {
    static constexpr int DT = (L + 1) * (L + 1);
    static constexpr int MF = m_floats_c(L);
    const UdArgs& a;
    const UdSmem& sm;
    const int NT, tid;
    // thread 0's CSR walk
    int64_t w_node, w_pos = 0, w_end = 0;
    bool w_open = false;                          // a node is at hand and not yet closed by a `last` batch
    int d_slot = 0;                               // ring slots of the batch `it + 3` (descriptor), `it + 2` (edge inputs),
    int r_slot2 = 2, r_slot1 = 1, r_slot0 = 0;    // `it + 1`, `it`; rotated at the end of an iteration

    int64_t n_s0 = 0, n_s1 = 0;                   // segment of the node after w_node, fetched ahead

    __device__ __forceinline__ UdPipe(const UdArgs& a_, const UdSmem& sm_, int NT_)
        : a(a_), sm(sm_), NT(NT_), tid(threadIdx.x), w_node((int64_t)(blockIdx.x / (SP ? a_.H : 1)) - (int64_t)(gridDim.x / (SP ? a_.H : 1))) {
        const int64_t n0 = blockIdx.x / (SP ? a.H : 1);
        if (tid == 0 && n0 < a.N) { n_s0 = a.row_ptr[n0]; n_s1 = a.row_ptr[n0 + 1]; }
    }
    // copies the CTA's channels of a [DT][Cf] feature row into [DT][C] shared floats, 16 bytes at a time
    __device__ __forceinline__ void copy_row(float* dst, const float* src) const {
        const int C = a.C;
        const int row_chunks = DT * C / 4;
        if (!SP) {
            for (int i = tid; i < row_chunks; i += NT) cp_async16(dst + 4 * i, src + 4 * i);
        } else {
            const int c4n = C / 4;
            const float* s0 = src + (blockIdx.x % a.H) * C;
            for (int i = tid; i < row_chunks; i += NT) {
                const int t = i / c4n, c4 = i - t * c4n;
                cp_async16(dst + 4 * i, s0 + t * a.Cf + 4 * c4);
            }
        }
    }
    __device__ __forceinline__ int4 desc_now() const { return sm.desc[(d_slot + 1) & 3]; }
    __device__ __forceinline__ void rotate(int it) {
        d_slot = (d_slot + 1) & 3;
        if (it >= -2) { const int t = r_slot0; r_slot0 = r_slot1; r_slot1 = r_slot2; r_slot2 = t; }
    }
    __device__ __forceinline__ void prefetch(int it) {
        const int C = a.C;
        cp_async_wait_all();
        __syncthreads();
        // ---- T: descriptor of batch it + 3
        if (tid == 0) {
            bool first = false;
            if (!w_open) {
                w_node += gridDim.x / (SP ? a.H : 1);
                if (w_node < a.N) {
                    // the bounds were fetched when the node before was opened (no load latency under the CTA barrier)
                    const int64_t s0 = n_s0 < 0 ? 0 : (n_s0 > a.E ? a.E : n_s0);
                    const int64_t s1 = n_s1 < s0 ? s0 : (n_s1 > a.E ? a.E : n_s1);
                    if ((s0 != n_s0 || s1 != n_s1) && a.status) atomicExch(a.status, (int)SOBEK_ERR_GRAPH);
                    w_pos = s0; w_end = s1; w_open = first = true;
                    const int64_t nx = w_node + gridDim.x / (SP ? a.H : 1);
                    if (nx < a.N) { n_s0 = a.row_ptr[nx]; n_s1 = a.row_ptr[nx + 1]; }
                }
            }
            int4 d = make_int4(0, 0, 0, -1);
            if (w_open) {
                const int nb = (int)min((int64_t)TB, w_end - w_pos);
                const bool last = w_pos + nb >= w_end;
                d = make_int4((int)(uint32_t)(uint64_t)w_pos, (int)((uint64_t)w_pos >> 32), nb | (last ? 256 : 0) | (first ? 512 : 0), (int)w_node);
                w_pos += nb;
                if (last) w_open = false;
            }
            sm.desc[d_slot] = d;
            if (a.perm && d.w >= 0)
                for (int i = 0; i < (d.z & 255); ++i) cp_async4(sm.eid + d_slot * TB + i, a.perm + (w_pos - (d.z & 255)) + i);
        }
        // ---- A: edge inputs of batch it + 2
        if (it >= -2) {
            const int4 d = sm.desc[(d_slot + 3) & 3];
            if (d.w >= 0) {
                const int64_t b0 = (int64_t)(((uint64_t)(uint32_t)d.y << 32) | (uint32_t)d.x);
                const int nb = d.z & 255;
                float* dphi = sm.phi + r_slot2 * (TB * KP);
                float* dY = sm.Y + r_slot2 * (TB * DT);
                const int32_t* eid = sm.eid + ((d_slot + 3) & 3) * TB;
                for (int i = tid; i < nb * KP; i += NT) {
                    const int e = i / KP, q = i - e * KP;
                    const int64_t ee = a.perm ? (int64_t)eid[e] : b0 + e;
                    if (q < a.K && id_ok(ee, a.E, a.status)) cp_async4(dphi + i, a.phi + ee * a.K + q);
                }
                for (int i = tid; i < nb * DT; i += NT) {
                    const int e = i / DT, b = i - e * DT;
                    const int64_t ee = a.perm ? (int64_t)eid[e] : b0 + e;
                    if (id_ok(ee, a.E, a.status)) cp_async4(dY + i, a.Y + ee * DT + b);
                }
                if (tid < nb) cp_async4(sm.sid + r_slot2 * TB + tid, a.ids + b0 + tid);
            }
        }
        // ---- B, C: sender rows and coupling matrices of batch it + 1
        if (it >= -1) {
            const int4 d = sm.desc[(d_slot + 2) & 3];
            if (d.w >= 0) {
                const int nb = d.z & 255;
                const int buf = (it + 1) & 1;
                float* dX = sm.X + (size_t)buf * TB * DT * C;
                const int32_t* sid = sm.sid + r_slot1 * TB;
                for (int e = 0; e < nb; ++e) {
                    const int32_t j = sid[e];
                    if (!id_ok(j, a.N, a.status)) continue;
                    copy_row(dX + e * DT * C, a.x + (int64_t)j * a.C_x);
                }
                if (a.own && (d.z & 512)) {           // the owning node's row (weight adjoint), with its first batch
                    copy_row(sm.own + (size_t)buf * DT * C, a.own + (int64_t)d.w * a.C_y);
                }
                float* dM = sm.M + buf * (TB * MF);
                const float* sY = sm.Y + r_slot1 * (TB * DT);
                for (int m = tid; m < a.nM; m += NT) {
                    const int2 en = sm.ent[m];
                    const int dst = en.x & 0xffff, cnt = en.x >> 16;
                    for (int e = 0; e < nb; ++e) {
                        float v = 0.f;
                        for (int k = en.y; k < en.y + cnt; ++k) { const int2 t = sm.nz[k]; v = fmaf(__int_as_float(t.y), sY[e * DT + t.x], v); }
                        dM[e * MF + dst] = v;
                    }
                }
            }
        }
    }
};

// The work of one thread share G of NG: see the header.  All shares run the same barrier sequence.
template <int L, int KP, int NG, int G, bool SP>
__device__ __forceinline__ void uvu_direct_share(const UdArgs& a, const UdSmem& sm, const int u) {
    constexpr int DT = (L + 1) * (L + 1);
    constexpr int NP = n_paths_c(L);
    constexpr int MF = m_floats_c(L);
    constexpr int NPG = (NP + NG - 1) / NG;
    const int C = a.C, NT = C * NG;

    // this channel's weights of the share's paths
    float rw[NPG * KP];
    {
        int pi = 0, pl = 0;
#pragma unroll
        for (int li = 0; li <= L; ++li)
#pragma unroll
            for (int ls = 0; ls <= L; ++ls)
#pragma unroll
                for (int lo = 0; lo <= L; ++lo) {
                    if (!path_ok(li, ls, lo, L)) continue;
                    if (pi * NG / NP == G) {
                        const float* Rp = a.R + __ldg(a.woff + pi) + (SP ? (blockIdx.x % a.H) * C : 0) + u;
#pragma unroll
                        for (int q = 0; q < KP; ++q) rw[pl * KP + q] = q < a.K ? __ldg(Rp + (int64_t)q * a.N_w) : 0.f;
                        ++pl;
                    }
                    ++pi;
                }
    }
    float acc[DT];
#pragma unroll
    for (int i = 0; i < DT; ++i) acc[i] = 0.f;

    UdPipe<L, KP, SP> pipe(a, sm, NT);
    for (int it = -3;; ++it) {
        pipe.prefetch(it);
        // ---- D: batch it
        if (it >= 0) {
            const int4 d = pipe.desc_now();
            if (d.w < 0) break;
            const int nb = d.z & 255;
            const int buf = it & 1;
            const float* bX = sm.X + (size_t)buf * TB * DT * C + u;
            const float* bM = sm.M + buf * (TB * MF);
            const float* bphi = sm.phi + pipe.r_slot0 * (TB * KP);
            const int32_t* sid = sm.sid + pipe.r_slot0 * TB;
            for (int e = 0; e < nb; ++e) {
                if ((uint32_t)sid[e] >= (uint64_t)a.N) continue;
                // w_e of the share's paths
                float w[NPG];
#pragma unroll
                for (int i = 0; i < NPG; ++i) w[i] = 0.f;
#pragma unroll
                for (int q4 = 0; q4 < KP; q4 += 4) {
                    const float4 f = *reinterpret_cast<const float4*>(bphi + e * KP + q4);
                    // (component by component: consecutive multiply-adds go to different sums)
#pragma unroll
                    for (int i = 0; i < NPG; ++i) w[i] = fmaf(f.x, rw[i * KP + q4], w[i]);
#pragma unroll
                    for (int i = 0; i < NPG; ++i) w[i] = fmaf(f.y, rw[i * KP + q4 + 1], w[i]);
#pragma unroll
                    for (int i = 0; i < NPG; ++i) w[i] = fmaf(f.z, rw[i * KP + q4 + 2], w[i]);
#pragma unroll
                    for (int i = 0; i < NPG; ++i) w[i] = fmaf(f.w, rw[i * KP + q4 + 3], w[i]);
                }
                const float* eX = bX + e * DT * C;
                const float* eM = bM + e * MF;
                int pi = 0, pl = 0, mo = 0, at_li = -1;
                float xv[2 * L + 1];
#pragma unroll
                for (int li = 0; li <= L; ++li) {
#pragma unroll
                    for (int ls = 0; ls <= L; ++ls) {
#pragma unroll
                        for (int lo = 0; lo <= L; ++lo) {
                            if (!path_ok(li, ls, lo, L)) continue;
                            const int di = 2 * li + 1, dO = 2 * lo + 1;
                            if (pi * NG / NP == G) {
                                if (at_li != li) {
#pragma unroll
                                    for (int s = 0; s < di; ++s) xv[s] = eX[(li * li + s) * C];
                                    at_li = li;
                                }
                                const float wp = w[pl];
                                if (ls == 0) {                               // a multiple of the identity
                                    const float wm = wp * eM[mo];
#pragma unroll
                                    for (int o = 0; o < dO; ++o) acc[lo * lo + o] = fmaf(wm, xv[o], acc[lo * lo + o]);
                                } else if (!m_transposed(di, dO)) {         // rows [a][o]
#pragma unroll
                                    for (int s = 0; s < di; ++s) {
                                        const float t = wp * xv[s];
#pragma unroll
                                        for (int o4 = 0; o4 < dO; o4 += 4) {
                                            const float4 r = *reinterpret_cast<const float4*>(eM + mo + s * pad4(dO) + o4);
                                            acc[lo * lo + o4] = fmaf(r.x, t, acc[lo * lo + o4]);
                                            if (o4 + 1 < dO) acc[lo * lo + o4 + 1] = fmaf(r.y, t, acc[lo * lo + o4 + 1]);
                                            if (o4 + 2 < dO) acc[lo * lo + o4 + 2] = fmaf(r.z, t, acc[lo * lo + o4 + 2]);
                                            if (o4 + 3 < dO) acc[lo * lo + o4 + 3] = fmaf(r.w, t, acc[lo * lo + o4 + 3]);
                                        }
                                    }
                                } else {                                     // rows [o][a]
#pragma unroll
                                    for (int o = 0; o < dO; ++o) {
                                        float c = 0.f;
#pragma unroll
                                        for (int s4 = 0; s4 < di; s4 += 4) {
                                            const float4 r = *reinterpret_cast<const float4*>(eM + mo + o * pad4(di) + s4);
                                            c = fmaf(r.x, xv[s4], c);
                                            if (s4 + 1 < di) c = fmaf(r.y, xv[s4 + 1], c);
                                            if (s4 + 2 < di) c = fmaf(r.z, xv[s4 + 2], c);
                                            if (s4 + 3 < di) c = fmaf(r.w, xv[s4 + 3], c);
                                        }
                                        acc[lo * lo + o] = fmaf(wp, c, acc[lo * lo + o]);
                                    }
                                }
                                ++pl;
                            }
                            ++pi; mo += m_block(li, ls, lo);
                        }
                    }
                }
            }
            if (d.z & 256) {                       // the receiver ends with this batch
                if (NG > 1) {
                    if (G > 0) {
#pragma unroll
                        for (int i = 0; i < DT; ++i) sm.out[((G - 1) * DT + i) * C + u] = acc[i];
                    }
                    __syncthreads();
                }
                if (G == 0) {
                    float* yp = a.y + (int64_t)d.w * a.C_y + (SP ? (blockIdx.x % a.H) * C : 0) + u;
#pragma unroll
                    for (int i = 0; i < DT; ++i) {
                        float v = acc[i];
#pragma unroll
                        for (int g = 1; g < NG; ++g) v += sm.out[((g - 1) * DT + i) * C + u];
                        yp[i * (SP ? a.Cf : C)] = v;
                    }
                }
#pragma unroll
                for (int i = 0; i < DT; ++i) acc[i] = 0.f;
            }
        }
        pipe.rotate(it);
    }
}

// carves the dynamic shared memory, loads the tables; the first barrier of the pipeline orders these writes before use
template <int L, int KP>
__device__ __forceinline__ UdSmem ud_setup(const UdArgs& a, unsigned char* p) {
    constexpr int DT = (L + 1) * (L + 1);
    constexpr int NG = n_groups_c(L, KP);
    constexpr int MF = m_floats_c(L);
    const int C = a.C, NT = C * NG, tid = threadIdx.x;
    UdSmem sm;
    sm.desc = reinterpret_cast<int4*>(p); p += 4 * sizeof(int4);
    sm.phi = reinterpret_cast<float*>(p); p += 3 * TB * KP * 4;
    sm.Y = reinterpret_cast<float*>(p); p += pad4(3 * TB * DT) * 4;
    sm.sid = reinterpret_cast<int32_t*>(p); p += 3 * TB * 4;
    sm.eid = reinterpret_cast<int32_t*>(p); p += 4 * TB * 4;
    sm.M = reinterpret_cast<float*>(p); p += 2 * TB * MF * 4;
    sm.X = reinterpret_cast<float*>(p); p += (size_t)2 * TB * DT * C * 4;
    sm.out = reinterpret_cast<float*>(p); p += (size_t)(NG - 1) * DT * C * 4;
    sm.own = reinterpret_cast<float*>(p); p += (size_t)2 * DT * C * 4;
    sm.ent = reinterpret_cast<int2*>(p); p += (size_t)a.nM * 8;
    sm.nz = reinterpret_cast<int2*>(p);
    for (int i = tid; i < 3 * TB * KP; i += NT) sm.phi[i] = 0.f;       // the columns q >= K stay zero
    for (int i = tid; i < a.nM; i += NT) sm.ent[i] = a.ent[i];
    for (int i = tid; i < a.n_nz; i += NT) sm.nz[i] = a.nz[i];
    return sm;
}
template <int L, int KP>
constexpr size_t ud_smem_bytes(int C, size_t tables) {
    constexpr int DT = (L + 1) * (L + 1), NG = n_groups_c(L, KP), MF = m_floats_c(L);
    return 4 * sizeof(int4) + (size_t)3 * TB * KP * 4 + (size_t)pad4(3 * TB * DT) * 4 + 7 * TB * 4 + (size_t)2 * TB * MF * 4 +
           (size_t)2 * TB * DT * C * 4 + (size_t)(NG - 1) * DT * C * 4 + (size_t)2 * DT * C * 4 + tables;
}

template <int L, int KP, bool SP>
__global__ void __launch_bounds__(256) k_uvu_direct_fwd(const UdArgs a) {
    constexpr int NG = n_groups_c(L, KP);
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const UdSmem sm = ud_setup<L, KP>(a, smem_raw);
    const int g = threadIdx.x / a.C, u = threadIdx.x - g * a.C;
    if (NG == 1 || g == 0) uvu_direct_share<L, KP, NG, 0, SP>(a, sm, u);
    else if (NG == 2 || g == 1) uvu_direct_share<L, KP, NG, (NG > 1 ? 1 : 0), SP>(a, sm, u);
    else if (NG == 3 || g == 2) uvu_direct_share<L, KP, NG, (NG > 2 ? 2 : 0), SP>(a, sm, u);
    else uvu_direct_share<L, KP, NG, (NG > 3 ? 3 : 0), SP>(a, sm, u);
}

// Weight adjoint of the channelwise mode on the same pipeline (Eq. adjoints):
//   gR[q, w_off(pi) + u] = sum_e phi_e[q] gw_e[pi, u],   gw_e[pi, u] = sum_{a, o} M_e^pi[a, o] x_{j(e)}[l_in, u, a] gy_{i(e)}[l_out, u, o].
// Thread (u, share) keeps the K x paths sums of its channel in registers over all receivers of its CTA and the
// receiver's gy components beside them; the CTA's sums go to its own slice of `part`, summed over CTAs in a fixed
// order by the caller.
template <int L, int KP, int NG, int G, bool SP>
__device__ __forceinline__ void uvu_direct_wgrad_share(const UdArgs& a, const UdSmem& sm, const int u) {
    constexpr int DT = (L + 1) * (L + 1);
    constexpr int NP = n_paths_c(L);
    constexpr int MF = m_floats_c(L);
    constexpr int NPG = (NP + NG - 1) / NG;
    const int C = a.C, NT = C * NG;
    float ga[NPG * KP];
#pragma unroll
    for (int i = 0; i < NPG * KP; ++i) ga[i] = 0.f;
    float gyr[DT];
#pragma unroll
    for (int i = 0; i < DT; ++i) gyr[i] = 0.f;
    UdPipe<L, KP, SP> pipe(a, sm, NT);
    for (int it = -3;; ++it) {
        pipe.prefetch(it);
        if (it >= 0) {
            const int4 d = pipe.desc_now();
            if (d.w < 0) break;
            const int nb = d.z & 255;
            const int buf = it & 1;
            const float* bX = sm.X + (size_t)buf * TB * DT * C + u;
            const float* bM = sm.M + buf * (TB * MF);
            const float* bphi = sm.phi + pipe.r_slot0 * (TB * KP);
            const int32_t* sid = sm.sid + pipe.r_slot0 * TB;
            if (d.z & 512) {                       // a new receiver: its gy components
#pragma unroll
                for (int i = 0; i < DT; ++i) gyr[i] = sm.own[((size_t)buf * DT + i) * C + u];
            }
            for (int e = 0; e < nb; ++e) {
                if ((uint32_t)sid[e] >= (uint64_t)a.N) continue;
                const float* eX = bX + e * DT * C;
                const float* eM = bM + e * MF;
                float gw[NPG];
                int pi = 0, pl = 0, mo = 0, at_li = -1;
                float xv[2 * L + 1];
#pragma unroll
                for (int li = 0; li <= L; ++li) {
#pragma unroll
                    for (int ls = 0; ls <= L; ++ls) {
#pragma unroll
                        for (int lo = 0; lo <= L; ++lo) {
                            if (!path_ok(li, ls, lo, L)) continue;
                            const int di = 2 * li + 1, dO = 2 * lo + 1;
                            if (pi * NG / NP == G) {
                                if (at_li != li) {
#pragma unroll
                                    for (int s = 0; s < di; ++s) xv[s] = eX[(li * li + s) * C];
                                    at_li = li;
                                }
                                float c = 0.f;
                                if (ls == 0) {
#pragma unroll
                                    for (int o = 0; o < dO; ++o) c = fmaf(xv[o], gyr[lo * lo + o], c);
                                    c *= eM[mo];
                                } else if (!m_transposed(di, dO)) {         // rows [a][o]
#pragma unroll
                                    for (int s = 0; s < di; ++s) {
                                        float r = 0.f;
#pragma unroll
                                        for (int o4 = 0; o4 < dO; o4 += 4) {
                                            const float4 m = *reinterpret_cast<const float4*>(eM + mo + s * pad4(dO) + o4);
                                            r = fmaf(m.x, gyr[lo * lo + o4], r);
                                            if (o4 + 1 < dO) r = fmaf(m.y, gyr[lo * lo + o4 + 1], r);
                                            if (o4 + 2 < dO) r = fmaf(m.z, gyr[lo * lo + o4 + 2], r);
                                            if (o4 + 3 < dO) r = fmaf(m.w, gyr[lo * lo + o4 + 3], r);
                                        }
                                        c = fmaf(r, xv[s], c);
                                    }
                                } else {                                     // rows [o][a]
#pragma unroll
                                    for (int o = 0; o < dO; ++o) {
                                        float r = 0.f;
#pragma unroll
                                        for (int s4 = 0; s4 < di; s4 += 4) {
                                            const float4 m = *reinterpret_cast<const float4*>(eM + mo + o * pad4(di) + s4);
                                            r = fmaf(m.x, xv[s4], r);
                                            if (s4 + 1 < di) r = fmaf(m.y, xv[s4 + 1], r);
                                            if (s4 + 2 < di) r = fmaf(m.z, xv[s4 + 2], r);
                                            if (s4 + 3 < di) r = fmaf(m.w, xv[s4 + 3], r);
                                        }
                                        c = fmaf(r, gyr[lo * lo + o], c);
                                    }
                                }
                                gw[pl] = c;
                                ++pl;
                            }
                            ++pi; mo += m_block(li, ls, lo);
                        }
                    }
                }
#pragma unroll
                for (int q4 = 0; q4 < KP; q4 += 4) {
                    const float4 f = *reinterpret_cast<const float4*>(bphi + e * KP + q4);
#pragma unroll
                    for (int i = 0; i < NPG; ++i) {
                        if (i < pl) {
                            ga[i * KP + q4] = fmaf(f.x, gw[i], ga[i * KP + q4]);
                            ga[i * KP + q4 + 1] = fmaf(f.y, gw[i], ga[i * KP + q4 + 1]);
                            ga[i * KP + q4 + 2] = fmaf(f.z, gw[i], ga[i * KP + q4 + 2]);
                            ga[i * KP + q4 + 3] = fmaf(f.w, gw[i], ga[i * KP + q4 + 3]);
                        }
                    }
                }
            }
        }
        pipe.rotate(it);
    }
    // this CTA's sums
    float* out = a.part + (int64_t)(blockIdx.x / (SP ? a.H : 1)) * a.K * a.N_w + (SP ? (blockIdx.x % a.H) * C : 0) + u;
    int pi = 0, pl = 0;
#pragma unroll
    for (int li = 0; li <= L; ++li)
#pragma unroll
        for (int ls = 0; ls <= L; ++ls)
#pragma unroll
            for (int lo = 0; lo <= L; ++lo) {
                if (!path_ok(li, ls, lo, L)) continue;
                if (pi * NG / NP == G) {
                    const int32_t wo = __ldg(a.woff + pi);
#pragma unroll
                    for (int q = 0; q < KP; ++q)
                        if (q < a.K) out[(int64_t)q * a.N_w + wo] = ga[pl * KP + q];
                    ++pl;
                }
                ++pi;
            }
}

template <int L, int KP, bool SP>
__global__ void __launch_bounds__(256) k_uvu_direct_wgrad(const UdArgs a) {
    constexpr int NG = n_groups_c(L, KP);
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const UdSmem sm = ud_setup<L, KP>(a, smem_raw);
    const int g = threadIdx.x / a.C, u = threadIdx.x - g * a.C;
    if (NG == 1 || g == 0) uvu_direct_wgrad_share<L, KP, NG, 0, SP>(a, sm, u);
    else if (NG == 2 || g == 1) uvu_direct_wgrad_share<L, KP, NG, (NG > 1 ? 1 : 0), SP>(a, sm, u);
    else if (NG == 3 || g == 2) uvu_direct_wgrad_share<L, KP, NG, (NG > 2 ? 2 : 0), SP>(a, sm, u);
    else uvu_direct_wgrad_share<L, KP, NG, (NG > 3 ? 3 : 0), SP>(a, sm, u);
}

}  // namespace

// Whether the plan's profile is  C x 0e + C x 1o + ... + C x L  on both sides with l_max = L <= 3, C a multiple of 16
// that splits into slices of at most 256 / (thread shares) channels; fills the per-path and per-entry tables in the kernel's static path order and
// padded M_e layout.
void build_uvu_direct(sobek_plan* p, const sobek_irrep* in, int n_in, const sobek_irrep* out, int n_out) {
    UvuDirect& D = p->ud;
    D = UvuDirect{};
    if (!p->uvu || n_in != n_out || n_in < 1 || n_in > 4 || p->l_max != n_in - 1 || p->K > KMAX) return;
    const int L = n_in - 1, C = in[0].mul;
    const int NG = n_groups_c(L, p->K <= 8 ? 8 : 16);
    // a CTA takes C / H channels (a multiple of 16) so that its (channel, share) threads number at most 256
    const int H = (C * NG + 255) / 256;
    if (C < 16 || (C & 15) || NG > 4 || C % H != 0 || ((C / H) & 15)) return;
    for (int i = 0; i < n_in; ++i) {
        const int par = (i & 1) ? -1 : 1;
        if (in[i].l != i || out[i].l != i || in[i].mul != C || out[i].mul != C || in[i].parity != par || out[i].parity != par) return;
    }
    const Direction& dir = p->fwd;
    for (int tr = 0; tr < 2; ++tr) {
        // tr = 1: the walk position (la, ls, lb) stands for the path (l_in = lb, l_sh = ls, l_out = la), whose coupling
        // matrix is used transposed: gx_j[l_in, u, a] += w_e M_e[a, o] gy_i[l_out, u, o]
        std::vector<int32_t> woff;
        std::vector<int2> ent, nz;
        int mo = 0;
        for (int la = 0; la <= L; ++la)
            for (int ls = 0; ls <= L; ++ls)
                for (int lb = 0; lb <= L; ++lb) {
                    if (!path_ok(la, ls, lb, L)) continue;
                    const int li = tr ? lb : la, lo = tr ? la : lb;
                    const DPath* P = nullptr;
                    for (size_t gi = 0; gi < dir.groups.size() && !P; ++gi) {
                        const DGroup& G = dir.groups[gi];
                        if (G.dst_off != lo * lo * C || G.d_dst != 2 * lo + 1) continue;
                        for (int k = G.path_begin; k < G.path_end; ++k) {
                            const DPath& Q = dir.paths[k];
                            if (Q.src_off == li * li * C && Q.d_src == 2 * li + 1 && Q.sh_off == ls * ls && Q.d_sh == 2 * ls + 1) { P = &Q; break; }
                        }
                    }
                    if (!P || P->c_src != C || P->c_dst != C) return;
                    woff.push_back((int32_t)P->w_off);
                    const int dA = 2 * la + 1, dB = 2 * lb + 1;      // gathered side, accumulated side
                    // sparse terms of the entry (a, b) of the walk's matrix
                    auto terms = [&](int ia, int ib) {
                        const int t = P->tabM + (tr ? ib * P->d_dst + ia : ia * P->d_dst + ib);
                        return std::make_pair(p->tab_ptr[t], p->tab_ptr[t + 1]);
                    };
                    auto emit = [&](int ia, int ib, int dst) {
                        const auto [k0, k1] = terms(ia, ib);
                        ent.push_back(make_int2(dst | ((k1 - k0) << 16), (int)nz.size()));
                        for (int k = k0; k < k1; ++k) {
                            int bits; const float cf = p->tab_coef[k]; memcpy(&bits, &cf, 4);
                            nz.push_back(make_int2(P->sh_off + p->tab_idx[k], bits));
                        }
                    };
                    if (ls == 0) {
                        // an equivariant map between equal irreps is a multiple of the identity; the kernel keeps only
                        // that multiple, so check that the table says the same
                        const auto [a0, a1] = terms(0, 0);
                        if (a1 - a0 != 1) return;
                        for (int ia = 0; ia < dA; ++ia)
                            for (int ib = 0; ib < dB; ++ib) {
                                const auto [k0, k1] = terms(ia, ib);
                                if (ia != ib) { if (k1 != k0) return; continue; }
                                if (k1 - k0 != 1 || p->tab_idx[k0] != p->tab_idx[a0] ||
                                    std::fabs(p->tab_coef[k0] - p->tab_coef[a0]) > 1e-6f * std::fabs(p->tab_coef[a0])) return;
                            }
                        emit(0, 0, mo);
                    } else if (!m_transposed(dA, dB)) {
                        for (int ia = 0; ia < dA; ++ia)
                            for (int ib = 0; ib < dB; ++ib) emit(ia, ib, mo + ia * pad4(dB) + ib);
                    } else {
                        for (int ia = 0; ia < dA; ++ia)
                            for (int ib = 0; ib < dB; ++ib) emit(ia, ib, mo + ib * pad4(dA) + ia);
                    }
                    mo += m_block(la, ls, lb);
                }
        if (woff.size() != dir.paths.size() || mo != m_floats_c(L) || mo >= 65536 || nz.size() >= 32768) return;
        D.dir[tr].woff = woff; D.dir[tr].ent = ent; D.dir[tr].nz = nz;
    }
    D.L = L; D.C = C; D.H = H;
    D.ok = true;
}

namespace {
template <int L, int KP>
cudaError_t launch_ud(const UdArgs& a, size_t tables, int max_grid, int* grid_out, cudaStream_t s) {
    constexpr int NG = n_groups_c(L, KP);
    const int NT = a.C * NG;                  // a.C: channels of a CTA
    const size_t sh = ud_smem_bytes<L, KP>(a.C, tables);
    auto kern = a.part ? (a.H > 1 ? k_uvu_direct_wgrad<L, KP, true> : k_uvu_direct_wgrad<L, KP, false>)
                       : (a.H > 1 ? k_uvu_direct_fwd<L, KP, true> : k_uvu_direct_fwd<L, KP, false>);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, NT, sh);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    // H CTAs (one per channel slice) walk the same nodes: the grid is a multiple of H
    int64_t walks = std::min<int64_t>(a.N, std::max<int64_t>(1, (int64_t)sms * per_sm / a.H));
    if (max_grid > 0) walks = std::min<int64_t>(walks, max_grid);
    if (grid_out) *grid_out = (int)walks;
    kern<<<(int)(walks * a.H), NT, sh, s>>>(a);
    return cudaGetLastError();
}
cudaError_t dispatch_ud(int L, bool k8, const UdArgs& a, size_t tables, int max_grid, int* grid_out, cudaStream_t s) {
    switch (L) {
        case 0: return k8 ? launch_ud<0, 8>(a, tables, max_grid, grid_out, s) : launch_ud<0, 16>(a, tables, max_grid, grid_out, s);
        case 1: return k8 ? launch_ud<1, 8>(a, tables, max_grid, grid_out, s) : launch_ud<1, 16>(a, tables, max_grid, grid_out, s);
        case 2: return k8 ? launch_ud<2, 8>(a, tables, max_grid, grid_out, s) : launch_ud<2, 16>(a, tables, max_grid, grid_out, s);
        default: return k8 ? launch_ud<3, 8>(a, tables, max_grid, grid_out, s) : launch_ud<3, 16>(a, tables, max_grid, grid_out, s);
    }
}
}  // namespace

cudaError_t launch_uvu_direct(const sobek_plan* p, const EdgeView& ev, int transposed, const float* src, const float* Y,
                              const float* phi, const float* R, float* dst, int* status, cudaStream_t s) {
    const UvuDirect& D = p->ud;
    const UvuDirectTables& T = D.dir[transposed ? 1 : 0];
    if (!D.ok || !T.d_woff || !T.d_ent || !T.d_nz || (transposed && (!ev.perm || !ev.recv))) return cudaErrorInvalidValue;
    UdArgs a{};
    a.row_ptr = ev.ptr; a.ids = transposed ? ev.recv : ev.col; a.perm = transposed ? ev.perm : nullptr; a.N = ev.N; a.E = ev.E;
    a.x = src; a.Y = Y; a.phi = phi; a.R = R; a.y = dst;
    a.woff = T.d_woff; a.ent = T.d_ent; a.nz = T.d_nz; a.n_nz = (int32_t)T.nz.size();
    a.C = D.C / D.H; a.Cf = D.C; a.H = D.H; a.K = p->K; a.nM = (int32_t)T.ent.size(); a.N_w = (int32_t)p->N_w;
    a.C_x = transposed ? p->C_y : p->C_x; a.C_y = transposed ? p->C_x : p->C_y; a.status = status;
    const size_t tables = (size_t)(T.ent.size() + T.nz.size()) * 8 + 16;
    KernelTimer kt(K_STATE, s);
    const cudaError_t e = dispatch_ud(D.L, p->K <= 8, a, tables, 0, nullptr, s);
    count_launch();
    return e;
}

// part[0 .. *n_parts)[K * N_w] = per-CTA sums of the weight adjoint over the receivers of `ev` (the receiver view);
// at most max_parts slices are written.  The caller adds them up in order.
cudaError_t launch_uvu_direct_wgrad(const sobek_plan* p, const EdgeView& ev, const float* x, const float* Y, const float* phi,
                                    const float* gy, float* part, int max_parts, int* n_parts, int* status, cudaStream_t s) {
    const UvuDirect& D = p->ud;
    const UvuDirectTables& T = D.dir[0];
    if (!D.ok || !T.d_woff || !T.d_ent || !T.d_nz || !part || max_parts < 1 || ev.perm) return cudaErrorInvalidValue;
    UdArgs a{};
    a.row_ptr = ev.ptr; a.ids = ev.col; a.perm = nullptr; a.N = ev.N; a.E = ev.E;
    a.x = x; a.Y = Y; a.phi = phi; a.R = nullptr; a.y = nullptr; a.own = gy; a.part = part;
    a.woff = T.d_woff; a.ent = T.d_ent; a.nz = T.d_nz; a.n_nz = (int32_t)T.nz.size();
    a.C = D.C / D.H; a.Cf = D.C; a.H = D.H; a.K = p->K; a.nM = (int32_t)T.ent.size(); a.N_w = (int32_t)p->N_w;
    a.C_x = p->C_x; a.C_y = p->C_y; a.status = status;
    const size_t tables = (size_t)(T.ent.size() + T.nz.size()) * 8 + 16;
    KernelTimer kt(K_STATE, s);
    const cudaError_t e = dispatch_ud(D.L, p->K <= 8, a, tables, max_parts, n_parts, s);
    count_launch();
    return e;
}

}  // namespace sobek
