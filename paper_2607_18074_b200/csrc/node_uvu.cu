// Node-side kernels of the channelwise (uvu) mode, Eq. uvu_connection.
//
// With tied multiplicities the receiver state Z_i[pi,u,q,o] (Eq. receiver_state) is the same as in the
// fully connected mode, but the radial projection no longer mixes channels: the three node-side
// contractions of the receiver program (Eqs. receiver_mixing, receiver_adjoint) lose their sum over a
// second multiplicity index and become elementwise products followed by short sums,
//     y_i[g,u,o]       = sum_{pi in P_g} sum_q Z_i[pi,u,q,o] * R[q, w_off(pi) + u]
//     Zbar_i[pi,u,q,o] = gy_i[g,u,o] * R[q, w_off(pi) + u]
//     gR[q, w_off(pi)+u] = sum_i sum_o Z_i[pi,u,q,o] * gy_i[g,u,o]
// so there is no GEMM: each kernel streams the bf16 (hi, lo) state of a node chunk once and is bound by HBM.
// The state layout is the one the edge kernels write and read: per destination group, rows (node, o) of
// pitch ld, column k = koff(pi) + q*c + u.  All paths of a group share its multiplicity c, hence
// k = (pl*K + q)*c + u with pl the path's index inside the group.
#include <cuda_bf16.h>

#include <algorithm>

#include "internal.h"

namespace sobek {
namespace {

__device__ __forceinline__ float bf_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
__device__ __forceinline__ float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf1(uint16_t v) { return __uint_as_float((uint32_t)v << 16); }

// V consecutive multiplicities of the state, hi + lo, starting at element index i (a multiple of V)
template <int V>
__device__ __forceinline__ void load_state(const uint16_t* __restrict__ zh, const uint16_t* __restrict__ zl, int64_t i,
                                           float* z) {
    if (V == 8) {
        const uint4 h = *reinterpret_cast<const uint4*>(zh + i), l = *reinterpret_cast<const uint4*>(zl + i);
        const uint32_t hw[4] = {h.x, h.y, h.z, h.w}, lw[4] = {l.x, l.y, l.z, l.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            z[2 * j] = bf_lo(hw[j]) + bf_lo(lw[j]);
            z[2 * j + 1] = bf_hi(hw[j]) + bf_hi(lw[j]);
        }
    } else if (V == 2) {
        const uint32_t h = *reinterpret_cast<const uint32_t*>(zh + i), l = *reinterpret_cast<const uint32_t*>(zl + i);
        z[0] = bf_lo(h) + bf_lo(l);
        z[1] = bf_hi(h) + bf_hi(l);
    } else {
        z[0] = bf1(zh[i]) + bf1(zl[i]);
    }
}

struct UvuGroup {
    const DPath* paths;   // the group's paths (device)
    int32_t np;           // paths in the group
    int32_t K;
    int64_t N_w;
    int32_t c, d;         // multiplicity and 2l+1 of the destination block
    int64_t rows;         // chunk nodes * d
    int64_t ld;           // row pitch of the bf16 state
    int64_t C_dst;        // row length of the destination feature matrix
};

// dst[(node, o), u] (+)= sum_{pi, q} Z[(node, o), (pl*K + q)*c + u] * R[q, w_off(pi) + u]
template <int V>
__global__ void k_uvu_mix(UvuGroup g, const uint16_t* __restrict__ zh, const uint16_t* __restrict__ zl,
                          const float* __restrict__ R, float* __restrict__ dst, int accumulate) {
    const int cv = g.c / V;
    const int64_t total = g.rows * cv;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / cv;
        const int u = (int)(i - r * cv) * V;
        float acc[V];
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] = 0.f;
        const int64_t zrow = r * g.ld + u;
        for (int pl = 0; pl < g.np; ++pl) {
            const int64_t wcol = g.paths[pl].w_off + u;
            const int64_t zp = zrow + (int64_t)pl * g.K * g.c;
#pragma unroll 4
            for (int q = 0; q < g.K; ++q) {
                float z[V];
                load_state<V>(zh, zl, zp + (int64_t)q * g.c, z);
#pragma unroll
                for (int v = 0; v < V; ++v) acc[v] = fmaf(z[v], __ldg(R + q * g.N_w + wcol + v), acc[v]);
            }
        }
        float* o = dst + (r / g.d) * g.C_dst + (r % g.d) * g.c + u;
#pragma unroll
        for (int v = 0; v < V; ++v) o[v] = accumulate ? o[v] + acc[v] : acc[v];
    }
}

// Zbar[(node, o), (pl*K + q)*c + u] = gy[(node, o), u] * R[q, w_off(pi) + u], as fp32 or as bf16 (hi, lo)
template <int V>
__global__ void k_uvu_zbar(UvuGroup g, const float* __restrict__ gy, const float* __restrict__ R,
                           float* __restrict__ zf, int64_t ldf, uint16_t* __restrict__ zh, uint16_t* __restrict__ zl) {
    const int cv = g.c / V;
    const int64_t per_row = (int64_t)g.np * g.K * cv;
    const int64_t total = g.rows * per_row;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / per_row;
        const int64_t j = i - r * per_row;
        const int pq = (int)(j / cv);
        const int u = (int)(j - (int64_t)pq * cv) * V;
        const int pl = pq / g.K, q = pq - pl * g.K;
        const float* gr = gy + (r / g.d) * g.C_dst + (r % g.d) * g.c + u;
        const float* Rr = R + q * g.N_w + g.paths[pl].w_off + u;
        float val[V];
#pragma unroll
        for (int v = 0; v < V; ++v) val[v] = gr[v] * __ldg(Rr + v);
        const int64_t k = (int64_t)pq * g.c + u;
        if (zf) {
#pragma unroll
            for (int v = 0; v < V; ++v) zf[r * ldf + k + v] = val[v];
        } else {
            __nv_bfloat16 h[V], l[V];
#pragma unroll
            for (int v = 0; v < V; ++v) {
                h[v] = __float2bfloat16_rn(val[v]);
                l[v] = __float2bfloat16_rn(val[v] - __bfloat162float(h[v]));
            }
            if (V == 8) {
                uint32_t hw[4], lw[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const __nv_bfloat162 hp = __halves2bfloat162(h[2 * j], h[2 * j + 1]), lp = __halves2bfloat162(l[2 * j], l[2 * j + 1]);
                    hw[j] = *reinterpret_cast<const uint32_t*>(&hp);
                    lw[j] = *reinterpret_cast<const uint32_t*>(&lp);
                }
                *reinterpret_cast<uint4*>(zh + r * g.ld + k) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                *reinterpret_cast<uint4*>(zl + r * g.ld + k) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
            } else if (V == 2) {
                *reinterpret_cast<__nv_bfloat162*>(zh + r * g.ld + k) = __halves2bfloat162(h[0], h[1]);
                *reinterpret_cast<__nv_bfloat162*>(zl + r * g.ld + k) = __halves2bfloat162(l[0], l[1]);
            } else {
                reinterpret_cast<__nv_bfloat16*>(zh)[r * g.ld + k] = h[0];
                reinterpret_cast<__nv_bfloat16*>(zl)[r * g.ld + k] = l[0];
            }
        }
    }
}

// part[z][q, w_off(pi) + u] = sum over the z-th slice of rows (node, o) of Z[(node, o), k] * gy[(node, o), u]
template <int V>
__global__ void k_uvu_wgrad(UvuGroup g, const uint16_t* __restrict__ zh, const uint16_t* __restrict__ zl,
                            const float* __restrict__ gy, float* __restrict__ part, int64_t part_stride, int splits) {
    const int cv = g.c / V;
    const int64_t cols = (int64_t)g.np * g.K * cv;
    const int z = blockIdx.y;
    const int64_t nodes = g.rows / g.d;
    const int64_t n_lo = nodes * z / splits, n_hi = nodes * (z + 1) / splits;
    for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < cols; j += (int64_t)gridDim.x * blockDim.x) {
        const int pq = (int)(j / cv);
        const int u = (int)(j - (int64_t)pq * cv) * V;
        const int pl = pq / g.K, q = pq - pl * g.K;
        const int64_t k = (int64_t)pq * g.c + u;
        float acc[V];
#pragma unroll
        for (int v = 0; v < V; ++v) acc[v] = 0.f;
        for (int64_t n = n_lo; n < n_hi; ++n)
            for (int o = 0; o < g.d; ++o) {
                float zv[V];
                load_state<V>(zh, zl, (n * g.d + o) * g.ld + k, zv);
                const float* gr = gy + n * g.C_dst + o * g.c + u;
#pragma unroll
                for (int v = 0; v < V; ++v) acc[v] = fmaf(zv[v], gr[v], acc[v]);
            }
        float* out = part + z * part_stride + q * g.N_w + g.paths[pl].w_off + u;
#pragma unroll
        for (int v = 0; v < V; ++v) out[v] = acc[v];
    }
}

// ---- multiplicities that are multiples of 8: one block per state row, threads (x = 8 multiplicities, y = (path, q)) ----
// Zbar row = gy row (x) R as bf16 (hi, lo) or fp32: thread (x, y) keeps its 8 output-adjoint values and walks the
// (path, q) pairs pq = y, y + blockDim.y, ...
__global__ void k_uvu_zbar_row(UvuGroup g, const float* __restrict__ gy, const float* __restrict__ R,
                               float* __restrict__ zf, int64_t ldf, uint16_t* __restrict__ zh, uint16_t* __restrict__ zl) {
    const int cv = g.c >> 3;
    const int64_t r = blockIdx.x;
    const float* gr = gy + (r / g.d) * g.C_dst + (r % g.d) * g.c;
    for (int x = threadIdx.x; x < cv; x += blockDim.x) {
        const int u = x << 3;
        float gv[8];
#pragma unroll
        for (int v = 0; v < 8; ++v) gv[v] = gr[u + v];
        for (int pq = threadIdx.y; pq < g.np * g.K; pq += blockDim.y) {
            const int pl = pq / g.K, q = pq - pl * g.K;
            const float* Rr = R + q * g.N_w + g.paths[pl].w_off + u;
            float val[8];
#pragma unroll
            for (int v = 0; v < 8; ++v) val[v] = gv[v] * __ldg(Rr + v);
            const int64_t k = (int64_t)pq * g.c + u;
            if (zf) {
#pragma unroll
                for (int v = 0; v < 8; ++v) zf[r * ldf + k + v] = val[v];
            } else {
                uint32_t hw[4], lw[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const __nv_bfloat162 hp = __floats2bfloat162_rn(val[2 * j], val[2 * j + 1]);
                    const float2 hf = __bfloat1622float2(hp);
                    const __nv_bfloat162 lp = __floats2bfloat162_rn(val[2 * j] - hf.x, val[2 * j + 1] - hf.y);
                    hw[j] = *reinterpret_cast<const uint32_t*>(&hp);
                    lw[j] = *reinterpret_cast<const uint32_t*>(&lp);
                }
                *reinterpret_cast<uint4*>(zh + r * g.ld + k) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                *reinterpret_cast<uint4*>(zl + r * g.ld + k) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
            }
        }
    }
}

// block shape of the row kernels: x covers the 8-multiplicity pieces of a row (at most 32), y the rest of 256 threads
dim3 row_block(int c, int ny_max) {
    const int bx = std::max(1, std::min(c / 8, 32));
    const int by = std::max(1, std::min(ny_max, 256 / bx));
    return dim3((unsigned)bx, (unsigned)by);
}

UvuGroup make_group(const sobek_plan* p, const Direction& dir, size_t gi, int64_t nn) {
    const DGroup& G = dir.groups[gi];
    UvuGroup g{};
    g.paths = dir.d_paths + G.path_begin;
    g.np = G.path_end - G.path_begin;
    g.K = p->K;
    g.N_w = p->N_w;
    g.c = G.c_dst;
    g.d = G.d_dst;
    g.rows = nn * G.d_dst;
    g.ld = dir.nk_ld[gi];
    g.C_dst = dir.C_dst;
    return g;
}

int grid_for(int64_t total) { return (int)std::max<int64_t>(1, std::min<int64_t>((total + 255) / 256, 148 * 16)); }

}  // namespace

cudaError_t launch_uvu_mix(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const void* zh,
                           const void* zl, const float* R, float* dst, int accumulate, cudaStream_t s0) {
    Fork fork(p, s0);
    for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
        const DGroup& G = dir.groups[gi];
        if (G.path_end == G.path_begin) continue;
        cudaStream_t s = fork.pick();
        const UvuGroup g = make_group(p, dir, gi, nn);
        const uint16_t* h = (const uint16_t*)zh + nn * dir.zb_off[gi];
        const uint16_t* l = (const uint16_t*)zl + nn * dir.zb_off[gi];
        float* d = dst + n0 * dir.C_dst + G.dst_off;
        KernelTimer kt(K_GEMM, s);
        if (g.c % 8 == 0) k_uvu_mix<8><<<grid_for(g.rows * (g.c / 8)), 256, 0, s>>>(g, h, l, R, d, accumulate);
        else if (g.c % 2 == 0) k_uvu_mix<2><<<grid_for(g.rows * (g.c / 2)), 256, 0, s>>>(g, h, l, R, d, accumulate);
        else k_uvu_mix<1><<<grid_for(g.rows * g.c), 256, 0, s>>>(g, h, l, R, d, accumulate);
        count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return fork.join();
}

cudaError_t launch_uvu_zbar(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const float* gy,
                            const float* R, float* Zbar, void* zqh, void* zql, cudaStream_t s0) {
    Fork fork(p, s0);
    for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
        const DGroup& G = dir.groups[gi];
        if (G.path_end == G.path_begin) continue;
        cudaStream_t s = fork.pick();
        const UvuGroup g = make_group(p, dir, gi, nn);
        const float* gsrc = gy + n0 * dir.C_dst + G.dst_off;
        float* zf = zqh ? nullptr : Zbar + nn * G.z_off;
        uint16_t* h = zqh ? (uint16_t*)zqh + nn * dir.zb_off[gi] : nullptr;
        uint16_t* l = zqh ? (uint16_t*)zql + nn * dir.zb_off[gi] : nullptr;
        const int64_t total = g.rows * (int64_t)g.np * g.K * g.c;
        KernelTimer kt(K_GEMM, s);
        if (g.c % 8 == 0) k_uvu_zbar_row<<<(unsigned)g.rows, row_block(g.c, g.np * g.K), 0, s>>>(g, gsrc, R, zf, G.D, h, l);
        else if (g.c % 2 == 0) k_uvu_zbar<2><<<grid_for(total / 2), 256, 0, s>>>(g, gsrc, R, zf, G.D, h, l);
        else k_uvu_zbar<1><<<grid_for(total), 256, 0, s>>>(g, gsrc, R, zf, G.D, h, l);
        count_launch();
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return fork.join();
}

cudaError_t launch_uvu_wgrad(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const void* zh,
                             const void* zl, const float* gy, float* gR_acc, float* part, int splits,
                             cudaStream_t s0) {
    const int64_t KN = (int64_t)p->K * p->N_w;
    const int sp = (int)std::max<int64_t>(1, std::min<int64_t>(splits, nn));
    {
        Fork fork(p, s0);
        for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
            const DGroup& G = dir.groups[gi];
            if (G.path_end == G.path_begin) continue;
            cudaStream_t s = fork.pick();
            const UvuGroup g = make_group(p, dir, gi, nn);
            const uint16_t* h = (const uint16_t*)zh + nn * dir.zb_off[gi];
            const uint16_t* l = (const uint16_t*)zl + nn * dir.zb_off[gi];
            const float* gsrc = gy + n0 * dir.C_dst + G.dst_off;
            const int V = g.c % 8 == 0 ? 8 : g.c % 2 == 0 ? 2 : 1;
            const int64_t cols = (int64_t)g.np * g.K * (g.c / V);
            dim3 grid((unsigned)std::max<int64_t>(1, (cols + 127) / 128), (unsigned)sp);
            KernelTimer kt(K_GEMM, s);
            if (V == 8) k_uvu_wgrad<8><<<grid, 128, 0, s>>>(g, h, l, gsrc, part, KN, sp);
            else if (V == 2) k_uvu_wgrad<2><<<grid, 128, 0, s>>>(g, h, l, gsrc, part, KN, sp);
            else k_uvu_wgrad<1><<<grid, 128, 0, s>>>(g, h, l, gsrc, part, KN, sp);
            count_launch();
            cudaError_t e = cudaGetLastError();
            if (e != cudaSuccess) return e;
        }
        cudaError_t e = fork.join();
        if (e != cudaSuccess) return e;
    }
    // every column of R belongs to exactly one path, so the groups' kernels together wrote all of part[0..sp)
    return launch_reduce_parts(gR_acc, part, KN, KN, sp, s0);
}

}  // namespace sobek
