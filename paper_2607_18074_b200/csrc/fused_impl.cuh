// Fused edge stream + node contraction (sm_100a): the receiver state never leaves the SM.
//
// One CTA owns a tile of NT consecutive nodes of one destination group, i.e. up to 128 rows
// (node, output component) of the group's contraction  dst = Z * Rp  (Eqs. receiver_state,
// receiver_mixing, receiver_matrix_product).  The contraction axis is walked in STAGES of 256
// columns = (path, block of 256/KP multiplicities, KP radial components):
//   * 8 producer warps stream the edges of the tile's nodes (lanes <-> multiplicities, one or two
//     nodes per warp) and accumulate Z[pi,u,q,o] = sum_e phi_e[q] C_e[pi,u,o] in registers, then
//     write the stage's slab of Z as split-bf16 (hi, lo) into shared memory in the 128-byte-swizzled
//     K-major layout the tensor core reads;
//   * one thread of warp 9 streams the matching slabs of R (bf16 hi, lo; B operand) from global
//     memory with TMA into a small ring;
//   * one thread of warp 8 issues tcgen05.mma (a_hi*b_hi + a_lo*b_hi + a_hi*b_lo, fp32 accumulator in
//     TMEM) per 64-column slab and commits to mbarriers that free the B slot / the A buffer;
//   * after the last stage warps 0..3 read the accumulator from TMEM and write the destination rows.
// Producers compute stage s+1 in registers while the tensor core consumes stage s; they only wait
// for the A buffer when they are ready to write.  With DUAL the producers build the directional
// state dZ of the double backward (Eq. receiver_double_adjoint) in one pass.  The same kernel runs
// the sender-owned transposed traversal.  Every mbarrier wait is bounded (ptx::mbar_wait).
#pragma once
#include <cuda_bf16.h>

#include "guard.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace sobek {
namespace {

using namespace ptx;

constexpr int FW = 8;                 // producer warps
constexpr int F_THREADS = (FW + 2) * 32;
constexpr int A_SLAB = 128 * 128;     // bytes of one 64-column slab of the A tile (128 rows x 128 B)
constexpr int A_BYTES = 4 * A_SLAB;   // 256 columns

__device__ __forceinline__ int64_t f_owner_of(const int64_t* __restrict__ row_ptr, int64_t N, int64_t e) {
    int64_t lo = 0, hi = N;
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (__ldg(row_ptr + mid) <= e) lo = mid; else hi = mid;
    }
    return lo;
}

// One producer task: the stage's slab of Z for RW nodes and one chunk of output components.
template <int D, int OC, int KP, int DS, bool DUAL>
__device__ __forceinline__ void produce(const FusedArgs& a, const FStage st, const DPath& P, const int64_t n0,
                                        const int nt, const int rb, const int o0, const int oc, float* sm,
                                        uint8_t* A_hi, uint8_t* A_lo, const uint32_t bar_empty_a,
                                        const uint32_t bar_full_a, const int stage_idx, const int lane) {
    constexpr int US = 256 / KP;      // multiplicities per stage
    constexpr int RW = 32 / US;       // nodes per warp
    const int sub = lane / US, ul = lane % US;
    const int t = rb * RW + sub;
    const bool has_node = t < nt;
    const int u = st.u0 + ul;
    const bool act_u = u < P.c_src;
    const int EB = a.EB, MS = a.MS, YS = a.dsh + 1;
    float* base = sm + sub * a.sub_floats;
    float* sM = base;                               // [EB][MS]
    float* sPhi = sM + EB * MS;                     // [EB][KP]
    float* sY = sPhi + EB * KP;                     // [EB][YS]
    int32_t* sSrc = (int32_t*)(sY + EB * YS);       // [EB]
    int32_t* sE = sSrc + EB;                        // [EB]
    float* sdM = (float*)(sE + EB);                 // DUAL: [EB][MS]
    float* sVphi = sdM + EB * MS;                   // DUAL: [EB][KP]
    float* sVY = sVphi + EB * KP;                   // DUAL: [EB][YS]
    const bool has_vx = DUAL && a.vsrc != nullptr, has_vY = DUAL && a.vY != nullptr,
               has_vphi = DUAL && a.vphi != nullptr;

    int64_t seg0 = 0, seg1 = 0;
    if (has_node) seg_bounds(a.ev.ptr, n0 + t, a.ev.E, a.status, seg0, seg1);
    int deg = (int)(seg1 - seg0);
    int maxdeg = deg;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) maxdeg = max(maxdeg, __shfl_xor_sync(0xffffffffu, maxdeg, o));

    float acc[OC][KP];
#pragma unroll
    for (int o = 0; o < OC; ++o)
#pragma unroll
        for (int q = 0; q < KP; ++q) acc[o][q] = 0.f;

    for (int b0 = 0; b0 < maxdeg; b0 += EB) {
        const int nb = max(0, min(EB, deg - b0));       // edges of this lane's node in the batch
        __syncwarp();
        if (ul < nb) {
            const int64_t pos = seg0 + b0 + ul;
            // an id out of range is reported; the edge then reads edge 0 / node 0 (valid memory, wrong data)
            int64_t eid = a.ev.perm ? (int64_t)a.ev.perm[pos] : pos;
            if (!id_ok(eid, a.ev.E, a.status)) eid = 0;
            sE[ul] = (int32_t)eid;
            int64_t sn = a.ev.transposed ? f_owner_of(a.ev.row_ptr, a.ev.N, eid) : (int64_t)a.ev.col[eid];
            if (!id_ok(sn, a.ev.N, a.status)) sn = 0;
            sSrc[ul] = (int32_t)sn;
        }
        __syncwarp();
        for (int i = ul; i < nb * a.dsh; i += US) {
            const int el = i / a.dsh, b = i - el * a.dsh;
            const int64_t g = (int64_t)sE[el] * a.dsh + b;
            sY[el * YS + b] = a.Y[g];
            if (has_vY) sVY[el * YS + b] = a.vY[g];
        }
        for (int i = ul; i < nb * KP; i += US) {
            const int el = i / KP, q = i - el * KP;
            const bool in = st.q0 + q < a.K;
            const int64_t g = (int64_t)sE[el] * a.K + st.q0 + q;
            sPhi[i] = in ? a.phi[g] : 0.f;
            if (has_vphi) sVphi[i] = in ? a.vphi[g] : 0.f;
        }
        __syncwarp();
        if (ul < nb) {      // M (and dM) of this lane's edge, own output components only
            const float* y = sY + ul * YS + P.sh_off;
            const float* vy = sVY + ul * YS + P.sh_off;
            for (int s = 0; s < P.d_src; ++s)
                for (int o = 0; o < OC; ++o) {
                    float m = 0.f, dm = 0.f;
                    if (o < oc) {
                        const int tt = P.tabM + s * D + o0 + o;
                        const int t0 = __ldg(a.tab_ptr + tt), t1 = __ldg(a.tab_ptr + tt + 1);
                        for (int k = t0; k < t1; ++k) {
                            const float c = __ldg(a.tab_coef + k);
                            const int b = __ldg(a.tab_idx + k);
                            m = fmaf(c, y[b], m);
                            if (has_vY) dm = fmaf(c, vy[b], dm);
                        }
                    }
                    sM[ul * MS + s * OC + o] = m;
                    if (has_vY) sdM[ul * MS + s * OC + o] = dm;
                }
        }
        __syncwarp();
        int maxnb = nb;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) maxnb = max(maxnb, __shfl_xor_sync(0xffffffffu, maxnb, o));
        constexpr int PB = (32 / (DS * (DUAL ? 2 : 1))) >= 8 ? 8 : ((32 / (DS * (DUAL ? 2 : 1))) >= 4 ? 4 : 2);
        for (int el0 = 0; el0 < maxnb; el0 += PB) {
            float xb[PB][DS], vxb[PB][DS];
#pragma unroll
            for (int pe = 0; pe < PB; ++pe) {
                const bool ok = (el0 + pe < nb) && act_u;
                const int64_t row = ok ? (int64_t)sSrc[el0 + pe] : 0;
                const float* xr = a.src + row * a.C_src + P.src_off + u;
#pragma unroll
                for (int s = 0; s < DS; ++s) xb[pe][s] = (ok && s < P.d_src) ? __ldg(xr + s * P.c_src) : 0.f;
                if (DUAL) {
                    const float* vr = a.vsrc + row * a.C_src + P.src_off + u;
#pragma unroll
                    for (int s = 0; s < DS; ++s) vxb[pe][s] = (has_vx && ok && s < P.d_src) ? __ldg(vr + s * P.c_src) : 0.f;
                }
            }
#pragma unroll
            for (int pe = 0; pe < PB; ++pe) {
                const int el = el0 + pe;
                if (el < nb) {
                    const float4* Me = reinterpret_cast<const float4*>(sM + el * MS);
                    const float4* dMe = reinterpret_cast<const float4*>(sdM + el * MS);
                    float C[OC], dC[OC];
#pragma unroll
                    for (int o = 0; o < OC; ++o) { C[o] = 0.f; dC[o] = 0.f; }
                    float4 mv = make_float4(0.f, 0.f, 0.f, 0.f), dmv = mv;
#pragma unroll
                    for (int s = 0; s < DS; ++s) {
                        if (s < P.d_src) {
#pragma unroll
                            for (int o = 0; o < OC; ++o) {
                                const int tt = s * OC + o;    // static after unrolling
                                if ((tt & 3) == 0) { mv = Me[tt >> 2]; if (has_vY) dmv = dMe[tt >> 2]; }
                                const float m = (tt & 3) == 0 ? mv.x : ((tt & 3) == 1 ? mv.y : ((tt & 3) == 2 ? mv.z : mv.w));
                                C[o] = fmaf(xb[pe][s], m, C[o]);
                                if (has_vx) dC[o] = fmaf(vxb[pe][s], m, dC[o]);
                                if (has_vY) {
                                    const float dm = (tt & 3) == 0 ? dmv.x : ((tt & 3) == 1 ? dmv.y : ((tt & 3) == 2 ? dmv.z : dmv.w));
                                    dC[o] = fmaf(xb[pe][s], dm, dC[o]);
                                }
                            }
                        }
                    }
                    const float4* ph4 = reinterpret_cast<const float4*>(sPhi + el * KP);
                    const float4* vph4 = reinterpret_cast<const float4*>(sVphi + el * KP);
#pragma unroll
                    for (int q4 = 0; q4 < KP / 4; ++q4) {
                        const float4 pv = ph4[q4];
                        const float pq[4] = {pv.x, pv.y, pv.z, pv.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j)
#pragma unroll
                            for (int o = 0; o < OC; ++o)
                                acc[o][4 * q4 + j] = fmaf(pq[j], DUAL ? dC[o] : C[o], acc[o][4 * q4 + j]);
                        if (has_vphi) {
                            const float4 vv = vph4[q4];
                            const float vq[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
                            for (int j = 0; j < 4; ++j)
#pragma unroll
                                for (int o = 0; o < OC; ++o) acc[o][4 * q4 + j] = fmaf(vq[j], C[o], acc[o][4 * q4 + j]);
                        }
                    }
                }
            }
        }
    }
    // ---- hand the slab to the tensor core: wait until the previous stage has been consumed.  The
    // "consumed" barriers form a ring of FW: a warp's tasks are at most FW stages apart, so the use of
    // barrier (s-1) % FW it waits for is never more than one phase away from the barrier's current phase.
    if (stage_idx > 0)
        mbar_wait(bar_empty_a + 8 * ((stage_idx - 1) % FW), (uint32_t)(((stage_idx - 1) / FW) & 1), a.status);
    if (has_node) {
#pragma unroll
        for (int o = 0; o < OC; ++o) {
            if (o < oc) {
                const int r = t * D + o0 + o;
#pragma unroll
                for (int c = 0; c < KP / 8; ++c) {       // 16-byte chunks of 8 bf16
                    const int k = ul * KP + 8 * c;        // column inside the stage
                    const int slab = k >> 6, chunk = (k & 63) >> 3;
                    const uint32_t off = slab * A_SLAB + (r >> 3) * 1024 + (r & 7) * 128 + ((chunk ^ (r & 7)) << 4);
                    __align__(16) __nv_bfloat16 h[8], l[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float v = act_u ? acc[o][8 * c + j] : 0.f;
                        h[j] = __float2bfloat16_rn(v);
                        l[j] = __float2bfloat16_rn(v - __bfloat162float(h[j]));
                    }
                    *reinterpret_cast<uint4*>(A_hi + off) = *reinterpret_cast<const uint4*>(h);
                    *reinterpret_cast<uint4*>(A_lo + off) = *reinterpret_cast<const uint4*>(l);
                }
            }
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncwarp();
    if (lane == 0) mbar_arrive(bar_full_a);
}

template <int D, int KP, bool DUAL>
__global__ void __launch_bounds__(F_THREADS, 1)
k_fused(const __grid_constant__ CUtensorMap tmBh, const __grid_constant__ CUtensorMap tmBl, const FusedArgs a) {
    constexpr int OC = D <= 5 ? D : (D == 7 ? 4 : 5);
    constexpr int NCH = D <= 5 ? 1 : 2;
    constexpr int US = 256 / KP, RW = 32 / US;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* A_hi = smem;
    uint8_t* A_lo = smem + A_BYTES;
    const uint32_t b_slab = (uint32_t)a.BN * 128;                       // bytes of one B slab (hi or lo)
    uint8_t* Bring = smem + 2 * A_BYTES;                                // [slots][hi, lo]
    uint64_t* bars = (uint64_t*)(Bring + (size_t)a.nb_slots * 2 * b_slab);
    // bars: [0] full_a, [1] accum, [2 .. 2+FW) empty_a ring, then [.. +S) full_b, [.. +S) empty_b
    uint32_t* tmem_holder = (uint32_t*)(bars + 2 + FW + 2 * a.nb_slots);
    float* prod = (float*)(((uintptr_t)(tmem_holder + 4) + 15) & ~(uintptr_t)15);
    const uint32_t bar0 = smem_u32(bars);
    const uint32_t bar_full_a = bar0, bar_acc = bar0 + 8, bar_empty_a = bar0 + 16;
    const uint32_t bar_b = bar0 + 8 * (2 + FW);
    const int S = a.nb_slots;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const int64_t n0 = (int64_t)blockIdx.x * a.NT;
    const int nt = (int)min((int64_t)a.NT, a.N - n0);
    const int TPS = (nt + RW - 1) / RW;          // producer tasks per (stage, component chunk)
    const int TPSC = TPS * NCH;
    const int nst = a.fs_count;

    if (threadIdx.x == 0) {
        mbar_init(bar_full_a, (uint32_t)TPSC);
        mbar_init(bar_acc, 1);
        for (int s = 0; s < FW; ++s) mbar_init(bar_empty_a + 8 * s, 1);
        for (int s = 0; s < S; ++s) { mbar_init(bar_b + 8 * s, 1); mbar_init(bar_b + 8 * (S + s), 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == FW) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"((uint32_t)a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp < FW) {
        // ---------------- producers
        float* sm = prod + (size_t)warp * RW * a.sub_floats;
        const int total = nst * TPSC;
        for (int tau = warp; tau < total; tau += FW) {
            const int si = tau / TPSC, r = tau - si * TPSC;
            const int ch = r / TPS, rb = r - ch * TPS;
            const FStage st = a.stages[a.fs_begin + si];
            const DPath P = a.paths[st.path];
            const int o0 = ch * OC, oc = min(OC, D - o0);
            if (P.d_src <= 3) produce<D, OC, KP, 3, DUAL>(a, st, P, n0, nt, rb, o0, oc, sm, A_hi, A_lo, bar_empty_a, bar_full_a, si, lane);
            else if (P.d_src <= 5) produce<D, OC, KP, 5, DUAL>(a, st, P, n0, nt, rb, o0, oc, sm, A_hi, A_lo, bar_empty_a, bar_full_a, si, lane);
            else produce<D, OC, KP, 9, DUAL>(a, st, P, n0, nt, rb, o0, oc, sm, A_hi, A_lo, bar_empty_a, bar_full_a, si, lane);
        }
        // ---------------- epilogue (warps 0..3 own TMEM lanes 32*warp .. +31)
        if (warp < 4) {
            mbar_wait(bar_acc, 0, a.status);
            tc_fence_after();
            const int r = warp * 32 + lane;
            const int t = r / D, o = r - t * D;
            float* drow = nullptr;
            if (t < nt) drow = a.dst + (n0 + t) * a.C_dst + a.G.dst_off + (int64_t)o * a.G.c_dst;
            for (int c0 = 0; c0 < a.BN; c0 += 16) {
                float v[16];
                tc_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
                if (drow) {
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (c0 + j < a.G.c_dst) drow[c0 + j] = a.accumulate ? drow[c0 + j] + v[j] : v[j];
                }
            }
        }
    } else if (warp == FW) {
        // ---------------- tensor-core issue
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(a.BN >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            const uint32_t ah = smem_u32(A_hi), al = smem_u32(A_lo), b0 = smem_u32(Bring);
            int sl = 0;
            for (int si = 0; si < nst; ++si) {
                mbar_wait(bar_full_a, (uint32_t)(si & 1), a.status);
                tc_fence_after();
                for (int j = 0; j < 4; ++j, ++sl) {
                    const int slot = sl % S;
                    mbar_wait(bar_b + 8 * slot, (uint32_t)((sl / S) & 1), a.status);
                    tc_fence_after();
                    const uint32_t bh = b0 + slot * 2 * b_slab, bl = bh + b_slab;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t dAh = make_desc(ah + j * A_SLAB + 32 * k, 16, 1024);
                        const uint64_t dAl = make_desc(al + j * A_SLAB + 32 * k, 16, 1024);
                        const uint64_t dBh = make_desc(bh + 32 * k, 16, 1024);
                        const uint64_t dBl = make_desc(bl + 32 * k, 16, 1024);
                        tc_mma_bf16(tmem_base, dAh, dBh, idesc, (sl > 0 || k > 0) ? 1u : 0u);
                        tc_mma_bf16(tmem_base, dAl, dBh, idesc, 1u);
                        tc_mma_bf16(tmem_base, dAh, dBl, idesc, 1u);
                    }
                    tc_commit(bar_b + 8 * (S + slot));          // B slot free when these MMAs retire
                }
                tc_commit(bar_empty_a + 8 * (si % FW));         // A buffer free
            }
            tc_commit(bar_acc);
        }
    } else {
        // ---------------- B operand loader
        if (lane == 0) {
            const uint32_t b0 = smem_u32(Bring);
            const int total = nst * 4;
            for (int sl = 0; sl < total; ++sl) {
                const int slot = sl % S;
                mbar_wait(bar_b + 8 * (S + slot), (uint32_t)(((sl / S) & 1) ^ 1), a.status);
                const uint32_t full = bar_b + 8 * slot;
                mbar_expect_tx(full, 2 * b_slab);
                const uint32_t bh = b0 + slot * 2 * b_slab;
                tma_load_2d(bh, &tmBh, sl * 64, 0, full);
                tma_load_2d(bh + b_slab, &tmBl, sl * 64, 0, full);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == FW) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols) : "memory");
    }
}

template <int KP, bool DUAL>
cudaError_t launch_fused_d(int D, const CUtensorMap& th, const CUtensorMap& tl, const FusedArgs& a, int grid, size_t sh,
                           cudaStream_t s) {
#define SOBEK_FUSED_CASE(DD)                                                                                  \
    case DD: {                                                                                                \
        auto kern = k_fused<DD, KP, DUAL>;                                                                    \
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh);     \
        if (e != cudaSuccess) return e;                                                                       \
        kern<<<grid, F_THREADS, sh, s>>>(th, tl, a);                                                          \
        return cudaGetLastError();                                                                            \
    }
    switch (D) {
        SOBEK_FUSED_CASE(1)
        SOBEK_FUSED_CASE(3)
        SOBEK_FUSED_CASE(5)
        SOBEK_FUSED_CASE(7)
        SOBEK_FUSED_CASE(9)
        default: return cudaErrorInvalidValue;
    }
#undef SOBEK_FUSED_CASE
}

}  // namespace
}  // namespace sobek
