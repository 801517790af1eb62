// Receiver-owned edge pass on the tensor cores (sm_100a, tcgen05 / TMEM), warp-specialised.
//
// The two edge outputs of the backward program (Section "Receiver-factorized backward";
// Eqs. streamed_radial_adjoints, streamed_operand_adjoints) share, per receiver i, source irrep block and
// batch of 16 edges, the dense contraction over the multiplicity u
//     D[(s,e), (comp,q)] = sum_u x_{src(e)}[s,u] * Zbar_i[(comp,q), u]
// whose operands are plain copies: the gathered bf16 (hi, lo) sender rows (rows (s,e), K-major) and the
// bf16 (hi, lo) rows of the adjoint state Zbar = gy R^T of the receiver (rows (comp,q), K-major), both in
// the 128-byte-swizzled layout that tcgen05.mma reads.  The FP32 pipes only run the epilogue
//     gM_e[s,comp] = sum_q phi_e[q] * D[(s,e),(comp,q)]          -> gY_e[b]  = sum c[s,b,comp] gM_e[s,comp]
//     gphi_e[q]    = sum_{s,comp} M_e[s,comp] * D[(s,e),(comp,q)]
// with one thread per accumulator row (s,e).  fp32 parity comes from the split-bf16 product
// a*b ~= a_hi*b_hi + a_lo*b_hi + a_hi*b_lo.  Every output element has exactly one writer and every sum
// runs in a fixed order (bitwise reproducible).
//
// With DUAL the pass evaluates the second-order terms that share Zbar (Eq. streamed_operand_second_adjoints)
//     hphi_e += <Zbar, C(vx,Y) + C(x,vY)>,   hY_e += CG^T_Y(vx, phi Zbar) + CG^T_Y(x, vphi Zbar)
// from D (sender rows of x) and Dv (sender rows of vx):
//     gM = sum_q ( vphi[q] D + phi[q] Dv ),   gphi[q] += dM D + M Dv.
//
// One launch per set of accumulator tiles (the first writes the outputs, the others accumulate).  The batch
// size tb of a set is the largest power of two (16..128) whose rows (s, e) = d_src * tb still fill one
// 128-row tile, so that the accumulator rows - one epilogue thread each - are used as fully as possible.
// Roles of a CTA (one receiver at a time, its edges in batches of tb): loader warps (cp.async of the Zbar slabs of a set, of the batch's phi / Y
// rows and of the sender rows into a two-stage ring), one MMA thread (two TMEM accumulator buffers), and
// compute warps (coupling matrices M_e from the sparse CG table, epilogue, fixed-order reductions, output).
// Every mbarrier wait is bounded.
#include <cuda_bf16.h>

#include <algorithm>

#include "geometry.cuh"
#include "guard.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace sobek {
namespace {

using namespace ptx;

// Warps of a CTA: NCW = 8 compute warps, NLW = 3 loader warps, one MMA warp (twelve warps: registers are handed out as
// if a CTA had a multiple of four warps, so the third loader warp is free).  MINB = CTAs per SM the kernel is compiled
// for: 2 where the shared memory of a set allows it, else 1 with the whole register file.
constexpr int NS = 2;           // ring stages

struct EtArgs {
    const TSet* sets;
    const TUnit* units;
    const TBlk* blks;
    const EntS* ents;           // of the launch's set
    const NzS* nz;
    const CompS* comps;
    const int32_t* inv_ptr;     // of the launch's set: dsh+1 offsets into inv (b -> terms (entry, coef))
    const NzS* inv;             // terms: b field = entry inside the set
    const int64_t* row_ptr;
    const int32_t* col;
    int64_t node0, n_nodes;
    const int4* oseg;           // the chunk's nodes in processing order {local node, segment begin, end} or NULL
    int64_t N, E;               // sizes of the graph: every gathered id and segment bound is checked against them
    const __nv_bfloat16* sh;
    const __nv_bfloat16* sl;
    const __nv_bfloat16* vsh;
    const __nv_bfloat16* vsl;
    const float* Y;
    const float* vY;
    const float* phi;
    const float* vphi;
    const __nv_bfloat16* zqh;   // bf16 (hi, lo) adjoint state of the chunk, laid out like the stream's state
    const __nv_bfloat16* zql;
    float* gphi;
    float* gY;
    // geometry mode: Y and phi are recomputed from the edge vectors [E][3] (Y, phi are NULL), and the adjoints of
    // both are contracted with their Jacobians into the adjoint of the edge vectors g_rvec [E][3] (gphi, gY are NULL;
    // phi_mode = Y_mode = mode of g_rvec)
    const float* rvec;
    float* g_rvec;
    float geo_rc;
    int32_t geo_basis, geo_p;
    int32_t phi_mode, Y_mode;   // 0 skip, 1 overwrite, 2 accumulate
    int32_t K, dsh, C_src, set;
    int32_t tb, lg;             // edges per batch (power of two) and its log2
    int32_t x_cap, z_cap, nent, tmem_cols, acc_cols, nnz, ninv, nunit, ncomp;
    int* status;
};

// Everything the roles look up per batch or row lives in shared memory (with most of the SM's L1 given to
// the operand regions, table reads from global memory would mostly go to L2).
struct UInfo {     // a unit of the launch's set
    uint32_t idesc, z_off, z_kb, x_off, x_kb, ksteps, nmt, npad, ncomp, comp_begin, d_src, c_src;
};

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// i / d for the small index ranges of the loaders (0 <= i, i * d < 2^20) by one multiplication: an integer division
// costs some thirty instructions, which the loader warps cannot hide
struct SmallDiv {
    uint32_t m;
    __device__ __forceinline__ explicit SmallDiv(int d) : m((1u << 20) / (uint32_t)d + 1u) {}
    __device__ __forceinline__ int operator()(int i) const { return (int)(((uint32_t)i * m) >> 20); }
};
template <int NCW>
__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory"); }
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async4_zfill(uint32_t dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
// the wait for the tensor-memory loads in flight; the loaded registers pass through it so that nothing that reads
// them can be scheduled ahead of it
__device__ __forceinline__ void tc_wait_ld16(float* v) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+f"(v[0]), "+f"(v[1]), "+f"(v[2]), "+f"(v[3]), "+f"(v[4]), "+f"(v[5]), "+f"(v[6]), "+f"(v[7]),
                   "+f"(v[8]), "+f"(v[9]), "+f"(v[10]), "+f"(v[11]), "+f"(v[12]), "+f"(v[13]), "+f"(v[14]), "+f"(v[15])
                 :: "memory");
}
__device__ __forceinline__ void tc_ld8_nowait(uint32_t taddr, float* v) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
#pragma unroll
    for (int i = 8; i < 16; ++i) v[i] = 0.f;
}

// per-stage raw area (floats): phi rows [tb][KP], (vphi), Y written transposed [dsh][tb], (vY), sender ids [tb]
__host__ __device__ inline int raw_floats(int KP, bool dual, int dsh, int tb) {
    const int n = dual ? 2 : 1;
    return n * tb * KP + n * dsh * tb + tb;
}

// GEO: the geometry mode (edge inputs recomputed from edge vectors, adjoint of the edge vectors out); plain pass only
// segment of the node at position v of the chunk's processing order; returns the node's local index
__device__ __forceinline__ int64_t et_bounds(const EtArgs& a, int64_t v, int* status, int64_t& s0, int64_t& s1) {
    if (a.oseg) { const int4 q = __ldg(a.oseg + v); s0 = q.y; s1 = q.z; return q.x; }
    seg_bounds(a.row_ptr, a.node0 + v, a.E, status, s0, s1);
    return v;
}

template <int KP, bool DUAL, int NCW, int NLW, bool GEO, int MINB>
__global__ void __launch_bounds__((NCW + NLW + 1) * 32, MINB) k_edge_tc(const EtArgs a) {
    constexpr int TT = (NCW + NLW + 1) * 32;
    // geometry mode: the last loader warp does not copy but recomputes phi and Y of every batch from the edge vectors
    constexpr int NLG = GEO ? NLW - 1 : NLW;
    constexpr int NH = NCW / 4;            // column parts of an accumulator tile: one per group of four compute warps
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    constexpr int NRAW = DUAL ? 2 : 1;     // raw stages: phi and Y, plus their directions
    const int tb = a.tb, lg = a.lg, PS = a.tb;       // PS: row pitch of the per-entry arrays (a warp holds whole rows of tb
                                                     // edges: no padding is needed, and shared memory decides the number of sets)
    const uint32_t raw_bytes = (uint32_t)((raw_floats(KP, DUAL, a.dsh, tb) * 4 + 1023) & ~1023);
    const uint32_t stage_bytes = (uint32_t)(2 * a.x_cap) + raw_bytes;
    uint8_t* sRing = smem;                                     // stages: Xh Xl raw
    uint8_t* sZ = sRing + (size_t)NS * stage_bytes;            // Zbar slabs of the set: hi, lo
    uint8_t* meta = sZ + (size_t)2 * a.z_cap;
    float* sM = reinterpret_cast<float*>(meta);                // [nent][PS] coupling matrices of the batch
    float* sdM = sM + (size_t)a.nent * PS;                     // DUAL
    float* sGM = sdM + (DUAL ? (size_t)a.nent * PS : 0);       // [nent][PS]
    float* sPphi = sGM + (size_t)a.nent * PS;                  // [NCW*32][KP]: one row per compute thread
    float* sGeo = sPphi + NCW * 32 * KP;                       // [tb][KP + dsh]: gphi and gY of the batch (geometry mode)
    uint64_t* bars = reinterpret_cast<uint64_t*>(sGeo + (size_t)tb * (KP + a.dsh));
    // bars: full[NS], free[NS], acc_full[2], acc_free[2], (tmem address), zfull[nunit], zfree[nunit]
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * NS + 6);
    UInfo* sU = reinterpret_cast<UInfo*>(bars + 2 * NS + 8 + 2 * a.nunit);     // [nunit]
    TBlk* sBlk = reinterpret_cast<TBlk*>(sU + a.nunit);                // [nunit]
    CompS* sComp = reinterpret_cast<CompS*>(sBlk + a.nunit);           // [ncomp]
    EntS* sEnt = reinterpret_cast<EntS*>(sComp + a.ncomp);             // [nent]
    NzS* sNz = reinterpret_cast<NzS*>(sEnt + a.nent);                  // [nnz]
    NzS* sInv = sNz + a.nnz;                                           // [ninv]
    int32_t* sInvPtr = reinterpret_cast<int32_t*>(sInv + a.ninv);      // [dsh + 1]
    const uint32_t bar0 = smem_u32(bars);
    // the Zbar slabs of a unit have a pair of barriers of their own: a unit's slabs are refilled for the next receiver
    // as soon as the last batch's MMAs of that unit have retired, while the later units are still being multiplied
    const uint32_t bar_full = bar0, bar_free = bar0 + 8 * NS, bar_accfull = bar0 + 16 * NS, bar_accfree = bar_accfull + 16,
                   bar_zfull = bar0 + 8 * (2 * NS + 8), bar_zfree = bar_zfull + 8 * (uint32_t)a.nunit;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool has_vx = DUAL && a.vsh != nullptr, has_vY = DUAL && a.vY != nullptr, has_vphi = DUAL && a.vphi != nullptr;
    const bool use_x = !DUAL || has_vY || has_vphi;     // D (rows of x) is needed
    const bool use_vx = has_vx;                         // Dv (rows of vx) is needed
    const bool any_op = use_x || use_vx;
    // sub-batches per batch of edges: one per product that is needed (op = 0: rows of x, op = 1: rows of vx)
    const int nsub = (use_x ? 1 : 0) + (use_vx ? 1 : 0);
    const TSet S = a.sets[a.set];

    if (tid == 0) {
        // a stage is released by the commit of the batch's MMAs and by every compute thread (raw rows read)
        for (int s = 0; s < NS; ++s) { mbar_init(bar_full + 8 * s, NLW * 32); mbar_init(bar_free + 8 * s, 2); }
        for (int u = 0; u < a.nunit; ++u) { mbar_init(bar_zfull + 8 * u, NLG * 32); mbar_init(bar_zfree + 8 * u, 1); }
        for (int t = 0; t < 2; ++t) { mbar_init(bar_accfull + 8 * t, 1); mbar_init(bar_accfree + 8 * t, NCW); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // zero what is never written later: the raw rows of padded radial components / absent directions, and the
    // Zbar slab rows of padded radial components (they meet zeros of phi, but must stay finite)
    {
        const int words = (int)(stage_bytes / 4), x_words = 2 * a.x_cap / 4;
        for (int i = tid; i < NS * words; i += TT) {
            const int st = i / words, w = i - st * words;
            if (w >= x_words) reinterpret_cast<uint32_t*>(sRing + (size_t)st * stage_bytes)[w] = 0u;
        }
        for (int i = tid; i < 2 * a.z_cap / 4; i += TT) reinterpret_cast<uint32_t*>(sZ)[i] = 0u;
    }
    // tables of the set
    for (int i = tid; i < S.nunit; i += TT) {
        const TUnit U = a.units[S.unit_begin + i];
        const TBlk B = a.blks[U.blk];
        UInfo u;
        u.npad = (uint32_t)U.pad[0];
        // D = F32, A = B = BF16, both K-major, M = 128, N = npad
        u.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((u.npad >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        u.z_off = (uint32_t)U.a_off; u.z_kb = (uint32_t)U.slab_stride;
        u.x_off = (uint32_t)B.b_off; u.x_kb = (uint32_t)B.atom_stride;
        u.ksteps = (uint32_t)(B.c_src >> 4); u.nmt = (uint32_t)((B.d_src * tb + 127) / 128);
        u.ncomp = (uint32_t)U.ncomp; u.comp_begin = (uint32_t)(U.comp_begin - a.units[S.unit_begin].comp_begin);
        u.d_src = (uint32_t)B.d_src; u.c_src = (uint32_t)B.c_src;
        sU[i] = u;
    }
    for (int i = tid; i < S.nblk; i += TT) sBlk[i] = a.blks[S.blk_begin + i];
    {
        const int c0 = a.units[S.unit_begin].comp_begin;
        for (int i = tid; i < a.ncomp; i += TT) sComp[i] = a.comps[c0 + i];
    }
    for (int i = tid; i < S.nent; i += TT) sEnt[i] = a.ents[i];
    for (int i = tid; i < a.nnz; i += TT) sNz[i] = a.nz[i];
    for (int i = tid; i <= a.dsh; i += TT) sInvPtr[i] = a.inv_ptr[i];
    for (int i = tid; i < a.ninv; i += TT) sInv[i] = a.inv[i];
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"((uint32_t)a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;

    if (warp >= NCW && warp < NCW + NLG) {
        // =========================== loader warps ===========================
        const int lt = (warp - NCW) * 32 + lane;
        uint32_t it = 0, zi = 0;
        for (int64_t v = blockIdx.x; v < a.n_nodes; v += gridDim.x) {
            int64_t seg0, seg1;
            const int64_t nl = et_bounds(a, v, a.status, seg0, seg1);
            if (!any_op) seg1 = seg0;
            if (seg1 <= seg0) continue;
            // ---- Zbar slabs, unit by unit (each once the previous receiver's MMAs of that unit have read theirs);
            // a loader warp takes whole components: K rows of c_src multiplicities, contiguous in the state
            auto load_zbar = [&]() {
                for (int ui = 0; ui < S.nunit; ++ui) {
                    const UInfo U = sU[ui];
                    if (zi > 0) mbar_wait(bar_zfree + 8 * ui, (zi - 1) & 1, a.status);
                    const int cpr = (int)U.c_src >> 3;
                    const int n_it = a.K * cpr;
                    const SmallDiv by_cpr(cpr);
                    for (int cl = warp - NCW; cl < (int)U.ncomp; cl += NLG) {
                        const CompS cp = sComp[U.comp_begin + cl];
                        const int64_t g0 = a.n_nodes * cp.zoff + (nl * cp.d_dst + cp.o) * (int64_t)cp.ld + cp.koff;
                        const __nv_bfloat16* gh = a.zqh + g0;
                        const __nv_bfloat16* gl = a.zql + g0;
                        const uint32_t d0 = smem_u32(sZ) + U.z_off + (uint32_t)(cl * KP) * 128u;
                        for (int i = lane; i < n_it; i += 32) {
                            const int q = by_cpr(i), j = i - q * cpr;
                            const int r = cl * KP + q;
                            const uint32_t d = d0 + (uint32_t)((j >> 3) * U.z_kb + q * 128 + (((j & 7) ^ (r & 7)) << 4));
                            cp_async16_zfill(d, gh + 8 * i, 16);
                            cp_async16_zfill(d + (uint32_t)a.z_cap, gl + 8 * i, 16);
                        }
                    }
                    cp_async_arrive(bar_zfull + 8 * ui);
                }
                ++zi;
            };
            // ---- the batches of the receiver; the first one is staged ahead of the Zbar slabs (its stage does not wait
            // for the previous receiver's MMAs to end)
            const int nbat = (int)((seg1 - seg0 + tb - 1) >> lg) * nsub;
            for (int bi_ = 0; bi_ < nbat; ++bi_, ++it) {
                if (bi_ == 1) load_zbar();
                const int bq = nsub == 2 ? bi_ >> 1 : bi_;
                const int64_t b0 = seg0 + (int64_t)bq * tb;
                const int sb = bi_ - bq * nsub;
                const int op = use_x ? sb : 1;
                const int nb = (int)min((int64_t)tb, seg1 - b0);
                const int st = (int)(it % NS);
                if (it >= NS) mbar_wait(bar_free + 8 * st, ((it / NS) & 1) ^ 1, a.status);
                uint8_t* stage = sRing + (size_t)st * stage_bytes;
                const uint32_t stage_u = smem_u32(stage);
                const uint32_t raw_u = stage_u + (uint32_t)(2 * a.x_cap);
                // sender ids of the batch (each loader warp keeps its own copy of all of them)
                int32_t* sIds = reinterpret_cast<int32_t*>(stage + 2 * a.x_cap) + NRAW * tb * KP + NRAW * a.dsh * PS + (warp - NCW) * 0;
                for (int e = lane; e < tb; e += 32) {      // -1: no such edge, or a sender id out of range (reported)
                    int32_t sid = -1;
                    if (e < nb) { sid = a.col[b0 + e]; if (!id_ok(sid, a.N, a.status)) sid = -1; }
                    sIds[e] = sid;
                }
                __syncwarp();
                if constexpr (GEO) {
                    // phi and Y of the stage come from the geometry warp
                } else {
                {
                    const bool v16 = (a.K & 3) == 0;
                    const int per = v16 ? a.K / 4 : a.K;
                    const int n_it = tb * per;
                    const SmallDiv by_per(per);
                    for (int i = lt; i < n_it; i += NLG * 32) {
                        const int e = by_per(i), j = i - e * per;
                        const int64_t ee = b0 + min(e, nb - 1);
                        const uint32_t ok = e < nb ? 1u : 0u;
                        if (v16) {
                            cp_async16_zfill(raw_u + (uint32_t)(e * KP + 4 * j) * 4, a.phi + ee * a.K + 4 * j, ok * 16);
                            if (has_vphi) cp_async16_zfill(raw_u + (uint32_t)(tb * KP + e * KP + 4 * j) * 4, a.vphi + ee * a.K + 4 * j, ok * 16);
                        } else {
                            cp_async4_zfill(raw_u + (uint32_t)(e * KP + j) * 4, a.phi + ee * a.K + j, ok * 4);
                            if (has_vphi) cp_async4_zfill(raw_u + (uint32_t)(tb * KP + e * KP + j) * 4, a.vphi + ee * a.K + j, ok * 4);
                        }
                    }
                }
                {   // Y (and vY), transposed: raw[b][PS + e]
                    const uint32_t y_u = raw_u + (uint32_t)(NRAW * tb * KP) * 4;
                    const int n_it = tb * a.dsh;
                    const SmallDiv by_dsh(a.dsh);
                    for (int i = lt; i < n_it; i += NLG * 32) {
                        const int e = by_dsh(i), b = i - e * a.dsh;
                        const int64_t ee = b0 + min(e, nb - 1);
                        const uint32_t ok = e < nb ? 4u : 0u;
                        cp_async4_zfill(y_u + (uint32_t)(b * PS + e) * 4, a.Y + ee * a.dsh + b, ok);
                        if (has_vY) cp_async4_zfill(y_u + (uint32_t)(a.dsh * PS + b * PS + e) * 4, a.vY + ee * a.dsh + b, ok);
                    }
                }
                }
                // sender rows: rows (s, e) of 128 bytes per 64 multiplicities, 128-byte swizzle
                for (int bi = 0; bi < S.nblk; ++bi) {
                    const TBlk B = sBlk[bi];
                    const int cpr = B.c_src >> 3;
                    const int npair = tb * cpr;
                    const SmallDiv by_cpr(cpr);
                    for (int pr = lt; pr < npair; pr += NLG * 32) {
                        const int e = by_cpr(pr), j = pr - e * cpr;
                        const int32_t sid = sIds[e];
                        const uint32_t ok = sid >= 0 ? 16u : 0u;
                        const int u = 8 * j;
                        uint32_t d = stage_u + (uint32_t)(B.b_off + (u >> 6) * B.atom_stride + e * 128 + ((((u & 63) >> 3) ^ (e & 7)) << 4));
                        const int64_t g = (int64_t)max(sid, 0) * a.C_src + B.src_off + u;
                        const __nv_bfloat16* ph = (op == 0 ? a.sh : a.vsh) + g;
                        const __nv_bfloat16* pl = (op == 0 ? a.sl : a.vsl) + g;
                        for (int sdx = 0; sdx < B.d_src; ++sdx) {
                            cp_async16_zfill(d, ph, ok);
                            cp_async16_zfill(d + (uint32_t)a.x_cap, pl, ok);
                            d += (uint32_t)B.slab_bytes; ph += B.c_src; pl += B.c_src;
                        }
                    }
                }
                cp_async_arrive(bar_full + 8 * st);
            }
            if (nbat == 1) load_zbar();
        }
    } else if (GEO && warp == NCW + NLG) {
        // =========================== geometry warp ===========================
        // walks the same receivers and batches as the loaders; lane <-> (edge, share of the radial indices and components)
        uint32_t it = 0;
        for (int64_t v = blockIdx.x; v < a.n_nodes; v += gridDim.x) {
            int64_t seg0, seg1;
            et_bounds(a, v, nullptr, seg0, seg1);
            if (!any_op) seg1 = seg0;
            for (int64_t b0 = seg0; b0 < seg1; b0 += tb, ++it) {
                const int nb = (int)min((int64_t)tb, seg1 - b0);
                const int st = (int)(it % NS);
                if (it >= NS) mbar_wait(bar_free + 8 * st, ((it / NS) & 1) ^ 1, a.status);
                uint8_t* stage = sRing + (size_t)st * stage_bytes;
                float* rawf = reinterpret_cast<float*>(stage + 2 * a.x_cap);       // phi rows [tb][KP]
                float* yT = rawf + NRAW * tb * KP;                                 // Y transposed [dsh][PS]
                const int nsh = max(1, 32 >> lg);
                const int qw = (a.K + nsh - 1) / nsh, bw = (a.dsh + nsh - 1) / nsh;
                for (int i = lane; i < tb * nsh; i += 32) {
                    const int e = i & (tb - 1), sh = i >> lg;
                    const bool okb = e < nb;
                    float rx = 0.f, ry = 0.f, rz = 1.f;
                    if (okb) { const float* rp = a.rvec + (b0 + e) * 3; rx = __ldg(rp); ry = __ldg(rp + 1); rz = __ldg(rp + 2); }
                    const float r = sqrtf(rx * rx + ry * ry + rz * rz), ir = 1.f / r;
                    const int q_lo = sh * qw, q_hi = min(a.K, q_lo + qw), b_lo = sh * bw, b_hi = min(a.dsh, b_lo + bw);
                    geo_radial(r, a.K, a.geo_rc, a.geo_basis, a.geo_p, [&](int q, float f, float) {
                        if (q >= q_lo && q < q_hi) rawf[e * KP + q] = okb ? f : 0.f;
                    });
                    geo_sh(rx * ir, ry * ir, rz * ir, [&](int b, float yb, float, float, float) {
                        if (b >= b_lo && b < b_hi) yT[b * PS + e] = okb ? yb : 0.f;
                    });
                }
                mbar_arrive(bar_full + 8 * st);      // release: the stores above are visible to whoever sees the stage full
            }
        }
    } else if (warp == NCW + NLW) {
        // =========================== MMA warp ===========================
        if (lane == 0) {
            uint32_t it = 0, zi = 0, ai = 0;
            const uint32_t sZ_u = smem_u32(sZ);
            for (int64_t v = blockIdx.x; v < a.n_nodes; v += gridDim.x) {
                int64_t seg0, seg1;
                et_bounds(a, v, nullptr, seg0, seg1);
                if (!any_op) seg1 = seg0;
                if (seg1 <= seg0) continue;
                for (int64_t b0 = seg0; b0 < seg1; b0 += tb)
                for (int sb = 0; sb < nsub; ++sb, ++it) {
                    const bool first = b0 == seg0 && sb == 0, last = b0 + tb >= seg1 && sb == nsub - 1;
                    const int st = (int)(it % NS);
                    mbar_wait(bar_full + 8 * st, (it / NS) & 1, a.status);
                    fence_async_smem();
                    tc_fence_after();
                    const uint32_t sX_u = smem_u32(sRing + (size_t)st * stage_bytes);
                    for (int ui = 0; ui < S.nunit; ++ui, ++ai) {
                        const UInfo U = sU[ui];
                        const uint32_t buf = ai & 1;
                        if (first) mbar_wait(bar_zfull + 8 * ui, zi & 1, a.status);
                        if (ai >= 2) mbar_wait(bar_accfree + 8 * buf, ((ai >> 1) & 1) ^ 1, a.status);
                        fence_async_smem();
                        tc_fence_after();
                        for (uint32_t mt = 0; mt < U.nmt; ++mt) {
                            const uint32_t d_tmem = tmem_base + buf * (uint32_t)a.acc_cols + mt * U.npad;
                            for (uint32_t ks = 0; ks < U.ksteps; ++ks) {
                                const uint32_t kb = ks >> 2, kk = ks & 3;
                                const uint32_t xh = sX_u + U.x_off + kb * U.x_kb + mt * (128u * 128u) + 32u * kk;
                                const uint32_t xl = xh + a.x_cap;
                                const uint32_t zh = sZ_u + U.z_off + kb * U.z_kb + 32u * kk;
                                const uint32_t zl = zh + a.z_cap;
                                const uint64_t dXh = make_desc(xh, 16, 1024), dXl = make_desc(xl, 16, 1024);
                                const uint64_t dZh = make_desc(zh, 16, 1024), dZl = make_desc(zl, 16, 1024);
                                tc_mma_bf16(d_tmem, dXh, dZh, U.idesc, ks > 0 ? 1u : 0u);
                                tc_mma_bf16(d_tmem, dXl, dZh, U.idesc, 1u);
                                tc_mma_bf16(d_tmem, dXh, dZl, U.idesc, 1u);
                            }
                        }
                        tc_commit(bar_accfull + 8 * buf);
                        if (last) tc_commit(bar_zfree + 8 * ui);
                    }
                    tc_commit(bar_free + 8 * st);
                }
                ++zi;
            }
        }
    } else {
        // =========================== compute warps ===========================
        uint32_t it = 0, ai = 0;
        const int quarter = warp & 3, half = warp >> 2;      // half: this warp's column part (0 .. NH-1)
        const int row0 = quarter * 32 + lane;        // this thread's accumulator row inside a 128-row tile
        const int e = row0 & (tb - 1);               // its edge (the same in every tile: 128 is a multiple of tb)
        const int t8 = tb >> 3;                      // 8-edge octets per batch
        const int GW = KP + a.dsh;                   // row pitch of sGeo
        // bounds of the next receiver, requested one receiver ahead
        int64_t nx0 = 0, nx1 = 0;
        if ((int64_t)blockIdx.x < a.n_nodes) et_bounds(a, blockIdx.x, nullptr, nx0, nx1);
        for (int64_t v = blockIdx.x; v < a.n_nodes; v += gridDim.x) {
            const int64_t seg0 = nx0, seg1 = any_op ? nx1 : nx0;
            if (v + gridDim.x < a.n_nodes) et_bounds(a, v + gridDim.x, nullptr, nx0, nx1);
            {
                for (int64_t b0 = seg0; b0 < seg1; b0 += tb) {
                    const int nb = (int)min((int64_t)tb, seg1 - b0);     // edges of the batch
                    float pphi[KP];
#pragma unroll
                    for (int q = 0; q < KP; ++q) pphi[q] = 0.f;
                    for (int sb = 0; sb < nsub; ++sb, ++it) {
                        const int op = use_x ? sb : 1;           // D (rows of x) or Dv (rows of vx)
                        const int st = (int)(it % NS);
                        mbar_wait(bar_full + 8 * st, (it / NS) & 1, a.status);
                        const float* raw = reinterpret_cast<const float*>(sRing + (size_t)st * stage_bytes + (size_t)2 * a.x_cap);
                        const float* sYT = raw + NRAW * tb * KP;
                        const float* sVYT = sYT + a.dsh * PS;
                        // weights of this sub-batch: gM += sum_q aw[q] * D,  gphi[q] += mw * D
                        //   plain: aw = phi, mw = M;   dual, op 0: aw = vphi, mw = dM;   dual, op 1: aw = phi, mw = M
                        float aw[KP];
#pragma unroll
                        for (int q = 0; q < KP; ++q) aw[q] = (DUAL && op == 0) ? raw[tb * KP + e * KP + q] : raw[e * KP + q];
                        // ---- coupling matrices of the set, once per batch (both sub-batches share them; the previous
                        // batch's readers are all past the barrier that follows its epilogue): thread <-> (entry, 8 edges)
                        if (sb == 0)
                        for (int i = tid; i < S.nent * t8; i += NCW * 32) {
                            const int j = i >> (lg - 3), o8 = 8 * (i - j * t8);
                            const EntS en = sEnt[j];
                            float m[8], dm[8];
#pragma unroll
                            for (int x = 0; x < 8; ++x) { m[x] = 0.f; dm[x] = 0.f; }
                            for (int k = en.nz_begin; k < en.nz_begin + en.nz_count; ++k) {
                                const NzS t = sNz[k];
                                float y[8];
                                *reinterpret_cast<float4*>(y) = *reinterpret_cast<const float4*>(sYT + t.b * PS + o8);
                                *reinterpret_cast<float4*>(y + 4) = *reinterpret_cast<const float4*>(sYT + t.b * PS + o8 + 4);
#pragma unroll
                                for (int x = 0; x < 8; ++x) m[x] = fmaf(t.coef, y[x], m[x]);
                                if (DUAL) {
                                    *reinterpret_cast<float4*>(y) = *reinterpret_cast<const float4*>(sVYT + t.b * PS + o8);
                                    *reinterpret_cast<float4*>(y + 4) = *reinterpret_cast<const float4*>(sVYT + t.b * PS + o8 + 4);
#pragma unroll
                                    for (int x = 0; x < 8; ++x) dm[x] = fmaf(t.coef, y[x], dm[x]);
                                }
                            }
                            *reinterpret_cast<float4*>(sM + j * PS + o8) = *reinterpret_cast<const float4*>(m);
                            *reinterpret_cast<float4*>(sM + j * PS + o8 + 4) = *reinterpret_cast<const float4*>(m + 4);
                            if (DUAL) {
                                *reinterpret_cast<float4*>(sdM + j * PS + o8) = *reinterpret_cast<const float4*>(dm);
                                *reinterpret_cast<float4*>(sdM + j * PS + o8 + 4) = *reinterpret_cast<const float4*>(dm + 4);
                            }
                        }
                        compute_sync<NCW>();     // coupling matrices complete; the previous batch's reductions are done
                        // the raw rows of the stage are consumed by every compute thread (the stage is released when
                        // they are and the batch's MMAs, which read the sender rows, have retired)
                        if (tid == 0) mbar_arrive(bar_free + 8 * st);
                        // ---- epilogue: this thread owns the accumulator rows (s, e) = (row >> lg, row & (tb-1))
                        int ent_u = 0;                // first entry of the unit inside the set
                        for (int ui = 0; ui < S.nunit; ++ui, ++ai) {
                            const UInfo U = sU[ui];
                            const int npad = (int)U.npad, nmt = (int)U.nmt, d_src = (int)U.d_src;
                            const uint32_t buf = ai & 1;
                            mbar_wait(bar_accfull + 8 * buf, (ai >> 1) & 1, a.status);
                            tc_fence_after();
                            const int chalf = ((int)U.ncomp + NH - 1) / NH;
                            const int c_lo = half * chalf, c_hi = min((int)U.ncomp, c_lo + chalf);
                            // 16 accumulator columns per TMEM load: two components at KP = 8, one at KP = 16.  The loads
                            // of a tile whose rows of this warp carry no (s, e) are skipped; the others run one ahead of
                            // the arithmetic (two register sets).
                            constexpr int CPL = 16 / KP;
                            const uint32_t t0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * (uint32_t)a.acc_cols;
                            const int ncl = (c_hi - c_lo + CPL - 1) / CPL;       // loads per tile
                            int nmt_w = 0;                                       // tiles with rows of this warp (a prefix)
                            for (int mt = 0; mt < nmt; ++mt) if (((mt * 128 + quarter * 32) >> lg) < d_src) nmt_w = mt + 1;
                            const int nch = ncl > 0 ? ncl * nmt_w : 0;
                            int mt_i = 0, cl_i = c_lo, mt_p = 0, cl_p = c_lo;      // the next load's and the next use's (tile, component)
                            auto issue = [&](float* v) {
                                const int mt = mt_i, cl = cl_i;
                                cl_i += CPL; if (cl_i >= c_hi) { cl_i = c_lo; ++mt_i; }
                                const uint32_t ad = t0 + (uint32_t)(mt * npad + cl * KP);
                                if (cl + CPL <= c_hi) tc_ld16_nowait(ad, v); else tc_ld8_nowait(ad, v);     // warp-uniform
                            };
                            auto process = [&](const float* v) {
                                const int mt = mt_p, cl = cl_p;
                                cl_p += CPL; if (cl_p >= c_hi) { cl_p = c_lo; ++mt_p; }
                                const int s = (mt * 128 + row0) >> lg;
                                if (s >= d_src) return;       // rows past the block's (s, e) range hold whatever the tile read
#pragma unroll
                                for (int c2 = 0; c2 < CPL; ++c2) {
                                    if (cl + c2 >= c_hi) break;
                                    const int ent = ent_u + (cl + c2) * d_src + s;
                                    const float mw = (DUAL && op == 0) ? sdM[ent * PS + e] : sM[ent * PS + e];
                                    float gp[4] = {0.f, 0.f, 0.f, 0.f};       // four partial sums: short dependent chains
#pragma unroll
                                    for (int x = 0; x < KP; ++x) {
                                        gp[x & 3] = fmaf(aw[x], v[c2 * KP + x], gp[x & 3]);
                                        pphi[x] = fmaf(mw, v[c2 * KP + x], pphi[x]);
                                    }
                                    const float gm = (gp[0] + gp[1]) + (gp[2] + gp[3]);
                                    sGM[ent * PS + e] = (sb == 0 ? 0.f : sGM[ent * PS + e]) + gm;
                                }
                            };
                            float va[16];
                            if constexpr (MINB == 2) {      // two CTAs per SM: half the registers, one load at a time
                                for (int ch = 0; ch < nch; ++ch) { issue(va); tc_wait_ld16(va); process(va); }
                            } else {
                            float vb[16];
                            if (nch > 0) issue(va);
                            for (int ch = 0; ch < nch; ch += 2) {
                                tc_wait_ld16(va);
                                if (ch + 1 < nch) issue(vb);
                                process(va);
                                if (ch + 1 < nch) {
                                    tc_wait_ld16(vb);
                                    if (ch + 2 < nch) issue(va);
                                    process(vb);
                                }
                            }
                            }
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar_accfree + 8 * buf);
                            ent_u += (int)U.ncomp * d_src;
                        }
                    }   // sub-batches
#pragma unroll
                    for (int q = 0; q < KP; ++q) sPphi[tid * KP + q] = pphi[q];
                    compute_sync<NCW>();
                    // ---- fixed-order reductions, written straight to the outputs: every (edge, q) and (edge, b) of the
                    // batch is produced here exactly once per launch (edge id = position in the receiver-sorted order).
                    // The threads that share an edge are those whose row is congruent to it modulo tb, in both column halves.
                    if (a.phi_mode)
                        for (int i = tid; i < tb * KP; i += NCW * 32) {
                            const int ee = i / KP, q = i - ee * KP;
                            if (ee < nb && q < a.K) {
                                float v = 0.f;
                                for (int r = ee; r < 128; r += tb)
#pragma unroll
                                    for (int h = 0; h < NH; ++h) v += sPphi[(128 * h + r) * KP + q];
                                if constexpr (GEO) { sGeo[ee * GW + q] = v; continue; }
                                float* p = a.gphi + (b0 + ee) * a.K + q;
                                // one add per element and launch, launches in stream order: the sum has a fixed order
                                if (a.phi_mode == 2) atomicAdd(p, v); else *p = v;
                            }
                        }
                    // gY: thread <-> (b, edge); the sparse terms of b are the same for the lanes that share it
                    if (a.Y_mode)
                        for (int i = tid; i < a.dsh * tb; i += NCW * 32) {
                            const int b = i >> lg, ee = i & (tb - 1);
                            if (ee < nb) {
                                float g0 = 0.f, g1 = 0.f;                  // two partial sums, fixed order
                                const int k1 = sInvPtr[b + 1];
                                int k = sInvPtr[b];
                                for (; k + 1 < k1; k += 2) {
                                    const NzS t0 = sInv[k], t1 = sInv[k + 1];
                                    g0 = fmaf(t0.coef, sGM[t0.b * PS + ee], g0);
                                    g1 = fmaf(t1.coef, sGM[t1.b * PS + ee], g1);
                                }
                                if (k < k1) { const NzS t0 = sInv[k]; g0 = fmaf(t0.coef, sGM[t0.b * PS + ee], g0); }
                                const float g = g0 + g1;
                                if constexpr (GEO) { sGeo[ee * GW + KP + b] = g; continue; }
                                float* p = a.gY + (b0 + ee) * a.dsh + b;
                                if (a.Y_mode == 2) atomicAdd(p, g); else *p = g;
                            }
                        }
                    // geometry mode: g_r = (sum_q gphi_q dphi_q/dr) u + (I - u u^T) (sum_b gY_b grad F_b) / |r|, one thread per edge
                    if constexpr (GEO) {
                        compute_sync<NCW>();
                        for (int ee = tid; ee < nb; ee += NCW * 32) {
                            const float* rp = a.rvec + (b0 + ee) * 3;
                            const float rx = __ldg(rp), ry = __ldg(rp + 1), rz = __ldg(rp + 2);
                            const float r = sqrtf(rx * rx + ry * ry + rz * rz), ir = 1.f / r;
                            const float ux = rx * ir, uy = ry * ir, uz = rz * ir;
                            const float* ge = sGeo + ee * GW;
                            float gr = 0.f, Gx = 0.f, Gy = 0.f, Gz = 0.f;
                            geo_radial(r, a.K, a.geo_rc, a.geo_basis, a.geo_p, [&](int q, float, float df) { gr = fmaf(ge[q], df, gr); });
                            const int dsh = a.dsh;
                            geo_sh(ux, uy, uz, [&](int b, float, float fx, float fy, float fz) {
                                if (b < dsh) { const float w = ge[KP + b]; Gx = fmaf(w, fx, Gx); Gy = fmaf(w, fy, Gy); Gz = fmaf(w, fz, Gz); }
                            });
                            const float un = ux * Gx + uy * Gy + uz * Gz;
                            const float o0 = gr * ux + (Gx - un * ux) * ir, o1 = gr * uy + (Gy - un * uy) * ir, o2 = gr * uz + (Gz - un * uz) * ir;
                            float* p = a.g_rvec + (b0 + ee) * 3;
                            if (a.phi_mode == 2) { atomicAdd(p, o0); atomicAdd(p + 1, o1); atomicAdd(p + 2, o2); }
                            else { p[0] = o0; p[1] = o1; p[2] = o2; }
                        }
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols) : "memory");
    }
}

// shared bytes of a launch
int smem_need(int KP, bool dual, int dsh, int tb, int x_cap, int z_cap, int nent, int nunit, int ncomp, int nnz, int ninv) {
    constexpr int NCW = 8;
    const int nop = dual ? 2 : 1;
    const int PS = tb;
    const int stage = 2 * x_cap + ((raw_floats(KP, dual, dsh, tb) * 4 + 1023) & ~1023);
    const size_t meta = (size_t)nop * nent * PS + (size_t)nent * PS + (size_t)NCW * 32 * KP + (size_t)tb * (KP + dsh);
    const int tables = nunit * (int)(sizeof(UInfo) + sizeof(TBlk)) + ncomp * (int)sizeof(CompS) + nent * (int)sizeof(EntS) +
                       (nnz + ninv) * (int)sizeof(NzS) + (dsh + 2) * 4;
    return 1024 + NS * stage + 2 * z_cap + (int)(meta * 4) + (2 * NS + 8 + 2 * nunit) * 8 + tables;
}

}  // namespace

// Units and sets of the tensor-core edge pass (receiver direction) for the plain ([0]) and dual ([1]) pass.
// Every set is one launch with its own batch size and shared-memory layout.
void build_tc_edge_sets(const sobek_plan* p, Direction& dir) {
    const int KP = p->K <= 8 ? 8 : 16;
    const int dsh = p->dim_sh;
    for (int dual = 0; dual < 2; ++dual) {
        TcSets& T = dir.etc[dual];
        T = TcSets{};
        if (p->K > 16) continue;
        bool ok = true;
        for (const DPath& P : dir.paths)
            if ((P.c_src & 15) || P.c_src > 128 || (P.src_off & 7)) ok = false;
        if (!ok || (dir.C_src & 7) || dir.paths.empty()) continue;
        struct Blk { int so, c_src, d_src; std::vector<SComp> comps; };
        std::vector<Blk> blocks;
        for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
            const DGroup& G = dir.groups[gi];
            for (int k = G.path_begin; k < G.path_end; ++k) {
                const DPath& P = dir.paths[k];
                auto it = std::find_if(blocks.begin(), blocks.end(), [&](const Blk& b) { return b.so == P.src_off; });
                if (it == blocks.end()) { blocks.push_back(Blk{P.src_off, P.c_src, P.d_src, {}}); it = blocks.end() - 1; }
                for (int o = 0; o < G.d_dst; ++o)
                    it->comps.push_back(SComp{P.tabM + o, G.d_dst, P.sh_off, (int)gi, o, P.koff, G.d_dst, 0});
            }
        }
        std::sort(blocks.begin(), blocks.end(), [](const Blk& x, const Blk& y) { return x.so < y.so; });
        struct Cand { int blk, c0, nc; };
        // accumulator tiles of up to 16 components (128 columns at K <= 8, 256 above); if the wide tiles of a
        // K > 8 profile do not fit shared memory, tiles of 8 components
        for (int comps_per_tile = 16; comps_per_tile >= 128 / KP && !T.ok; comps_per_tile >>= 1) {
        std::vector<Cand> cands;
        for (size_t b = 0; b < blocks.size(); ++b) {
            const int nc = (int)blocks[b].comps.size();
            const int ntile = (nc + comps_per_tile - 1) / comps_per_tile;
            const int per = (nc + ntile - 1) / ntile;
            for (int c0 = 0; c0 < nc; c0 += per) cands.push_back(Cand{(int)b, c0, std::min(per, nc - c0)});
        }
        auto nkb = [&](int b) { return (blocks[b].c_src + 63) / 64; };
        auto npad = [&](const Cand& c) { return (c.nc * KP + 15) & ~15; };
        auto unit_z = [&](const Cand& c) { return npad(c) * 128 * nkb(c.blk); };
        auto cand_nz = [&](const Cand& c) {
            int n = 0;
            for (int cl = 0; cl < c.nc; ++cl) {
                const SComp& cp = blocks[c.blk].comps[c.c0 + cl];
                for (int sdx = 0; sdx < blocks[c.blk].d_src; ++sdx) {
                    const int t = cp.tab0 + sdx * cp.tstride;
                    n += p->tab_ptr[t + 1] - p->tab_ptr[t];
                }
            }
            return n;
        };
        // batch size of a set: the largest power of two in 16..128 whose rows d_src * tb fit one 128-row tile
        auto batch_of = [&](int d_src_max) { int tb = 16; while (tb < 128 && d_src_max * tb * 2 <= 128) tb *= 2; return tb; };
        struct Par { int tb, x, z, nent, nnz, ncomp, cols, need; };
        // the launch parameters of the set of candidates [i, j): the largest batch size (at most the one that
        // fills a 128-row tile) whose shared memory stays within the budget
        auto eval = [&](size_t i, size_t j, int budget) {
            int dmax = 0;
            std::vector<int> blks;
            for (size_t k = i; k < j; ++k) {
                dmax = std::max(dmax, blocks[cands[k].blk].d_src);
                if (std::find(blks.begin(), blks.end(), cands[k].blk) == blks.end()) blks.push_back(cands[k].blk);
            }
            Par r{};
            for (int tb = batch_of(dmax); tb >= 16; tb >>= 1) {
                r = Par{};
                r.tb = tb;
                for (int b : blks) r.x += blocks[b].d_src * r.tb * 128 * nkb(b);
                for (size_t k = i; k < j; ++k) {
                    const Cand& c = cands[k];
                    r.z += unit_z(c); r.nent += c.nc * blocks[c.blk].d_src; r.nnz += cand_nz(c); r.ncomp += c.nc;
                    r.cols = std::max(r.cols, ((blocks[c.blk].d_src * r.tb + 127) / 128) * npad(c));
                }
                // a 128-row MMA tile may read past the rows of a block: what follows in shared memory (the other
                // copy, the next stage, the Zbar slabs) is at least 16 KiB, hence the floor on the slab size
                r.x = (r.x + 1023) & ~1023;
                r.z = std::max(8192, (r.z + 1023) & ~1023);
                r.need = smem_need(KP, dual, dsh, r.tb, r.x, r.z, r.nent, (int)(j - i), r.ncomp, r.nnz, r.nnz);
                if (r.need <= budget) break;
            }
            return r;
        };
        // sets of at most `maxu` units each: the largest grouping that fits the budget of two CTAs per SM
        // (attempt 0) or of one CTA per SM (attempt 1)
        auto pack = [&](int attempt) {
          TcSets T;
          for (int maxu = (int)cands.size(); maxu >= 1 && !T.ok; --maxu) {
            const int budget = (attempt == 0 ? 113 : 226) * 1024;
            const int col_budget = attempt == 0 ? 128 : 256;
            T = TcSets{};
            bool fits = true;
            size_t i = 0;
            while (i < cands.size() && fits) {
                size_t j = i;
                while (j < cands.size() && (int)(j - i) < maxu) {
                    const Par r = eval(i, j + 1, budget);
                    if (r.need > budget || r.cols > col_budget) break;
                    ++j;
                }
                if (j == i) { fits = false; break; }
                const Par r = eval(i, j, budget);
                TSet S{};
                S.unit_begin = (int)T.units.size(); S.blk_begin = (int)T.blks.size(); S.ent_begin = (int)T.ents.size();
                int z_off = 0, x_off = 0;
                std::vector<int> local_blk;
                for (size_t k = i; k < j; ++k) {
                    const Cand& c = cands[k];
                    const Blk& Bk = blocks[c.blk];
                    int bi = -1;
                    for (size_t m = 0; m < local_blk.size(); ++m) if (local_blk[m] == c.blk) bi = S.blk_begin + (int)m;
                    if (bi < 0) {
                        TBlk tb{};
                        tb.src_off = Bk.so; tb.c_src = Bk.c_src; tb.d_src = Bk.d_src; tb.ncols = 0;
                        tb.b_off = x_off; tb.slab_bytes = r.tb * 128; tb.atom_stride = Bk.d_src * r.tb * 128;
                        x_off += Bk.d_src * r.tb * 128 * nkb(c.blk);
                        bi = (int)T.blks.size();
                        T.blks.push_back(tb);
                        local_blk.push_back(c.blk);
                    }
                    TUnit U{};
                    U.blk = bi; U.comp_begin = (int)T.comps.size(); U.ncomp = c.nc; U.a_off = z_off;
                    U.slab_stride = npad(c) * 128; U.tmem_col = 0; U.pad[0] = npad(c);
                    for (int cl = 0; cl < c.nc; ++cl) {
                        const SComp& cp = Bk.comps[c.c0 + cl];
                        T.comps.push_back(cp);
                        for (int s = 0; s < Bk.d_src; ++s) T.ents.push_back(TEnt{cp.tab0 + s * cp.tstride, cp.sh_off, 0, 0});
                    }
                    z_off += unit_z(c);
                    T.units.push_back(U);
                }
                S.nunit = (int)T.units.size() - S.unit_begin; S.nblk = (int)T.blks.size() - S.blk_begin;
                S.nent = (int)T.ents.size() - S.ent_begin;
                T.sets.push_back(S);
                int lg = 0; while ((1 << lg) < r.tb) ++lg;
                int tc = 32; while (tc < 2 * r.cols) tc <<= 1;
                TcSets::ESetPar ep{};
                ep.tb = r.tb; ep.lg = lg; ep.x_cap = r.x; ep.z_cap = r.z; ep.smem = r.need; ep.tmem_cols = tc; ep.acc_cols = r.cols;
                ep.ctas = (r.need <= 113 * 1024 && tc <= 256) ? 2 : 1;
                ep.nnz = r.nnz; ep.ninv = r.nnz; ep.ncomp = r.ncomp;
                T.epar.push_back(ep);
                if (r.need > 227 * 1024 || tc > 512) fits = false;
                i = j;
            }
            if (!fits) continue;
            // shared-memory images of the tables, per set: entries with their sparse terms, the inverse table
            // b -> (entry inside the set, coef), and the components with their group layout resolved
            for (TSet& S : T.sets) {
                S.b_items = (int)T.nz.size();
                for (int j = 0; j < S.nent; ++j) {
                    const TEnt& E = T.ents[S.ent_begin + j];
                    EntS es{0, (int)T.nz.size() - S.b_items, p->tab_ptr[E.tab + 1] - p->tab_ptr[E.tab], 0};
                    for (int k = p->tab_ptr[E.tab]; k < p->tab_ptr[E.tab + 1]; ++k) T.nz.push_back(NzS{E.sh_off + p->tab_idx[k], p->tab_coef[k]});
                    T.ents_s.push_back(es);
                }
                S.pad = (int)T.nz.size() - S.b_items;
                T.inv_base.push_back((int)T.inv.size());
                const int base = (int)T.inv.size();
                for (int b = 0; b < dsh; ++b) {
                    T.inv_ptr.push_back((int)T.inv.size() - base);
                    for (int en = 0; en < S.nent; ++en) {
                        const TEnt& E = T.ents[S.ent_begin + en];
                        for (int k = p->tab_ptr[E.tab]; k < p->tab_ptr[E.tab + 1]; ++k)
                            if (E.sh_off + p->tab_idx[k] == b) T.inv.push_back(NzS{en, p->tab_coef[k]});
                    }
                }
                T.inv_ptr.push_back((int)T.inv.size() - base);
            }
            for (const SComp& cp : T.comps)
                T.comps_s.push_back(CompS{dir.zb_off[cp.group], dir.nk_ld[cp.group], cp.d_dst, cp.o, cp.koff, {0, 0}});
            T.ok = true;
          }
          return T;
        };
        // two CTAs per SM hide the latency of the short batches better, unless that takes many more sets (each set
        // is a launch of its own that stages the edge data again)
        TcSets T0 = pack(0), T1 = pack(1);
        T = (T0.ok && (!T1.ok || T0.sets.size() <= T1.sets.size() + 2)) ? T0 : T1;
        }   // tile widths
    }
}

cudaError_t launch_edge_pass_tc(const sobek_plan* p, const Direction& dir, const EdgeView& ev, int64_t node0,
                                int64_t n_nodes, const SplitSrc& ss, const float* Y, const float* vY, const float* phi,
                                const float* vphi, int dual, const void* zqh, const void* zql, float* gphi, float* gY,
                                int phi_mode, int Y_mode, int* status, cudaStream_t s) {
    const TcSets& T = dir.etc[dual ? 1 : 0];
    if (!T.ok || !ss.h || !ss.l) return cudaErrorInvalidValue;
    if (n_nodes <= 0) return cudaSuccess;
    EtArgs a{};
    a.sets = T.d_sets; a.units = T.d_units; a.blks = T.d_blks; a.comps = T.d_comps_s;
    a.row_ptr = ev.ptr; a.col = ev.col; a.node0 = node0; a.n_nodes = n_nodes; a.N = ev.N; a.E = ev.E;
    a.sh = (const __nv_bfloat16*)ss.h; a.sl = (const __nv_bfloat16*)ss.l;
    a.vsh = (const __nv_bfloat16*)ss.vh; a.vsl = (const __nv_bfloat16*)ss.vl;
    a.Y = Y; a.vY = vY; a.phi = phi; a.vphi = vphi;
    a.zqh = (const __nv_bfloat16*)zqh; a.zql = (const __nv_bfloat16*)zql;
    a.gphi = gphi; a.gY = gY;
    a.rvec = ss.rvec; a.g_rvec = ss.g_rvec; a.geo_rc = ss.geo_rc; a.geo_basis = ss.geo_basis; a.geo_p = ss.geo_p;
    a.oseg = ss.oseg ? ss.oseg + node0 : nullptr;
    a.K = p->K; a.dsh = p->dim_sh; a.C_src = dir.C_src;
    a.status = status;
    const bool k8 = p->K <= 8;
    if (ss.rvec && dual) return cudaErrorNotSupported;
    void (*kern2)(const EtArgs) = k8 ? (dual ? k_edge_tc<8, true, 8, 3, false, 2> : k_edge_tc<8, false, 8, 3, false, 2>)
                                     : (dual ? k_edge_tc<16, true, 8, 3, false, 2> : k_edge_tc<16, false, 8, 3, false, 2>);
    void (*kern1)(const EtArgs) = k8 ? (dual ? k_edge_tc<8, true, 8, 3, false, 1> : k_edge_tc<8, false, 8, 3, false, 1>)
                                     : (dual ? k_edge_tc<16, true, 8, 3, false, 1> : k_edge_tc<16, false, 8, 3, false, 1>);
    if (ss.rvec) {
        kern2 = k8 ? k_edge_tc<8, false, 8, 3, true, 2> : k_edge_tc<16, false, 8, 3, true, 2>;
        kern1 = k8 ? k_edge_tc<8, false, 8, 3, true, 1> : k_edge_tc<16, false, 8, 3, true, 1>;
    }
    int max_smem = 0;
    for (const auto& ep : T.epar) max_smem = std::max(max_smem, ep.smem);
    cudaError_t e = cudaFuncSetAttribute(kern2, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(kern1, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e != cudaSuccess) return e;
    // one launch per set of accumulator tiles: the first writes in the caller's mode, the others accumulate
    for (size_t si = 0; si < T.sets.size(); ++si) {
        const TSet& S = T.sets[si];
        const TcSets::ESetPar& ep = T.epar[si];
        a.set = (int)si;
        a.tb = ep.tb; a.lg = ep.lg; a.x_cap = ep.x_cap; a.z_cap = ep.z_cap; a.nent = S.nent;
        a.tmem_cols = ep.tmem_cols; a.acc_cols = ep.acc_cols; a.nnz = ep.nnz; a.ninv = ep.ninv; a.nunit = S.nunit; a.ncomp = ep.ncomp;
        a.ents = T.d_ents_s + S.ent_begin; a.nz = T.d_nz + S.b_items;
        a.inv_ptr = T.d_inv_ptr + si * (size_t)(p->dim_sh + 1); a.inv = T.d_inv + T.inv_base[si];
        a.phi_mode = phi_mode ? (si == 0 ? phi_mode : 2) : 0;
        a.Y_mode = Y_mode ? (si == 0 ? Y_mode : 2) : 0;
        const int grid = (int)std::min<int64_t>(n_nodes, (int64_t)148 * ep.ctas);
        KernelTimer kt(K_EDGE, s);
        if (ep.ctas == 2) kern2<<<grid, (8 + 3 + 1) * 32, ep.smem, s>>>(a);
        else kern1<<<grid, (8 + 3 + 1) * 32, ep.smem, s>>>(a);
        count_launch();
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace sobek
