// Edge stream on the tensor cores (sm_100a, tcgen05 / TMEM), warp-specialised.
//
// For one receiver i and one source irrep block the fold of its edges into the bounded state
// (Eqs. angular_path_contraction, receiver_state)
//     Z_i[(comp,q), u] = sum_e phi_e[q] * sum_s M_e[s,comp] * x_{src(e)}[s,u]
// is a dense contraction over k = (s, e) of
//     A[(comp,q), k] = phi_e[q] * M_e[s,comp]      (built per edge on the FP32 pipes; independent of u)
//     B[k, u]        = x_{src(e)}[s,u]             (the gathered sender rows, as they lie in memory)
// so the work that scales with the multiplicity runs on tcgen05.mma.  fp32 parity comes from the
// split-bf16 product a*b ~= a_hi*b_hi + a_lo*b_hi + a_hi*b_lo (fp32 accumulation in TMEM); the sender
// rows are read from bf16 (hi, lo) copies of the source features made once per call.
//
// A CTA works through (set of accumulator tiles, receiver) items in set-major order, edges in batches of 16,
// with three roles:
//   loader warps  run ahead (segment bounds and edge / sender ids are requested one step early): cp.async of
//                 the batch's phi rows, of its Y rows (written transposed) and of the sender rows straight
//                 into the B slabs (16 edges x c_src, MN-major, 128-byte swizzle) of a two-stage ring; the
//                 copies signal the stage's mbarrier themselves when they land;
//   compute warps expand the coupling matrices M_e[s,comp] of the set from the sparse CG table (kept in shared
//                 memory, like every other table the kernel looks up), build the A slabs (one per s: 128 rows
//                 x 16 edges, K-major, no swizzle, bf16 hi / lo), and - one item behind - drain the finished
//                 accumulator (tcgen05.ld), split it into bf16 hi / lo and write the rows of the node GEMM's
//                 A operand (contraction index k = koff + q*c_src + u, so a row of 16-byte pieces per thread);
//   MMA warp      one thread issues the batch's MMAs into one of two TMEM accumulator buffers and commits
//                 to the mbarriers that release the A region, the ring stage and the accumulator.
// With DUAL the kernel produces the directional state of the double backward
//     dZ = sum_e ( vphi (x) C(x,Y) + phi (x) [ C(vx,Y) + C(x,vY) ] )       (Eq. receiver_double_adjoint)
// as  [vphi*M + phi*dM] x B(x)  +  [phi*M] x B(vx).
// The same kernel runs the sender-owned transposed traversal.  Every mbarrier wait is bounded.
#include <cuda_bf16.h>

#include <algorithm>

#include "guard.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace sobek {
namespace {

using namespace ptx;

constexpr int TB = 16;          // edges per batch = k extent of one MMA
constexpr int NCW = 8;          // compute warps
constexpr int NLW = 2;          // loader warps
constexpr int TT = (NCW + NLW + 1) * 32;   // threads per CTA
constexpr int NS = 2;           // ring stages
constexpr int PS = 20;          // row pitch (floats) of the transposed stages: 16 values + 4 (bank spread)

struct TcArgs {
    const TSet* sets;
    const TUnit* units;
    const TBlk* blks;
    const EntS* ents;      // per set (TSet::ent_begin)
    const NzS* nz;         // per set (TSet::b_items = first term, TSet::pad = number of terms)
    const CompS* comps;
    EdgeView ev;
    int64_t node0, n_nodes;
    const __nv_bfloat16* sh;    // bf16 hi / lo copies of the source features [N][C_src]
    const __nv_bfloat16* sl;
    const __nv_bfloat16* vsh;   // DUAL: the same for the source direction; NULL without it
    const __nv_bfloat16* vsl;
    const float* Y;
    const float* vY;
    const float* phi;
    const float* vphi;
    __nv_bfloat16* zh;
    __nv_bfloat16* zl;
    int32_t K, dsh, C_src, nsets;
    int32_t a_cap, b_cap, max_ent, tmem_cols, acc_cols, n_units, n_blks, n_comps, max_nz;
    int32_t concat;        // 1: multiplicities <= 32, the lo copy of a gathered row sits 32 columns beside the hi copy
    int* status;
};

__device__ __forceinline__ int64_t owner_of(const int64_t* __restrict__ row_ptr, int64_t N, int64_t e) {
    int64_t lo = 0, hi = N;   // row_ptr[lo] <= e < row_ptr[hi]
    while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (__ldg(row_ptr + mid) <= e) lo = mid; else hi = mid;
    }
    return lo;
}

// Everything the roles look up per item, batch or row lives in shared memory: with most of the SM's
// L1 given to the operand regions, table reads from global memory would mostly go to L2.
struct UInfo {     // a unit, as the MMA thread and the drain need it
    uint32_t idesc, tmem_col, a_off, slab_stride, b_off, slab_bytes, d_src, comp_begin, ncomp, c_src, ncols, pad;
    // operand descriptors of slab 0 (hi copies; stage 0 of the ring for B): the other slabs, copies and stages differ
    // only in the 16-byte-granular address field, so the MMA thread reaches them with one addition each
    uint64_t dA0, dB0;
    uint32_t idesc_wide, pad2;   // concat: the same instruction with N = 64 columns ([B_hi | B_lo])
};
// shared-memory operand descriptor without swizzle (K-major core matrices of 8 rows x 16 bytes)
__device__ __forceinline__ uint64_t make_desc_none(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;   // version
    return d;
}

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void compute_sync() { asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory"); }

// cp.async with zero fill: copies `bytes` (0 or the full size) and fills the rest with zeros
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async4_zfill(uint32_t dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void tc_ld8(uint32_t taddr, float* v) {
    uint32_t r[8];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

// (hi, lo) bf16 split of two floats: hi pair, lo pair (element 0 in the low half)
__device__ __forceinline__ void split2(float a, float b, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    hi = *reinterpret_cast<const uint32_t*>(&h);
    const float ra = a - __uint_as_float(hi << 16);
    const float rb = b - __uint_as_float(hi & 0xffff0000u);
    const __nv_bfloat162 l = __floats2bfloat162_rn(ra, rb);
    lo = *reinterpret_cast<const uint32_t*>(&l);
}
__device__ __forceinline__ void split8(const float* p, uint4& h, uint4& l) {
    split2(p[0], p[1], h.x, l.x);
    split2(p[2], p[3], h.y, l.y);
    split2(p[4], p[5], h.z, l.z);
    split2(p[6], p[7], h.w, l.w);
}

// per-stage raw area (floats): phi rows [TB][KP], (vphi), and Y written transposed [dsh][PS], (vY)
__host__ __device__ inline int raw_floats(int KP, bool dual, int dsh) {
    const int n = dual ? 2 : 1;
    return n * TB * KP + n * dsh * PS;
}

template <int KP, bool DUAL>
__global__ void __launch_bounds__(TT, 2) k_stream_tc(const TcArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    constexpr int NOP = 1;                 // operand pairs held at once (the dual stream runs its two pairs in turn)
    constexpr int NRAW = DUAL ? 2 : 1;     // raw / transposed stages: phi and Y, plus their directions
    const int YS = a.dsh + 1;
    // A region (single buffer): A1h A1l (A2h A2l)
    uint8_t* sA = smem;
    // ring stages: B1h B1l (B2h B2l), then the raw phi / Y rows
    const uint32_t stage_bytes = (uint32_t)(2 * NOP * a.b_cap + ((raw_floats(KP, DUAL, a.dsh) * 4 + 1023) & ~1023));
    uint8_t* sRing = sA + (size_t)2 * NOP * a.a_cap;
    uint8_t* meta = sRing + (size_t)NS * stage_bytes;
    float* sM0 = reinterpret_cast<float*>(meta);             // [2][max_ent][PS]: coupling matrices, double buffered
    float* sdM0 = sM0 + (size_t)2 * a.max_ent * PS;          // DUAL
    float* sPhiT0 = sdM0 + (DUAL ? (size_t)2 * a.max_ent * PS : 0);   // [2][NRAW][KP][PS]
    uint64_t* bars = reinterpret_cast<uint64_t*>(sPhiT0 + 2 * NRAW * KP * PS);
    // bars: full[NS], freeS[NS], ready, afree, acc_full[2], acc_free[2]
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 2 * NS + 6);
    UInfo* sU = reinterpret_cast<UInfo*>(bars + 2 * NS + 8);           // [n_units]
    TSet* sSet = reinterpret_cast<TSet*>(sU + a.n_units);               // [nsets]
    TBlk* sBlk = reinterpret_cast<TBlk*>(sSet + a.nsets);               // [n_blks]
    CompS* sComp = reinterpret_cast<CompS*>(sBlk + a.n_blks);           // [n_comps]
    EntS* sEnt = reinterpret_cast<EntS*>(sComp + a.n_comps);            // [max_ent]  (current set)
    NzS* sNz = reinterpret_cast<NzS*>(sEnt + a.max_ent);                // [max_nz]   (current set)
    const uint32_t bar0 = smem_u32(bars);
    const uint32_t bar_full = bar0, bar_free = bar0 + 8 * NS, bar_ready = bar0 + 16 * NS, bar_afree = bar_ready + 8,
                   bar_accfull = bar_ready + 16, bar_accfree = bar_ready + 32;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool has_vx = DUAL && a.vsh != nullptr, has_vY = DUAL && a.vY != nullptr, has_vphi = DUAL && a.vphi != nullptr;
    const bool has_a1 = !DUAL || has_vY || has_vphi;   // operand 1: [phi*M] (plain) or [vphi*M + phi*dM] (dual), times x
    const bool has_a2 = has_vx;                        // operand 2 (dual): [phi*M] times vx
    const bool any_op = has_a1 || has_a2;
    // sub-batches per batch of edges: one per operand pair that is present (op = 0: x rows, op = 1: vx rows)
    const int nsub = (has_a1 ? 1 : 0) + (has_a2 ? 1 : 0);

    if (tid == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(bar_full + 8 * s, NLW * 32); mbar_init(bar_free + 8 * s, 1); }
        mbar_init(bar_ready, NCW * 32);
        mbar_init(bar_afree, 1);
        for (int t = 0; t < 2; ++t) { mbar_init(bar_accfull + 8 * t, 1); mbar_init(bar_accfree + 8 * t, NCW * 32); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // the raw rows of padded radial components (q >= K) and of absent directions stay zero for ever
    {
        const int words = (int)(stage_bytes / 4), b_words = 2 * NOP * a.b_cap / 4;
        for (int i = tid; i < NS * words; i += TT) {
            const int st = i / words, w = i - st * words;
            if (w >= b_words) reinterpret_cast<uint32_t*>(sRing + (size_t)st * stage_bytes)[w] = 0u;
        }
    }
    for (int i = tid; i < a.n_units; i += TT) {
        const TUnit U = a.units[i];
        const TBlk B = a.blks[U.blk];
        UInfo u;
        // D = F32, A = B = BF16, A K-major, B MN-major, M = 128, N = ncols
        u.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(B.ncols >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        u.tmem_col = (uint32_t)U.tmem_col; u.a_off = (uint32_t)U.a_off; u.slab_stride = (uint32_t)U.slab_stride;
        u.b_off = (uint32_t)B.b_off; u.slab_bytes = (uint32_t)B.slab_bytes; u.d_src = (uint32_t)B.d_src;
        u.comp_begin = (uint32_t)U.comp_begin; u.ncomp = (uint32_t)U.ncomp; u.c_src = (uint32_t)B.c_src;
        u.ncols = (uint32_t)B.ncols; u.pad = 0;
        u.idesc_wide = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(64 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        u.pad2 = 0;
        u.dA0 = make_desc_none(smem_u32(sA) + u.a_off, 128, 256);
        u.dB0 = make_desc(smem_u32(sRing) + u.b_off, 2048, 1024);
        sU[i] = u;
    }
    for (int i = tid; i < a.nsets; i += TT) sSet[i] = a.sets[i];
    for (int i = tid; i < a.n_blks; i += TT) sBlk[i] = a.blks[i];
    for (int i = tid; i < a.n_comps; i += TT) sComp[i] = a.comps[i];
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"((uint32_t)a.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    const int64_t total = a.n_nodes * a.nsets;
    // (local node, set) of an item, advanced without divisions: items are set-major, a CTA takes every gridDim.x-th
    struct ItemPos {
        int64_t nl; int set;
        __device__ void init(int64_t item, int64_t n) { nl = item % n; set = (int)(item / n); }
        __device__ void step(int64_t by, int64_t n) { nl += by; while (nl >= n) { nl -= n; ++set; } }
    };

    if (warp >= NCW && warp < NCW + NLW) {
        // =========================== loader warps ===========================
        // The segment bounds of the next item and the ids of the next batch are requested one step ahead,
        // so that their latency overlaps the issue of the current batch's copies; the copies themselves
        // signal the stage's mbarrier when they land (no wait in this warp).
        const int lt = (warp - NCW) * 32 + lane;   // thread index among the loaders
        int64_t p_item = blockIdx.x, p_seg0 = 0, p_seg1 = 0;     // prefetched item
        ItemPos lp; lp.init(p_item, a.n_nodes);
        auto prefetch_item = [&]() {
            if (p_item < total) {
                seg_bounds(a.ev.ptr, a.node0 + lp.nl, a.ev.E, a.status, p_seg0, p_seg1);
                if (!any_op) p_seg1 = p_seg0;
            }
        };
        prefetch_item();
        struct Cur { int set; int64_t b0, seg1; int sub; };
        auto next_batch = [&](Cur& c, bool first) -> bool {
            if (!first) {
                if (c.sub + 1 < nsub) { ++c.sub; return true; }
                c.sub = 0; c.b0 += TB;
            }
            while (first || c.b0 >= c.seg1) {
                first = false;
                if (p_item >= total) return false;
                c.set = lp.set; c.b0 = p_seg0; c.seg1 = p_seg1; c.sub = 0;
                p_item += gridDim.x; lp.step(gridDim.x, a.n_nodes);
                prefetch_item();
            }
            return true;
        };
        // lane e < 16 holds edge e of the batch; bit e of msk says that the edge exists and that its ids are in
        // range (an id that is not turns the edge's copies into zero fills and is reported in the status word)
        auto load_ids = [&](const Cur& c, int64_t& eid, int32_t& sn, uint32_t& msk) {
            eid = 0; sn = 0;
            bool ok = false;
            if (c.b0 + lane < c.seg1 && lane < TB) {
                const int64_t pos = c.b0 + lane;
                eid = a.ev.perm ? (int64_t)a.ev.perm[pos] : pos;
                ok = id_ok(eid, a.ev.E, a.status);
                if (ok) {
                    const int64_t v = a.ev.transposed ? (a.ev.recv ? (int64_t)a.ev.recv[pos] : owner_of(a.ev.row_ptr, a.ev.N, eid))
                                                      : (int64_t)a.ev.col[eid];
                    ok = id_ok(v, a.ev.N, a.status);
                    sn = ok ? (int32_t)v : 0;
                } else {
                    eid = 0;
                }
            }
            msk = __ballot_sync(0xffffffffu, ok);
        };
        Cur cur{0, 0, 0, 0};
        bool have = next_batch(cur, true);
        int64_t eid = 0; int32_t sn = 0; uint32_t msk = 0;
        if (have) load_ids(cur, eid, sn, msk);
        for (uint32_t it = 0; have; ++it) {
            Cur nxt = cur;
            const bool have_n = next_batch(nxt, false);
            int64_t eid_n = 0; int32_t sn_n = 0; uint32_t msk_n = 0;
            if (have_n) load_ids(nxt, eid_n, sn_n, msk_n);
            const TSet S = sSet[cur.set];
            const int op = has_a1 ? cur.sub : 1;
            const int st = (int)(it % NS);
            if (it >= NS) mbar_wait(bar_free + 8 * st, ((it / NS) & 1) ^ 1, a.status);
            const uint32_t stage_u = smem_u32(sRing + (size_t)st * stage_bytes);
            const uint32_t raw_u = stage_u + (uint32_t)(2 * NOP * a.b_cap);
            // phi (and vphi) rows: raw[e][KP]   (all lanes run every iteration: the loops hold shuffles)
            {
                const bool v16 = (a.K & 3) == 0;
                const int per = v16 ? a.K / 4 : a.K;         // pieces per edge
                const int n_it = TB * per;
                for (int i0 = 0; i0 < n_it; i0 += NLW * 32) {
                    const int i = i0 + lt;
                    const int e = min(i / per, TB - 1), j = i - (i / per) * per;
                    const int64_t ee = __shfl_sync(0xffffffffu, eid, e);
                    if (i < n_it) {
                        const uint32_t ok = (msk >> e) & 1u;
                        if (v16) {
                            cp_async16_zfill(raw_u + (uint32_t)(e * KP + 4 * j) * 4, a.phi + ee * a.K + 4 * j, ok * 16);
                            if (has_vphi) cp_async16_zfill(raw_u + (uint32_t)(TB * KP + e * KP + 4 * j) * 4, a.vphi + ee * a.K + 4 * j, ok * 16);
                        } else {
                            cp_async4_zfill(raw_u + (uint32_t)(e * KP + j) * 4, a.phi + ee * a.K + j, ok * 4);
                            if (has_vphi) cp_async4_zfill(raw_u + (uint32_t)(TB * KP + e * KP + j) * 4, a.vphi + ee * a.K + j, ok * 4);
                        }
                    }
                }
            }
            // Y (and vY), transposed: raw[b][PS + e].  Thread <-> (edge e = lane mod 16, b = lt / 16, + 4, ...)
            const int le = lane & (TB - 1);
            const int64_t ee_own = __shfl_sync(0xffffffffu, eid, le);
            {
                const uint32_t y_u = raw_u + (uint32_t)(NRAW * TB * KP) * 4;
                const uint32_t ok = ((msk >> le) & 1u) * 4u;
                const float* yr = a.Y + ee_own * a.dsh;
                const float* vyr = has_vY ? a.vY + ee_own * a.dsh : nullptr;
                for (int b = lt >> 4; b < a.dsh; b += NLW * 32 / TB) {
                    cp_async4_zfill(y_u + (uint32_t)(b * PS + le) * 4, yr + b, ok);
                    if (has_vY) cp_async4_zfill(y_u + (uint32_t)(a.dsh * PS + b * PS + le) * 4, vyr + b, ok);
                }
            }
            // sender rows -> B slabs (hi and lo), 16 bytes = 8 multiplicities per copy
            {
                // lanes 2e, 2e+1 of each loader warp serve edge e; a thread walks pieces j0, j0 + 4, ... of the row
                const int re = (lane >> 1) & (TB - 1);
                const int32_t sne = __shfl_sync(0xffffffffu, sn, re);
                const uint32_t ok = ((msk >> re) & 1u) * 16u;
                const int j0 = (lane & 1) | ((lt >> 5) << 1);
                const int64_t grow = (int64_t)sne * a.C_src;
                const __nv_bfloat16* srch = (op == 0 ? a.sh : a.vsh) + grow;
                const __nv_bfloat16* srcl = (op == 0 ? a.sl : a.vsl) + grow;
                for (int bi = 0; bi < S.nblk; ++bi) {
                    const TBlk B = sBlk[S.blk_begin + bi];
                    const int cpr = B.c_src >> 3;                  // 16-byte pieces per row
                    for (int j = j0; j < cpr; j += 2 * NLW) {
                        const int u = 8 * j;
                        uint32_t d = stage_u + (uint32_t)(B.b_off + (u >> 6) * B.atom_stride + re * 128 + ((((u & 63) >> 3) ^ (re & 7)) << 4));
                        const __nv_bfloat16* ph = srch + B.src_off + u;
                        const __nv_bfloat16* pl = srcl + B.src_off + u;
                        // the lo copy: a slab of its own, or (concat) columns 32.. of the same swizzled row
                        uint32_t dl = a.concat ? stage_u + (uint32_t)(B.b_off + re * 128 + ((((u >> 3) + 4) ^ (re & 7)) << 4))
                                               : d + (uint32_t)a.b_cap;
                        for (int sdx = 0; sdx < B.d_src; ++sdx) {
                            cp_async16_zfill(d, ph, ok);
                            cp_async16_zfill(dl, pl, ok);
                            d += (uint32_t)B.slab_bytes; dl += (uint32_t)B.slab_bytes; ph += B.c_src; pl += B.c_src;
                        }
                    }
                }
            }
            // this thread's arrival on the stage's barrier fires when all its copies above have landed
            asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar_full + 8 * st) : "memory");
            cur = nxt; have = have_n; eid = eid_n; sn = sn_n; msk = msk_n;
        }
    } else if (warp == NCW + NLW) {
        // =========================== MMA warp ===========================
        if (lane == 0) {
            uint32_t it = 0, mi = 0;
            int64_t nx0 = 0, nx1 = 0;
            ItemPos mp; mp.init(blockIdx.x, a.n_nodes);      // position of the item whose bounds are in flight
            if ((int64_t)blockIdx.x < total) seg_bounds(a.ev.ptr, a.node0 + mp.nl, a.ev.E, nullptr, nx0, nx1);
            const uint64_t acap16 = (uint64_t)(a.a_cap >> 4), bcap16 = (uint64_t)(a.b_cap >> 4);
            for (int64_t item = blockIdx.x; item < total; item += gridDim.x) {
                const TSet S = sSet[mp.set];
                const int64_t seg0 = nx0, seg1 = any_op ? nx1 : nx0;
                mp.step(gridDim.x, a.n_nodes);
                if (item + gridDim.x < total)       // the next item's bounds, requested one item ahead
                    seg_bounds(a.ev.ptr, a.node0 + mp.nl, a.ev.E, nullptr, nx0, nx1);
                if (seg1 <= seg0) continue;
                const uint32_t buf = mi & 1;
                if (mi >= 2) mbar_wait(bar_accfree + 8 * buf, ((mi >> 1) & 1) ^ 1, a.status);
                tc_fence_after();
                for (int64_t b0 = seg0; b0 < seg1; b0 += TB) {
                    for (int sb = 0; sb < nsub; ++sb, ++it) {
                        const int st = (int)(it % NS);
                        mbar_wait(bar_ready, it & 1, a.status);
                        tc_fence_after();
                        const uint64_t st16 = (uint64_t)((uint32_t)st * (stage_bytes >> 4));
                        const uint32_t acc0 = (b0 == seg0 && sb == 0) ? 0u : 1u;
                        for (int ui = 0; ui < S.nunit; ++ui) {
                            const UInfo& U = sU[S.unit_begin + ui];
                            const uint32_t d_tmem = tmem_base + buf * (uint32_t)a.acc_cols + U.tmem_col;
                            const uint32_t idesc = U.idesc, nslab = U.d_src;
                            const uint64_t sa16 = U.slab_stride >> 4, sb16 = U.slab_bytes >> 4;
                            uint64_t dAh = U.dA0, dBh = U.dB0 + st16;
                            if (a.concat) {
                                // two instructions per slab instead of three: A_hi x [B_hi | B_lo] (64 columns; the second
                                // 32 are summed into the first at the drain) and A_lo x B_hi.  An MMA of up to 64 columns
                                // costs the same fixed time, so this takes a third off the tensor-pipe time.
                                const uint32_t iw = U.idesc_wide;
                                tc_mma_bf16(d_tmem, dAh, dBh, iw, acc0);
                                tc_mma_bf16(d_tmem, dAh + acap16, dBh, idesc, 1u);
                                for (uint32_t s = 1; s < nslab; ++s) {
                                    dAh += sa16; dBh += sb16;
                                    tc_mma_bf16(d_tmem, dAh, dBh, iw, 1u);
                                    tc_mma_bf16(d_tmem, dAh + acap16, dBh, idesc, 1u);
                                }
                                continue;
                            }
                            tc_mma_bf16(d_tmem, dAh, dBh, idesc, acc0);
                            tc_mma_bf16(d_tmem, dAh + acap16, dBh, idesc, 1u);
                            tc_mma_bf16(d_tmem, dAh, dBh + bcap16, idesc, 1u);
                            for (uint32_t s = 1; s < nslab; ++s) {
                                dAh += sa16; dBh += sb16;
                                tc_mma_bf16(d_tmem, dAh, dBh, idesc, 1u);
                                tc_mma_bf16(d_tmem, dAh + acap16, dBh, idesc, 1u);
                                tc_mma_bf16(d_tmem, dAh, dBh + bcap16, idesc, 1u);
                            }
                        }
                        tc_commit(bar_afree);
                        tc_commit(bar_free + 8 * st);
                        if (b0 + TB >= seg1 && sb == nsub - 1) tc_commit(bar_accfull + 8 * buf);
                    }
                }
                ++mi;
            }
        }
    } else {
        // =========================== compute warps ===========================
        uint32_t it = 0, mi = 0;
        int cur_set = -1;
        int64_t cx0 = 0, cx1 = 0;
        ItemPos cp_; cp_.init(blockIdx.x, a.n_nodes);        // position of the item whose bounds are in flight
        if ((int64_t)blockIdx.x < total) seg_bounds(a.ev.ptr, a.node0 + cp_.nl, a.ev.E, nullptr, cx0, cx1);
        // the item whose accumulator is drained next (one behind the one being built)
        int64_t p_nl = -1; int p_set = 0; uint32_t p_mi = 0; bool p_wrote = false;

        auto drain = [&](int64_t nl, int set, uint32_t dmi, bool wrote) {
            const TSet S = sSet[set];
            const uint32_t buf = dmi & 1;
            if (wrote) {
                mbar_wait(bar_accfull + 8 * buf, (dmi >> 1) & 1, a.status);
                tc_fence_after();
            }
            const int quarter = warp & 3, half = warp >> 2;
            for (int ui = 0; ui < S.nunit; ++ui) {
                const UInfo U = sU[S.unit_begin + ui];
                struct { int ncols, c_src; } B{(int)U.ncols, (int)U.c_src};
                const int r = quarter * 32 + lane;
                const int cl = r / KP, q = r - cl * KP;
                const bool rv = cl < (int)U.ncomp && q < a.K;
                int64_t off = 0;
                if (rv) {
                    const CompS cp = sComp[U.comp_begin + cl];
                    off = a.n_nodes * cp.zoff + (nl * cp.d_dst + cp.o) * (int64_t)cp.ld + cp.koff + (int64_t)q * B.c_src;
                }
                const int hc = B.ncols >> 1;       // columns per warp half (multiple of 8)
                const uint32_t trow = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * (uint32_t)a.acc_cols + U.tmem_col;
                if ((hc & 15) == 0) {              // 16 columns per TMEM load: half as many load round trips
                    for (int cc = half * hc; cc < (half + 1) * hc; cc += 16) {
                        float v[16];
                        if (wrote) {
                            tc_ld16(trow + (uint32_t)cc, v);
                            if (a.concat) {     // + A_hi x B_lo, accumulated 32 columns further on
                                float w[16];
                                tc_ld16(trow + 32u + (uint32_t)cc, w);
#pragma unroll
                                for (int i = 0; i < 16; ++i) v[i] += w[i];
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] = 0.f;
                        }
#pragma unroll
                        for (int g8 = 0; g8 < 16; g8 += 8) {
                            if (rv && cc + g8 < B.c_src) {
                                uint4 h, l;
                                split8(v + g8, h, l);
                                *reinterpret_cast<uint4*>(a.zh + off + cc + g8) = h;
                                *reinterpret_cast<uint4*>(a.zl + off + cc + g8) = l;
                            }
                        }
                    }
                } else {
                    for (int cc = half * hc; cc < (half + 1) * hc; cc += 8) {
                        float v[8];
                        if (wrote) {
                            tc_ld8(trow + (uint32_t)cc, v);
                            if (a.concat) {
                                float w[8];
                                tc_ld8(trow + 32u + (uint32_t)cc, w);
#pragma unroll
                                for (int i = 0; i < 8; ++i) v[i] += w[i];
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i) v[i] = 0.f;
                        }
                        if (rv && cc < B.c_src) {
                            uint4 h, l;
                            split8(v, h, l);
                            *reinterpret_cast<uint4*>(a.zh + off + cc) = h;
                            *reinterpret_cast<uint4*>(a.zl + off + cc) = l;
                        }
                    }
                }
            }
            if (wrote) {
                tc_fence_before();
                mbar_arrive(bar_accfree + 8 * buf);
            }
        };

        for (int64_t item = blockIdx.x; item < total; item += gridDim.x) {
            const int64_t nl = cp_.nl;
            const int set = cp_.set;
            const TSet S = sSet[set];
            const int64_t seg0 = cx0, seg1 = any_op ? cx1 : cx0;
            cp_.step(gridDim.x, a.n_nodes);
            if (item + gridDim.x < total)       // the next item's bounds, requested one item ahead
                seg_bounds(a.ev.ptr, a.node0 + cp_.nl, a.ev.E, nullptr, cx0, cx1);
            if (set != cur_set && seg1 > seg0) {     // entry and sparse-term tables of the set
                compute_sync();
                for (int i = tid; i < S.nent; i += NCW * 32) sEnt[i] = a.ents[S.ent_begin + i];
                for (int i = tid; i < S.pad; i += NCW * 32) sNz[i] = a.nz[S.b_items + i];
                compute_sync();
                cur_set = set;
            }
            for (int64_t b0 = seg0; b0 < seg1; b0 += TB)
            for (int sb = 0; sb < nsub; ++sb, ++it) {
                const int op = has_a1 ? sb : 1;          // which operand pair this sub-batch builds
                const int st = (int)(it % NS);
                mbar_wait(bar_full + 8 * st, (it / NS) & 1, a.status);
                const float* raw = reinterpret_cast<const float*>(sRing + (size_t)st * stage_bytes + (size_t)2 * NOP * a.b_cap);
                const float* sYT = raw + NRAW * TB * KP;
                const float* sVYT = sYT + a.dsh * PS;
                float* sM = sM0 + (size_t)(it & 1) * a.max_ent * PS;
                float* sdM = sdM0 + (size_t)(it & 1) * a.max_ent * PS;
                float* sPhiT = sPhiT0 + (size_t)(it & 1) * NRAW * KP * PS;     // [KP][PS] (+ vphi)
                float* sVphiT = sPhiT + KP * PS;
                // ---- transpose phi: [e][q] -> [q][e]   (same double buffer and barrier as the coupling matrices)
                for (int i = tid; i < TB * KP; i += NCW * 32) {
                    const int e = i / KP, q = i - e * KP;
                    sPhiT[q * PS + e] = raw[i];
                    if (DUAL) sVphiT[q * PS + e] = raw[TB * KP + i];
                }
                // ---- coupling matrices of the set: thread <-> (entry, 8 edges)
                for (int i = tid; i < 2 * S.nent; i += NCW * 32) {
                    const int j = i >> 1, h = i & 1;
                    const EntS en = sEnt[j];
                    float m[8], dm[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) { m[e] = 0.f; dm[e] = 0.f; }
                    for (int k = en.nz_begin; k < en.nz_begin + en.nz_count; ++k) {
                        const NzS t = sNz[k];
                        const float cf = t.coef;
                        const int b = t.b;
                        float y[8];
                        *reinterpret_cast<float4*>(y) = *reinterpret_cast<const float4*>(sYT + b * PS + 8 * h);
                        *reinterpret_cast<float4*>(y + 4) = *reinterpret_cast<const float4*>(sYT + b * PS + 8 * h + 4);
#pragma unroll
                        for (int e = 0; e < 8; ++e) m[e] = fmaf(cf, y[e], m[e]);
                        if (DUAL) {
                            *reinterpret_cast<float4*>(y) = *reinterpret_cast<const float4*>(sVYT + b * PS + 8 * h);
                            *reinterpret_cast<float4*>(y + 4) = *reinterpret_cast<const float4*>(sVYT + b * PS + 8 * h + 4);
#pragma unroll
                            for (int e = 0; e < 8; ++e) dm[e] = fmaf(cf, y[e], dm[e]);
                        }
                    }
                    *reinterpret_cast<float4*>(sM + j * PS + 8 * h) = *reinterpret_cast<const float4*>(m);
                    *reinterpret_cast<float4*>(sM + j * PS + 8 * h + 4) = *reinterpret_cast<const float4*>(m + 4);
                    if (DUAL) {
                        *reinterpret_cast<float4*>(sdM + j * PS + 8 * h) = *reinterpret_cast<const float4*>(dm);
                        *reinterpret_cast<float4*>(sdM + j * PS + 8 * h + 4) = *reinterpret_cast<const float4*>(dm + 4);
                    }
                }
                compute_sync();
                // the previous batch's MMAs must have read the A region before it is rewritten
                if (it > 0) mbar_wait(bar_afree, (it - 1) & 1, a.status);
                // ---- A slabs: thread <-> (entry, q), both 8-edge halves
                for (int i = tid; i < S.nent * KP; i += NCW * 32) {
                    const int j = i / KP, q = i - j * KP;
                    const int a_off = sEnt[j].a_off + (q >> 3) * 256 + (q & 7) * 16;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        float mv[8], ph[8], p1[8];
                        uint4 hh, ll;
                        *reinterpret_cast<float4*>(mv) = *reinterpret_cast<const float4*>(sM + j * PS + 8 * h);
                        *reinterpret_cast<float4*>(mv + 4) = *reinterpret_cast<const float4*>(sM + j * PS + 8 * h + 4);
                        *reinterpret_cast<float4*>(ph) = *reinterpret_cast<const float4*>(sPhiT + q * PS + 8 * h);
                        *reinterpret_cast<float4*>(ph + 4) = *reinterpret_cast<const float4*>(sPhiT + q * PS + 8 * h + 4);
                        if (!DUAL) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) p1[e] = ph[e] * mv[e];
                            split8(p1, hh, ll);
                            *reinterpret_cast<uint4*>(sA + a_off + 128 * h) = hh;
                            *reinterpret_cast<uint4*>(sA + a.a_cap + a_off + 128 * h) = ll;
                        } else if (op == 0) {
                            float dmv[8], vph[8];
                            *reinterpret_cast<float4*>(dmv) = *reinterpret_cast<const float4*>(sdM + j * PS + 8 * h);
                            *reinterpret_cast<float4*>(dmv + 4) = *reinterpret_cast<const float4*>(sdM + j * PS + 8 * h + 4);
                            *reinterpret_cast<float4*>(vph) = *reinterpret_cast<const float4*>(sVphiT + q * PS + 8 * h);
                            *reinterpret_cast<float4*>(vph + 4) = *reinterpret_cast<const float4*>(sVphiT + q * PS + 8 * h + 4);
#pragma unroll
                            for (int e = 0; e < 8; ++e) p1[e] = fmaf(vph[e], mv[e], ph[e] * dmv[e]);
                            split8(p1, hh, ll);
                            *reinterpret_cast<uint4*>(sA + a_off + 128 * h) = hh;
                            *reinterpret_cast<uint4*>(sA + a.a_cap + a_off + 128 * h) = ll;
                        } else {
#pragma unroll
                            for (int e = 0; e < 8; ++e) p1[e] = ph[e] * mv[e];
                            split8(p1, hh, ll);
                            *reinterpret_cast<uint4*>(sA + a_off + 128 * h) = hh;
                            *reinterpret_cast<uint4*>(sA + a.a_cap + a_off + 128 * h) = ll;
                        }
                    }
                }
                fence_async_smem();
                mbar_arrive(bar_ready);
            }
            // one item behind: the previous item's accumulator drains while this item's last MMAs run
            if (p_nl >= 0) drain(p_nl, p_set, p_mi, p_wrote);
            p_nl = nl; p_set = set; p_mi = mi; p_wrote = seg1 > seg0;
            if (seg1 > seg0) ++mi;
        }
        if (p_nl >= 0) drain(p_nl, p_set, p_mi, p_wrote);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)a.tmem_cols) : "memory");
    }
}

// shared bytes of the kernel for given region sizes
int smem_need(int KP, bool dual, int dsh, int a_cap, int b_cap, int max_ent, int n_units, int n_sets, int n_comps, int max_nz) {
    const int nop = dual ? 2 : 1;     // phi / Y / M come with their directions in the dual stream
    const int stage = 2 * b_cap + ((raw_floats(KP, dual, dsh) * 4 + 1023) & ~1023);
    size_t meta = (size_t)2 * nop * max_ent * PS + (size_t)2 * nop * KP * PS;
    meta = (meta + 1) & ~size_t(1);
    // tables: units (and at most as many blocks), sets, components, entries and sparse terms of one set
    const int tables = n_units * (int)(sizeof(UInfo) + sizeof(TBlk)) + n_sets * (int)sizeof(TSet) + n_comps * (int)sizeof(CompS) +
                       max_ent * (int)sizeof(EntS) + max_nz * (int)sizeof(NzS);
    return 1024 + 2 * a_cap + NS * stage + (int)(meta * 4) + (2 * NS + 8) * 8 + tables;
}

}  // namespace

// Units, sets and entries of one direction for the plain ([0]) and the dual ([1]) stream.
void build_tc_sets(const sobek_plan* p, Direction& dir) {
    const int KP = p->K <= 8 ? 8 : 16;
    for (int dual = 0; dual < 2; ++dual) {
        TcSets& T = dir.tc[dual];
        T = TcSets{};
        if (p->K > 16) continue;
        bool ok = true;
        for (const DPath& P : dir.paths)
            if ((P.c_src & 7) || P.c_src > 128 || (P.src_off & 7)) ok = false;
        if (!ok || (dir.C_src & 7) || dir.paths.empty()) continue;
        // distinct source blocks in order of appearance, with the components of all paths reading them
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
        // candidate units
        struct Cand { int blk, c0, nc; };
        std::vector<Cand> cands;
        const int comps_per_tile = 128 / KP;
        for (size_t b = 0; b < blocks.size(); ++b) {
            const int nc = (int)blocks[b].comps.size();
            const int ntile = (nc + comps_per_tile - 1) / comps_per_tile;
            const int per = (nc + ntile - 1) / ntile;
            for (int c0 = 0; c0 < nc; c0 += per) cands.push_back(Cand{(int)b, c0, std::min(per, nc - c0)});
        }
        auto unit_a = [&](const Cand& c) { return blocks[c.blk].d_src * (c.nc * KP) * 32; };
        auto blk_b = [&](int b) { return blocks[b].d_src * 2048 * ((blocks[b].c_src + 63) / 64); };
        auto ncols = [&](int b) { return (blocks[b].c_src + 15) & ~15; };
        // with every multiplicity <= 32 the lo copy of a gathered row fits beside the hi copy inside one 64-column
        // swizzle row: [B_hi | B_lo] is then one 64-column operand and a tile takes 64 accumulator columns
        bool concat = true;
        for (const Blk& b : blocks) concat = concat && b.c_src <= 32;
        auto cols32 = [&](int b) { return concat ? 64 : (ncols(b) + 31) & ~31; };
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
        int n_comps_total = 0;
        for (const Blk& b : blocks) n_comps_total += (int)b.comps.size();
        // greedy packing under a shared-memory budget: first for two CTAs per SM, else for one
        // sets of at most `maxu` units: the largest grouping that fits two CTAs per SM, else one CTA per SM
        for (int trial = 0; trial < 2 * (int)cands.size() && !T.ok; ++trial) {
            const int attempt = trial / (int)cands.size();
            const int maxu = (int)cands.size() - trial % (int)cands.size();
            const int budget = (attempt == 0 ? 113 : 226) * 1024;
            const int col_budget = attempt == 0 ? 128 : 256;     // two accumulator buffers per CTA
            T = TcSets{};
            bool fits = true;
            size_t i = 0;
            while (i < cands.size() && fits) {
                int a_bytes = 0, b_bytes = 0, cols = 0, nent = 0, nnz = 0;
                std::vector<int> set_blks;
                size_t j = i;
                for (; j < cands.size() && (int)(j - i) < maxu; ++j) {
                    const Cand& c = cands[j];
                    const bool new_blk = std::find(set_blks.begin(), set_blks.end(), c.blk) == set_blks.end();
                    const int a2 = a_bytes + unit_a(c), b2 = b_bytes + (new_blk ? blk_b(c.blk) : 0);
                    const int c2 = cols + cols32(c.blk), e2 = nent + c.nc * blocks[c.blk].d_src, n2 = nnz + cand_nz(c);
                    // the kernel sizes its regions by the maxima over all sets
                    const int acap = std::max(T.a_cap, (a2 + 4096 + 1023) & ~1023), bcap = std::max(T.b_cap, (b2 + 1023) & ~1023);
                    const int need = smem_need(KP, dual, p->dim_sh, acap, bcap, std::max(T.max_ent, e2), (int)cands.size(), (int)cands.size(),
                                               n_comps_total, std::max(T.max_nz, n2));
                    if (need > budget || c2 > col_budget) break;
                    a_bytes = a2; b_bytes = b2; cols = c2; nent = e2; nnz = n2;
                    if (new_blk) set_blks.push_back(c.blk);
                }
                if (j == i) { fits = false; break; }
                // emit the set
                TSet S{};
                S.unit_begin = (int)T.units.size(); S.blk_begin = (int)T.blks.size(); S.ent_begin = (int)T.ents.size();
                int a_off = 0, b_off = 0, col = 0;
                std::vector<int> local_blk;   // block index -> index in T.blks
                for (size_t k = i; k < j; ++k) {
                    const Cand& c = cands[k];
                    const Blk& Bk = blocks[c.blk];
                    int bi = -1;
                    for (size_t m = 0; m < local_blk.size(); ++m) if (local_blk[m] == c.blk) bi = S.blk_begin + (int)m;
                    if (bi < 0) {
                        TBlk tb{};
                        tb.src_off = Bk.so; tb.c_src = Bk.c_src; tb.d_src = Bk.d_src; tb.ncols = ncols(c.blk);
                        tb.b_off = b_off; tb.slab_bytes = 2048 * ((Bk.c_src + 63) / 64); tb.atom_stride = 2048;
                        b_off += blk_b(c.blk);
                        S.b_items += Bk.d_src * TB * (Bk.c_src / 8);
                        bi = (int)T.blks.size();
                        T.blks.push_back(tb);
                        local_blk.push_back(c.blk);
                    }
                    TUnit U{};
                    U.blk = bi; U.comp_begin = (int)T.comps.size(); U.ncomp = c.nc; U.a_off = a_off;
                    U.slab_stride = c.nc * KP * 32; U.tmem_col = col;
                    for (int cl = 0; cl < c.nc; ++cl) {
                        const SComp& cp = Bk.comps[c.c0 + cl];
                        T.comps.push_back(cp);
                        for (int s = 0; s < Bk.d_src; ++s)
                            T.ents.push_back(TEnt{cp.tab0 + s * cp.tstride, cp.sh_off, a_off + s * U.slab_stride + cl * KP * 32, 0});
                    }
                    a_off += unit_a(c);
                    col += cols32(c.blk);
                    T.units.push_back(U);
                }
                S.nunit = (int)T.units.size() - S.unit_begin; S.nblk = (int)T.blks.size() - S.blk_begin;
                S.nent = (int)T.ents.size() - S.ent_begin;
                T.sets.push_back(S);
                T.a_cap = std::max(T.a_cap, (a_off + 4096 + 1023) & ~1023);
                T.b_cap = std::max(T.b_cap, (b_off + 1023) & ~1023);
                T.max_ent = std::max(T.max_ent, S.nent);
                T.max_nz = std::max(T.max_nz, nnz);
                T.acc_cols = std::max(T.acc_cols, col);
                i = j;
            }
            if (!fits) continue;
            int tc = 32; while (tc < 2 * T.acc_cols) tc <<= 1;
            T.tmem_cols = tc;
            T.smem_bytes = smem_need(KP, dual, p->dim_sh, T.a_cap, T.b_cap, T.max_ent, (int)cands.size(), (int)cands.size(), n_comps_total, T.max_nz);
            if (T.smem_bytes > 227 * 1024 || T.tmem_cols > 512) continue;
            T.ctas_per_sm = (T.smem_bytes <= 113 * 1024 && T.tmem_cols <= 256) ? 2 : 1;
            T.concat = concat ? 1 : 0;
            // shared-memory images of the tables
            for (TSet& S : T.sets) {
                S.b_items = (int)T.nz.size();
                for (int j = 0; j < S.nent; ++j) {
                    const TEnt& E = T.ents[S.ent_begin + j];
                    EntS es{E.a_off, (int)T.nz.size() - S.b_items, p->tab_ptr[E.tab + 1] - p->tab_ptr[E.tab], 0};
                    for (int k = p->tab_ptr[E.tab]; k < p->tab_ptr[E.tab + 1]; ++k) T.nz.push_back(NzS{E.sh_off + p->tab_idx[k], p->tab_coef[k]});
                    T.ents_s.push_back(es);
                }
                S.pad = (int)T.nz.size() - S.b_items;
            }
            for (const SComp& cp : T.comps)
                T.comps_s.push_back(CompS{dir.zb_off[cp.group], dir.nk_ld[cp.group], cp.d_dst, cp.o, cp.koff, {0, 0}});
            T.ok = true;
        }
    }
}

cudaError_t launch_stream_tc(const sobek_plan* p, const Direction& dir, const EdgeView& ev, int64_t node0,
                             int64_t n_nodes, const SplitSrc& ss, const float* Y, const float* vY, const float* phi,
                             const float* vphi, int dual, void* zh, void* zl, int* status, cudaStream_t s) {
    const TcSets& T = dir.tc[dual ? 1 : 0];
    if (!T.ok || !ss.h || !ss.l) return cudaErrorInvalidValue;
    if (n_nodes <= 0) return cudaSuccess;
    TcArgs a{};
    a.sets = T.d_sets; a.units = T.d_units; a.blks = T.d_blks; a.ents = T.d_ents_s; a.nz = T.d_nz; a.comps = T.d_comps_s;
    a.ev = ev; a.node0 = node0; a.n_nodes = n_nodes;
    a.sh = (const __nv_bfloat16*)ss.h; a.sl = (const __nv_bfloat16*)ss.l;
    a.vsh = (const __nv_bfloat16*)ss.vh; a.vsl = (const __nv_bfloat16*)ss.vl;
    a.Y = Y; a.vY = vY; a.phi = phi; a.vphi = vphi;
    a.zh = (__nv_bfloat16*)zh; a.zl = (__nv_bfloat16*)zl;
    a.K = p->K; a.dsh = p->dim_sh; a.C_src = dir.C_src; a.nsets = (int)T.sets.size();
    a.a_cap = T.a_cap; a.b_cap = T.b_cap; a.max_ent = T.max_ent; a.tmem_cols = T.tmem_cols; a.acc_cols = T.acc_cols; a.concat = T.concat; a.n_units = (int)T.units.size(); a.n_blks = (int)T.blks.size(); a.n_comps = (int)T.comps.size(); a.max_nz = T.max_nz;
    a.status = status;
    const bool k8 = p->K <= 8;
    void (*kern)(const TcArgs) = k8 ? (dual ? k_stream_tc<8, true> : k_stream_tc<8, false>)
                                    : (dual ? k_stream_tc<16, true> : k_stream_tc<16, false>);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, T.smem_bytes);
    if (e != cudaSuccess) return e;
    const int64_t total = n_nodes * a.nsets;
    const int grid = (int)std::min<int64_t>(total, (int64_t)148 * T.ctas_per_sm);
    KernelTimer kt(K_STATE, s);
    kern<<<grid, TT, T.smem_bytes, s>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace sobek
