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
// The A operand never touches shared memory: the thread that owns accumulator row (comp,q) computes the 16
// values of one slab (one s, 16 edges) in registers, splits them and stores them with tcgen05.st into a ring
// of slab slots in tensor memory, from where tcgen05.mma reads them (A in TMEM, B from a shared-memory
// descriptor).  Shared-memory bandwidth is then spent on the gathered rows only.
//
// One CTA per SM works through (pass, receiver) items in pass-major order (a pass = the accumulator tiles that
// fit one of two TMEM accumulator buffers), edges in batches of 16, with four roles:
//   loader warps   run ahead (segment bounds and edge / sender ids are requested one step early): cp.async of
//                  the batch's phi rows, of its Y rows (written transposed) and of the sender rows straight
//                  into the B slabs (16 edges x c_src, MN-major, 128-byte swizzle) of a ring of stages; the
//                  copies signal the stage's mbarrier themselves when they land;
//   builder warps  three groups of four (one warp per TMEM lane quarter).  Group g produces every third A slab of
//                  the batch into its two TMEM slots (the slabs of a pass are listed tile after tile in turn, so
//                  that the groups and the MMA threads are evenly loaded whatever the mix of source orders).  Per
//                  batch it first expands the coupling values M_e[s,comp] of its own slabs from the sparse CG
//                  table (kept in shared memory, like every other table the kernel looks up) into a buffer of
//                  its own: one barrier among its 128 threads per batch, none with the other groups;
//   MMA threads    three, in three warps (one thread gets a tcgen05.mma accepted every ~110 cycles whatever its
//                  size, the pipe takes them three times as fast); thread t owns the accumulator tiles
//                  unit = t mod 3 of the pass (a tile's products all come from one thread, in a fixed order), issues
//                  the three products of a slab of theirs as soon as its slot is full, and commits to the
//                  mbarriers that release the slot, the ring stage and the accumulator buffer;
//   drain warps    read a finished accumulator (tcgen05.ld), split it into bf16 hi / lo and write the rows of
//                  the node GEMM's A operand (contraction index k = koff + q*c_src + u, so a row of 16-byte
//                  pieces per thread) while the next receiver's products run into the other buffer.
// With DUAL the kernel produces the directional state of the double backward
//     dZ = sum_e ( vphi (x) C(x,Y) + phi (x) [ C(vx,Y) + C(x,vY) ] )       (Eq. receiver_double_adjoint)
// as  [vphi*M + phi*dM] x B(x)  +  [phi*M] x B(vx).
// The same kernel runs the sender-owned transposed traversal.  Every mbarrier wait is bounded.
#include <cuda_bf16.h>

#include <algorithm>

#include "geometry.cuh"
#include "guard.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace sobek {
namespace {

using namespace ptx;

constexpr int TB = 16;          // edges per batch = k extent of one MMA
constexpr int NBG = 3;          // builder groups (four warps each: one per TMEM lane quarter)
constexpr int NBW = 4 * NBG;    // builder warps
constexpr int NDW = 4;          // drain warps
constexpr int NLW = 4;          // loader warps
constexpr int NMW = 3;          // MMA warps (one issuing thread each; a unit's products all come from one of them)
constexpr int W_DRAIN = NBW, W_LOAD = NBW + NDW, W_MMA = NBW + NDW + NLW;
constexpr int W_GEO = W_MMA + NMW;           // the last warp: recomputes phi and Y from edge vectors in geometry mode, else idle
constexpr int TT = (W_GEO + 1) * 32;         // threads per CTA (a multiple of 128)
constexpr int MAXNS = 4;        // ring stages: 2..4, as many as shared memory holds
constexpr int NSLOT = 2 * NBG;  // A slab slots in tensor memory, two per builder group: 16 columns each (8 hi + 8 lo)
constexpr int TMEM_COLS = 512;
constexpr int RING0 = TMEM_COLS - NSLOT * 16;      // first column of the slot ring
constexpr int DRAIN_BYTES = NDW * 32 * 64 * 2;   // per drain warp: 32 rows x 32 columns, bf16 hi and lo
constexpr int ACC_BUDGET = RING0 / 2;              // columns of one accumulator buffer (two buffers)
constexpr int PS = 20;          // row pitch (floats) of the transposed stages: 16 values + 4 (bank spread)
static_assert(NSLOT % NBG == 0, "slab j of a batch goes to slot j mod NSLOT, built by group j mod NBG");

struct TcArgs {
    const TSet* sets;
    const TUnit* units;
    const TBlk* blks;
    const EntS* ents;      // per set (TSet::ent_begin)
    const NzS* nz;         // per set (TSet::b_items = first term, TSet::pad = number of terms)
    const CompS* comps;
    EdgeView ev;
    int64_t node0, n_nodes;
    const int4* oseg;           // the chunk's nodes in processing order {local node, segment begin, end} or NULL
    const __nv_bfloat16* sh;    // bf16 hi / lo copies of the source features [N][C_src]
    const __nv_bfloat16* sl;
    const __nv_bfloat16* vsh;   // DUAL: the same for the source direction; NULL without it
    const __nv_bfloat16* vsl;
    const float* Y;
    const float* vY;
    const float* phi;
    const float* vphi;
    const float* rvec;     // edge vectors [E][3]: when set, Y and phi are recomputed from them (Y, phi are NULL then)
    const float* vrvec;    // DUAL, geometry mode: direction on the edge vectors; vY = J_Y vrvec, vphi = J_phi vrvec
    float geo_rc;          // cutoff radius of the radial basis
    int32_t geo_basis, geo_p;
    int32_t geo_inline;    // geometry mode: 0 = the geometry warp recomputes phi and Y (the default: nearly free, the warp has
                           // nothing else to do); 1 = the loader warps do it themselves between their copies (measured
                           // 5 - 20 % slower in the forward; the loader is close to the critical path)
    __nv_bfloat16* zh;
    __nv_bfloat16* zl;
    int32_t K, dsh, C_src, nsets;
    int32_t b_cap, max_ent, acc_cols, n_units, n_blks, n_comps, max_nz, ns, n_slab;
    int32_t nbuf;           // accumulator buffers: 2 (a set's tiles fit half of the accumulator columns; the drain of one item
                            // overlaps the MMAs of the next) or 1 (wider sets, the MMAs wait for the drain)
    int32_t max_own;        // slabs of a batch that one builder group builds, at most
    const uint32_t* slabs;  // per set (TSet::sched_begin, nslab): two words per slab, in build order (see SlabW)
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

// Everything the roles look up per item, batch or slab lives in shared memory: with most of the SM's
// L1 given to the operand regions, table reads from global memory would mostly go to L2.
struct UInfo {     // a unit, as the MMA thread, the builders and the drain need it
    uint32_t idesc, tmem_col, d_src, comp_begin, ncomp, c_src, ncols, ent0;
    uint64_t dB0;    // operand descriptor of the unit's B slab 0 (hi copy, stage 0 of the ring): the other slabs,
    uint64_t sb16;   // copies and stages differ only in the 16-byte-granular address field (sb16 per slab)
};

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// hand-over by a count in shared memory that only grows: the producer adds with release semantics, the consumer
// polls with acquire semantics until the count reaches its target (bounded like every other wait of the kernel)
__device__ __forceinline__ void count_add(uint32_t addr) {
    asm volatile("red.release.cta.shared::cta.add.u32 [%0], 1;" ::"r"(addr) : "memory");
}
__device__ __forceinline__ void count_wait(uint32_t addr, uint32_t target, int* status) {
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        uint32_t v;
        asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
        if ((int32_t)(v - target) >= 0) return;
        if ((it & 255u) == 0) {
            uint64_t t1;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
            if (it == 0) t0 = t1;
            else if (t1 - t0 > 2000000000ull) break;
        }
    }
    atomicExch(status, (int)SOBEK_ERR_DEVICE_TIMEOUT);
}
__device__ __forceinline__ void group_sync(int grp) { asm volatile("bar.sync %0, 128;" ::"r"(2 + grp) : "memory"); }
__device__ __forceinline__ void builder_sync() { asm volatile("bar.sync 1, %0;" ::"n"(NBW * 32) : "memory"); }
// A slab of a pass in build order, as two words.
//   bw: (first entry of the tile + s) | d_src << 16 | ncomp << 24         what the builders need
//   mw: tile in the pass | s << 8 | next slab of the same MMA thread << 16 (255: none)
struct SlabW { uint32_t bw, mw; };

// cp.async with zero fill: copies `bytes` (0 or the full size) and fills the rest with zeros
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async4_zfill(uint32_t dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
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
__global__ void __launch_bounds__(TT, 1) k_stream_tc(const TcArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    constexpr int NRAW = DUAL ? 2 : 1;     // raw / transposed stages: phi and Y, plus their directions
    const int NS = a.ns;
    // ring stages: Bh Bl, then the raw phi / Y rows
    const uint32_t stage_bytes = (uint32_t)(2 * a.b_cap + ((raw_floats(KP, DUAL, a.dsh) * 4 + 1023) & ~1023));
    uint8_t* sRing = smem;
    uint8_t* sDrain = sRing + (size_t)NS * stage_bytes;      // staging of the drain warps (DRAIN_BYTES)
    uint8_t* meta = sDrain + DRAIN_BYTES;
    // coupling values of a group's own slabs of one batch, double buffered: [NBG][2][max_own][MC][PS] (+ directions)
    constexpr int MC = 128 / KP;                              // components of a tile at most
    const size_t mbuf_floats = (size_t)a.max_own * MC * PS;
    float* sM0 = reinterpret_cast<float*>(meta);
    float* sdM0 = sM0 + (size_t)NBG * 2 * mbuf_floats;        // DUAL
    uint64_t* bars = reinterpret_cast<uint64_t*>(sdM0 + (DUAL ? (size_t)NBG * 2 * mbuf_floats : 0));
    // bars: full[MAXNS], sfree[MAXNS], slot_free[NSLOT], acc_full[2], acc_free[2]
    constexpr int NBAR = 2 * MAXNS + NSLOT + 4;
    // slot_fill[s]: warps that have finished storing into slot s, counted over the whole kernel (4 per use).  A slot is
    // consumed by whichever MMA thread owns the slab's tile, so its hand-over is a count that only grows (an mbarrier's
    // parity could be misread by a thread that is two uses ahead of another).
    uint32_t* slot_fill = reinterpret_cast<uint32_t*>(bars + NBAR);
    uint32_t* tmem_holder = slot_fill + NSLOT + (NSLOT & 1);
    UInfo* sU = reinterpret_cast<UInfo*>(tmem_holder + 2);             // [n_units]
    TSet* sSet = reinterpret_cast<TSet*>(sU + a.n_units);               // [nsets]
    TBlk* sBlk = reinterpret_cast<TBlk*>(sSet + a.nsets);               // [n_blks]
    CompS* sComp = reinterpret_cast<CompS*>(sBlk + a.n_blks);           // [n_comps]
    EntS* sEnt = reinterpret_cast<EntS*>(sComp + a.n_comps);            // [max_ent]  (current set)
    NzS* sNz = reinterpret_cast<NzS*>(sEnt + a.max_ent);                // [max_nz]   (current set)
    SlabW* sSlab = reinterpret_cast<SlabW*>(sNz + a.max_nz);            // [n_slab]
    const uint32_t bar0 = smem_u32(bars);
    const uint32_t bar_full = bar0, bar_sfree = bar0 + 8 * MAXNS, bar_slotfree = bar0 + 16 * MAXNS,
                   bar_accfull = bar_slotfree + 8 * NSLOT, bar_accfree = bar_accfull + 16;
    const uint32_t fill0 = smem_u32(slot_fill);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool has_vx = DUAL && a.vsh != nullptr, has_vY = DUAL && (a.rvec ? a.vrvec != nullptr : a.vY != nullptr),
               has_vphi = DUAL && (a.rvec ? a.vrvec != nullptr : a.vphi != nullptr);
    const bool has_a1 = !DUAL || has_vY || has_vphi;   // operand 1: [phi*M] (plain) or [vphi*M + phi*dM] (dual), times x
    const bool has_a2 = has_vx;                        // operand 2 (dual): [phi*M] times vx
    const bool any_op = has_a1 || has_a2;
    // sub-batches per batch of edges: one per operand pair that is present (op = 0: x rows, op = 1: vx rows)
    const int nsub = (has_a1 ? 1 : 0) + (has_a2 ? 1 : 0);

    if (tid == 0) {
        // a stage is full when every loader thread's copies have landed (and the geometry warp, where it runs, has stored phi and Y)
        for (int s = 0; s < MAXNS; ++s) { mbar_init(bar_full + 8 * s, NLW * 32 + ((a.rvec && !a.geo_inline) ? 32 : 0)); mbar_init(bar_sfree + 8 * s, NMW); }
        for (int s = 0; s < NSLOT; ++s) { mbar_init(bar_slotfree + 8 * s, 1); slot_fill[s] = 0u; }
        for (int t = 0; t < 2; ++t) { mbar_init(bar_accfull + 8 * t, NMW); mbar_init(bar_accfree + 8 * t, NDW); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // every slot starts out free: its first phase completes here, so that the builders wait on it like on any other
        for (int s = 0; s < NSLOT; ++s) mbar_arrive(bar_slotfree + 8 * s);
    }
    // the raw rows of padded radial components (q >= K) and of absent directions stay zero for ever
    {
        const int words = (int)(stage_bytes / 4), b_words = 2 * a.b_cap / 4;
        for (int i = tid; i < NS * words; i += TT) {
            const int st = i / words, w = i - st * words;
            if (w >= b_words) reinterpret_cast<uint32_t*>(sRing + (size_t)st * stage_bytes)[w] = 0u;
        }
    }
    for (int i = tid; i < a.n_units; i += TT) {
        const TUnit U = a.units[i];
        const TBlk B = a.blks[U.blk];
        UInfo u;
        // D = F32, A = B = BF16, A K-major (tensor memory), B MN-major, M = 128, N = ncols
        u.idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(B.ncols >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        u.tmem_col = (uint32_t)U.tmem_col; u.d_src = (uint32_t)B.d_src;
        u.comp_begin = (uint32_t)U.comp_begin; u.ncomp = (uint32_t)U.ncomp; u.c_src = (uint32_t)B.c_src;
        u.ncols = (uint32_t)B.ncols; u.ent0 = (uint32_t)U.a_off;
        u.dB0 = make_desc(smem_u32(sRing) + (uint32_t)B.b_off, 2048, 1024);
        u.sb16 = (uint64_t)(B.slab_bytes >> 4);
        sU[i] = u;
    }
    for (int i = tid; i < a.nsets; i += TT) sSet[i] = a.sets[i];
    for (int i = tid; i < a.n_blks; i += TT) sBlk[i] = a.blks[i];
    for (int i = tid; i < a.n_comps; i += TT) sComp[i] = a.comps[i];
    for (int i = tid; i < 2 * a.n_slab; i += TT) reinterpret_cast<uint32_t*>(sSlab)[i] = a.slabs[i];
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(tmem_holder)), "r"((uint32_t)TMEM_COLS) : "memory");
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
    // segment of the node at position v of the chunk's processing order; returns the node's local index
    auto item_bounds = [&](int64_t v, int* status, int64_t& s0, int64_t& s1) -> int64_t {
        if (a.oseg) { const int4 q = __ldg(a.oseg + v); s0 = q.y; s1 = q.z; return q.x; }
        seg_bounds(a.ev.ptr, a.node0 + v, a.ev.E, status, s0, s1);
        return v;
    };

    if (warp >= W_LOAD && warp < W_LOAD + NLW) {
        // =========================== loader warps ===========================
        // The segment bounds of the next item and the ids of the next batch are requested one step ahead,
        // so that their latency overlaps the issue of the current batch's copies; the copies themselves
        // signal the stage's mbarrier when they land (no wait in this warp).
        const int lt = (warp - W_LOAD) * 32 + lane;   // thread index among the loaders
        int64_t p_item = blockIdx.x, p_seg0 = 0, p_seg1 = 0;     // prefetched item
        ItemPos lp; lp.init(p_item, a.n_nodes);
        auto prefetch_item = [&]() {
            if (p_item < total) {
                item_bounds(lp.nl, a.status, p_seg0, p_seg1);
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
        int st = 0; uint32_t round = 0;      // stage of the batch and how often the ring has wrapped
        for (; have;) {
            Cur nxt = cur;
            const bool have_n = next_batch(nxt, false);
            int64_t eid_n = 0; int32_t sn_n = 0; uint32_t msk_n = 0;
            if (have_n) load_ids(nxt, eid_n, sn_n, msk_n);
            const TSet S = sSet[cur.set];
            const int op = has_a1 ? cur.sub : 1;
            if (round > 0) mbar_wait(bar_sfree + 8 * st, (round & 1) ^ 1, a.status);
            const uint32_t stage_u = smem_u32(sRing + (size_t)st * stage_bytes);
            const uint32_t raw_u = stage_u + (uint32_t)(2 * a.b_cap);
            const int le = lane & (TB - 1);
            const int64_t ee_own = __shfl_sync(0xffffffffu, eid, le);
            if (a.rvec) {
                if (a.geo_inline) {
                // recomputed from the edge vector: thread <-> (edge le, share g8 of the components and radial indices)
                const int g8 = lt >> 4;
                const bool okb = (msk >> le) & 1u;
                float rx = 0.f, ry = 0.f, rz = 1.f;
                if (okb) { const float* rp = a.rvec + ee_own * 3; rx = __ldg(rp); ry = __ldg(rp + 1); rz = __ldg(rp + 2); }
                const float r = sqrtf(rx * rx + ry * ry + rz * rz), ir = 1.f / r;
                float* rawf = reinterpret_cast<float*>(sRing + (size_t)st * stage_bytes + (size_t)2 * a.b_cap);
                float* yT = rawf + NRAW * TB * KP;
                geo_radial(r, a.K, a.geo_rc, a.geo_basis, a.geo_p, [&](int q, float f, float) {
                    if ((q & 7) == g8) rawf[le * KP + q] = okb ? f : 0.f;
                });
                const int dsh = a.dsh;
                geo_sh(rx * ir, ry * ir, rz * ir, [&](int b, float yb, float, float, float) {
                    if (b < dsh && (b & 7) == g8) yT[b * PS + le] = okb ? yb : 0.f;
                });
                __threadfence_block();       // the stores above are ordered before this thread's arrival on the stage
                }
            } else {
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
            // Y (and vY), transposed: raw[b][PS + e].  Thread <-> (edge e = lane mod 16, b = lt / 16, + 8, ...)
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
            }
            // sender rows -> B slabs (hi and lo), 16 bytes = 8 multiplicities per copy
            {
                // Eight consecutive loader threads serve one edge (four or two for blocks of fewer than 64 / 32
                // multiplicities): a copy instruction then reads whole 128-byte runs of four sender rows instead of 32 bytes
                // of sixteen.  A thread walks pieces j0, j0 + 8, ... of its edge's row.
                const __nv_bfloat16* baseh = op == 0 ? a.sh : a.vsh;
                const __nv_bfloat16* basel = op == 0 ? a.sl : a.vsl;
                for (int bi = 0; bi < S.nblk; ++bi) {
                    const TBlk B = sBlk[S.blk_begin + bi];
                    const int cpr = B.c_src >> 3;                  // 16-byte pieces per row
                    const int lgp = cpr >= 8 ? 3 : (cpr >= 4 ? 2 : 1);
                    const int re = lt >> lgp, j0 = lt & ((1 << lgp) - 1);
                    const int32_t sne = __shfl_sync(0xffffffffu, sn, re & (TB - 1));
                    if (re < TB) {
                        const uint32_t ok = ((msk >> re) & 1u) * 16u;
                        const int64_t grow = (int64_t)sne * a.C_src + B.src_off;
                        for (int j = j0; j < cpr; j += 1 << lgp) {
                            const int u = 8 * j;
                            uint32_t d = stage_u + (uint32_t)(B.b_off + (u >> 6) * B.atom_stride + re * 128 + ((((u & 63) >> 3) ^ (re & 7)) << 4));
                            const __nv_bfloat16* ph = baseh + grow + u;
                            const __nv_bfloat16* pl = basel + grow + u;
                            for (int sdx = 0; sdx < B.d_src; ++sdx) {
                                cp_async16_zfill(d, ph, ok);
                                cp_async16_zfill(d + (uint32_t)a.b_cap, pl, ok);
                                d += (uint32_t)B.slab_bytes; ph += B.c_src; pl += B.c_src;
                            }
                        }
                    }
                }
            }
            // this thread's arrival on the stage's barrier fires when all its copies above have landed
            asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar_full + 8 * st) : "memory");
            cur = nxt; have = have_n; eid = eid_n; sn = sn_n; msk = msk_n;
            if (++st == NS) { st = 0; ++round; }
        }
    } else if (warp == W_GEO) {
        // =========================== geometry warp ===========================
        // Walks the same batches as the loaders and fills the stage's phi rows and transposed Y from the edge vectors
        // (lane <-> edge lane & 15, half of the radial indices / components each).
        if (a.rvec != nullptr && !a.geo_inline) {
            int64_t p_item = blockIdx.x, p_seg0 = 0, p_seg1 = 0;
            ItemPos lp; lp.init(p_item, a.n_nodes);
            auto prefetch_item = [&]() {
                if (p_item < total) {
                    item_bounds(lp.nl, nullptr, p_seg0, p_seg1);
                    if (!any_op) p_seg1 = p_seg0;
                }
            };
            prefetch_item();
            int64_t b0 = 0, seg1 = 0;
            auto next_batch = [&](bool first) -> bool {
                if (!first) b0 += TB;
                while (first || b0 >= seg1) {
                    first = false;
                    if (p_item >= total) return false;
                    b0 = p_seg0; seg1 = p_seg1;
                    p_item += gridDim.x; lp.step(gridDim.x, a.n_nodes);
                    prefetch_item();
                }
                return true;
            };
            const int le = lane & (TB - 1), hf = lane >> 4;
            int st = 0; uint32_t round = 0;
            for (bool have = next_batch(true); have; have = next_batch(false)) {
                const int64_t pos = b0 + le;
                bool okb = pos < seg1;
                int64_t ee = 0;
                if (okb) { ee = a.ev.perm ? (int64_t)a.ev.perm[pos] : pos; okb = ee >= 0 && ee < a.ev.E; }
                float rx = 0.f, ry = 0.f, rz = 1.f;
                if (okb) { const float* rp = a.rvec + ee * 3; rx = __ldg(rp); ry = __ldg(rp + 1); rz = __ldg(rp + 2); }
                const float r = sqrtf(rx * rx + ry * ry + rz * rz), ir = 1.f / r;
                // every sub-batch of the batch (one per operand pair of the dual pass) has a stage of its own and needs the same rows
                for (int sub = 0; sub < nsub; ++sub) {
                if (round > 0) mbar_wait(bar_sfree + 8 * st, (round & 1) ^ 1, a.status);
                float* rawf = reinterpret_cast<float*>(sRing + (size_t)st * stage_bytes + (size_t)2 * a.b_cap);
                float* yT = rawf + NRAW * TB * KP;
                const float ux = rx * ir, uy = ry * ir, uz = rz * ir;
                // DUAL: the directions vphi = phi'(r) (u . v) and vY = grad F . (v - u (u . v)) / r of the edge-vector direction v
                float uv = 0.f, tx = 0.f, ty = 0.f, tz = 0.f;
                const bool dirs = DUAL && a.vrvec != nullptr;
                if (dirs && okb) {
                    const float* vp = a.vrvec + ee * 3;
                    const float vx_ = __ldg(vp), vy_ = __ldg(vp + 1), vz_ = __ldg(vp + 2);
                    uv = ux * vx_ + uy * vy_ + uz * vz_;
                    tx = (vx_ - ux * uv) * ir; ty = (vy_ - uy * uv) * ir; tz = (vz_ - uz * uv) * ir;
                }
                geo_radial(r, a.K, a.geo_rc, a.geo_basis, a.geo_p, [&](int q, float f, float df) {
                    if ((q & 1) == hf) {
                        rawf[le * KP + q] = okb ? f : 0.f;
                        if (dirs) rawf[TB * KP + le * KP + q] = okb ? df * uv : 0.f;
                    }
                });
                const int dsh = a.dsh;
                geo_sh(ux, uy, uz, [&](int b, float yb, float fx, float fy, float fz) {
                    if (b < dsh && (b & 1) == hf) {
                        yT[b * PS + le] = okb ? yb : 0.f;
                        if (dirs) yT[dsh * PS + b * PS + le] = okb ? fx * tx + fy * ty + fz * tz : 0.f;
                    }
                });
                mbar_arrive(bar_full + 8 * st);      // release: the stores above are visible to whoever sees the stage full
                if (++st == NS) { st = 0; ++round; }
                }
            }
        }
    } else if (warp >= W_MMA && warp < W_MMA + NMW) {
        // =========================== MMA warps ===========================
        if (lane == 0) {
            const uint32_t me = (uint32_t)(warp - W_MMA);
            uint32_t mi = 0;
            uint32_t uses[NSLOT];            // how often every slot has been used before the current batch
#pragma unroll
            for (int s = 0; s < NSLOT; ++s) uses[s] = 0u;
            int st = 0; uint32_t round = 0;
            int64_t nx0 = 0, nx1 = 0;
            ItemPos mp; mp.init(blockIdx.x, a.n_nodes);      // position of the item whose bounds are in flight
            if ((int64_t)blockIdx.x < total) item_bounds(mp.nl, nullptr, nx0, nx1);
            const uint64_t bcap16 = (uint64_t)(a.b_cap >> 4);
            for (int64_t item = blockIdx.x; item < total; item += gridDim.x) {
                const TSet S = sSet[mp.set];
                const int64_t seg0 = nx0, seg1 = any_op ? nx1 : nx0;
                mp.step(gridDim.x, a.n_nodes);
                if (item + gridDim.x < total)       // the next item's bounds, requested one item ahead
                    item_bounds(mp.nl, nullptr, nx0, nx1);
                if (seg1 <= seg0) continue;
                const uint32_t buf = a.nbuf == 2 ? (mi & 1) : 0u, gen = a.nbuf == 2 ? (mi >> 1) : mi;    // buffer and its use count
                if (mi >= (uint32_t)a.nbuf) mbar_wait(bar_accfree + 8 * buf, (gen & 1) ^ 1, a.status);
                tc_fence_after();
                const SlabW* slabs = sSlab + S.sched_begin;
                const uint32_t j0 = ((uint32_t)S.mfirst >> (8 * me)) & 255u;     // first slab of this thread (255: none)
                for (int64_t b0 = seg0; b0 < seg1; b0 += TB) {
                    for (int sb = 0; sb < nsub; ++sb) {
                        mbar_wait(bar_full + 8 * st, round & 1, a.status);
                        fence_async_smem();      // the gathered rows were written through the generic proxy
                        const uint64_t st16 = (uint64_t)((uint32_t)st * (stage_bytes >> 4));
                        const bool first = b0 == seg0 && sb == 0;
                        for (uint32_t j = j0; j != 255u;) {
                            const uint32_t mw = slabs[j].mw, ui = mw & 255u, sl = (mw >> 8) & 255u;
                            const UInfo& U = sU[S.unit_begin + ui];
                            const uint32_t d_tmem = tmem_base + buf * (uint32_t)a.acc_cols + U.tmem_col;
                            const uint64_t dBh = U.dB0 + st16 + sl * U.sb16;
                            const uint32_t idesc = U.idesc;
                            const uint32_t slot = j % NSLOT, use = j / NSLOT;
                            uint32_t before = 0;
#pragma unroll
                            for (int s = 0; s < NSLOT; ++s) before = slot == (uint32_t)s ? uses[s] : before;
                            count_wait(fill0 + 4 * slot, 4u * (before + use + 1u), a.status);
                            tc_fence_after();
                            const uint32_t a_h = tmem_base + (uint32_t)RING0 + slot * 16u, a_l = a_h + 8u;
                            tc_mma_bf16_ts(d_tmem, a_h, dBh, idesc, (first && sl == 0) ? 0u : 1u);
                            tc_mma_bf16_ts(d_tmem, a_l, dBh, idesc, 1u);
                            tc_mma_bf16_ts(d_tmem, a_h, dBh + bcap16, idesc, 1u);
                            tc_commit(bar_slotfree + 8 * slot);
                            j = (mw >> 16) & 255u;
                        }
#pragma unroll
                        for (int s = 0; s < NSLOT; ++s) uses[s] += (uint32_t)(S.nslab + NSLOT - 1 - s) / NSLOT;
                        // (a commit with nothing outstanding arrives at once: every MMA thread takes part)
                        tc_commit(bar_sfree + 8 * st);
                        if (b0 + TB >= seg1 && sb == nsub - 1) tc_commit(bar_accfull + 8 * buf);
                        if (++st == NS) { st = 0; ++round; }
                    }
                }
                ++mi;
            }
        }
    } else if (warp >= W_DRAIN && warp < W_DRAIN + NDW) {
        // =========================== drain warps ===========================
        // one thread per accumulator row (TMEM lane); a warp reaches the 32 lanes of its quarter only
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;
        const int cl = r / KP, q = r - cl * KP;
        uint32_t mi = 0;
        int64_t dx0 = 0, dx1 = 0;
        ItemPos dp; dp.init(blockIdx.x, a.n_nodes);
        int64_t dnl = 0;                 // local index of the node whose bounds are in flight
        if ((int64_t)blockIdx.x < total) dnl = item_bounds(dp.nl, nullptr, dx0, dx1);
        for (int64_t item = blockIdx.x; item < total; item += gridDim.x) {
            const int64_t nl = dnl;
            const TSet S = sSet[dp.set];
            const int64_t seg0 = dx0, seg1 = any_op ? dx1 : dx0;
            dp.step(gridDim.x, a.n_nodes);
            if (item + gridDim.x < total) dnl = item_bounds(dp.nl, nullptr, dx0, dx1);
            const bool wrote = seg1 > seg0;      // a node without edges has a state of zeros
            const uint32_t buf = a.nbuf == 2 ? (mi & 1) : 0u, gen = a.nbuf == 2 ? (mi >> 1) : mi;
            if (wrote) {
                mbar_wait(bar_accfull + 8 * buf, gen & 1, a.status);
                tc_fence_after();
            }
            // A lane owns an accumulator row, but 16-byte stores of 32 lanes to 32 different state rows cost the load/store
            // unit 32 line requests per instruction.  So the warp stages 32 columns of its 32 rows in shared memory (bf16
            // hi and lo, 64 bytes per row, 16-byte pieces XOR-swizzled: conflict-free both ways) and writes them back with
            // four lanes per row: 64 contiguous bytes per row, eight rows per instruction.
            uint8_t* stg = sDrain + (size_t)(warp - W_DRAIN) * (32 * 64 * 2);
            const int wr = lane >> 2, wp = lane & 3;             // write-back: row wr (+ 8 per pass), piece wp
            for (int ui = 0; ui < S.nunit; ++ui) {
                const UInfo& U = sU[S.unit_begin + ui];
                const int c_src = (int)U.c_src, ncols = (int)U.ncols;
                const bool rv = cl < (int)U.ncomp && q < a.K;
                int64_t off = -1;
                if (rv) {
                    const CompS cp = sComp[U.comp_begin + cl];
                    off = a.n_nodes * cp.zoff + (nl * cp.d_dst + cp.o) * (int64_t)cp.ld + cp.koff + (int64_t)q * c_src;
                }
                int64_t roff[4];                                 // state offsets of the four rows this lane writes back
#pragma unroll
                for (int t = 0; t < 4; ++t) roff[t] = __shfl_sync(0xffffffffu, off, 8 * t + wr);
                const uint32_t trow = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * (uint32_t)a.acc_cols + U.tmem_col;
#pragma unroll 1
                for (int cc = 0; cc < ncols; cc += 32) {         // ncols is a multiple of 16, c_src of 8
                    const int sw = (lane >> 1) & 3;
#pragma unroll
                    for (int h2 = 0; h2 < 2; ++h2) {
                        float v[16];
                        if (wrote && cc + 16 * h2 < ncols) {
                            tc_ld16(trow + (uint32_t)(cc + 16 * h2), v);
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] = 0.f;
                        }
                        uint4 h, l;
                        split8(v, h, l);
                        *reinterpret_cast<uint4*>(stg + lane * 64 + (((2 * h2) ^ sw) << 4)) = h;
                        *reinterpret_cast<uint4*>(stg + 2048 + lane * 64 + (((2 * h2) ^ sw) << 4)) = l;
                        split8(v + 8, h, l);
                        *reinterpret_cast<uint4*>(stg + lane * 64 + (((2 * h2 + 1) ^ sw) << 4)) = h;
                        *reinterpret_cast<uint4*>(stg + 2048 + lane * 64 + (((2 * h2 + 1) ^ sw) << 4)) = l;
                    }
                    __syncwarp();
                    const int col = cc + 8 * wp;
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        const int row = 8 * t + wr;
                        if (roff[t] >= 0 && col < c_src) {
                            const int so = row * 64 + ((wp ^ ((row >> 1) & 3)) << 4);
                            *reinterpret_cast<uint4*>(a.zh + roff[t] + col) = *reinterpret_cast<const uint4*>(stg + so);
                            *reinterpret_cast<uint4*>(a.zl + roff[t] + col) = *reinterpret_cast<const uint4*>(stg + 2048 + so);
                        }
                    }
                    __syncwarp();
                }
            }
            if (wrote) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_accfree + 8 * buf);
                ++mi;
            }
        }
    } else if (warp < NBW) {
        // =========================== builder warps ===========================
        // group grp = warp / 4 builds the slabs j = grp, grp + NBG, ... of every batch; its four warps cover the 128 rows
        const int grp = warp >> 2, quarter = warp & 3;
        const int r = quarter * 32 + lane;                    // this thread's accumulator row = TMEM lane
        const int cl = r / KP, q = r - cl * KP;
        const uint32_t ring_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)RING0;
        const int gt = tid & 127;                             // thread index inside the group
        uint32_t it = 0;
        uint32_t par = 0;                // bit s: how often slot s has been used so far, modulo 2
        int st = 0; uint32_t round = 0;
        int cur_set = -1;
        int64_t cx0 = 0, cx1 = 0;
        ItemPos cp_; cp_.init(blockIdx.x, a.n_nodes);        // position of the item whose bounds are in flight
        if ((int64_t)blockIdx.x < total) item_bounds(cp_.nl, nullptr, cx0, cx1);
        for (int64_t item = blockIdx.x; item < total; item += gridDim.x) {
            const int set = cp_.set;
            const TSet S = sSet[set];
            const int64_t seg0 = cx0, seg1 = any_op ? cx1 : cx0;
            cp_.step(gridDim.x, a.n_nodes);
            if (item + gridDim.x < total)       // the next item's bounds, requested one item ahead
                item_bounds(cp_.nl, nullptr, cx0, cx1);
            if (set != cur_set && seg1 > seg0) {     // entry and sparse-term tables of the set
                builder_sync();
                for (int i = tid; i < S.nent; i += NBW * 32) sEnt[i] = a.ents[S.ent_begin + i];
                for (int i = tid; i < S.pad; i += NBW * 32) sNz[i] = a.nz[S.b_items + i];
                builder_sync();
                cur_set = set;
            }
            const SlabW* slabs = sSlab + S.sched_begin;
            for (int64_t b0 = seg0; b0 < seg1; b0 += TB)
            for (int sb = 0; sb < nsub; ++sb, ++it) {
                const int op = has_a1 ? sb : 1;          // which operand pair this sub-batch builds
                mbar_wait(bar_full + 8 * st, round & 1, a.status);
                const float* raw = reinterpret_cast<const float*>(sRing + (size_t)st * stage_bytes + (size_t)2 * a.b_cap);
                const float* sYT = raw + NRAW * TB * KP;
                const float* sVYT = sYT + a.dsh * PS;
                // the two sub-batches of a batch of the dual pass share the coupling values: built with the first one
                const uint32_t mpar = nsub == 2 ? (it >> 1) & 1u : it & 1u;
                float* sM = sM0 + ((size_t)grp * 2 + mpar) * mbuf_floats;
                float* sdM = sdM0 + ((size_t)grp * 2 + mpar) * mbuf_floats;
                // ---- coupling values of this group's own slabs: thread <-> (own slab k, component c, 8 edges)
                const int nown = (S.nslab - grp + NBG - 1) / NBG;
                const bool build_m = nsub == 1 || sb == 0;
#pragma unroll 1
                for (int i = gt; build_m && i < nown * 2 * MC; i += 128) {
                    const int k = i / (2 * MC), c = (i >> 1) & (MC - 1), h = i & 1;
                    const uint32_t bw = slabs[grp + k * NBG].bw;
                    if (c >= (int)(bw >> 24)) continue;
                    const EntS en = sEnt[(int)(bw & 0xffffu) + c * (int)((bw >> 16) & 255u)];
                    float m[8], dm[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) { m[e] = 0.f; dm[e] = 0.f; }
                    for (int kk = en.nz_begin; kk < en.nz_begin + en.nz_count; ++kk) {
                        const NzS t = sNz[kk];
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
                    float* d = sM + (size_t)(k * MC + c) * PS + 8 * h;
                    *reinterpret_cast<float4*>(d) = *reinterpret_cast<const float4*>(m);
                    *reinterpret_cast<float4*>(d + 4) = *reinterpret_cast<const float4*>(m + 4);
                    if (DUAL) {
                        float* dd = sdM + (size_t)(k * MC + c) * PS + 8 * h;
                        *reinterpret_cast<float4*>(dd) = *reinterpret_cast<const float4*>(dm);
                        *reinterpret_cast<float4*>(dd + 4) = *reinterpret_cast<const float4*>(dm + 4);
                    }
                }
                if (build_m) group_sync(grp);
                // ---- this row's radial factors of the 16 edges (rows of padded q read the zeros left at start-up)
                float ph[TB];
#pragma unroll
                for (int e = 0; e < TB; ++e) ph[e] = raw[e * KP + q];
                const float* vph = raw + TB * KP + q;      // DUAL: the direction's factors are read where they are used
                // ---- this group's A slabs of the batch, one slot each.  The stores of a slab stay in flight while the
                // next one is computed: its slot is handed over after that.
                int pend = -1;
                const float* mrow = sM + (size_t)cl * PS;
                const float* dmrow = sdM + (size_t)cl * PS;
#pragma unroll 1
                for (int j = grp; j < S.nslab; j += NBG, mrow += MC * PS, dmrow += MC * PS) {
                    const uint32_t bw = slabs[j].bw;
                    const bool rv = cl < (int)(bw >> 24) && q < a.K;
                    const uint32_t slot = (uint32_t)j % NSLOT, use = (uint32_t)j / NSLOT;
                    mbar_wait(bar_slotfree + 8 * slot, ((par >> slot) ^ use) & 1u, a.status);
                    tc_fence_after();
                    uint32_t hl[16];                 // columns 0..7: hi pairs, 8..15: lo pairs
                    uint32_t* const hi = hl;
                    uint32_t* const lo = hl + 8;
                    if (rv) {
#pragma unroll
                        for (int e4 = 0; e4 < TB; e4 += 4) {
                            const float4 mv = *reinterpret_cast<const float4*>(mrow + e4);
                            float p0, p1, p2, p3;
                            if (DUAL && op == 0) {
                                const float4 dv = *reinterpret_cast<const float4*>(dmrow + e4);
                                p0 = fmaf(vph[e4 * KP], mv.x, ph[e4] * dv.x);
                                p1 = fmaf(vph[(e4 + 1) * KP], mv.y, ph[e4 + 1] * dv.y);
                                p2 = fmaf(vph[(e4 + 2) * KP], mv.z, ph[e4 + 2] * dv.z);
                                p3 = fmaf(vph[(e4 + 3) * KP], mv.w, ph[e4 + 3] * dv.w);
                            } else {
                                p0 = ph[e4] * mv.x; p1 = ph[e4 + 1] * mv.y; p2 = ph[e4 + 2] * mv.z; p3 = ph[e4 + 3] * mv.w;
                            }
                            split2(p0, p1, hi[e4 >> 1], lo[e4 >> 1]);
                            split2(p2, p3, hi[(e4 >> 1) + 1], lo[(e4 >> 1) + 1]);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) hl[i] = 0u;
                    }
                    __syncwarp();
                    if (pend >= 0) {
                        tc_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) count_add(fill0 + 4 * (uint32_t)pend);
                    }
                    tc_st16(ring_row + slot * 16u, hl);
                    pend = (int)slot;
                }
                if (pend >= 0) {
                    tc_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) count_add(fill0 + 4 * (uint32_t)pend);
                }
                par ^= (uint32_t)S.oddmask;
                if (++st == NS) { st = 0; ++round; }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS) : "memory");
    }
}

// shared bytes of the kernel for given region sizes
int smem_need(int KP, bool dual, int dsh, int ns, int b_cap, int max_ent, int n_units, int n_sets, int n_comps, int max_nz, int n_slab, int max_own) {
    const int nop = dual ? 2 : 1;     // M comes with its direction in the dual stream
    const int stage = 2 * b_cap + ((raw_floats(KP, dual, dsh) * 4 + 1023) & ~1023);
    size_t meta = (size_t)NBG * 2 * nop * max_own * (128 / KP) * PS;     // coupling values of a group's own slabs, double buffered
    meta = (meta + 1) & ~size_t(1);
    // tables: units (and at most as many blocks), sets, components, entries and sparse terms of one set, slabs
    const int tables = n_units * (int)(sizeof(UInfo) + sizeof(TBlk)) + n_sets * (int)sizeof(TSet) + n_comps * (int)sizeof(CompS) +
                       max_ent * (int)sizeof(EntS) + max_nz * (int)sizeof(NzS) + n_slab * (int)sizeof(SlabW) + 16;
    return 1024 + ns * stage + DRAIN_BYTES + (int)(meta * 4) + (2 * MAXNS + 2 * NSLOT + 4 + 4) * 8 + tables;
}

}  // namespace

// Units, passes ("sets") and entries of one direction for the plain ([0]) and the dual ([1]) stream.
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
        // candidate units: accumulator tiles of up to 128 / KP components of one source block, split evenly
        struct Cand { int blk, c0, nc; };
        std::vector<Cand> cands;
        const int comps_per_tile = 128 / KP;
        for (size_t b = 0; b < blocks.size(); ++b) {
            const int nc = (int)blocks[b].comps.size();
            const int ntile = (nc + comps_per_tile - 1) / comps_per_tile;
            const int per = (nc + ntile - 1) / ntile;
            for (int c0 = 0; c0 < nc; c0 += per) cands.push_back(Cand{(int)b, c0, std::min(per, nc - c0)});
        }
        auto blk_b = [&](int b) { return blocks[b].d_src * 2048 * ((blocks[b].c_src + 63) / 64); };
        auto ncols = [&](int b) { return (blocks[b].c_src + 15) & ~15; };
        auto cols32 = [&](int b) { return (ncols(b) + 31) & ~31; };
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
        int n_comps_total = 0, n_slab = 0;
        for (const Blk& b : blocks) n_comps_total += (int)b.comps.size();
        for (const Cand& c : cands) n_slab += blocks[c.blk].d_src;        // one slab per (tile, s)
        // greedy packing of consecutive units into passes: the accumulator tiles of a pass fit one of the two TMEM
        // buffers and its operand regions fit shared memory with at least two ring stages
        const int budget = 227 * 1024;
        // Two accumulator buffers (the drain of one receiver overlaps the MMAs of the next) when at least two of the
        // widest tiles fit half of the accumulator columns; else one buffer over all of them: with 128-column tiles a
        // half holds a single tile, a set then has one to nine slabs per batch and most builder groups idle, which
        // costs more than the wait for the drain (measured: 128-wide profiles 10 - 17 % faster with one buffer, 32- and
        // 64-wide ones 2 - 10 % slower).
        int widest = 0;
        for (const Cand& c : cands) widest = std::max(widest, cols32(c.blk));
        T.nbuf = 2 * widest > ACC_BUDGET ? 1 : 2;
        const int acc_budget = T.nbuf == 2 ? ACC_BUDGET : RING0;
        bool fits = true;
        size_t i = 0;
        while (i < cands.size() && fits) {
            int b_bytes = 0, cols = 0, nent = 0, nnz = 0, slabs_in = 0;
            std::vector<int> set_blks;
            size_t j = i;
            for (; j < cands.size(); ++j) {
                const Cand& c = cands[j];
                const bool new_blk = std::find(set_blks.begin(), set_blks.end(), c.blk) == set_blks.end();
                const int b2 = b_bytes + (new_blk ? blk_b(c.blk) : 0);
                const int c2 = cols + cols32(c.blk), e2 = nent + c.nc * blocks[c.blk].d_src, n2 = nnz + cand_nz(c);
                // the kernel sizes its regions by the maxima over all passes
                const int bcap = std::max(T.b_cap, (b2 + 1023) & ~1023);
                const int own2 = (slabs_in + blocks[c.blk].d_src + NBG - 1) / NBG;
                const int need = smem_need(KP, dual, p->dim_sh, 2, bcap, std::max(T.max_ent, e2), (int)cands.size(), (int)cands.size(),
                                           n_comps_total, std::max(T.max_nz, n2), n_slab, std::max(T.max_units, own2));
                if (need > budget || c2 > acc_budget) break;
                b_bytes = b2; cols = c2; nent = e2; nnz = n2; slabs_in += blocks[c.blk].d_src;
                if (new_blk) set_blks.push_back(c.blk);
            }
            if (j == i) { fits = false; break; }
            TSet S{};
            S.unit_begin = (int)T.units.size(); S.blk_begin = (int)T.blks.size(); S.ent_begin = (int)T.ents.size();
            int b_off = 0, col = 0, ent = 0;
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
                    bi = (int)T.blks.size();
                    T.blks.push_back(tb);
                    local_blk.push_back(c.blk);
                }
                TUnit U{};
                U.blk = bi; U.comp_begin = (int)T.comps.size(); U.ncomp = c.nc;
                U.a_off = ent;                 // first entry of the unit inside the pass: entry = a_off + cl * d_src + s
                U.slab_stride = 0; U.tmem_col = col;
                for (int cl = 0; cl < c.nc; ++cl) {
                    const SComp& cp = Bk.comps[c.c0 + cl];
                    T.comps.push_back(cp);
                    for (int s = 0; s < Bk.d_src; ++s) T.ents.push_back(TEnt{cp.tab0 + s * cp.tstride, cp.sh_off, 0, 0});
                }
                ent += c.nc * Bk.d_src;
                col += cols32(c.blk);
                T.units.push_back(U);
            }
            S.nunit = (int)T.units.size() - S.unit_begin; S.nblk = (int)T.blks.size() - S.blk_begin;
            S.nent = (int)T.ents.size() - S.ent_begin;
            // build order of the pass's slabs: tile after tile in turn (s = 0 of every tile, then s = 1, ...), so that
            // the builder groups (slab j mod NBG) and the MMA threads (tile mod NMW) find work at the same rate
            S.sched_begin = (int)T.slabs.size() / 2;
            std::vector<uint32_t> order;      // (tile << 8) | s
            for (int sdx = 0, more = 1; more; ++sdx) {
                more = 0;
                for (int u = 0; u < S.nunit; ++u)
                    if (sdx < T.blks[T.units[S.unit_begin + u].blk].d_src) { order.push_back(((uint32_t)u << 8) | (uint32_t)sdx); more = 1; }
            }
            S.nslab = (int)order.size();
            S.mfirst = 0x00ffffff;
            S.oddmask = 0;
            for (int sl = 0; sl < NSLOT; ++sl)
                if (((S.nslab - sl + NSLOT - 1) / NSLOT) & 1) S.oddmask |= 1 << sl;      // slots used an odd number of times per batch
            for (int j = 0; j < S.nslab; ++j) {
                const int u = (int)(order[j] >> 8), sdx = (int)(order[j] & 255u);
                const TUnit& Uu = T.units[S.unit_begin + u];
                const int d = T.blks[Uu.blk].d_src;
                uint32_t next = 255;
                for (int k = j + 1; k < S.nslab && next == 255; ++k)
                    if ((int)(order[k] >> 8) % NMW == u % NMW) next = (uint32_t)k;
                T.slabs.push_back((uint32_t)(Uu.a_off + sdx) | ((uint32_t)d << 16) | ((uint32_t)Uu.ncomp << 24));
                T.slabs.push_back((uint32_t)u | ((uint32_t)sdx << 8) | (next << 16));
                const int t = u % NMW;
                if (((S.mfirst >> (8 * t)) & 255) == 255) S.mfirst = (S.mfirst & ~(255 << (8 * t))) | (j << (8 * t));
            }
            if (S.nslab > 254) fits = false;
            T.max_units = std::max(T.max_units, (S.nslab + NBG - 1) / NBG);      // own slabs of a builder group at most
            T.sets.push_back(S);
            T.b_cap = std::max(T.b_cap, (b_off + 1023) & ~1023);
            T.max_ent = std::max(T.max_ent, S.nent);
            T.max_nz = std::max(T.max_nz, nnz);
            T.acc_cols = std::max(T.acc_cols, col);
            i = j;
        }
        if (!fits) { T = TcSets{}; continue; }
        // as many ring stages as shared memory holds (the loaders run that many batches ahead)
        int ns = 2;
        while (ns < MAXNS && smem_need(KP, dual, p->dim_sh, ns + 1, T.b_cap, T.max_ent, (int)cands.size(), (int)cands.size(),
                                       n_comps_total, T.max_nz, n_slab, T.max_units) <= budget) ++ns;
        T.ctas_per_sm = 1;
        T.ring_stages = ns;
        T.tmem_cols = TMEM_COLS;
        T.smem_bytes = smem_need(KP, dual, p->dim_sh, ns, T.b_cap, T.max_ent, (int)cands.size(), (int)cands.size(), n_comps_total, T.max_nz, n_slab, T.max_units);
        // shared-memory images of the tables
        for (TSet& S : T.sets) {
            S.b_items = (int)T.nz.size();
            for (int j = 0; j < S.nent; ++j) {
                const TEnt& E = T.ents[S.ent_begin + j];
                EntS es{0, (int)T.nz.size() - S.b_items, p->tab_ptr[E.tab + 1] - p->tab_ptr[E.tab], 0};
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
    a.rvec = ss.rvec; a.geo_rc = ss.geo_rc; a.geo_basis = ss.geo_basis; a.geo_p = ss.geo_p; a.geo_inline = 0;
    a.oseg = ss.oseg ? ss.oseg + node0 : nullptr;
    a.vrvec = dual ? ss.vrvec : nullptr;
    a.zh = (__nv_bfloat16*)zh; a.zl = (__nv_bfloat16*)zl;
    a.K = p->K; a.dsh = p->dim_sh; a.C_src = dir.C_src; a.nsets = (int)T.sets.size();
    a.b_cap = T.b_cap; a.max_ent = T.max_ent; a.acc_cols = T.acc_cols; a.ns = T.ring_stages; a.nbuf = T.nbuf;
    a.n_units = (int)T.units.size(); a.n_blks = (int)T.blks.size(); a.n_comps = (int)T.comps.size(); a.max_nz = T.max_nz;
    a.slabs = T.d_slabs; a.n_slab = (int)T.slabs.size() / 2; a.max_own = T.max_units;
    a.status = status;
    const bool k8 = p->K <= 8;
    void (*kern)(const TcArgs) = k8 ? (dual ? k_stream_tc<8, true> : k_stream_tc<8, false>)
                                    : (dual ? k_stream_tc<16, true> : k_stream_tc<16, false>);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, T.smem_bytes);
    if (e != cudaSuccess) return e;
    const int64_t total = n_nodes * a.nsets;
    const int grid = (int)std::min<int64_t>(total, (int64_t)148);
    KernelTimer kt(K_STATE, s);
    kern<<<grid, TT, T.smem_bytes, s>>>(a);
    count_launch();
    return cudaGetLastError();
}

}  // namespace sobek
