// C-ABI entry points: argument checks, workspace carving and the launch schedules of
// forward, backward and double backward.  Everything here only enqueues work on the
// caller's stream.
#include <algorithm>

#include "internal.h"

using namespace sobek;

namespace {

inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

struct Workspace {
    int* status;
    // bf16 (hi, lo) copies of R as tensor-core operands
    uint16_t *fNKh, *fNKl;    // receiver direction, [w][k]   (y = Z Rp)
    uint16_t *fKNh, *fKNl;    // receiver direction, [k][w]   (Zbar = gy Rp^T)
    uint16_t *tNKh, *tNKl;    // sender direction,   [u][k']  (gx = V Rt)
    uint16_t *vfNKh, *vfNKl, *vfKNh, *vfKNl, *vtNKh, *vtNKl;   // the same for vR
    uint16_t *fFKh, *fFKl, *tFKh, *tFKl, *vfFKh, *vfFKl, *vtFKh, *vtFKl;   // stage-ordered copies (fused kernels)
    bool fused_f, fused_t;    // fused kernels usable for the receiver / sender direction
    float* gRp;               // fp32 accumulator of the R adjoint, packed [k][w] per group
    float* part;              // split-K partial results of the weight-adjoint GEMM
    int splits;
    float* zbar;              // fp32 adjoint state Zbar of one chunk (input of the edge pass)
    uint16_t *zbh, *zbl;      // bf16 (hi, lo) node state Z / dZ / V of one chunk
    uint16_t *gbh, *gbl;      // bf16 (hi, lo) rows of the chunk's output adjoint
    // bf16 (hi, lo) copies of x, gy and vx, [N][C] each: the gathered operand of the tensor-core stream
    uint16_t *xsh, *xsl, *gsh, *gsl, *vsh, *vsl;
    uint16_t *zqh, *zql;      // bf16 (hi, lo) adjoint state of one chunk (input of the tensor-core edge pass)
    int4 *oseg_r, *oseg_s;    // processing order of the nodes of every chunk, receiver / sender view (launch_chunk_order)
    // mul_ir plans: ir_mul copies of the node feature arrays of a call (inputs x, gy, vx; outputs on C_y, on C_x)
    float *lx, *lgy, *lvx, *ly, *lgx;
    int64_t chunk;
    size_t bytes;
};

constexpr int64_t kOrderMinChunk = 4 * 148;   // nodes per chunk from which the processing order is balanced
constexpr int kOrderPeriod = 148;             // persistent CTAs of the edge kernels (one per SM)

Workspace carve(const sobek_plan* p, int64_t N, int order, void* ws) {
    Workspace w{};
    char* c = (char*)ws;
    size_t off = kHeaderBytes;
    auto take = [&](size_t bytes) { char* r = c + off; off += align256(bytes); return r; };
    w.status = (int*)c;
    w.fused_f = fused_supported(p, p->fwd);
    w.fused_t = fused_supported(p, p->tr);
    if (w.fused_f) { w.fFKh = (uint16_t*)take(p->fwd.fk_elems * 2); w.fFKl = (uint16_t*)take(p->fwd.fk_elems * 2); }
    if (w.fused_f && order >= 2) { w.vfFKh = (uint16_t*)take(p->fwd.fk_elems * 2); w.vfFKl = (uint16_t*)take(p->fwd.fk_elems * 2); }
    if (w.fused_t && order >= 1) { w.tFKh = (uint16_t*)take(p->tr.fk_elems * 2); w.tFKl = (uint16_t*)take(p->tr.fk_elems * 2); }
    if (w.fused_t && order >= 2) { w.vtFKh = (uint16_t*)take(p->tr.fk_elems * 2); w.vtFKl = (uint16_t*)take(p->tr.fk_elems * 2); }
    if (order == 0 && w.fused_f) {   // the forward needs nothing else: the state stays on chip
        w.chunk = 0;
        if (p->mul_ir) {
            w.lx = (float*)take((size_t)std::max<int64_t>(N, 0) * (size_t)p->C_x * 4);
            w.ly = (float*)take((size_t)std::max<int64_t>(N, 0) * (size_t)p->C_y * 4);
        }
        w.bytes = off;
        return w;
    }
    const bool gemm = !p->uvu;   // the channelwise mode has no GEMM, hence no operand copies of R
    if (gemm) { w.fNKh = (uint16_t*)take(p->fwd.nk_elems * 2); w.fNKl = (uint16_t*)take(p->fwd.nk_elems * 2); }
    if (order >= 1) {
        if (gemm) {
            w.fKNh = (uint16_t*)take(p->fwd.kn_elems * 2); w.fKNl = (uint16_t*)take(p->fwd.kn_elems * 2);
            w.tNKh = (uint16_t*)take(p->tr.nk_elems * 2); w.tNKl = (uint16_t*)take(p->tr.nk_elems * 2);
        }
        w.gRp = (float*)take((size_t)p->K * (size_t)p->N_w * 4);
        w.splits = (int)std::max<size_t>(1, std::min<size_t>(gemm ? kMaxSplits : kMaxSplitsUvu,
                                                             kPartBudgetBytes / ((size_t)p->K * (size_t)p->N_w * 4)));
        w.part = (float*)take((size_t)w.splits * (size_t)p->K * (size_t)p->N_w * 4);
    }
    if (order >= 2 && gemm) {
        w.vfNKh = (uint16_t*)take(p->fwd.nk_elems * 2); w.vfNKl = (uint16_t*)take(p->fwd.nk_elems * 2);
        w.vfKNh = (uint16_t*)take(p->fwd.kn_elems * 2); w.vfKNl = (uint16_t*)take(p->fwd.kn_elems * 2);
        w.vtNKh = (uint16_t*)take(p->tr.nk_elems * 2); w.vtNKl = (uint16_t*)take(p->tr.nk_elems * 2);
    }
    w.chunk = chunk_nodes(p, N, order);
    int64_t zb = p->fwd.zb_elems;
    if (order >= 1) zb = std::max(zb, p->tr.zb_elems);
    w.zbh = (uint16_t*)take((size_t)w.chunk * (size_t)zb * 2);
    w.zbl = (uint16_t*)take((size_t)w.chunk * (size_t)zb * 2);
    if (order >= 1) {
        if (gemm) {
            w.gbh = (uint16_t*)take((size_t)w.chunk * (size_t)p->fwd.gb_elems * 2);
            w.gbl = (uint16_t*)take((size_t)w.chunk * (size_t)p->fwd.gb_elems * 2);
        }
        if (p->use_tc_edge && p->fwd.etc[0].ok) {
            // the adjoint state of a chunk is made after the chunk's state has been consumed (by the mixing and
            // weight-adjoint contractions): the two share one buffer
            w.zqh = w.zbh;
            w.zql = w.zbl;
        } else {
            w.zbar = (float*)take((size_t)w.chunk * (size_t)p->fwd.state_floats * 4);
        }
    }
    if (p->use_tc_stream || (p->use_tc_edge && p->fwd.etc[0].ok)) {
        const size_t nx = (size_t)std::max<int64_t>(N, 0) * (size_t)p->C_x * 2, ny = (size_t)std::max<int64_t>(N, 0) * (size_t)p->C_y * 2;
        if (p->fwd.tc[0].ok || (order >= 2 && p->fwd.tc[1].ok) || (order >= 1 && w.zqh)) { w.xsh = (uint16_t*)take(nx); w.xsl = (uint16_t*)take(nx); }
        if (order >= 1 && (p->tr.tc[0].ok || (order >= 2 && p->tr.tc[1].ok))) { w.gsh = (uint16_t*)take(ny); w.gsl = (uint16_t*)take(ny); }
        if (order >= 2 && (p->fwd.tc[1].ok || (w.zqh && p->fwd.etc[1].ok))) { w.vsh = (uint16_t*)take(nx); w.vsl = (uint16_t*)take(nx); }
        // load balance of the persistent edge kernels: only where a CTA takes several nodes of a chunk
        if (w.chunk >= kOrderMinChunk && N >= kOrderMinChunk) {
            w.oseg_r = (int4*)take((size_t)N * sizeof(int4));
            if (order >= 1) w.oseg_s = (int4*)take((size_t)N * sizeof(int4));
        }
    }
    if (p->mul_ir) {
        const size_t nx = (size_t)std::max<int64_t>(N, 0) * (size_t)p->C_x * 4, ny = (size_t)std::max<int64_t>(N, 0) * (size_t)p->C_y * 4;
        w.lx = (float*)take(nx);
        w.ly = (float*)take(ny);            // y (order 0), ggy (order 2)
        if (order >= 1) { w.lgy = (float*)take(ny); w.lgx = (float*)take(nx); }
        if (order >= 2) w.lvx = (float*)take(nx);
    }
    w.bytes = off;
    return w;
}

// whole feature matrix [N][C] -> bf16 (hi, lo)
cudaError_t split_features(const float* src, int64_t N, int C, uint16_t* h, uint16_t* l, cudaStream_t s) {
    return launch_split(src, C, 0, 1, N, C, C, h, l, s);
}

// several of them in one launch
struct FeatureSplits {
    SplitJob j[kMaxSplitJobs];
    int n = 0;
    void add(const float* src, int64_t N, int C, uint16_t* h, uint16_t* l) { j[n++] = SplitJob{src, C, 0, 1, N, C, C, h, l}; }
    cudaError_t flush(cudaStream_t s) { const int k = n; n = 0; return launch_split_jobs(j, k, s); }
};

int check_common(const sobek_plan* p, const sobek_graph* g, void* ws, size_t ws_bytes, int order) {
    if (!p || !g) return SOBEK_ERR_INVALID_ARG;
    if (g->N < 0 || g->E < 0) return SOBEK_ERR_INVALID_ARG;
    if (g->N >= (int64_t(1) << 31) || g->E >= (int64_t(1) << 31)) return SOBEK_ERR_UNSUPPORTED;
    if (g->N > 0 && !g->row_ptr) return SOBEK_ERR_INVALID_ARG;
    if (g->E > 0 && !g->col) return SOBEK_ERR_INVALID_ARG;
    if (p->device < 0) return SOBEK_ERR_CUDA;
    if (!ws || ((uintptr_t)ws & 255)) return SOBEK_ERR_WORKSPACE;
    if (ws_bytes < sobek_workspace_bytes(p, g->N, g->E, order)) return SOBEK_ERR_WORKSPACE;
    return SOBEK_OK;
}

// every floating-point array argument must start on a 16-byte boundary (NULL passes: "not given")
template <class... P>
bool aligned16(P... ptrs) {
    uintptr_t m = 0;
    ((m |= (uintptr_t)ptrs), ...);
    return (m & 15) == 0;
}

#define CK(expr)                                              \
    do {                                                      \
        cudaError_t e__ = (expr);                             \
        if (e__ != cudaSuccess) {                             \
            (void)cudaGetLastError();                         \
            return SOBEK_ERR_CUDA;                            \
        }                                                     \
    } while (0)

EdgeView receiver_view(const sobek_graph* g) {
    return EdgeView{g->row_ptr, nullptr, g->col, g->row_ptr, g->N, g->E, 0};
}
EdgeView sender_view(const sobek_graph* g) {
    return EdgeView{g->src_ptr, g->src_perm, g->col, g->row_ptr, g->N, g->E, 1, g->src_recv};
}

bool has_uncovered(const Direction& d) {
    for (const DGroup& G : d.groups)
        if (G.path_end == G.path_begin) return true;
    return false;
}


// rows (node, o) of the chunk's output adjoint -> bf16 (hi, lo), group by group
cudaError_t split_adjoint(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const float* gdst,
                          uint16_t* gh, uint16_t* gl, cudaStream_t s) {
    SplitJob jobs[kMaxSplitJobs];
    int nj = 0;
    for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
        const DGroup& G = dir.groups[gi];
        if (G.path_end == G.path_begin) continue;
        jobs[nj++] = SplitJob{gdst + n0 * dir.C_dst + G.dst_off, dir.C_dst, G.c_dst, G.d_dst, nn * G.d_dst, G.c_dst, dir.kn_ld[gi],
                              gh + nn * dir.gb_off[gi], gl + nn * dir.gb_off[gi]};
        if (nj == kMaxSplitJobs) {
            cudaError_t e = launch_split_jobs(jobs, nj, s);
            if (e != cudaSuccess) return e;
            nj = 0;
        }
    }
    return launch_split_jobs(jobs, nj, s);
}

// dst_g (+)= Z_g * Rp_g        (Eq. receiver_matrix_product)
cudaError_t mix_tc(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const uint16_t* zh,
                   const uint16_t* zl, const uint16_t* nkh, const uint16_t* nkl, float* dst, int accumulate,
                   int* status, cudaStream_t s) {
    GemmBatch gb;                 // the groups' products run as one launch
    for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
        const DGroup& G = dir.groups[gi];
        if (G.path_end == G.path_begin) continue;
        cudaError_t e = gemm_tc_add(gb, zh + nn * dir.zb_off[gi], zl + nn * dir.zb_off[gi], dir.nk_ld[gi],
                                    nkh + dir.nk_off[gi], nkl + dir.nk_off[gi], dir.nk_ld[gi],
                                    dst + n0 * dir.C_dst + G.dst_off, dir.C_dst, G.c_dst, G.d_dst,
                                    nn * G.d_dst, G.c_dst, G.D, accumulate, 0, status, s, 1, 0, nullptr, nullptr, p->gemm_passes);
        if (e != cudaSuccess) return e;
    }
    return gemm_tc_flush(gb, s, p);
}

// Zbar_g = gy_g * Rp_g^T       (Eq. receiver_adjoint)
// With zqh / zql the result is written as bf16 (hi, lo) rows in the layout of the stream's state instead.
cudaError_t state_adjoint_tc(const sobek_plan* p, const Direction& dir, int64_t nn, const uint16_t* gh,
                             const uint16_t* gl, const uint16_t* knh, const uint16_t* knl, float* Zbar, int* status,
                             cudaStream_t s, uint16_t* zqh = nullptr, uint16_t* zql = nullptr) {
    GemmBatch gb;
    for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
        const DGroup& G = dir.groups[gi];
        if (G.path_end == G.path_begin) continue;
        cudaError_t e;
        if (zqh)
            e = gemm_tc_add(gb, gh + nn * dir.gb_off[gi], gl + nn * dir.gb_off[gi], dir.kn_ld[gi],
                            knh + dir.kn_off[gi], knl + dir.kn_off[gi], dir.kn_ld[gi], nullptr, dir.nk_ld[gi], 0, 1,
                            nn * G.d_dst, G.D, G.c_dst, 0, 0, status, s, 1, 0, zqh + nn * dir.zb_off[gi],
                            zql + nn * dir.zb_off[gi], p->gemm_passes);
        else
            e = gemm_tc_add(gb, gh + nn * dir.gb_off[gi], gl + nn * dir.gb_off[gi], dir.kn_ld[gi],
                            knh + dir.kn_off[gi], knl + dir.kn_off[gi], dir.kn_ld[gi],
                            Zbar + nn * G.z_off, G.D, 0, 1, nn * G.d_dst, G.D, G.c_dst, 0, 0, status, s, 1, 0, nullptr, nullptr,
                            p->gemm_passes);
        if (e != cudaSuccess) return e;
    }
    return gemm_tc_flush(gb, s, p);
}

// gRp_g += Z_g^T * gy_g        (Eq. receiver_adjoint).  The contraction runs over every (node, component)
// row of the chunk; it is cut into `splits` pieces that run concurrently and are summed in a fixed order.
cudaError_t weight_grad_tc(const sobek_plan* p, const Direction& dir, int64_t nn, const uint16_t* zh,
                           const uint16_t* zl, const uint16_t* gh, const uint16_t* gl, float* gRp, float* part,
                           int splits, int* status, cudaStream_t s0) {
    const int64_t KN = (int64_t)p->K * p->N_w;
    GemmBatch gb;
    for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
        const DGroup& G = dir.groups[gi];
        if (G.path_end == G.path_begin) continue;
        const int64_t kblocks = (nn * G.d_dst + 63) / 64;
        const int sp = (int)std::max<int64_t>(1, std::min<int64_t>(splits, kblocks));
        cudaError_t e = gemm_tc_add(gb, zh + nn * dir.zb_off[gi], zl + nn * dir.zb_off[gi], dir.nk_ld[gi],
                                    gh + nn * dir.gb_off[gi], gl + nn * dir.gb_off[gi], dir.kn_ld[gi],
                                    part + G.rp_off, G.c_dst, 0, 1, G.D, G.c_dst, nn * G.d_dst, 0, 1, status, s0,
                                    sp, KN, nullptr, nullptr, p->gemm_passes);
        if (e != cudaSuccess) return e;
    }
    cudaError_t e = gemm_tc_flush(gb, s0, p);
    if (e != cudaSuccess) return e;
    // the pieces of every group, summed in a fixed order: one launch over the groups' column ranges
    ReduceRange rr[kMaxReduceRanges];
    int nr = 0;
    for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
        const DGroup& G = dir.groups[gi];
        if (G.path_end == G.path_begin) continue;
        const int64_t kblocks = (nn * G.d_dst + 63) / 64;
        rr[nr++] = ReduceRange{G.rp_off, (int64_t)G.D * G.c_dst, (int)std::max<int64_t>(1, std::min<int64_t>(splits, kblocks))};
        if (nr == kMaxReduceRanges) {
            e = launch_reduce_ranges(gRp, part, KN, rr, nr, s0);
            if (e != cudaSuccess) return e;
            nr = 0;
        }
    }
    return launch_reduce_ranges(gRp, part, KN, rr, nr, s0);
}

// ---- the node-side steps in either multiplicity mode: tensor-core GEMMs on the packed copies of R (uvw), or
// the elementwise kernels on R itself (uvu, Eq. uvu_connection) --------------------------------------------
cudaError_t pack_R(const sobek_plan* p, const Direction& dir, int transposed, int n_major, const float* R, void* hi,
                   void* lo, cudaStream_t s) {
    return p->uvu ? cudaSuccess : launch_pack_R_bf16(p, dir, transposed, n_major, R, hi, lo, s);
}
cudaError_t split_gy(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const float* gdst,
                     uint16_t* gh, uint16_t* gl, cudaStream_t s) {
    return p->uvu ? cudaSuccess : split_adjoint(p, dir, n0, nn, gdst, gh, gl, s);
}
cudaError_t mix(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const uint16_t* zh,
                const uint16_t* zl, const uint16_t* nkh, const uint16_t* nkl, const float* Rraw, float* dst,
                int accumulate, int* status, cudaStream_t s) {
    if (p->uvu) return launch_uvu_mix(p, dir, n0, nn, zh, zl, Rraw, dst, accumulate, s);
    return mix_tc(p, dir, n0, nn, zh, zl, nkh, nkl, dst, accumulate, status, s);
}
cudaError_t state_adjoint(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const uint16_t* gh,
                          const uint16_t* gl, const uint16_t* knh, const uint16_t* knl, const float* gy,
                          const float* Rraw, float* Zbar, int* status, cudaStream_t s, uint16_t* zqh = nullptr,
                          uint16_t* zql = nullptr) {
    if (p->uvu) return launch_uvu_zbar(p, dir, n0, nn, gy, Rraw, Zbar, zqh, zql, s);
    return state_adjoint_tc(p, dir, nn, gh, gl, knh, knl, Zbar, status, s, zqh, zql);
}
cudaError_t weight_grad(const sobek_plan* p, const Direction& dir, int64_t n0, int64_t nn, const uint16_t* zh,
                        const uint16_t* zl, const uint16_t* gh, const uint16_t* gl, const float* gy, float* gRp,
                        float* part, int splits, int* status, cudaStream_t s) {
    if (p->uvu) return launch_uvu_wgrad(p, dir, n0, nn, zh, zl, gy, gRp, part, splits, s);
    return weight_grad_tc(p, dir, nn, zh, zl, gh, gl, gRp, part, splits, status, s);
}
// the accumulated weight adjoint -> the caller's [K, N_w] array (already in that layout in the uvu mode)
cudaError_t unpack_R(const sobek_plan* p, const Direction& dir, const float* Rp, float* R, cudaStream_t s) {
    if (p->uvu) return cudaMemcpyAsync(R, Rp, (size_t)p->K * (size_t)p->N_w * 4, cudaMemcpyDeviceToDevice, s);
    return launch_unpack_R(p, dir, Rp, R, s);
}

}  // namespace

extern "C" size_t sobek_workspace_bytes(const sobek_plan* p, int64_t N, int64_t E, int order) {
    (void)E;   // by construction: nothing edge-sized is ever held
    if (!p || order < 0 || order > 2 || N < 0) return 0;
    return carve(p, N, order, nullptr).bytes;
}

extern "C" size_t sobek_graph_prepare_bytes(int64_t N, int64_t E) {
    if (N < 0 || E < 0) return 0;
    return graph_prepare_bytes(N, E);
}

extern "C" int sobek_graph_prepare(int64_t N, int64_t E, const int64_t* row_ptr, const int32_t* col,
                                   int64_t* src_ptr, int32_t* src_perm, void* ws, size_t ws_bytes,
                                   void* stream) {
    return graph_prepare(N, E, row_ptr, col, src_ptr, src_perm, ws, ws_bytes, (cudaStream_t)stream);
}

extern "C" int sobek_graph_receivers(int64_t N, int64_t E, const int64_t* row_ptr, const int32_t* src_perm,
                                     int32_t* src_recv, void* stream) {
    return graph_receivers(N, E, row_ptr, src_perm, src_recv, (cudaStream_t)stream);
}

namespace {
// Geometry mode (Y and phi recomputed from edge vectors inside the edge kernels) exists in the tensor-core edge
// kernels only: the plan must run them in both directions, unfused, in the ir_mul layout, with l_max <= 4.
bool geo_supported(const sobek_plan* p, const Workspace& w, int order) {
    if (!p->use_tc_stream || !p->fwd.tc[0].ok || !w.xsh || w.fused_f || p->mul_ir || p->dim_sh > 25) return false;
    return order == 0 || (p->tr.tc[0].ok && p->fwd.etc[0].ok && w.gsh && w.zqh && !w.fused_t);
}
// `order` is the workspace layout to use (0, or 1 when the state is to be found by a following backward call);
// *retained is set to 1 when the state of every receiver is left in the workspace (one chunk, state schedule)
int conv_fwd_core(const sobek_plan* p, const sobek_graph* g, const float* x, const float* Y,
                  const float* phi, const float* R, float* y, void* ws, size_t ws_bytes,
                  void* stream, int order = 0, int* retained = nullptr, const SplitSrc* geo = nullptr) {
    if (retained) *retained = 0;
    int rc = check_common(p, g, ws, ws_bytes, order);
    if (rc) return rc;
    if (!y || !R || (g->N > 0 && !x) || (g->E > 0 && !geo && (!Y || !phi))) return SOBEK_ERR_INVALID_ARG;
    if (!aligned16(x, Y, phi, R, y)) return SOBEK_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w = carve(p, g->N, order, ws);
    if (geo && !geo_supported(p, w, 0)) return SOBEK_ERR_UNSUPPORTED;
    CK(cudaMemsetAsync(w.status, 0, kHeaderBytes, s));
    if (g->N == 0) return SOBEK_OK;
    if (g->E == 0 || has_uncovered(p->fwd)) CK(launch_fill_zero(y, g->N * (int64_t)p->C_y, s));
    if (g->E == 0) return SOBEK_OK;
    const EdgeView rv = receiver_view(g);
    if (p->uvu && p->ud.ok && !p->uvu_state && !geo && order == 0) {
        // channelwise mode, uniform natural-parity profile: the direct kernel (no state, no node-side pass)
        CK(launch_uvu_direct(p, rv, 0, x, Y, phi, R, y, w.status, s));
        return SOBEK_OK;
    }
    if (w.fused_f) {
        CK(launch_pack_R_fused(p, p->fwd, 0, R, w.fFKh, w.fFKl, s));
        CK(launch_fused(p, p->fwd, rv, x, nullptr, Y, nullptr, phi, nullptr, 0, w.fFKh, w.fFKl, y, 0, w.status, s));
        return SOBEK_OK;
    }
    CK(pack_R(p, p->fwd, 0, 1, R, w.fNKh, w.fNKl, s));
    SplitSrc xs{};
    if (geo) xs = *geo;
    if (w.oseg_r) { CK(launch_chunk_order(rv, w.chunk, kOrderPeriod, w.oseg_r, w.status, s)); xs.oseg = w.oseg_r; }
    if (w.xsh) { CK(split_features(x, g->N, p->C_x, w.xsh, w.xsl, s)); xs.h = w.xsh; xs.l = w.xsl; }
    for (int64_t n0 = 0; n0 < g->N; n0 += w.chunk) {
        const int64_t nn = std::min(w.chunk, g->N - n0);
        CK(launch_stream(p, p->fwd, rv, n0, nn, x, nullptr, xs, Y, nullptr, phi, nullptr, 0, w.zbh, w.zbl, w.status, s));
        CK(mix(p, p->fwd, n0, nn, w.zbh, w.zbl, w.fNKh, w.fNKl, R, y, 0, w.status, s));
    }
    if (retained && w.chunk >= g->N) *retained = 1;
    return SOBEK_OK;
}

// z_valid: the workspace still holds the state Z of all receivers, left by conv_fwd_core(order = 1) on the same inputs
int conv_bwd_core(const sobek_plan* p, const sobek_graph* g, const float* x, const float* Y,
                  const float* phi, const float* R, const float* gy, float* gx, float* gY,
                  float* gphi, float* gR, void* ws, size_t ws_bytes, void* stream, int z_valid = 0,
                  const SplitSrc* geo = nullptr) {
    int rc = check_common(p, g, ws, ws_bytes, 1);
    if (rc) return rc;
    if (!R || (g->N > 0 && (!x || !gy)) || (g->E > 0 && !geo && (!Y || !phi))) return SOBEK_ERR_INVALID_ARG;
    if (!aligned16(x, Y, phi, R, gy, gx, gY, gphi, gR)) return SOBEK_ERR_INVALID_ARG;
    if (gx && g->E > 0 && (!g->src_ptr || !g->src_perm)) return SOBEK_ERR_NEED_TRANSPOSE;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w = carve(p, g->N, 1, ws);
    if (geo && !geo_supported(p, w, 1)) return SOBEK_ERR_UNSUPPORTED;
    CK(cudaMemsetAsync(w.status, 0, kHeaderBytes, s));
    const int64_t KN = (int64_t)p->K * p->N_w;
    if (g->N == 0 || g->E == 0) {
        if (gx && g->N > 0) CK(launch_fill_zero(gx, g->N * (int64_t)p->C_x, s));
        if (gR) CK(launch_fill_zero(gR, KN, s));
        return SOBEK_OK;
    }
    const EdgeView rv = receiver_view(g);
    SplitSrc xs{}, gs{};
    if (geo) { xs = *geo; gs = *geo; gs.g_rvec = nullptr; }
    const bool g_edge = geo && geo->g_rvec;       // geometry mode: the edge pass writes the adjoint of the edge vectors
    if (g_edge) { gphi = geo->g_rvec; gY = geo->g_rvec; }      // (stand-ins: "wanted"; the kernel writes g_rvec only)
    const bool tc_edge = w.zqh != nullptr;
    const bool gx_direct = p->uvu && p->ud.ok && !p->uvu_state && !geo && g->src_recv;      // channelwise mode: no state for gx
    const bool gR_direct = gR && p->uvu && p->ud.ok && !p->uvu_state && !geo && !z_valid;   // nor for gR
    if (gR_direct) {
        int n_parts = 0;
        CK(launch_fill_zero(gR, KN, s));
        CK(launch_uvu_direct_wgrad(p, rv, x, Y, phi, gy, w.part, w.splits, &n_parts, w.status, s));
        CK(launch_reduce_parts(gR, w.part, KN, KN, n_parts, s));
        gR = nullptr;
    }
    if (w.oseg_r && (gR || gphi || gY)) { CK(launch_chunk_order(rv, w.chunk, kOrderPeriod, w.oseg_r, w.status, s)); xs.oseg = w.oseg_r; }
    if (w.oseg_s && gx && !gx_direct && !w.fused_t) {
        CK(launch_chunk_order(sender_view(g), w.chunk, kOrderPeriod, w.oseg_s, w.status, s));
        gs.oseg = w.oseg_s;
    }
    FeatureSplits fs;
    if (w.xsh && (gR || ((gphi || gY) && tc_edge))) { fs.add(x, g->N, p->C_x, w.xsh, w.xsl); xs.h = w.xsh; xs.l = w.xsl; }
    if (w.gsh && gx && !w.fused_t && !gx_direct) { fs.add(gy, g->N, p->C_y, w.gsh, w.gsl); gs.h = w.gsh; gs.l = w.gsl; }
    CK(fs.flush(s));
    PackQueue pq(p);              // every operand layout of R this call needs, one launch
    if (gphi || gY) pq.add(p->fwd, 0, 0, R, w.fKNh, w.fKNl);
    if (gx && !gx_direct && !w.fused_t) pq.add(p->tr, 1, 1, R, w.tNKh, w.tNKl);
    CK(pq.flush(s));
    if (gR || gphi || gY) {
        if (gR) CK(launch_fill_zero(w.gRp, KN, s));
        for (int64_t n0 = 0; n0 < g->N; n0 += w.chunk) {
            const int64_t nn = std::min(w.chunk, g->N - n0);
            CK(split_gy(p, p->fwd, n0, nn, gy, w.gbh, w.gbl, s));
            if (gR) {     // gR = Z^T gy with Z re-streamed, unless the forward left it in place for all receivers
                if (!(z_valid && w.chunk >= g->N))
                    CK(launch_stream(p, p->fwd, rv, n0, nn, x, nullptr, xs, Y, nullptr, phi, nullptr, 0, w.zbh, w.zbl, w.status, s));
                CK(weight_grad(p, p->fwd, n0, nn, w.zbh, w.zbl, w.gbh, w.gbl, gy, w.gRp, w.part, w.splits, w.status, s));
            }
            if (gphi || gY) {
                if (tc_edge) {
                    CK(state_adjoint(p, p->fwd, n0, nn, w.gbh, w.gbl, w.fKNh, w.fKNl, gy, R, nullptr, w.status, s, w.zqh, w.zql));
                    CK(launch_edge_pass_tc(p, p->fwd, rv, n0, nn, xs, Y, nullptr, phi, nullptr, 0, w.zqh, w.zql,
                                           g_edge ? nullptr : gphi, g_edge ? nullptr : gY, gphi ? 1 : 0, gY ? 1 : 0, w.status, s));
                } else {
                    CK(state_adjoint(p, p->fwd, n0, nn, w.gbh, w.gbl, w.fKNh, w.fKNl, gy, R, w.zbar, w.status, s));
                    CK(launch_edge_pass(p, p->fwd, rv, n0, nn, x, nullptr, Y, nullptr, phi, nullptr, 0, w.zbar, gphi, gY,
                                        gphi ? 1 : 0, gY ? 1 : 0, w.status, s));
                }
            }
        }
        if (gR) CK(unpack_R(p, p->fwd, w.gRp, gR, s));
    }
    if (gx) {
        if (has_uncovered(p->tr)) CK(launch_fill_zero(gx, g->N * (int64_t)p->C_x, s));
        const EdgeView sv = sender_view(g);
        if (gx_direct) {
            // channelwise mode, uniform natural-parity profile: the direct kernel on the sender view
            CK(launch_uvu_direct(p, sv, 1, gy, Y, phi, R, gx, w.status, s));
        } else if (w.fused_t) {
            CK(launch_pack_R_fused(p, p->tr, 1, R, w.tFKh, w.tFKl, s));
            CK(launch_fused(p, p->tr, sv, gy, nullptr, Y, nullptr, phi, nullptr, 0, w.tFKh, w.tFKl, gx, 0, w.status, s));
        } else {
            for (int64_t n0 = 0; n0 < g->N; n0 += w.chunk) {
                const int64_t nn = std::min(w.chunk, g->N - n0);
                CK(launch_stream(p, p->tr, sv, n0, nn, gy, nullptr, gs, Y, nullptr, phi, nullptr, 0, w.zbh, w.zbl, w.status, s));
                CK(mix(p, p->tr, n0, nn, w.zbh, w.zbl, w.tNKh, w.tNKl, R, gx, 0, w.status, s));
            }
        }
    }
    return SOBEK_OK;
}

int conv_dbwd_core(const sobek_plan* p, const sobek_graph* g, const float* x, const float* Y,
                   const float* phi, const float* R, const float* gy, const float* vx,
                   const float* vY, const float* vphi, const float* vR, float* ggy,
                   float* hx, float* hY, float* hphi, float* hR, void* ws, size_t ws_bytes,
                   void* stream, const SplitSrc* geo = nullptr) {
    int rc = check_common(p, g, ws, ws_bytes, 2);
    if (rc) return rc;
    if (!R || (g->N > 0 && (!x || !gy)) || (g->E > 0 && !geo && (!Y || !phi))) return SOBEK_ERR_INVALID_ARG;
    if (geo) {
        // geometry mode: the direction on the edge vectors stands for both vY and vphi (the dual stream passes compute
        // J_Y v and J_phi v themselves); the second-order edge adjoints are not provided
        if (hY || hphi) return SOBEK_ERR_UNSUPPORTED;
        vY = vphi = geo->vrvec;
    }
    if (!aligned16(x, Y, phi, R, gy, vx, vY, vphi, vR, ggy, hx, hY, hphi, hR)) return SOBEK_ERR_INVALID_ARG;
    if (hx && g->E > 0 && (!g->src_ptr || !g->src_perm)) return SOBEK_ERR_NEED_TRANSPOSE;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w = carve(p, g->N, 2, ws);
    if (geo && !(geo_supported(p, w, 1) && p->fwd.tc[1].ok && p->tr.tc[1].ok && w.vsh)) return SOBEK_ERR_UNSUPPORTED;
    CK(cudaMemsetAsync(w.status, 0, kHeaderBytes, s));
    const int64_t KN = (int64_t)p->K * p->N_w;
    const bool any_edge_dir = vx || vY || vphi;
    // outputs that no term reaches are plain zeros
    auto zero_out = [&](float*& ptr, int64_t n) -> int {
        if (ptr && n > 0) CK(launch_fill_zero(ptr, n, s));
        ptr = nullptr;
        return SOBEK_OK;
    };
    if (g->N == 0 || g->E == 0) {
        if ((rc = zero_out(ggy, g->N * (int64_t)p->C_y))) return rc;
        if ((rc = zero_out(hx, g->N * (int64_t)p->C_x))) return rc;
        if ((rc = zero_out(hR, KN))) return rc;
        return SOBEK_OK;
    }
    if (!(any_edge_dir || vR)) { if ((rc = zero_out(ggy, g->N * (int64_t)p->C_y))) return rc; }
    if (!any_edge_dir) { if ((rc = zero_out(hR, KN))) return rc; }
    if (!(vx || vY || vR)) { if ((rc = zero_out(hphi, g->E * (int64_t)p->K))) return rc; }
    if (!(vx || vphi || vR)) { if ((rc = zero_out(hY, g->E * (int64_t)p->dim_sh))) return rc; }
    if (!(vY || vphi || vR)) { if ((rc = zero_out(hx, g->N * (int64_t)p->C_x))) return rc; }

    const EdgeView rv = receiver_view(g);
    SplitSrc xs{}, gs{};
    if (geo) { xs = *geo; gs = *geo; }
    const bool tc_edge_plain = w.zqh != nullptr, tc_edge_dual = tc_edge_plain && p->fwd.etc[1].ok && (!vx || w.vsh);
    if (w.oseg_r && (ggy || hR || hphi || hY)) { CK(launch_chunk_order(rv, w.chunk, kOrderPeriod, w.oseg_r, w.status, s)); xs.oseg = w.oseg_r; }
    if (w.oseg_s && hx && !w.fused_t) {
        CK(launch_chunk_order(sender_view(g), w.chunk, kOrderPeriod, w.oseg_s, w.status, s));
        gs.oseg = w.oseg_s;
    }
    FeatureSplits fs;
    if (w.xsh && (ggy || hR || ((hphi || hY) && tc_edge_plain))) {
        fs.add(x, g->N, p->C_x, w.xsh, w.xsl); xs.h = w.xsh; xs.l = w.xsl;
        if (vx && w.vsh) { fs.add(vx, g->N, p->C_x, w.vsh, w.vsl); xs.vh = w.vsh; xs.vl = w.vsl; }
    }
    if (w.gsh && hx && !w.fused_t) { fs.add(gy, g->N, p->C_y, w.gsh, w.gsl); gs.h = w.gsh; gs.l = w.gsl; }
    CK(fs.flush(s));
    {
        // every operand layout of R and vR this call needs, one launch (the fused schedule packs its own)
        const bool fuse_ggy = ggy && w.fused_f, fuse_dz = fuse_ggy && !hR;
        PackQueue pq(p);
        if (ggy && any_edge_dir && !fuse_dz) pq.add(p->fwd, 0, 1, R, w.fNKh, w.fNKl);
        if (ggy && vR && !fuse_ggy) pq.add(p->fwd, 0, 1, vR, w.vfNKh, w.vfNKl);
        if ((hphi || hY) && any_edge_dir) pq.add(p->fwd, 0, 0, R, w.fKNh, w.fKNl);
        if ((hphi || hY) && vR) pq.add(p->fwd, 0, 0, vR, w.vfKNh, w.vfKNl);
        if (hx && !w.fused_t) {
            if (vY || vphi) pq.add(p->tr, 1, 1, R, w.tNKh, w.tNKl);
            if (vR) pq.add(p->tr, 1, 1, vR, w.vtNKh, w.vtNKl);
        }
        CK(pq.flush(s));
    }
    if (ggy || hR || hphi || hY) {
        if (ggy && has_uncovered(p->fwd)) CK(launch_fill_zero(ggy, g->N * (int64_t)p->C_y, s));
        // ggy = Z vR + dZ R.  The fused kernels produce it without leaving the SM; when hR is wanted too the
        // directional state dZ is materialised chunk by chunk (it also feeds hR = dZ^T gy).
        const bool fuse_ggy = ggy && w.fused_f;
        const bool fuse_dz = fuse_ggy && !hR;
        int ggy_done = 0;
        if (fuse_ggy && vR) {
            CK(launch_pack_R_fused(p, p->fwd, 0, vR, w.vfFKh, w.vfFKl, s));
            CK(launch_fused(p, p->fwd, rv, x, nullptr, Y, nullptr, phi, nullptr, 0, w.vfFKh, w.vfFKl, ggy, 0, w.status, s));
            ggy_done = 1;
        }
        if (fuse_dz && any_edge_dir) {
            CK(launch_pack_R_fused(p, p->fwd, 0, R, w.fFKh, w.fFKl, s));
            CK(launch_fused(p, p->fwd, rv, x, vx, Y, vY, phi, vphi, 1, w.fFKh, w.fFKl, ggy, ggy_done, w.status, s));
            ggy_done = 1;
        }
        if (hR) CK(launch_fill_zero(w.gRp, KN, s));
        for (int64_t n0 = 0; n0 < g->N; n0 += w.chunk) {
            const int64_t nn = std::min(w.chunk, g->N - n0);
            if (hR || hphi || hY) CK(split_gy(p, p->fwd, n0, nn, gy, w.gbh, w.gbl, s));
            // ggy = Z vR + dZ R,  hR = dZ^T gy      (Eq. receiver_double_adjoint with d(gy) = 0)
            int ggy_written = ggy_done;
            if (ggy && vR && !fuse_ggy) {
                CK(launch_stream(p, p->fwd, rv, n0, nn, x, nullptr, xs, Y, nullptr, phi, nullptr, 0, w.zbh, w.zbl, w.status, s));
                CK(mix(p, p->fwd, n0, nn, w.zbh, w.zbl, w.vfNKh, w.vfNKl, vR, ggy, 0, w.status, s));
                ggy_written = 1;
            }
            if (((ggy && !fuse_dz) || hR) && any_edge_dir) {
                // dZ = sum_e ( vphi (x) C(x,Y) + phi (x) [C(vx,Y) + C(x,vY)] ) in one pass
                CK(launch_stream(p, p->fwd, rv, n0, nn, x, vx, xs, Y, vY, phi, vphi, 1, w.zbh, w.zbl, w.status, s));
                if (ggy && !fuse_dz) CK(mix(p, p->fwd, n0, nn, w.zbh, w.zbl, w.fNKh, w.fNKl, R, ggy, ggy_written, w.status, s));
                if (hR) CK(weight_grad(p, p->fwd, n0, nn, w.zbh, w.zbl, w.gbh, w.gbl, gy, w.gRp, w.part, w.splits, w.status, s));
            }
            if (hphi || hY) {
                int pm = 1, ym = 1;   // first writer overwrites, later ones accumulate
                if (any_edge_dir) {
                    // the three direction terms that share Zbar = gy R^T, in one pass
                    if (tc_edge_dual) {
                        CK(state_adjoint(p, p->fwd, n0, nn, w.gbh, w.gbl, w.fKNh, w.fKNl, gy, R, nullptr, w.status, s, w.zqh, w.zql));
                        CK(launch_edge_pass_tc(p, p->fwd, rv, n0, nn, xs, Y, vY, phi, vphi, 1, w.zqh, w.zql, hphi, hY,
                                               hphi ? pm : 0, hY ? ym : 0, w.status, s));
                    } else {
                        CK(state_adjoint(p, p->fwd, n0, nn, w.gbh, w.gbl, w.fKNh, w.fKNl, gy, R, w.zbar, w.status, s));
                        CK(launch_edge_pass(p, p->fwd, rv, n0, nn, x, vx, Y, vY, phi, vphi, 1, w.zbar, hphi, hY,
                                            hphi ? pm : 0, hY ? ym : 0, w.status, s));
                    }
                    pm = ym = 2;
                }
                if (vR) {   // the term through dZbar = gy vR^T
                    if (tc_edge_plain) {
                        CK(state_adjoint(p, p->fwd, n0, nn, w.gbh, w.gbl, w.vfKNh, w.vfKNl, gy, vR, nullptr, w.status, s, w.zqh, w.zql));
                        SplitSrc xp{}; xp.h = xs.h; xp.l = xs.l;
                        CK(launch_edge_pass_tc(p, p->fwd, rv, n0, nn, xp, Y, nullptr, phi, nullptr, 0, w.zqh, w.zql, hphi, hY,
                                               hphi ? pm : 0, hY ? ym : 0, w.status, s));
                    } else {
                        CK(state_adjoint(p, p->fwd, n0, nn, w.gbh, w.gbl, w.vfKNh, w.vfKNl, gy, vR, w.zbar, w.status, s));
                        CK(launch_edge_pass(p, p->fwd, rv, n0, nn, x, nullptr, Y, nullptr, phi, nullptr, 0, w.zbar, hphi, hY,
                                            hphi ? pm : 0, hY ? ym : 0, w.status, s));
                    }
                }
            }
        }
        if (hR) CK(unpack_R(p, p->fwd, w.gRp, hR, s));
    }
    if (hx) {
        if (has_uncovered(p->tr)) CK(launch_fill_zero(hx, g->N * (int64_t)p->C_x, s));
        const EdgeView sv = sender_view(g);
        if (w.fused_t) {
            int wrote = 0;
            if (vY || vphi) {   // dV = V(gy; vY, phi) + V(gy; Y, vphi) in one pass
                CK(launch_pack_R_fused(p, p->tr, 1, R, w.tFKh, w.tFKl, s));
                CK(launch_fused(p, p->tr, sv, gy, nullptr, Y, vY, phi, vphi, 1, w.tFKh, w.tFKl, hx, 0, w.status, s));
                wrote = 1;
            }
            if (vR) {
                CK(launch_pack_R_fused(p, p->tr, 1, vR, w.vtFKh, w.vtFKl, s));
                CK(launch_fused(p, p->tr, sv, gy, nullptr, Y, nullptr, phi, nullptr, 0, w.vtFKh, w.vtFKl, hx, wrote, w.status, s));
            }
            return SOBEK_OK;
        }
        for (int64_t n0 = 0; n0 < g->N; n0 += w.chunk) {
            const int64_t nn = std::min(w.chunk, g->N - n0);
            int wrote = 0;
            if (vY || vphi) {   // dV = V(gy; vY, phi) + V(gy; Y, vphi) in one pass
                CK(launch_stream(p, p->tr, sv, n0, nn, gy, nullptr, gs, Y, vY, phi, vphi, 1, w.zbh, w.zbl, w.status, s));
                CK(mix(p, p->tr, n0, nn, w.zbh, w.zbl, w.tNKh, w.tNKl, R, hx, 0, w.status, s));
                wrote = 1;
            }
            if (vR) {
                CK(launch_stream(p, p->tr, sv, n0, nn, gy, nullptr, gs, Y, nullptr, phi, nullptr, 0, w.zbh, w.zbl, w.status, s));
                CK(mix(p, p->tr, n0, nn, w.zbh, w.zbl, w.vtNKh, w.vtNKl, vR, hx, wrote, w.status, s));
            }
        }
    }
    return SOBEK_OK;
}

// ---- boundary layout: a mul_ir plan re-lays the node feature arrays through the workspace around the ir_mul core
struct Relay {
    const sobek_plan* p; int64_t N; cudaStream_t s;
    // ir_mul copy of an input on C_x (in = 1) or C_y columns; NULL stays NULL
    int in_x(const float* src, float* tmp, const float** out) const {
        *out = src;
        if (!src || !p->mul_ir) return SOBEK_OK;
        CK(launch_relayout(src, tmp, N, p->C_x, p->d_in_blocks, (int)p->in.size(), 1, s));
        *out = tmp; return SOBEK_OK;
    }
    int in_y(const float* src, float* tmp, const float** out) const {
        *out = src;
        if (!src || !p->mul_ir) return SOBEK_OK;
        CK(launch_relayout(src, tmp, N, p->C_y, p->d_out_blocks, (int)p->out.size(), 1, s));
        *out = tmp; return SOBEK_OK;
    }
    int out_x(const float* tmp, float* dst) const {
        if (!dst || !p->mul_ir) return SOBEK_OK;
        CK(launch_relayout(tmp, dst, N, p->C_x, p->d_in_blocks, (int)p->in.size(), 0, s));
        return SOBEK_OK;
    }
    int out_y(const float* tmp, float* dst) const {
        if (!dst || !p->mul_ir) return SOBEK_OK;
        CK(launch_relayout(tmp, dst, N, p->C_y, p->d_out_blocks, (int)p->out.size(), 0, s));
        return SOBEK_OK;
    }
};
}  // namespace

extern "C" int sobek_conv_fwd(const sobek_plan* p, const sobek_graph* g, const float* x, const float* Y,
                              const float* phi, const float* R, float* y, void* ws, size_t ws_bytes,
                              void* stream) {
    if (!p || !p->mul_ir) return conv_fwd_core(p, g, x, Y, phi, R, y, ws, ws_bytes, stream);
    int rc = check_common(p, g, ws, ws_bytes, 0);
    if (rc) return rc;
    if (!y || (g->N > 0 && !x)) return SOBEK_ERR_INVALID_ARG;
    const Workspace w = carve(p, g->N, 0, ws);
    const Relay r{p, g->N, (cudaStream_t)stream};
    const float* xi;
    if ((rc = r.in_x(x, w.lx, &xi))) return rc;
    if ((rc = conv_fwd_core(p, g, xi, Y, phi, R, w.ly, ws, ws_bytes, stream))) return rc;
    return r.out_y(w.ly, y);
}

extern "C" int sobek_conv_bwd(const sobek_plan* p, const sobek_graph* g, const float* x, const float* Y,
                              const float* phi, const float* R, const float* gy, float* gx, float* gY,
                              float* gphi, float* gR, void* ws, size_t ws_bytes, void* stream) {
    if (!p || !p->mul_ir) return conv_bwd_core(p, g, x, Y, phi, R, gy, gx, gY, gphi, gR, ws, ws_bytes, stream);
    int rc = check_common(p, g, ws, ws_bytes, 1);
    if (rc) return rc;
    if (g->N > 0 && (!x || !gy)) return SOBEK_ERR_INVALID_ARG;
    const Workspace w = carve(p, g->N, 1, ws);
    const Relay r{p, g->N, (cudaStream_t)stream};
    const float *xi, *gyi;
    if ((rc = r.in_x(x, w.lx, &xi)) || (rc = r.in_y(gy, w.lgy, &gyi))) return rc;
    if ((rc = conv_bwd_core(p, g, xi, Y, phi, R, gyi, gx ? w.lgx : nullptr, gY, gphi, gR, ws, ws_bytes, stream))) return rc;
    return r.out_x(w.lgx, gx);
}

namespace {
int geo_source(const float* rvec, int basis, float r_cut, int envelope_p, SplitSrc* geo) {
    if (!rvec || (basis != SOBEK_BASIS_BESSEL && basis != SOBEK_BASIS_GAUSSIAN) || !(r_cut > 0.f) ||
        (basis == SOBEK_BASIS_BESSEL && (envelope_p < 1 || envelope_p > 16)))
        return SOBEK_ERR_INVALID_ARG;
    geo->rvec = rvec; geo->geo_basis = basis; geo->geo_rc = r_cut; geo->geo_p = envelope_p;
    return SOBEK_OK;
}
}  // namespace

extern "C" int sobek_edge_vectors(const sobek_graph* g, const float* pos, float* rvec, void* stream) {
    return edge_vectors(g, pos, rvec, (cudaStream_t)stream);
}

extern "C" int sobek_position_gradient(const sobek_graph* g, const float* g_rvec, float* gpos, void* stream) {
    return position_gradient(g, g_rvec, gpos, (cudaStream_t)stream);
}

extern "C" int sobek_conv_geo_fwd(const sobek_plan* p, const sobek_graph* g, const float* rvec, int basis, float r_cut,
                                  int envelope_p, const float* x, const float* R, float* y, void* ws, size_t ws_bytes,
                                  void* stream) {
    SplitSrc geo{};
    if (g && g->E > 0) { const int rc = geo_source(rvec, basis, r_cut, envelope_p, &geo); if (rc) return rc; }
    else geo.rvec = rvec ? rvec : reinterpret_cast<const float*>(&geo);      // no edge is read
    return conv_fwd_core(p, g, x, nullptr, nullptr, R, y, ws, ws_bytes, stream, 0, nullptr, &geo);
}

extern "C" int sobek_conv_geo_bwd(const sobek_plan* p, const sobek_graph* g, const float* rvec, int basis, float r_cut,
                                  int envelope_p, const float* x, const float* R, const float* gy, float* gx,
                                  float* g_rvec, float* gR, void* ws, size_t ws_bytes, void* stream) {
    SplitSrc geo{};
    if (g && g->E > 0) { const int rc = geo_source(rvec, basis, r_cut, envelope_p, &geo); if (rc) return rc; }
    else geo.rvec = rvec ? rvec : reinterpret_cast<const float*>(&geo);
    geo.g_rvec = g_rvec;
    return conv_bwd_core(p, g, x, nullptr, nullptr, R, gy, gx, nullptr, nullptr, gR, ws, ws_bytes, stream, 0, &geo);
}

extern "C" int sobek_conv_geo_dbwd(const sobek_plan* p, const sobek_graph* g, const float* rvec, int basis, float r_cut,
                                   int envelope_p, const float* x, const float* R, const float* gy, const float* vx,
                                   const float* v_rvec, const float* vR, float* ggy, float* hx, float* hR, void* ws,
                                   size_t ws_bytes, void* stream) {
    SplitSrc geo{};
    if (g && g->E > 0) { const int rc = geo_source(rvec, basis, r_cut, envelope_p, &geo); if (rc) return rc; }
    else geo.rvec = rvec ? rvec : reinterpret_cast<const float*>(&geo);
    geo.vrvec = v_rvec;
    return conv_dbwd_core(p, g, x, nullptr, nullptr, R, gy, vx, nullptr, nullptr, vR, ggy, hx, nullptr, nullptr, hR, ws,
                          ws_bytes, stream, &geo);
}

// the eight edge arrays of sobek_conv_geo_dbwd_full behind the workspace of the stored-input calls
namespace {
struct GeoFullWs { size_t core; float *Y, *vY, *gY, *hY, *phi, *vphi, *gphi, *hphi; size_t bytes; };
GeoFullWs geo_full_carve(const sobek_plan* p, int64_t N, int64_t E, void* ws) {
    GeoFullWs w{};
    w.core = (std::max(sobek_workspace_bytes(p, N, E, 1), sobek_workspace_bytes(p, N, E, 2)) + 255) & ~size_t(255);
    size_t off = w.core;
    auto take = [&](size_t n) { float* q = ws ? reinterpret_cast<float*>((char*)ws + off) : nullptr; off += (n * 4 + 255) & ~size_t(255); return q; };
    const size_t ny = (size_t)E * p->dim_sh, nk = (size_t)E * p->K;
    w.Y = take(ny); w.vY = take(ny); w.gY = take(ny); w.hY = take(ny);
    w.phi = take(nk); w.vphi = take(nk); w.gphi = take(nk); w.hphi = take(nk);
    w.bytes = off;
    return w;
}
}  // namespace

extern "C" size_t sobek_geo_dbwd_full_workspace_bytes(const sobek_plan* p, int64_t N, int64_t E) {
    if (!p || N < 0 || E < 0) return 0;
    return geo_full_carve(p, N, E, nullptr).bytes;
}

extern "C" int sobek_conv_geo_dbwd_full(const sobek_plan* p, const sobek_graph* g, const float* rvec, int basis, float r_cut,
                                        int envelope_p, const float* x, const float* R, const float* gy, const float* vx,
                                        const float* v_rvec, const float* vR, float* ggy, float* hx, float* hR,
                                        float* h_rvec, void* ws, size_t ws_bytes, void* stream) {
    if (!p || !g) return SOBEK_ERR_INVALID_ARG;
    if (g->E > 0 && !rvec) return SOBEK_ERR_INVALID_ARG;
    if (basis != SOBEK_BASIS_BESSEL && basis != SOBEK_BASIS_GAUSSIAN) return SOBEK_ERR_INVALID_ARG;
    if (!(r_cut > 0.f) || (basis == SOBEK_BASIS_BESSEL && envelope_p < 1)) return SOBEK_ERR_INVALID_ARG;
    if (!geo_second_supported(p->l_max, p->K)) return SOBEK_ERR_UNSUPPORTED;
    if (!aligned16(rvec, v_rvec, h_rvec)) return SOBEK_ERR_INVALID_ARG;
    if (!ws || ((uintptr_t)ws & 255)) return SOBEK_ERR_WORKSPACE;
    const GeoFullWs w = geo_full_carve(p, g->N, g->E, ws);
    if (ws_bytes < w.bytes) return SOBEK_ERR_WORKSPACE;
    cudaStream_t s = (cudaStream_t)stream;
    CK(launch_geo_edge_inputs(rvec, v_rvec, g->E, p->l_max, p->K, r_cut, basis, envelope_p, w.Y, w.phi, w.vY, w.vphi, s));
    int rc;
    if (h_rvec) {       // the first-order edge adjoints, which the derivative of the Jacobians is contracted with
        if ((rc = sobek_conv_bwd(p, g, x, w.Y, w.phi, R, gy, nullptr, w.gY, w.gphi, nullptr, ws, w.core, stream))) return rc;
    }
    const float* vYp = v_rvec ? w.vY : nullptr;
    const float* vpp = v_rvec ? w.vphi : nullptr;
    if ((rc = sobek_conv_dbwd(p, g, x, w.Y, w.phi, R, gy, vx, vYp, vpp, vR, ggy, hx, h_rvec ? w.hY : nullptr,
                              h_rvec ? w.hphi : nullptr, hR, ws, w.core, stream)))
        return rc;
    if (h_rvec)
        CK(launch_geo_second_adjoint(rvec, v_rvec, g->E, p->l_max, p->K, r_cut, basis, envelope_p, w.gY, w.gphi, w.hY, w.hphi,
                                     h_rvec, s));
    return SOBEK_OK;
}

extern "C" int sobek_conv_fwd_retain(const sobek_plan* p, const sobek_graph* g, const float* x, const float* Y,
                                     const float* phi, const float* R, float* y, void* ws, size_t ws_bytes,
                                     void* stream, int* retained) {
    if (!retained) return SOBEK_ERR_INVALID_ARG;
    *retained = 0;
    if (!p || !p->mul_ir) return conv_fwd_core(p, g, x, Y, phi, R, y, ws, ws_bytes, stream, 1, retained);
    int rc = check_common(p, g, ws, ws_bytes, 1);
    if (rc) return rc;
    if (!y || (g->N > 0 && !x)) return SOBEK_ERR_INVALID_ARG;
    const Workspace w = carve(p, g->N, 1, ws);
    const Relay r{p, g->N, (cudaStream_t)stream};
    const float* xi;
    if ((rc = r.in_x(x, w.lx, &xi))) return rc;
    if ((rc = conv_fwd_core(p, g, xi, Y, phi, R, w.ly, ws, ws_bytes, stream, 1, retained))) return rc;
    return r.out_y(w.ly, y);
}

extern "C" int sobek_conv_bwd_retained(const sobek_plan* p, const sobek_graph* g, const float* x, const float* Y,
                                       const float* phi, const float* R, const float* gy, float* gx, float* gY,
                                       float* gphi, float* gR, void* ws, size_t ws_bytes, void* stream, int retained) {
    if (!p || !p->mul_ir) return conv_bwd_core(p, g, x, Y, phi, R, gy, gx, gY, gphi, gR, ws, ws_bytes, stream, retained);
    int rc = check_common(p, g, ws, ws_bytes, 1);
    if (rc) return rc;
    if (g->N > 0 && (!x || !gy)) return SOBEK_ERR_INVALID_ARG;
    const Workspace w = carve(p, g->N, 1, ws);
    const Relay r{p, g->N, (cudaStream_t)stream};
    const float *xi, *gyi;
    if ((rc = r.in_x(x, w.lx, &xi)) || (rc = r.in_y(gy, w.lgy, &gyi))) return rc;
    if ((rc = conv_bwd_core(p, g, xi, Y, phi, R, gyi, gx ? w.lgx : nullptr, gY, gphi, gR, ws, ws_bytes, stream, retained))) return rc;
    return r.out_x(w.lgx, gx);
}

extern "C" int sobek_conv_dbwd(const sobek_plan* p, const sobek_graph* g, const float* x, const float* Y,
                               const float* phi, const float* R, const float* gy, const float* vx,
                               const float* vY, const float* vphi, const float* vR, float* ggy,
                               float* hx, float* hY, float* hphi, float* hR, void* ws, size_t ws_bytes,
                               void* stream) {
    if (!p || !p->mul_ir)
        return conv_dbwd_core(p, g, x, Y, phi, R, gy, vx, vY, vphi, vR, ggy, hx, hY, hphi, hR, ws, ws_bytes, stream);
    int rc = check_common(p, g, ws, ws_bytes, 2);
    if (rc) return rc;
    if (g->N > 0 && (!x || !gy)) return SOBEK_ERR_INVALID_ARG;
    const Workspace w = carve(p, g->N, 2, ws);
    const Relay r{p, g->N, (cudaStream_t)stream};
    const float *xi, *gyi, *vxi;
    if ((rc = r.in_x(x, w.lx, &xi)) || (rc = r.in_y(gy, w.lgy, &gyi)) || (rc = r.in_x(vx, w.lvx, &vxi))) return rc;
    if ((rc = conv_dbwd_core(p, g, xi, Y, phi, R, gyi, vxi, vY, vphi, vR, ggy ? w.ly : nullptr, hx ? w.lgx : nullptr, hY, hphi,
                             hR, ws, ws_bytes, stream)))
        return rc;
    if ((rc = r.out_y(w.ly, ggy))) return rc;
    return r.out_x(w.lgx, hx);
}

extern "C" int sobek_selftest_wait_timeout(void* ws, unsigned limit_ms, void* stream) {
    if (!ws || ((uintptr_t)ws & 255) || limit_ms == 0 || limit_ms > 2000) return SOBEK_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    CK(cudaMemsetAsync(ws, 0, kHeaderBytes, s));
    CK(launch_wait_selftest((int*)ws, (uint64_t)limit_ms * 1000000ull, s));
    return SOBEK_OK;
}

extern "C" int sobek_last_device_status(void* ws, void* stream) {
    if (!ws) return SOBEK_ERR_INVALID_ARG;
    int h = 0;
    cudaError_t e = cudaMemcpyAsync(&h, ws, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return SOBEK_ERR_CUDA; }
    return h;
}
