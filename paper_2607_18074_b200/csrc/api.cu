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
    float* Rp;     // R   packed for the receiver direction
    float* Rt;     // R   packed for the sender direction
    float* gRp;    // packed accumulator of the R adjoint
    float* vRp;    // vR  packed, receiver direction
    float* vRt;    // vR  packed, sender direction
    float* state;  // bounded node state (Z / Zbar / V) of one chunk
    int64_t chunk;
    size_t bytes;
};

Workspace carve(const sobek_plan* p, int64_t N, int order, void* ws) {
    Workspace w{};
    char* c = (char*)ws;
    const size_t rbytes = align256((size_t)p->K * (size_t)p->N_w * 4);
    size_t off = kHeaderBytes;
    w.status = (int*)c;
    w.Rp = (float*)(c + off); off += rbytes;
    if (order >= 1) {
        w.Rt = (float*)(c + off); off += rbytes;
        w.gRp = (float*)(c + off); off += rbytes;
    }
    if (order >= 2) {
        w.vRp = (float*)(c + off); off += rbytes;
        w.vRt = (float*)(c + off); off += rbytes;
    }
    w.chunk = chunk_nodes(p, N, order);
    int64_t per = p->fwd.state_floats;
    if (order >= 1) per = std::max(per, p->tr.state_floats);
    w.state = (float*)(c + off);
    off += align256((size_t)w.chunk * (size_t)per * 4);
    w.bytes = off;
    return w;
}

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
    return EdgeView{g->src_ptr, g->src_perm, g->col, g->row_ptr, g->N, g->E, 1};
}

bool has_uncovered(const Direction& d) {
    for (const DGroup& G : d.groups)
        if (G.path_end == G.path_begin) return true;
    return false;
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

extern "C" int sobek_conv_fwd(const sobek_plan* p, const sobek_graph* g, const float* x, const float* Y,
                              const float* phi, const float* R, float* y, void* ws, size_t ws_bytes,
                              void* stream) {
    int rc = check_common(p, g, ws, ws_bytes, 0);
    if (rc) return rc;
    if (!y || !R || (g->N > 0 && !x) || (g->E > 0 && (!Y || !phi))) return SOBEK_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w = carve(p, g->N, 0, ws);
    CK(cudaMemsetAsync(w.status, 0, kHeaderBytes, s));
    if (g->N == 0) return SOBEK_OK;
    if (g->E == 0 || has_uncovered(p->fwd)) CK(launch_fill_zero(y, g->N * (int64_t)p->C_y, s));
    if (g->E == 0) return SOBEK_OK;
    CK(launch_pack_R(p, p->fwd, 0, R, w.Rp, s));
    const EdgeView rv = receiver_view(g);
    for (int64_t n0 = 0; n0 < g->N; n0 += w.chunk) {
        const int64_t nn = std::min(w.chunk, g->N - n0);
        CK(launch_state(p, p->fwd, rv, n0, nn, x, Y, phi, w.state, 0, s));
        CK(launch_mix(p, p->fwd, n0, nn, w.state, w.Rp, y, 0, s));
    }
    return SOBEK_OK;
}

extern "C" int sobek_conv_bwd(const sobek_plan* p, const sobek_graph* g, const float* x, const float* Y,
                              const float* phi, const float* R, const float* gy, float* gx, float* gY,
                              float* gphi, float* gR, void* ws, size_t ws_bytes, void* stream) {
    int rc = check_common(p, g, ws, ws_bytes, 1);
    if (rc) return rc;
    if (!R || (g->N > 0 && (!x || !gy)) || (g->E > 0 && (!Y || !phi))) return SOBEK_ERR_INVALID_ARG;
    if (gx && g->E > 0 && (!g->src_ptr || !g->src_perm)) return SOBEK_ERR_NEED_TRANSPOSE;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w = carve(p, g->N, 1, ws);
    CK(cudaMemsetAsync(w.status, 0, kHeaderBytes, s));
    const int64_t KN = (int64_t)p->K * p->N_w;
    if (g->N == 0 || g->E == 0) {
        if (gx && g->N > 0) CK(launch_fill_zero(gx, g->N * (int64_t)p->C_x, s));
        if (gR) CK(launch_fill_zero(gR, KN, s));
        return SOBEK_OK;
    }
    CK(launch_pack_R(p, p->fwd, 0, R, w.Rp, s));
    if (gR) CK(launch_fill_zero(w.gRp, KN, s));
    const EdgeView rv = receiver_view(g);
    if (gR || gphi || gY) {
        for (int64_t n0 = 0; n0 < g->N; n0 += w.chunk) {
            const int64_t nn = std::min(w.chunk, g->N - n0);
            if (gR) {
                CK(launch_state(p, p->fwd, rv, n0, nn, x, Y, phi, w.state, 0, s));
                CK(launch_weight_grad(p, p->fwd, n0, nn, w.state, gy, w.gRp, 1, s));
            }
            if (gphi || gY) {
                CK(launch_state_adjoint(p, p->fwd, n0, nn, gy, w.Rp, w.state, s));
                CK(launch_edge_pass(p, p->fwd, rv, n0, nn, x, Y, phi, w.state, gphi, gY, gphi ? 1 : 0,
                                    gY ? 1 : 0, s));
            }
        }
    }
    if (gR) CK(launch_unpack_R(p, p->fwd, w.gRp, gR, s));
    if (gx) {
        if (has_uncovered(p->tr)) CK(launch_fill_zero(gx, g->N * (int64_t)p->C_x, s));
        CK(launch_pack_R(p, p->tr, 1, R, w.Rt, s));
        const EdgeView sv = sender_view(g);
        for (int64_t n0 = 0; n0 < g->N; n0 += w.chunk) {
            const int64_t nn = std::min(w.chunk, g->N - n0);
            CK(launch_state(p, p->tr, sv, n0, nn, gy, Y, phi, w.state, 0, s));
            CK(launch_mix(p, p->tr, n0, nn, w.state, w.Rt, gx, 0, s));
        }
    }
    return SOBEK_OK;
}

extern "C" int sobek_conv_dbwd(const sobek_plan* p, const sobek_graph* g, const float* x, const float* Y,
                               const float* phi, const float* R, const float* gy, const float* vx,
                               const float* vY, const float* vphi, const float* vR, float* ggy,
                               float* hx, float* hY, float* hphi, float* hR, void* ws, size_t ws_bytes,
                               void* stream) {
    int rc = check_common(p, g, ws, ws_bytes, 2);
    if (rc) return rc;
    if (!R || (g->N > 0 && (!x || !gy)) || (g->E > 0 && (!Y || !phi))) return SOBEK_ERR_INVALID_ARG;
    if (hx && g->E > 0 && (!g->src_ptr || !g->src_perm)) return SOBEK_ERR_NEED_TRANSPOSE;
    cudaStream_t s = (cudaStream_t)stream;
    Workspace w = carve(p, g->N, 2, ws);
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
    if (!(any_edge_dir || vR)) {
        if ((rc = zero_out(ggy, g->N * (int64_t)p->C_y))) return rc;
    }
    if (!any_edge_dir) { if ((rc = zero_out(hR, KN))) return rc; }
    if (!(vx || vY || vR)) { if ((rc = zero_out(hphi, g->E * (int64_t)p->K))) return rc; }
    if (!(vx || vphi || vR)) { if ((rc = zero_out(hY, g->E * (int64_t)p->dim_sh))) return rc; }
    if (!(vY || vphi || vR)) { if ((rc = zero_out(hx, g->N * (int64_t)p->C_x))) return rc; }

    CK(launch_pack_R(p, p->fwd, 0, R, w.Rp, s));
    if (vR) CK(launch_pack_R(p, p->fwd, 0, vR, w.vRp, s));
    if (hR) CK(launch_fill_zero(w.gRp, KN, s));
    const EdgeView rv = receiver_view(g);
    if (ggy && has_uncovered(p->fwd)) CK(launch_fill_zero(ggy, g->N * (int64_t)p->C_y, s));

    if (ggy || hR || hphi || hY) {
        for (int64_t n0 = 0; n0 < g->N; n0 += w.chunk) {
            const int64_t nn = std::min(w.chunk, g->N - n0);
            // ggy = Z vR + dZ R,  hR = dZ^T gy      (Eq. receiver_double_adjoint, d(gy) = 0)
            int ggy_written = 0;
            if (ggy && vR) {
                CK(launch_state(p, p->fwd, rv, n0, nn, x, Y, phi, w.state, 0, s));
                CK(launch_mix(p, p->fwd, n0, nn, w.state, w.vRp, ggy, 0, s));
                ggy_written = 1;
            }
            if ((ggy || hR) && any_edge_dir) {
                int acc = 0;   // dZ = Z(vx,Y,phi) + Z(x,vY,phi) + Z(x,Y,vphi)
                if (vx) { CK(launch_state(p, p->fwd, rv, n0, nn, vx, Y, phi, w.state, acc, s)); acc = 1; }
                if (vY) { CK(launch_state(p, p->fwd, rv, n0, nn, x, vY, phi, w.state, acc, s)); acc = 1; }
                if (vphi) { CK(launch_state(p, p->fwd, rv, n0, nn, x, Y, vphi, w.state, acc, s)); acc = 1; }
                if (ggy) CK(launch_mix(p, p->fwd, n0, nn, w.state, w.Rp, ggy, ggy_written, s));
                if (hR) CK(launch_weight_grad(p, p->fwd, n0, nn, w.state, gy, w.gRp, 1, s));
            }
            if (hphi || hY) {
                int pm = 1, ym = 1;   // first writer overwrites, later ones accumulate
                if (any_edge_dir) {
                    CK(launch_state_adjoint(p, p->fwd, n0, nn, gy, w.Rp, w.state, s));
                    if (vx) {
                        CK(launch_edge_pass(p, p->fwd, rv, n0, nn, vx, Y, phi, w.state, hphi, hY,
                                            hphi ? pm : 0, hY ? ym : 0, s));
                        pm = ym = 2;
                    }
                    if (vY && hphi) {
                        CK(launch_edge_pass(p, p->fwd, rv, n0, nn, x, vY, phi, w.state, hphi, hY, pm, 0, s));
                        pm = 2;
                    }
                    if (vphi && hY) {
                        CK(launch_edge_pass(p, p->fwd, rv, n0, nn, x, Y, vphi, w.state, hphi, hY, 0, ym, s));
                        ym = 2;
                    }
                }
                if (vR) {
                    CK(launch_state_adjoint(p, p->fwd, n0, nn, gy, w.vRp, w.state, s));
                    CK(launch_edge_pass(p, p->fwd, rv, n0, nn, x, Y, phi, w.state, hphi, hY, hphi ? pm : 0,
                                        hY ? ym : 0, s));
                }
            }
        }
    }
    if (hR) CK(launch_unpack_R(p, p->fwd, w.gRp, hR, s));
    if (hx) {
        if (has_uncovered(p->tr)) CK(launch_fill_zero(hx, g->N * (int64_t)p->C_x, s));
        CK(launch_pack_R(p, p->tr, 1, R, w.Rt, s));
        if (vR) CK(launch_pack_R(p, p->tr, 1, vR, w.vRt, s));
        const EdgeView sv = sender_view(g);
        for (int64_t n0 = 0; n0 < g->N; n0 += w.chunk) {
            const int64_t nn = std::min(w.chunk, g->N - n0);
            int wrote = 0;
            if (vY || vphi) {
                int acc = 0;
                if (vY) { CK(launch_state(p, p->tr, sv, n0, nn, gy, vY, phi, w.state, acc, s)); acc = 1; }
                if (vphi) { CK(launch_state(p, p->tr, sv, n0, nn, gy, Y, vphi, w.state, acc, s)); acc = 1; }
                CK(launch_mix(p, p->tr, n0, nn, w.state, w.Rt, hx, 0, s));
                wrote = 1;
            }
            if (vR) {
                CK(launch_state(p, p->tr, sv, n0, nn, gy, Y, phi, w.state, 0, s));
                CK(launch_mix(p, p->tr, n0, nn, w.state, w.vRt, hx, wrote, s));
            }
        }
    }
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
