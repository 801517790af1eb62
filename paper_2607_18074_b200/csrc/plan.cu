// Plan creation: path enumeration, real Clebsch-Gordan tensors, sparse tables, traversal
// descriptors (host), and their upload.
//
// The coupling tensors are obtained numerically as the rotation-invariant element of
// (l_in x l_sh x l_out): a seed tensor is averaged over SO(3) with an exact quadrature in
// ZYZ Euler angles, using real Wigner matrices D^l(g) that are solved from the defining
// relation Y_l(g r) = D^l(g) Y_l(r) of the real spherical harmonics.  The invariant
// subspace is one-dimensional, so the result is fixed up to scale and sign; it is scaled
// to unit Frobenius norm, its first nonzero entry (lexicographic in m_in, m_sh, m_out) is
// made positive, and the path normalisation sqrt(2 l_out + 1) of Eq. angular_path_contraction
// is applied.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>

#include "internal.h"

namespace sobek {
namespace {

constexpr int LM = SOBEK_MAX_L;
constexpr int DMAX = 2 * LM + 1;
const double kPi = 3.14159265358979323846;

// Orthonormal real spherical harmonics up to order lmax at the direction (x,y,z) (unit).
// Components m = -l..l, sine-type for m < 0, no Condon-Shortley sign.
void real_sh(int lmax, double x, double y, double z, double* out) {
    double P[LM + 1][LM + 1];  // P[l][m]
    const double s = sqrt(std::max(0.0, 1.0 - z * z));
    for (int m = 0; m <= lmax; ++m) {
        double pmm = 1.0;
        for (int k = 1; k <= m; ++k) pmm *= (2 * k - 1) * s;
        P[m][m] = pmm;
        if (m + 1 <= lmax) P[m + 1][m] = z * (2 * m + 1) * pmm;
        for (int l = m + 2; l <= lmax; ++l)
            P[l][m] = ((2 * l - 1) * z * P[l - 1][m] - (l + m - 1) * P[l - 2][m]) / (l - m);
    }
    const double ph = atan2(y, x);
    for (int l = 0; l <= lmax; ++l) {
        const int base = l * l + l;
        for (int m = 0; m <= l; ++m) {
            double f = (2 * l + 1) / (4 * kPi);
            for (int k = l - m + 1; k <= l + m; ++k) f /= k;
            const double n = sqrt(f);
            if (m == 0) {
                out[base] = n * P[l][0];
            } else {
                out[base + m] = sqrt(2.0) * n * P[l][m] * cos(m * ph);
                out[base - m] = sqrt(2.0) * n * P[l][m] * sin(m * ph);
            }
        }
    }
}

// In-place inverse of a d x d matrix (row-major, leading dimension DMAX), partial pivoting.
bool invert(double a[DMAX][DMAX], int d) {
    double inv[DMAX][DMAX] = {};
    for (int i = 0; i < d; ++i) inv[i][i] = 1.0;
    for (int c = 0; c < d; ++c) {
        int piv = c;
        for (int r = c + 1; r < d; ++r)
            if (fabs(a[r][c]) > fabs(a[piv][c])) piv = r;
        if (fabs(a[piv][c]) < 1e-10) return false;
        for (int k = 0; k < d; ++k) {
            std::swap(a[c][k], a[piv][k]);
            std::swap(inv[c][k], inv[piv][k]);
        }
        const double f = 1.0 / a[c][c];
        for (int k = 0; k < d; ++k) { a[c][k] *= f; inv[c][k] *= f; }
        for (int r = 0; r < d; ++r) {
            if (r == c) continue;
            const double g = a[r][c];
            if (g == 0.0) continue;
            for (int k = 0; k < d; ++k) { a[r][k] -= g * a[c][k]; inv[r][k] -= g * inv[c][k]; }
        }
    }
    memcpy(a, inv, sizeof(inv));
    return true;
}

struct WignerSampler {
    // fixed, generic sample directions and, per order, the inverse of [Y_l(r_k)]
    double pts[DMAX][3];
    double Ainv[LM + 1][DMAX][DMAX];
    bool ok = true;
    WignerSampler() {
        for (int k = 0; k < DMAX; ++k) {
            // deterministic, well spread directions
            const double zz = -0.93 + 1.86 * (k + 0.37) / DMAX;
            const double ph = 2.399963229728653 * k + 0.41;   // golden angle
            const double s = sqrt(1 - zz * zz);
            pts[k][0] = s * cos(ph); pts[k][1] = s * sin(ph); pts[k][2] = zz;
        }
        for (int l = 0; l <= LM; ++l) {
            const int d = 2 * l + 1;
            double A[DMAX][DMAX] = {};
            for (int k = 0; k < d; ++k) {
                double sh[(LM + 1) * (LM + 1)];
                real_sh(l, pts[k][0], pts[k][1], pts[k][2], sh);
                for (int m = 0; m < d; ++m) A[m][k] = sh[l * l + m];
            }
            ok = ok && invert(A, d);
            memcpy(Ainv[l], A, sizeof(A));
        }
    }
    // D^l(g) for l = 0..lmax;  g is a 3x3 rotation acting on column vectors
    void wigner(const double g[3][3], int lmax, double D[LM + 1][DMAX][DMAX]) const {
        double B[LM + 1][DMAX][DMAX];
        for (int k = 0; k < DMAX; ++k) {
            double r[3];
            for (int i = 0; i < 3; ++i)
                r[i] = g[i][0] * pts[k][0] + g[i][1] * pts[k][1] + g[i][2] * pts[k][2];
            double sh[(LM + 1) * (LM + 1)];
            real_sh(lmax, r[0], r[1], r[2], sh);
            for (int l = 0; l <= lmax; ++l)
                if (k < 2 * l + 1)
                    for (int m = 0; m < 2 * l + 1; ++m) B[l][m][k] = sh[l * l + m];
        }
        for (int l = 0; l <= lmax; ++l) {
            const int d = 2 * l + 1;
            for (int i = 0; i < d; ++i)
                for (int j = 0; j < d; ++j) {
                    double s = 0;
                    for (int k = 0; k < d; ++k) s += B[l][i][k] * Ainv[l][k][j];
                    D[l][i][j] = s;
                }
        }
    }
};

void euler_zyz(double a, double b, double c, double g[3][3]) {
    const double ca = cos(a), sa = sin(a), cb = cos(b), sb = sin(b), cc = cos(c), sc = sin(c);
    // Rz(a) Ry(b) Rz(c)
    g[0][0] = ca * cb * cc - sa * sc; g[0][1] = -ca * cb * sc - sa * cc; g[0][2] = ca * sb;
    g[1][0] = sa * cb * cc + ca * sc; g[1][1] = -sa * cb * sc + ca * cc; g[1][2] = sa * sb;
    g[2][0] = -sb * cc;               g[2][1] = sb * sc;                 g[2][2] = cb;
}

void gauss_legendre(int n, std::vector<double>& x, std::vector<double>& w) {
    x.resize(n); w.resize(n);
    for (int i = 0; i < n; ++i) {
        double z = cos(kPi * (i + 0.75) / (n + 0.5));
        for (int it = 0; it < 100; ++it) {
            double p0 = 1, p1 = z;
            for (int k = 2; k <= n; ++k) { double p2 = ((2 * k - 1) * z * p1 - (k - 1) * p0) / k; p0 = p1; p1 = p2; }
            const double dp = n * (z * p1 - p0) / (z * z - 1);
            const double dz = p1 / dp;
            z -= dz;
            if (fabs(dz) < 1e-15) break;
        }
        double p0 = 1, p1 = z;
        for (int k = 2; k <= n; ++k) { double p2 = ((2 * k - 1) * z * p1 - (k - 1) * p0) / k; p0 = p1; p1 = p2; }
        const double dp = n * (z * p1 - p0) / (z * z - 1);
        x[i] = z;
        w[i] = 2 / ((1 - z * z) * dp * dp);
    }
}

// All invariant tensors needed by `triples` at once (one pass over the quadrature).
bool invariant_tensors(const std::vector<int>& triples /* l1,l2,l3 ... */,
                       std::vector<std::vector<double>>& out) {
    static const WignerSampler ws;
    if (!ws.ok) return false;
    const int nt = (int)triples.size() / 3;
    out.assign(nt, {});
    int Lmax = 0, lmax = 0;
    for (int t = 0; t < nt; ++t) {
        Lmax = std::max(Lmax, triples[3 * t] + triples[3 * t + 1] + triples[3 * t + 2]);
        for (int k = 0; k < 3; ++k) lmax = std::max(lmax, triples[3 * t + k]);
    }
    const int na = Lmax + 2, nb = Lmax / 2 + 2;
    std::vector<double> gx, gw;
    gauss_legendre(nb, gx, gw);
    for (int attempt = 0; attempt < 6; ++attempt) {
        bool all_ok = true;
        std::vector<std::vector<double>> acc(nt);
        std::vector<char> todo(nt, 0);
        for (int t = 0; t < nt; ++t)
            if (out[t].empty()) {
                todo[t] = 1;
                acc[t].assign((2 * triples[3 * t] + 1) * (2 * triples[3 * t + 1] + 1) * (2 * triples[3 * t + 2] + 1), 0.0);
            }
        // seed vectors (deterministic, different for the three slots and per attempt)
        auto seed = [&](int slot, int l, int m) {
            return sin(1.7 * m + 0.9 * l + 2.3 * slot + 0.61 * attempt + 0.3) + 0.25 * cos(0.8 * m * (slot + 1) + attempt);
        };
        for (int ia = 0; ia < na; ++ia)
            for (int ib = 0; ib < nb; ++ib)
                for (int ic = 0; ic < na; ++ic) {
                    double g[3][3];
                    euler_zyz(2 * kPi * ia / na, acos(gx[ib]), 2 * kPi * ic / na, g);
                    double D[LM + 1][DMAX][DMAX];
                    ws.wigner(g, lmax, D);
                    const double wq = 0.5 * gw[ib] / (double(na) * na);
                    for (int t = 0; t < nt; ++t) {
                        if (!todo[t]) continue;
                        const int l1 = triples[3 * t], l2 = triples[3 * t + 1], l3 = triples[3 * t + 2];
                        const int d1 = 2 * l1 + 1, d2 = 2 * l2 + 1, d3 = 2 * l3 + 1;
                        double v1[DMAX], v2[DMAX], v3[DMAX];
                        for (int i = 0; i < d1; ++i) { double s = 0; for (int j = 0; j < d1; ++j) s += D[l1][i][j] * seed(0, l1, j); v1[i] = s; }
                        for (int i = 0; i < d2; ++i) { double s = 0; for (int j = 0; j < d2; ++j) s += D[l2][i][j] * seed(1, l2, j); v2[i] = s; }
                        for (int i = 0; i < d3; ++i) { double s = 0; for (int j = 0; j < d3; ++j) s += D[l3][i][j] * seed(2, l3, j); v3[i] = s; }
                        double* a = acc[t].data();
                        for (int i = 0; i < d1; ++i)
                            for (int j = 0; j < d2; ++j) {
                                const double f = wq * v1[i] * v2[j];
                                for (int k = 0; k < d3; ++k) a[(i * d2 + j) * d3 + k] += f * v3[k];
                            }
                    }
                }
        for (int t = 0; t < nt; ++t) {
            if (!todo[t]) continue;
            double n2 = 0;
            for (double v : acc[t]) n2 += v * v;
            if (n2 < 1e-6) { all_ok = false; continue; }   // seed nearly orthogonal: try another
            const double inv = 1.0 / sqrt(n2);
            double sign = 0;
            for (double& v : acc[t]) {
                v *= inv;
                if (fabs(v) < 1e-11) v = 0.0;
                if (sign == 0 && fabs(v) > 1e-9) sign = v > 0 ? 1.0 : -1.0;
            }
            for (double& v : acc[t]) v *= sign;
            out[t] = acc[t];
        }
        if (all_ok) break;
    }
    for (int t = 0; t < nt; ++t)
        if (out[t].empty()) return false;
    // verify invariance under one generic rotation
    double g[3][3];
    euler_zyz(0.7345, 1.2211, 2.4127, g);
    double D[LM + 1][DMAX][DMAX];
    ws.wigner(g, lmax, D);
    for (int t = 0; t < nt; ++t) {
        const int l1 = triples[3 * t], l2 = triples[3 * t + 1], l3 = triples[3 * t + 2];
        const int d1 = 2 * l1 + 1, d2 = 2 * l2 + 1, d3 = 2 * l3 + 1;
        const double* c = out[t].data();
        double err = 0;
        for (int i = 0; i < d1; ++i)
            for (int j = 0; j < d2; ++j)
                for (int k = 0; k < d3; ++k) {
                    double s = 0;
                    for (int a = 0; a < d1; ++a)
                        for (int b = 0; b < d2; ++b) {
                            const double f = D[l1][i][a] * D[l2][j][b];
                            for (int e = 0; e < d3; ++e) s += f * D[l3][k][e] * c[(a * d2 + b) * d3 + e];
                        }
                    err = std::max(err, fabs(s - c[(i * d2 + j) * d3 + k]));
                }
        if (err > 1e-9) return false;
    }
    return true;
}

template <class T>
cudaError_t upload(const std::vector<T>& h, T** d) {
    *d = nullptr;
    if (h.empty()) return cudaSuccess;
    cudaError_t e = cudaMalloc((void**)d, h.size() * sizeof(T));
    if (e != cudaSuccess) return e;
    return cudaMemcpy(*d, h.data(), h.size() * sizeof(T), cudaMemcpyHostToDevice);
}

// Build one traversal direction.  transposed = 0: groups are output irreps; 1: input irreps.
void build_direction(sobek_plan* p, int transposed, Direction& dir) {
    const auto& dst_ir = transposed ? p->in : p->out;
    dir.C_src = transposed ? p->C_y : p->C_x;
    dir.C_dst = transposed ? p->C_x : p->C_y;
    int64_t z_off = 0, rp_off = 0;
    int dst_off = 0;
    for (int g = 0; g < (int)dst_ir.size(); ++g) {
        const int d_dst = 2 * dst_ir[g].l + 1;
        DGroup G{};
        G.dst_off = dst_off;
        G.c_dst = dst_ir[g].mul;
        G.d_dst = d_dst;
        G.path_begin = (int)dir.paths.size();
        G.wt_begin = (int)dir.wtasks.size();
        int koff = 0, m_off = 0;
        for (const HPath& hp : p->paths) {
            const sobek_path_info& pi = hp.info;
            if ((transposed ? pi.i_in : pi.i_out) != g) continue;
            DPath P{};
            const int d_in = 2 * pi.l_in + 1, d_sh = 2 * pi.l_sh + 1, d_out = 2 * pi.l_out + 1;
            P.src_off = transposed ? pi.out_off : pi.in_off;
            P.c_src = transposed ? pi.c_out : pi.c_in;
            P.d_src = transposed ? d_out : d_in;
            P.sh_off = pi.sh_off;
            P.d_sh = d_sh;
            P.d_dst = d_dst;
            P.c_dst = G.c_dst;
            P.koff = koff;
            P.m_off = m_off;
            P.w_off = pi.w_off;
            P.rp_off = rp_off;
            P.c_in = pi.c_in;
            P.c_out = pi.c_out;
            // sparse tables.  entry = s*d_dst + o with (s, o) = (m_in, m_out) forward and
            // (m_out, m_in) transposed; value c[m_in][m_sh][m_out].
            auto cval = [&](int s, int b, int o) {
                return transposed ? hp.cg[(size_t(o) * d_sh + b) * d_out + s]
                                  : hp.cg[(size_t(s) * d_sh + b) * d_out + o];
            };
            P.tabM = (int)p->tab_ptr.size();
            for (int s = 0; s < P.d_src; ++s)
                for (int o = 0; o < d_dst; ++o) {
                    p->tab_ptr.push_back((int)p->tab_idx.size());
                    for (int b = 0; b < d_sh; ++b) {
                        const double c = cval(s, b, o);
                        if (c != 0.0) { p->tab_idx.push_back(b); p->tab_coef.push_back((float)c); }
                    }
                }
            p->tab_ptr.push_back((int)p->tab_idx.size());
            P.tabY = (int)p->tab_ptr.size();
            for (int b = 0; b < d_sh; ++b) {
                p->tab_ptr.push_back((int)p->tab_idx.size());
                for (int s = 0; s < P.d_src; ++s)
                    for (int o = 0; o < d_dst; ++o) {
                        const double c = cval(s, b, o);
                        if (c != 0.0) { p->tab_idx.push_back(s * d_dst + o); p->tab_coef.push_back((float)c); }
                    }
            }
            p->tab_ptr.push_back((int)p->tab_idx.size());
            for (int u0 = 0; u0 < P.c_src; u0 += 32) dir.wtasks.push_back(WTask{(int)dir.paths.size(), u0});
            koff += p->K * P.c_src;
            m_off += P.d_src * d_dst;
            dir.paths.push_back(P);
        }
        G.path_end = (int)dir.paths.size();
        G.wt_end = (int)dir.wtasks.size();
        G.D = koff;
        G.m_entries = m_off;
        G.z_off = z_off;
        G.rp_off = rp_off;
        dst_off += G.c_dst * d_dst;
        if (G.path_end > G.path_begin) {
            z_off += int64_t(d_dst) * G.D;
            rp_off += int64_t(G.D) * G.c_dst;
            dir.max_m_entries = std::max(dir.max_m_entries, m_off);
        }
        dir.groups.push_back(G);   // groups without paths are kept (their block is zero-filled)
    }
    dir.state_floats = z_off;
    // bf16 operand layouts
    auto r8 = [](int64_t v) { return (v + 7) & ~int64_t(7); };
    dir.path_group.assign(dir.paths.size(), 0);
    for (size_t gi = 0; gi < dir.groups.size(); ++gi) {
        const DGroup& G = dir.groups[gi];
        dir.kn_off.push_back(dir.kn_elems); dir.nk_off.push_back(dir.nk_elems);
        dir.kn_ld.push_back((int32_t)r8(G.c_dst)); dir.nk_ld.push_back((int32_t)r8(G.D));
        dir.zb_off.push_back(dir.zb_elems); dir.gb_off.push_back(dir.gb_elems);
        if (G.path_end == G.path_begin) continue;
        dir.kn_elems += int64_t(G.D) * r8(G.c_dst);
        dir.nk_elems += int64_t(G.c_dst) * r8(G.D);
        dir.zb_elems += int64_t(G.d_dst) * r8(G.D);
        dir.gb_elems += int64_t(G.d_dst) * r8(G.c_dst);
        for (int k = G.path_begin; k < G.path_end; ++k) dir.path_group[k] = (int32_t)gi;
    }
}

}  // namespace

int64_t chunk_nodes(const sobek_plan* p, int64_t N, int order) {
    // bytes per node held at once: the bf16 (hi, lo) state (its adjoint takes the same buffer in turn) and, for
    // orders >= 1, the bf16 (hi, lo) rows of the output adjoint and - FP32-pipe edge pass only - the fp32 adjoint state
    int64_t zb = p->fwd.zb_elems;
    if (order >= 1) zb = std::max(zb, p->tr.zb_elems);
    const bool tc_edge = p->use_tc_edge && p->fwd.etc[0].ok;     // else the edge pass reads an fp32 adjoint state
    int64_t per = 4 * zb + (order >= 1 ? (tc_edge ? 0 : 4 * p->fwd.state_floats) + 4 * p->fwd.gb_elems : 0);
    per = std::max<int64_t>(per, 1);
    // the budget bounds the chunk, but a chunk never has fewer than kMinChunkNodes nodes: below that the
    // node-side kernels cannot fill the machine
    int64_t n = (int64_t)(p->state_budget / (size_t)per);
    n = std::max<int64_t>(n, kMinChunkNodes);
    return std::min<int64_t>(std::max<int64_t>(N, 1), n);
}

}  // namespace sobek

using namespace sobek;

extern "C" int sobek_plan_create(const sobek_irrep* in, int n_in, const sobek_irrep* out, int n_out,
                                 int l_max, int K, uint32_t flags, sobek_plan** plan) {
    if (!in || !out || !plan || n_in < 1 || n_out < 1 || K < 1 || (flags & 0xFFFu & ~uint32_t(SOBEK_FLAG_UVU | SOBEK_FLAG_MUL_IR | SOBEK_FLAG_FAST_GEMM | SOBEK_FLAG_FUSED_FP32 | SOBEK_FLAG_FP32_STREAM | SOBEK_FLAG_FP32_EDGE | SOBEK_FLAG_UVU_STATE)) != 0 || l_max < 0)
        return SOBEK_ERR_INVALID_ARG;
    *plan = nullptr;
    if (l_max > SOBEK_MAX_L) return SOBEK_ERR_UNSUPPORTED;
    for (int i = 0; i < n_in; ++i) {
        if (in[i].mul < 1 || in[i].l < 0 || (in[i].parity != 1 && in[i].parity != -1)) return SOBEK_ERR_INVALID_ARG;
        if (in[i].l > SOBEK_MAX_L) return SOBEK_ERR_UNSUPPORTED;
    }
    for (int i = 0; i < n_out; ++i) {
        if (out[i].mul < 1 || out[i].l < 0 || (out[i].parity != 1 && out[i].parity != -1)) return SOBEK_ERR_INVALID_ARG;
        if (out[i].l > SOBEK_MAX_L) return SOBEK_ERR_UNSUPPORTED;
    }
    sobek_plan* p = new (std::nothrow) sobek_plan();
    if (!p) return SOBEK_ERR_INVALID_ARG;
    p->in.assign(in, in + n_in);
    p->out.assign(out, out + n_out);
    p->l_max = l_max;
    p->K = K;
    p->uvu = (flags & SOBEK_FLAG_UVU) != 0;
    p->mul_ir = (flags & SOBEK_FLAG_MUL_IR) != 0;
    p->gemm_passes = (flags & SOBEK_FLAG_FAST_GEMM) ? 1 : 3;
    p->dim_sh = (l_max + 1) * (l_max + 1);
    std::vector<int> in_off(n_in), out_off(n_out);
    for (int i = 0; i < n_in; ++i) { in_off[i] = p->C_x; p->C_x += in[i].mul * (2 * in[i].l + 1); }
    for (int i = 0; i < n_out; ++i) { out_off[i] = p->C_y; p->C_y += out[i].mul * (2 * out[i].l + 1); }
    // paths in nested order (input irrep, SH order, output irrep), Eq. cg_selection_rules
    std::vector<int> triples;
    for (int ii = 0; ii < n_in; ++ii)
        for (int ls = 0; ls <= l_max; ++ls)
            for (int io = 0; io < n_out; ++io) {
                const int li = in[ii].l, lo = out[io].l;
                const int ps = (ls % 2 == 0) ? 1 : -1;
                if (lo < abs(li - ls) || lo > li + ls || out[io].parity != in[ii].parity * ps) continue;
                HPath hp;
                hp.info = sobek_path_info{ii, ls, io, li, lo, in[ii].mul, out[io].mul, in_off[ii], ls * ls,
                                          out_off[io], p->N_w};
                if (p->uvu) {
                    // tied multiplicities: the instruction needs C_out = C_in and owns C_in weights
                    if (in[ii].mul != out[io].mul) { delete p; return SOBEK_ERR_UNSUPPORTED; }
                    p->N_w += in[ii].mul;
                } else {
                    p->N_w += int64_t(in[ii].mul) * out[io].mul;
                }
                p->paths.push_back(hp);
                triples.push_back(li); triples.push_back(ls); triples.push_back(lo);
            }
    if (p->paths.empty()) { delete p; return SOBEK_ERR_UNSUPPORTED; }
    // unique triples -> invariant tensors
    std::vector<int> uniq;
    std::vector<int> which(p->paths.size());
    for (size_t k = 0; k < p->paths.size(); ++k) {
        int found = -1;
        for (size_t t = 0; t < uniq.size() / 3; ++t)
            if (uniq[3 * t] == triples[3 * k] && uniq[3 * t + 1] == triples[3 * k + 1] && uniq[3 * t + 2] == triples[3 * k + 2]) found = (int)t;
        if (found < 0) {
            found = (int)uniq.size() / 3;
            uniq.insert(uniq.end(), triples.begin() + 3 * k, triples.begin() + 3 * k + 3);
        }
        which[k] = found;
    }
    std::vector<std::vector<double>> tens;
    if (!invariant_tensors(uniq, tens)) { delete p; return SOBEK_ERR_UNSUPPORTED; }
    for (size_t k = 0; k < p->paths.size(); ++k) {
        p->paths[k].cg = tens[which[k]];
        const double nrm = sqrt(2.0 * p->paths[k].info.l_out + 1.0);
        for (double& v : p->paths[k].cg) v *= nrm;
    }
    p->use_fused = (flags & SOBEK_FLAG_FUSED_FP32) != 0 && !p->uvu;   // the fused kernels contain the channel-mixing GEMM
    p->use_tc_stream = (flags & SOBEK_FLAG_FP32_STREAM) == 0;
    p->use_tc_edge = (flags & SOBEK_FLAG_FP32_EDGE) == 0;
    if (const uint32_t mb = flags >> 12) p->state_budget = size_t(mb) << 20;
    build_direction(p, 0, p->fwd);
    build_direction(p, 1, p->tr);
    build_stream_tasks(p, p->fwd);
    build_stream_tasks(p, p->tr);
    build_tc_sets(p, p->fwd);
    build_tc_sets(p, p->tr);
    build_tc_edge_sets(p, p->fwd);
    p->uvu_state = (flags & SOBEK_FLAG_UVU_STATE) != 0;
    build_uvu_direct(p, in, n_in, out, n_out);
    build_edge_tasks(p, p->fwd);
    build_fused_stages(p, p->fwd);
    build_fused_stages(p, p->tr);
    cudaError_t e = cudaGetDevice(&p->device);
    if (e != cudaSuccess) {
        // No CUDA device: the plan stays usable for inspection (info, paths, CG tensors);
        // every sobek_conv_* call on it fails with SOBEK_ERR_CUDA.
        (void)cudaGetLastError();
        p->device = -1;
        *plan = p;
        return SOBEK_OK;
    }
    if (e == cudaSuccess) e = upload(p->tab_ptr, &p->d_tab_ptr);
    if (e == cudaSuccess) e = upload(p->tab_idx, &p->d_tab_idx);
    if (e == cudaSuccess) e = upload(p->tab_coef, &p->d_tab_coef);
    if (p->ud.ok) {
        for (UvuDirectTables& T : p->ud.dir) {
            if (e == cudaSuccess) e = upload(T.woff, &T.d_woff);
            if (e == cudaSuccess) e = upload(T.ent, &T.d_ent);
            if (e == cudaSuccess) e = upload(T.nz, &T.d_nz);
        }
    }
    {
        std::vector<int4> bi, bo;
        for (int i = 0; i < n_in; ++i) bi.push_back(make_int4(in_off[i], in[i].mul, 2 * in[i].l + 1, 0));
        for (int i = 0; i < n_out; ++i) bo.push_back(make_int4(out_off[i], out[i].mul, 2 * out[i].l + 1, 0));
        if (e == cudaSuccess) e = upload(bi, &p->d_in_blocks);
        if (e == cudaSuccess) e = upload(bo, &p->d_out_blocks);
    }
    for (Direction* d : {&p->fwd, &p->tr}) {
        if (e == cudaSuccess) e = upload(d->paths, &d->d_paths);
        if (e == cudaSuccess) e = upload(d->groups, &d->d_groups);
        if (e == cudaSuccess) e = upload(d->wtasks, &d->d_wtasks);
        if (e == cudaSuccess) e = upload(d->kn_off, &d->d_kn_off);
        if (e == cudaSuccess) e = upload(d->nk_off, &d->d_nk_off);
        if (e == cudaSuccess) e = upload(d->kn_ld, &d->d_kn_ld);
        if (e == cudaSuccess) e = upload(d->nk_ld, &d->d_nk_ld);
        if (e == cudaSuccess) e = upload(d->path_group, &d->d_path_group);
        if (e == cudaSuccess) e = upload(d->stasks, &d->d_stasks);
        if (e == cudaSuccess) e = upload(d->scomps, &d->d_scomps);
        if (e == cudaSuccess) e = upload(d->etasks, &d->d_etasks);
        if (e == cudaSuccess) e = upload(d->ecomps, &d->d_ecomps);
        if (e == cudaSuccess) e = upload(d->zb_off, &d->d_zb_off);
        if (e == cudaSuccess) e = upload(d->fstages, &d->d_fstages);
        if (e == cudaSuccess) e = upload(d->fs_begin, &d->d_fs_begin);
        if (e == cudaSuccess) e = upload(d->fs_count, &d->d_fs_count);
        if (e == cudaSuccess) e = upload(d->fk_off, &d->d_fk_off);
        for (TcSets* tp : {&d->tc[0], &d->tc[1], &d->etc[0], &d->etc[1]}) {
            TcSets& t = *tp;
            if (!t.ok) continue;
            if (e == cudaSuccess) e = upload(t.ents_s, &t.d_ents_s);
            if (e == cudaSuccess) e = upload(t.nz, &t.d_nz);
            if (e == cudaSuccess) e = upload(t.comps_s, &t.d_comps_s);
            if (e == cudaSuccess) e = upload(t.slabs, &t.d_slabs);
            if (e == cudaSuccess) e = upload(t.inv_ptr, &t.d_inv_ptr);
            if (e == cudaSuccess) e = upload(t.inv, &t.d_inv);
            if (e == cudaSuccess) e = upload(t.sets, &t.d_sets);
            if (e == cudaSuccess) e = upload(t.units, &t.d_units);
            if (e == cudaSuccess) e = upload(t.blks, &t.d_blks);
            if (e == cudaSuccess) e = upload(t.ents, &t.d_ents);
            if (e == cudaSuccess) e = upload(t.comps, &t.d_comps);
        }
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        sobek_plan_destroy(p);
        return SOBEK_ERR_CUDA;
    }
    // side streams (optional: without them everything runs on the caller's stream)
    if (cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming) == cudaSuccess) {
        for (int i = 0; i < sobek_plan::kSide; ++i) {
            if (cudaStreamCreateWithFlags(&p->side[i], cudaStreamNonBlocking) != cudaSuccess ||
                cudaEventCreateWithFlags(&p->ev_join[i], cudaEventDisableTiming) != cudaSuccess)
                break;
            p->n_side = i + 1;
        }
    }
    (void)cudaGetLastError();
    *plan = p;
    return SOBEK_OK;
}

extern "C" void sobek_plan_destroy(sobek_plan* p) {
    if (!p) return;
    for (int i = 0; i < sobek_plan::kSide; ++i) {
        if (p->side[i]) cudaStreamDestroy(p->side[i]);
        if (p->ev_join[i]) cudaEventDestroy(p->ev_join[i]);
    }
    if (p->ev_fork) cudaEventDestroy(p->ev_fork);
    cudaFree(p->d_tab_ptr); cudaFree(p->d_tab_idx); cudaFree(p->d_tab_coef);
    for (UvuDirectTables& T : p->ud.dir) { cudaFree(T.d_woff); cudaFree(T.d_ent); cudaFree(T.d_nz); }
    cudaFree(p->d_in_blocks); cudaFree(p->d_out_blocks);
    for (Direction* d : {&p->fwd, &p->tr}) {
        cudaFree(d->d_paths); cudaFree(d->d_groups); cudaFree(d->d_wtasks);
        cudaFree(d->d_kn_off); cudaFree(d->d_nk_off); cudaFree(d->d_kn_ld); cudaFree(d->d_nk_ld); cudaFree(d->d_path_group);
        cudaFree(d->d_stasks); cudaFree(d->d_scomps); cudaFree(d->d_etasks); cudaFree(d->d_ecomps); cudaFree(d->d_zb_off);
        cudaFree(d->d_fstages); cudaFree(d->d_fs_begin); cudaFree(d->d_fs_count); cudaFree(d->d_fk_off);
        for (TcSets* tp : {&d->tc[0], &d->tc[1], &d->etc[0], &d->etc[1]}) {
            TcSets& t = *tp;
            cudaFree(t.d_inv_ptr); cudaFree(t.d_inv);
            cudaFree(t.d_ents_s); cudaFree(t.d_nz); cudaFree(t.d_comps_s); cudaFree(t.d_slabs);
            cudaFree(t.d_sets); cudaFree(t.d_units); cudaFree(t.d_blks); cudaFree(t.d_ents); cudaFree(t.d_comps);
        }
    }
    (void)cudaGetLastError();
    delete p;
}

extern "C" int sobek_plan_info(const sobek_plan* p, sobek_info* info) {
    if (!p || !info) return SOBEK_ERR_INVALID_ARG;
    info->C_x = p->C_x; info->C_y = p->C_y; info->dim_sh = p->dim_sh; info->K = p->K;
    info->n_paths = (int)p->paths.size(); info->l_max = p->l_max; info->N_w = p->N_w;
    info->state_floats_fwd = p->fwd.state_floats; info->state_floats_bwd = p->tr.state_floats;
    return SOBEK_OK;
}

extern "C" int sobek_plan_path(const sobek_plan* p, int path, sobek_path_info* info) {
    if (!p || !info || path < 0 || path >= (int)p->paths.size()) return SOBEK_ERR_INVALID_ARG;
    *info = p->paths[path].info;
    return SOBEK_OK;
}

extern "C" int sobek_plan_cg(const sobek_plan* p, int path, double* dense) {
    if (!p || !dense || path < 0 || path >= (int)p->paths.size()) return SOBEK_ERR_INVALID_ARG;
    memcpy(dense, p->paths[path].cg.data(), p->paths[path].cg.size() * sizeof(double));
    return SOBEK_OK;
}

extern "C" const char* sobek_status_string(int s) {
    switch (s) {
        case SOBEK_OK: return "ok";
        case SOBEK_ERR_INVALID_ARG: return "invalid argument";
        case SOBEK_ERR_UNSUPPORTED: return "unsupported descriptor";
        case SOBEK_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case SOBEK_ERR_GRAPH: return "graph is not a valid receiver-sorted CSR";
        case SOBEK_ERR_NEED_TRANSPOSE: return "sender-sorted view required";
        case SOBEK_ERR_CUDA: return "CUDA error";
        case SOBEK_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}
