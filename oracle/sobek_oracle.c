/*
 * TEST INFRASTRUCTURE -- fp64 CPU oracle of the edge-conditioned tensor-product
 * convolution in its conventional MATERIALISED form.  Not part of the product; it
 * shares no code with the CUDA library and is only called by the tests, the smoke
 * check and the benchmark's CPU-baseline leg.
 *
 * What it computes, in the paper's order and with nothing reassociated:
 *   O1  W_e[pi,a]   = sum_q phi_e[q] A[q,pi,a]                 (Eq. radial_projection_background)
 *   O2  M_e         = sum_pi sum_a W_e[pi,a] T_{pi,a}(x_j, Y_e)  (Eq. uvw_connection; the
 *       angular contribution T is the CG coupling of Eq. angular_path_contraction)
 *   O3  m_i         = sum_{e into i} M_e                       (Eq. standard_tpconv_background)
 *   O4  first-order adjoints via h_e = <mbar_i, T>              (Eqs. streamed_weight_adjoint,
 *       streamed_radial_adjoints, streamed_operand_adjoints), with the full rows W_e and
 *       h_e (= the edge-weight adjoint) materialised per edge
 *   O5  second order by the product rule on O4 (Eqs. streamed_directional_terms ..
 *       streamed_operand_second_adjoints) with the direction on the output adjoint set
 *       to zero: the routine returns the vector-Jacobian product of the backward map.
 *
 * Notation: x = node features, Y = spherical harmonics, phi = radial embedding,
 * A (named R at the library boundary) = radial projection, gy = mbar.
 * Layouts: features [N, C] in ir_mul order (block offset + m*mult + u); Y [E, dsh];
 * phi [E, K]; A [K, N_w] with column w_off(pi) + u*C_out + w.
 *
 * Channelwise mode (Eq. uvu_connection): a path marked `tied` couples input multiplicity u
 * only to output multiplicity u (C_out = C_in) and owns C_in weights, column w_off(pi) + u.
 * Every loop over the output multiplicity w below then runs over the single value w = u.
 *
 * Every routine works on a list of ACTIVE RECEIVERS: only edges into those nodes are
 * visited.  With the full list this is the whole operator; with a sample it gives the
 * rows of y / the edge outputs for that sample, and the node/parameter adjoints that
 * an output adjoint supported on the sample produces.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int64_t in_off, c_in, d_in, sh_off, d_sh, out_off, c_out, d_out, w_off, cg_off, tied;
} opath;

/* range of output multiplicities coupled to input multiplicity u, and the weight column of (u, w) */
static int64_t w_lo(const opath* p, int64_t u) { return p->tied ? u : 0; }
static int64_t w_hi(const opath* p, int64_t u) { return p->tied ? u + 1 : p->c_out; }
static int64_t w_col(const opath* p, int64_t u, int64_t w) {
    return p->tied ? p->w_off + u : p->w_off + u * p->c_out + w;
}

static int nthreads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int oracle_threads(void) { return nthreads(); }

/* t[u*d_out + o] = sum_{a,b} c[a,b,o] xs[a*c_in + u] Ys[b]   (angular contraction) */
static void angular(const opath* p, const double* cg, const double* xs, const double* Ys,
                    double* t) {
    const double* c = cg + p->cg_off;
    for (int64_t u = 0; u < p->c_in; ++u)
        for (int64_t o = 0; o < p->d_out; ++o) {
            double s = 0.0;
            for (int64_t a = 0; a < p->d_in; ++a)
                for (int64_t b = 0; b < p->d_sh; ++b)
                    s += c[(a * p->d_sh + b) * p->d_out + o] * xs[a * p->c_in + u] * Ys[b];
            t[u * p->d_out + o] = s;
        }
}

static void radial_row(int64_t K, int64_t N_w, const double* phi_e, const double* A, double* W) {
    for (int64_t n = 0; n < N_w; ++n) W[n] = 0.0;
    for (int64_t q = 0; q < K; ++q)
        for (int64_t n = 0; n < N_w; ++n) W[n] += phi_e[q] * A[q * N_w + n];
}

static int64_t max_t(const opath* P, int64_t np) {
    int64_t m = 1;
    for (int64_t k = 0; k < np; ++k) {
        int64_t v = P[k].c_in * (P[k].d_out > P[k].d_in ? P[k].d_out : P[k].d_in);
        if (v > m) m = v;
    }
    return m;
}

/* ---------------------------------------------------------------- forward */
void oracle_fwd(int64_t n_act, const int64_t* act, const int64_t* row_ptr, const int32_t* col,
                int64_t np, const opath* P, const double* cg,
                int64_t C_x, int64_t C_y, int64_t dsh, int64_t K, int64_t N_w,
                const double* x, const double* Y, const double* phi, const double* A,
                double* y /* [N, C_y], rows of active receivers are overwritten */) {
    const int64_t mt = max_t(P, np);
#pragma omp parallel
    {
        double* W = (double*)malloc(sizeof(double) * (size_t)N_w);
        double* M = (double*)malloc(sizeof(double) * (size_t)C_y);
        double* t = (double*)malloc(sizeof(double) * (size_t)mt);
#pragma omp for schedule(dynamic, 4)
        for (int64_t r = 0; r < n_act; ++r) {
            const int64_t i = act[r];
            double* yi = y + i * C_y;
            for (int64_t c = 0; c < C_y; ++c) yi[c] = 0.0;
            for (int64_t e = row_ptr[i]; e < row_ptr[i + 1]; ++e) {
                const int64_t j = col[e];
                radial_row(K, N_w, phi + e * K, A, W);                       /* O1 */
                for (int64_t c = 0; c < C_y; ++c) M[c] = 0.0;
                for (int64_t k = 0; k < np; ++k) {                           /* O2 */
                    const opath* p = P + k;
                    angular(p, cg, x + j * C_x + p->in_off, Y + e * dsh + p->sh_off, t);
                    for (int64_t u = 0; u < p->c_in; ++u)
                        for (int64_t w = w_lo(p, u); w < w_hi(p, u); ++w) {
                            const double Wuw = W[w_col(p, u, w)];
                            for (int64_t o = 0; o < p->d_out; ++o)
                                M[p->out_off + o * p->c_out + w] += Wuw * t[u * p->d_out + o];
                        }
                }
                for (int64_t c = 0; c < C_y; ++c) yi[c] += M[c];             /* O3 */
            }
        }
        free(W); free(M); free(t);
    }
}

/* ---------------------------------------------------------------- backward */
void oracle_bwd(int64_t n_act, const int64_t* act, const int64_t* row_ptr, const int32_t* col,
                int64_t np, const opath* P, const double* cg,
                int64_t C_x, int64_t C_y, int64_t dsh, int64_t K, int64_t N_w,
                const double* x, const double* Y, const double* phi, const double* A,
                const double* gy,
                double* gx   /* [N, C_x]  accumulated into (caller zeroes) */,
                double* gY   /* [E, dsh]  rows of visited edges overwritten */,
                double* gphi /* [E, K]    rows of visited edges overwritten */,
                double* gA   /* [K, N_w]  accumulated into (caller zeroes) */) {
    const int64_t mt = max_t(P, np);
    const int nt = nthreads();
    double* gA_all = (double*)calloc((size_t)nt * (size_t)K * (size_t)N_w, sizeof(double));
#pragma omp parallel
    {
#ifdef _OPENMP
        double* gAt = gA_all + (size_t)omp_get_thread_num() * (size_t)K * (size_t)N_w;
#else
        double* gAt = gA_all;
#endif
        double* W = (double*)malloc(sizeof(double) * (size_t)N_w);
        double* h = (double*)malloc(sizeof(double) * (size_t)N_w);
        double* t = (double*)malloc(sizeof(double) * (size_t)mt);
        double* s = (double*)malloc(sizeof(double) * (size_t)mt);
#pragma omp for schedule(dynamic, 4)
        for (int64_t r = 0; r < n_act; ++r) {
            const int64_t i = act[r];
            const double* gyi = gy + i * C_y;
            for (int64_t e = row_ptr[i]; e < row_ptr[i + 1]; ++e) {
                const int64_t j = col[e];
                const double* xj = x + j * C_x;
                const double* Ye = Y + e * dsh;
                radial_row(K, N_w, phi + e * K, A, W);
                for (int64_t b = 0; b < dsh; ++b) gY[e * dsh + b] = 0.0;
                for (int64_t k = 0; k < np; ++k) {
                    const opath* p = P + k;
                    const double* c = cg + p->cg_off;
                    angular(p, cg, xj + p->in_off, Ye + p->sh_off, t);
                    for (int64_t u = 0; u < p->c_in; ++u) {
                        /* h = <mbar_i, T_{pi,(u,w)}>  and  s = sum_w W mbar (weighted adjoint
                           of the angular contraction) */
                        for (int64_t o = 0; o < p->d_out; ++o) s[u * p->d_out + o] = 0.0;
                        for (int64_t w = w_lo(p, u); w < w_hi(p, u); ++w) {
                            double acc = 0.0;
                            const double Wuw = W[w_col(p, u, w)];
                            for (int64_t o = 0; o < p->d_out; ++o) {
                                const double g = gyi[p->out_off + o * p->c_out + w];
                                acc += g * t[u * p->d_out + o];
                                s[u * p->d_out + o] += Wuw * g;
                            }
                            h[w_col(p, u, w)] = acc;
                        }
                        /* operand adjoints: D_x T^* and D_Y T^* applied to s */
                        for (int64_t a = 0; a < p->d_in; ++a) {
                            double gxa = 0.0;
                            for (int64_t b = 0; b < p->d_sh; ++b)
                                for (int64_t o = 0; o < p->d_out; ++o) {
                                    const double cc = c[(a * p->d_sh + b) * p->d_out + o];
                                    gxa += cc * Ye[p->sh_off + b] * s[u * p->d_out + o];
                                    gY[e * dsh + p->sh_off + b] +=
                                        cc * xj[p->in_off + a * p->c_in + u] * s[u * p->d_out + o];
                                }
#pragma omp atomic
                            gx[j * C_x + p->in_off + a * p->c_in + u] += gxa;
                        }
                    }
                }
                for (int64_t q = 0; q < K; ++q) {
                    const double pq = phi[e * K + q];
                    double acc = 0.0;
                    for (int64_t n = 0; n < N_w; ++n) {
                        gAt[q * N_w + n] += pq * h[n];
                        acc += A[q * N_w + n] * h[n];
                    }
                    gphi[e * K + q] = acc;
                }
            }
        }
        free(W); free(h); free(t); free(s);
    }
    for (int tt = 0; tt < nt; ++tt)
        for (int64_t n = 0; n < K * N_w; ++n) gA[n] += gA_all[(size_t)tt * (size_t)K * (size_t)N_w + n];
    free(gA_all);
}

/* ---------------------------------------------------------------- double backward
 * Directions (vx, vY, vphi, vA) on the four inputs; the direction on gy is zero.
 * Outputs: ggy = m-dot; hx, hY, hphi, hA = the directional derivatives of the four
 * first-order adjoints. */
void oracle_dbwd(int64_t n_act, const int64_t* act, const int64_t* row_ptr, const int32_t* col,
                 int64_t np, const opath* P, const double* cg,
                 int64_t C_x, int64_t C_y, int64_t dsh, int64_t K, int64_t N_w,
                 const double* x, const double* Y, const double* phi, const double* A,
                 const double* gy,
                 const double* vx, const double* vY, const double* vphi, const double* vA,
                 double* ggy  /* [N, C_y] rows of active receivers overwritten */,
                 double* hx   /* [N, C_x] accumulated into */,
                 double* hY   /* [E, dsh] visited rows overwritten */,
                 double* hphi /* [E, K]   visited rows overwritten */,
                 double* hA   /* [K, N_w] accumulated into */) {
    const int64_t mt = max_t(P, np);
    const int nt = nthreads();
    double* hA_all = (double*)calloc((size_t)nt * (size_t)K * (size_t)N_w, sizeof(double));
#pragma omp parallel
    {
#ifdef _OPENMP
        double* hAt = hA_all + (size_t)omp_get_thread_num() * (size_t)K * (size_t)N_w;
#else
        double* hAt = hA_all;
#endif
        double* W = (double*)malloc(sizeof(double) * (size_t)N_w);
        double* dW = (double*)malloc(sizeof(double) * (size_t)N_w);
        double* tmpW = (double*)malloc(sizeof(double) * (size_t)N_w);
        double* h = (double*)malloc(sizeof(double) * (size_t)N_w);
        double* dh = (double*)malloc(sizeof(double) * (size_t)N_w);
        double* t = (double*)malloc(sizeof(double) * (size_t)mt);
        double* dt = (double*)malloc(sizeof(double) * (size_t)mt);
        double* t2 = (double*)malloc(sizeof(double) * (size_t)mt);
        double* s = (double*)malloc(sizeof(double) * (size_t)mt);
        double* ds = (double*)malloc(sizeof(double) * (size_t)mt);
#pragma omp for schedule(dynamic, 4)
        for (int64_t r = 0; r < n_act; ++r) {
            const int64_t i = act[r];
            const double* gyi = gy + i * C_y;
            double* ggyi = ggy + i * C_y;
            for (int64_t c = 0; c < C_y; ++c) ggyi[c] = 0.0;
            for (int64_t e = row_ptr[i]; e < row_ptr[i + 1]; ++e) {
                const int64_t j = col[e];
                const double *xj = x + j * C_x, *vxj = vx + j * C_x;
                const double *Ye = Y + e * dsh, *vYe = vY + e * dsh;
                /* w and w-dot (Eq. streamed_directional_terms) */
                radial_row(K, N_w, phi + e * K, A, W);
                radial_row(K, N_w, vphi + e * K, A, dW);
                radial_row(K, N_w, phi + e * K, vA, tmpW);
                for (int64_t n = 0; n < N_w; ++n) dW[n] += tmpW[n];
                for (int64_t b = 0; b < dsh; ++b) hY[e * dsh + b] = 0.0;
                for (int64_t k = 0; k < np; ++k) {
                    const opath* p = P + k;
                    const double* c = cg + p->cg_off;
                    /* T and T-dot = D_x T[vx] + D_Y T[vY] */
                    angular(p, cg, xj + p->in_off, Ye + p->sh_off, t);
                    angular(p, cg, vxj + p->in_off, Ye + p->sh_off, dt);
                    angular(p, cg, xj + p->in_off, vYe + p->sh_off, t2);
                    for (int64_t n = 0; n < p->c_in * p->d_out; ++n) dt[n] += t2[n];
                    for (int64_t u = 0; u < p->c_in; ++u) {
                        for (int64_t o = 0; o < p->d_out; ++o) {
                            s[u * p->d_out + o] = 0.0;
                            ds[u * p->d_out + o] = 0.0;
                        }
                        for (int64_t w = w_lo(p, u); w < w_hi(p, u); ++w) {
                            const int64_t n = w_col(p, u, w);
                            double a0 = 0.0, a1 = 0.0;
                            for (int64_t o = 0; o < p->d_out; ++o) {
                                const int64_t yo = p->out_off + o * p->c_out + w;
                                const double g = gyi[yo];
                                /* m-dot = w-dot T + w T-dot */
                                ggyi[yo] += dW[n] * t[u * p->d_out + o] + W[n] * dt[u * p->d_out + o];
                                a0 += g * t[u * p->d_out + o];
                                a1 += g * dt[u * p->d_out + o];
                                s[u * p->d_out + o] += W[n] * g;
                                ds[u * p->d_out + o] += dW[n] * g;
                            }
                            h[n] = a0;   /* h     = <mbar, T>      */
                            dh[n] = a1;  /* h-dot = <mbar, T-dot>  */
                        }
                        /* x-bar-dot and Y-bar-dot = w-dot B + w B-dot: B^x = D_xT^* mbar depends on
                           Y, B^Y = D_YT^* mbar depends on x; s = w*mbar, ds = w-dot*mbar. */
                        for (int64_t a = 0; a < p->d_in; ++a) {
                            double hxa = 0.0;
                            const double xa = xj[p->in_off + a * p->c_in + u];
                            const double vxa = vxj[p->in_off + a * p->c_in + u];
                            for (int64_t b = 0; b < p->d_sh; ++b)
                                for (int64_t o = 0; o < p->d_out; ++o) {
                                    const double cc = c[(a * p->d_sh + b) * p->d_out + o];
                                    const double so = s[u * p->d_out + o], dso = ds[u * p->d_out + o];
                                    hxa += cc * (Ye[p->sh_off + b] * dso + vYe[p->sh_off + b] * so);
                                    hY[e * dsh + p->sh_off + b] += cc * (xa * dso + vxa * so);
                                }
#pragma omp atomic
                            hx[j * C_x + p->in_off + a * p->c_in + u] += hxa;
                        }
                    }
                }
                /* A-bar-dot and phi-bar-dot (Eq. streamed_radial_second_adjoints) */
                for (int64_t q = 0; q < K; ++q) {
                    const double pq = phi[e * K + q], vpq = vphi[e * K + q];
                    double acc = 0.0;
                    for (int64_t n = 0; n < N_w; ++n) {
                        hAt[q * N_w + n] += vpq * h[n] + pq * dh[n];
                        acc += vA[q * N_w + n] * h[n] + A[q * N_w + n] * dh[n];
                    }
                    hphi[e * K + q] = acc;
                }
            }
        }
        free(W); free(dW); free(tmpW); free(h); free(dh); free(t); free(dt); free(t2); free(s); free(ds);
    }
    for (int tt = 0; tt < nt; ++tt)
        for (int64_t n = 0; n < K * N_w; ++n) hA[n] += hA_all[(size_t)tt * (size_t)K * (size_t)N_w + n];
    free(hA_all);
}
