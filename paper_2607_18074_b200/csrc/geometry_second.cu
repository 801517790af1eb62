// Second-order geometry: what the double backward needs when the derivative with respect to the edge vectors
// themselves is wanted (h_rvec = d Phi / d rvec for Phi = <vx, gx> + <v_r, g_r> + <vR, gR>, the adjoints of the
// geometry-mode backward; Table memory_complexity "stored or recomputed", Eq. energy_force_symmetry).
//
//   h_rvec_e = J_Y^T hY_e + J_phi^T hphi_e + d/dr [ <J_Y(r) v_e, gY_e> + <J_phi(r) v_e, gphi_e> ]   (gY, gphi held fixed)
//
// with hY, hphi the second-order and gY, gphi the first-order edge adjoints of the convolution on the inputs
// Y_e = Y(r_e), phi_e = phi(|r_e|) and the directions vY_e = J_Y v_e, vphi_e = J_phi v_e.  Nothing here is differentiated
// by hand: the spherical harmonics and the radial bases are evaluated in hyper-dual arithmetic
//   a + a1 e1 + a2 e2 + a12 e1 e2,   e1^2 = e2^2 = 0,
// at r_e + e1 v_e + e2 u_j (u_j a coordinate direction).  The e1 part of Y is J_Y v (the direction the double backward
// takes), its e2 part is dY / dr_j and its e1 e2 part is u_j^T (d^2 Y / dr^2) v, so that
//   h_rvec_e[j] = sum_b (Y_b.e2 hY_b + Y_b.e12 gY_b) + sum_q (phi_q.e2 hphi_q + phi_q.e12 gphi_q).
// Two elementwise kernels around the stored-input calls of the library: k_geo_edge_inputs writes Y, phi, vY, vphi of every
// edge, k_geo_second_adjoint folds the four edge adjoints into h_rvec.  The harmonics follow the same Cartesian
// recurrences as the in-kernel geometry (A_m + i B_m = (x + iy)^m, Q_l^m by the three-term recurrence in z; component
// normalisation, no Condon-Shortley sign, index l*l + l + m), written over a number type.
#include <cuda_runtime.h>

#include <algorithm>

#include "internal.h"

namespace sobek {
namespace {

constexpr int LMAX2 = 4;                 // as in the in-kernel geometry
constexpr int DSH2 = (LMAX2 + 1) * (LMAX2 + 1);
constexpr int KMAX2 = 32;

struct HD {                              // hyper-dual number
    float v, d1, d2, d12;
};
__device__ __forceinline__ HD hd(float v) { return HD{v, 0.f, 0.f, 0.f}; }
__device__ __forceinline__ HD operator+(HD a, HD b) { return HD{a.v + b.v, a.d1 + b.d1, a.d2 + b.d2, a.d12 + b.d12}; }
__device__ __forceinline__ HD operator-(HD a, HD b) { return HD{a.v - b.v, a.d1 - b.d1, a.d2 - b.d2, a.d12 - b.d12}; }
__device__ __forceinline__ HD operator*(HD a, HD b) {
    return HD{a.v * b.v, a.d1 * b.v + a.v * b.d1, a.d2 * b.v + a.v * b.d2, a.d12 * b.v + a.d1 * b.d2 + a.d2 * b.d1 + a.v * b.d12};
}
__device__ __forceinline__ HD operator*(float s, HD a) { return HD{s * a.v, s * a.d1, s * a.d2, s * a.d12}; }
// f(a) for a scalar function with value f0, first derivative f1 and second derivative f2 at a.v
__device__ __forceinline__ HD chain(HD a, float f0, float f1, float f2) {
    return HD{f0, f1 * a.d1, f1 * a.d2, f1 * a.d12 + f2 * a.d1 * a.d2};
}
__device__ __forceinline__ HD hd_inv(HD a) { const float i = 1.f / a.v; return chain(a, i, -i * i, 2.f * i * i * i); }
__device__ __forceinline__ HD hd_sqrt(HD a) { const float s = sqrtf(a.v); return chain(a, s, 0.5f / s, -0.25f / (s * a.v)); }
__device__ __forceinline__ HD hd_sin(HD a) { float s, c; sincosf(a.v, &s, &c); return chain(a, s, c, -s); }
__device__ __forceinline__ HD hd_exp(HD a) { const float e = expf(a.v); return chain(a, e, e, e); }

__device__ __forceinline__ float norm_lm(int l, int m) {      // sqrt((2l+1) (l-m)! / (l+m)!), times sqrt(2) for m > 0
    double f = 2.0 * l + 1.0;
    for (int k = l - m + 1; k <= l + m; ++k) f /= (double)k;
    return (float)sqrt(m > 0 ? 2.0 * f : f);
}

// Y[b] for b < (l_max+1)^2 at the edge vector (rx, ry, rz) (any length > 0)
__device__ void sh_eval(HD rx, HD ry, HD rz, int l_max, HD* Y) {
    const HD il = hd_inv(hd_sqrt(rx * rx + ry * ry + rz * rz));
    const HD x = rx * il, y = ry * il, z = rz * il;
    HD A[LMAX2 + 1], B[LMAX2 + 1];
    A[0] = hd(1.f); B[0] = hd(0.f);
    for (int m = 1; m <= l_max; ++m) { A[m] = x * A[m - 1] - y * B[m - 1]; B[m] = y * A[m - 1] + x * B[m - 1]; }
    for (int m = 0; m <= l_max; ++m) {
        HD q2 = hd(0.f), q1 = hd(0.f);                       // Q_{l-2}^m, Q_{l-1}^m
        for (int l = m; l <= l_max; ++l) {
            HD q;
            if (l == m) {
                float dfact = 1.f;
                for (int k = 1; k <= m; ++k) dfact *= (float)(2 * k - 1);
                q = hd(dfact);
            } else if (l == m + 1) {
                q = (float)(2 * m + 1) * (z * q1);
            } else {
                q = (1.f / (float)(l - m)) * ((float)(2 * l - 1) * (z * q1) - (float)(l + m - 1) * q2);
            }
            const float c = norm_lm(l, m);
            const int b0 = l * l + l;
            if (m == 0) Y[b0] = c * q;
            else { Y[b0 + m] = c * (q * A[m]); Y[b0 - m] = c * (q * B[m]); }
            q2 = q1; q1 = q;
        }
    }
}

// phi[q] for q < K at the length r: the two radial bases of the geometry front end
__device__ void radial_eval(HD r, int K, float r_c, int basis, int p, HD* phi) {
    if (basis == SOBEK_BASIS_BESSEL) {
        const HD d = (1.f / r_c) * r, ir = hd_inv(r);
        HD dp = hd(1.f);                                      // d^p
        for (int k = 0; k < p; ++k) dp = dp * d;
        const float fp = (float)p;
        const HD u = hd(1.f) - (0.5f * (fp + 1.f) * (fp + 2.f)) * dp + (fp * (fp + 2.f)) * (dp * d) - (0.5f * fp * (fp + 1.f)) * (dp * d * d);
        const float w = 3.14159265358979323846f / r_c, nrm = sqrtf(2.f / r_c);
        for (int q = 0; q < K; ++q) phi[q] = nrm * (hd_sin(((float)(q + 1) * w) * r) * ir * u);
    } else {
        const float step = r_c / (float)(K > 1 ? K - 1 : 1), i2 = 1.f / (step * step);
        for (int q = 0; q < K; ++q) {
            const HD t = r - hd((float)q * step);
            phi[q] = hd_exp((-0.5f * i2) * (t * t));
        }
    }
}

__global__ void k_geo_edge_inputs(const float* __restrict__ rvec, const float* __restrict__ vrvec, int64_t E, int l_max, int K,
                                  float r_c, int basis, int p, float* __restrict__ Y, float* __restrict__ phi,
                                  float* __restrict__ vY, float* __restrict__ vphi) {
    const int dsh = (l_max + 1) * (l_max + 1);
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < E; e += (int64_t)gridDim.x * blockDim.x) {
        const float* r = rvec + 3 * e;
        const float v0 = vrvec ? vrvec[3 * e] : 0.f, v1 = vrvec ? vrvec[3 * e + 1] : 0.f, v2 = vrvec ? vrvec[3 * e + 2] : 0.f;
        const HD rx{r[0], v0, 0.f, 0.f}, ry{r[1], v1, 0.f, 0.f}, rz{r[2], v2, 0.f, 0.f};
        HD y[DSH2], f[KMAX2];
        sh_eval(rx, ry, rz, l_max, y);
        radial_eval(hd_sqrt(rx * rx + ry * ry + rz * rz), K, r_c, basis, p, f);
        for (int b = 0; b < dsh; ++b) { Y[e * dsh + b] = y[b].v; vY[e * dsh + b] = y[b].d1; }
        for (int q = 0; q < K; ++q) { phi[e * K + q] = f[q].v; vphi[e * K + q] = f[q].d1; }
    }
}

__global__ void k_geo_second_adjoint(const float* __restrict__ rvec, const float* __restrict__ vrvec, int64_t E, int l_max, int K,
                                     float r_c, int basis, int p, const float* __restrict__ gY, const float* __restrict__ gphi,
                                     const float* __restrict__ hY, const float* __restrict__ hphi, float* __restrict__ h_rvec) {
    const int dsh = (l_max + 1) * (l_max + 1);
    // thread <-> (edge, coordinate j)
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < 3 * E; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t e = i / 3;
        const int j = (int)(i - 3 * e);
        const float* r = rvec + 3 * e;
        const float v0 = vrvec ? vrvec[3 * e] : 0.f, v1 = vrvec ? vrvec[3 * e + 1] : 0.f, v2 = vrvec ? vrvec[3 * e + 2] : 0.f;
        const HD rx{r[0], v0, j == 0 ? 1.f : 0.f, 0.f}, ry{r[1], v1, j == 1 ? 1.f : 0.f, 0.f}, rz{r[2], v2, j == 2 ? 1.f : 0.f, 0.f};
        HD y[DSH2], f[KMAX2];
        sh_eval(rx, ry, rz, l_max, y);
        radial_eval(hd_sqrt(rx * rx + ry * ry + rz * rz), K, r_c, basis, p, f);
        float s = 0.f;
        for (int b = 0; b < dsh; ++b) s += y[b].d2 * hY[e * dsh + b] + y[b].d12 * gY[e * dsh + b];
        for (int q = 0; q < K; ++q) s += f[q].d2 * hphi[e * K + q] + f[q].d12 * gphi[e * K + q];
        h_rvec[i] = s;
    }
}

int grid_for_edges(int64_t n) { return (int)std::max<int64_t>(1, std::min<int64_t>((n + 127) / 128, 148 * 8)); }

}  // namespace

bool geo_second_supported(int l_max, int K) { return l_max >= 0 && l_max <= LMAX2 && K >= 1 && K <= KMAX2; }

cudaError_t launch_geo_edge_inputs(const float* rvec, const float* vrvec, int64_t E, int l_max, int K, float r_c, int basis, int p,
                                   float* Y, float* phi, float* vY, float* vphi, cudaStream_t s) {
    if (E <= 0) return cudaSuccess;
    k_geo_edge_inputs<<<grid_for_edges(E), 128, 0, s>>>(rvec, vrvec, E, l_max, K, r_c, basis, p, Y, phi, vY, vphi);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_geo_second_adjoint(const float* rvec, const float* vrvec, int64_t E, int l_max, int K, float r_c, int basis,
                                      int p, const float* gY, const float* gphi, const float* hY, const float* hphi,
                                      float* h_rvec, cudaStream_t s) {
    if (E <= 0) return cudaSuccess;
    k_geo_second_adjoint<<<grid_for_edges(3 * E), 128, 0, s>>>(rvec, vrvec, E, l_max, K, r_c, basis, p, gY, gphi, hY, hphi, h_rvec);
    count_launch();
    return cudaGetLastError();
}

}  // namespace sobek
