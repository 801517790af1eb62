// Edge inputs recomputed from the edge vector r_e = pos[sender] - pos[receiver] inside the edge kernels
// (Table memory_complexity: the spherical harmonics are "stored or recomputed"; Section "Peak memory"):
// Y_e = real spherical harmonics of r_e / |r_e| (component normalisation, sum_m Y_lm^2 = 2l+1, no Condon-Shortley
// sign, index l*l + l + m, negative m = sine branch) and phi_e = radial basis of |r_e|; and the way back,
// g_r = J_Y^T gY + J_phi^T gphi, which is what reaches the positions (forces, Eq. energy_force_symmetry).
//
// Cartesian route, no trigonometry for the angular part: with the unit vector (x, y, z),
//   s^m cos(m az) = A_m = Re (x + iy)^m,   s^m sin(m az) = B_m = Im (x + iy)^m,   P_l^m(z) = s^m Q_l^m(z),
//   Q_m^m = (2m-1)!!,  Q_{m+1}^m = (2m+1) z Q_m^m,  (l-m) Q_l^m = (2l-1) z Q_{l-1}^m - (l+m-1) Q_{l-2}^m,
// so that Y_{l,m} = c_lm Q_l^m A_m, Y_{l,-m} = c_lm Q_l^m B_m, Y_{l,0} = c_l0 Q_l^0.  These expressions extend Y off
// the unit sphere; the gradient with respect to r_e is the tangential part of the extension's gradient over |r_e|:
//   grad_r Y(r / |r|) = (I - u u^T) grad F(u) / |r|.
#pragma once
#include <cuda_runtime.h>

namespace sobek {

constexpr int GEO_LMAX = 4;
constexpr int GEO_DSH = (GEO_LMAX + 1) * (GEO_LMAX + 1);
enum { GEO_BESSEL = 0, GEO_GAUSSIAN = 1 };

// c_lm = sqrt((2l+1) (l-m)! / (l+m)!), times sqrt(2) for m > 0
__device__ __forceinline__ float geo_c(int l, int m) {
    constexpr float c[5][5] = {
        {1.0f, 0.f, 0.f, 0.f, 0.f},
        {1.7320508075688772f, 1.7320508075688772f, 0.f, 0.f, 0.f},
        {2.23606797749979f, 1.2909944487358058f, 0.6454972243679029f, 0.f, 0.f},
        {2.6457513110645907f, 1.0801234497346435f, 0.34156502553198664f, 0.13944333775567927f, 0.f},
        {3.0f, 0.9486832980505139f, 0.223606797749979f, 0.05976143046671968f, 0.021128856368212916f}};
    return c[l][m];
}

// emit(b, Y_b, Gx, Gy, Gz) for every b < (GEO_LMAX+1)^2 of the unit vector (x, y, z): the harmonic and the gradient
// of its extension (still to be projected on the tangent plane and divided by |r|).  Fully unrolled: b is a constant
// inside emit.
template <class Emit>
__device__ __forceinline__ void geo_sh(float x, float y, float z, Emit&& emit) {
    float A[GEO_LMAX + 1], B[GEO_LMAX + 1];
    A[0] = 1.f; B[0] = 0.f;
#pragma unroll
    for (int m = 1; m <= GEO_LMAX; ++m) { A[m] = x * A[m - 1] - y * B[m - 1]; B[m] = y * A[m - 1] + x * B[m - 1]; }
#pragma unroll
    for (int m = 0; m <= GEO_LMAX; ++m) {
        float q2 = 0.f, q1 = 0.f, d2 = 0.f, d1 = 0.f;      // Q_{l-2}^m, Q_{l-1}^m and their z-derivatives
#pragma unroll
        for (int l = m; l <= GEO_LMAX; ++l) {
            float q, d;
            if (l == m) {
                q = 1.f;
#pragma unroll
                for (int k = 1; k <= m; ++k) q *= (float)(2 * k - 1);
                d = 0.f;
            } else if (l == m + 1) {
                q = (float)(2 * m + 1) * z * q1;
                d = (float)(2 * m + 1) * q1;
            } else {
                const float inv = 1.f / (float)(l - m);
                q = ((float)(2 * l - 1) * z * q1 - (float)(l + m - 1) * q2) * inv;
                d = ((float)(2 * l - 1) * (q1 + z * d1) - (float)(l + m - 1) * d2) * inv;
            }
            const float c = geo_c(l, m);
            const int b0 = l * l + l;
            if (m == 0) {
                emit(b0, c * q, 0.f, 0.f, c * d);
            } else {
                const float fm = (float)m;
                emit(b0 + m, c * q * A[m], c * q * fm * A[m - 1], -c * q * fm * B[m - 1], c * d * A[m]);
                emit(b0 - m, c * q * B[m], c * q * fm * B[m - 1], c * q * fm * A[m - 1], c * d * B[m]);
            }
            q2 = q1; q1 = q; d2 = d1; d1 = d;
        }
    }
}

// Radial basis of the length r: emit(q, f_q, df_q / dr) for q < K.
//   bessel:   sqrt(2 / r_c) sin(n pi r / r_c) / r * u(r / r_c),  n = q + 1,
//             u(d) = 1 - (p+1)(p+2)/2 d^p + p(p+2) d^(p+1) - p(p+1)/2 d^(p+2),  u'(d) = -p(p+1)(p+2)/2 d^(p-1) (1 - d)^2
//   gaussian: exp(-(r - mu_q)^2 / (2 s^2)),  mu_q = q s,  s = r_c / (K - 1)
template <class Emit>
__device__ __forceinline__ void geo_radial(float r, int K, float r_c, int basis, int p, Emit&& emit) {
    if (basis == GEO_BESSEL) {
        const float d = r / r_c, inv_r = 1.f / r;
        float dp1 = 1.f;                                    // d^(p-1)
        for (int k = 1; k < p; ++k) dp1 *= d;
        const float dp = dp1 * d, fp = (float)p;
        const float u = 1.f - 0.5f * (fp + 1.f) * (fp + 2.f) * dp + fp * (fp + 2.f) * dp * d - 0.5f * fp * (fp + 1.f) * dp * d * d;
        const float du = -0.5f * fp * (fp + 1.f) * (fp + 2.f) * dp1 * (1.f - d) * (1.f - d) / r_c;      // du / dr
        const float w = 3.14159265358979323846f / r_c, nrm = sqrtf(2.f / r_c);
        float s1, c1;
        __sincosf(w * r, &s1, &c1);      // argument in (0, pi) for r below the cutoff: absolute error ~ 2^-21
        float sn = s1, cn = c1;                             // sin, cos of n w r by the angle-addition recurrence
#pragma unroll 1
        for (int q = 0; q < K; ++q) {
            const float b = nrm * sn * inv_r;
            emit(q, b * u, (nrm * (float)(q + 1) * w * cn * inv_r - b * inv_r) * u + b * du);
            const float s2 = sn * c1 + cn * s1;
            cn = cn * c1 - sn * s1; sn = s2;
        }
    } else {
        const float step = r_c / (float)(K > 1 ? K - 1 : 1), i2 = 1.f / (step * step);
#pragma unroll 1
        for (int q = 0; q < K; ++q) {
            const float t = r - (float)q * step;
            const float v = expf(-0.5f * t * t * i2);
            emit(q, v, -t * i2 * v);
        }
    }
}

}  // namespace sobek
