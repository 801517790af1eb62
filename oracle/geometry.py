"""TEST INFRASTRUCTURE -- fp64 CPU oracle of the geometry front end of the convolution.

Not part of the product: only the tests, the smoke check and the benchmark's CPU-baseline
leg may import this.  It shares no code with the CUDA library.

The convolution takes the edge inputs Y (spherical harmonics of the edge direction) and phi
(radial embedding of the edge length) as given (Section "Edge-conditioned equivariant tensor
product convolution").  They are edge-sized and "stored or recomputed" (Table memory_complexity);
here they are recomputed from the edge vectors r_e = pos[sender] - pos[receiver], which is also
what carries a gradient back to the positions (forces, Eq. energy_force_symmetry).

The definitions are written out plainly in torch fp64:
  Y_{l,m}(r)  = sqrt(2) N_lm P_l^m(cos theta) cos(m phi)   (m > 0)
  Y_{l,0}(r)  = N_l0 P_l(cos theta)
  Y_{l,-m}(r) = sqrt(2) N_lm P_l^m(cos theta) sin(m phi)   (m > 0)
with N_lm^2 = (2l+1) (l-m)! / (l+m)!  (component normalisation: sum_m Y_lm^2 = 2l+1), P_l^m without the
Condon-Shortley sign, and (theta, phi) the polar angles of r / |r|; index l*l + l + m.
Radial bases (the paper does not fix one; these are the two the synthetic workloads use):
  bessel:   phi_q(r) = sqrt(2 / r_c) sin(q pi r / r_c) / r * u(r / r_c),  q = 1..K,
            u(d) = 1 - (p+1)(p+2)/2 d^p + p(p+2) d^(p+1) - p(p+1)/2 d^(p+2)
  gaussian: phi_q(r) = exp(-(r - mu_q)^2 / (2 s^2)),  mu_q = q r_c / (K-1), s = r_c / (K-1), q = 0..K-1
Derivatives are taken by torch.autograd of these very expressions, so the adjoint is the derivative
of the forward by construction; the pins check the forward against closed forms, the addition theorem,
quadrature orthonormality and the coupling tables, and the derivative against central differences.
"""
from __future__ import annotations

import math

import numpy as np
import torch

BESSEL, GAUSSIAN = 0, 1


def real_sh(rvec: torch.Tensor, l_max: int) -> torch.Tensor:
    """[n, 3] edge vectors (any length > 0) -> [n, (l_max+1)^2], differentiable."""
    r = torch.linalg.norm(rvec, dim=-1)
    x, y, z = rvec[:, 0] / r, rvec[:, 1] / r, rvec[:, 2] / r
    ct = z
    st = torch.sqrt(torch.clamp(1.0 - z * z, min=0.0))
    az = torch.atan2(y, x)
    # associated Legendre functions P_l^m(cos theta), no Condon-Shortley sign
    P = {}
    for m in range(l_max + 1):
        pmm = torch.ones_like(z)
        for k in range(1, m + 1):
            pmm = pmm * (2 * k - 1) * st
        P[(m, m)] = pmm
        if m + 1 <= l_max:
            P[(m + 1, m)] = (2 * m + 1) * ct * pmm
        for l in range(m + 2, l_max + 1):
            P[(l, m)] = ((2 * l - 1) * ct * P[(l - 1, m)] - (l + m - 1) * P[(l - 2, m)]) / (l - m)
    cols = [None] * (l_max + 1) ** 2
    for l in range(l_max + 1):
        for m in range(l + 1):
            n = math.sqrt((2 * l + 1) * math.factorial(l - m) / math.factorial(l + m))
            if m == 0:
                cols[l * l + l] = n * P[(l, 0)]
            else:
                cols[l * l + l + m] = math.sqrt(2.0) * n * P[(l, m)] * torch.cos(m * az)
                cols[l * l + l - m] = math.sqrt(2.0) * n * P[(l, m)] * torch.sin(m * az)
    return torch.stack(cols, dim=1)


def radial(r: torch.Tensor, K: int, r_c: float, basis: int = BESSEL, p: int = 6) -> torch.Tensor:
    """[n] edge lengths -> [n, K], differentiable."""
    if basis == BESSEL:
        q = torch.arange(1, K + 1, dtype=r.dtype)
        b = math.sqrt(2.0 / r_c) * torch.sin(q[None, :] * math.pi * r[:, None] / r_c) / r[:, None]
        d = r / r_c
        u = 1.0 - (p + 1) * (p + 2) / 2.0 * d**p + p * (p + 2) * d ** (p + 1) - p * (p + 1) / 2.0 * d ** (p + 2)
        return b * u[:, None]
    if basis == GAUSSIAN:
        step = r_c / max(K - 1, 1)
        mu = torch.arange(K, dtype=r.dtype) * step
        return torch.exp(-((r[:, None] - mu[None, :]) ** 2) / (2 * step * step))
    raise ValueError("basis")


def edge_inputs(rvec, l_max: int, K: int, r_c: float, basis: int = BESSEL, p: int = 6):
    """numpy [E, 3] -> (Y [E, dsh], phi [E, K]) in fp64."""
    t = torch.as_tensor(np.asarray(rvec, dtype=np.float64))
    return real_sh(t, l_max).numpy(), radial(torch.linalg.norm(t, dim=-1), K, r_c, basis, p).numpy()


def edge_vectors(col, recv, pos):
    """r_e = pos[sender(e)] - pos[receiver(e)]"""
    pos = np.asarray(pos, dtype=np.float64)
    return pos[np.asarray(col)] - pos[np.asarray(recv)]


def position_gradient(col, recv, g_rvec, N: int):
    """Adjoint of edge_vectors: gpos[j] += g_r[e] for the sender, gpos[i] -= g_r[e] for the receiver."""
    g = np.zeros((N, 3))
    np.add.at(g, np.asarray(col), g_rvec)
    np.subtract.at(g, np.asarray(recv), g_rvec)
    return g


def geo_fwd(orc, row_ptr, col, rvec, x, R, r_c: float, basis: int = BESSEL, p: int = 6, act=None):
    """y of the convolution with Y, phi recomputed from the edge vectors; `orc` is a conv.Oracle, `act` an optional
    subset of receivers (as in conv.Oracle.fwd)."""
    Y, phi = edge_inputs(rvec, orc.l_max, orc.K, r_c, basis, p)
    return orc.fwd(row_ptr, col, x, Y, phi, R, act=act)


def geo_bwd(orc, row_ptr, col, rvec, x, R, gy, r_c: float, basis: int = BESSEL, p: int = 6, act=None):
    """(gx, g_rvec, gR): adjoints of geo_fwd.  g_rvec[e] = J_Y(r_e)^T gY_e + J_phi(r_e)^T gphi_e."""
    t = torch.as_tensor(np.asarray(rvec, dtype=np.float64)).clone().requires_grad_(True)
    Y = real_sh(t, orc.l_max)
    phi = radial(torch.linalg.norm(t, dim=-1), orc.K, r_c, basis, p)
    gx, gY, gphi, gR = orc.bwd(row_ptr, col, x, Y.detach().numpy(), phi.detach().numpy(), R, gy, act=act)
    s = (Y * torch.as_tensor(gY)).sum() + (phi * torch.as_tensor(gphi)).sum()
    (g_rvec,) = torch.autograd.grad(s, t)
    return gx, g_rvec.numpy(), gR


def geo_dbwd(orc, row_ptr, col, rvec, x, R, gy, vx, v_rvec, vR, r_c: float, basis: int = BESSEL, p: int = 6, act=None,
             with_h_rvec: bool = False):
    """(ggy, hx, hR): derivatives of  Phi = <vx, gx> + <v_rvec, g_rvec> + <vR, gR>  (the adjoints of geo_bwd) with respect
    to gy, x and R -- what a loss on the forces needs for its parameter and feature gradients.  Since
    <v_rvec, g_rvec> = <J_Y v_rvec, gY> + <J_phi v_rvec, gphi>, this is the double backward of the convolution with the
    directions vY = J_Y v_rvec and vphi = J_phi v_rvec (Jacobian-vector products of the definitions above, by
    torch.autograd).

    with_h_rvec: also h_rvec = dPhi / d rvec, returned as a fourth array.  Phi depends on the edge vector of an edge
    through Y_e, phi_e (inside gx, gR, gY, gphi: the convolution's own second-order edge adjoints hY, hphi, pulled back
    through the Jacobians) and through the Jacobians in g_rvec = J_Y^T gY + J_phi^T gphi themselves (second derivatives
    of both bases, contracted with the first-order adjoints gY, gphi and the direction):
        h_rvec_e = J_Y^T hY_e + J_phi^T hphi_e + d/dr [ <J_Y(r) v_e, gY_e> + <J_phi(r) v_e, gphi_e> ]  (gY, gphi held fixed)."""
    t = torch.as_tensor(np.asarray(rvec, dtype=np.float64))
    v = torch.as_tensor(np.asarray(v_rvec, dtype=np.float64))
    sh = lambda r: real_sh(r, orc.l_max)
    rad = lambda r: radial(torch.linalg.norm(r, dim=-1), orc.K, r_c, basis, p)
    Y, vY = torch.autograd.functional.jvp(sh, t, v)
    phi, vphi = torch.autograd.functional.jvp(rad, t, v)
    ggy, hx, hY, hphi, hR = orc.dbwd(row_ptr, col, x, Y.numpy(), phi.numpy(), R, gy, vx, vY.numpy(), vphi.numpy(), vR, act=act)
    if not with_h_rvec:
        return ggy, hx, hR
    _, gY, gphi, _ = orc.bwd(row_ptr, col, x, Y.numpy(), phi.numpy(), R, gy, act=act)
    tt = t.clone().requires_grad_(True)
    # first part: the pull-back of hY, hphi; second part: the derivative of the Jacobians along v, with gY, gphi fixed
    first = (sh(tt) * torch.as_tensor(hY)).sum() + (rad(tt) * torch.as_tensor(hphi)).sum()
    _, Yv = torch.autograd.functional.jvp(sh, tt, v, create_graph=True)
    _, phiv = torch.autograd.functional.jvp(rad, tt, v, create_graph=True)
    second = (Yv * torch.as_tensor(gY)).sum() + (phiv * torch.as_tensor(gphi)).sum()
    (h_rvec,) = torch.autograd.grad(first + second, tt)
    return ggy, hx, hR, h_rvec.numpy()
