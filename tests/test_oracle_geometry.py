"""Pins for the geometry oracle (spherical harmonics and radial bases recomputed from edge vectors, and the
gradient that reaches the positions).  None of them re-types the oracle's expressions: closed Cartesian forms,
the addition theorem, quadrature orthonormality, the coupling tables, boundary behaviour of the radial bases,
central differences, and the symmetry of energies and forces (Eq. energy_force_symmetry)."""
import math

import numpy as np
import pytest
import torch

from oracle import conv, geometry, tables
from workloads import synth

P = synth.parse_irreps


def _units(n, seed=0):
    v = np.random.default_rng(seed).standard_normal((n, 3))
    return v / np.linalg.norm(v, axis=1, keepdims=True)


def _sh(v, l_max):
    return geometry.real_sh(torch.as_tensor(v), l_max).numpy()


def test_closed_cartesian_forms_up_to_l2():
    v = _units(50, 1)
    x, y, z = v.T
    Y = _sh(v * np.random.default_rng(2).uniform(0.3, 4.0, (50, 1)), 2)      # any length: only the direction counts
    assert np.allclose(Y[:, 0], 1.0)
    assert np.allclose(Y[:, 1:4], math.sqrt(3) * np.stack([y, z, x], 1), atol=1e-12)
    want = np.stack([math.sqrt(15) * x * y, math.sqrt(15) * y * z, math.sqrt(5) / 2 * (3 * z * z - 1),
                     math.sqrt(15) * x * z, math.sqrt(15) / 2 * (x * x - y * y)], 1)
    assert np.allclose(Y[:, 4:9], want, atol=1e-12)


@pytest.mark.parametrize("l", range(5))
def test_addition_theorem(l):
    a, b = _units(40, 3), _units(40, 4)
    Ya, Yb = _sh(a, 4)[:, l * l:(l + 1) ** 2], _sh(b, 4)[:, l * l:(l + 1) ** 2]
    c = np.zeros(l + 1); c[l] = 1.0
    leg = np.polynomial.legendre.legval((a * b).sum(1), c)
    assert np.allclose((Ya * Yb).sum(1), (2 * l + 1) * leg, atol=1e-11)


def test_orthonormal_on_the_sphere():
    # Gauss-Legendre in cos(theta) times a uniform grid in the azimuth: exact for the products involved
    ct, w = np.polynomial.legendre.leggauss(12)
    az = (np.arange(24) + 0.5) * 2 * math.pi / 24
    st = np.sqrt(1 - ct * ct)
    pts = np.stack([np.outer(st, np.cos(az)), np.outer(st, np.sin(az)), np.outer(ct, np.ones_like(az))], -1).reshape(-1, 3)
    wt = np.repeat(w, 24) / (2 * 24)
    Y = _sh(pts, 4)
    assert np.allclose(np.einsum("n,na,nb->ab", wt, Y, Y), np.eye(25), atol=1e-12)


@pytest.mark.parametrize("l1,l2,l3", [(1, 1, 2), (1, 2, 3), (2, 2, 4), (2, 2, 2), (1, 3, 4), (4, 4, 4), (3, 4, 1), (1, 1, 0)])
def test_products_couple_through_the_oracles_tables(l1, l2, l3):
    """sum_ab w3j[a,b,c] Y_l1[a] Y_l2[b] is proportional to Y_l3[c] with one constant for every direction:
    ties the basis (order and signs of the components) to the coupling tensors the convolution uses."""
    v = _units(30, 5)
    Y = _sh(v, 4)
    sl = lambda l: Y[:, l * l:(l + 1) ** 2]
    lhs = np.einsum("abc,na,nb->nc", tables.real_w3j(l1, l2, l3), sl(l1), sl(l2))
    k = (lhs * sl(l3)).sum() / (sl(l3) ** 2).sum()
    assert abs(k) > 1e-3
    assert np.allclose(lhs, k * sl(l3), atol=1e-10)


def test_workload_generator_agrees():
    """The workloads' own generator (numpy, written separately) feeds the same functions."""
    v = _units(64, 6) * np.random.default_rng(7).uniform(0.2, 0.9, (64, 1))
    r = np.linalg.norm(v, axis=1)
    Y, phi = geometry.edge_inputs(v, 4, 8, 1.0, geometry.BESSEL)
    assert np.allclose(Y, synth.real_sph_harm(4, v), atol=1e-12)
    assert np.allclose(phi, synth.bessel_basis(r, 8, 1.0), atol=1e-12)
    assert np.allclose(geometry.edge_inputs(v, 2, 6, 1.0, geometry.GAUSSIAN)[1], synth.gaussian_basis(r, 6, 1.0), atol=1e-12)


def test_radial_boundary_behaviour():
    rc, K = 1.7, 6
    r = torch.tensor([rc, 1e-4], dtype=torch.float64, requires_grad=True)
    f = geometry.radial(r, K, rc, geometry.BESSEL, 6)
    assert np.allclose(f[0].detach().numpy(), 0.0, atol=1e-12)           # vanishes at the cutoff
    for q in range(K):                                                     # ... with zero slope (smooth envelope)
        (g,) = torch.autograd.grad(f[0, q], r, retain_graph=True)
        assert abs(g[0].item()) < 1e-9
    # r -> 0: sin(q pi r / rc) / r -> q pi / rc
    assert np.allclose(f[1].detach().numpy(), math.sqrt(2 / rc) * np.arange(1, K + 1) * math.pi / rc, rtol=1e-6)
    # the bare Bessel functions are orthonormal on [0, rc] with weight r^2 (envelope exponent -> infinity removes it: use quadrature
    # of the un-enveloped ratio instead)
    x, w = np.polynomial.legendre.leggauss(80)
    rr = 0.5 * rc * (x + 1); ww = 0.5 * rc * w
    d = rr / rc
    u = 1 - 28 * d**6 + 48 * d**7 - 21 * d**8
    b = geometry.radial(torch.as_tensor(rr), K, rc, geometry.BESSEL, 6).numpy() / u[:, None]
    assert np.allclose(np.einsum("n,na,nb->ab", ww * rr * rr, b, b), np.eye(K), atol=1e-10)
    g = geometry.radial(torch.tensor([0.0, rc / 5 * 2, rc], dtype=torch.float64), 6, rc, geometry.GAUSSIAN).numpy()
    assert np.allclose([g[0, 0], g[1, 2], g[2, 5]], 1.0)                  # unit peaks at the centres
    assert np.allclose(g[0, 1], math.exp(-0.5))


def _tiny(seed=3, basis="bessel"):
    ii, io, lm, K = P("2x0e+2x1o+1x2e"), P("3x0e+1x1o+1x2e+1x3o"), 3, 4
    w = synth.Workload("t", ii, io, lm, K, 9, 1.0, 0.8, basis, seed=seed)
    o = conv.Oracle(ii, io, lm, K)
    return o, w, synth.make_inputs(w, o.col_std(), dtype=np.float64)


@pytest.mark.parametrize("basis", ["bessel", "gaussian"])
def test_forward_equals_the_convolution_on_precomputed_inputs(basis):
    o, w, d = _tiny(basis=basis)
    rv = geometry.edge_vectors(d.col, d.recv, d.pos)
    b = geometry.BESSEL if basis == "bessel" else geometry.GAUSSIAN
    y = geometry.geo_fwd(o, d.row_ptr, d.col, rv, d.x, d.R, w.r_c, b)
    assert np.abs(y).max() > 1e-3
    assert np.allclose(y, o.fwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R), atol=1e-12)


@pytest.mark.parametrize("basis", [geometry.BESSEL, geometry.GAUSSIAN])
def test_edge_vector_gradient_by_central_differences(basis):
    o, w, d = _tiny(basis="bessel" if basis == geometry.BESSEL else "gaussian")
    rv = geometry.edge_vectors(d.col, d.recv, d.pos)
    gx, g_rv, gR = geometry.geo_bwd(o, d.row_ptr, d.col, rv, d.x, d.R, d.gy, w.r_c, basis)
    L = lambda r: (geometry.geo_fwd(o, d.row_ptr, d.col, r, d.x, d.R, w.r_c, basis) * d.gy).sum()
    rng = np.random.default_rng(0)
    h = 1e-6
    for _ in range(12):
        e, c = rng.integers(rv.shape[0]), rng.integers(3)
        dp = np.zeros_like(rv); dp[e, c] = h
        fd = (L(rv + dp) - L(rv - dp)) / (2 * h)
        assert abs(fd - g_rv[e, c]) < 1e-6 * max(1.0, abs(fd))
    # the other two adjoints are those of the convolution itself
    gx0, _, _, gR0 = o.bwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R, d.gy)
    assert np.allclose(gx, gx0, atol=1e-12) and np.allclose(gR, gR0, atol=1e-12)
    # the direction part of the gradient is tangential: scaling an edge vector changes only phi
    Y_only = geometry.geo_bwd(o, d.row_ptr, d.col, rv, d.x, d.R, d.gy, 1e9, geometry.GAUSSIAN)       # flat radial basis
    assert np.abs((Y_only[1] * rv).sum(1)).max() < 1e-9 * np.abs(Y_only[1]).max() + 1e-12


def test_energy_is_invariant_and_forces_rotate():
    """Eq. energy_force_symmetry for E = sum of the scalar outputs: E(R r) = E(r), F(R r) = R F(r), sum_i F_i = 0."""
    o, w, d = _tiny(seed=5)
    n0 = sum(c for c, l, p in o.irreps_out if l == 0)                      # the 0e block comes first
    gy = np.zeros_like(d.gy); gy[:, :n0] = np.random.default_rng(1).standard_normal(n0)[None, :]

    def energy_forces(pos):
        rv = geometry.edge_vectors(d.col, d.recv, pos)
        y = geometry.geo_fwd(o, d.row_ptr, d.col, rv, d.x_scalar, d.R, w.r_c)
        _, g_rv, _ = geometry.geo_bwd(o, d.row_ptr, d.col, rv, d.x_scalar, d.R, gy, w.r_c)
        return (y * gy).sum(), -geometry.position_gradient(d.col, d.recv, g_rv, pos.shape[0])

    # features that are themselves invariant (only the scalar block is non-zero), so that E depends on geometry alone
    d.x_scalar = np.zeros_like(d.x)
    c0 = sum(c for c, l, p in o.irreps_in if l == 0)
    d.x_scalar[:, :c0] = d.x[:, :c0]
    E0, F0 = energy_forces(d.pos)
    assert np.abs(F0).max() > 1e-6
    assert np.abs(F0.sum(0)).max() < 1e-12 * max(1.0, np.abs(F0).max()) + 1e-13
    q = np.random.default_rng(2).standard_normal(4); q /= np.linalg.norm(q)
    a, b, c, e = q
    Rm = np.array([[a*a+b*b-c*c-e*e, 2*(b*c-a*e), 2*(b*e+a*c)],
                   [2*(b*c+a*e), a*a-b*b+c*c-e*e, 2*(c*e-a*b)],
                   [2*(b*e-a*c), 2*(c*e+a*b), a*a-b*b-c*c+e*e]])
    E1, F1 = energy_forces(d.pos @ Rm.T + np.array([0.3, -1.0, 2.0]))
    assert abs(E1 - E0) < 1e-10 * max(1.0, abs(E0))
    assert np.allclose(F1, F0 @ Rm.T, atol=1e-10)
    # forces are minus the derivative of the energy with respect to a position
    h = 1e-6
    for i, k in [(0, 0), (3, 2), (7, 1)]:
        dp = np.zeros_like(d.pos); dp[i, k] = h
        fd = (energy_forces(d.pos + dp)[0] - energy_forces(d.pos - dp)[0]) / (2 * h)
        assert abs(-fd - F0[i, k]) < 1e-6 * max(1.0, abs(fd))


def test_force_loss_double_backward_by_central_differences():
    """geo_dbwd against central differences of  Phi = <vx, gx> + <v_r, g_r> + <vR, gR>  evaluated with geo_bwd, with
    respect to entries of x (hx), R (hR) and gy (ggy; Phi is linear in gy, so that one is exact up to rounding)."""
    o, w, d = _tiny(seed=7)
    rv = geometry.edge_vectors(d.col, d.recv, d.pos)
    rng = np.random.default_rng(11)
    v_r = rng.standard_normal(rv.shape)
    ggy, hx, hR = geometry.geo_dbwd(o, d.row_ptr, d.col, rv, d.x, d.R, d.gy, d.vx, v_r, d.vR, w.r_c)

    def Phi(x, R, gy):
        gx, g_r, gR = geometry.geo_bwd(o, d.row_ptr, d.col, rv, x, R, gy, w.r_c)
        return (d.vx * gx).sum() + (v_r * g_r).sum() + (d.vR * gR).sum()

    h = 1e-5
    for arr, grad, k in ((d.x, hx, 0), (d.R, hR, 1), (d.gy, ggy, 2)):
        scale = np.abs(grad).max()
        assert scale > 1e-6
        for _ in range(6):
            idx = tuple(rng.integers(n) for n in arr.shape)
            dp = np.zeros_like(arr); dp[idx] = h
            args = [d.x, d.R, d.gy]
            args[k] = arr + dp; fp = Phi(*args)
            args[k] = arr - dp; fm = Phi(*args)
            assert abs((fp - fm) / (2 * h) - grad[idx]) < 1e-6 * scale + 1e-9
    # with no direction on the edge vectors it is the stored-input double backward with vY = vphi = 0
    g2 = geometry.geo_dbwd(o, d.row_ptr, d.col, rv, d.x, d.R, d.gy, d.vx, np.zeros_like(rv), d.vR, w.r_c)
    ref = o.dbwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R, d.gy, d.vx, np.zeros_like(d.vY), np.zeros_like(d.vphi), d.vR)
    assert np.allclose(g2[0], ref[0], atol=1e-11) and np.allclose(g2[1], ref[1], atol=1e-11) and np.allclose(g2[2], ref[4], atol=1e-11)


def test_second_order_edge_vector_adjoint_by_central_differences():
    """h_rvec of geo_dbwd (with_h_rvec) against central differences of  Phi = <vx, gx> + <v_r, g_r> + <vR, gR>  with
    respect to entries of the edge vectors, Phi evaluated with geo_bwd; both radial bases."""
    for basis, seed in ((geometry.BESSEL, 5), (geometry.GAUSSIAN, 6)):
        o, w, d = _tiny(seed=seed)
        rv = geometry.edge_vectors(d.col, d.recv, d.pos)
        rng = np.random.default_rng(13)
        v_r = rng.standard_normal(rv.shape)
        out = geometry.geo_dbwd(o, d.row_ptr, d.col, rv, d.x, d.R, d.gy, d.vx, v_r, d.vR, w.r_c, basis, with_h_rvec=True)
        assert len(out) == 4
        h_r = out[3]
        # the first three outputs do not depend on the flag
        for a, b in zip(out[:3], geometry.geo_dbwd(o, d.row_ptr, d.col, rv, d.x, d.R, d.gy, d.vx, v_r, d.vR, w.r_c, basis)):
            assert np.allclose(a, b, rtol=1e-12, atol=1e-12 * np.abs(b).max())

        def Phi(r):
            gx, g_r, gR = geometry.geo_bwd(o, d.row_ptr, d.col, r, d.x, d.R, d.gy, w.r_c, basis)
            return (d.vx * gx).sum() + (v_r * g_r).sum() + (d.vR * gR).sum()

        scale = np.abs(h_r).max()
        assert scale > 1e-6
        h = 1e-5
        for _ in range(8):
            e, k = int(rng.integers(rv.shape[0])), int(rng.integers(3))
            dp = np.zeros_like(rv); dp[e, k] = h
            fd = (Phi(rv + dp) - Phi(rv - dp)) / (2 * h)
            assert abs(fd - h_r[e, k]) < 2e-6 * scale + 1e-9
