"""Pins for the fp64 oracle of the convolution and its two derivative orders.

None of these re-types the oracle's formula: they check it against equivariance under
random rotations (with Wigner-D matrices obtained from the spherical harmonics
themselves), textbook special cases, an independently ordered (reassociated) evaluation,
exact multilinearity, adjoint identities and finite differences."""
import math

import numpy as np
import pytest

from oracle import conv, tables
from workloads import synth


def _rand_rot(rng):
    q = rng.standard_normal(4)
    q /= np.linalg.norm(q)
    a, b, c, d = q
    return np.array([[a*a+b*b-c*c-d*d, 2*(b*c-a*d), 2*(b*d+a*c)],
                     [2*(b*c+a*d), a*a-b*b+c*c-d*d, 2*(c*d-a*b)],
                     [2*(b*d-a*c), 2*(c*d+a*b), a*a-b*b-c*c+d*d]])


def wigner_D(l, g, rng):
    """Real D^l(g) defined by Y_l(g r) = D^l(g) Y_l(r), solved from sample directions."""
    pts = rng.standard_normal((4 * (2 * l + 1), 3))
    A = synth.real_sph_harm(l, pts)[:, l * l:]
    B = synth.real_sph_harm(l, pts @ g.T)[:, l * l:]
    D, *_ = np.linalg.lstsq(A, B, rcond=None)
    return D.T


def block_D(irreps, g, rng, improper=False):
    """Action on an ir_mul feature vector: D acts on m, identity on multiplicity."""
    dim = synth.irreps_dim(irreps)
    M = np.zeros((dim, dim))
    o = 0
    for c, l, p in irreps:
        D = wigner_D(l, g, rng)
        if improper:
            D = D * p
        M[o:o + (2 * l + 1) * c, o:o + (2 * l + 1) * c] = np.kron(D, np.eye(c))
        o += (2 * l + 1) * c
    return M


def tiny(irreps_in, irreps_out, l_max, K, N=7, seed=1, r_c=0.75):
    w = synth.Workload("t", irreps_in, irreps_out, l_max, K, N, 1.0, r_c, "gaussian", seed=seed)
    o = conv.Oracle(irreps_in, irreps_out, l_max, K)
    inp = synth.make_inputs(w, o.col_std(), dtype=np.float64)
    return o, inp


P = synth.parse_irreps
CASES = [
    (P("3x0e+2x1o"), P("2x0e+3x1o+1x2e"), 2, 3),
    (P("2x0e+2x1o+1x1e+2x2e"), P("1x0e+1x0o+2x1o+2x1e+1x2e+1x2o+1x3o"), 3, 2),   # includes odd-sum paths
    (P("2x0e+1x1o+1x2e+1x3o+1x4e"), P("1x0e+1x1o+1x2e+1x3o+2x4e"), 4, 2),
]


@pytest.mark.parametrize("case", CASES, ids=["l2", "l3-mixed-parity", "l4"])
def test_equivariance(case):
    ii, io, lm, K = case
    o, d = tiny(ii, io, lm, K)
    rng = np.random.default_rng(5)
    y0 = o.fwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R)
    assert np.abs(y0).max() > 1e-3
    for improper in (False, True):
        g = _rand_rot(rng)
        gg = -g if improper else g
        # rotate the geometry: recompute Y from rotated positions; phi is invariant
        rij = (d.pos[d.col] - d.pos[d.recv]) @ gg.T
        Yr = synth.real_sph_harm(lm, rij)
        Dsh = block_D([(1, l, (-1) ** l) for l in range(lm + 1)], g, rng, improper)
        assert np.allclose(Yr, d.Y @ Dsh.T, atol=1e-10)
        xr = d.x @ block_D(ii, g, rng, improper).T
        yr = o.fwd(d.row_ptr, d.col, xr, Yr, d.phi, d.R)
        assert np.allclose(yr, y0 @ block_D(io, g, rng, improper).T, atol=1e-10)


@pytest.mark.parametrize("case", CASES, ids=["l2", "l3-mixed-parity", "l4"])
def test_materialised_equals_reassociated(case):
    ii, io, lm, K = case
    o, d = tiny(ii, io, lm, K, N=9)
    y0 = o.fwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R)
    y1 = o.reassociated_fwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R)
    assert np.allclose(y0, y1, atol=1e-12 * max(1.0, np.abs(y0).max()))


def test_scalar_only_is_weighted_adjacency_matmul():
    """All-scalar irreps with l_max = 0: y = sum_q (A_q X) R_q, A_q the phi_q-weighted
    adjacency matrix."""
    ii, io = P("5x0e"), P("4x0e")
    o, d = tiny(ii, io, 0, 3, N=12)
    y = o.fwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R)
    ref = np.zeros_like(y)
    for q in range(3):
        A = np.zeros((d.N, d.N))
        np.add.at(A, (d.recv, d.col), d.phi[:, q] * d.Y[:, 0])
        ref += A @ d.x @ d.R[q].reshape(5, 4)
    assert np.allclose(y, ref, atol=1e-12)


def test_single_edge_vector_formulas():
    """One edge, one path: scalar*vector, dot product and cross product, written in
    Cartesian coordinates (our l=1 component order is (y, z, x))."""
    row_ptr = np.array([0, 1, 1]); col = np.array([1], dtype=np.int32)
    rng = np.random.default_rng(3)
    r = rng.standard_normal(3); r /= np.linalg.norm(r)
    Y = synth.real_sph_harm(1, r[None])
    yzx = lambda v: np.array([v[1], v[2], v[0]])
    phi = np.array([[0.7]])
    v = rng.standard_normal(3)
    # 1o x Y1 -> 0e : c = delta/sqrt(3)  =>  y = R*phi * (v . sqrt(3) r)/sqrt(3)
    o = conv.Oracle(P("1x1o"), P("1x0e"), 1, 1)
    x = np.zeros((2, 3)); x[1] = yzx(v)
    y = o.fwd(row_ptr, col, x, Y, phi, np.array([[1.3]]))
    assert abs(y[0, 0] - 1.3 * 0.7 * v @ r) < 1e-12 and np.all(y[1] == 0)
    # 0e x Y1 -> 1o : y = s * sqrt(3) r
    o = conv.Oracle(P("1x0e"), P("1x1o"), 1, 1)
    x = np.zeros((2, 1)); x[1] = 2.0
    y = o.fwd(row_ptr, col, x, Y, phi, np.array([[1.3]]))
    assert np.allclose(y[0], 1.3 * 0.7 * 2.0 * math.sqrt(3) * yzx(r), atol=1e-12)
    # 1o x Y1 -> 1e : +-sqrt(3/2) (v x r) ... with the sign pin: positive first entry
    o = conv.Oracle(P("1x1o"), P("1x1e"), 1, 1)
    x = np.zeros((2, 3)); x[1] = yzx(v)
    y = o.fwd(row_ptr, col, x, Y, phi, np.array([[1.0]]))
    cr = yzx(np.cross(v, r)) * 0.7 * math.sqrt(3) * math.sqrt(3) / math.sqrt(6)
    assert np.allclose(y[0], cr, atol=1e-12) or np.allclose(y[0], -cr, atol=1e-12)


def test_unit_radial_is_plain_tensor_product_of_neighbour_sum():
    """K = 1, phi = 1, Y constant over edges (same direction): y_i = TP(sum_j x_j, Y)."""
    ii, io = P("2x0e+2x1o"), P("2x0e+2x1o+2x2e")
    o, d = tiny(ii, io, 2, 1, N=8)
    Y = np.tile(d.Y[:1], (d.E, 1)); phi = np.ones((d.E, 1))
    y = o.fwd(d.row_ptr, d.col, d.x, Y, phi, d.R)
    xs = np.zeros_like(d.x)
    np.add.at(xs, d.recv, d.x[d.col])
    # a graph of self-loops fed with the neighbour sums
    rp = np.arange(d.N + 1); cl = np.arange(d.N, dtype=np.int32)
    y2 = o.fwd(rp, cl, xs, np.tile(d.Y[:1], (d.N, 1)), np.ones((d.N, 1)), d.R)
    assert np.allclose(y, y2, atol=1e-12)


@pytest.mark.parametrize("case", CASES, ids=["l2", "l3-mixed-parity", "l4"])
def test_backward_is_the_adjoint_of_forward(case):
    ii, io, lm, K = case
    o, d = tiny(ii, io, lm, K)
    g = (d.row_ptr, d.col)
    gx, gY, gphi, gR = o.bwd(*g, d.x, d.Y, d.phi, d.R, d.gy)
    f = lambda x, Y, phi, R: o.fwd(*g, x, Y, phi, R)
    # y is linear in each argument separately: <gy, f(.. v ..)> = <v, grad>
    assert np.isclose((d.gy * f(d.vx, d.Y, d.phi, d.R)).sum(), (d.vx * gx).sum(), rtol=1e-11)
    assert np.isclose((d.gy * f(d.x, d.vY, d.phi, d.R)).sum(), (d.vY * gY).sum(), rtol=1e-11)
    assert np.isclose((d.gy * f(d.x, d.Y, d.vphi, d.R)).sum(), (d.vphi * gphi).sum(), rtol=1e-11)
    assert np.isclose((d.gy * f(d.x, d.Y, d.phi, d.vR)).sum(), (d.vR * gR).sum(), rtol=1e-11)


@pytest.mark.parametrize("case", CASES[:2], ids=["l2", "l3-mixed-parity"])
def test_backward_elementwise_by_linearity(case):
    """Because y is linear in x (and in Y, phi, R), d<gy,y>/dx_k = <gy, f(e_k)> exactly."""
    ii, io, lm, K = case
    o, d = tiny(ii, io, lm, K, N=5)
    g = (d.row_ptr, d.col)
    gx, gY, gphi, gR = o.bwd(*g, d.x, d.Y, d.phi, d.R, d.gy)
    rng = np.random.default_rng(0)
    for arr, grad, slot in ((d.x, gx, 0), (d.Y, gY, 1), (d.phi, gphi, 2), (d.R, gR, 3)):
        for _ in range(6):
            k = tuple(rng.integers(0, s) for s in arr.shape)
            e = np.zeros_like(arr); e[k] = 1.0
            args = [d.x, d.Y, d.phi, d.R]; args[slot] = e
            assert np.isclose((d.gy * o.fwd(*g, *args)).sum(), grad[k], rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("case", CASES, ids=["l2", "l3-mixed-parity", "l4"])
def test_double_backward_central_differences(case):
    """dbwd returns d/d(theta, gy) of <v, bwd(theta, gy)>: compare with central
    differences of the backward map along random directions (exact up to rounding for a
    cubic in the step, so the step can be large)."""
    ii, io, lm, K = case
    o, d = tiny(ii, io, lm, K)
    g = (d.row_ptr, d.col)
    ggy, hx, hY, hphi, hR = o.dbwd(*g, d.x, d.Y, d.phi, d.R, d.gy, d.vx, d.vY, d.vphi, d.vR)

    def scalar(x, Y, phi, R, gy):
        gx, gY, gphi, gR = o.bwd(*g, x, Y, phi, R, gy)
        return (d.vx * gx).sum() + (d.vY * gY).sum() + (d.vphi * gphi).sum() + (d.vR * gR).sum()

    rng = np.random.default_rng(11)
    base = [d.x, d.Y, d.phi, d.R, d.gy]
    grads = [hx, hY, hphi, hR, ggy]
    for slot in range(5):
        dirn = rng.standard_normal(base[slot].shape)
        eps = 1e-3
        # scalar is a polynomial of degree <= 2 in any single argument's step => the
        # central difference is exact
        a = list(base); a[slot] = base[slot] + eps * dirn
        b = list(base); b[slot] = base[slot] - eps * dirn
        fd = (scalar(*a) - scalar(*b)) / (2 * eps)
        an = (grads[slot] * dirn).sum()
        assert np.isclose(fd, an, rtol=1e-7, atol=1e-9), (slot, fd, an)


@pytest.mark.parametrize("case", CASES[:2], ids=["l2", "l3-mixed-parity"])
def test_double_backward_substitution_form_and_hessian_symmetry(case):
    """<gy, y> is linear in each of its five arguments, so the second-order outputs are
    sums of first-order maps with one argument replaced by its direction."""
    ii, io, lm, K = case
    o, d = tiny(ii, io, lm, K)
    g = (d.row_ptr, d.col)
    ggy, hx, hY, hphi, hR = o.dbwd(*g, d.x, d.Y, d.phi, d.R, d.gy, d.vx, d.vY, d.vphi, d.vR)
    f = lambda x, Y, phi, R: o.fwd(*g, x, Y, phi, R)
    s = f(d.vx, d.Y, d.phi, d.R) + f(d.x, d.vY, d.phi, d.R) + f(d.x, d.Y, d.vphi, d.R) + f(d.x, d.Y, d.phi, d.vR)
    assert np.allclose(ggy, s, atol=1e-11)
    b = lambda x, Y, phi, R: o.bwd(*g, x, Y, phi, R, d.gy)
    bx, bY, bp, bR = b(d.vx, d.Y, d.phi, d.R), b(d.x, d.vY, d.phi, d.R), b(d.x, d.Y, d.vphi, d.R), b(d.x, d.Y, d.phi, d.vR)
    assert np.allclose(hx, bY[0] + bp[0] + bR[0], atol=1e-11)
    assert np.allclose(hY, bx[1] + bp[1] + bR[1], atol=1e-11)
    assert np.allclose(hphi, bx[2] + bY[2] + bR[2], atol=1e-11)
    assert np.allclose(hR, bx[3] + bY[3] + bp[3], atol=1e-11)
    # Hessian symmetry <v1, H v2> = <v2, H v1>
    rng = np.random.default_rng(2)
    u = [rng.standard_normal(a.shape) for a in (d.x, d.Y, d.phi, d.R)]
    _, ax, aY, ap, aR = o.dbwd(*g, d.x, d.Y, d.phi, d.R, d.gy, *u)
    lhs = (d.vx * ax).sum() + (d.vY * aY).sum() + (d.vphi * ap).sum() + (d.vR * aR).sum()
    rhs = (u[0] * hx).sum() + (u[1] * hY).sum() + (u[2] * hphi).sum() + (u[3] * hR).sum()
    assert np.isclose(lhs, rhs, rtol=1e-10)


def test_active_receiver_subset():
    ii, io, lm, K = CASES[0]
    o, d = tiny(ii, io, lm, K, N=10)
    g = (d.row_ptr, d.col)
    act = np.array([1, 4, 7])
    y = o.fwd(*g, d.x, d.Y, d.phi, d.R)
    ys = o.fwd(*g, d.x, d.Y, d.phi, d.R, act=act)
    assert np.array_equal(ys[act], y[act])
    gym = np.zeros_like(d.gy); gym[act] = d.gy[act]
    full = o.bwd(*g, d.x, d.Y, d.phi, d.R, gym)
    part = o.bwd(*g, d.x, d.Y, d.phi, d.R, d.gy, act=act)
    for a, b in zip(full, part):
        assert np.allclose(a, b, atol=1e-13)


def test_sender_view_is_a_stable_sort():
    _, d = tiny(*CASES[0], N=20)
    sp, perm = conv.sender_view(d.row_ptr, d.col)
    assert np.array_equal(perm, np.argsort(d.col, kind="stable").astype(np.int32))
    assert np.array_equal(sp, np.concatenate([[0], np.cumsum(np.bincount(d.col, minlength=d.N))]))


def test_empty_receivers_self_loops_duplicates():
    ii, io, lm, K = CASES[0]
    o = conv.Oracle(ii, io, lm, K)
    rng = np.random.default_rng(0)
    row_ptr = np.array([0, 0, 3, 3, 4]); col = np.array([1, 2, 2, 0], dtype=np.int32)  # self loop, duplicate
    E, N = 4, 4
    x = rng.standard_normal((N, o.C_x)); Y = rng.standard_normal((E, 9)); phi = rng.standard_normal((E, K))
    R = rng.standard_normal((K, o.N_w))
    y = o.fwd(row_ptr, col, x, Y, phi, R)
    assert np.all(y[0] == 0) and np.all(y[2] == 0)
    # duplicates are summed: doubling one copy equals two copies
    rp2 = np.array([0, 0, 2, 2, 3]); cl2 = np.array([1, 2, 0], dtype=np.int32)
    Y2 = Y[[0, 1, 3]]; phi2 = phi[[0, 1, 3]].copy()
    Ysame = Y.copy(); Ysame[2] = Y[1]; phis = phi.copy(); phis[2] = phi[1]
    phi2[1] *= 2
    assert np.allclose(o.fwd(row_ptr, col, x, Ysame, phis, R), o.fwd(rp2, cl2, x, Y2, phi2, R), atol=1e-12)


# ---------------------------------------------------------------------------------------
# channelwise (uvu) mode, Eq. uvu_connection
# ---------------------------------------------------------------------------------------
UVU_CASES = [
    (P("3x0e+3x1o"), 1, 3),
    (P("2x0e+2x1o+2x2e"), 2, 2),
]


def _uvu_pair(ir, l_max, K, seed=2):
    """A uvu oracle, a uvw oracle on the same irreps, inputs for the first, and the map that embeds
    the tied weights on the diagonal of the fully connected ones: A[q, pi, u, w] = delta_uw a[q, pi, u]."""
    w = synth.Workload("t", ir, ir, l_max, K, 7, 1.0, 0.75, "gaussian", seed=seed)
    try:
        ou = conv.Oracle(ir, ir, l_max, K, mode="uvu")
    except ValueError:
        return None
    ow = conv.Oracle(ir, ir, l_max, K)
    inp = synth.make_inputs(w, ou.col_std(), dtype=np.float64)

    def embed(a):
        A = np.zeros((K, ow.N_w))
        for pu, pw in zip(ou.paths, ow.paths):
            for u in range(pu.c_in):
                A[:, pw.w_off + u * pw.c_out + u] = a[:, pu.w_off + u]
        return A

    def diag(A):
        a = np.zeros((K, ou.N_w))
        for pu, pw in zip(ou.paths, ow.paths):
            for u in range(pu.c_in):
                a[:, pu.w_off + u] = A[:, pw.w_off + u * pw.c_out + u]
        return a

    return ou, ow, inp, embed, diag


def test_uvu_rejects_unequal_multiplicities():
    with pytest.raises(ValueError):
        conv.Oracle(P("2x0e+3x1o"), P("2x0e+3x1o"), 1, 2, mode="uvu")     # 0e x 1o -> 1o couples 2 with 3
    with pytest.raises(ValueError):
        conv.Oracle(P("2x0e+3x1o"), P("2x0e+3x1o+1x2e"), 2, 2, mode="uvu")
    conv.Oracle(P("3x0e+3x1o"), P("3x0e+3x1o"), 1, 2, mode="uvu")


@pytest.mark.parametrize("case", UVU_CASES)
def test_uvu_is_uvw_with_diagonal_weights(case):
    """The tied mode is the fully connected one restricted to weights that vanish off the diagonal u = w
    (Eqs. uvw_connection, uvu_connection): all three orders must agree, with the weight adjoints read off the
    diagonal.  This pins the uvu oracle to the uvw oracle, which the tests above pin independently."""
    ir, l_max, K = case
    ou, ow, d, embed, diag = _uvu_pair(ir, l_max, K)
    assert ou.N_w == sum(p.c_in for p in ou.paths) and len(ou.paths) == len(ow.paths)
    A, vA = embed(d.R), embed(d.vR)
    g = (d.row_ptr, d.col, d.x, d.Y, d.phi)
    assert np.allclose(ou.fwd(*g, d.R), ow.fwd(*g, A), rtol=1e-12, atol=1e-13)
    bu, bw = ou.bwd(*g, d.R, d.gy), ow.bwd(*g, A, d.gy)
    for a, b in zip(bu[:3], bw[:3]):
        assert np.allclose(a, b, rtol=1e-12, atol=1e-13)
    assert np.allclose(bu[3], diag(bw[3]), rtol=1e-12, atol=1e-13)
    du = ou.dbwd(*g, d.R, d.gy, d.vx, d.vY, d.vphi, d.vR)
    dw = ow.dbwd(*g, A, d.gy, d.vx, d.vY, d.vphi, vA)
    for a, b in zip(du[:4], dw[:4]):
        assert np.allclose(a, b, rtol=1e-12, atol=1e-13)
    assert np.allclose(du[4], diag(dw[4]), rtol=1e-12, atol=1e-13)
    assert np.abs(du[0]).max() > 1e-3 and np.abs(du[4]).max() > 1e-3


@pytest.mark.parametrize("case", UVU_CASES)
def test_uvu_materialised_equals_reassociated(case):
    ir, l_max, K = case
    ou, _, d, _, _ = _uvu_pair(ir, l_max, K)
    g = (d.row_ptr, d.col, d.x, d.Y, d.phi, d.R)
    assert np.allclose(ou.fwd(*g), ou.reassociated_fwd(*g), rtol=1e-11, atol=1e-12)


def test_uvu_channels_do_not_mix():
    """Changing input channel u changes output channel u only, in every block."""
    ir, l_max, K = UVU_CASES[1]
    ou, _, d, _, _ = _uvu_pair(ir, l_max, K)
    g = (d.row_ptr, d.col)
    y0 = ou.fwd(*g, d.x, d.Y, d.phi, d.R)
    x1 = d.x.copy()
    o = 0
    for c, l, _ in ir:                      # perturb channel 0 of every input block
        for m in range(2 * l + 1):
            x1[:, o + m * c + 0] += 1.0
        o += c * (2 * l + 1)
    dy = ou.fwd(*g, x1, d.Y, d.phi, d.R) - y0
    o = 0
    for c, l, _ in ir:
        blk = dy[:, o:o + c * (2 * l + 1)].reshape(-1, 2 * l + 1, c)
        assert np.abs(blk[:, :, 1:]).max() == 0.0 and np.abs(blk[:, :, 0]).max() > 0.0
        o += c * (2 * l + 1)


def test_uvu_mixed_multiplicity_blocks_that_do_not_couple():
    """Blocks of different multiplicity are allowed as long as no path joins them."""
    ir = P("2x0e+3x1e")          # 0e x l_sh -> needs parity (-1)^l_sh: with l_max = 0 only 0e->0e and 1e->1e
    ou = conv.Oracle(ir, ir, 0, 2, mode="uvu")
    assert [(p.c_in, p.c_out) for p in ou.paths] == [(2, 2), (3, 3)] and ou.N_w == 5
