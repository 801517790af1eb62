"""GPU parity of the geometry front end (Y and phi recomputed from edge vectors inside the edge kernels; the
adjoint of the edge vectors and of the positions) against the fp64 geometry oracle, through the C ABI.
Tolerances as for the convolution: forward 1e-4 * max|ref|, backward 5e-4 * max|ref|."""
import numpy as np
import pytest

from oracle import geometry
from gpu_util import BWD_TOL, FWD_TOL, Case, rel_err
from workloads import synth

pytestmark = pytest.mark.gpu
P = synth.parse_irreps


def _cases():
    c = {}
    c["cfg2_N200"] = synth.scaled(synth.config("cfg2"), 200)
    c["cfg3_N120"] = synth.scaled(synth.config("cfg3"), 120)
    c["cfg4_N150"] = synth.scaled(synth.config("cfg4"), 150)           # K = 16
    c["cfg5_N60"] = synth.scaled(synth.config("cfg5"), 60)             # l_max = 4, several sets per launch
    c["tc_K6_dense"] = synth.Workload("tc_K6_dense", P("16x0e+16x1o"), P("16x0e+16x1o+16x2e"), 2, 6, 160, 4.0, 3.6,
                                      "bessel", seed=5)                 # K not a multiple of 4, ~100 edges per receiver
    c["gauss_K12"] = synth.Workload("gauss_K12", P("48x0e+16x1o+16x2e"), P("16x0e+48x1o"), 2, 12, 70, 4.0, 2.2,
                                    "gaussian", seed=6)
    return c


CASES = _cases()


class GeoCase(Case):
    def __init__(self, w, **kw):
        super().__init__(w, **kw)
        import torch
        d = self.d
        self.basis = geometry.BESSEL if w.basis == "bessel" else geometry.GAUSSIAN
        self.pos = torch.from_numpy(np.ascontiguousarray(d.pos, dtype=np.float32)).to("cuda:0")
        self.rvec = self._new(self.E, 3)
        self.sb.edge_vectors(self.graph, self.pos, self.rvec)
        # the oracle starts from the same fp32 positions
        self.o_rvec = geometry.edge_vectors(d.col, d.recv, self.pos.cpu().numpy().astype(np.float64))

    def geo_fwd(self):
        y = self._new(self.N, self.plan.info.C_y)
        self.sb.conv_geo_fwd(self.plan, self.graph, self.rvec, self.basis, self.w.r_c, 6, self.x, self.R, y, self.ws(0))
        assert self.sb.last_device_status(self.ws(0)) == 0
        return y.cpu().numpy()

    def geo_bwd(self, want=(True, True, True)):
        i = self.plan.info
        gx, g_rv, gR = self._new(self.N, i.C_x), self._new(self.E, 3), self._new(i.K, i.N_w)
        out = [t if on else None for t, on in zip((gx, g_rv, gR), want)]
        self.sb.conv_geo_bwd(self.plan, self.graph, self.rvec, self.basis, self.w.r_c, 6, self.x, self.R, self.gy,
                             *out, self.ws(1))
        assert self.sb.last_device_status(self.ws(1)) == 0
        return [None if t is None else t.cpu().numpy() for t in out]


@pytest.mark.parametrize("name", list(CASES))
def test_edge_vectors_and_forward(name):
    c = GeoCase(CASES[name])
    d = c.d
    assert np.abs(c.rvec.cpu().numpy() - c.o_rvec).max() < 1e-6
    y = c.geo_fwd()
    ref = geometry.geo_fwd(c.oracle, d.row_ptr, d.col, c.o_rvec, d.x, d.R, c.w.r_c, c.basis)
    assert np.isfinite(y).all() and np.abs(ref).max() > 1e-3
    assert rel_err(y, ref) <= FWD_TOL
    # and it is the stored-input forward on the same geometry (both within tolerance of the oracle)
    assert rel_err(y, c.fwd()) <= 2 * FWD_TOL


@pytest.mark.parametrize("name", list(CASES))
def test_backward_and_position_gradient(name):
    c = GeoCase(CASES[name])
    d = c.d
    gx, g_rv, gR = c.geo_bwd()
    rx, r_rv, rR = geometry.geo_bwd(c.oracle, d.row_ptr, d.col, c.o_rvec, d.x, d.R, d.gy, c.w.r_c, c.basis)
    assert all(np.isfinite(a).all() for a in (gx, g_rv, gR))
    assert rel_err(gx, rx) <= BWD_TOL and rel_err(gR, rR) <= BWD_TOL
    assert np.abs(r_rv).max() > 1e-3 and rel_err(g_rv, r_rv) <= BWD_TOL
    # positions: the fixed-order segment sums against numpy's scatter of the oracle's edge gradient
    import torch
    gpos = c._new(c.N, 3)
    c.sb.position_gradient(c.graph, torch.from_numpy(r_rv.astype(np.float32)).to("cuda:0"), gpos)
    ref = geometry.position_gradient(d.col, d.recv, r_rv, c.N)
    assert rel_err(gpos.cpu().numpy(), ref) <= 1e-5
    # bitwise the same on a second run (every sum has a fixed order)
    again = c.geo_bwd()
    assert all(np.array_equal(a, b) for a, b in zip((gx, g_rv, gR), again))


FULL = {"cfg3": (synth.config("cfg3"), 6), "cfg4_1e6": (synth.config("cfg4", edges=1e6), 8), "cfg5": (synth.config("cfg5"), 3)}


@pytest.mark.parametrize("name", list(FULL))
def test_full_size_sampled(name):
    """The benchmark configurations at full size: sampled receivers (first, last and some between, so that several
    chunks are hit) against the oracle, output adjoint zero outside the sample."""
    w, n_sample = FULL[name]
    c = GeoCase(w)
    d = c.d
    act = np.sort(np.random.default_rng(123).choice(c.N, size=n_sample, replace=False))
    act[0], act[-1] = 0, c.N - 1
    act = np.unique(act)
    ed = c.edges_into(act)
    y = c.geo_fwd()
    ref = geometry.geo_fwd(c.oracle, d.row_ptr, d.col, c.o_rvec, d.x, d.R, w.r_c, c.basis, act=act)
    assert np.isfinite(y).all() and rel_err(y[act], ref[act]) <= FWD_TOL
    c.gy = c.masked_gy(act)
    gx, g_rv, gR = c.geo_bwd()
    gym = c.gy.cpu().numpy().astype(np.float64)
    rx, r_rv, rR = geometry.geo_bwd(c.oracle, d.row_ptr, d.col, c.o_rvec, d.x, d.R, gym, w.r_c, c.basis, act=act)
    assert rel_err(gx, rx) <= BWD_TOL and rel_err(gR, rR) <= BWD_TOL
    assert rel_err(g_rv[ed], r_rv[ed]) <= BWD_TOL
    mask = np.ones(c.E, dtype=bool); mask[ed] = False
    assert np.all(g_rv[mask] == 0)


@pytest.mark.parametrize("name", list(CASES))
def test_force_loss_double_backward(name):
    """ggy, hx, hR for cotangents on (gx, g_rvec, gR): all three directions, single directions, partial outputs."""
    import torch
    c = GeoCase(CASES[name])
    d, i = c.d, c.plan.info
    v_r = np.random.default_rng(17).standard_normal((c.E, 3))
    v_rt = torch.from_numpy(v_r.astype(np.float32)).to("cuda:0")
    v_r = v_rt.cpu().numpy().astype(np.float64)

    def run(dirs=(True, True, True), outs=(True, True, True)):
        res = [c._new(c.N, i.C_y), c._new(c.N, i.C_x), c._new(i.K, i.N_w)]
        o = [t if on else None for t, on in zip(res, outs)]
        v = [t if on else None for t, on in zip((c.vx, v_rt, c.vR), dirs)]
        c.sb.conv_geo_dbwd(c.plan, c.graph, c.rvec, c.basis, c.w.r_c, 6, c.x, c.R, c.gy, *v, *o, c.ws(2))
        assert c.sb.last_device_status(c.ws(2)) == 0
        return [None if t is None else t.cpu().numpy() for t in o]

    def ref(dirs=(True, True, True)):
        z = lambda a, on: a if on else np.zeros_like(a)
        return geometry.geo_dbwd(c.oracle, d.row_ptr, d.col, c.o_rvec, d.x, d.R, d.gy, z(d.vx, dirs[0]), z(v_r, dirs[1]),
                                 z(d.vR, dirs[2]), c.w.r_c, c.basis)

    got, want = run(), ref()
    for a, b in zip(got, want):
        assert np.isfinite(a).all() and np.abs(b).max() > 1e-3 and rel_err(a, b) <= BWD_TOL
    # the direction on the edge vectors alone (the force term proper), and without it
    for dirs in [(False, True, False), (True, False, True)]:
        got, want = run(dirs), ref(dirs)
        for a, b in zip(got, want):
            assert rel_err(a, b) <= BWD_TOL if np.abs(b).max() > 0 else np.all(a == 0)
    full = run()
    part = run(outs=(False, True, False))
    assert part[0] is None and part[2] is None and np.array_equal(part[1], full[1])


@pytest.mark.parametrize("name", ["cfg2_N200", "cfg5_N60", "tc_K6_dense", "gauss_K12"])
def test_second_order_edge_vector_adjoint(name):
    """sobek_conv_geo_dbwd_full: ggy, hx, hR as the streaming double backward, and h_rvec = d<v, b>/d rvec (second
    derivatives of the spherical harmonics and the radial basis) against the oracle; single directions; NULL outputs."""
    import torch
    c = GeoCase(CASES[name])
    d, i = c.d, c.plan.info
    v_r = np.random.default_rng(19).standard_normal((c.E, 3))
    v_rt = torch.from_numpy(v_r.astype(np.float32)).to("cuda:0")
    v_r = v_rt.cpu().numpy().astype(np.float64)
    ws = torch.empty(c.sb.geo_dbwd_full_workspace_bytes(c.plan, c.N, c.E), dtype=torch.uint8, device="cuda:0")

    def run(dirs=(True, True, True), outs=(True, True, True, True)):
        res = [c._new(c.N, i.C_y), c._new(c.N, i.C_x), c._new(i.K, i.N_w), c._new(c.E, 3)]
        o = [t if on else None for t, on in zip(res, outs)]
        v = [t if on else None for t, on in zip((c.vx, v_rt, c.vR), dirs)]
        c.sb.conv_geo_dbwd_full(c.plan, c.graph, c.rvec, c.basis, c.w.r_c, 6, c.x, c.R, c.gy, *v, *o, ws)
        assert c.sb.last_device_status(ws) == 0
        return [None if t is None else t.cpu().numpy() for t in o]

    def ref(dirs=(True, True, True)):
        z = lambda a, on: a if on else np.zeros_like(a)
        return geometry.geo_dbwd(c.oracle, d.row_ptr, d.col, c.o_rvec, d.x, d.R, d.gy, z(d.vx, dirs[0]), z(v_r, dirs[1]),
                                 z(d.vR, dirs[2]), c.w.r_c, c.basis, with_h_rvec=True)

    got, want = run(), ref()
    for a, b, nm in zip(got, want, ("ggy", "hx", "hR", "h_rvec")):
        assert np.isfinite(a).all() and np.abs(b).max() > 1e-3 and rel_err(a, b) <= BWD_TOL, nm
    for dirs in [(False, True, False), (True, False, True)]:
        got, want = run(dirs), ref(dirs)
        for a, b, nm in zip(got, want, ("ggy", "hx", "hR", "h_rvec")):
            assert (rel_err(a, b) <= BWD_TOL if np.abs(b).max() > 0 else np.all(a == 0)), (dirs, nm)
    full = run()
    part = run(outs=(False, False, False, True))
    assert part[0] is None and part[1] is None and part[2] is None and np.array_equal(part[3], full[3])
    # the streaming entry point computes the same three outputs
    three = [c._new(c.N, i.C_y), c._new(c.N, i.C_x), c._new(i.K, i.N_w)]
    c.sb.conv_geo_dbwd(c.plan, c.graph, c.rvec, c.basis, c.w.r_c, 6, c.x, c.R, c.gy, c.vx, v_rt, c.vR, *three, c.ws(2))
    for a, t in zip(full[:3], three):
        assert rel_err(a, t.cpu().numpy().astype(np.float64)) <= BWD_TOL


def test_partial_outputs_and_argument_errors():
    c = GeoCase(CASES["cfg3_N120"])
    full = c.geo_bwd()
    for want in [(True, False, False), (False, True, False), (False, False, True), (True, True, False)]:
        got = c.geo_bwd(want)
        for a, b, on in zip(got, full, want):
            assert (a is None) == (not on)
            if on:
                assert np.array_equal(a, b)
    sb = c.sb
    y = c._new(c.N, c.plan.info.C_y)
    for bad in [dict(basis=7), dict(r_cut=0.0), dict(p=0)]:
        with pytest.raises(sb.SobekError) as e:
            sb.conv_geo_fwd(c.plan, c.graph, c.rvec, bad.get("basis", 0), bad.get("r_cut", 1.0), bad.get("p", 6),
                            c.x, c.R, y, c.ws(0))
        assert e.value.code == -1
    with pytest.raises(sb.SobekError) as e:
        sb.conv_geo_fwd(c.plan, c.graph, None, 0, 1.0, 6, c.x, c.R, y, c.ws(0))
    assert e.value.code == -1
    # a plan that runs the FP32-pipe edge kernels has no geometry mode
    c2 = GeoCase(CASES["cfg3_N120"], tc_stream=False)
    with pytest.raises(sb.SobekError) as e:
        c2.geo_fwd()
    assert e.value.code == -2


@pytest.mark.parametrize("name", ["uvu_16x3", "uvu_32x4_K16"])
def test_channelwise_mode(name):
    """The geometry front end in the channelwise (uvu) mode: same edge kernels, elementwise node-side steps."""
    import torch
    W = synth.Workload
    w = {"uvu_16x3": W("uvu_16x3", P("16x0e+16x1o+16x2e"), P("16x0e+16x1o+16x2e"), 2, 8, 150, 4.0, 1.5, "bessel", seed=7, mode="uvu"),
         "uvu_32x4_K16": W("uvu_32x4_K16", P("32x0e+32x1o+32x2e+32x3o"), P("32x0e+32x1o+32x2e+32x3o"), 3, 16, 80, 4.0, 1.7, "bessel",
                           seed=8, mode="uvu")}[name]
    c = GeoCase(w)
    d, i = c.d, c.plan.info
    y = c.geo_fwd()
    assert rel_err(y, geometry.geo_fwd(c.oracle, d.row_ptr, d.col, c.o_rvec, d.x, d.R, w.r_c, c.basis)) <= FWD_TOL
    got = c.geo_bwd()
    ref = geometry.geo_bwd(c.oracle, d.row_ptr, d.col, c.o_rvec, d.x, d.R, d.gy, w.r_c, c.basis)
    for a, b in zip(got, ref):
        assert np.abs(b).max() > 1e-4 and rel_err(a, b) <= BWD_TOL
    v_rt = torch.randn(c.E, 3, generator=torch.Generator().manual_seed(3)).to("cuda:0")
    ggy, hx, hR = c._new(c.N, i.C_y), c._new(c.N, i.C_x), c._new(i.K, i.N_w)
    c.sb.conv_geo_dbwd(c.plan, c.graph, c.rvec, c.basis, w.r_c, 6, c.x, c.R, c.gy, c.vx, v_rt, c.vR, ggy, hx, hR, c.ws(2))
    assert c.sb.last_device_status(c.ws(2)) == 0
    ref = geometry.geo_dbwd(c.oracle, d.row_ptr, d.col, c.o_rvec, d.x, d.R, d.gy, d.vx, v_rt.cpu().numpy().astype(np.float64),
                            d.vR, w.r_c, c.basis)
    for a, b in zip((ggy, hx, hR), ref):
        assert rel_err(a.cpu().numpy(), b) <= BWD_TOL


def test_graph_without_edges():
    """E = 0: zeros out, no edge array needed; and receivers without edges inside a graph give zero rows."""
    import torch
    import paper_2607_18074_b200 as sb
    w = CASES["cfg3_N120"]
    plan = sb.Plan(w.irreps_in, w.irreps_out, w.l_max, w.K)
    i, N = plan.info, 9
    dev = "cuda:0"
    rp = torch.zeros(N + 1, dtype=torch.int64, device=dev)
    col = torch.zeros(0, dtype=torch.int32, device=dev)
    g = sb.make_graph(rp, col, rp.clone(), col.clone(), col.clone())
    x = torch.randn(N, i.C_x, device=dev); R = torch.randn(i.K, i.N_w, device=dev); gy = torch.randn(N, i.C_y, device=dev)
    nan = lambda *s: torch.full(s, float("nan"), device=dev)
    ws = torch.empty(sb.workspace_bytes(plan, N, 0, 2), dtype=torch.uint8, device=dev)
    y = nan(N, i.C_y)
    sb.conv_geo_fwd(plan, g, None, 0, 1.0, 6, x, R, y, ws)
    gx, gR = nan(N, i.C_x), nan(i.K, i.N_w)
    sb.conv_geo_bwd(plan, g, None, 0, 1.0, 6, x, R, gy, gx, None, gR, ws)
    ggy, hx, hR = nan(N, i.C_y), nan(N, i.C_x), nan(i.K, i.N_w)
    sb.conv_geo_dbwd(plan, g, None, 0, 1.0, 6, x, R, gy, x, None, R, ggy, hx, hR, ws)
    gpos = nan(N, 3)
    sb.position_gradient(g, None, gpos)
    for t in (y, gx, gR, ggy, hx, hR, gpos):
        assert torch.all(t == 0)
    # a real graph in which the last three receivers lose their edges
    c = GeoCase(w)
    d = c.d
    cut = int(d.row_ptr[c.N - 3])
    rp2 = torch.from_numpy(np.minimum(d.row_ptr, cut).astype(np.int64)).to(dev)
    col2 = c.col[:cut].contiguous()
    sp, perm = sb.graph_prepare(rp2, col2)
    g2 = sb.make_graph(rp2, col2, sp, perm, sb.graph_receivers(rp2, perm))
    rvec2 = c.rvec[:cut].contiguous()
    y2 = c._new(c.N, c.plan.info.C_y)
    ws2 = torch.empty(sb.workspace_bytes(c.plan, c.N, cut, 1), dtype=torch.uint8, device=dev)
    sb.conv_geo_fwd(c.plan, g2, rvec2, c.basis, w.r_c, 6, c.x, c.R, y2, ws2)
    assert sb.last_device_status(ws2) == 0
    ref = geometry.geo_fwd(c.oracle, np.minimum(d.row_ptr, cut), d.col[:cut], c.o_rvec[:cut], d.x, d.R, w.r_c, c.basis)
    assert torch.all(y2[c.N - 3:] == 0) and rel_err(y2.cpu().numpy(), ref) <= FWD_TOL


def test_forces_rotate_with_the_positions():
    """Eq. energy_force_symmetry on the GPU path: the energy sum_i a . y_i[scalars] of invariant features is unchanged
    by a rotation of the positions and the forces rotate with them."""
    import torch
    w = CASES["cfg3_N120"]
    c = GeoCase(w)
    i = c.plan.info
    n0 = sum(m for m, l, p in w.irreps_out if l == 0)
    c0 = sum(m for m, l, p in w.irreps_in if l == 0)
    c.x[:, c0:] = 0
    a = torch.randn(n0, generator=torch.Generator().manual_seed(1)).to("cuda:0")
    c.gy.zero_(); c.gy[:, :n0] = a[None, :]

    def energy_forces(pos):
        c.sb.edge_vectors(c.graph, pos, c.rvec)
        y = torch.from_numpy(c.geo_fwd()).to("cuda:0")
        _, g_rv, _ = c.geo_bwd((False, True, False))
        gpos = c._new(c.N, 3)
        c.sb.position_gradient(c.graph, torch.from_numpy(g_rv).to("cuda:0"), gpos)
        return float((y * c.gy).sum()), -gpos.cpu().numpy()

    E0, F0 = energy_forces(c.pos)
    q = np.random.default_rng(3).standard_normal(4); q /= np.linalg.norm(q)
    a_, b_, c_, d_ = q
    Rm = np.array([[a_*a_+b_*b_-c_*c_-d_*d_, 2*(b_*c_-a_*d_), 2*(b_*d_+a_*c_)],
                   [2*(b_*c_+a_*d_), a_*a_-b_*b_+c_*c_-d_*d_, 2*(c_*d_-a_*b_)],
                   [2*(b_*d_-a_*c_), 2*(c_*d_+a_*b_), a_*a_-b_*b_-c_*c_+d_*d_]], dtype=np.float32)
    E1, F1 = energy_forces(c.pos @ torch.from_numpy(Rm.T.copy()).to("cuda:0"))
    scale = np.abs(F0).max()
    assert scale > 1e-3
    assert abs(E1 - E0) <= 1e-4 * max(1.0, abs(E0))
    assert np.abs(F1 - F0 @ Rm.T).max() <= 1e-3 * scale
    assert np.abs(F0.sum(0)).max() <= 1e-3 * scale * np.sqrt(c.N)
