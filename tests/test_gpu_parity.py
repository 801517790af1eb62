"""GPU parity: the CUDA library, called through its C ABI, against the fp64 oracle on the same
seeded inputs.  Element by element on small cases that still span several node chunks and
ragged multiplicities; on sampled receivers at the benchmark's full sizes."""
import numpy as np
import pytest

from oracle import conv as oconv
from workloads import synth

pytestmark = pytest.mark.gpu

from gpu_util import BWD_TOL, FWD_TOL, Case, rel_err  # noqa: E402

P = synth.parse_irreps


def small_cases():
    c = {}
    c["cfg1"] = synth.config("cfg1")
    c["cfg2_N200"] = synth.scaled(synth.config("cfg2"), 200)
    c["cfg3_N120"] = synth.scaled(synth.config("cfg3"), 120)
    c["cfg4_N150"] = synth.scaled(synth.config("cfg4"), 150)
    c["cfg5_N60"] = synth.scaled(synth.config("cfg5"), 60)
    c["cfg2_N700"] = synth.scaled(synth.config("cfg2"), 700)      # a chunk of 592 nodes or more: balanced processing order
    # ragged multiplicities, odd K, mixed parities (odd-sum paths), a block with no path
    c["ragged"] = synth.Workload("ragged", P("5x0e+3x1o+2x1e+33x2e"), P("7x0e+1x0o+35x1o+2x2e+3x3o+2x4e"),
                                 3, 3, 40, 4.0, 1.9, "gaussian", seed=3)
    c["K20"] = synth.Workload("K20", P("6x0e+4x1o"), P("6x0e+4x1o+2x2e"), 2, 20, 50, 4.0, 1.8, "bessel", seed=4)
    # tensor-core kernels off their main path: K below the padded width (and not a multiple of 4), multiplicities
    # that are multiples of 16 but not of 32, and receivers with well over 64 / 128 edges (several output groups)
    c["tc_K6_dense"] = synth.Workload("tc_K6_dense", P("16x0e+16x1o"), P("16x0e+16x1o+16x2e"), 2, 6, 160, 4.0, 3.6,
                                      "gaussian", seed=5)
    # a group whose paths mix a multiplicity that is a multiple of 4 with one that is not (row pitch and path offset
    # of the adjoint state are then odd): FP32-pipe kernels one way, tensor-core stream the other way
    c["mixed_align"] = synth.Workload("mixed_align", P("5x0e+96x1o"), P("16x0e+96x2e"), 2, 3, 114, 4.0, 1.9, "bessel", seed=11)
    c["tc_K12"] = synth.Workload("tc_K12", P("48x0e+16x1o+16x2e"), P("16x0e+48x1o"), 2, 12, 70, 4.0, 2.2, "bessel", seed=6)
    return c


CASES = small_cases()


@pytest.fixture(scope="module")
def cases():
    return {}


def get(cases, name):
    if name not in cases:
        cases[name] = Case(CASES[name])
    return cases[name]


@pytest.mark.parametrize("name", list(CASES))
def test_forward(cases, name):
    c = get(cases, name)
    assert rel_err(c.fwd(), c.o_fwd()) <= FWD_TOL


@pytest.mark.parametrize("name", list(CASES))
def test_backward(cases, name):
    c = get(cases, name)
    for got, ref, nm in zip(c.bwd(), c.o_bwd(), ("gx", "gY", "gphi", "gR")):
        assert rel_err(got, ref) <= BWD_TOL, nm


@pytest.mark.parametrize("name", list(CASES))
def test_double_backward(cases, name):
    c = get(cases, name)
    for got, ref, nm in zip(c.dbwd(), c.o_dbwd(), ("ggy", "hx", "hY", "hphi", "hR")):
        assert rel_err(got, ref) <= BWD_TOL, nm


@pytest.mark.parametrize("dirs", [(1, 0, 0, 0), (0, 1, 0, 0), (0, 0, 1, 0), (0, 0, 0, 1), (0, 0, 0, 0), (1, 0, 1, 0)])
def test_double_backward_null_directions(cases, dirs):
    c = get(cases, "cfg1")
    dirs = tuple(bool(v) for v in dirs)
    for got, ref, nm in zip(c.dbwd(dirs=dirs), c.o_dbwd(dirs=dirs), ("ggy", "hx", "hY", "hphi", "hR")):
        if np.abs(ref).max() == 0:
            assert np.all(got == 0), nm
        else:
            assert rel_err(got, ref) <= BWD_TOL, nm


def test_partial_outputs(cases):
    """NULL outputs are skipped and do not change the others."""
    import torch
    c = get(cases, "cfg1")
    sb, i = c.sb, c.plan.info
    full = c.bwd()
    gphi = torch.full((c.E, i.K), float("nan"), device="cuda:0")
    sb.conv_bwd(c.plan, c.graph, c.x, c.Y, c.phi, c.R, c.gy, None, None, gphi, None, c.ws(1))
    assert np.array_equal(gphi.cpu().numpy(), full[2])
    gx = torch.full((c.N, i.C_x), float("nan"), device="cuda:0")
    sb.conv_bwd(c.plan, c.graph, c.x, c.Y, c.phi, c.R, c.gy, gx, None, None, None, c.ws(1))
    assert np.array_equal(gx.cpu().numpy(), full[0])


def test_bitwise_reproducible(cases):
    c = get(cases, "cfg2_N200")
    assert np.array_equal(c.fwd(), c.fwd())
    for a, b in zip(c.bwd(), c.bwd()):
        assert np.array_equal(a, b)
    for a, b in zip(c.dbwd(), c.dbwd()):
        assert np.array_equal(a, b)


def test_graph_prepare_bit_exact(cases):
    for name in ("cfg1", "cfg2_N200", "ragged"):
        c = get(cases, name)
        sp, perm = oconv.sender_view(c.d.row_ptr, c.d.col)
        assert np.array_equal(c.src_ptr.cpu().numpy(), sp)
        assert np.array_equal(c.src_perm.cpu().numpy(), perm)
        # receiver of every edge of the sender-sorted view
        recv_of_edge = np.repeat(np.arange(c.d.N), np.diff(c.d.row_ptr))
        assert np.array_equal(c.src_recv.cpu().numpy(), recv_of_edge[perm].astype(np.int32))


def test_graph_prepare_large_and_hub():
    """A hub sender with thousands of out-edges and many empty rows."""
    import torch
    import paper_2607_18074_b200 as sb
    rng = np.random.default_rng(0)
    N, E = 5000, 60000
    recv = np.sort(rng.integers(0, N // 2, E))          # upper half of the nodes receives nothing
    col = rng.integers(0, N, E).astype(np.int32)
    col[rng.random(E) < 0.2] = 17                         # hub
    row_ptr = np.concatenate([[0], np.cumsum(np.bincount(recv, minlength=N))]).astype(np.int64)
    sp, perm = sb.graph_prepare(torch.from_numpy(row_ptr).cuda(), torch.from_numpy(col).cuda())
    assert np.array_equal(perm.cpu().numpy(), np.argsort(col, kind="stable").astype(np.int32))
    assert np.array_equal(sp.cpu().numpy(), np.concatenate([[0], np.cumsum(np.bincount(col, minlength=N))]))


def test_graph_prepare_rejects_bad_graphs():
    import torch
    import paper_2607_18074_b200 as sb
    rp = torch.tensor([0, 2, 1, 3], dtype=torch.int64, device="cuda:0")       # not monotone
    col = torch.tensor([0, 1, 2], dtype=torch.int32, device="cuda:0")
    with pytest.raises(sb.SobekError) as ei:
        sb.graph_prepare(rp, col)
    assert ei.value.code == -4
    rp = torch.tensor([0, 1, 2, 3], dtype=torch.int64, device="cuda:0")
    col = torch.tensor([0, 7, 2], dtype=torch.int32, device="cuda:0")         # sender out of range
    with pytest.raises(sb.SobekError) as ei:
        sb.graph_prepare(rp, col)
    assert ei.value.code == -4


def test_degenerate_graphs():
    """No edges at all; empty receivers, self loops and duplicate edges."""
    import torch
    import paper_2607_18074_b200 as sb
    ii, io = P("3x0e+2x1o"), P("2x0e+3x1o+1x2e")
    o = oconv.Oracle(ii, io, 2, 4)
    plan = sb.Plan(ii, io, 2, 4)
    rng = np.random.default_rng(0)
    for row_ptr, col in [(np.zeros(6, dtype=np.int64), np.zeros(0, dtype=np.int32)),
                         (np.array([0, 0, 3, 3, 4, 4], dtype=np.int64), np.array([1, 2, 2, 0], dtype=np.int32))]:
        N, E = 5, col.shape[0]
        f = lambda *s: rng.standard_normal(s).astype(np.float32)
        x, Y, phi, R, gy = f(N, o.C_x), f(E, 9), f(E, 4), f(4, o.N_w), f(N, o.C_y)
        t = lambda a: torch.from_numpy(a).cuda()
        rp_d, col_d = t(row_ptr), t(col)
        sp, perm = sb.graph_prepare(rp_d, col_d)
        g = sb.make_graph(rp_d, col_d, sp, perm)
        ws = torch.empty(sb.workspace_bytes(plan, N, E, 1), dtype=torch.uint8, device="cuda:0")
        y = torch.full((N, o.C_y), float("nan"), device="cuda:0")
        sb.conv_fwd(plan, g, t(x), t(Y), t(phi), t(R), y, ws)
        ref = o.fwd(row_ptr, col, x, Y, phi, R)
        assert np.abs(y.cpu().numpy() - ref).max() <= FWD_TOL * max(np.abs(ref).max(), 1e-30)
        outs = [torch.full(s, float("nan"), device="cuda:0") for s in ((N, o.C_x), (E, 9), (E, 4), (4, o.N_w))]
        sb.conv_bwd(plan, g, t(x), t(Y), t(phi), t(R), t(gy), *outs, ws)
        for got, r in zip(outs, o.bwd(row_ptr, col, x, Y, phi, R, gy)):
            assert rel_err(got.cpu().numpy(), r) <= BWD_TOL


def test_errors_on_device_calls(cases):
    import ctypes
    import torch
    c = get(cases, "cfg1")
    sb = c.sb
    y = torch.empty(c.N, c.plan.info.C_y, device="cuda:0")
    small = torch.empty(256, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(sb.SobekError) as ei:
        sb.conv_fwd(c.plan, c.graph, c.x, c.Y, c.phi, c.R, y, small)
    assert ei.value.code == -3
    g = sb.make_graph(c.row_ptr, c.col)          # no sender view
    gx = torch.empty(c.N, c.plan.info.C_x, device="cuda:0")
    with pytest.raises(sb.SobekError) as ei:
        sb.conv_bwd(c.plan, g, c.x, c.Y, c.phi, c.R, c.gy, gx, None, None, None, c.ws(1))
    assert ei.value.code == -5


@pytest.mark.parametrize("name,fp32_pipe", [("cfg1", False), ("cfg1", True), ("tc_K6_dense", False), ("cfg2_N700", False)])
def test_stale_graph_arrays_are_reported_not_followed(name, fp32_pipe):
    """The graph arrays are the caller's: an entry that is out of range when a kernel reads it (a freed or
    overwritten buffer) must end in SOBEK_ERR_GRAPH in the status word with finite outputs, never in an
    access through the bad value.  One corrupted entry per array, positive and negative, all three orders."""
    import torch
    opts = dict(tc_stream=False, tc_edge=False) if fp32_pipe else {}
    c = Case(CASES[name], **opts)          # cfg1: tensor-core stream + FP32-pipe edge pass; tc_K6_dense: both on tensor cores
    sb, i = c.sb, c.plan.info
    names = ("row_ptr", "col", "src_ptr", "src_perm", "src_recv")
    new = lambda *s: torch.full(s, float("nan"), dtype=torch.float32, device="cuda:0")
    for which, pos, bad in (("col", 5, c.N + 1000), ("col", 0, -3), ("src_recv", 7, 2 ** 30), ("src_recv", 1, -1),
                            ("src_perm", 3, c.E + 5), ("src_perm", c.E - 1, -7), ("row_ptr", c.N, c.E + 1000),
                            ("row_ptr", 3, -4), ("src_ptr", 2, 2 ** 40)):
        arrs = {n: getattr(c, n).clone() for n in names}
        arrs[which][pos] = bad
        g = sb.make_graph(*[arrs[n] for n in names])
        assert all(a is b for a, b in zip(g.tensors, [arrs[n] for n in names]))     # the descriptor keeps them alive
        touched = {"col": (0, 1, 2), "row_ptr": (0, 1, 2)}.get(which, (1, 2))        # the forward reads only the receiver CSR
        if which == "src_recv" and fp32_pipe:
            touched = ()          # the FP32-pipe traversal looks receivers up in row_ptr and never reads src_recv
        for order in (0, 1, 2):
            ws = c.ws(order)
            if order == 0:
                outs = [new(c.N, i.C_y)]
                sb.conv_fwd(c.plan, g, c.x, c.Y, c.phi, c.R, *outs, ws)
            elif order == 1:
                outs = [new(c.N, i.C_x), new(c.E, i.dim_sh), new(c.E, i.K), new(i.K, i.N_w)]
                sb.conv_bwd(c.plan, g, c.x, c.Y, c.phi, c.R, c.gy, *outs, ws)
            else:
                outs = [new(c.N, i.C_y), new(c.N, i.C_x), new(c.E, i.dim_sh), new(c.E, i.K), new(i.K, i.N_w)]
                sb.conv_dbwd(c.plan, g, c.x, c.Y, c.phi, c.R, c.gy, c.vx, c.vY, c.vphi, c.vR, *outs, ws)
            status = sb.last_device_status(ws)
            assert status == (-4 if order in touched else 0), (which, pos, order, status)
            for o in outs:
                assert torch.isfinite(o).all(), (which, pos, order)
    # and the context is intact: the untouched graph still gives the right answer
    assert rel_err(c.fwd(), c.o_fwd()) <= FWD_TOL


def test_misaligned_arrays_are_refused(cases):
    """Floating-point arrays must start on a 16-byte boundary (16-byte pieces of their rows are copied)."""
    import torch
    c = get(cases, "cfg1")
    sb = c.sb
    y = torch.empty(c.N, c.plan.info.C_y, device="cuda:0")
    buf = torch.empty(c.phi.numel() + 4, dtype=torch.float32, device="cuda:0")
    phi1 = buf[1:1 + c.phi.numel()].view_as(c.phi)       # 4 bytes off
    phi1.copy_(c.phi)
    with pytest.raises(sb.SobekError) as ei:
        sb.conv_fwd(c.plan, c.graph, c.x, c.Y, phi1, c.R, y, c.ws(0))
    assert ei.value.code == -1


# ---------------------------------------------------------------------------------------
# benchmark-sized workloads, in the configuration bench.py times: sampled receivers
# ---------------------------------------------------------------------------------------
FULL = {
    "cfg2": (synth.config("cfg2"), 48, (0, 1, 2)),
    "cfg3": (synth.config("cfg3"), 6, (0, 1, 2)),
    "cfg4_1e5": (synth.config("cfg4", edges=1e5), 8, (0, 1)),
    "cfg4_1e6": (synth.config("cfg4", edges=1e6), 8, (0, 1)),
    "cfg4t_10": (synth.config("cfg4t_10"), 8, (0, 1)),          # 1e7 edges: ten copies of the 1e6-edge graph
    "cfg5": (synth.config("cfg5"), 3, (0, 1, 2)),
}


@pytest.mark.parametrize("name", list(FULL))
def test_full_size_sampled(name):
    w, n_sample, orders = FULL[name]
    c = Case(w)
    rng = np.random.default_rng(123)
    # spread the sample over the node range so that several chunks are hit
    act = np.sort(rng.choice(c.N, size=n_sample, replace=False))
    act[0], act[-1] = 0, c.N - 1
    act = np.unique(act)
    ed = c.edges_into(act)
    y = c.fwd()
    assert np.isfinite(y).all()
    assert rel_err(y[act], c.o_fwd(act)[act]) <= FWD_TOL
    gym = c.masked_gy(act)
    if 1 in orders:
        got = c.bwd(gy=gym)
        ref = c.o_bwd(act)
        assert rel_err(got[0], ref[0]) <= BWD_TOL          # gx: every sender
        assert rel_err(got[3], ref[3]) <= BWD_TOL          # gR
        assert rel_err(got[1][ed], ref[1][ed]) <= BWD_TOL and rel_err(got[2][ed], ref[2][ed]) <= BWD_TOL
        mask = np.ones(c.E, dtype=bool); mask[ed] = False
        assert np.all(got[1][mask] == 0) and np.all(got[2][mask] == 0)
    if 2 in orders:
        got = c.dbwd(gy=gym)
        ref = c.o_dbwd(act)
        assert rel_err(got[0][act], ref[0][act]) <= BWD_TOL
        assert rel_err(got[1], ref[1]) <= BWD_TOL and rel_err(got[4], ref[4]) <= BWD_TOL
        assert rel_err(got[2][ed], ref[2][ed]) <= BWD_TOL and rel_err(got[3][ed], ref[3][ed]) <= BWD_TOL


# ---------------------------------------------------------------------------------------
# the top of the edge-scaling sweep (section "Scaling axes"): 5e7, 1e8 and 1.4e8 edges
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("copies", [50, 100, 140])
def test_edge_sweep_top_sampled(copies):
    """Forward and backward of the sweep profile on `copies` disjoint copies of its 1e6-edge graph (5.0e7 / 1.0e8 /
    1.4e8 edges, up to 4.4 M nodes; with 140 copies E*K and N*C_x both pass 2^31, so that every offset of the kernels
    has to be 64-bit).  A receiver only sees its own copy, so the oracle is run on single copies: on the sampled
    receivers of three copies (first, middle, last) with that copy's features, with the output adjoint zero outside the
    sample.  Checked: y of the sampled receivers, gY / gphi of their edges, gx of the three copies (and exact zeros in
    the copies in between), gR (= the sum over the copies' oracle runs)."""
    import torch
    import paper_2607_18074_b200 as sb
    w = synth.config(f"cfg4t_{copies}")
    oracle = oconv.Oracle(w.irreps_in, w.irreps_out, w.l_max, w.K)
    plan = sb.Plan(w.irreps_in, w.irreps_out, w.l_max, w.K)
    d = synth.make_inputs(w, oracle.col_std(), with_cotangents=False)
    n1, B = w.N, copies
    e1 = d.E // B
    assert d.N == n1 * B and d.E == e1 * B
    if copies == 140:
        assert d.E * w.K > 2 ** 31 and d.N * plan.info.C_x > 2 ** 31
    dev = "cuda:0"
    t = lambda a: torch.from_numpy(a).to(dev)
    row_ptr, col = t(d.row_ptr.astype(np.int64)), t(d.col)
    src_ptr, src_perm = sb.graph_prepare(row_ptr, col)
    src_recv = sb.graph_receivers(row_ptr, src_perm)
    g = sb.make_graph(row_ptr, col, src_ptr, src_perm, src_recv)
    x, Y, phi, R = t(d.x), t(d.Y), t(d.phi), t(d.R)
    rng = np.random.default_rng(7)
    check = [0, B // 2, B - 1]
    local = {b: np.unique(np.concatenate([[0, n1 - 1], rng.choice(n1, size=2, replace=False)])) for b in check}
    i = plan.info
    # ---- forward
    ws = torch.empty(sb.workspace_bytes(plan, d.N, d.E, 0), dtype=torch.uint8, device=dev)
    y = torch.full((d.N, i.C_y), float("nan"), dtype=torch.float32, device=dev)
    sb.conv_fwd(plan, g, x, Y, phi, R, y, ws)
    assert sb.last_device_status(ws) == 0
    assert bool(torch.isfinite(y).all())
    base_rp = d.row_ptr[:n1 + 1].astype(np.int64)
    base_col = d.col[:e1].astype(np.int32)
    for b in check:
        act = local[b]
        ref = oracle.fwd(base_rp, base_col, d.x[b * n1:(b + 1) * n1], d.Y[b * e1:(b + 1) * e1], d.phi[b * e1:(b + 1) * e1],
                         d.R, act=act)
        got = y[b * n1 + torch.from_numpy(act).to(dev)].cpu().numpy()
        assert rel_err(got, ref[act]) <= FWD_TOL, b
    del y, ws
    torch.cuda.empty_cache()
    # ---- backward, output adjoint supported on the sampled receivers
    gy_host = np.zeros((d.N, i.C_y), dtype=np.float32)
    for b in check:
        gy_host[b * n1 + local[b]] = d.gy[b * n1 + local[b]]
    gy = t(gy_host)
    ws = torch.empty(sb.workspace_bytes(plan, d.N, d.E, 1), dtype=torch.uint8, device=dev)
    new = lambda *s: torch.full(s, float("nan"), dtype=torch.float32, device=dev)
    gx, gY, gphi, gR = new(d.N, i.C_x), new(d.E, i.dim_sh), new(d.E, i.K), new(i.K, i.N_w)
    sb.conv_bwd(plan, g, x, Y, phi, R, gy, gx, gY, gphi, gR, ws)
    assert sb.last_device_status(ws) == 0
    gR_ref = np.zeros((i.K, i.N_w))
    for b in check:
        act = local[b]
        rx, rY, rphi, rR = oracle.bwd(base_rp, base_col, d.x[b * n1:(b + 1) * n1], d.Y[b * e1:(b + 1) * e1],
                                      d.phi[b * e1:(b + 1) * e1], d.R, gy_host[b * n1:(b + 1) * n1], act=act)
        gR_ref += rR
        assert rel_err(gx[b * n1:(b + 1) * n1].cpu().numpy(), rx) <= BWD_TOL, b
        ed = np.concatenate([np.arange(base_rp[r], base_rp[r + 1]) for r in act])
        ge = torch.from_numpy(b * e1 + ed).to(dev)
        assert rel_err(gY[ge].cpu().numpy(), rY[ed]) <= BWD_TOL, b
        assert rel_err(gphi[ge].cpu().numpy(), rphi[ed]) <= BWD_TOL, b
    assert rel_err(gR.cpu().numpy(), gR_ref) <= BWD_TOL
    # copies without a sampled receiver get exact zeros
    other = 1 if B > 3 else None
    if other is not None:
        assert float(gx[other * n1:(other + 1) * n1].abs().max()) == 0.0
        assert float(gY[other * e1:(other + 1) * e1].abs().max()) == 0.0
    assert bool(torch.isfinite(gx).all()) and bool(torch.isfinite(gphi).all())


# ---------------------------------------------------------------------------------------
# the fused schedule (edge stream feeding the tensor core without leaving the SM)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["cfg2_N200", "cfg4_N150", "cfg5_N60", "ragged", "K20"])
def test_fused_schedule(name):
    """The plan-level schedule switch (SOBEK_FLAG_FUSED_FP32) selects the fused stream+contraction kernels for
    y, gx, ggy and hx; results must match the oracle to the same tolerances."""
    c = Case(CASES[name], fused=True)
    assert rel_err(c.fwd(), c.o_fwd()) <= FWD_TOL
    for got, ref, nm in zip(c.bwd(), c.o_bwd(), ("gx", "gY", "gphi", "gR")):
        assert rel_err(got, ref) <= BWD_TOL, nm
    # hR not requested: ggy then comes from the fused directional kernel as well
    import torch
    i = c.plan.info
    new = lambda *s: torch.full(s, float("nan"), dtype=torch.float32, device="cuda:0")
    ggy, hx = new(c.N, i.C_y), new(c.N, i.C_x)
    c.sb.conv_dbwd(c.plan, c.graph, c.x, c.Y, c.phi, c.R, c.gy, c.vx, c.vY, c.vphi, c.vR, ggy, hx, None, None,
                   None, c.ws(2))
    ref = c.o_dbwd()
    assert rel_err(ggy.cpu().numpy(), ref[0]) <= BWD_TOL and rel_err(hx.cpu().numpy(), ref[1]) <= BWD_TOL
    for got, r, nm in zip(c.dbwd(), ref, ("ggy", "hx", "hY", "hphi", "hR")):
        assert rel_err(got, r) <= BWD_TOL, nm


# ---------------------------------------------------------------------------------------
# the FP32-pipe edge kernels (used where the tensor-core kernels do not apply), forced for whole plans
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["cfg1", "cfg2_N200", "cfg4_N150", "ragged"])
def test_fp32_pipe_edge_kernels(name):
    """SOBEK_FLAG_FP32_STREAM / SOBEK_FLAG_FP32_EDGE at plan creation select the FP32-pipe stream and edge pass
    for every traversal; all three orders must match the oracle to the same tolerances."""
    c = Case(CASES[name], tc_stream=False, tc_edge=False)
    assert rel_err(c.fwd(), c.o_fwd()) <= FWD_TOL
    for got, ref, nm in zip(c.bwd(), c.o_bwd(), ("gx", "gY", "gphi", "gR")):
        assert rel_err(got, ref) <= BWD_TOL, nm
    for got, ref, nm in zip(c.dbwd(), c.o_dbwd(), ("ggy", "hx", "hY", "hphi", "hR")):
        assert rel_err(got, ref) <= BWD_TOL, nm


def test_sender_view_without_receiver_ids(cases):
    """src_recv is optional: without it the transposed traversal looks the receivers up in row_ptr."""
    import paper_2607_18074_b200 as sb
    c = get(cases, "cfg2_N200")
    g = sb.make_graph(c.row_ptr, c.col, c.src_ptr, c.src_perm)
    import torch
    gx = torch.full((c.N, c.plan.info.C_x), float("nan"), dtype=torch.float32, device="cuda:0")
    sb.conv_bwd(c.plan, g, c.x, c.Y, c.phi, c.R, c.gy, gx, None, None, None, c.ws(1))
    assert rel_err(gx.cpu().numpy(), c.o_bwd()[0]) <= BWD_TOL


# ---------------------------------------------------------------------------------------
# the paper's scaling axes (section "Scaling axes"): long neighbourhoods, many small graphs
# ---------------------------------------------------------------------------------------
AXES = {
    "deg_4": (6, (0, 1, 2)),         # mean degree 4: isolated receivers and receivers with one edge
    "deg_1023": (2, (0, 1, 2)),      # 341 ... 1850 edges per receiver (dozens of edge batches each)
    "graphs_31": (6, (0, 1, 2)),     # one 128-node graph repeated 31 times
}


@pytest.mark.parametrize("name", list(AXES))
def test_scaling_axes_sampled(name):
    n_sample, orders = AXES[name]
    FULL[name] = (synth.config(name), n_sample, orders)
    try:
        test_full_size_sampled(name)
    finally:
        del FULL[name]


def test_balanced_processing_order():
    """From 592 nodes per chunk on, the tensor-core edge kernels take the nodes of a chunk longest neighbourhood first
    in alternating rounds (a per-chunk counting sort of the degrees) instead of by index: every output of every order
    against the oracle on a graph large enough for that, with hubs, isolated nodes and several chunks."""
    w = synth.scaled(synth.config("cfg2"), 1500)
    c = Case(w, state_budget_mib=32)             # about 35 KB of state per node: two chunks of 750 to 1,100 nodes
    assert rel_err(c.fwd(), c.o_fwd()) <= FWD_TOL
    for got, ref, nm in zip(c.bwd(), c.o_bwd(), ("gx", "gY", "gphi", "gR")):
        assert rel_err(got, ref) <= BWD_TOL, nm
    for got, ref, nm in zip(c.dbwd(), c.o_dbwd(), ("ggy", "hx", "hY", "hphi", "hR")):
        assert rel_err(got, ref) <= BWD_TOL, nm
    assert np.array_equal(c.fwd(), c.fwd())


def test_scratch_budget():
    """The scratch budget (section "Runtime scratch-budget policy") only changes the chunking: with the
    paper's 128 MiB the workspace shrinks and every output still matches the oracle."""
    import paper_2607_18074_b200 as sb
    w = synth.scaled(synth.config("cfg4", edges=1e5), 1500)
    big = Case(w)
    small = Case(w, inputs=big.d, state_budget_mib=128)
    for order in (0, 1, 2):
        assert sb.workspace_bytes(small.plan, w.N, small.E, order) < sb.workspace_bytes(big.plan, w.N, big.E, order)
    rng = np.random.default_rng(5)
    act = np.unique(np.concatenate([[0, big.N - 1], rng.choice(big.N, size=6, replace=False)]))
    ed = big.edges_into(act)
    assert rel_err(small.fwd()[act], big.o_fwd(act)[act]) <= FWD_TOL
    assert np.array_equal(small.fwd(), big.fwd())            # the forward does not depend on the chunking at all
    got = small.bwd(gy=small.masked_gy(act))
    ref = big.o_bwd(act)
    assert rel_err(got[0], ref[0]) <= BWD_TOL and rel_err(got[3], ref[3]) <= BWD_TOL
    assert rel_err(got[1][ed], ref[1][ed]) <= BWD_TOL and rel_err(got[2][ed], ref[2][ed]) <= BWD_TOL
    got = small.dbwd(gy=small.masked_gy(act))
    ref = big.o_dbwd(act)
    assert rel_err(got[0][act], ref[0][act]) <= BWD_TOL
    assert rel_err(got[1], ref[1]) <= BWD_TOL and rel_err(got[4], ref[4]) <= BWD_TOL
    assert rel_err(got[2][ed], ref[2][ed]) <= BWD_TOL and rel_err(got[3][ed], ref[3][ed]) <= BWD_TOL


@pytest.mark.parametrize("name", ["cfg2_N200", "uvu_32x4_K16"])
def test_cuda_graph_capture(cases, name):
    """A call neither allocates nor synchronises, and its side streams fork from and join the caller's
    stream with events, so the three orders can be captured into one CUDA graph and replayed (fully connected mode;
    channelwise mode with its direct kernels)."""
    import torch
    import paper_2607_18074_b200 as sb
    c = get(cases, name) if name in CASES else Case(uvu_cases()[name])
    i = c.plan.info
    eager = [c.fwd()] + c.bwd() + c.dbwd()
    new = lambda *s: torch.full(s, float("nan"), dtype=torch.float32, device="cuda:0")
    y = new(c.N, i.C_y)
    gx, gY, gphi, gR = new(c.N, i.C_x), new(c.E, i.dim_sh), new(c.E, i.K), new(i.K, i.N_w)
    ggy, hx, hY, hphi, hR = new(c.N, i.C_y), new(c.N, i.C_x), new(c.E, i.dim_sh), new(c.E, i.K), new(i.K, i.N_w)
    ws = c.ws(2)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        sb.conv_fwd(c.plan, c.graph, c.x, c.Y, c.phi, c.R, y, ws)
        sb.conv_bwd(c.plan, c.graph, c.x, c.Y, c.phi, c.R, c.gy, gx, gY, gphi, gR, ws)
        sb.conv_dbwd(c.plan, c.graph, c.x, c.Y, c.phi, c.R, c.gy, c.vx, c.vY, c.vphi, c.vR,
                     ggy, hx, hY, hphi, hR, ws)
    outs = (y, gx, gY, gphi, gR, ggy, hx, hY, hphi, hR)
    for _ in range(2):
        for t in outs:
            t.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert sb.last_device_status(ws) == 0
        for got, ref in zip(outs, eager):
            assert np.array_equal(got.cpu().numpy(), ref)


# ---------------------------------------------------------------------------------------
# channelwise (uvu) mode, Eq. uvu_connection: same edge kernels, elementwise node-side steps
# ---------------------------------------------------------------------------------------
def uvu_cases():
    W = synth.Workload
    c = {}
    # tensor-core edge kernels (multiplicities that are multiples of 16), several node chunks' worth of rows
    c["uvu_16x3"] = W("uvu_16x3", P("16x0e+16x1o+16x2e"), P("16x0e+16x1o+16x2e"), 2, 8, 150, 4.0, 1.5, "bessel", seed=7,
                      mode="uvu")
    c["uvu_32x4_K16"] = W("uvu_32x4_K16", P("32x0e+32x1o+32x2e+32x3o"), P("32x0e+32x1o+32x2e+32x3o"), 3, 16, 80, 4.0, 1.7,
                          "bessel", seed=8, mode="uvu")
    # 128 channels x 3 thread shares: the direct kernels split the channels into two slices of 64, one CTA each
    c["uvu_128x4_K16"] = W("uvu_128x4_K16", P("128x0e+128x1o+128x2e+128x3o"), P("128x0e+128x1o+128x2e+128x3o"), 3, 16, 40,
                           4.0, 1.7, "bessel", seed=11, mode="uvu")
    # FP32-pipe edge kernels: odd multiplicities, blocks of different multiplicity that no path couples, an
    # output block without an input twin (3x3e, fed by 4e only), a multiplicity above 128
    c["uvu_ragged"] = W("uvu_ragged", P("5x0e+5x1o+3x4e+2x0o"), P("5x0e+5x1o+3x4e+3x3e+2x0o"), 2, 3, 40, 4.0, 1.9,
                        "gaussian", seed=9, mode="uvu")
    c["uvu_wide"] = W("uvu_wide", P("144x0e+144x1o"), P("144x0e+144x1o"), 1, 8, 60, 4.0, 1.8, "bessel", seed=10, mode="uvu")
    return c


UVU = uvu_cases()


@pytest.fixture(scope="module")
def ucases():
    return {}


def uget(ucases, name):
    if name not in ucases:
        ucases[name] = Case(UVU[name])
    return ucases[name]


@pytest.mark.parametrize("name", list(UVU))
def test_uvu_forward(ucases, name):
    c = uget(ucases, name)
    assert c.plan.info.N_w == c.oracle.N_w
    assert rel_err(c.fwd(), c.o_fwd()) <= FWD_TOL


@pytest.mark.parametrize("name", list(UVU))
def test_uvu_backward(ucases, name):
    c = uget(ucases, name)
    for got, ref in zip(c.bwd(), c.o_bwd()):
        assert rel_err(got, ref) <= BWD_TOL


@pytest.mark.parametrize("name", list(UVU))
def test_uvu_double_backward(ucases, name):
    c = uget(ucases, name)
    for got, ref in zip(c.dbwd(), c.o_dbwd()):
        assert rel_err(got, ref) <= BWD_TOL


@pytest.mark.parametrize("dirs", [(1, 0, 0, 0), (0, 1, 0, 0), (0, 0, 1, 0), (0, 0, 0, 1)])
def test_uvu_double_backward_single_directions(ucases, dirs):
    c = uget(ucases, "uvu_16x3")
    for got, ref in zip(c.dbwd(dirs=dirs), c.o_dbwd(dirs=dirs)):
        assert rel_err(got, ref) <= BWD_TOL


def test_uvu_bitwise_reproducible_and_fp32_pipe_kernels(ucases):
    c = uget(ucases, "uvu_16x3")
    for a, b in zip([c.fwd()] + c.bwd() + c.dbwd(), [c.fwd()] + c.bwd() + c.dbwd()):
        assert np.array_equal(a, b)
    f = Case(UVU["uvu_16x3"], inputs=c.d, tc_stream=False, tc_edge=False)
    assert rel_err(f.fwd(), c.o_fwd()) <= FWD_TOL
    for got, ref in zip(f.bwd(), c.o_bwd()):
        assert rel_err(got, ref) <= BWD_TOL
    for got, ref in zip(f.dbwd(), c.o_dbwd()):
        assert rel_err(got, ref) <= BWD_TOL


@pytest.mark.parametrize("name", ["uvu_16x3", "uvu_32x4_K16", "uvu_128x4_K16"])
def test_uvu_direct_and_state_route_agree(name):
    """Uniform natural-parity profiles take the direct channelwise kernels for y, gx and gR by default; the route through
    the receiver state (SOBEK_FLAG_UVU_STATE) computes the same thing.  Both against the oracle."""
    c = Case(UVU[name])
    s = Case(UVU[name], inputs=c.d, uvu_state=True)
    ref = c.o_fwd()
    y_direct, y_state = c.fwd(), s.fwd()
    assert rel_err(y_direct, ref) <= FWD_TOL and rel_err(y_state, ref) <= FWD_TOL
    assert not np.array_equal(y_direct, y_state)        # two different kernels did run
    assert np.array_equal(y_direct, c.fwd())            # and the direct one repeats bitwise
    b_direct, b_state, b_ref = c.bwd(), s.bwd(), c.o_bwd()
    for got in (b_direct, b_state):
        for g, r in zip(got, b_ref):
            assert rel_err(g, r) <= BWD_TOL
    again = c.bwd()
    for k in (0, 3):                                    # gx and gR: direct kernels, repeatable bitwise
        assert not np.array_equal(b_direct[k], b_state[k])
        assert np.array_equal(b_direct[k], again[k])
    for k in (1, 2):                                    # gY, gphi take the same kernels on both plans
        assert np.array_equal(b_direct[k], b_state[k])


def test_uvu_full_size_sampled():
    """The paper's 128/128/128 channelwise profile (K = 16) on 31 copies of its 128-node graph."""
    FULL["uvu_128x3_31"] = (synth.config("uvu_128x3_31"), 6, (0, 1, 2))
    try:
        test_full_size_sampled("uvu_128x3_31")
    finally:
        del FULL["uvu_128x3_31"]


def test_uvu_plan_contract():
    import paper_2607_18074_b200 as sb
    ir = P("64x0e+64x1o+64x2e+64x3o")
    assert sb.Plan(ir, ir, 3, 16, mode="uvu").info.N_w == 1472          # Table uvu_capacity_matched
    with pytest.raises(sb.SobekError):
        sb.Plan(P("8x0e+4x1o"), P("8x0e+4x1o"), 1, 4, mode="uvu")      # 0e x 1o -> 1o would tie 8 to 4


# ---------------------------------------------------------------------------------------
# mul_ir boundary layout (SOBEK_FLAG_MUL_IR): the same operator with node features transposed per block
# ---------------------------------------------------------------------------------------
def _to_mul_ir(a, irreps):
    """[N, C] in ir_mul order (block offset + m*c + u) -> mul_ir order (block offset + u*d + m)."""
    out = np.empty_like(a)
    o = 0
    for c, l, _ in irreps:
        d = 2 * l + 1
        out[:, o:o + c * d] = a[:, o:o + c * d].reshape(-1, d, c).transpose(0, 2, 1).reshape(-1, c * d)
        o += c * d
    return out


@pytest.mark.parametrize("name,mode", [("cfg2_N200", "uvw"), ("ragged", "uvw"), ("uvu_16x3", "uvu")])
def test_mul_ir_layout(name, mode):
    import torch
    import paper_2607_18074_b200 as sb
    w = (UVU if mode == "uvu" else CASES)[name]
    ref = Case(w)                                   # ir_mul plan: outputs to compare with
    plan = sb.Plan(w.irreps_in, w.irreps_out, w.l_max, w.K, mode=mode, layout="mul_ir")
    assert plan.layout == "mul_ir" and plan.info.N_w == ref.plan.info.N_w
    d, i = ref.d, plan.info
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to("cuda:0")
    x, gy, vx = t(_to_mul_ir(d.x, w.irreps_in)), t(_to_mul_ir(d.gy, w.irreps_out)), t(_to_mul_ir(d.vx, w.irreps_in))
    ws = torch.empty(sb.workspace_bytes(plan, d.N, d.E, 2), dtype=torch.uint8, device="cuda:0")
    assert ws.numel() > sb.workspace_bytes(ref.plan, d.N, d.E, 2)
    new = lambda *s: torch.full(s, float("nan"), dtype=torch.float32, device="cuda:0")
    y = new(d.N, i.C_y)
    sb.conv_fwd(plan, ref.graph, x, ref.Y, ref.phi, ref.R, y, ws)
    assert np.array_equal(y.cpu().numpy(), _to_mul_ir(ref.fwd(), w.irreps_out))       # same kernels, same bits
    gx, gY, gphi, gR = new(d.N, i.C_x), new(d.E, i.dim_sh), new(d.E, i.K), new(i.K, i.N_w)
    sb.conv_bwd(plan, ref.graph, x, ref.Y, ref.phi, ref.R, gy, gx, gY, gphi, gR, ws)
    rb = ref.bwd()
    assert np.array_equal(gx.cpu().numpy(), _to_mul_ir(rb[0], w.irreps_in))
    for got, r in zip((gY, gphi, gR), rb[1:]):
        assert np.array_equal(got.cpu().numpy(), r)
    ggy, hx, hY, hphi, hR = new(d.N, i.C_y), new(d.N, i.C_x), new(d.E, i.dim_sh), new(d.E, i.K), new(i.K, i.N_w)
    sb.conv_dbwd(plan, ref.graph, x, ref.Y, ref.phi, ref.R, gy, vx, ref.vY, ref.vphi, ref.vR, ggy, hx, hY, hphi, hR, ws)
    rd = ref.dbwd()
    assert np.array_equal(ggy.cpu().numpy(), _to_mul_ir(rd[0], w.irreps_out))
    assert np.array_equal(hx.cpu().numpy(), _to_mul_ir(rd[1], w.irreps_in))
    for got, r in zip((hY, hphi, hR), rd[2:]):
        assert np.array_equal(got.cpu().numpy(), r)
    assert sb.last_device_status(ws) == 0
    # and against the oracle directly (forward), so that the layout itself is pinned, not only its consistency
    assert rel_err(y.cpu().numpy(), _to_mul_ir(ref.o_fwd(), w.irreps_out)) <= FWD_TOL
    # partial outputs through the re-layout: only hx
    hx2 = new(d.N, i.C_x)
    sb.conv_dbwd(plan, ref.graph, x, ref.Y, ref.phi, ref.R, gy, vx, ref.vY, ref.vphi, ref.vR, None, hx2, None, None, None, ws)
    assert np.array_equal(hx2.cpu().numpy(), hx.cpu().numpy())


def test_bounded_wait_gives_up_and_reports():
    """A device-side wait whose partner never arrives runs out after its limit, records DEVICE_TIMEOUT in the status
    word and the kernel returns: the context stays usable (the next call computes correct results)."""
    import time
    import torch
    import paper_2607_18074_b200 as sb
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda:0")
    t0 = time.time()
    sb.selftest_wait_timeout(ws, 200)
    assert sb.last_device_status(ws) == -7            # SOBEK_ERR_DEVICE_TIMEOUT
    dt = time.time() - t0
    assert 0.15 < dt < 5.0
    assert "timeout" in sb.status_string(-7).lower() or "wait" in sb.status_string(-7).lower()
    c = Case(CASES["cfg1"])
    assert rel_err(c.fwd(), c.o_fwd()) <= FWD_TOL


# ---------------------------------------------------------------------------------------
# randomised profiles: multiplicities, orders, parities, K, mode and graph drawn from a seed
# ---------------------------------------------------------------------------------------
def _random_workload(rng, it):
    mults = [8, 16, 24, 32, 48, 64, 96, 128, 5, 12]
    mode = "uvu" if rng.random() < 0.35 else "uvw"
    l_max = int(rng.integers(1, 4))
    K = int(rng.choice([3, 4, 8, 11, 16, 20]))

    def irreps(n, fixed=None):
        out = []
        for l in sorted(rng.choice(np.arange(0, 4), size=n, replace=False).tolist()):
            par = 1 if l % 2 == 0 else -1
            if rng.random() < 0.15:
                par = -par
            out.append((fixed if fixed is not None else int(rng.choice(mults)), int(l), par))
        return out

    n_in, n_out = int(rng.integers(1, 4)), int(rng.integers(1, 4))
    m = int(rng.choice(mults)) if mode == "uvu" else None
    ir_in, ir_out = irreps(n_in, m), irreps(n_out, m)
    big = rng.random() < 0.15
    N = int(rng.integers(600, 1200)) if big else int(rng.integers(20, 120))
    deg = float(rng.choice([3, 12])) if big else float(rng.choice([3, 12, 40]))
    L = 4.0 * (N / 60.0) ** (1 / 3)
    return synth.Workload(f"rnd{it}", ir_in, ir_out, l_max, K, N, L, float(synth.cutoff_for_edges(N, deg * N, L)), "bessel",
                          seed=int(rng.integers(1 << 30)), mode=mode)


@pytest.mark.parametrize("seed", [1, 2])
def test_random_profiles(seed):
    """Profiles nobody hand-picked: mixed and odd multiplicities, sparse path sets, both modes, K off the padded
    widths, tiny and multi-chunk graphs.  (A sweep of this kind found the odd-row-pitch profile `mixed_align`.)"""
    import paper_2607_18074_b200 as sb
    rng = np.random.default_rng(seed)
    ran = 0
    for it in range(45):
        w = _random_workload(rng, it)
        try:
            c = Case(w)
        except (sb.SobekError, ValueError):
            continue                  # no allowed path, or a uvu path between unequal multiplicities
        tag = f"seed {seed} case {it}: {w.mode} {w.irreps_in} -> {w.irreps_out} l_max={w.l_max} K={w.K} N={w.N}"
        assert rel_err(c.fwd(), c.o_fwd()) <= FWD_TOL, tag
        for got, ref in zip(c.bwd(), c.o_bwd()):
            assert rel_err(got, ref) <= BWD_TOL, tag
        for got, ref in zip(c.dbwd(), c.o_dbwd()):
            assert rel_err(got, ref) <= BWD_TOL, tag
        ran += 1
    assert ran >= 25


@pytest.mark.parametrize("name,mode", [("cfg2_N200", "uvw"), ("ragged", "uvw"), ("uvu_16x3", "uvu")])
def test_state_retained_from_forward(name, mode):
    """sobek_conv_fwd_retain leaves the receiver state in the workspace; sobek_conv_bwd_retained then computes gR
    from it without streaming the edges again: same bits as the plain calls, one stream launch fewer."""
    import torch
    import paper_2607_18074_b200 as sb
    # (a retaining forward goes through the state in either mode; the plain uvu forward compared with it must too)
    c = Case(UVU[name], uvu_state=True) if mode == "uvu" else Case(CASES[name])
    i = c.plan.info
    y_ref, b_ref = c.fwd(), c.bwd()
    new = lambda *s: torch.full(s, float("nan"), dtype=torch.float32, device="cuda:0")
    ws = c.ws(1)
    y = new(c.N, i.C_y)
    kept = sb.conv_fwd_retain(c.plan, c.graph, c.x, c.Y, c.phi, c.R, y, ws)
    assert kept == 1 and np.array_equal(y.cpu().numpy(), y_ref)
    outs = [new(c.N, i.C_x), new(c.E, i.dim_sh), new(c.E, i.K), new(i.K, i.N_w)]
    l0 = sb.launch_count()
    sb.conv_bwd_retained(c.plan, c.graph, c.x, c.Y, c.phi, c.R, c.gy, *outs, ws, kept)
    n_ret = sb.launch_count() - l0
    assert sb.last_device_status(ws) == 0
    for got, ref in zip(outs, b_ref):
        assert np.array_equal(got.cpu().numpy(), ref)
    l0 = sb.launch_count()
    sb.conv_bwd(c.plan, c.graph, c.x, c.Y, c.phi, c.R, c.gy, *outs, ws)
    assert sb.launch_count() - l0 > n_ret               # the plain call streams the edges once more
    # retained = 0 is the plain backward
    sb.conv_bwd_retained(c.plan, c.graph, c.x, c.Y, c.phi, c.R, c.gy, *outs, ws, 0)
    for got, ref in zip(outs, b_ref):
        assert np.array_equal(got.cpu().numpy(), ref)
    # a scratch budget that needs several chunks: nothing is retained, the results stay right
    if c.N >= 100:
        w2 = synth.scaled(synth.config("cfg2"), 1300)
        c2 = Case(w2, state_budget_mib=1)
        y2 = new(c2.N, c2.plan.info.C_y)
        assert sb.conv_fwd_retain(c2.plan, c2.graph, c2.x, c2.Y, c2.phi, c2.R, y2, c2.ws(1)) == 0
        assert np.array_equal(y2.cpu().numpy(), c2.fwd())


def test_fast_gemm_flag(cases):
    """SOBEK_FLAG_FAST_GEMM: the node-side GEMMs as single bf16 products.  Optional and outside the stated tolerances:
    close to the oracle at bf16 level, and not the same numbers as the default three-pass plan."""
    import torch
    import paper_2607_18074_b200 as sb
    c = get(cases, "cfg2_N200")
    w = c.w
    plan = sb.Plan(w.irreps_in, w.irreps_out, w.l_max, w.K, flags=sb.FLAG_FAST_GEMM)
    i = plan.info
    ws = torch.empty(sb.workspace_bytes(plan, c.N, c.E, 2), dtype=torch.uint8, device="cuda:0")
    new = lambda *s: torch.full(s, float("nan"), dtype=torch.float32, device="cuda:0")
    y = new(c.N, i.C_y)
    sb.conv_fwd(plan, c.graph, c.x, c.Y, c.phi, c.R, y, ws)
    e = rel_err(y.cpu().numpy(), c.o_fwd())
    assert FWD_TOL < e < 2e-2
    outs = [new(c.N, i.C_x), new(c.E, i.dim_sh), new(c.E, i.K), new(i.K, i.N_w)]
    sb.conv_bwd(plan, c.graph, c.x, c.Y, c.phi, c.R, c.gy, *outs, ws)
    for got, ref in zip(outs, c.o_bwd()):
        assert rel_err(got.cpu().numpy(), ref) < 2e-2
    outs = [new(c.N, i.C_y), new(c.N, i.C_x), new(c.E, i.dim_sh), new(c.E, i.K), new(i.K, i.N_w)]
    sb.conv_dbwd(plan, c.graph, c.x, c.Y, c.phi, c.R, c.gy, c.vx, c.vY, c.vphi, c.vR, *outs, ws)
    for got, ref in zip(outs, c.o_dbwd()):
        assert rel_err(got.cpu().numpy(), ref) < 2e-2
    assert sb.last_device_status(ws) == 0
