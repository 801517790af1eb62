"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares,
its host-side plan logic (path enumeration, Clebsch-Gordan tensors from the library's own
numerical route) agrees with the oracle's closed-form route, and argument errors are
reported as status codes.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2607_18074_b200 as sb
from oracle import tables
from workloads import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2607_18074_b200 import build
    build.build()


def test_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "sobek.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(sobek_[a-z_0-9]+)\s*\(", hdr))
    assert declared == set(sb.EXPORTS)
    L = ctypes.CDLL(sb.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings():
    assert sb.status_string(0) == "ok"
    for c in range(-7, 0):
        assert sb.status_string(c) not in ("ok", "unknown status")


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
def test_plan_paths_and_cg_match_oracle(name):
    w = synth.config(name)
    plan = sb.Plan(w.irreps_in, w.irreps_out, w.l_max, w.K)
    paths, n_w = tables.enumerate_paths(w.irreps_in, w.irreps_out, w.l_max)
    assert plan.info.N_w == n_w and plan.info.n_paths == len(paths)
    assert plan.info.C_x == synth.irreps_dim(w.irreps_in) and plan.info.C_y == synth.irreps_dim(w.irreps_out)
    for k, p in enumerate(paths):
        q = plan.path(k)
        assert (q.i_in, q.l_sh, q.i_out, q.l_in, q.l_out, q.c_in, q.c_out, q.in_off, q.sh_off, q.out_off,
                q.w_off) == (p.i_in, p.l_sh, p.i_out, p.l_in, p.l_out, p.c_in, p.c_out, p.in_off, p.sh_off,
                             p.out_off, p.w_off)
        assert np.abs(plan.cg(k) - p.cg).max() < 1e-9
    assert np.allclose(synth.plan_col_std(plan), tables.weight_col_std(w.irreps_in, w.irreps_out, w.l_max, w.K))


def test_cg_all_triples_including_odd_sums():
    ir_in = [(1, l, p) for l in range(5) for p in (1, -1)]
    plan = sb.Plan(ir_in, ir_in, 4, 1)
    paths, _ = tables.enumerate_paths(ir_in, ir_in, 4)
    assert plan.info.n_paths == len(paths)
    seen = set()
    for k, p in enumerate(paths):
        seen.add((p.l_in, p.l_sh, p.l_out))
        assert np.abs(plan.cg(k) - p.cg).max() < 1e-9
    assert len(seen) == sum(1 for a in range(5) for b in range(5) for c in range(abs(a - b), min(a + b, 4) + 1))


def test_state_widths():
    w = synth.config("cfg4")
    plan = sb.Plan(w.irreps_in, w.irreps_out, w.l_max, w.K)
    assert plan.info.state_floats_fwd == 35840          # K*F
    w = synth.config("cfg3")
    plan = sb.Plan(w.irreps_in, w.irreps_out, w.l_max, w.K)
    assert plan.info.state_floats_fwd == 40960 and plan.info.state_floats_bwd == 8 * 2816


def test_workspace_does_not_grow_with_edges():
    w = synth.config("cfg4")
    plan = sb.Plan(w.irreps_in, w.irreps_out, w.l_max, w.K, state_budget_mib=2048)      # (the default depends on the device)
    for order in (0, 1, 2):
        a = sb.workspace_bytes(plan, 3125, 10**5, order)
        assert a > 0
        # same node count, any edge count
        assert sb.workspace_bytes(plan, 3125, 10**9, order) == a
        # more nodes: the chunked state is bounded by its budget; what grows is only the bf16 (hi, lo)
        # copy of the node features that the tensor-core stream gathers from (4 bytes per feature)
        C_x, C_y = plan.info.C_x, plan.info.C_y
        per_node = 4 * (C_x + (C_y if order >= 1 else 0) + (C_x if order >= 2 else 0))
        per_node += 16 * (1 if order == 0 else 2)      # and the chunks' processing order of each view (one int4 per node)
        grow = sb.workspace_bytes(plan, 3 * 10**6, 10**8, order) - sb.workspace_bytes(plan, 10**6, 10**8, order)
        assert abs(grow - 2 * 10**6 * per_node) < 4096
        assert sb.workspace_bytes(plan, 10**6, 10**8, order) - 10**6 * per_node < 4300 * 2**20
    # the widest benchmark contract: bounded by the state budget (or 512 nodes) plus the feature copies, whatever the edge count
    w = synth.config("cfg5")
    plan = sb.Plan(w.irreps_in, w.irreps_out, w.l_max, w.K, state_budget_mib=2048)
    a = sb.workspace_bytes(plan, 50000, 2 * 10**6, 2)
    assert a == sb.workspace_bytes(plan, 50000, 4 * 10**8, 2)
    assert a - 50000 * 4 * (2 * plan.info.C_x + plan.info.C_y) < 5400 * 2**20


def test_argument_errors_are_status_codes():
    L = sb.lib()
    h = ctypes.c_void_p()
    ok = sb._irreps([(2, 0, 1)])
    assert L.sobek_plan_create(None, 1, ok, 1, 0, 4, 0, ctypes.byref(h)) == -1
    assert L.sobek_plan_create(ok, 1, ok, 1, 0, 0, 0, ctypes.byref(h)) == -1            # K < 1
    assert L.sobek_plan_create(ok, 1, ok, 1, 5, 4, 0, ctypes.byref(h)) == -2            # l_max too high
    assert L.sobek_plan_create(sb._irreps([(2, 0, 3)]), 1, ok, 1, 0, 4, 0, ctypes.byref(h)) == -1   # parity
    assert L.sobek_plan_create(sb._irreps([(2, 7, 1)]), 1, ok, 1, 0, 4, 0, ctypes.byref(h)) == -2   # l too high
    # no valid path: 0e x (0e) -> 0o
    assert L.sobek_plan_create(ok, 1, sb._irreps([(2, 0, -1)]), 1, 0, 4, 0, ctypes.byref(h)) == -2
    plan = sb.Plan([(2, 0, 1)], [(2, 0, 1)], 0, 4)
    g = sb.Graph(4, 0, None, None, None, None)
    assert L.sobek_conv_fwd(None, ctypes.byref(g), None, None, None, None, None, None, 0, None) == -1
    assert L.sobek_plan_path(plan.handle, 99, ctypes.byref(sb.PathInfo())) == -1
    assert sb.workspace_bytes(plan, 4, 0, 7) == 0
    assert L.sobek_last_device_status(None, None) == -1
    # geometry front end: null descriptors and arguments are refused before anything is launched
    assert L.sobek_edge_vectors(None, None, None, None) == -1
    assert L.sobek_position_gradient(None, None, None, None) == -1
    assert L.sobek_conv_geo_fwd(None, ctypes.byref(g), None, 0, 1.0, 6, None, None, None, None, 0, None) == -1
    g1 = sb.Graph(4, 1, None, None, None, None)
    assert L.sobek_conv_geo_fwd(plan.handle, ctypes.byref(g1), None, 0, 1.0, 6, None, None, None, None, 0, None) == -1   # no rvec
    assert L.sobek_conv_geo_bwd(plan.handle, ctypes.byref(g1), None, 5, 1.0, 6, None, None, None, None, None, None, None, 0, None) == -1
    assert L.sobek_conv_geo_dbwd(plan.handle, ctypes.byref(g1), None, 0, 1.0, 6, *([None] * 10), 0, None) == -1
    assert L.sobek_conv_geo_dbwd_full(None, ctypes.byref(g1), None, 0, 1.0, 6, *([None] * 11), 0, None) == -1
    assert L.sobek_conv_geo_dbwd_full(plan.handle, ctypes.byref(g1), None, 0, 1.0, 6, *([None] * 11), 0, None) == -1    # no rvec
    assert L.sobek_geo_dbwd_full_workspace_bytes(None, 4, 8) == 0


def test_uvu_plan_weight_counts_match_the_paper():
    """Channelwise mode (Eq. uvu_connection): N_w = sum of C_in over the paths; the paper prints it for nine
    profiles (Table uvu_capacity_matched)."""
    n = 0
    for line in open(os.path.join(ROOT, "tests", "golden", "paper_weight_counts.txt")):
        tok = line.split()
        if not tok or tok[0] != "uvu":
            continue
        mults = [int(v) for v in tok[1].split("/")]
        ir = [(m, l, 1 if l % 2 == 0 else -1) for l, m in enumerate(mults)]
        plan = sb.Plan(ir, ir, len(mults) - 1, 16, mode="uvu")
        assert plan.info.N_w == int(tok[2])
        paths, n_w = tables.enumerate_paths(ir, ir, len(mults) - 1, "uvu")
        assert [plan.path(k).w_off for k in range(plan.info.n_paths)] == [p.w_off for p in paths]
        n += 1
    assert n == 9


def test_uvu_plan_errors_and_workspace():
    P = synth.parse_irreps
    with pytest.raises(sb.SobekError):
        sb.Plan(P("8x0e+4x1o"), P("8x0e+4x1o"), 1, 4, mode="uvu")       # 0e x 1o -> 1o would tie 8 channels to 4
    with pytest.raises(sb.SobekError):
        sb.Plan(P("8x0e"), P("8x0e"), 0, 4, flags=1 << 10)              # unknown flag bit
    ir = P("64x0e+64x1o+64x2e")
    u, w = sb.Plan(ir, ir, 2, 16, mode="uvu"), sb.Plan(ir, ir, 2, 16)
    assert u.mode == "uvu" and w.mode == "uvw" and u.info.C_y == w.info.C_y
    for order in (0, 1, 2):
        a = sb.workspace_bytes(u, 3125, 10**5, order)
        assert a == sb.workspace_bytes(u, 3125, 10**9, order)            # nothing edge-sized
        assert a <= sb.workspace_bytes(w, 3125, 10**5, order)            # no GEMM operand copies of R


def test_mul_ir_flag_and_workspace():
    P = synth.parse_irreps
    ir = P("32x0e+32x1o+32x2e")
    a, b = sb.Plan(ir, ir, 2, 8), sb.Plan(ir, ir, 2, 8, layout="mul_ir")
    assert (a.layout, b.layout) == ("ir_mul", "mul_ir") and a.info.N_w == b.info.N_w
    N = 5000
    # the re-layout copies: x, y | + gy, gx | + vx   (4 bytes per node feature and array, 256-byte aligned)
    al = lambda n: (n + 255) & ~255
    cx = cy = a.info.C_x
    extra = [al(4 * N * cx) + al(4 * N * cy), 2 * (al(4 * N * cx) + al(4 * N * cy)), 3 * al(4 * N * cx) + 2 * al(4 * N * cy)]
    for order in (0, 1, 2):
        assert sb.workspace_bytes(b, N, 10**5, order) - sb.workspace_bytes(a, N, 10**5, order) == extra[order]
    assert sb.Plan(ir, ir, 2, 8, mode="uvu", layout="mul_ir").mode == "uvu"


def test_binding_declares_every_signature():
    """ctypes without argtypes passes Python ints as 32-bit C ints: a workspace size above 4 GiB would be truncated.
    Every exported entry point that takes arguments must have its signature declared."""
    L = sb.lib()
    no_args = {"sobek_static_scratch_bytes", "sobek_launch_count", "sobek_timing_classes"}
    for name in sb.EXPORTS:
        if name in no_args:
            continue
        assert getattr(L, name).argtypes is not None, name


def test_graph_descriptor_keeps_its_tensors_alive():
    """make_graph stores raw addresses in the C struct, so the returned object must hold the tensors."""
    import torch
    rp = torch.tensor([0, 1, 2], dtype=torch.int64)
    col = torch.tensor([1, 0], dtype=torch.int32)
    sp, perm, recv = rp.clone(), col.clone(), col.clone()
    g = sb.make_graph(rp, col, sp, perm, recv)
    assert g.N == 2 and g.E == 2
    assert [id(t) for t in g.tensors] == [id(t) for t in (rp, col, sp, perm, recv)]
    assert g.row_ptr == rp.data_ptr() and g.src_recv == recv.data_ptr()
    g2 = sb.make_graph(rp, col)
    assert g2.tensors[2] is None and not g2.src_ptr


def test_plan_option_flags():
    ir = [(8, 0, 1), (8, 1, -1)]
    for kw in (dict(fused=True), dict(tc_stream=False), dict(tc_edge=False), dict(state_budget_mib=128), dict(mode="uvu", uvu_state=True)):
        sb.Plan(ir, ir, 2, 8, **kw)
    with pytest.raises(sb.SobekError):
        sb.Plan(ir, ir, 2, 8, flags=1 << 11)            # an undefined flag bit
    with pytest.raises(ValueError):
        sb.Plan(ir, ir, 2, 8, state_budget_mib=0)
