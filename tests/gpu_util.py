"""Helpers for the GPU parity tests: run the CUDA library through its C ABI (via the thin
binding) and the fp64 oracle on the same seeded inputs."""
import numpy as np

from oracle import conv as oconv
from workloads import synth

FWD_TOL, BWD_TOL = 1e-4, 5e-4   # max|delta| <= tol * max|ref|


def rel_err(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    if ref.size == 0:
        return 0.0
    return float(np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30))


class Case:
    """One workload on the GPU and in the oracle."""

    def __init__(self, w: synth.Workload, inputs=None, **plan_options):
        import torch
        import paper_2607_18074_b200 as sb
        self.sb, self.torch = sb, torch
        self.w = w
        self.oracle = oconv.Oracle(w.irreps_in, w.irreps_out, w.l_max, w.K, mode=w.mode)
        self.plan = sb.Plan(w.irreps_in, w.irreps_out, w.l_max, w.K, mode=w.mode, **plan_options)
        self.d = inputs if inputs is not None else synth.make_inputs(w, self.oracle.col_std())
        d = self.d
        dev = "cuda:0"
        t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
        self.row_ptr, self.col = t(d.row_ptr.astype(np.int64)), t(d.col.astype(np.int32))
        self.x, self.Y, self.phi, self.R, self.gy = t(d.x), t(d.Y), t(d.phi), t(d.R), t(d.gy)
        self.vx, self.vY, self.vphi, self.vR = t(d.vx), t(d.vY), t(d.vphi), t(d.vR)
        self.src_ptr, self.src_perm = sb.graph_prepare(self.row_ptr, self.col)
        self.src_recv = sb.graph_receivers(self.row_ptr, self.src_perm)
        self.graph = sb.make_graph(self.row_ptr, self.col, self.src_ptr, self.src_perm, self.src_recv)
        self.N, self.E = d.N, d.E
        self._ws = {}

    def ws(self, order):
        if order not in self._ws:
            n = self.sb.workspace_bytes(self.plan, self.N, self.E, order)
            self._ws[order] = self.torch.empty(n, dtype=self.torch.uint8, device="cuda:0")
        return self._ws[order]

    def _new(self, *shape):
        # poison so that unwritten outputs are caught
        return self.torch.full(shape, float("nan"), dtype=self.torch.float32, device="cuda:0")

    def fwd(self):
        y = self._new(self.N, self.plan.info.C_y)
        self.sb.conv_fwd(self.plan, self.graph, self.x, self.Y, self.phi, self.R, y, self.ws(0))
        assert self.sb.last_device_status(self.ws(0)) == 0
        return y.cpu().numpy()

    def bwd(self, gy=None):
        i = self.plan.info
        gy = self.gy if gy is None else gy
        gx, gY = self._new(self.N, i.C_x), self._new(self.E, i.dim_sh)
        gphi, gR = self._new(self.E, i.K), self._new(i.K, i.N_w)
        self.sb.conv_bwd(self.plan, self.graph, self.x, self.Y, self.phi, self.R, gy, gx, gY, gphi, gR,
                         self.ws(1))
        assert self.sb.last_device_status(self.ws(1)) == 0
        return [a.cpu().numpy() for a in (gx, gY, gphi, gR)]

    def dbwd(self, gy=None, dirs=(True, True, True, True)):
        i = self.plan.info
        gy = self.gy if gy is None else gy
        ggy, hx, hY = self._new(self.N, i.C_y), self._new(self.N, i.C_x), self._new(self.E, i.dim_sh)
        hphi, hR = self._new(self.E, i.K), self._new(i.K, i.N_w)
        v = [t if on else None for t, on in zip((self.vx, self.vY, self.vphi, self.vR), dirs)]
        self.sb.conv_dbwd(self.plan, self.graph, self.x, self.Y, self.phi, self.R, gy, *v,
                          ggy, hx, hY, hphi, hR, self.ws(2))
        assert self.sb.last_device_status(self.ws(2)) == 0
        return [a.cpu().numpy() for a in (ggy, hx, hY, hphi, hR)]

    # oracle side
    def o_fwd(self, act=None):
        d = self.d
        return self.oracle.fwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R, act=act)

    def o_bwd(self, act=None):
        d = self.d
        return self.oracle.bwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R, d.gy, act=act)

    def o_dbwd(self, act=None, dirs=(True, True, True, True)):
        d = self.d
        v = [a if on else np.zeros_like(a) for a, on in zip((d.vx, d.vY, d.vphi, d.vR), dirs)]
        return self.oracle.dbwd(d.row_ptr, d.col, d.x, d.Y, d.phi, d.R, d.gy, *v, act=act)

    def masked_gy(self, act):
        m = self.torch.zeros_like(self.gy)
        idx = self.torch.from_numpy(np.asarray(act, dtype=np.int64)).to("cuda:0")
        m[idx] = self.gy[idx]
        return m

    def edges_into(self, act):
        d = self.d
        return np.concatenate([np.arange(d.row_ptr[i], d.row_ptr[i + 1]) for i in act]).astype(np.int64)
