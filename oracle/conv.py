"""TEST INFRASTRUCTURE -- Python front end of the fp64 CPU oracle.

Not part of the product: only the tests, the smoke check and the benchmark's
CPU-baseline leg may import this.  It shares no code with the CUDA library.

`Oracle(irreps_in, irreps_out, l_max, K)` builds the path table (tables.py) and calls
the materialised C routines (sobek_oracle.c: O1 radial projection, O2 message, O3
scatter, O4 first-order adjoints, O5 second order).  `reassociated_fwd` is the
receiver-state form (Eqs. angular_path_contraction, receiver_state, receiver_mixing)
written with numpy, used to check that the two orders of summation agree.
`sender_view` is the stable sender-sorted view of a receiver-sorted CSR graph.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

from . import tables

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libsobek_oracle.so")
_SRC = os.path.join(_HERE, "sobek_oracle.c")


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c99",
                               "-o", _SO, _SRC, "-lm"])
    return _SO


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(_load().oracle_threads())


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _d(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


class Oracle:
    def __init__(self, irreps_in, irreps_out, l_max: int, K: int, mode: str = "uvw"):
        self.irreps_in, self.irreps_out, self.l_max, self.K = list(irreps_in), list(irreps_out), l_max, K
        self.mode = mode   # "uvw" (Eq. uvw_connection) or "uvu" (Eq. uvu_connection)
        self.paths, self.N_w = tables.enumerate_paths(irreps_in, irreps_out, l_max, mode)
        self.C_x = sum(c * (2 * l + 1) for c, l, _ in irreps_in)
        self.C_y = sum(c * (2 * l + 1) for c, l, _ in irreps_out)
        self.dsh = (l_max + 1) ** 2
        rows, cg, off = [], [], 0
        for p in self.paths:
            di, ds, do = 2 * p.l_in + 1, 2 * p.l_sh + 1, 2 * p.l_out + 1
            rows.append([p.in_off, p.c_in, di, p.sh_off, ds, p.out_off, p.c_out, do, p.w_off, off,
                         1 if mode == "uvu" else 0])
            cg.append(p.cg.ravel())
            off += di * ds * do
        self._P = np.ascontiguousarray(np.array(rows, dtype=np.int64).reshape(-1, 11))
        self._cg = np.ascontiguousarray(np.concatenate(cg)) if cg else np.zeros(1)

    def col_std(self):
        return tables.weight_col_std(self.irreps_in, self.irreps_out, self.l_max, self.K, self.mode)

    # -- helpers ------------------------------------------------------------
    def _graph(self, row_ptr, col, act):
        rp = np.ascontiguousarray(np.asarray(row_ptr, dtype=np.int64))
        cl = np.ascontiguousarray(np.asarray(col, dtype=np.int32))
        N = rp.shape[0] - 1
        if act is None:
            act = np.arange(N, dtype=np.int64)
        act = np.ascontiguousarray(np.asarray(act, dtype=np.int64))
        return rp, cl, act, N, int(cl.shape[0])

    def _common(self, rp, cl, act):
        i64 = ctypes.c_int64
        return [i64(act.shape[0]), _p(act), _p(rp), _p(cl), i64(len(self.paths)), _p(self._P),
                _p(self._cg), i64(self.C_x), i64(self.C_y), i64(self.dsh), i64(self.K), i64(self.N_w)]

    # -- the three orders -----------------------------------------------------
    def fwd(self, row_ptr, col, x, Y, phi, R, act=None):
        rp, cl, act, N, E = self._graph(row_ptr, col, act)
        x, Y, phi, R = _d(x), _d(Y), _d(phi), _d(R)
        y = np.zeros((N, self.C_y))
        _load().oracle_fwd(*self._common(rp, cl, act), _p(x), _p(Y), _p(phi), _p(R), _p(y))
        return y

    def bwd(self, row_ptr, col, x, Y, phi, R, gy, act=None):
        rp, cl, act, N, E = self._graph(row_ptr, col, act)
        x, Y, phi, R, gy = _d(x), _d(Y), _d(phi), _d(R), _d(gy)
        gx = np.zeros((N, self.C_x)); gY = np.zeros((E, self.dsh)); gphi = np.zeros((E, self.K))
        gR = np.zeros((self.K, self.N_w))
        _load().oracle_bwd(*self._common(rp, cl, act), _p(x), _p(Y), _p(phi), _p(R), _p(gy),
                           _p(gx), _p(gY), _p(gphi), _p(gR))
        return gx, gY, gphi, gR

    def dbwd(self, row_ptr, col, x, Y, phi, R, gy, vx, vY, vphi, vR, act=None):
        rp, cl, act, N, E = self._graph(row_ptr, col, act)
        x, Y, phi, R, gy = _d(x), _d(Y), _d(phi), _d(R), _d(gy)
        vx, vY, vphi, vR = _d(vx), _d(vY), _d(vphi), _d(vR)
        ggy = np.zeros((N, self.C_y)); hx = np.zeros((N, self.C_x)); hY = np.zeros((E, self.dsh))
        hphi = np.zeros((E, self.K)); hR = np.zeros((self.K, self.N_w))
        _load().oracle_dbwd(*self._common(rp, cl, act), _p(x), _p(Y), _p(phi), _p(R), _p(gy),
                            _p(vx), _p(vY), _p(vphi), _p(vR),
                            _p(ggy), _p(hx), _p(hY), _p(hphi), _p(hR))
        return ggy, hx, hY, hphi, hR

    # -- receiver-state form, numpy -------------------------------------------
    def reassociated_fwd(self, row_ptr, col, x, Y, phi, R):
        """m = S A with S_{i,pi,q,u,mo} = sum_j phi_q C_{pi,u,mo}(x_j, Y_ij)."""
        rp = np.asarray(row_ptr, dtype=np.int64)
        cl = np.asarray(col, dtype=np.int64)
        x, Y, phi, R = _d(x), _d(Y), _d(phi), _d(R)
        N = rp.shape[0] - 1
        y = np.zeros((N, self.C_y))
        recv = np.repeat(np.arange(N), np.diff(rp))
        for p in self.paths:
            di, ds, do = 2 * p.l_in + 1, 2 * p.l_sh + 1, 2 * p.l_out + 1
            xs = x[cl][:, p.in_off:p.in_off + di * p.c_in].reshape(-1, di, p.c_in)
            Ys = Y[:, p.sh_off:p.sh_off + ds]
            C = np.einsum("abo,eau,eb->euo", p.cg, xs, Ys)            # angular contraction
            S = np.zeros((N, self.K, p.c_in, do))
            np.add.at(S, recv, phi[:, :, None, None] * C[:, None, :, :])  # receiver state
            if self.mode == "uvu":
                A = R[:, p.w_off:p.w_off + p.c_in]
                m = np.einsum("iquo,qu->iou", S, A)                     # tied channels: no mixing
            else:
                A = R[:, p.w_off:p.w_off + p.c_in * p.c_out].reshape(self.K, p.c_in, p.c_out)
                m = np.einsum("iquo,quw->iow", S, A)                    # channel mixing
            y[:, p.out_off:p.out_off + do * p.c_out] += m.reshape(N, -1)
        return y


def sender_view(row_ptr, col):
    """Stable sender-sorted view of a receiver-sorted CSR graph: src_ptr[N+1] (int64)
    and src_perm[E] (int32, positions in the receiver-sorted order), edges of one sender
    kept in increasing receiver-sorted position."""
    rp = np.asarray(row_ptr, dtype=np.int64)
    cl = np.asarray(col, dtype=np.int64)
    N = rp.shape[0] - 1
    cnt = np.zeros(N + 1, dtype=np.int64)
    for e in range(cl.shape[0]):
        cnt[cl[e] + 1] += 1
    src_ptr = np.cumsum(cnt)
    cur = src_ptr[:-1].copy()
    perm = np.zeros(cl.shape[0], dtype=np.int32)
    for e in range(cl.shape[0]):
        perm[cur[cl[e]]] = e
        cur[cl[e]] += 1
    return src_ptr, perm
