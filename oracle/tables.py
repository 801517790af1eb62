"""TEST INFRASTRUCTURE -- fp64 reference tables for the tensor-product convolution.

Nothing under `oracle/` is part of the product: only the tests, the smoke check and
the benchmark's CPU-baseline leg may import it, and it shares no code with the CUDA
library.

What is here
  * `enumerate_paths`  -- the valid (input irrep, SH order, output irrep) triples
    under the Clebsch-Gordan selection rules (Eq. cg_selection_rules), in nested
    order (input irrep, SH order, output irrep), each with n_pi = C_in*C_out
    weights (Section "Edge-conditioned tensor product convolution"; Eq. num_weights).
  * `real_w3j`         -- the rotation-invariant coupling tensor of three real
    irreps, from the Racah closed form of the complex Wigner 3j symbol and the
    unitary complex->real change of basis.
  * `path_cg`          -- c^pi = sqrt(2 l_out + 1) * real_w3j: the "sparse
    Clebsch-Gordan coefficient with the path normalisation" of
    Eq. angular_path_contraction.

Readings of points the paper leaves open:
  real basis m = -l..l with sine-type components at m < 0, Condon-Shortley phase
  cancelled (l = 1 is (y, z, x)); unit Frobenius norm for the 3j tensor; sign fixed
  so that the first nonzero entry in lexicographic (m_in, m_sh, m_out) order is
  positive; normalisation sqrt(2 l_out+1) (so that, per output component,
  sum_{m_in,m_sh} c^2 = 1) and no further per-path factor.
"""
from __future__ import annotations

import math
from fractions import Fraction
from functools import lru_cache

import numpy as np


def _f(n: int) -> int:
    return math.factorial(n)


def su2_cg(j1: int, m1: int, j2: int, m2: int, j3: int, m3: int) -> float:
    """<j1 m1 j2 m2 | j3 m3>, integer spins, Racah's formula in exact rationals."""
    if m1 + m2 != m3 or not (abs(j1 - j2) <= j3 <= j1 + j2):
        return 0.0
    if abs(m1) > j1 or abs(m2) > j2 or abs(m3) > j3:
        return 0.0
    pref = Fraction((2 * j3 + 1) * _f(j3 + j1 - j2) * _f(j3 - j1 + j2) * _f(j1 + j2 - j3),
                    _f(j1 + j2 + j3 + 1))
    pref *= _f(j3 + m3) * _f(j3 - m3) * _f(j1 - m1) * _f(j1 + m1) * _f(j2 - m2) * _f(j2 + m2)
    s = Fraction(0)
    for k in range(0, j1 + j2 - j3 + 1):
        d = [k, j1 + j2 - j3 - k, j1 - m1 - k, j2 + m2 - k, j3 - j2 + m1 + k, j3 - j1 - m2 + k]
        if min(d) < 0:
            continue
        den = 1
        for t in d:
            den *= _f(t)
        s += Fraction((-1) ** k, den)
    return math.sqrt(pref) * float(s)


def wigner_3j(j1, m1, j2, m2, j3, m3) -> float:
    if m1 + m2 + m3 != 0:
        return 0.0
    return (-1) ** (j1 - j2 - m3) / math.sqrt(2 * j3 + 1) * su2_cg(j1, m1, j2, m2, j3, -m3)


def complex_to_real(l: int) -> np.ndarray:
    """U with Y^real_a = sum_m U[a, m] Y_l^m (rows a = -l..l real, columns m complex).

    m > 0: sqrt(2) (-1)^m Re Y_l^m;  m < 0: sqrt(2) (-1)^m Im Y_l^|m|;  m = 0: Y_l^0,
    using Y_l^{-m} = (-1)^m conj(Y_l^m).
    """
    U = np.zeros((2 * l + 1, 2 * l + 1), dtype=np.complex128)
    U[l, l] = 1.0
    for m in range(1, l + 1):
        sg = (-1) ** m
        U[l + m, l + m] = sg / math.sqrt(2)
        U[l + m, l - m] = 1 / math.sqrt(2)
        U[l - m, l + m] = sg / (1j * math.sqrt(2))
        U[l - m, l - m] = -1 / (1j * math.sqrt(2))
    return U


@lru_cache(maxsize=None)
def _real_w3j_cached(l1: int, l2: int, l3: int):
    w = np.zeros((2 * l1 + 1, 2 * l2 + 1, 2 * l3 + 1))
    for m1 in range(-l1, l1 + 1):
        for m2 in range(-l2, l2 + 1):
            m3 = -m1 - m2
            if abs(m3) <= l3:
                w[l1 + m1, l2 + m2, l3 + m3] = wigner_3j(l1, m1, l2, m2, l3, m3)
    # invariant = sum 3j * Y^{m1} Y^{m2} Y^{m3}, and Y^m = sum_a conj(U[a, m]) Y^real_a
    U1, U2, U3 = (np.conj(complex_to_real(l)) for l in (l1, l2, l3))
    t = np.einsum("am,bn,co,mno->abc", U1, U2, U3, w.astype(np.complex128))
    re, im = np.abs(t.real).max(), np.abs(t.imag).max()
    r = t.real if re >= im else t.imag
    assert min(re, im) < 1e-12 * max(re, im, 1e-300), "3j tensor neither real nor imaginary"
    r = r / np.linalg.norm(r)
    flat = r.ravel()
    first = flat[np.nonzero(np.abs(flat) > 1e-9)[0][0]]
    if first < 0:
        r = -r
    r[np.abs(r) < 1e-14] = 0.0
    return r


def real_w3j(l1: int, l2: int, l3: int) -> np.ndarray:
    if not (abs(l1 - l2) <= l3 <= l1 + l2):
        raise ValueError("triangle rule violated")
    return _real_w3j_cached(l1, l2, l3).copy()


def path_cg(l_in: int, l_sh: int, l_out: int) -> np.ndarray:
    """c^pi[m_in, m_sh, m_out] of Eq. angular_path_contraction."""
    return math.sqrt(2 * l_out + 1) * real_w3j(l_in, l_sh, l_out)


class Path:
    __slots__ = ("i_in", "l_sh", "i_out", "l_in", "l_out", "c_in", "c_out", "in_off", "sh_off",
                 "out_off", "w_off", "cg")

    def __repr__(self):
        return (f"Path(in#{self.i_in} l={self.l_in} x sh l={self.l_sh} -> out#{self.i_out} "
                f"l={self.l_out}, {self.c_in}x{self.c_out} @ {self.w_off})")


def enumerate_paths(irreps_in, irreps_out, l_max: int, mode: str = "uvw"):
    """All (input irrep, SH order, output irrep) triples allowed by
    Eq. cg_selection_rules; SH irreps are one copy per order with parity (-1)^l.
    mode "uvw": C_in*C_out weights per path (Eq. uvw_connection); mode "uvu": the output
    multiplicity is tied to the input one, C_in weights per path (Eq. uvu_connection), and
    a path between blocks of different multiplicity is an error.  Returns (paths, N_w)."""
    if mode not in ("uvw", "uvu"):
        raise ValueError(mode)
    in_offs, o = [], 0
    for c, l, p in irreps_in:
        in_offs.append(o)
        o += c * (2 * l + 1)
    out_offs, o = [], 0
    for c, l, p in irreps_out:
        out_offs.append(o)
        o += c * (2 * l + 1)
    paths, w_off = [], 0
    for ii, (ci, li, pi) in enumerate(irreps_in):
        for ls in range(l_max + 1):
            ps = 1 if ls % 2 == 0 else -1
            for io, (co, lo, po) in enumerate(irreps_out):
                if abs(li - ls) <= lo <= li + ls and po == pi * ps:
                    p = Path()
                    p.i_in, p.l_sh, p.i_out = ii, ls, io
                    p.l_in, p.l_out, p.c_in, p.c_out = li, lo, ci, co
                    p.in_off, p.sh_off, p.out_off = in_offs[ii], ls * ls, out_offs[io]
                    p.w_off = w_off
                    p.cg = path_cg(li, ls, lo)
                    if mode == "uvu":
                        if ci != co:
                            raise ValueError("uvu needs equal input and output multiplicity on every path")
                        w_off += ci
                    else:
                        w_off += ci * co
                    paths.append(p)
    return paths, w_off


def n_weights_uvu(irreps_in, irreps_out, l_max: int) -> int:
    """Weight count of the channelwise mode (Eq. uvu_connection): C_in per path,
    paths restricted to equal input/output multiplicity blocks.  Used only to pin
    the path enumeration against the counts the paper prints for that mode."""
    return enumerate_paths(irreps_in, irreps_out, l_max, "uvu")[1]


def weight_col_std(irreps_in, irreps_out, l_max: int, K: int, mode: str = "uvw") -> np.ndarray:
    """Per-column standard deviation 1/sqrt(fan_in) for drawing R, with
    fan_in = K * (sum of input multiplicities over the paths into that output block); in the
    channelwise mode an output channel is fed by one channel per path: fan_in = K * (paths into the block)."""
    paths, n_w = enumerate_paths(irreps_in, irreps_out, l_max, mode)
    fan = {}
    for p in paths:
        fan[p.i_out] = fan.get(p.i_out, 0) + (1 if mode == "uvu" else p.c_in)
    std = np.zeros(n_w)
    for p in paths:
        n = p.c_in if mode == "uvu" else p.c_in * p.c_out
        std[p.w_off:p.w_off + n] = 1.0 / math.sqrt(K * fan[p.i_out])
    return std
