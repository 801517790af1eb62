"""Seeded synthetic inputs for the edge-conditioned tensor-product convolution.

This module produces *inputs only*: irreps descriptors, radius graphs in
receiver-sorted CSR form, spherical harmonics Y of the edge directions, radial
embeddings phi, and Gaussian features / weights / cotangents.  It holds none of
the operator's arithmetic (no Clebsch-Gordan tables, no contractions), so both
the fp64 oracle and the CUDA library may be fed from it.

Conventions (they are inputs to the operator, fixed here):
  * r_ij = r_j - r_i for the edge j -> i (Section "Edge-conditioned tensor
    product convolution"), Y_ij = real spherical harmonics of r_ij / |r_ij|.
  * real SH basis: components m = -l..l; m < 0 sine-type, m > 0 cosine-type,
    Condon-Shortley phase cancelled, so l = 1 reads sqrt(3)*(y, z, x);
    component normalisation sum_m Y_lm^2 = 2l+1.
  * features are in `ir_mul` layout: irrep blocks in descriptor order and, inside
    a block, index m*C + u (multiplicity contiguous).
"""
from __future__ import annotations

import math
import re
from dataclasses import dataclass, field

import numpy as np

# ----------------------------------------------------------------------------
# irreps descriptors
# ----------------------------------------------------------------------------

_IR = re.compile(r"^\s*(?:(\d+)\s*x\s*)?(\d+)\s*([eo])\s*$")


def parse_irreps(text: str):
    """'32x0e+32x1o' -> [(32, 0, +1), (32, 1, -1)] as (mul, l, parity)."""
    out = []
    for tok in text.split("+"):
        m = _IR.match(tok)
        if not m:
            raise ValueError(f"bad irrep token {tok!r}")
        mul = int(m.group(1)) if m.group(1) else 1
        out.append((mul, int(m.group(2)), 1 if m.group(3) == "e" else -1))
    return out


def irreps_dim(irreps) -> int:
    return sum(mul * (2 * l + 1) for mul, l, _ in irreps)


def profile_irreps(mults):
    """Paper profile '64/32/32' -> natural-parity irreps, ascending l."""
    return [(m, l, 1 if l % 2 == 0 else -1) for l, m in enumerate(mults)]


# ----------------------------------------------------------------------------
# spherical harmonics and radial embeddings (inputs)
# ----------------------------------------------------------------------------


def real_sph_harm(l_max: int, vec: np.ndarray) -> np.ndarray:
    """Component-normalised real SH of unit vectors, [n, (l_max+1)^2], fp64.

    Associated Legendre functions by the standard upward recurrences, without the
    Condon-Shortley sign; azimuth from atan2(y, x).
    """
    v = np.asarray(vec, dtype=np.float64)
    v = v / np.linalg.norm(v, axis=-1, keepdims=True)
    x, y, z = v[:, 0], v[:, 1], v[:, 2]
    phi = np.arctan2(y, x)
    s = np.sqrt(np.maximum(0.0, 1.0 - z * z))
    n = v.shape[0]
    out = np.empty((n, (l_max + 1) ** 2), dtype=np.float64)
    # P[m][l]
    P = {}
    for m in range(l_max + 1):
        pmm = np.ones(n)
        for k in range(1, m + 1):
            pmm = pmm * (2 * k - 1) * s
        P[(m, m)] = pmm
        if m + 1 <= l_max:
            P[(m + 1, m)] = z * (2 * m + 1) * pmm
        for l in range(m + 2, l_max + 1):
            P[(l, m)] = ((2 * l - 1) * z * P[(l - 1, m)] - (l + m - 1) * P[(l - 2, m)]) / (l - m)
    for l in range(l_max + 1):
        base = l * l + l
        for m in range(0, l + 1):
            # sqrt(4 pi) * N_lm with N_lm^2 = (2l+1)/(4 pi) (l-m)!/(l+m)!
            nlm = math.sqrt((2 * l + 1) * math.factorial(l - m) / math.factorial(l + m))
            if m == 0:
                out[:, base] = nlm * P[(l, 0)]
            else:
                out[:, base + m] = math.sqrt(2.0) * nlm * P[(l, m)] * np.cos(m * phi)
                out[:, base - m] = math.sqrt(2.0) * nlm * P[(l, m)] * np.sin(m * phi)
    return out


def gaussian_basis(r: np.ndarray, K: int, r_c: float) -> np.ndarray:
    mu = np.arange(K, dtype=np.float64) * r_c / max(K - 1, 1)
    sig = r_c / max(K - 1, 1)
    return np.exp(-((r[:, None] - mu[None, :]) ** 2) / (2 * sig * sig))


def bessel_basis(r: np.ndarray, K: int, r_c: float, p: int = 6) -> np.ndarray:
    q = np.arange(1, K + 1, dtype=np.float64)
    b = math.sqrt(2.0 / r_c) * np.sin(q[None, :] * math.pi * r[:, None] / r_c) / r[:, None]
    d = r / r_c
    env = (1.0 - (p + 1) * (p + 2) / 2.0 * d**p + p * (p + 2) * d ** (p + 1)
           - p * (p + 1) / 2.0 * d ** (p + 2))
    return b * env[:, None]


# ----------------------------------------------------------------------------
# radius graphs
# ----------------------------------------------------------------------------


def pair_cdf_unit_cube(t: float) -> float:
    """P(|a-b| < t) for a, b uniform in the unit cube, t <= 1."""
    return (4.0 / 3.0) * math.pi * t**3 - 1.5 * math.pi * t**4 + 1.6 * t**5 - t**6 / 6.0


def cutoff_for_edges(N: int, E_target: float, L: float) -> float:
    lo, hi = 0.0, 1.0
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if N * (N - 1) * pair_cdf_unit_cube(mid) < E_target:
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi) * L


def radius_graph(pos: np.ndarray, r_c: float):
    """Directed edges j -> i for every pair with 0 < |r_j - r_i| < r_c, both
    directions, sorted by (receiver i, sender j).  Returns row_ptr int64[N+1],
    col int32[E] (senders), recv int32[E]."""
    from scipy.spatial import cKDTree

    N = pos.shape[0]
    tree = cKDTree(pos)
    pairs = tree.query_pairs(r_c, output_type="ndarray")
    if pairs.size:
        d = np.linalg.norm(pos[pairs[:, 0]] - pos[pairs[:, 1]], axis=1)
        pairs = pairs[(d > 0) & (d < r_c)]
    recv = np.concatenate([pairs[:, 0], pairs[:, 1]]).astype(np.int64)
    send = np.concatenate([pairs[:, 1], pairs[:, 0]]).astype(np.int64)
    order = np.lexsort((send, recv))
    recv, send = recv[order], send[order]
    row_ptr = np.zeros(N + 1, dtype=np.int64)
    np.add.at(row_ptr, recv + 1, 1)
    row_ptr = np.cumsum(row_ptr)
    return row_ptr, send.astype(np.int32), recv.astype(np.int32)


# ----------------------------------------------------------------------------
# workloads
# ----------------------------------------------------------------------------


@dataclass
class Workload:
    name: str
    irreps_in: list
    irreps_out: list
    l_max: int
    K: int
    N: int
    L: float
    r_c: float
    basis: str  # "gaussian" | "bessel"
    orders: tuple = (0, 1, 2)
    seed: int = 0
    note: str = ""
    copies: int = 1  # the graph of N nodes repeated this many times (disjoint copies, one batch)
    mode: str = "uvw"  # multiplicity mode of the operator: "uvw" fully connected, "uvu" channelwise


def _cube(N, rho):
    return (N / rho) ** (1.0 / 3.0)


def config(name: str, **kw) -> Workload:
    """The five benchmark configurations (synthetic stand-ins for the paper's
    unpublished radius graphs: uniform positions in a non-periodic cube)."""
    P = parse_irreps
    if name == "cfg1":
        return Workload("cfg1", P("8x0e+8x1o"), P("8x0e+8x1o"), 2, 8, 64, 6.0, 3.0, "gaussian")
    if name == "cfg2":
        ir = P("32x0e+32x1o+32x2e")
        N = 5000
        L = _cube(N, 0.1)
        return Workload("cfg2", ir, ir, 2, 8, N, L, cutoff_for_edges(N, 30.0 * N, L), "bessel",
                        orders=(0, 1))
    if name == "cfg3":
        N = 20000
        L = _cube(N, 0.1)
        return Workload("cfg3", P("128x0e+128x1o"), P("128x0e+128x1o+128x2e+128x3o"), 3, 8, N, L,
                        cutoff_for_edges(N, 30.0 * N, L), "bessel")
    if name.startswith("cfg4t_"):
        # the edge-scaling sweep beyond 1e6 edges: the 1e6-edge graph of the sweep repeated B times (disjoint copies in
        # one batch; the node features are drawn for every copy), so that 1e7 ... 1e8 edges are generated in seconds
        base = config("cfg4", edges=1e6)
        B = int(name.split("_")[1])
        return Workload(name, base.irreps_in, base.irreps_out, 2, 16, base.N, base.L, base.r_c, "bessel", orders=(0, 1),
                        copies=B, note=f"{B} copies of cfg4_1e6")
    if name.startswith("cfg4"):
        E = float(kw.get("edges", name.split("_")[1] if "_" in name else 1e5))
        ir = P("64x0e+64x1o+64x2e")
        N = int(round(E / 32))
        L = _cube(N, 0.1)
        return Workload(f"cfg4_{E:.0e}".replace("+0", ""), ir, ir, 2, 16, N, L,
                        cutoff_for_edges(N, E, L), "bessel", orders=(0, 1))
    if name == "cfg5":
        ir = P("64x0e+64x1o+64x2e+64x3o+64x4e")
        N = 50000
        L = _cube(N, 0.1)
        return Workload("cfg5", ir, ir, 4, 16, N, L, cutoff_for_edges(N, 40.0 * N, L), "bessel")
    if name.startswith("uvu_"):
        # channelwise mode on the paper's fixed 128-node, degree-32 graph repeated B times (appendix "Native
        # Channelwise Throughput"): uvu_<mult>x<blocks>_<B>, e.g. uvu_128x3_511 = profile 128/128/128, K = 16
        _, prof, B = name.split("_")
        mult, nb = (int(v) for v in prof.split("x"))
        base = config(f"graphs_{int(B)}")
        ir = [(mult, l, 1 if l % 2 == 0 else -1) for l in range(nb)]
        return Workload(name, ir, ir, nb - 1, 16, base.N, base.L, base.r_c, "bessel", copies=base.copies, mode="uvu")
    if name.startswith("deg_") or name.startswith("graphs_"):
        # the paper's two scaling axes (section "Scaling axes"), on its 128/64/64 profile with K = 16:
        # longer neighbourhoods on 2,048 nodes, or one 128-node graph of mean degree 32 repeated B times
        ir = P("128x0e+64x1o+64x2e")
        v = int(name.split("_")[1])
        if name.startswith("deg_"):
            N, deg, copies = 2048, float(v), 1
        else:
            N, deg, copies = 128, 32.0, v
        L = _cube(N, 0.1)
        # cutoff from the realised positions (same seeded draw as make_inputs), so that the mean degree is exact
        pos = L * np.random.default_rng(np.random.SeedSequence(0).spawn(8)[0]).random((N, 3))
        iu = np.triu_indices(N, 1)
        dist = np.sort(np.linalg.norm(pos[iu[0]] - pos[iu[1]], axis=1))
        n_pairs = min(int(round(deg * N / 2)), dist.size - 1)
        r_c = 0.5 * (dist[n_pairs - 1] + dist[n_pairs])
        return Workload(name, ir, ir, 2, 16, N, L, float(r_c), "bessel", copies=copies)
    raise KeyError(name)


def scaled(w: Workload, N: int, name: str | None = None) -> Workload:
    """Same irreps, density and mean degree, fewer nodes (for parity tests)."""
    rho = w.N / w.L**3
    L = _cube(N, rho)
    deg = w.N * (w.N - 1) * pair_cdf_unit_cube(min(1.0, w.r_c / w.L)) / w.N
    return Workload(name or f"{w.name}_N{N}", w.irreps_in, w.irreps_out, w.l_max, w.K, N, L,
                    cutoff_for_edges(N, deg * N, L), w.basis, w.orders, w.seed, w.note)


@dataclass
class Inputs:
    w: Workload
    N: int
    E: int
    row_ptr: np.ndarray
    col: np.ndarray
    recv: np.ndarray
    x: np.ndarray
    Y: np.ndarray
    phi: np.ndarray
    R: np.ndarray
    gy: np.ndarray
    vx: np.ndarray
    vY: np.ndarray
    vphi: np.ndarray
    vR: np.ndarray
    pos: np.ndarray = field(default=None, repr=False)


def weight_col_std(paths, K: int, N_w: int, mode: str = "uvw") -> np.ndarray:
    """1/sqrt(fan_in) per column of R, the scale of the synthetic weights: fan_in = K * (sum of the input
    multiplicities over the paths into the column's output block; the number of those paths in the channelwise
    mode).  `paths` is a sequence of records with fields i_out, c_in, c_out, w_off (the path table of a plan)."""
    uvu = mode == "uvu"
    fan = {}
    for p in paths:
        fan[p.i_out] = fan.get(p.i_out, 0) + (1 if uvu else p.c_in)
    std = np.zeros(N_w)
    for p in paths:
        std[p.w_off:p.w_off + (p.c_in if uvu else p.c_in * p.c_out)] = (K * fan[p.i_out]) ** -0.5
    return std


def plan_col_std(plan) -> np.ndarray:
    """weight_col_std for a library plan (anything with .info, .path(k) and .mode)."""
    return weight_col_std([plan.path(k) for k in range(plan.info.n_paths)], plan.info.K, plan.info.N_w, plan.mode)


def make_inputs(w: Workload, col_std: np.ndarray, dtype=np.float32,
                with_cotangents: bool = True) -> Inputs:
    """Draw every input of one workload.

    `col_std[N_w]` is the standard deviation of each column of R (the caller derives
    it from its own path table as 1/sqrt(fan_in), fan_in = K * sum of the input
    multiplicities feeding that column's output block), so that this module needs
    no knowledge of the path structure.
    """
    col_std = np.asarray(col_std, dtype=np.float64)
    N_w = int(col_std.shape[0])
    ss = np.random.SeedSequence(w.seed)
    s_pos, s_x, s_R, s_gy, s_vx, s_vY, s_vphi, s_vR = [np.random.default_rng(s) for s in ss.spawn(8)]
    pos = w.L * s_pos.random((w.N, 3))
    row_ptr, col, recv = radius_graph(pos, w.r_c)
    # edge inputs of the base graph (computed once, then repeated with the graph)
    e1 = int(col.shape[0])
    rij = pos[col] - pos[recv]
    r = np.linalg.norm(rij, axis=1)
    dsh = (w.l_max + 1) ** 2
    Y = real_sph_harm(w.l_max, rij) if e1 else np.zeros((0, dsh))
    phi = gaussian_basis(r, w.K, w.r_c) if w.basis == "gaussian" else bessel_basis(r, w.K, w.r_c)
    if w.copies > 1:
        # disjoint copies of the same graph: node ids of copy b are shifted by b * N; the edge inputs repeat, the
        # node features below are drawn for every node of every copy
        n1, B = w.N, int(w.copies)
        shift = (np.arange(B, dtype=np.int64) * n1)[:, None]
        col = (col[None, :].astype(np.int64) + shift).reshape(-1).astype(np.int32)
        recv = (recv[None, :].astype(np.int64) + shift).reshape(-1).astype(np.int32)
        row_ptr = np.concatenate([[0], (row_ptr[None, 1:] + (np.arange(B, dtype=np.int64) * e1)[:, None]).reshape(-1)])
        pos = np.tile(pos, (B, 1))
        Y = np.tile(Y.astype(dtype), (B, 1))
        phi = np.tile(phi.astype(dtype), (B, 1))
    N_tot = w.N * max(1, int(w.copies))
    E = int(col.shape[0])
    C_x, C_y = irreps_dim(w.irreps_in), irreps_dim(w.irreps_out)
    # node-sized Gaussians: in the target precision directly once they are large (the fp64 draw of a graph with millions
    # of nodes would need tens of gigabytes of host memory)
    big = N_tot * max(C_x, C_y) > 50_000_000
    normal = (lambda g, shape: g.standard_normal(shape, dtype=np.float32)) if (big and dtype == np.float32) else \
             (lambda g, shape: g.standard_normal(shape))
    x = normal(s_x, (N_tot, C_x))
    R = s_R.standard_normal((w.K, N_w)) * col_std[None, :]
    vR = s_vR.standard_normal((w.K, N_w)) * col_std[None, :]
    gy = normal(s_gy, (N_tot, C_y))
    if with_cotangents:
        vx = normal(s_vx, (N_tot, C_x))
        vY = normal(s_vY, (E, dsh))
        vphi = normal(s_vphi, (E, w.K))
    else:
        vx = np.zeros((0, C_x)); vY = np.zeros((0, dsh)); vphi = np.zeros((0, w.K))
    c = lambda a: np.ascontiguousarray(a if a.dtype == dtype else a.astype(dtype))
    return Inputs(w, N_tot, E, row_ptr, col, recv, c(x), c(Y), c(phi), c(R), c(gy), c(vx), c(vY),
                  c(vphi), c(vR), pos)
