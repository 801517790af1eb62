"""Pins for the oracle's tables: path enumeration against the weight counts the paper
prints, the byte model against its memory table, and the real Clebsch-Gordan tensors
against sum rules, closed forms and an independent quadrature route."""
import math
import os

import numpy as np
import pytest

from oracle import tables
from workloads import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append(line.split())
    return out


@pytest.mark.parametrize("row", _rows("paper_weight_counts.txt"), ids=lambda r: f"{r[0]}-{r[1]}")
def test_weight_counts_match_paper(row):
    mode, prof, n_w = row[0], [int(t) for t in row[1].split("/")], int(row[2])
    ir = synth.profile_irreps(prof)
    paths, nw = tables.enumerate_paths(ir, ir, len(prof) - 1)
    if mode == "uvw":
        assert nw == n_w
        assert len(paths) == {1: 4, 2: 11, 3: 23}[len(prof) - 1]
    else:
        assert tables.n_weights_uvu(ir, ir, len(prof) - 1) == n_w


@pytest.mark.parametrize("row", _rows("paper_weight_memory.txt"), ids=lambda r: f"{r[0]}-{r[1]}")
def test_weight_memory_model(row):
    kind, prof, val = row[0], [int(t) for t in row[1].split("/")], float(row[2])
    ir = synth.profile_irreps(prof)
    _, nw = tables.enumerate_paths(ir, ir, len(prof) - 1)
    if kind == "gib_at_1e6":
        assert abs(4 * nw * 1.0e6 / 2**30 - val) < 0.06
    else:
        assert abs(32 * 2**30 / (4 * nw) - val) / val < 0.03


def test_benchmark_config_shapes():
    """N_w, path counts and feature widths of the five configurations."""
    want = {"cfg1": (5, 320, 32, 32), "cfg2": (11, 11264, 288, 288), "cfg3": (10, 163840, 512, 2048),
            "cfg4": (11, 45056, 576, 576), "cfg5": (42, 172032, 1600, 1600)}
    for name, (npaths, nw, cx, cy) in want.items():
        w = synth.config(name)
        paths, n = tables.enumerate_paths(w.irreps_in, w.irreps_out, w.l_max)
        assert (len(paths), n, synth.irreps_dim(w.irreps_in), synth.irreps_dim(w.irreps_out)) == \
            (npaths, nw, cx, cy)


TRIPLES = [(a, b, c) for a in range(5) for b in range(5) for c in range(abs(a - b), min(a + b, 4) + 1)]


@pytest.mark.parametrize("l1,l2,l3", TRIPLES)
def test_cg_sum_rules(l1, l2, l3):
    c = tables.path_cg(l1, l2, l3)
    # per output component the coupling is orthonormal: sum_{a,b} c[a,b,o] c[a,b,o'] = delta
    g = np.einsum("abo,abp->op", c, c)
    assert np.allclose(g, np.eye(2 * l3 + 1), atol=1e-12)
    assert abs((c * c).sum() - (2 * l3 + 1)) < 1e-12
    # first nonzero entry positive
    flat = c.ravel()
    assert flat[np.nonzero(np.abs(flat) > 1e-9)[0][0]] > 0
    # swapping the two inputs transposes the tensor up to one global sign
    w, wt = tables.real_w3j(l1, l2, l3), tables.real_w3j(l2, l1, l3).transpose(1, 0, 2)
    assert np.allclose(w, wt, atol=1e-12) or np.allclose(w, -wt, atol=1e-12)
    # cyclic symmetry of the 3j tensor
    wc = tables.real_w3j(l3, l1, l2).transpose(1, 2, 0)
    assert np.allclose(w, wc, atol=1e-12) or np.allclose(w, -wc, atol=1e-12)


def test_cg_closed_forms():
    for l in range(5):
        c = tables.path_cg(l, 0, l)[:, 0, :]
        assert np.allclose(c, np.eye(2 * l + 1), atol=1e-12)            # scalar SH: identity
        c = tables.path_cg(0, l, l)[0, :, :]
        assert np.allclose(c, np.eye(2 * l + 1), atol=1e-12)
        d = tables.path_cg(l, l, 0)[:, :, 0]
        assert np.allclose(d, np.eye(2 * l + 1) / math.sqrt(2 * l + 1), atol=1e-12)  # dot product
    # 1 x 1 -> 1 is the cross product / sqrt(2), in the (y, z, x) component order
    c = tables.path_cg(1, 1, 1) / math.sqrt(3)
    eps = np.zeros((3, 3, 3))
    for (i, j, k) in [(0, 1, 2), (1, 2, 0), (2, 0, 1)]:
        eps[i, j, k], eps[j, i, k] = 1, -1
    # our axis order is (y, z, x), a cyclic permutation of (x, y, z): eps keeps its form
    assert np.allclose(c, eps / math.sqrt(6), atol=1e-12) or np.allclose(c, -eps / math.sqrt(6), atol=1e-12)
    # 1 x 1 -> 2 is symmetric and traceless in its two inputs
    c = tables.path_cg(1, 1, 2)
    assert np.allclose(c, c.transpose(1, 0, 2), atol=1e-12)
    assert np.allclose(np.einsum("aao->o", c), 0, atol=1e-12)


def test_nonzero_counts():
    nnz = lambda a, b, c: int((np.abs(tables.path_cg(a, b, c)) > 1e-9).sum())
    assert nnz(0, 0, 0) == 1 and nnz(0, 1, 1) == 3 and nnz(1, 1, 2) == 11
    assert nnz(2, 2, 2) == 25 and nnz(4, 4, 4) == 97


def _lebedev_like(n_theta=24, n_phi=48):
    xs, ws = np.polynomial.legendre.leggauss(n_theta)
    ph = (np.arange(n_phi) + 0.5) * 2 * math.pi / n_phi
    z = np.repeat(xs, n_phi)
    s = np.sqrt(1 - z * z)
    p = np.tile(ph, n_theta)
    pts = np.stack([s * np.cos(p), s * np.sin(p), z], axis=1)
    w = np.repeat(ws, n_phi) * (2 * math.pi / n_phi) / (4 * math.pi)
    return pts, w


@pytest.mark.parametrize("l1,l2,l3", [t for t in TRIPLES if sum(t) % 2 == 0])
def test_cg_against_gaunt_quadrature(l1, l2, l3):
    """For even l1+l2+l3 the integral of three real spherical harmonics over the sphere
    is proportional to the real 3j tensor: an independent route that also ties the
    tensor's basis to the spherical harmonics the workloads feed in."""
    pts, w = _lebedev_like()
    Y = synth.real_sph_harm(4, pts)
    sl = lambda l: Y[:, l * l:(l + 1) ** 2]
    G = np.einsum("n,na,nb,nc->abc", w, sl(l1), sl(l2), sl(l3))
    w3 = tables.real_w3j(l1, l2, l3)
    k = (G * w3).sum()
    assert abs(k) > 1e-6
    assert np.allclose(G, k * w3, atol=1e-10)
