"""Pins for the oracle's lattice part (Sec. 3.2: Eq. 2-5), independent of the oracle itself:
brute-force search over both cosets, lattice invariants, the E8 second-moment constant,
hand-derived examples of the tie conventions, field round trips."""
import itertools
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _brute_force_e8(Y):
    """Smallest squared distance from Y (float64) to D8 u (D8 + 1/2) and all minimisers.
    The covering radius of E8 is 1, so every coordinate of the nearest point is within 1 of Y."""
    best, arg = np.inf, []
    for c in (0, 1):
        base = np.floor(Y - 0.5 * c)
        offs = np.array(list(itertools.product((-1, 0, 1, 2), repeat=8)), dtype=np.float64)
        z = base[None, :] + offs
        z = z[(z.sum(axis=1) % 2) == 0]
        p = z + 0.5 * c
        d = ((Y[None, :] - p) ** 2).sum(axis=1)
        m = d.min()
        if m < best - 1e-12:
            best, arg = m, [tuple(q) for q in p[np.abs(d - m) < 1e-12]]
        elif abs(m - best) <= 1e-12:
            arg += [tuple(q) for q in p[np.abs(d - m) < 1e-12]]
    return best, arg


def test_e8_matches_brute_force():
    rng = np.random.default_rng(11)
    n_unique = 0
    for i in range(60):
        scale = (0.3, 1.0, 3.0)[i % 3]
        Y = (rng.standard_normal(8) * scale).astype(np.float32)
        c, z = oracle.e8_nearest(Y)
        p = z.astype(np.float64) + 0.5 * c
        d = ((Y.astype(np.float64) - p) ** 2).sum()
        best, arg = _brute_force_e8(Y.astype(np.float64))
        assert abs(d - best) < 1e-6, (Y, p, d, best)
        if len(arg) == 1:
            n_unique += 1
            assert tuple(p) == arg[0]
    assert n_unique > 40


def test_e8_brute_force_on_grid_ties():
    # inputs on a quarter grid hit many coordinate and parity ties; distances must still be minimal
    rng = np.random.default_rng(5)
    for _ in range(25):
        Y = (rng.integers(-8, 9, size=8) / 4.0).astype(np.float32)
        c, z = oracle.e8_nearest(Y)
        p = z.astype(np.float64) + 0.5 * c
        d = ((Y.astype(np.float64) - p) ** 2).sum()
        best, _ = _brute_force_e8(Y.astype(np.float64))
        assert abs(d - best) < 1e-9


def test_lattice_invariants_and_second_moment():
    # rows are uniform on a box, long enough that every row has nearly the same RMS; the
    # quantiser input (W / mu) / s is then uniform on a (scaled) box spanning many cells
    rng = np.random.default_rng(3)
    R, C = 10, 40000
    n = R * C // 8
    W = rng.uniform(-6, 6, size=(R, C)).astype(np.float32)
    s = np.float32(0.25)
    fields, mus = oracle.quantise(W, float(s))
    assert np.allclose(mus, [oracle.row_rms(W[r]) for r in range(R)], rtol=0, atol=0)
    Yeff = ((W / mus[:, None]) / s).reshape(n, 8)
    q = np.stack([oracle.point2_from_fields(f) for f in fields[:4000]])
    # all-integer or all-half-integer coordinates, even coordinate sum of z
    par = q & 1
    assert np.all(par == par[:, :1])
    z = (q - par) // 2
    assert np.all(z.sum(axis=1) % 2 == 0)
    # second moment per dimension of the E8 Voronoi cell (unit volume): 929/12960; covering radius 1
    allq = np.empty((n, 8), np.int64)
    c = fields[:, 0].astype(np.int64)
    allq[:, :7] = 2 * fields[:, 1:8] + c[:, None]
    pi = fields[:, 1:8].sum(axis=1) % 2
    allq[:, 7] = 2 * (2 * fields[:, 8] + pi) + c
    err = ((Yeff.astype(np.float64) - 0.5 * allq) ** 2).sum(axis=1)
    assert err.max() <= 1.0 + 1e-6
    G = err.mean() / 8.0
    assert abs(G - 929.0 / 12960.0) < 0.012 * 929.0 / 12960.0, G


def test_hand_examples_of_tie_conventions():
    for line in open(os.path.join(GOLDEN, "e8_examples.txt")):
        if line.startswith("#") or not line.strip():
            continue
        ys, cs, zs = line.split("|")
        Y = np.array([float(t) for t in ys.split()], np.float32)
        c, z = oracle.e8_nearest(Y)
        assert c == int(cs), line
        assert list(z) == [int(t) for t in zs.split()], line


def test_field_examples_and_round_trip():
    for line in open(os.path.join(GOLDEN, "field_examples.txt")):
        if line.startswith("#") or not line.strip():
            continue
        cs, zs, ms = line.split("|")
        c, z, m = int(cs), np.array([int(t) for t in zs.split()], np.int32), int(ms)
        f = oracle.fields_from_point(c, z)
        assert f[0] == c and list(f[1:8]) == list(z[:7]) and f[8] == m, line
        assert list(oracle.point2_from_fields(f)) == list(2 * z + c)
    rng = np.random.default_rng(7)
    for _ in range(500):
        z = rng.integers(-40, 41, size=8).astype(np.int32)
        if z.sum() % 2:
            z[rng.integers(0, 8)] += 1
        c = int(rng.integers(0, 2))
        f = oracle.fields_from_point(c, z)
        assert list(oracle.point2_from_fields(f)) == list(2 * z + c)


def test_row_rms_closed_form_and_floor():
    x = np.full(64, 3.0, np.float32)
    assert oracle.row_rms(x) == np.float32(3.0)
    x = np.array([3.0, 4.0] * 4, np.float32)
    assert oracle.row_rms(x) == np.float32(np.sqrt(12.5))
    assert oracle.row_rms(np.zeros(16, np.float32)) == np.float32(1e-12)
