"""Seeded synthetic atomic systems (positions, species, cell, masses, velocities).

Metal units throughout: lengths in Angstrom, masses in amu, time in ps,
temperature in K.  Everything is drawn from ``numpy.random.Generator(PCG64(seed))``
so a given description always yields the same bytes.
"""

import math

import numpy as np

KB_EV_PER_K = 8.617333262e-5
# 1 eV / amu = 9648.533 (Angstrom / ps)^2
EV_PER_AMU_IN_A2_PS2 = 9648.53321

_FCC_BASIS = np.array([[0.0, 0.0, 0.0], [0.5, 0.5, 0.0], [0.5, 0.0, 0.5], [0.0, 0.5, 0.5]])
_BCC_BASIS = np.array([[0.0, 0.0, 0.0], [0.5, 0.5, 0.5]])
_DIAMOND_BASIS = np.concatenate([_FCC_BASIS, _FCC_BASIS + 0.25])


def _lattice(basis, cells, a):
    idx = np.arange(cells)
    gx, gy, gz = np.meshgrid(idx, idx, idx, indexing="ij")
    origins = np.stack([gx.ravel(), gy.ravel(), gz.ravel()], axis=1).astype(np.float64)
    pos = (origins[:, None, :] + basis[None, :, :]).reshape(-1, 3) * a
    return pos, np.eye(3) * (cells * a)


def rsa_points(n, box, dmin, rng, max_rounds=400):
    """Random sequential insertion of ``n`` points in a periodic cube of edge
    ``box`` with pairwise minimum-image distance >= ``dmin``.

    Candidates are thrown in batches.  A candidate is kept when no earlier-accepted
    point and no earlier candidate of its own batch lies within ``dmin``.  A grid of
    cells with diagonal <= dmin (one point per cell at most), padded with periodic
    copies of its faces, makes each check a handful of table look-ups.
    """
    ncell = int(math.ceil(box / (dmin / math.sqrt(3.0))))
    g = box / ncell
    reach = int(math.ceil(dmin / g))
    npad = ncell + 2 * reach
    offs = np.array([(dx * npad + dy) * npad + dz
                     for dx in range(-reach, reach + 1)
                     for dy in range(-reach, reach + 1)
                     for dz in range(-reach, reach + 1)], dtype=np.int64)
    grid = np.full((ncell, ncell, ncell), -1, dtype=np.int64)
    pts = np.empty((n, 3), dtype=np.float64)
    count = 0
    d2min = dmin * dmin

    def conflicts(p, cidp, table3d, other_pts, only_earlier):
        """True where a point stored in ``table3d`` lies within dmin of ``p``."""
        tab = np.pad(table3d, reach, mode="wrap").ravel()
        bad = np.zeros(len(p), dtype=bool)
        live = np.arange(len(p))
        base = cidp
        for off in offs:
            if live.size == 0:
                break
            k = tab[base + off]
            has = k >= 0
            if only_earlier:
                has &= k < live
            if not has.any():
                continue
            li = live[has]
            d = other_pts[k[has]] - p[li]
            d -= box * np.round(d / box)
            hit = (d * d).sum(axis=1) < d2min
            if hit.any():
                bad[li[hit]] = True
                sel = ~bad[live]
                live = live[sel]
                base = base[sel]
        return bad

    for _ in range(max_rounds):
        remaining = n - count
        if remaining == 0:
            break
        m = max(4096, 2 * remaining)
        cand = rng.random((m, 3)) * box
        c = np.minimum((cand / g).astype(np.int64), ncell - 1)
        cid = (c[:, 0] * ncell + c[:, 1]) * ncell + c[:, 2]
        keep = grid.ravel()[cid] < 0
        # first candidate per cell only
        _, first = np.unique(cid, return_index=True)
        mask = np.zeros(m, dtype=bool)
        mask[first] = True
        keep &= mask
        cand, c, cid = cand[keep], c[keep], cid[keep]
        cidp = ((c[:, 0] + reach) * npad + c[:, 1] + reach) * npad + c[:, 2] + reach
        bad = conflicts(cand, cidp, grid, pts, only_earlier=False)
        cand, cid, cidp = cand[~bad], cid[~bad], cidp[~bad]
        tmp = np.full(ncell ** 3, -1, dtype=np.int64)
        tmp[cid] = np.arange(len(cand))
        bad = conflicts(cand, cidp, tmp.reshape(ncell, ncell, ncell), cand, only_earlier=True)
        cand, cid = cand[~bad], cid[~bad]
        take = min(len(cand), remaining)
        pts[count:count + take] = cand[:take]
        grid.ravel()[cid[:take]] = np.arange(count, count + take)
        count += take
    if count < n:
        raise RuntimeError(f"random sequential insertion stalled at {count}/{n} points")
    return pts


def _random_rotations(n, rng):
    q = rng.standard_normal((n, 4))
    q /= np.linalg.norm(q, axis=1, keepdims=True)
    w, x, y, z = q[:, 0], q[:, 1], q[:, 2], q[:, 3]
    R = np.empty((n, 3, 3))
    R[:, 0, 0] = 1 - 2 * (y * y + z * z)
    R[:, 0, 1] = 2 * (x * y - z * w)
    R[:, 0, 2] = 2 * (x * z + y * w)
    R[:, 1, 0] = 2 * (x * y + z * w)
    R[:, 1, 1] = 1 - 2 * (x * x + z * z)
    R[:, 1, 2] = 2 * (y * z - x * w)
    R[:, 2, 0] = 2 * (x * z - y * w)
    R[:, 2, 1] = 2 * (y * z + x * w)
    R[:, 2, 2] = 1 - 2 * (x * x + y * y)
    return R


def maxwell_boltzmann(masses_per_atom, temperature, rng):
    """Velocities in Angstrom/ps: Gaussian per component, centre-of-mass momentum
    removed, then rescaled so the kinetic temperature over 3N-3 degrees of freedom
    equals ``temperature`` exactly."""
    n = len(masses_per_atom)
    sig = np.sqrt(KB_EV_PER_K * temperature * EV_PER_AMU_IN_A2_PS2 / masses_per_atom)
    v = rng.standard_normal((n, 3)) * sig[:, None]
    p = (masses_per_atom[:, None] * v).sum(axis=0)
    v -= p / masses_per_atom.sum()
    ke = 0.5 * (masses_per_atom[:, None] * v * v).sum() / EV_PER_AMU_IN_A2_PS2
    dof = max(3 * n - 3, 1)
    t_now = 2.0 * ke / (dof * KB_EV_PER_K)
    if t_now > 0:
        v *= math.sqrt(temperature / t_now)
    return v


def make_system(desc, md=None):
    """Build a system from a description dict (see ``workloads.configs``).

    Returns a dict with ``pos`` float64 [N,3], ``types`` int32 [N], ``cell`` float64
    [3,3] (rows are cell vectors), ``pbc`` int32 [3], ``masses`` float64 [T] and,
    when ``md`` is given, ``vel`` float64 [N,3].
    """
    kind = desc["kind"]
    rng = np.random.Generator(np.random.PCG64(desc["seed"]))
    pbc = np.array(desc.get("pbc", [1, 1, 1]), dtype=np.int32)
    n_types = desc["n_types"]
    if kind in ("fcc", "bcc", "diamond"):
        basis = {"fcc": _FCC_BASIS, "bcc": _BCC_BASIS, "diamond": _DIAMOND_BASIS}[kind]
        pos, cell = _lattice(basis, desc["cells"], desc["a"])
        if "type_index" in desc:         # one species out of a larger type table
            types = np.full(len(pos), desc["type_index"], dtype=np.int32)
        elif n_types > 1:
            types = rng.integers(0, n_types, size=len(pos)).astype(np.int32)
        else:
            types = np.zeros(len(pos), dtype=np.int32)
        pos = pos + rng.standard_normal(pos.shape) * desc["jitter"]
    elif kind == "water":
        nmol = desc["molecules"]
        amu_g = 1.66053906660e-24
        vol_a3 = nmol * (15.999 + 2 * 1.008) * amu_g / desc["density_g_cm3"] * 1e24
        box = vol_a3 ** (1.0 / 3.0)
        cell = np.eye(3) * box
        o = rsa_points(nmol, box, desc["min_oo"], rng)
        R = _random_rotations(nmol, rng)
        half = math.radians(104.5) / 2.0
        h_local = 0.96 * np.array([[math.sin(half), 0.0, math.cos(half)],
                                   [-math.sin(half), 0.0, math.cos(half)]])
        h = o[:, None, :] + np.einsum("nab,kb->nka", R, h_local)
        pos = np.concatenate([o[:, None, :], h], axis=1).reshape(-1, 3)
        types = np.tile(np.array([0, 1, 1], dtype=np.int32), nmol)
    elif kind == "poisson_disk":
        n = desc["atoms"]
        box = (n / desc["density"]) ** (1.0 / 3.0)
        cell = np.eye(3) * box
        pos = rsa_points(n, box, desc["min_dist"], rng)
        types = rng.integers(0, n_types, size=n).astype(np.int32)
    elif kind == "random_box":
        # small test cells: uniform points with a minimum distance; the cell may be
        # orthorhombic with unequal edges, points are thrown in the unit cube and scaled
        n = desc["atoms"]
        edges = np.array(desc["edges"], dtype=np.float64)
        cell = np.diag(edges)
        pos = np.empty((0, 3))
        while len(pos) < n:
            cand = rng.random(3) * edges
            if len(pos):
                d = pos - cand
                if any(pbc):
                    d -= edges * np.round(d / edges) * pbc
                if (np.sqrt((d * d).sum(axis=1)) < desc["min_dist"]).any():
                    continue
            pos = np.vstack([pos, cand])
        types = rng.integers(0, n_types, size=n).astype(np.int32)
        if "shift" in desc:  # push some atoms outside the cell to exercise wrapping
            pos = pos + rng.integers(-2, 3, size=pos.shape) * edges * pbc
    else:
        raise ValueError(f"unknown system kind {kind!r}")
    masses = np.array(desc["masses"], dtype=np.float64)
    out = dict(pos=np.ascontiguousarray(pos, dtype=np.float64), types=types,
               cell=np.ascontiguousarray(cell, dtype=np.float64), pbc=pbc, masses=masses)
    if md is not None:
        vrng = np.random.Generator(np.random.PCG64(md["seed"]))
        out["vel"] = maxwell_boltzmann(masses[types], md["temperature"], vrng)
    return out
