"""Pins for the CPU oracle: values the paper prints, closed forms, invariants and
brute force on tiny inputs.  None of these re-types an oracle formula; each one checks
the oracle against something fixed outside it."""

import itertools
import math
import os

import numpy as np
import pytest
import scipy.special
import torch
from scipy.spatial import cKDTree

from oracle import dpa4c as orc
from workloads import SMALL_PROFILES, make_blob, make_system

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_rows(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


TOL = {k: float(v) for k, v in _golden_rows("verification_tolerances.txt")}


def _rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def _rand_unitish(n, seed):
    return torch.from_numpy(_rng(seed).standard_normal((n, 3)))


# ---------------------------------------------------------------- printed tables

def test_widths_table():
    for row in _golden_rows("widths_table.txt"):
        C0, C1, C2, K1, K2 = map(int, row[:5])
        for k, L in enumerate((2, 3, 4)):
            w = orc.widths(C0, L)
            assert (w["C1"], w["C2"], w["K1"], w["K2"]) == (C1, C2, K1, K2)
            assert w["S"] == int(row[5 + k])
            assert w["D_out"] == int(row[8 + k])


def test_worked_examples():
    w = orc.widths(32, 2)
    assert (w["C1"], w["C2"], w["S"], w["D_out"]) == (8, 4, 76, 144)


def test_parameter_counts():
    # 118 elements plus the zero padding row of the type table
    for name, C0, L, R, F, n in _golden_rows("parameter_counts.txt"):
        assert orc.parameter_count(int(C0), int(L), int(R), 16, 3, int(F), 119) == int(n), name


def test_triples_for_L4():
    assert orc.triples(4) == [(1, 1, 2), (1, 2, 3), (1, 3, 4), (2, 2, 2), (2, 2, 4), (2, 3, 3),
                              (2, 4, 4), (3, 3, 4), (4, 4, 4)]
    assert orc.triples(2) == [(1, 1, 2), (2, 2, 2)]
    assert orc.triples(3) == [(1, 1, 2), (1, 2, 3), (2, 2, 2), (2, 3, 3)]


def test_bispectrum_counts():
    # Eq. "bispectrum-count"
    for C0 in (8, 32, 128):
        K = orc.probe_ranks(C0, 4)
        for tr in orc.triples(4):
            l1, l2, l3 = tr
            n = len(orc.retained_entries(tr, K))
            if l1 == l2 == l3:
                k = K[l1]
                assert n == k * (k + 1) * (k + 2) // 6
            elif l1 == l2:
                assert n == K[l1] * (K[l1] + 1) // 2 * K[l3]
            elif l2 == l3:
                assert n == K[l2] * (K[l2] + 1) // 2 * K[l1]
            else:
                assert n == K[l1] * K[l2] * K[l3]


# ---------------------------------------------------------------- envelope

def test_envelope_is_incomplete_beta():
    rc = 6.0
    rho = torch.linspace(0.0, 7.0, 1401, dtype=torch.float64)
    chi = orc.envelope(rho, rc).numpy()
    x = np.clip(rho.numpy() / rc, 0, 1)
    ref = 1.0 - scipy.special.betainc(5, 4, x)
    assert np.abs(chi - ref).max() < 1e-15 * 8
    assert chi[0] == 1.0 and (chi[rho.numpy() >= rc] == 0).all()


def test_envelope_derivative_closed_form():
    rc = 6.0
    rho = torch.linspace(0.05, 5.95, 300, dtype=torch.float64, requires_grad=True)
    (d,) = torch.autograd.grad(orc.envelope(rho, rc).sum(), rho)
    x = rho.detach() / rc
    ref = -280.0 * x ** 4 * (1 - x) ** 3 / rc
    assert (d - ref).abs().max() < 1e-14


def test_envelope_c3_at_cutoff():
    rc = 6.0
    h = 1e-3
    for k in (1, 2, 3):
        # one-sided k-th difference quotient just inside the cutoff vanishes like h^(4-k)
        pts = torch.tensor([rc - j * h for j in range(k + 1)], dtype=torch.float64)
        vals = orc.envelope(pts, rc).numpy()
        coef = [(-1) ** j * math.comb(k, j) for j in range(k + 1)]
        dq = sum(c * v for c, v in zip(coef, vals)) / h ** k
        assert abs(dq) < 50 * h ** (4 - k)


# ---------------------------------------------------------------- radial basis

def test_bessel_basis_values_and_limit():
    omega = torch.tensor([0.5, 1.0, 3.0], dtype=torch.float64)
    rho = torch.tensor([0.0, 1e-9, 0.7, 5.0], dtype=torch.float64)
    f = orc.bessel_basis(rho, omega).numpy()
    assert np.allclose(f[0], omega.numpy(), rtol=0, atol=0)
    assert np.allclose(f[1], omega.numpy(), rtol=1e-15)
    assert np.allclose(f[2], np.sin(omega.numpy() * 0.7) / 0.7, rtol=1e-15)
    assert np.allclose(f[3], np.sin(omega.numpy() * 5.0) / 5.0, rtol=1e-14, atol=1e-17)


def test_gaussian_basis_against_the_normal_density():
    # fixed width sigma_g = rc / (N_rbf - 1): f_n is the normal density of that width, centred on
    # c_n, rescaled to 1 at its maximum; half maximum at sigma_g sqrt(2 ln 2); the family has no
    # cutoff factor, so it does not vanish at rc
    import scipy.stats
    rc, centers = 6.0, torch.tensor([0.0, 1.3, 2.0, 4.4, 6.0], dtype=torch.float64)
    sg = rc / 4
    rho = torch.tensor([0.0, 0.9, 2.0, 2.0 + sg, 2.0 - sg * math.sqrt(2 * math.log(2)), 6.0], dtype=torch.float64)
    f = orc.gaussian_basis(rho, centers, rc).numpy()
    ref = scipy.stats.norm.pdf(rho.numpy()[:, None], loc=centers.numpy()[None, :], scale=sg) * sg * math.sqrt(2 * math.pi)
    assert np.allclose(f, ref, rtol=1e-14, atol=0)
    assert f[2, 2] == 1.0 and abs(f[3, 2] - math.exp(-0.5)) < 1e-15 and abs(f[4, 2] - 0.5) < 1e-15
    assert f[5, 3] > 0.5                                  # at rho = rc, centre 4.4: no cutoff factor
    # the radial map routes through the family named in the blob header
    p = SMALL_PROFILES["p16_2_0"]
    ob, og = orc.Oracle(make_blob(p, seed=3)), orc.Oracle(make_blob(p, seed=3, basis="gaussian"))
    assert ob.p["basis"] == "bessel" and og.p["basis"] == "gaussian"
    r = torch.tensor([0.3, 2.5, 5.9], dtype=torch.float64)
    g, _ = orc.radial_map(r, og.prm, "gaussian", p["rc"])
    h = orc.swiglu(torch.from_numpy(scipy.stats.norm.pdf(r.numpy()[:, None], loc=og.prm["omega"].numpy()[None, :],
                                                         scale=p["rc"] / (p["N_rbf"] - 1))
                                    * p["rc"] / (p["N_rbf"] - 1) * math.sqrt(2 * math.pi)), og.prm["W_in"])
    assert np.allclose(g.numpy(), (h @ og.prm["W_out"]).numpy(), rtol=1e-13, atol=1e-15)


# ---------------------------------------------------------------- harmonics

def test_addition_theorem_degrees_0_to_4():
    u, v = _rand_unitish(200, 1), _rand_unitish(200, 2)
    Bu, Bv = orc.harmonics(u, 4), orc.harmonics(v, 4)
    nu, nv = u.norm(dim=1), v.norm(dim=1)
    c = ((u * v).sum(1) / (nu * nv)).numpy()
    for l in range(5):
        lhs = (Bu[l] * Bv[l]).sum(1).numpy()
        rhs = (nu * nv).numpy() ** l * scipy.special.eval_legendre(l, c)
        scale = np.maximum(1.0, np.abs(rhs))
        assert (np.abs(lhs - rhs) / scale).max() < 10 * TOL["addition_theorem"]


def test_harmonics_parity_exact():
    u = _rand_unitish(100, 3)
    Bp, Bm = orc.harmonics(u, 4), orc.harmonics(-u, 4)
    for l in range(5):
        assert torch.equal(Bm[l], (-1) ** l * Bp[l])


def test_harmonic_blocks_are_harmonic_and_orthogonal():
    # Laplacian of each component vanishes (solid harmonics) and distinct components are
    # orthogonal over the sphere with equal norms 4 pi / (2l+1) (from the addition theorem)
    xs, ws = np.polynomial.legendre.leggauss(16)
    ph = (np.arange(32) + 0.5) * (2 * math.pi / 32)
    ct, phg = np.meshgrid(xs, ph, indexing="ij")
    st = np.sqrt(1 - ct * ct)
    u = torch.from_numpy(np.stack([st * np.cos(phg), st * np.sin(phg), ct], -1).reshape(-1, 3))
    w = torch.from_numpy((ws[:, None] * np.full((1, 32), 2 * math.pi / 32)).reshape(-1))
    B = orc.harmonics(u, 4)
    for l in range(5):
        gram = torch.einsum("p,pa,pb->ab", w, B[l], B[l])
        assert (gram - torch.eye(2 * l + 1, dtype=torch.float64) * 4 * math.pi / (2 * l + 1)).abs().max() < 1e-13
    for l1, l2 in itertools.combinations(range(5), 2):
        assert torch.einsum("p,pa,pb->ab", w, B[l1], B[l2]).abs().max() < 1e-13


# ---------------------------------------------------------------- STF map

def test_stf_quadrupolar_form():
    u = _rand_unitish(100, 4)
    Q = orc.stf(orc.harmonics(u, 2)[2])
    s = (u * u).sum(1)
    ref = math.sqrt(1.5) * (u[:, :, None] * u[:, None, :] - s[:, None, None] / 3 * torch.eye(3, dtype=torch.float64))
    assert (Q - ref).abs().max() < 10 * TOL["quadrupolar_form"]


def test_stf_isometry_symmetric_tracefree():
    z = torch.from_numpy(_rng(5).standard_normal((100, 5)))
    z2 = torch.from_numpy(_rng(6).standard_normal((100, 5)))
    Q, Q2 = orc.stf(z), orc.stf(z2)
    assert ((Q * Q2).sum((1, 2)) - (z * z2).sum(1)).abs().max() < 10 * TOL["stf_isometry"]
    assert (Q - Q.transpose(1, 2)).abs().max() == 0
    assert Q.diagonal(dim1=1, dim2=2).sum(1).abs().max() < 1e-15


# ---------------------------------------------------------------- Gaunt couplings

def test_gaunt_unit_norm_and_axis_symmetry():
    for tr in orc.triples(4):
        Cc = orc.gaunt_coupling(tr)
        assert abs(torch.linalg.norm(Cc).item() - 1) < 1e-14
        if tr[0] == tr[1]:
            assert (Cc - Cc.permute(1, 0, 2)).abs().max() < 1e-15
        if tr[1] == tr[2]:
            assert (Cc - Cc.permute(0, 2, 1)).abs().max() < 1e-15


def test_gaunt_rotation_invariant_trilinear_form():
    # the coupling is an invariant trilinear form: contracting three rotated harmonic
    # blocks gives the same number as contracting the originals
    rng = _rng(7)
    A = rng.standard_normal((3, 3))
    Rm, _ = np.linalg.qr(A)
    Rm = torch.from_numpy(Rm * np.sign(np.linalg.det(Rm)))
    pts = [_rand_unitish(20, 8 + k) for k in range(3)]
    for tr in orc.triples(4):
        Cc = orc.gaunt_coupling(tr)
        a = torch.einsum("abc,na,nb,nc->n", Cc, *[orc.harmonics(p, 4)[l] for p, l in zip(pts, tr)])
        b = torch.einsum("abc,na,nb,nc->n", Cc, *[orc.harmonics(p @ Rm.T, 4)[l] for p, l in zip(pts, tr)])
        assert (a - b).abs().max() < 1e-12 * max(1.0, a.abs().max().item())


def test_closed_forms_against_gaunt_contraction():
    rng = _rng(9)
    v1 = torch.from_numpy(rng.standard_normal((50, 3)))
    v2 = torch.from_numpy(rng.standard_normal((50, 3)))
    z = [torch.from_numpy(rng.standard_normal((50, 5))) for _ in range(3)]
    Q = [orc.stf(t) for t in z]
    j112 = torch.einsum("abc,na,nb,nc->n", orc.gaunt_coupling((1, 1, 2)), v1, v2, z[0])
    ref112 = -(1 / math.sqrt(5)) * torch.einsum("na,nab,nb->n", v1, Q[0], v2)
    assert (j112 - ref112).abs().max() < 10 * TOL["closed_forms_vs_gaunt"]
    j222 = torch.einsum("abc,na,nb,nc->n", orc.gaunt_coupling((2, 2, 2)), z[0], z[1], z[2])
    ref222 = -math.sqrt(12 / 35) * torch.einsum("nab,nbc,nca->n", Q[0], Q[1], Q[2])
    assert (j222 - ref222).abs().max() < 10 * TOL["closed_forms_vs_gaunt"]


# ---------------------------------------------------------------- neighbor search

def _python_neighbors(pos, cell, pbc, r_list):
    """Independent plain-loop search over atoms and images."""
    N = len(pos)
    rng_ = orc.image_range(cell, pbc, r_list)
    rows = []
    for i in range(N):
        ent = []
        for j in range(N):
            for nx in range(-rng_[0], rng_[0] + 1):
                for ny in range(-rng_[1], rng_[1] + 1):
                    for nz in range(-rng_[2], rng_[2] + 1):
                        if j == i and nx == 0 and ny == 0 and nz == 0:
                            continue
                        s = nx * cell[0] + ny * cell[1] + nz * cell[2]
                        d = (pos[j] + s) - pos[i]
                        if math.sqrt(float(d @ d)) < r_list:
                            ent.append((j, nx, ny, nz))
        rows.append(sorted(ent))
    return rows


@pytest.mark.parametrize("edges,n,r_list", [((4.0, 4.5, 5.0), 6, 6.0), ((9.0, 13.0, 12.5), 14, 6.0),
                                            ((3.1, 14.0, 7.3), 8, 7.0)])
def test_neighbor_rows_match_plain_loops(edges, n, r_list):
    s = make_system(dict(kind="random_box", atoms=n, edges=edges, min_dist=1.2, seed=11, n_types=1,
                         masses=[1.0], shift=True))
    pos = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    assert (pos >= 0).all() and (pos <= np.diag(s["cell"])).all()
    rows = orc.neighbor_rows(pos, s["cell"], s["pbc"], r_list)
    ref = _python_neighbors(pos, s["cell"], s["pbc"], r_list)
    for a, b in zip(rows, ref):
        assert [tuple(x) for x in a.tolist()] == b
    # list is symmetric: (i <- j, n) iff (j <- i, -n)
    have = {(i, *e) for i, r in enumerate(rows) for e in map(tuple, r.tolist())}
    assert all((j, i, -nx, -ny, -nz) in have for (i, j, nx, ny, nz) in have)


def test_neighbor_rows_match_kdtree_counts():
    s = make_system(dict(kind="random_box", atoms=300, edges=(14.0, 15.0, 16.0), min_dist=1.5, seed=12,
                         n_types=1, masses=[1.0]))
    pos = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    rows = orc.neighbor_rows(pos, s["cell"], s["pbc"], 6.0)
    tree = cKDTree(pos % np.diag(s["cell"]), boxsize=np.diag(s["cell"]))
    counts = np.array([len(x) - 1 for x in tree.query_ball_point(pos % np.diag(s["cell"]), 6.0 - 1e-12)])
    assert (np.array([len(r) for r in rows]) == counts).all()


@pytest.mark.parametrize("pbc", [(1, 1, 1), (1, 0, 1)])
def test_general_cell_rows_match_plain_loops_and_a_rotated_box_keeps_its_energy(pbc):
    # a sheared cell against plain loops over images, and a rigidly rotated orthorhombic box (its
    # cell matrix is then full) against the unrotated one: same edge multiset, same energies
    s = make_system(dict(kind="random_box", atoms=10, edges=(6.0, 7.5, 8.0), min_dist=1.4, seed=31, n_types=1,
                         masses=[1.0], shift=True, pbc=list(pbc)))
    e = np.diag(np.asarray(s["cell"], dtype=np.float64))
    cell = np.array([[e[0], 0.0, 0.0], [0.3 * e[1], e[1], 0.0], [-0.2 * e[2], 0.25 * e[2], e[2]]])
    pos = orc.wrap_positions((s["pos"] / e) @ cell, cell, pbc)
    frac = pos @ np.linalg.inv(cell)
    per = np.asarray(pbc, bool)
    assert (frac[:, per] > -1e-12).all() and (frac[:, per] < 1 + 1e-12).all()
    rows = orc.neighbor_rows(pos, cell, pbc, 6.0)
    ref = _python_neighbors(pos, cell, pbc, 6.0)
    for a, b in zip(rows, ref):
        assert [tuple(x) for x in a.tolist()] == b

    o, s2 = _small_case(n=16, edges=(6.5, 7.0, 8.2), seed=33, pbc=pbc)
    base = o.compute(s2["pos"], s2["types"], s2["cell"], pbc)
    Rm = _random_rotation(8)
    rot = o.compute(s2["pos"] @ Rm.T, s2["types"], np.asarray(s2["cell"]) @ Rm.T, pbc)
    assert rot["n_edges"] == base["n_edges"]
    assert np.allclose(rot["E_i"], base["E_i"], rtol=1e-11, atol=1e-13)
    assert np.allclose(rot["F"], base["F"] @ Rm.T, rtol=1e-9, atol=1e-12)
    assert np.allclose(rot["virial"], Rm @ base["virial"] @ Rm.T, rtol=1e-9, atol=1e-11)


def test_non_periodic_cluster_has_no_images():
    s = make_system(dict(kind="random_box", atoms=12, edges=(6.0, 6.0, 6.0), min_dist=1.5, seed=13,
                         n_types=1, masses=[1.0], pbc=[0, 0, 0]))
    rows = orc.neighbor_rows(s["pos"], s["cell"], s["pbc"], 6.0)
    assert all((r[:, 1:] == 0).all() for r in rows)


# ---------------------------------------------------------------- model-level pins

def _small_case(profile="p16_3_2", n=24, edges=(7.5, 8.0, 9.1), seed=21, pbc=(1, 1, 1), **kw):
    p = SMALL_PROFILES[profile]
    blob = make_blob(p, seed=seed, bias_scale=0.3, e_ref_scale=0.5, **kw)
    s = make_system(dict(kind="random_box", atoms=n, edges=edges, min_dist=1.6, seed=seed + 1,
                         n_types=p["T"], masses=[1.0] * p["T"], pbc=list(pbc)))
    return orc.Oracle(blob), s


def _raw_descriptors(o, pos, types, cell, pbc):
    out = o.compute(pos, types, cell, pbc, want_grad=False)
    return out["D_raw"], out["E_i"]


def _random_rotation(seed, proper=True):
    A = _rng(seed).standard_normal((3, 3))
    Rm, _ = np.linalg.qr(A)
    if (np.linalg.det(Rm) > 0) != proper:
        Rm[:, 0] *= -1
    return Rm


def test_invariance_rotation_translation_permutation():
    o, s = _small_case()
    D0, E0 = _raw_descriptors(o, s["pos"], s["types"], s["cell"], s["pbc"])
    scale = np.abs(D0).max()
    Rm = _random_rotation(31, proper=True)
    D1, E1 = _raw_descriptors(o, s["pos"] @ Rm.T, s["types"], s["cell"] @ Rm.T, s["pbc"])
    assert np.abs(D1 - D0).max() / scale < 20 * TOL["rotation"]
    t = np.array([0.37, -1.9, 11.3])
    D2, E2 = _raw_descriptors(o, s["pos"] + t, s["types"], s["cell"], s["pbc"])
    assert np.abs(D2 - D0).max() / scale < 20 * TOL["translation"]
    perm = _rng(32).permutation(len(s["pos"]))
    D3, E3 = _raw_descriptors(o, s["pos"][perm], s["types"][perm], s["cell"], s["pbc"])
    assert np.abs(D3 - D0[perm]).max() / scale < 20 * TOL["permutation"]
    for E in (E1, E2):
        assert np.abs(E - E0).max() < 1e-12 * max(1.0, np.abs(E0).max())
    assert np.abs(E3 - E0[perm]).max() < 1e-12 * max(1.0, np.abs(E0).max())


def test_invariance_improper_rotation_and_inversion_on_cluster():
    o, s = _small_case(n=12, edges=(6.0, 6.0, 6.0), pbc=(0, 0, 0))
    D0, E0 = _raw_descriptors(o, s["pos"], s["types"], s["cell"], s["pbc"])
    D1, _ = _raw_descriptors(o, -s["pos"], s["types"], s["cell"], s["pbc"])
    assert np.abs(D1 - D0).max() == TOL["inversion"]
    Rm = _random_rotation(33, proper=False)
    D2, _ = _raw_descriptors(o, s["pos"] @ Rm.T, s["types"], s["cell"], s["pbc"])
    assert np.abs(D2 - D0).max() / np.abs(D0).max() < 20 * TOL["rotation"]


def test_odd_triple_would_not_be_invariant():
    # guards the parity selection rule: the (1,1,1) contraction with the Levi-Civita
    # tensor changes sign under inversion, which is why T_L keeps even sums only
    assert all(sum(t) % 2 == 0 for t in orc.triples(4))


def test_single_aggregation_equals_per_degree_sums():
    o, s = _small_case()
    p, prm = o.p, o.prm
    pos = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    rows = orc.neighbor_rows(pos, s["cell"], s["pbc"], p["rc"])
    dst, src, rij = orc.rows_to_edges(rows, np.arange(len(pos)), pos, s["cell"])
    ty = torch.from_numpy(s["types"].astype(np.int64))
    dst_t, r = torch.from_numpy(dst), torch.from_numpy(rij)
    A, s0, s1 = orc.aggregate(p, prm, o.pair, len(pos), dst_t, ty[dst_t], ty[torch.from_numpy(src)], r)
    # per-centre, per-degree plain loops over that centre's neighbours
    rho = torch.sqrt((r * r).sum(1) + orc.EPS_REG ** 2)
    chi = orc.envelope(rho, p["rc"]).numpy()
    for i in (0, 5, 17):
        sel = dst == i
        assert abs(s0[i].item() - (chi[sel] ** 2).sum()) < 1e-14 * max(1, s0[i].item())
        assert abs(s1[i].item() - (chi[sel] ** 4).sum()) < 1e-14 * max(1, s1[i].item())
    # order independence: shuffling the edge list leaves the sums unchanged to rounding
    perm = torch.from_numpy(_rng(41).permutation(len(dst)))
    A2, s02, s12 = orc.aggregate(p, prm, o.pair, len(pos), dst_t[perm], ty[dst_t][perm],
                                 ty[torch.from_numpy(src)][perm], r[perm])
    for a, b in zip(A, A2):
        assert (a - b).abs().max() < 20 * TOL["single_aggregation"] * max(1.0, a.abs().max().item())


def test_zeroed_learned_maps_reduce_to_envelope_sums():
    # With W_out = 0 and W_p_out = 0: g = 0, gamma = 1, beta = X0_i + X0_j, U = 0, so
    # psi = beta and A_{0,c} = sum_j chi_j (X0_i + X0_j)_c: pure envelope sums that plain
    # numpy reproduces from distances alone.
    p = SMALL_PROFILES["p16_2_0"]
    blob = bytearray(make_blob(p, seed=50))
    _, prm = orc.parse_blob(bytes(blob))
    o = orc.Oracle(bytes(blob))
    o.prm["W_out"].zero_()
    o.prm["W_p_out"].zero_()
    with torch.no_grad():
        o.pair = orc.pair_modulation(o.p, o.prm)
    s = make_system(dict(kind="random_box", atoms=20, edges=(8.0, 8.5, 9.0), min_dist=1.6, seed=51,
                         n_types=p["T"], masses=[1.0] * p["T"]))
    out = o.compute(s["pos"], s["types"], s["cell"], s["pbc"], want_grad=False)
    X0 = o.prm["X0"].numpy()
    pos = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    C0, C1 = p["C0"], p["C1"]
    for i in (0, 7, 19):
        sel = out["dst"] == i
        d = np.sqrt((out["rij"][sel] ** 2).sum(1))       # eps changes d by 1e-15
        x = d / p["rc"]
        chi = 1.0 - scipy.special.betainc(5, 4, np.clip(x, 0, 1))
        beta = X0[s["types"][i]][None, :] + X0[s["types"][out["src"][sel]]]
        M0 = math.sqrt(0.25 + (chi ** 2).sum())
        M1 = math.sqrt(0.25 + (chi ** 4).sum())
        A0 = (chi[:, None] * beta).sum(0)
        Dr = out["D_raw"][i]
        assert np.allclose(Dr[:C0], X0[s["types"][i]], rtol=0, atol=0)
        assert np.allclose(Dr[C0:2 * C0], A0 / M0, rtol=1e-12, atol=1e-14)
        assert abs(Dr[2 * C0] - M0) < 1e-13 and abs(Dr[2 * C0 + 1] - M1) < 1e-13
        # degree one: X_1[m, c] = sum chi^2 beta_c u_m / M1 ; G_1 = X~^T X~ with W_1 as drawn
        u = out["rij"][sel] / d[:, None]
        X1 = np.einsum("e,ec,em->mc", chi ** 2, beta[:, :C1], u) / M1
        Xt = X1 @ (np.eye(C1) + o.prm["W_1"].numpy())
        G = Xt.T @ Xt
        vech = [G[a, b] * (1 if a == b else math.sqrt(2)) for a in range(C1) for b in range(a, C1)]
        got = Dr[2 * C0 + 2:2 * C0 + 2 + len(vech)]
        assert np.allclose(got, vech, rtol=1e-10, atol=1e-13)
        # the half-vectorisation preserves the Frobenius norm
        assert abs(np.linalg.norm(got) - np.linalg.norm(G)) < 1e-12


def test_retained_bispectrum_preserves_tensor_norm():
    rng = _rng(60)
    K = orc.probe_ranks(128, 3)
    Z = {l: torch.from_numpy(rng.standard_normal((2 * l + 1, K[l]))) for l in (1, 2, 3)}
    for tr in orc.triples(3):
        J = torch.einsum("abc,ai,bj,ck->ijk", orc.gaunt_coupling(tr), Z[tr[0]], Z[tr[1]], Z[tr[2]])
        kept = torch.stack([J[i, j, k] * w for ((i, j, k), w) in orc.retained_entries(tr, K)])
        assert abs(kept.norm().item() - J.norm().item()) < 1e-13


def test_mlp_residual_layers_with_zero_weights_are_identity():
    p = dict(SMALL_PROFILES["p16_2_0"])
    blob = make_blob(p, seed=70, bias_scale=0.2, e_ref_scale=0.4)
    o, _ = orc.Oracle(blob), None
    D = torch.from_numpy(_rng(71).standard_normal((5, p["D_out"])))
    ty = torch.tensor([0, 1, 2, 1, 0])
    E_full = orc.mlp_energy(o.p, o.prm, D, ty)
    o.prm["Theta_2"].zero_()
    o.prm["b_2"].zero_()
    E_res = orc.mlp_energy(o.p, o.prm, D, ty)
    p1 = dict(o.p, n_hidden=1)
    E_one = orc.mlp_energy(p1, o.prm, D, ty)
    assert (E_res - E_one).abs().max() == 0 and (E_full - E_one).abs().max() > 1e-6
    # dead first layer: only head bias and reference energy remain
    o.prm["Theta_1"].zero_()
    o.prm["b_1"].zero_()
    E0 = orc.mlp_energy(o.p, o.prm, D, ty)
    assert (E0 - (o.prm["b_head"][0] + o.prm["E_ref"][ty])).abs().max() == 0


def test_first_layer_residual_only_when_widths_agree():
    p = SMALL_PROFILES["p32_2_0_res"]
    o = orc.Oracle(make_blob(p, seed=72))
    D = torch.from_numpy(_rng(73).standard_normal((3, p["D_out"])))
    ty = torch.zeros(3, dtype=torch.int64)
    o.prm["Theta_1"].zero_()
    o.prm["Theta_2"].zero_()
    E = orc.mlp_energy(o.p, o.prm, D, ty)
    assert (E - (D @ o.prm["w_head"] + o.prm["b_head"][0])).abs().max() < 1e-14


def test_pair_modulation_ranges_and_order():
    p = SMALL_PROFILES["p32_3_2"]
    o = orc.Oracle(make_blob(p, seed=74))
    gamma, beta, U = o.pair
    assert ((gamma > 0) & (gamma < 2)).all() and (U.abs() < 1).all()
    X0 = o.prm["X0"]
    assert ((beta - X0[:, None, :] - X0[None, :, :]).abs() < 1).all()
    assert (gamma[0, 1] - gamma[1, 0]).abs().max() > 1e-6          # ordered pairs differ
    assert U.shape == (p["T"], p["T"], p["C0"], p["R"])


def test_swiglu_gate_is_the_first_half_of_the_columns():
    # Eq. "swiglu": [x_g, x_v] = x W, output SiLU(x_g) * x_v with the gate in the FIRST H columns.
    # One input row, H = 2, every product written out by hand; swapping the halves would give
    # SiLU(x_v) * x_g = (-0.5249791874789399 * ..., ...) instead.
    x = torch.tensor([[0.5, -1.0, 2.0]], dtype=torch.float64)
    W = torch.tensor([[1.0, -2.0, 0.5, 3.0],
                      [0.0, 1.0, -1.0, 2.0],
                      [0.25, 0.5, 1.5, -0.5]], dtype=torch.float64)
    a_gate = np.array([0.5 * 1.0 + (-1.0) * 0.0 + 2.0 * 0.25, 0.5 * (-2.0) + (-1.0) * 1.0 + 2.0 * 0.5])   # 1.0, -1.0
    a_val = np.array([0.5 * 0.5 + (-1.0) * (-1.0) + 2.0 * 1.5, 0.5 * 3.0 + (-1.0) * 2.0 + 2.0 * (-0.5)])  # 4.25, -1.5
    expected = a_gate * scipy.special.expit(a_gate) * a_val
    got = orc.swiglu(x, W).numpy()[0]
    assert np.allclose(got, expected, rtol=1e-15, atol=0)
    # the same numbers as decimals: SiLU(1) = 0.7310585786300049, SiLU(-1) = -0.2689414213699951
    assert np.allclose(got, [0.7310585786300049 * 4.25, -0.2689414213699951 * -1.5], rtol=1e-14, atol=0)
    swapped = a_val * scipy.special.expit(a_val) * a_gate
    assert np.abs(got - swapped).max() > 0.5


def test_pair_modulation_against_a_hand_built_network():
    # Eq. "pairfilm" with C0 = 2, R = 1, T = 2 and weights chosen so that two hidden units carry
    # everything: h0 = SiLU(X0_a[0]) X0_b[0] (gate reads the centre, value the neighbour) and
    # h1 = SiLU(X0_b[1]) X0_a[1].  Then [s | t | w] = 0.1 (h0 row0 + h1 row1), gamma = 1 + tanh s,
    # beta = X0_a + X0_b + tanh t, U = tanh w.  A missing 0.1, a different block order or the
    # neighbour-first concatenation each change these numbers.
    C0, R, T = 2, 1, 2
    Hp = 8 * math.ceil(2 * C0 / 3)
    X0 = np.array([[0.8, -0.3], [-1.2, 0.6]])
    W_in = np.zeros((2 * C0, 2 * Hp))
    W_in[0, 0] = 1.0            # gate 0 <- centre feature 0 (z = [X0_a, X0_b])
    W_in[2, Hp + 0] = 1.0       # value 0 <- neighbour feature 0
    W_in[3, 1] = 1.0            # gate 1 <- neighbour feature 1
    W_in[1, Hp + 1] = 1.0       # value 1 <- centre feature 1
    row0 = np.array([1.0, -2.0, 3.0, 0.5, -1.5, 2.5])
    row1 = np.array([0.7, 1.1, -0.9, 2.0, 0.3, -0.6])
    W_out = np.zeros((Hp, C0 * (2 + R)))
    W_out[0], W_out[1] = row0, row1
    prm = dict(X0=torch.from_numpy(X0), W_p_in=torch.from_numpy(W_in), W_p_out=torch.from_numpy(W_out))
    gamma, beta, U = orc.pair_modulation(dict(T=T, C0=C0, R=R), prm)
    assert U.shape == (T, T, C0, R)

    def silu_(v):
        return v * scipy.special.expit(v)

    for a in range(T):
        for b in range(T):
            h0 = silu_(X0[a, 0]) * X0[b, 0]
            h1 = silu_(X0[b, 1]) * X0[a, 1]
            o = 0.1 * (h0 * row0 + h1 * row1)
            assert np.allclose(gamma[a, b].numpy(), 1.0 + np.tanh(o[0:2]), rtol=1e-14, atol=0)
            assert np.allclose(beta[a, b].numpy(), X0[a] + X0[b] + np.tanh(o[2:4]), rtol=1e-14, atol=0)
            assert np.allclose(U[a, b, :, 0].numpy(), np.tanh(o[4:6]), rtol=1e-13, atol=0)
    # one entry as plain decimals, centre species 0, neighbour species 1:
    # h0 = SiLU(0.8)(-1.2) = -0.662381, h1 = SiLU(0.6)(-0.3) = -0.116218, s_0 = 0.1 (h0 + 0.7 h1) = -0.0743734
    h0, h1 = -1.2 * 0.8 / (1 + math.exp(-0.8)), -0.3 * 0.6 / (1 + math.exp(-0.6))
    assert abs(gamma[0, 1, 0].item() - (1 + math.tanh(0.1 * (h0 * 1.0 + h1 * 0.7)))) < 1e-15
    assert abs(gamma[0, 1, 0].item() - 0.925764) < 1e-6
    # ordered pairs: (0, 1) and (1, 0) differ
    assert abs(gamma[0, 1, 0].item() - gamma[1, 0, 0].item()) > 1e-3


def _beta_only_oracle(profile, seed):
    """Oracle of a small profile with the learned radial map and the pair network's output layer
    zeroed (psi = beta = X0_i + X0_j), no alignment (W_l = 0) and probes that select the leading
    channels (A_l = leading columns of the identity)."""
    p = SMALL_PROFILES[profile]
    o = orc.Oracle(make_blob(p, seed=seed))
    for k in ("W_out", "W_mode", "W_p_out", "W_1", "W_2", "A_1", "A_2"):
        o.prm[k].zero_()
    for l in (1, 2):
        A = o.prm[f"A_{l}"]
        for k in range(A.shape[1]):
            A[k, k] = 1.0
    with torch.no_grad():
        o.pair = orc.pair_modulation(o.p, o.prm)
    return p, o


@pytest.mark.parametrize("profile", ["p32_3_2", "p32_4_2"])
def test_higher_degree_gram_blocks_follow_the_addition_theorem(profile):
    # With psi = beta the degree-l moments are X_l[m, c] = sum_j chi_j^2 beta_jc B_lm(u_j) / M_1 for
    # the LEADING C_l channels, and the addition theorem turns the Gram block into
    #   G_l[c, c'] = sum_jk chi_j^2 chi_k^2 beta_jc beta_kc' P_l(u_j . u_k) / M_1^2,
    # which needs only distances, directions and scipy's Legendre polynomials.  Pins the weight
    # chi^2 for every l >= 1, the shared normaliser M_1, the leading-channel rule (C_2 < C_1 here)
    # and the positions of vech(G_2), vech(G_3) in the feature vector.
    p, o = _beta_only_oracle(profile, 52)
    s = make_system(dict(kind="random_box", atoms=18, edges=(8.0, 8.5, 9.0), min_dist=1.6, seed=53,
                         n_types=p["T"], masses=[1.0] * p["T"]))
    out = o.compute(s["pos"], s["types"], s["cell"], s["pbc"], want_grad=False)
    X0 = o.prm["X0"].numpy()
    C0, Cs = p["C0"], {1: p["C1"], 2: p["C2"], 3: 1, 4: 1}
    assert Cs[2] < Cs[1]
    for i in (0, 6, 17):
        sel = out["dst"] == i
        d = np.sqrt((out["rij"][sel] ** 2).sum(1))
        chi = 1.0 - scipy.special.betainc(5, 4, np.clip(d / p["rc"], 0, 1))
        beta = X0[s["types"][i]][None, :] + X0[s["types"][out["src"][sel]]]
        M1sq = 0.25 + (chi ** 4).sum()
        u = out["rij"][sel] / d[:, None]
        cosjk = np.clip(u @ u.T, -1.0, 1.0)
        off = 2 * C0 + 2
        for l in range(1, p["L"] + 1):
            C = Cs[l]
            wb = (chi ** 2)[:, None] * beta[:, :C]                        # [edges, C_l]
            G = wb.T @ scipy.special.eval_legendre(l, cosjk) @ wb / M1sq
            vech = np.array([G[a, b] * (1 if a == b else math.sqrt(2)) for a in range(C) for b in range(a, C)])
            got = out["D_raw"][i][off:off + len(vech)]
            assert np.allclose(got, vech, rtol=1e-9, atol=1e-12 * np.abs(vech).max()), (i, l)
            off += len(vech)


def test_bispectrum_and_quartic_blocks_from_cartesian_tensors():
    # Same setting: the probes are v_k = sum_j chi_j^2 beta_jk u_j / M_1 and, by Eq. "stf",
    # Q_h = sum_j chi_j^2 beta_jh sqrt(3/2) (u_j u_j^T - I/3) / M_1, built here from directions
    # alone.  Eq. "closed-forms" then gives the (1,1,2) and (2,2,2) blocks and Eq. "quartic"
    # Pi[h, k] = |Q_h v_k|^2; the feature vector holds J(1,1,2) right after the Gram blocks,
    # J(2,2,2) after it (L = 2) and Pi, h-major, in its last K_1 K_2 entries.
    p, o = _beta_only_oracle("p32_2_4", 54)
    s = make_system(dict(kind="random_box", atoms=16, edges=(8.0, 8.5, 9.0), min_dist=1.6, seed=55,
                         n_types=p["T"], masses=[1.0] * p["T"]))
    out = o.compute(s["pos"], s["types"], s["cell"], s["pbc"], want_grad=False)
    X0 = o.prm["X0"].numpy()
    C0, C1, C2, K1, K2, D = p["C0"], p["C1"], p["C2"], p["K1"], p["K2"], p["D_out"]
    for i in (1, 9, 15):
        sel = out["dst"] == i
        d = np.sqrt((out["rij"][sel] ** 2).sum(1))
        chi = 1.0 - scipy.special.betainc(5, 4, np.clip(d / p["rc"], 0, 1))
        beta = X0[s["types"][i]][None, :] + X0[s["types"][out["src"][sel]]]
        M1 = math.sqrt(0.25 + (chi ** 4).sum())
        u = out["rij"][sel] / d[:, None]
        w = chi ** 2
        v = np.einsum("e,ek,ea->ka", w, beta[:, :K1], u) / M1                          # [K1, 3]
        quad = math.sqrt(1.5) * (u[:, :, None] * u[:, None, :] - np.eye(3)[None] / 3.0)
        Q = np.einsum("e,eh,eab->hab", w, beta[:, :K2], quad) / M1                    # [K2, 3, 3]
        Dr = out["D_raw"][i]
        Pi = np.array([[np.sum((Q[h] @ v[k]) ** 2) for k in range(K1)] for h in range(K2)])
        assert np.allclose(Dr[D - K1 * K2:], Pi.reshape(-1), rtol=1e-9, atol=1e-13 * np.abs(Pi).max())
        off = 2 * C0 + 2 + C1 * (C1 + 1) // 2 + C2 * (C2 + 1) // 2
        j112 = [-(1 / math.sqrt(5)) * (v[a] @ Q[h] @ v[b]) * (1.0 if a == b else math.sqrt(2))
                for a in range(K1) for b in range(a, K1) for h in range(K2)]
        assert np.allclose(Dr[off:off + len(j112)], j112, rtol=1e-9, atol=1e-13 * np.abs(j112).max())
        off += len(j112)
        j222 = []
        for a in range(K2):
            for b in range(a, K2):
                for c in range(b, K2):
                    fam = len(set(itertools.permutations((a, b, c))))
                    j222.append(-math.sqrt(12 / 35) * np.trace(Q[a] @ Q[b] @ Q[c]) * math.sqrt(fam))
        assert np.allclose(Dr[off:off + len(j222)], j222, rtol=1e-9, atol=1e-13 * np.abs(j222).max())
        assert off + len(j222) == D - K1 * K2


# ---------------------------------------------------------------- forces and virial

def _energy(o, pos, s, cell=None):
    return o.compute(pos, s["types"], s["cell"] if cell is None else cell, s["pbc"], want_grad=False)["E"]


@pytest.mark.parametrize("profile", ["p16_3_2", "p32_2_4", "p8_4_0"])
def test_forces_sum_to_zero_and_match_finite_differences(profile):
    o, s = _small_case(profile=profile, n=16, edges=(7.0, 7.7, 8.1), seed=80)
    out = o.compute(s["pos"], s["types"], s["cell"], s["pbc"])
    F = out["F"]
    assert np.abs(F.sum(0)).max() < 1e-12 * max(1.0, np.abs(F).max())
    h = 1e-4
    fscale = np.abs(F).max()
    for (k, a) in [(0, 0), (3, 1), (7, 2), (15, 0), (9, 1)]:
        pp, pm = s["pos"].copy(), s["pos"].copy()
        pp[k, a] += h
        pm[k, a] -= h
        fd = -(_energy(o, pp, s) - _energy(o, pm, s)) / (2 * h)
        assert abs(fd - F[k, a]) < 1e-6 * fscale, (k, a, fd, F[k, a])


def test_virial_is_strain_derivative_and_symmetric():
    o, s = _small_case(profile="p16_3_2", n=16, edges=(7.0, 7.7, 8.1), seed=81)
    out = o.compute(s["pos"], s["types"], s["cell"], s["pbc"])
    Xi = out["virial"]
    assert np.abs(Xi - Xi.T).max() < 1e-11 * max(1.0, np.abs(Xi).max())
    h = 1e-5
    for a in range(3):
        for b in range(3):
            eps = np.zeros((3, 3))
            eps[a, b] = h
            Ep = _energy(o, s["pos"] @ (np.eye(3) + eps).T, s, s["cell"] @ (np.eye(3) + eps).T)
            Em = _energy(o, s["pos"] @ (np.eye(3) - eps).T, s, s["cell"] @ (np.eye(3) - eps).T)
            dE = (Ep - Em) / (2 * h)
            assert abs(dE + Xi[a, b]) < 1e-6 * max(1.0, np.abs(Xi).max()), (a, b, dE, Xi[a, b])


def test_skin_shell_edges_contribute_nothing():
    o, s = _small_case(n=16, edges=(7.0, 7.7, 8.1), seed=82)
    pos = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    cs = np.arange(len(pos))
    r0 = orc.neighbor_rows(pos, s["cell"], s["pbc"], o.p["rc"])
    r1 = orc.neighbor_rows(pos, s["cell"], s["pbc"], o.p["rc"] + 1.0)
    assert sum(map(len, r1)) > sum(map(len, r0))
    E0 = o.evaluate_rows(pos, s["types"], s["cell"], r0, cs, want_grad=False)[0]
    E1 = o.evaluate_rows(pos, s["types"], s["cell"], r1, cs, want_grad=False)[0]
    assert np.abs(E0 - E1).max() < 1e-13 * max(1.0, np.abs(E0).max())


def test_force_on_single_atom_matches_whole_system():
    o, s = _small_case(n=20, edges=(12.5, 13.0, 12.2), seed=83)
    out = o.compute(s["pos"], s["types"], s["cell"], s["pbc"])
    Fk, Ei = o.force_on(s["pos"], s["types"], s["cell"], s["pbc"], 4)
    assert np.abs(Fk - out["F"][4]).max() < 1e-12 * max(1.0, np.abs(out["F"]).max())
    assert abs(Ei[4] - out["E_i"][4]) < 1e-13 * max(1.0, abs(out["E_i"][4]))


def test_atom_virials_sum_to_the_virial_and_split_a_dimer_evenly():
    p = SMALL_PROFILES["p8_2_0"]
    o = orc.Oracle(make_blob(p, seed=9))
    s = make_system(dict(kind="random_box", atoms=20, edges=(7.5, 8.0, 9.0), min_dist=1.6, seed=4, n_types=p["T"],
                         masses=[1.0] * p["T"]))
    res = o.compute(s["pos"], s["types"], s["cell"], s["pbc"])
    W = o.atom_virials(res)
    assert np.allclose(W.sum(axis=0), res["virial"], rtol=0, atol=1e-12 * max(1.0, np.abs(res["virial"]).max()))
    # an isolated pair of equal atoms: the two shares are equal, and each is -1/2 of the sum over
    # both directed edges; with F the force on atom 1 and d = r_1 - r_0 the virial is F (x) d
    pos = np.array([[10.0, 10.0, 10.0], [11.1, 10.4, 9.3]])
    big = [[40.0, 0, 0], [0, 40.0, 0], [0, 0, 40.0]]
    r2 = o.compute(pos, np.zeros(2, dtype=np.int64), big, (0, 0, 0))
    W2 = o.atom_virials(r2)
    assert np.allclose(W2[0], W2[1], rtol=1e-12, atol=1e-15)
    assert np.allclose(W2[0] + W2[1], np.outer(r2["F"][1], pos[1] - pos[0]), rtol=1e-10, atol=1e-14)
