"""Full-size parity: the three large workloads in the configuration bench.py times (list
radius r_c + skin, default node tiling, default MLP path), checked against the oracle on
sampled outputs that it can compute one by one, plus properties that hold at any size."""

import numpy as np
import pytest
import torch

from oracle import dpa4c as orc
from workloads import CONFIGS, make_system, workload_blob

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2608_19041_b200 import binding
    return binding


@pytest.mark.parametrize("name,n_force,n_rows,modes", [("cfg3_water32400", 3, 48, None), ("cfg4_hea128k", 3, 48, None),
                                                       ("cfg5_amorphous1m", 2, 24, None),
                                                       ("cfg3_water32400", 2, 24, 4),    # R = 4: the profile with shared radial modes
                                                       ("cfg5_amorphous1m", 1, 12, 4)])  # R = 4 with 64 species: modes read through the pair cache
def test_fullsize_sampled_parity(name, n_force, n_rows, modes):
    cfg = CONFIGS[name]
    s = make_system(cfg["system"])
    N = len(s["pos"])
    blob = workload_blob(name, modes)
    skin = cfg["md"]["skin"]
    m = _binding().Model(blob)
    pos = torch.as_tensor(s["pos"], dtype=torch.float64).cuda().contiguous()
    types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
    m.build_neighbors(pos, types, s["cell"], s["pbc"], skin)
    out = m.compute(pos, atom_energy=True)
    Ei = out["atom_energy"].cpu().numpy()
    F = out["forces"].cpu().numpy()
    assert np.isfinite(Ei).all() and np.isfinite(F).all()

    # ---- properties that hold at any size
    f_scale, e_scale = np.abs(F).max(), np.abs(Ei).max()
    assert abs(Ei.sum() - out["energy"]) <= 1e-9 * max(1.0, np.abs(Ei).sum())
    assert np.abs(F.sum(axis=0)).max() <= 2e-6 * f_scale * np.sqrt(N) * 10       # sum of forces ~ fp32 noise
    V = out["virial"]
    assert np.abs(V - V.T).max() <= 1e-5 * max(np.abs(V).max(), 1e-12)

    # ---- neighbor rows of sampled centres, bit-exact as sorted sets
    rng = np.random.Generator(np.random.PCG64(2024 + cfg["index"]))
    centers = np.sort(rng.choice(N, size=n_rows, replace=False))
    pos_w = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    ref_rows = orc.neighbor_rows(pos_w, s["cell"], s["pbc"], cfg["profile"]["rc"] + skin, centers=centers)
    row_ptr, src, shift = m.get_neighbors()
    rp = row_ptr.cpu().numpy()
    assert rp[-1] == m.query()["n_edges"]
    for c, ref in zip(centers, ref_rows):
        a, b = int(rp[c]), int(rp[c + 1])
        ent = np.concatenate([src[a:b].cpu().numpy()[:, None].astype(np.int64),
                              shift[a:b].cpu().numpy().astype(np.int64)], axis=1)
        ent = ent[np.lexsort((ent[:, 3], ent[:, 2], ent[:, 1], ent[:, 0]))]
        assert np.array_equal(ent, ref), c
    del row_ptr, src, shift

    # ---- forces on sampled atoms and energies of their whole neighbourhoods
    o = orc.Oracle(blob)
    for k in rng.choice(N, size=n_force, replace=False):
        Fk, E_near = o.force_on(s["pos"], s["types"], s["cell"], s["pbc"], int(k))
        assert np.abs(F[k] - Fk).max() <= min(1e-4, 2e-5 * f_scale + 2e-7), (k, F[k], Fk)
        for a, ea in E_near.items():
            assert abs(Ei[a] - ea) <= 1e-5 * e_scale, (a, Ei[a], ea)
    m.close()


@pytest.mark.parametrize("name", ["cfg3_water32400", "cfg4_hea128k", "cfg5_amorphous1m"])
def test_fullsize_nve_drift_over_the_configured_run(name):
    # the workload's own MD recipe (steps, time step, temperature, rebuild interval, skin) in the
    # configuration bench.py times; drift = slope of a least-squares line through (E_pot + E_kin) / N
    cfg = CONFIGS[name]
    md = cfg["md"]
    s = make_system(cfg["system"], md)
    N = len(s["pos"])
    m = _binding().Model(workload_blob(name))
    pos = torch.as_tensor(s["pos"], dtype=torch.float64).cuda().contiguous()
    vel = torch.as_tensor(s["vel"], dtype=torch.float64).cuda().contiguous()
    types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
    m.build_neighbors(pos, types, s["cell"], s["pbc"], md["skin"])
    m.set_md_state(pos, vel, s["masses"])
    chunk = max(1, md["steps"] // 10)
    t, e = [0.0], []
    ep, ek = m.step(0, md["dt_ps"], md["rebuild_every"])
    e.append((ep + ek) / N)
    for k in range(md["steps"] // chunk):
        ep, ek = m.step(chunk, md["dt_ps"], md["rebuild_every"])
        t.append((k + 1) * chunk * md["dt_ps"])
        e.append((ep + ek) / N)
    slope = np.polyfit(np.array(t), np.array(e), 1)[0]
    print(f"{name}: NVE drift {slope:.3e} eV/atom/ps over {t[-1]:.3f} ps, E/N {min(e):.8f}..{max(e):.8f}")
    assert np.isfinite(e).all()
    assert abs(slope) <= 1e-5
    m.close()


def _cluster_around(pos_w, cell, k, radius):
    """Atoms within `radius` of atom k (minimum image, orthorhombic cell), as an isolated
    cluster with atom k first: indices into the system and unwrapped coordinates."""
    L = np.array([cell[0][0], cell[1][1], cell[2][2]])
    d = pos_w - pos_w[k]
    d -= L * np.round(d / L)
    idx = np.nonzero((d * d).sum(axis=1) < radius * radius)[0]
    idx = np.concatenate([[k], idx[idx != k]])
    return idx, d[idx] + 0.5 * L


def test_just_below_2_31_edges():
    # the largest jittered-diamond box whose neighbor list the 32-bit verification export still takes
    # (6,859,000 atoms, 1.88e9 listed edges, 3 E > 2^32): properties that hold at any size, sampled
    # rows against brute force, and energies and forces of sampled atoms against the oracle run
    # on the isolated cluster that determines them (radius 2 r_c around the atom)
    name = "paper_nano_c1m"
    cfg = CONFIGS[name]
    s = make_system(dict(cfg["system"], cells=95))
    N = len(s["pos"])
    skin = cfg["md"]["skin"]
    rc = cfg["profile"]["rc"]
    blob = workload_blob(name)
    m = _binding().Model(blob)
    pos = torch.as_tensor(s["pos"], dtype=torch.float64).cuda().contiguous()
    types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
    m.build_neighbors(pos, types, s["cell"], s["pbc"], skin)
    E = m.query()["n_edges"]
    assert 3 * E > 2 ** 32 and E < 2 ** 31
    out = m.compute(pos, atom_energy=True)
    Ei = out["atom_energy"].cpu().numpy()
    F = out["forces"].cpu().numpy()
    assert np.isfinite(Ei).all() and np.isfinite(F).all()
    f_scale, e_scale = np.abs(F).max(), np.abs(Ei).max()
    assert abs(Ei.sum() - out["energy"]) <= 1e-9 * max(1.0, np.abs(Ei).sum())
    assert np.abs(F.sum(axis=0)).max() <= 2e-6 * f_scale * np.sqrt(N) * 10
    V = out["virial"]
    assert np.abs(V - V.T).max() <= 1e-5 * max(np.abs(V).max(), 1e-12)

    rng = np.random.Generator(np.random.PCG64(95))
    pos_w = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    row_ptr, src, shift = m.get_neighbors()
    rp = row_ptr.cpu().numpy()
    assert rp[-1] == E
    centers = np.sort(rng.choice(N, size=2, replace=False))
    for c, ref in zip(centers, orc.neighbor_rows(pos_w, s["cell"], s["pbc"], rc + skin, centers=centers)):
        a, b = int(rp[c]), int(rp[c + 1])
        ent = np.concatenate([src[a:b].cpu().numpy()[:, None].astype(np.int64),
                              shift[a:b].cpu().numpy().astype(np.int64)], axis=1)
        ent = ent[np.lexsort((ent[:, 3], ent[:, 2], ent[:, 1], ent[:, 0]))]
        assert np.array_equal(ent, ref), c
    del row_ptr, src, shift

    o = orc.Oracle(blob)
    big = [[1000.0, 0, 0], [0, 1000.0, 0], [0, 0, 1000.0]]
    for k in rng.choice(N, size=2, replace=False):
        idx, xyz = _cluster_around(pos_w, s["cell"], int(k), 2 * rc + 0.5)
        ref = o.compute(xyz, s["types"][idx], big, (0, 0, 0))
        assert np.abs(F[k] - ref["F"][0]).max() <= min(1e-4, 2e-5 * f_scale + 2e-7), (k, F[k], ref["F"][0])
        near = np.nonzero(((xyz - xyz[0]) ** 2).sum(axis=1) < rc * rc)[0]     # complete neighbourhoods
        assert np.abs(Ei[idx[near]] - ref["E_i"][near]).max() <= 1e-5 * e_scale
    m.close()


def test_more_than_2_31_edges():
    # 8,000,000 diamond atoms with the 1 A skin list 2.19e9 edges, more than a 32-bit offset holds:
    # edge offsets are 64-bit inside the library (only the verification export is 32-bit and says
    # so); energies and forces of sampled atoms against the oracle on their isolated clusters
    name = "paper_nano_c1m"
    cfg = CONFIGS[name]
    s = make_system(dict(cfg["system"], cells=100))
    N = len(s["pos"])
    rc = cfg["profile"]["rc"]
    blob = workload_blob(name)
    m = _binding().Model(blob)
    pos = torch.as_tensor(s["pos"], dtype=torch.float64).cuda().contiguous()
    types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
    m.build_neighbors(pos, types, s["cell"], s["pbc"], cfg["md"]["skin"])
    assert m.query()["n_edges"] > 2 ** 31
    with pytest.raises(_binding().UmlmdError) as e:
        m.get_neighbors()
    assert e.value.code == -9
    # the row-range export has 64-bit offsets: rows from the start, the middle and the end of the
    # caller's numbering against brute force
    pos_w0 = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    for c, ref_row in zip((0, N // 2 + 1, N - 1),
                          orc.neighbor_rows(pos_w0, s["cell"], s["pbc"], rc + cfg["md"]["skin"], centers=[0, N // 2 + 1, N - 1])):
        _, rsrc, rshift = m.get_neighbor_rows(c, 1)
        ent = np.concatenate([rsrc.cpu().numpy()[:, None].astype(np.int64), rshift.cpu().numpy().astype(np.int64)], axis=1)
        assert np.array_equal(ent[np.lexsort((ent[:, 3], ent[:, 2], ent[:, 1], ent[:, 0]))], ref_row), c
    out = m.compute(pos, atom_energy=True)
    Ei = out["atom_energy"].cpu().numpy()
    F = out["forces"].cpu().numpy()
    assert np.isfinite(Ei).all() and np.isfinite(F).all()
    f_scale, e_scale = np.abs(F).max(), np.abs(Ei).max()
    assert abs(Ei.sum() - out["energy"]) <= 1e-9 * max(1.0, np.abs(Ei).sum())
    assert np.abs(F.sum(axis=0)).max() <= 2e-6 * f_scale * np.sqrt(N) * 10
    rng = np.random.Generator(np.random.PCG64(100))
    pos_w = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    o = orc.Oracle(blob)
    big = [[1000.0, 0, 0], [0, 1000.0, 0], [0, 0, 1000.0]]
    # one atom from the end of the caller's numbering and two anywhere (the internal order is by cell)
    for k in [N - 1] + list(rng.choice(N, size=2, replace=False)):
        idx, xyz = _cluster_around(pos_w, s["cell"], int(k), 2 * rc + 0.5)
        ref = o.compute(xyz, s["types"][idx], big, (0, 0, 0))
        assert np.abs(F[k] - ref["F"][0]).max() <= min(1e-4, 2e-5 * f_scale + 2e-7), (k, F[k], ref["F"][0])
        near = np.nonzero(((xyz - xyz[0]) ** 2).sum(axis=1) < rc * rc)[0]
        assert np.abs(Ei[idx[near]] - ref["E_i"][near]).max() <= 1e-5 * e_scale
    m.close()
