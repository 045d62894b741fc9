"""GPU parity: the CUDA library, called through its C ABI, against the fp64 CPU oracle on
the same seeded inputs.

Tolerances (fp32 kernels against an fp64 reference):
  * neighbor lists: identical as sorted sets of (j, n) per centre;
  * aggregated sums and feature vector: 2e-5 of the largest entry of the block compared;
  * atomic energies: max |dE_i| <= 1e-5 * max_j |E_j| (relative to the largest atomic energy,
    the convention the paper uses for its own single-precision fidelity figures); total
    energy per atom likewise;
  * forces: max |dF| <= 1e-4 eV/Angstrom and <= 2e-5 of the largest force component;
    virial: |dXi| / N <= 1e-5 eV (times the force scale when that exceeds 1 eV/Angstrom).
Plain float32 PyTorch on the same inputs shows the same noise floor (about 1e-5 of the RMS
atomic energy on the near-centrosymmetric 108-atom crystal, whose odd-degree sums cancel).
"""

import numpy as np
import pytest
import torch

from oracle import dpa4c as orc
from workloads import CONFIGS, SMALL_PROFILES, load_calibration, make_blob, make_system, workload_blob

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2608_19041_b200 import binding
    return binding


def _dev(a, dtype):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype).cuda().contiguous()


def _rows_from_gpu(model, N):
    row_ptr, src, shift = model.get_neighbors()
    row_ptr, src, shift = row_ptr.cpu().numpy(), src.cpu().numpy(), shift.cpu().numpy()
    rows = []
    for i in range(N):
        a, b = row_ptr[i], row_ptr[i + 1]
        ent = np.concatenate([src[a:b, None].astype(np.int64), shift[a:b].astype(np.int64)], axis=1)
        order = np.lexsort((ent[:, 3], ent[:, 2], ent[:, 1], ent[:, 0]))
        rows.append(ent[order])
    return rows


def _build(blob, s, skin=0.0, **kw):
    m = _binding().Model(blob, **kw)
    pos = _dev(s["pos"], torch.float64)
    types = _dev(s["types"], torch.int32)
    m.build_neighbors(pos, types, s["cell"], s["pbc"], skin)
    return m, pos


TINY = [
    dict(kind="random_box", atoms=6, edges=(4.0, 4.5, 5.0), min_dist=1.2, seed=11, n_types=1, masses=[1.0], shift=True),
    dict(kind="random_box", atoms=14, edges=(9.0, 13.0, 12.5), min_dist=1.2, seed=12, n_types=1, masses=[1.0], shift=True),
    dict(kind="random_box", atoms=8, edges=(3.1, 14.0, 7.3), min_dist=1.2, seed=13, n_types=1, masses=[1.0]),
    dict(kind="random_box", atoms=40, edges=(14.5, 12.1, 19.0), min_dist=1.2, seed=14, n_types=1, masses=[1.0]),
    dict(kind="random_box", atoms=12, edges=(6.0, 6.0, 6.0), min_dist=1.5, seed=15, n_types=1, masses=[1.0], pbc=[0, 0, 0]),
    dict(kind="random_box", atoms=30, edges=(20.0, 7.0, 9.0), min_dist=1.5, seed=16, n_types=1, masses=[1.0], pbc=[0, 1, 1]),
    dict(kind="random_box", atoms=300, edges=(21.0, 22.5, 30.0), min_dist=1.5, seed=17, n_types=1, masses=[1.0], shift=True),
]


@pytest.mark.parametrize("desc", TINY, ids=lambda d: f"n{d['atoms']}_{'x'.join(map(str, d['edges']))}")
@pytest.mark.parametrize("skin", [0.0, 1.0])
def test_neighbor_lists_bit_exact_on_small_cells(desc, skin):
    s = make_system(desc)
    blob = make_blob(SMALL_PROFILES["p8_2_0"], seed=1)
    m, _ = _build(blob, s, skin=skin)
    got = _rows_from_gpu(m, len(s["pos"]))
    pos = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    ref = orc.neighbor_rows(pos, s["cell"], s["pbc"], 6.0 + skin)
    assert m.query()["n_edges"] == sum(len(r) for r in ref)
    for a, b in zip(got, ref):
        assert np.array_equal(a, b)


@pytest.mark.parametrize("name", ["cfg1_al108", "cfg2_cu4000"])
def test_neighbor_lists_bit_exact_on_workloads(name):
    cfg = CONFIGS[name]
    s = make_system(cfg["system"])
    blob = make_blob(SMALL_PROFILES["p8_2_0"], seed=1)
    for skin in (0.0, 1.0):
        m, _ = _build(blob, s, skin=skin)
        got = _rows_from_gpu(m, len(s["pos"]))
        pos = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
        ref = orc.neighbor_rows(pos, s["cell"], s["pbc"], 6.0 + skin)
        assert all(np.array_equal(a, b) for a, b in zip(got, ref))
        m.close()


def test_empty_system_and_single_atom():
    blob = make_blob(SMALL_PROFILES["p8_2_0"], seed=1, e_ref_scale=0.5, bias_scale=0.2)
    B = _binding()
    m = B.Model(blob)
    pos = torch.zeros((0, 3), dtype=torch.float64, device="cuda")
    types = torch.zeros((0,), dtype=torch.int32, device="cuda")
    m.build_neighbors(pos, types, np.eye(3) * 20.0)
    out = m.compute(pos)
    assert out["energy"] == 0.0 and np.all(out["virial"] == 0)
    # one isolated atom: no edges, energy = MLP of the empty-neighbourhood features
    s = dict(pos=np.array([[1.0, 2.0, 3.0]]), types=np.array([1], dtype=np.int32), cell=np.eye(3) * 20.0,
             pbc=np.array([1, 1, 1]))
    m, pos = _build(blob, s)
    assert m.query()["n_edges"] == 0
    out = m.compute(pos, atom_energy=True)
    ref = orc.Oracle(blob).compute(s["pos"], s["types"], s["cell"], s["pbc"])
    assert abs(out["energy"] - ref["E"]) < 1e-5 * max(1.0, abs(ref["E"]))
    assert out["forces"].abs().max().item() == 0.0


def _compare(blob, s, tol_scale=1.0, skin=0.0, check_intermediates=True, **kw):
    o = orc.Oracle(blob)
    ref = o.compute(s["pos"], s["types"], s["cell"], s["pbc"])
    m, pos = _build(blob, s, skin=skin, **kw)
    N = len(s["pos"])
    if check_intermediates:
        m.compute(pos, forces=False, virial=False)
        state, desc = m.get_intermediates()
        state, desc = state.cpu().numpy().astype(np.float64), desc.cpu().numpy().astype(np.float64)
        ty = torch.from_numpy(s["types"].astype(np.int64))
        dst_t = torch.from_numpy(ref["dst"])
        A, s0, s1 = orc.aggregate(o.p, o.prm, o.pair, N, dst_t, ty[dst_t], ty[torch.from_numpy(ref["src"])],
                                  torch.from_numpy(ref["rij"]))
        flat = torch.cat([a.reshape(N, -1) for a in A] + [s0[:, None], s1[:, None]], dim=1).numpy()
        off = 0
        for l, a in enumerate(A):
            w = a[0].numel()
            blk = flat[:, off:off + w]
            assert np.abs(state[:, off:off + w] - blk).max() <= 2e-5 * tol_scale * max(np.abs(blk).max(), 1e-30), f"A_{l}"
            off += w
        assert np.abs(state[:, off:] - flat[:, off:]).max() <= 2e-5 * np.abs(flat[:, off:]).max()
        Dref = (ref["D_raw"] - o.prm["mu"].numpy()) / o.prm["sigma"].numpy()
        err = np.abs(desc - Dref)
        assert err.max() <= 5e-5 * tol_scale * np.abs(Dref).max(), (err.max(), np.unravel_index(err.argmax(), err.shape))
    out = m.compute(pos, atom_energy=True)
    Ei = out["atom_energy"].cpu().numpy()
    F = out["forces"].cpu().numpy()
    e_scale = np.abs(ref["E_i"]).max()
    f_scale = np.abs(ref["F"]).max()
    assert np.abs(Ei - ref["E_i"]).max() <= 1e-5 * tol_scale * e_scale, np.abs(Ei - ref["E_i"]).max() / e_scale
    assert abs(out["energy"] - ref["E"]) / N <= 1e-5 * tol_scale * max(abs(ref["E"]) / N, e_scale)
    f_err = np.abs(F - ref["F"]).max()
    assert f_err <= 1e-4 * tol_scale and f_err <= 2e-5 * f_scale + 2e-7, (f_err, f_scale)
    assert np.abs(out["virial"] - ref["virial"]).max() / N <= 1e-5 * tol_scale * max(1.0, f_scale)
    m.close()
    return ref, out


SYS_SMALL = dict(kind="random_box", atoms=60, edges=(9.5, 10.5, 12.0), min_dist=1.7, seed=31, masses=[1.0] * 3)


@pytest.mark.parametrize("pair_table_mb", [-1, 0], ids=["pair_cache", "pair_tables"])
@pytest.mark.parametrize("name", sorted(SMALL_PROFILES))
def test_energy_force_virial_parity_small_profiles(name, pair_table_mb):
    # with and without the per-pair amplitude tables that the library builds when few species
    # are present (the oracle knows no such path)
    p = SMALL_PROFILES[name]
    blob = make_blob(p, seed=40, bias_scale=0.2, e_ref_scale=0.5)
    s = make_system(dict(SYS_SMALL, n_types=p["T"]))
    _compare(blob, s, pair_table_mb=pair_table_mb)


def test_parity_with_skin_and_multi_image_box():
    p = SMALL_PROFILES["p16_3_2"]
    blob = make_blob(p, seed=41, bias_scale=0.2)
    s = make_system(dict(kind="random_box", atoms=16, edges=(5.0, 7.7, 8.1), min_dist=1.6, seed=32,
                         n_types=p["T"], masses=[1.0] * p["T"], shift=True))
    _compare(blob, s, skin=1.0)


def test_parity_isolated_cluster():
    p = SMALL_PROFILES["p32_2_4"]
    blob = make_blob(p, seed=42)
    s = make_system(dict(kind="random_box", atoms=20, edges=(7.0, 7.0, 7.0), min_dist=1.6, seed=33,
                         n_types=p["T"], masses=[1.0] * p["T"], pbc=[0, 0, 0]))
    _compare(blob, s)


@pytest.mark.parametrize("name", ["p16_3_2", "p32_2_4", "p8_2_0"])
def test_parity_one_species_present_out_of_several(name):
    # all atoms of one species (not index 0): a single pair table, shared radial modes included
    p = SMALL_PROFILES[name]
    blob = make_blob(p, seed=44, bias_scale=0.2, e_ref_scale=0.5)
    s = make_system(dict(SYS_SMALL, n_types=p["T"]))
    s["types"] = np.full_like(s["types"], p["T"] - 1)
    _compare(blob, s)


def test_species_mix_may_change_between_builds_on_one_handle():
    p = SMALL_PROFILES["p32_3_2"]
    blob = make_blob(p, seed=45, bias_scale=0.2)
    s = make_system(dict(SYS_SMALL, n_types=p["T"]))
    assert len(np.unique(s["types"])) > 1
    one = dict(s, types=np.full_like(s["types"], 1 % p["T"]))
    o = orc.Oracle(blob)
    m, pos = _build(blob, one)
    two = dict(s, types=np.where(s["types"] == s["types"][0], 0, p["T"] - 1).astype(s["types"].dtype))
    for sysd in (one, s, two, one):
        m.build_neighbors(pos, _dev(sysd["types"], torch.int32), s["cell"], s["pbc"], 0.0)
        ref = o.compute(s["pos"], sysd["types"], s["cell"], s["pbc"])
        out = m.compute(pos)
        f_scale = np.abs(ref["F"]).max()
        assert np.abs(out["forces"].cpu().numpy() - ref["F"]).max() <= 2e-5 * f_scale + 2e-7
        assert abs(out["energy"] - ref["E"]) <= 1e-5 * len(s["pos"]) * np.abs(ref["E_i"]).max()
    m.close()


@pytest.mark.parametrize("name", ["p16_3_2", "p32_2_0_res"])
def test_parity_gaussian_radial_family(name):
    # only the create-time table differs: Gaussian basis functions with the centres in the blob
    p = SMALL_PROFILES[name]
    blob = make_blob(p, seed=47, bias_scale=0.2, basis="gaussian")
    s = make_system(dict(SYS_SMALL, n_types=p["T"]))
    _compare(blob, s)


def test_parity_with_node_tiling():
    # several workspace tiles with a ragged last tile
    p = SMALL_PROFILES["p16_2_0"]
    blob = make_blob(p, seed=43, bias_scale=0.2)
    s = make_system(dict(SYS_SMALL, n_types=p["T"], atoms=75))
    _compare(blob, s, check_intermediates=False, node_tile=32)


@pytest.mark.parametrize("name", ["cfg1_al108", "cfg2_cu4000"])
def test_parity_on_workloads(name):
    cfg = CONFIGS[name]
    s = make_system(cfg["system"])
    blob = workload_blob(name)
    _compare(blob, s)


def test_results_are_bitwise_reproducible():
    cfg = CONFIGS["cfg1_al108"]
    s = make_system(cfg["system"])
    blob = workload_blob("cfg1_al108")
    m, pos = _build(blob, s)
    a = m.compute(pos)
    b = m.compute(pos)
    assert a["energy"] == b["energy"] and torch.equal(a["forces"], b["forces"])
    assert np.array_equal(a["virial"], b["virial"])


def test_stale_list_is_reported():
    p = SMALL_PROFILES["p8_2_0"]
    blob = make_blob(p, seed=44)
    s = make_system(dict(SYS_SMALL, n_types=p["T"]))
    m, pos = _build(blob, s, skin=0.4)
    moved = pos.clone()
    moved[3, 0] += 0.15
    m.compute(moved)                       # within skin/2
    moved[3, 0] += 0.2
    with pytest.raises(_binding().UmlmdError) as e:
        m.compute(moved)
    assert e.value.code == -6
    m.compute(pos)                         # the handle stays usable


@pytest.mark.parametrize("bad", [-1, 2])
def test_species_index_out_of_range_is_refused(bad):
    # the index would address the pair cache out of bounds: the build reports it, nothing reads it
    p = SMALL_PROFILES["p8_2_0"]
    assert p["T"] == 2
    blob = make_blob(p, seed=44)
    s = make_system(dict(SYS_SMALL, n_types=p["T"]))
    m, pos = _build(blob, s)
    types = s["types"].copy()
    types[7] = bad
    with pytest.raises(_binding().UmlmdError) as e:
        m.build_neighbors(pos, _dev(types, torch.int32), s["cell"], s["pbc"], 0.0)
    assert e.value.code == -1
    with pytest.raises(_binding().UmlmdError) as e:
        m.compute(pos)                     # no list: the failed build left none
    assert e.value.code == -5
    m.build_neighbors(pos, _dev(s["types"], torch.int32), s["cell"], s["pbc"], 0.0)
    m.compute(pos)                         # the handle stays usable
    m.close()


@pytest.mark.parametrize("path", [2, 3])
@pytest.mark.parametrize("name", ["p16_3_2", "p32_2_4", "p32_2_0_res"])
def test_tensor_core_mlp_path_small_profiles(name, path):
    # both tensor-core GEMM variants (2: persistent 256-row items, 3: one tile per CTA) with
    # ragged everything: fewer rows than a tile, widths that are not multiples of the tile
    p = SMALL_PROFILES[name]
    blob = make_blob(p, seed=45, bias_scale=0.2, e_ref_scale=0.5)
    s = make_system(dict(SYS_SMALL, n_types=p["T"], atoms=150, edges=(12.5, 13.5, 14.0)))
    _compare(blob, s, check_intermediates=False, mlp_path=path)


def test_table_spacing_sweep_against_the_continuous_model():
    # the paper's fidelity experiment on random weights: the tabulated path against the
    # continuous model for a range of table spacings.  The library stores the cubic two-point
    # interpolant, whose error grows like the fourth power of the spacing (third for the
    # derivative), with its quadratic and cubic coefficients packed into one word, which adds a
    # derivative error proportional to the spacing; up to 0.002 A the result sits at the
    # single-precision floor, and the forces, which see the derivative of the table, resolve
    # the spacing first.
    p = SMALL_PROFILES["p32_3_2"]
    blob = make_blob(p, seed=46)
    s = make_system(dict(SYS_SMALL, n_types=p["T"]))
    o = orc.Oracle(blob)
    ref = o.compute(s["pos"], s["types"], s["cell"], s["pbc"])
    Dref = (ref["D_raw"] - o.prm["mu"].numpy()) / o.prm["sigma"].numpy()
    dev = {}
    for dx in (0.0005, 0.002, 0.005, 0.01, 0.02, 0.05):
        m, pos = _build(blob, s, table_dx=dx)
        m.compute(pos, forces=False, virial=False)
        _, desc = m.get_intermediates()
        desc = desc.cpu().numpy().astype(np.float64)
        out = m.compute(pos)
        dev[dx] = (np.abs(desc - Dref).max() / np.abs(Dref).max(),
                   np.abs(out["forces"].cpu().numpy() - ref["F"]).max() / np.abs(ref["F"]).max())
        m.close()
    for dx in (0.0005, 0.002):
        assert dev[dx][0] <= 2e-6 and dev[dx][1] <= 5e-6, (dx, dev[dx])
    assert dev[0.005][0] <= 2e-6 and dev[0.005][1] <= 1e-5, dev[0.005]
    assert dev[0.01][1] <= 5e-5 and dev[0.02][1] <= 3e-4 and dev[0.05][1] <= 3e-3, dev
    assert dev[0.05][1] > 10 * dev[0.002][1]                 # the coarse end is resolvably worse


@pytest.mark.parametrize("name", ["paper_nano_c1m", "paper_air_c1m", "paper_plus_c1m"])
def test_paper_variants_on_small_diamond_cell(name):
    # the paper's model variants (118-species type table, carbon only) on a 512-atom cell of its
    # jittered-diamond workload: 158 neighbours per atom, box < 2 (r_c + skin)
    cfg = CONFIGS[name]
    s = make_system(dict(cfg["system"], cells=4))
    blob = make_blob(cfg["profile"], seed=cfg["weights_seed"], calibration=load_calibration(name), bias_scale=0.1,
                     e_ref_scale=0.5)
    # a nearly perfect lattice, like the 108-atom Al cell: the odd-degree invariants almost cancel and
    # single-precision noise in them is amplified by the calibration; the per-variant error is printed
    for skin in (0.0, 1.0):
        ref, out = _compare(blob, s, check_intermediates=False, skin=skin)
        err = np.abs(out["atom_energy"].cpu().numpy() - ref["E_i"]).max() / np.abs(ref["E_i"]).max()
        print(f"{name} skin {skin}: max|dE_i| / max|E_i| = {err:.2e}")


def test_tensor_core_mlp_path_matches_cuda_core_path_on_cu4000():
    name = "cfg2_cu4000"
    s = make_system(CONFIGS[name]["system"])
    blob = workload_blob(name)
    outs = []
    for path in (1, 2, 3):
        m, pos = _build(blob, s, mlp_path=path, node_tile=1536)    # three tiles, ragged last one (928 = 3 * 256 + 160 rows)
        outs.append(m.compute(pos, atom_energy=True))
        m.close()
    a = outs[0]
    e_scale = a["atom_energy"].abs().max().item()
    f_scale = a["forces"].abs().max().item()
    for b in outs[1:]:
        # the tensor core truncates when it aligns partial sums, a ~2e-6 relative one-sided bias
        assert (a["atom_energy"] - b["atom_energy"]).abs().max().item() <= 5e-6 * e_scale
        assert (a["forces"] - b["forces"]).abs().max().item() <= 1e-5 * f_scale
        assert np.abs(a["virial"] - b["virial"]).max() <= 1e-5 * np.abs(a["virial"]).max()
    # (at this tile size path 2 also picks the one-tile kernel, which keeps the cross terms in an
    # accumulator of their own and carries a third of the persistent kernel's truncation bias)
    d2 = (a["atom_energy"] - outs[1]["atom_energy"]).abs().max().item()
    d3 = (a["atom_energy"] - outs[2]["atom_energy"]).abs().max().item()
    print(f"max|dE_i| vs CUDA-core path: path 2 {d2 / e_scale:.2e}, path 3 {d3 / e_scale:.2e} of max|E_i|")


@pytest.mark.parametrize("name", ["p32_2_4", "p128_3_4"])
def test_persistent_tensor_core_kernels_match_the_cuda_core_path(name):
    # enough rows that path 2 takes the one-CTA persistent kernel and path 4 the two-CTA one (both
    # fall back to one tile per CTA on small systems); ragged last row tile, widths that are not
    # multiples of the column tile
    p = SMALL_PROFILES[name]
    blob = make_blob(p, seed=50, bias_scale=0.2, e_ref_scale=0.5)
    s = make_system(dict(kind="fcc", cells=18, a=4.05, jitter=0.05, seed=6, n_types=p["T"], masses=[1.0] * p["T"]))
    outs = {}
    for path in (1, 2, 4):
        m, pos = _build(blob, s, mlp_path=path)
        outs[path] = m.compute(pos, atom_energy=True)
        m.close()
    a = outs[1]
    e_scale = a["atom_energy"].abs().max().item()
    f_scale = a["forces"].abs().max().item()
    for path in (2, 4):
        b = outs[path]
        de = (a["atom_energy"] - b["atom_energy"]).abs().max().item()
        print(f"{name} path {path}: max|dE_i| vs CUDA-core path {de / e_scale:.2e} of max|E_i|")
        assert de <= 5e-6 * e_scale
        assert (a["forces"] - b["forces"]).abs().max().item() <= 1e-5 * f_scale
        assert np.abs(a["virial"] - b["virial"]).max() <= 1e-5 * np.abs(a["virial"]).max()


# ------------------------------------------------------------------ general (triclinic) cells

def _sheared(desc, tilt, flip=False):
    """The random box of `desc` mapped into a general cell: same fractional coordinates, cell rows
    a = (ex, 0, 0), b = (t0 ey, ey, 0), c = (t1 ez, t2 ez, ez); `flip` swaps two rows (left-handed)."""
    s = make_system(desc)
    e = np.diag(np.asarray(s["cell"], dtype=np.float64))
    cell = np.array([[e[0], 0.0, 0.0], [tilt[0] * e[1], e[1], 0.0], [tilt[1] * e[2], tilt[2] * e[2], e[2]]])
    frac = s["pos"] / e
    if flip:
        cell, frac = cell[[1, 0, 2]], frac[:, [1, 0, 2]]
        s["pbc"] = [s["pbc"][1], s["pbc"][0], s["pbc"][2]]
    s["pos"] = frac @ cell
    s["cell"] = cell.tolist()
    return s


TRI = [
    (dict(kind="random_box", atoms=14, edges=(9.0, 13.0, 12.5), min_dist=1.4, seed=52, n_types=1, masses=[1.0], shift=True), (0.3, -0.2, 0.25), False),
    (dict(kind="random_box", atoms=8, edges=(4.1, 14.0, 7.3), min_dist=1.4, seed=53, n_types=1, masses=[1.0]), (0.45, 0.1, -0.35), False),
    (dict(kind="random_box", atoms=300, edges=(21.0, 22.5, 30.0), min_dist=1.6, seed=57, n_types=1, masses=[1.0], shift=True), (-0.4, 0.3, 0.2), False),
    (dict(kind="random_box", atoms=30, edges=(20.0, 7.0, 9.0), min_dist=1.6, seed=56, n_types=1, masses=[1.0], pbc=[0, 1, 1]), (0.2, 0.2, -0.3), False),
    (dict(kind="random_box", atoms=40, edges=(14.5, 12.1, 19.0), min_dist=1.4, seed=54, n_types=1, masses=[1.0]), (0.25, 0.15, 0.3), True),
]


@pytest.mark.parametrize("case", range(len(TRI)))
@pytest.mark.parametrize("skin", [0.0, 1.0])
def test_neighbor_lists_in_general_cells(case, skin):
    desc, tilt, flip = TRI[case]
    s = _sheared(desc, tilt, flip)
    blob = make_blob(SMALL_PROFILES["p8_2_0"], seed=1)
    m, _ = _build(blob, s, skin=skin)
    got = _rows_from_gpu(m, len(s["pos"]))
    pos = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    ref = orc.neighbor_rows(pos, s["cell"], s["pbc"], 6.0 + skin)
    assert m.query()["n_edges"] == sum(len(r) for r in ref)
    for a, b in zip(got, ref):
        assert np.array_equal(a, b)
    m.close()


@pytest.mark.parametrize("name,case", [("p16_3_2", 0), ("p32_2_4", 1), ("p32_3_2", 2), ("p8_2_0", 3), ("p16_2_0", 4)])
def test_parity_in_general_cells(name, case):
    p = SMALL_PROFILES[name]
    desc, tilt, flip = TRI[case]
    blob = make_blob(p, seed=48, bias_scale=0.2)
    s = _sheared(dict(desc, n_types=p["T"], masses=[1.0] * p["T"]), tilt, flip)
    _compare(blob, s, skin=0.5 * (case % 2))


def test_singular_cell_is_refused():
    p = SMALL_PROFILES["p8_2_0"]
    blob = make_blob(p, seed=1)
    s = make_system(dict(SYS_SMALL, n_types=p["T"]))
    m, pos = _build(blob, s)
    bad = [[9.5, 0.0, 0.0], [19.0, 0.0, 0.0], [0.0, 0.0, 12.0]]
    with pytest.raises(_binding().UmlmdError) as e:
        m.build_neighbors(pos, _dev(s["types"], torch.int32), bad, s["pbc"], 0.0)
    assert e.value.code == -4
    m.close()


@pytest.mark.parametrize("general_cell", [False, True])
def test_atom_virials(general_cell):
    p = SMALL_PROFILES["p32_3_2"]
    blob = make_blob(p, seed=49, bias_scale=0.2)
    desc = dict(SYS_SMALL, n_types=p["T"])
    s = _sheared(desc, (0.3, -0.2, 0.25)) if general_cell else make_system(desc)
    o = orc.Oracle(blob)
    ref = o.compute(s["pos"], s["types"], s["cell"], s["pbc"])
    Wref = o.atom_virials(ref)
    m, pos = _build(blob, s, skin=0.7)
    with pytest.raises(_binding().UmlmdError):
        m.atom_virial()                            # nothing evaluated yet
    out = m.compute(pos)
    W = m.atom_virial().cpu().numpy()
    scale = max(np.abs(Wref).max(), 1e-12)
    assert np.abs(W - Wref).max() <= 2e-5 * scale
    # the total is accumulated from single-precision products in the edge kernel
    assert np.abs(W.sum(axis=0) - out["virial"]).max() <= 1e-5 * np.abs(out["virial"]).max() + 1e-5 * scale
    m.compute(pos, forces=False, virial=False)     # an energy-only evaluation leaves no edge gradients
    with pytest.raises(_binding().UmlmdError):
        m.atom_virial()
    m.close()
