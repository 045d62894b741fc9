"""Batched multi-frame evaluation against the oracle, frame by frame."""

import numpy as np
import pytest
import torch

from oracle import dpa4c as orc
from workloads import CONFIGS, SMALL_PROFILES, make_blob, make_system, workload_blob

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2608_19041_b200 import binding
    return binding


def _dev(a, dtype):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype).cuda().contiguous()


def _frames(p, pbc):
    """A handful of different small frames: sizes, cells (one sheared, one smaller than the cutoff)."""
    descs = [dict(atoms=40, edges=(9.5, 10.5, 12.0), seed=61), dict(atoms=14, edges=(9.0, 13.0, 12.5), seed=62),
             dict(atoms=8, edges=(4.5, 14.0, 7.3), seed=63), dict(atoms=60, edges=(11.0, 12.5, 13.0), seed=64),
             dict(atoms=1, edges=(20.0, 20.0, 20.0), seed=65)]
    out = []
    for k, dsc in enumerate(descs):
        s = make_system(dict(kind="random_box", min_dist=1.6, n_types=p["T"], masses=[1.0] * p["T"], pbc=list(pbc), **dsc))
        cell = np.asarray(s["cell"], dtype=np.float64)
        if k == 1:      # shear the second frame: same fractional coordinates in a general cell
            e = np.diag(cell)
            sheared = np.array([[e[0], 0, 0], [0.3 * e[1], e[1], 0], [-0.2 * e[2], 0.25 * e[2], e[2]]])
            s["pos"] = (s["pos"] / e) @ sheared
            cell = sheared
        out.append(dict(pos=s["pos"], types=s["types"], cell=cell))
    return out


@pytest.mark.parametrize("name,pbc", [("p32_3_2", (1, 1, 1)), ("p16_2_0", (1, 0, 1)), ("p8_4_0", (1, 1, 1))])
def test_batch_matches_the_oracle_frame_by_frame(name, pbc):
    p = SMALL_PROFILES[name]
    blob = make_blob(p, seed=66, bias_scale=0.2, e_ref_scale=0.5)
    frames = _frames(p, pbc)
    frames.insert(2, dict(pos=np.zeros((0, 3)), types=np.zeros(0, dtype=np.int32), cell=np.eye(3) * 9.0))   # an empty frame
    off = np.concatenate([[0], np.cumsum([len(f["pos"]) for f in frames])])
    pos = _dev(np.concatenate([f["pos"] for f in frames]), torch.float64)
    types = _dev(np.concatenate([f["types"] for f in frames]), torch.int32)
    cells = np.stack([f["cell"] for f in frames])
    m = _binding().Model(blob)
    out = m.compute_batch(off, pos, types, cells, pbc, atom_energy=True)
    F, Ei = out["forces"].cpu().numpy(), out["atom_energy"].cpu().numpy()
    o = orc.Oracle(blob)
    for k, f in enumerate(frames):
        a, b = off[k], off[k + 1]
        if a == b:
            assert out["energies"][k] == 0.0 and np.all(out["virials"][k] == 0.0)
            continue
        ref = o.compute(f["pos"], f["types"], f["cell"], pbc)
        e_scale, f_scale, n = np.abs(ref["E_i"]).max(), np.abs(ref["F"]).max(), b - a
        assert np.abs(Ei[a:b] - ref["E_i"]).max() <= 1e-5 * e_scale, k
        assert abs(out["energies"][k] - ref["E"]) / n <= 1e-5 * max(abs(ref["E"]) / n, e_scale), k
        assert np.abs(F[a:b] - ref["F"]).max() <= min(1e-4, 2e-5 * f_scale + 2e-7), k
        assert np.abs(out["virials"][k] - ref["virial"]).max() / n <= 1e-5 * max(1.0, f_scale), k
    # the handle's list was replaced: a plain evaluation needs a new build
    with pytest.raises(_binding().UmlmdError) as e:
        m.compute(pos)
    assert e.value.code == -5
    m.close()


def test_batch_of_copies_equals_the_single_evaluation():
    name = "cfg1_al108"
    s = make_system(CONFIGS[name]["system"])
    blob = workload_blob(name)
    m = _binding().Model(blob)
    pos1, types1 = _dev(s["pos"], torch.float64), _dev(s["types"], torch.int32)
    m.build_neighbors(pos1, types1, s["cell"], s["pbc"], 0.0)
    single = m.compute(pos1, atom_energy=True)
    nf, n = 7, len(s["pos"])
    off = np.arange(nf + 1) * n
    pos = _dev(np.tile(s["pos"], (nf, 1)), torch.float64)
    types = _dev(np.tile(s["types"], nf), torch.int32)
    out = m.compute_batch(off, pos, types, np.tile(np.asarray(s["cell"], dtype=np.float64).reshape(1, 9), (nf, 1)), s["pbc"],
                          atom_energy=True)
    e_scale = single["atom_energy"].abs().max().item()
    f_scale = single["forces"].abs().max().item()
    for k in range(nf):
        # same arithmetic per edge; only the order of the edges inside a row differs from the cell-list build
        assert (out["atom_energy"][k * n:(k + 1) * n] - single["atom_energy"]).abs().max().item() <= 2e-6 * e_scale
        assert (out["forces"][k * n:(k + 1) * n] - single["forces"]).abs().max().item() <= 2e-6 * f_scale
        assert abs(out["energies"][k] - single["energy"]) <= 2e-6 * n * e_scale
        assert np.abs(out["virials"][k] - single["virial"]).max() <= 2e-6 * n * max(1.0, f_scale)
    # every copy is bit for bit the same as the first
    assert np.all(out["energies"] == out["energies"][0])
    assert torch.equal(out["forces"][:n], out["forces"][3 * n:4 * n])
    m.close()


def test_oversized_frame_is_refused():
    p = SMALL_PROFILES["p8_2_0"]
    m = _binding().Model(make_blob(p, seed=1))
    n = 16385
    pos = torch.zeros((n, 3), dtype=torch.float64, device="cuda")
    types = torch.zeros(n, dtype=torch.int32, device="cuda")
    with pytest.raises(_binding().UmlmdError) as e:
        m.compute_batch([0, n], pos, types, np.eye(3).reshape(1, 9) * 100.0)
    assert e.value.code == -9
    m.close()
