"""CPU-only checks of the C-ABI library: it loads, exports what the header declares,
validates its inputs, and its create-time products (radial table, pair cache, widths) agree
with the oracle's continuous model."""

import ctypes
import os
import re
import struct

import numpy as np
import pytest
import torch

from oracle import dpa4c as orc
from paper_2608_19041_b200 import binding
from workloads import CONFIGS, SMALL_PROFILES, make_blob

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _header_functions():
    text = open(os.path.join(ROOT, "include", "umlmd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(umlmd_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2608_19041_b200", "libumlmd.so"))
    names = _header_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_profile_widths_match_printed_table():
    rows = [l.split() for l in open(os.path.join(ROOT, "tests", "golden", "widths_table.txt"))
            if l.strip() and not l.startswith("#")]
    for row in rows:
        C0, C1, C2, K1, K2 = map(int, row[:5])
        for k, L in enumerate((2, 3, 4)):
            w = binding.profile_widths(C0, L)
            assert (w["C1"], w["C2"], w["K1"], w["K2"]) == (C1, C2, K1, K2)
            assert w["S"] == int(row[5 + k]) and w["D_out"] == int(row[8 + k])
            ow = orc.widths(C0, L)
            assert (w["H"], w["H_pair"]) == (ow["H"], ow["Hp"])
    for bad in [(12, 2, 0), (32, 1, 0), (32, 5, 0), (32, 2, 3)]:
        with pytest.raises(binding.UmlmdError):
            binding.profile_widths(*bad)


def test_workload_profiles_are_consistent_with_both_width_formulas():
    for cfg in list(CONFIGS.values()):
        p = cfg["profile"]
        w = binding.profile_widths(p["C0"], p["L"], p["R"])
        o = orc.widths(p["C0"], p["L"], p["R"])
        for k in ("C1", "C2", "K1", "K2", "S", "D_out", "H"):
            assert p[k] == w[k] == o[k], k
        assert p["Hp"] == w["H_pair"] == o["Hp"]


def test_create_rejects_bad_blobs():
    p = SMALL_PROFILES["p8_2_0"]
    blob = make_blob(p, seed=1)
    binding.Model(blob).close()
    with pytest.raises(binding.UmlmdError) as e:
        binding.Model(blob[:-4])
    assert e.value.code == -2
    with pytest.raises(binding.UmlmdError) as e:
        binding.Model(b"XXXXXXXX" + blob[8:])
    assert e.value.code == -2
    bad = bytearray(blob)
    bad[12:16] = struct.pack("<I", 12)          # C0 = 12
    with pytest.raises(binding.UmlmdError) as e:
        binding.Model(bytes(bad))
    assert e.value.code == -3
    nan = bytearray(blob)
    nan[-8:-4] = struct.pack("<f", float("nan"))
    with pytest.raises(binding.UmlmdError) as e:
        binding.Model(bytes(nan))
    assert e.value.code == -2
    lib = binding.lib()
    assert lib.umlmd_create(None, 0, None, None, None) == -1


def test_calls_before_a_neighbor_build_fail_cleanly():
    m = binding.Model(make_blob(SMALL_PROFILES["p8_2_0"], seed=1))
    lib = binding.lib()
    e = ctypes.c_double()
    assert lib.umlmd_compute(m._h, None, ctypes.byref(e), None, None, None) == -5
    assert lib.umlmd_step(m._h, 1, 0.001, 0, None, None) == -5
    assert lib.umlmd_step_nvt(m._h, 1, 0.001, 0, 300.0, 0.1, None, None, None) == -5
    assert lib.umlmd_step_nvt(None, 1, 0.001, 0, 300.0, 0.1, None, None, None) == -1
    assert b"build_neighbors" in lib.umlmd_last_error(m._h)
    q = m.query()
    assert q["n_atoms"] == 0 and q["table_rows"] == 3000 and q["rc"] == 6.0


@pytest.mark.parametrize("basis", ["bessel", "gaussian"])
@pytest.mark.parametrize("name", ["p16_2_0", "p32_2_4", "p32_3_2"])
def test_radial_table_reproduces_continuous_radial_map(name, basis):
    # the paper reports 1.3e-7 .. 1.8e-7 (relative to the largest entry) for these three
    # (C0, L, R) at a spacing of 0.002 Angstrom in single precision
    p = SMALL_PROFILES[name]
    blob = make_blob(p, seed=5, basis=basis)
    m = binding.Model(blob)
    o = orc.Oracle(blob)
    assert o.p["basis"] == basis
    rho = np.random.default_rng(0).uniform(0.0, p["rc"], 4000)
    rho[:3] = [0.0, 1e-9, p["rc"] - 1e-9]
    g, dg = m.eval_radial_table(rho)
    r = torch.from_numpy(rho).requires_grad_(True)
    go, qo = orc.radial_map(r, o.prm, basis, p["rc"])
    ref = torch.cat([go, qo], dim=1)
    scale = ref.abs().max().item()
    assert np.abs(g - ref.detach().numpy()).max() / scale < 3e-7
    dref = torch.stack([torch.autograd.grad(ref[:, c].sum(), r, retain_graph=True)[0]
                        for c in range(ref.shape[1])], dim=1).numpy()
    assert np.abs(dg - dref).max() / np.abs(dref).max() < 3e-6


def test_radial_table_spacing_override_and_knot_continuity():
    p = SMALL_PROFILES["p16_2_0"]
    blob = make_blob(p, seed=6)
    m = binding.Model(blob, table_dx=0.01)
    assert m.query()["table_rows"] == 600
    # value and slope are continuous across knots (two-point Hermite)
    k = np.arange(1, 599) * 0.01
    gl, dl = m.eval_radial_table(k - 1e-12)
    gr, dr = m.eval_radial_table(k + 1e-12)
    assert np.abs(gl - gr).max() < 1e-6 * np.abs(gl).max()
    assert np.abs(dl - dr).max() < 1e-5 * np.abs(dl).max()


@pytest.mark.parametrize("name", ["p16_2_0", "p32_3_2"])
def test_pair_cache_matches_pair_modulation(name):
    p = SMALL_PROFILES[name]
    blob = make_blob(p, seed=7)
    m = binding.Model(blob)
    o = orc.Oracle(blob)
    gamma, beta, U = o.pair
    for a in range(p["T"]):
        for b in range(p["T"]):
            got = m.eval_pair_cache(a, b)
            assert np.abs(got[0] - gamma[a, b].numpy()).max() < 2e-7
            assert np.abs(got[1] - beta[a, b].numpy()).max() < 2e-7 * max(1.0, beta.abs().max().item())
            for q in range(p["R"]):
                assert np.abs(got[2 + q] - U[a, b, :, q].numpy()).max() < 2e-7
