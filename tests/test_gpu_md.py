"""GPU tests of the velocity-Verlet NVE driver (umlmd_step)."""

import numpy as np
import pytest
import torch

from oracle import dpa4c as orc
from workloads import CONFIGS, SMALL_PROFILES, make_blob, make_system, workload_blob
from workloads.systems import EV_PER_AMU_IN_A2_PS2, KB_EV_PER_K

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2608_19041_b200 import binding
    return binding


def _setup(name):
    cfg = CONFIGS[name]
    s = make_system(cfg["system"], cfg["md"])
    blob = workload_blob(name)
    m = _binding().Model(blob)
    pos = torch.as_tensor(s["pos"], dtype=torch.float64).cuda().contiguous()
    vel = torch.as_tensor(s["vel"], dtype=torch.float64).cuda().contiguous()
    types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
    m.build_neighbors(pos, types, s["cell"], s["pbc"], cfg["md"]["skin"])
    m.set_md_state(pos, vel, s["masses"])
    return cfg, s, blob, m, pos, vel, types


def test_initial_velocities_have_the_requested_temperature():
    cfg, s, *_ = _setup("cfg2_cu4000")
    m = s["masses"][s["types"]]
    ke = 0.5 * (m[:, None] * s["vel"] ** 2).sum() / EV_PER_AMU_IN_A2_PS2
    T = 2 * ke / ((3 * len(m) - 3) * KB_EV_PER_K)
    assert abs(T - cfg["md"]["temperature"]) < 1e-9 * cfg["md"]["temperature"]
    assert np.abs((m[:, None] * s["vel"]).sum(0)).max() < 1e-9


def test_step_equals_hand_written_velocity_verlet():
    cfg, s, blob, m, pos, vel, types = _setup("cfg2_cu4000")
    dt = cfg["md"]["dt_ps"]
    # reference integration with the library's own forces, arithmetic in torch float64
    m2 = _binding().Model(blob)
    p2, v2 = pos.clone(), vel.clone()
    m2.build_neighbors(p2, types, s["cell"], s["pbc"], cfg["md"]["skin"])
    inv_m = torch.as_tensor(1.0 / s["masses"][s["types"]], dtype=torch.float64).cuda()[:, None]
    f = m2.compute(p2)["forces"]
    for _ in range(3):
        v2 += 0.5 * dt * EV_PER_AMU_IN_A2_PS2 * inv_m * f
        p2 += dt * v2
        out = m2.compute(p2)
        f = out["forces"]
        v2 += 0.5 * dt * EV_PER_AMU_IN_A2_PS2 * inv_m * f
    e_pot, e_kin = m.step(3, dt, 0)
    assert (pos - p2).abs().max().item() < 1e-12
    assert (vel - v2).abs().max().item() < 1e-10
    assert abs(e_pot - out["energy"]) < 1e-9 * max(1.0, abs(e_pot))
    ke = 0.5 * (torch.as_tensor(s["masses"][s["types"]]).cuda()[:, None] * v2 ** 2).sum().item() / EV_PER_AMU_IN_A2_PS2
    assert abs(e_kin - ke) < 1e-10 * ke


def test_nve_energy_drift_on_cu4000():
    cfg, s, blob, m, pos, vel, types = _setup("cfg2_cu4000")
    md = cfg["md"]
    N = len(s["pos"])
    chunk = 50
    t, e = [0.0], []
    ep, ek = m.step(0, md["dt_ps"], md["rebuild_every"])
    e.append((ep + ek) / N)
    for k in range(md["steps"] // chunk):
        ep, ek = m.step(chunk, md["dt_ps"], md["rebuild_every"])
        t.append((k + 1) * chunk * md["dt_ps"])
        e.append((ep + ek) / N)
    slope = np.polyfit(np.array(t), np.array(e), 1)[0]
    print(f"NVE drift {slope:.3e} eV/atom/ps over {t[-1]:.2f} ps; E range {min(e):.6f}..{max(e):.6f}; "
          f"final T = {2 * ek / ((3 * N - 3) * KB_EV_PER_K):.1f} K")
    assert abs(slope) <= 1e-5


def test_forces_on_a_later_md_frame_match_the_oracle():
    cfg, s, blob, m, pos, vel, types = _setup("cfg2_cu4000")
    md = cfg["md"]
    m.step(60, md["dt_ps"], md["rebuild_every"])
    frame = pos.cpu().numpy().copy()
    m2 = _binding().Model(blob)
    p2 = torch.as_tensor(frame).cuda().contiguous()
    m2.build_neighbors(p2, types, s["cell"], s["pbc"], 0.0)
    out = m2.compute(p2, atom_energy=True)
    F = out["forces"].cpu().numpy()
    Ei = out["atom_energy"].cpu().numpy()
    o = orc.Oracle(blob)
    e_scale, f_scale = np.abs(Ei).max(), np.abs(F).max()
    for k in (0, 1234, 3999):
        Fk, E_near = o.force_on(frame, s["types"], s["cell"], s["pbc"], k)
        assert np.abs(F[k] - Fk).max() <= min(1e-4, 2e-5 * f_scale + 2e-7)
        for a, ea in E_near.items():
            assert abs(Ei[a] - ea) <= 1e-5 * e_scale


def test_rebuild_keeps_results_continuous():
    # same trajectory with and without intermediate rebuilds (list covers the motion either way)
    p = SMALL_PROFILES["p16_2_0"]
    blob = make_blob(p, seed=60)
    s = make_system(dict(kind="random_box", atoms=80, edges=(13.0, 14.0, 15.0), min_dist=1.8, seed=61,
                         n_types=p["T"], masses=[20.0, 30.0, 40.0]),
                    dict(seed=62, temperature=300.0))
    res = []
    for every in (0, 3):
        m = _binding().Model(blob)
        pos = torch.as_tensor(s["pos"], dtype=torch.float64).cuda().contiguous()
        vel = torch.as_tensor(s["vel"], dtype=torch.float64).cuda().contiguous()
        types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
        m.build_neighbors(pos, types, s["cell"], s["pbc"], 1.0)
        m.set_md_state(pos, vel, s["masses"])
        ep, ek = m.step(12, 0.001, every)
        res.append((pos.clone(), ep, ek))
    assert (res[0][0] - res[1][0]).abs().max().item() < 1e-6
    assert abs(res[0][1] - res[1][1]) < 1e-6 * max(1.0, abs(res[0][1]))


def test_displacement_triggered_rebuild():
    # a thin skin that the motion outruns: a fixed list fails as stale, the displacement-triggered
    # mode (rebuild_every < 0) rebuilds when needed and follows the frequently rebuilt trajectory
    p = SMALL_PROFILES["p16_2_0"]
    blob = make_blob(p, seed=60)
    s = make_system(dict(kind="random_box", atoms=80, edges=(13.0, 14.0, 15.0), min_dist=1.8, seed=61,
                         n_types=p["T"], masses=[20.0, 30.0, 40.0]),
                    dict(seed=62, temperature=3000.0))
    res = {}
    for every in (0, -1, 1):
        m = _binding().Model(blob)
        pos = torch.as_tensor(s["pos"], dtype=torch.float64).cuda().contiguous()
        vel = torch.as_tensor(s["vel"], dtype=torch.float64).cuda().contiguous()
        types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
        m.build_neighbors(pos, types, s["cell"], s["pbc"], 0.2)
        m.set_md_state(pos, vel, s["masses"])
        if every == 0:
            with pytest.raises(_binding().UmlmdError) as e:
                m.step(60, 0.001, every)
            assert e.value.code == -6
        else:
            ep, ek = m.step(60, 0.001, every)
            res[every] = (pos.clone(), ep, ek, m.query()["kernel_launches"])
        m.close()
    assert (res[-1][0] - res[1][0]).abs().max().item() < 1e-6
    assert abs(res[-1][1] - res[1][1]) < 1e-6 * max(1.0, abs(res[1][1]))
    assert res[-1][3] < res[1][3]          # fewer builds than one per step

