"""GPU tests of the spatial decomposition (paper_2608_19041_b200/domain.py) on one GPU: the ranks of a
brick grid run as threads of this process, each with a library handle of its own, and exchange
their messages through an in-process communicator.  No kernel of one rank waits for a kernel of
another: the ranks meet on host barriers only.  The results must be those of the undivided system.
"""

import threading

import numpy as np
import pytest
import torch

from workloads import CONFIGS, SMALL_PROFILES, make_blob, make_system, workload_blob

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2608_19041_b200 import binding
    return binding


class _Shared:
    def __init__(self, world):
        self.box = [None] * world
        self.barrier = threading.Barrier(world, timeout=300)


class ThreadComm:
    """Ranks = threads of one process; a message is a reference handed over between two barriers."""

    def __init__(self, shared, rank, world):
        self.s, self.rank, self.world = shared, rank, world

    def _exchange(self, mine):
        self.s.box[self.rank] = mine
        self.s.barrier.wait()
        everything = list(self.s.box)
        self.s.barrier.wait()
        return everything

    def all_gather(self, t):
        return [x.clone() for x in self._exchange(t)]

    def all_to_all(self, send, recv_counts=None):
        recv = [per_rank[self.rank].clone() for per_rank in self._exchange(send)]
        if recv_counts is not None:
            assert [int(r.shape[0]) for r in recv] == list(recv_counts)
        return recv

    def all_reduce_sum(self, t):
        total = torch.stack(self._exchange(t)).sum(0)        # rank order: the same value on every rank
        return total


def _run_ranks(world, fn):
    shared = _Shared(world)
    out, errors = [None] * world, []

    def body(rank):
        try:
            out[rank] = fn(ThreadComm(shared, rank, world))
        except BaseException as e:          # noqa: BLE001 - reported below; the others must not wait forever
            errors.append((rank, e))
            shared.barrier.abort()

    threads = [threading.Thread(target=body, args=(r,)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    real = [e for e in errors if not isinstance(e[1], threading.BrokenBarrierError)]
    if real or errors:
        raise (real or errors)[0][1]
    return out


def _reference(blob, s, skin):
    B = _binding()
    m = B.Model(blob)
    pos = torch.as_tensor(s["pos"], dtype=torch.float64).cuda().contiguous()
    types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
    m.build_neighbors(pos, types, s["cell"], s["pbc"], skin)
    return m, pos, types


@pytest.mark.parametrize("grid", [(1, 1, 1), (2, 1, 1), (2, 2, 1), (2, 2, 2), (3, 1, 2)])
def test_bricks_with_ghosts_reproduce_the_undivided_evaluation(grid):
    from paper_2608_19041_b200.domain import Domain
    p = SMALL_PROFILES["p32_3_2"]
    # 864 atoms in a 24.3 A cube: bricks of 12 A and 8 A are narrower than the 7 A halo on each
    # side is wide, so a brick holds several images of the same atom
    s = make_system(dict(kind="fcc", cells=6, a=4.05, jitter=0.08, seed=12, n_types=p["T"], masses=[20.0] * p["T"]))
    blob = make_blob(p, seed=47, bias_scale=0.2, e_ref_scale=0.5)
    skin = 1.0
    ref_model, pos, types = _reference(blob, s, skin)
    ref = ref_model.compute(pos, atom_energy=True)
    lengths = np.diag(s["cell"])
    world = int(np.prod(grid))
    B = _binding()

    def rank_fn(comm):
        m = B.Model(blob)
        d = Domain(m, comm, lengths, grid, p["rc"], skin, s["masses"])
        d.distribute(s["pos"], np.zeros_like(s["pos"]), s["types"])
        d.start()
        e_pot, e_kin, virial = d.totals()
        _, _, force = d.gather()
        res = dict(e_pot=e_pot, virial=virial, force=force.clone(), n_own=d.n_own, n_ghost=d.n_ghost)
        m.close()
        return res

    out = _run_ranks(world, rank_fn)
    assert sum(o["n_own"] for o in out) == len(s["pos"])
    f_ref = ref["forces"]
    scale_f = f_ref.abs().max().item()
    print(f"grid {grid}: ghosts per rank {[o['n_ghost'] for o in out]}, |dE| {abs(out[0]['e_pot'] - ref['energy']):.2e} of "
          f"sum|E_i| {ref['atom_energy'].abs().sum().item():.3e}, max|dF| {(out[0]['force'] - f_ref).abs().max().item():.2e} of {scale_f:.2e}")
    for o in out:
        # fp32 sums run in another order in a brick's list than in the whole cell's
        assert abs(o["e_pot"] - ref["energy"]) <= 2e-6 * ref["atom_energy"].abs().sum().item()
        assert (o["force"] - f_ref).abs().max().item() <= 2e-5 * scale_f
        assert np.abs(o["virial"] - ref["virial"]).max() <= 2e-5 * max(1.0, np.abs(ref["virial"]).max())
    if world > 1:
        assert all(o["n_ghost"] > 0 for o in out)
    ref_model.close()


def test_a_brick_without_atoms_of_its_own_takes_part_in_the_exchange():
    # a slab with 17 A of vacuum along x, cut into three bricks along x: the third owns nothing and
    # holds only images of the slab's first layers; energies and forces are those of the whole cell
    from paper_2608_19041_b200.domain import Domain
    p = SMALL_PROFILES["p16_3_2"]
    s = make_system(dict(kind="fcc", cells=6, a=4.05, jitter=0.08, seed=13, n_types=p["T"], masses=[20.0] * p["T"]))
    s["cell"] = np.array(s["cell"], dtype=np.float64)
    s["cell"][0, 0] *= 1.7
    s["pos"] = np.array(s["pos"], dtype=np.float64)
    s["pos"][:, 0] += 1.0                               # keeps the jittered first layer from wrapping to the far side
    blob = make_blob(p, seed=49, bias_scale=0.2, e_ref_scale=0.5)
    ref_model, pos, types = _reference(blob, s, 1.0)
    ref = ref_model.compute(pos, atom_energy=True)
    grid = (3, 1, 1)
    B = _binding()

    def rank_fn(comm):
        m = B.Model(blob)
        d = Domain(m, comm, np.diag(s["cell"]), grid, p["rc"], 1.0, s["masses"])
        d.distribute(s["pos"], np.zeros_like(s["pos"]), s["types"])
        d.start()
        e_pot, _, virial = d.totals()
        _, _, force = d.gather()
        res = dict(e_pot=e_pot, virial=virial, force=force.clone(), n_own=d.n_own, n_ghost=d.n_ghost)
        m.close()
        return res

    out = _run_ranks(3, rank_fn)
    assert out[2]["n_own"] == 0 and out[2]["n_ghost"] > 0
    assert sum(o["n_own"] for o in out) == len(s["pos"])
    f_ref = ref["forces"]
    for o in out:
        assert abs(o["e_pot"] - ref["energy"]) <= 2e-6 * ref["atom_energy"].abs().sum().item()
        assert (o["force"] - f_ref).abs().max().item() <= 2e-5 * f_ref.abs().max().item()
        assert np.abs(o["virial"] - ref["virial"]).max() <= 2e-5 * max(1.0, np.abs(ref["virial"]).max())
    ref_model.close()


def test_exchange_over_an_nccl_process_group_of_one_rank():
    # the production communicator (torch.distributed over NCCL) with a single rank: the brick's
    # ghosts are its own periodic images and every exchange is a message to itself, through the
    # same all_to_all_single / all_gather / all_reduce calls that several GPUs would use
    import socket

    import torch.distributed as dist

    from paper_2608_19041_b200.domain import Domain, TorchComm
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    try:
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                                device_id=torch.device("cuda", torch.cuda.current_device()))
    except Exception as e:                              # no usable NCCL bootstrap on this machine
        pytest.skip(f"NCCL process group could not be created: {e}")
    try:
        name = "cfg2_cu4000"
        cfg = CONFIGS[name]
        desc = dict(cfg["system"])
        desc["cells"] = 6
        s = make_system(desc, cfg["md"])
        md = cfg["md"]
        blob = workload_blob(name)
        B = _binding()
        ref_model, pos, types = _reference(blob, s, md["skin"])
        vel = torch.as_tensor(s["vel"], dtype=torch.float64).cuda().contiguous()
        ref_model.set_md_state(pos, vel, s["masses"])
        e_pot_ref, e_kin_ref = ref_model.step(12, md["dt_ps"], md["rebuild_every"])
        m = B.Model(blob)
        d = Domain(m, TorchComm(), np.diag(s["cell"]), (1, 1, 1), ref_model.query()["rc"], md["skin"], s["masses"])
        d.distribute(s["pos"], s["vel"], s["types"])
        d.start()
        d.step(12, md["dt_ps"], md["rebuild_every"])
        e_pot, e_kin, _ = d.totals()
        p, v, _ = d.gather()
        L = torch.as_tensor(np.array(np.diag(s["cell"]))).cuda()
        dp = p - pos
        dp -= torch.round(dp / L) * L
        assert dp.abs().max().item() < 2e-6 and (v - vel).abs().max().item() < 2e-4
        assert abs(e_pot - e_pot_ref) < 2e-6 * len(s["pos"]) and abs(e_kin - e_kin_ref) < 2e-6 * len(s["pos"])
        assert d.n_ghost > 0
        m.close()
        ref_model.close()
    finally:
        dist.destroy_process_group()


def test_ghost_atoms_have_no_energy_and_owned_forces_need_their_return():
    # one handle, hand-made ghosts: the first half of a small cluster is owned, the rest are ghosts.
    # The energy is the owned atoms' share, and the forces are the derivative of that share
    # (checked against a central difference of the same call).
    p = SMALL_PROFILES["p16_3_2"]
    s = make_system(dict(kind="random_box", atoms=60, edges=(9.0, 9.5, 10.0), min_dist=1.7, seed=33,
                         n_types=p["T"], masses=[1.0] * p["T"], pbc=[0, 0, 0]))
    blob = make_blob(p, seed=48, bias_scale=0.2, e_ref_scale=0.5)
    B = _binding()
    m = B.Model(blob)
    pos = torch.as_tensor(s["pos"], dtype=torch.float64).cuda().contiguous()
    types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
    m.build_neighbors(pos, types, s["cell"], (0, 0, 0), 0.5)
    full = m.compute(pos, atom_energy=True)
    n_own = 25
    m.set_owned_atoms(n_own)
    with pytest.raises(B.UmlmdError):                    # the list has to be rebuilt: owned atoms come first inside
        m.compute(pos)
    m.build_neighbors(pos, types, s["cell"], (0, 0, 0), 0.5)
    part = m.compute(pos, atom_energy=True)
    # (the rows list their neighbours in another order now: fp32 sums differ in the last bits)
    assert (part["atom_energy"][:n_own] - full["atom_energy"][:n_own]).abs().max().item() < 2e-6 * full["atom_energy"].abs().max().item()
    assert part["atom_energy"][n_own:].abs().max().item() == 0.0
    assert abs(part["energy"] - part["atom_energy"].sum().item()) < 1e-9 * abs(full["energy"])
    h = 2e-3
    for k, ax in ((3, 0), (n_own + 4, 1), (n_own + 20, 2)):      # an owned atom and two ghosts
        pp, pm = pos.clone(), pos.clone()
        pp[k, ax] += h
        pm[k, ax] -= h
        fd = -(m.compute(pp, forces=False, virial=False)["energy"] - m.compute(pm, forces=False, virial=False)["energy"]) / (2 * h)
        assert abs(fd - part["forces"][k, ax].item()) < 5e-3 * part["forces"].abs().max().item()
    with pytest.raises(B.UmlmdError):
        vel = torch.zeros_like(pos)
        m.set_md_state(pos, vel, s["masses"])
        m.step(1, 0.001, 0)
    m.set_owned_atoms(-1)
    m.build_neighbors(pos, types, s["cell"], (0, 0, 0), 0.5)
    again = m.compute(pos, atom_energy=True)
    assert again["energy"] == full["energy"] and torch.equal(again["forces"], full["forces"])
    m.close()


def test_decomposed_md_follows_the_undivided_run():
    from paper_2608_19041_b200.domain import Domain
    name = "cfg2_cu4000"
    cfg = CONFIGS[name]
    desc = dict(cfg["system"])
    desc["cells"] = 7                                   # 1372 atoms, 25.3 A
    s = make_system(desc, cfg["md"])
    blob = workload_blob(name)
    md = cfg["md"]
    B = _binding()
    ref_model, pos, types = _reference(blob, s, md["skin"])
    vel = torch.as_tensor(s["vel"], dtype=torch.float64).cuda().contiguous()
    ref_model.set_md_state(pos, vel, s["masses"])
    steps = 25
    e_pot_ref, e_kin_ref = ref_model.step(steps, md["dt_ps"], md["rebuild_every"])
    grid = (2, 2, 1)
    lengths = np.diag(s["cell"])
    rc = ref_model.query()["rc"]

    def rank_fn(comm):
        m = B.Model(blob)
        d = Domain(m, comm, lengths, grid, rc, md["skin"], s["masses"])
        d.distribute(s["pos"], s["vel"], s["types"])
        d.start()
        e0 = d.totals()
        d.step(steps, md["dt_ps"], md["rebuild_every"])
        e1 = d.totals()
        p, v, _ = d.gather()
        m.close()
        return dict(e0=e0, e1=e1, pos=p.clone(), vel=v.clone())

    out = _run_ranks(4, rank_fn)
    L = torch.as_tensor(np.array(lengths)).cuda()
    print(f"decomposed MD, {steps} steps: max|dr| {((out[0]['pos'] - pos) - torch.round((out[0]['pos'] - pos) / L) * L).abs().max().item():.2e} A, "
          f"max|dv| {(out[0]['vel'] - vel).abs().max().item():.2e} A/ps, E drift {(out[0]['e1'][0] + out[0]['e1'][1]) - (out[0]['e0'][0] + out[0]['e0'][1]):.2e} eV")
    for o in out:
        dpos = o["pos"] - pos
        dpos -= torch.round(dpos / L) * L                # the decomposed run wraps at its rebuilds
        assert dpos.abs().max().item() < 2e-6
        assert (o["vel"] - vel).abs().max().item() < 2e-4
        e_pot, e_kin, _ = o["e1"]
        assert abs(e_pot - e_pot_ref) < 2e-6 * len(s["pos"]) and abs(e_kin - e_kin_ref) < 2e-6 * len(s["pos"])
        # and it conserves energy like the undivided run does
        assert abs((o["e1"][0] + o["e1"][1]) - (o["e0"][0] + o["e0"][1])) < 2e-5 * len(s["pos"])
    ref_model.close()
