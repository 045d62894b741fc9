"""The host side of the spatial decomposition (paper_2608_19041_b200/domain.py) as two gloo ranks on
CPU: ownership, periodic ghost images, the exchange plan, the forward exchange of coordinates, the
reverse exchange of ghost forces and the migration at a rebuild.  The model is a stand-in with the
library's ghost semantics (a smooth pair energy summed over the owned atoms' neighbours, forces on
every atom by automatic differentiation), so that the plumbing is checked against the undivided
periodic sum without a GPU."""

import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

RC, SKIN = 3.0, 0.6
LENGTHS = (11.0, 9.0, 10.0)


def _pair_energy(r2):
    x = r2 / (RC * RC)
    return torch.where(x < 1.0, (1.0 - x) ** 3, torch.zeros_like(x))


class PairModel:
    """Stand-in for binding.Model on CPU tensors: E = sum over owned i, all j != i of phi(r_ij)
    (open boundaries: periodic images arrive as ghost atoms), forces = -dE/dr of every atom."""

    def __init__(self):
        self.n_owned = -1

    def set_owned_atoms(self, n):
        self.n_owned = n

    def build_neighbors(self, pos, types, cell, pbc, skin):
        assert tuple(pbc) == (0, 0, 0)
        box = np.diag(np.asarray(cell)).copy()
        assert (pos >= 0).all() and (pos < torch.as_tensor(box)).all()      # ghosts and owned atoms inside the brick's box
        self.n = pos.shape[0]

    def compute(self, pos, forces=True, virial=True, out_forces=None):
        x = pos.detach().clone().requires_grad_(True)
        n_own = self.n if self.n_owned < 0 else self.n_owned
        d = x[None, :, :] - x[:n_own, None, :]
        r2 = (d * d).sum(-1)
        mask = ~torch.eye(self.n, dtype=torch.bool)[:n_own]
        e = (_pair_energy(r2) * mask).sum()
        e.backward()
        f = -x.grad
        if out_forces is not None:
            out_forces.copy_(f)
        return dict(energy=float(e.detach()), forces=out_forces if out_forces is not None else f, virial=np.zeros((3, 3)))


def _whole_system(pos):
    """Energy and forces of the undivided periodic system by brute force over images."""
    x = pos.clone().requires_grad_(True)
    L = torch.tensor(LENGTHS, dtype=torch.float64)
    e = x.new_zeros(())
    for nx in (-1, 0, 1):
        for ny in (-1, 0, 1):
            for nz in (-1, 0, 1):
                sh = torch.tensor([nx, ny, nz], dtype=torch.float64) * L
                d = x[None, :, :] + sh - x[:, None, :]
                r2 = (d * d).sum(-1)
                if nx == ny == nz == 0:
                    r2 = r2 + torch.eye(len(x), dtype=torch.float64) * 1e6
                e = e + _pair_energy(r2).sum()
    e.backward()
    return float(e.detach()), -x.grad


def _system(n=160, seed=5):
    g = torch.Generator().manual_seed(seed)
    pos = torch.rand((n, 3), dtype=torch.float64, generator=g) * torch.tensor(LENGTHS, dtype=torch.float64)
    types = (torch.arange(n) % 2).to(torch.int32)
    return pos, types


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, grid, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2608_19041_b200.domain import Domain, TorchComm
    pos, types = _system()
    d = Domain(PairModel(), TorchComm(), LENGTHS, grid, RC, SKIN, [1.0, 2.0], device="cpu")
    d.distribute(pos, torch.zeros_like(pos), types)
    d.start()
    e0, _, _ = d.totals()
    p0, _, f0 = d.gather()
    n_own0, n_ghost0 = d.n_own, d.n_ghost
    # move every atom a little (less than skin / 2): same lists, new coordinates through the exchange
    g = torch.Generator().manual_seed(17)
    shift_all = 0.2 * (torch.rand((len(pos), 3), dtype=torch.float64, generator=g) - 0.5)
    d.pos += shift_all[d.gid]
    d.forward()
    d.evaluate()
    e1, _, _ = d.totals()
    p1, _, f1 = d.gather()
    # a larger move that carries atoms across brick faces and cell faces, then a rebuild (migration)
    d.vel.copy_(d.gid[:, None].to(torch.float64) * torch.tensor([1.0, 10.0, 100.0], dtype=torch.float64))
    jump = 2.5 * (torch.rand((len(pos), 3), dtype=torch.float64, generator=g) - 0.5)
    d.pos += jump[d.gid]
    d.rebuild()
    d.forward()
    d.evaluate()
    e2, _, _ = d.totals()
    p2, v2, f2 = d.gather()
    out.put((rank, dict(e=(e0, e1, e2), p=[t.numpy().copy() for t in (p0, p1, p2)], f=[t.numpy().copy() for t in (f0, f1, f2)],
                        v2=v2.numpy().copy(), own=(n_own0, d.n_own), ghost=(n_ghost0, d.n_ghost))))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("grid", [(2, 1, 1), (1, 1, 2)])
def test_two_ranks_exchange_ghosts_and_reproduce_the_periodic_sum(grid):
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, grid, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=300) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    pos, _ = _system()
    L = torch.tensor(LENGTHS, dtype=torch.float64)
    n = len(pos)
    assert sum(res[r]["own"][0] for r in range(world)) == n and sum(res[r]["own"][1] for r in range(world)) == n
    assert all(res[r]["ghost"][0] > 0 for r in range(world))
    for r in range(world):
        for k in range(3):
            pk = torch.as_tensor(res[r]["p"][k])
            # (both sides sum phi over ordered pairs: centre i, any neighbour or image j)
            e_ref, f_ref = _whole_system(pk)
            assert res[r]["e"][k] == pytest.approx(e_ref, rel=1e-12)
            assert (torch.as_tensor(res[r]["f"][k]) - f_ref).abs().max().item() < 1e-11 * max(1.0, f_ref.abs().max().item())
        # both ranks hold the same gathered arrays
        assert np.array_equal(res[r]["p"][2], res[0]["p"][2]) and np.array_equal(res[r]["f"][2], res[0]["f"][2])
        # positions after the rebuild are the moved ones, wrapped into the cell; velocities moved with their atoms
        assert ((res[r]["p"][2] >= 0) & (res[r]["p"][2] < L.numpy())).all()
        expect_v = np.arange(n, dtype=np.float64)[:, None] * np.array([1.0, 10.0, 100.0])
        assert np.array_equal(res[r]["v2"], expect_v)


def test_one_rank_holds_its_own_periodic_images():
    from paper_2608_19041_b200.domain import Domain, SerialComm, brick_grid
    pos, types = _system(n=90, seed=8)
    d = Domain(PairModel(), SerialComm(), LENGTHS, (1, 1, 1), RC, SKIN, [1.0, 2.0], device="cpu")
    d.distribute(pos, torch.zeros_like(pos), types)
    d.start()
    e, _, _ = d.totals()
    p, _, f = d.gather()
    e_ref, f_ref = _whole_system(p)
    assert e == pytest.approx(e_ref, rel=1e-12)
    assert (f - f_ref).abs().max().item() < 1e-11 * max(1.0, f_ref.abs().max().item())
    assert d.n_own == 90 and d.n_ghost > 0
    assert brick_grid(8) == (2, 2, 2) and brick_grid(4) == (2, 2, 1) and brick_grid(6) == (3, 2, 1) and brick_grid(1) == (1, 1, 1)
