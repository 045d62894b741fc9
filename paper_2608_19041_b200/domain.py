"""Spatial decomposition of one periodic system over the ranks of a process group.

The paper's distributed runs cut the simulation cell into regions, one per GPU: a rank owns the
atoms inside its region, holds ghost copies of every atom (periodic images included) within the
neighbor-list radius around it, receives the ghosts' coordinates before each evaluation and sends
the forces on them back to their owners afterwards.  Nothing learned crosses a boundary, because
the model has a single aggregation layer: an owned atom's energy depends only on the coordinates
and species of the atoms inside its cutoff sphere (Results, "Distributed scaling"; Supplementary
"Distributed V100 scaling").

This module is that scheme for orthorhombic cells and a grid of px x py x pz bricks, on top of the
library's ghost-atom evaluation (``Model.set_owned_atoms``): host logic and message plumbing only.
Per MD step a rank makes one forward exchange (positions of the atoms its neighbours hold as
ghosts), one evaluation, one reverse exchange (forces on its ghosts), and the velocity Verlet
updates of its own atoms (``binding.vv_update``); energies and the virial are summed over ranks on
request.  Every ``rebuild_every`` steps the atoms are wrapped and re-assigned to bricks, velocities
migrating with them, ghosts are searched again and the neighbor list of the brick is rebuilt.

The re-assignment gathers coordinates, velocities and species of all atoms on every rank (60 bytes
per atom per rebuild); the per-step exchanges move only the ghost layers.  Messages go through a
small communicator interface: ``TorchComm`` (torch.distributed, NCCL or gloo) in production,
``SerialComm`` for a single rank, and in-process stand-ins in the tests.
"""

import math

import numpy as np
import torch


class SerialComm:
    """Communicator of a single rank (periodic images of the rank's own atoms are still exchanged
    through it, so the one-rank path runs the same code)."""

    rank, world = 0, 1

    def all_gather(self, t):
        return [t]

    def all_to_all(self, send, recv_counts=None):
        return [send[0]]

    def all_reduce_sum(self, t):
        return t


class TorchComm:
    """Communicator over a torch.distributed process group (NCCL for CUDA tensors, gloo for CPU)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self._dist, self._group = dist, group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)

    def _counts(self, n, device):
        mine = torch.tensor([n], dtype=torch.int64, device=device)
        out = [torch.empty_like(mine) for _ in range(self.world)]
        self._dist.all_gather(out, mine, group=self._group)
        return [int(c.item()) for c in out]

    def all_gather(self, t):
        """Rows of every rank's tensor (first dimensions may differ), in rank order."""
        counts = self._counts(t.shape[0], t.device)
        cap = max(counts)
        padded = torch.zeros((cap,) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        padded[: t.shape[0]] = t
        out = [torch.empty_like(padded) for _ in range(self.world)]
        self._dist.all_gather(out, padded, group=self._group)
        return [o[:c] for o, c in zip(out, counts)]

    def all_to_all(self, send, recv_counts=None):
        """send[q] goes to rank q; returns what each rank sent here.  recv_counts: rows to expect
        from each rank, when the caller knows them (saves the exchange of counts)."""
        dev, dtype, tail = send[0].device, send[0].dtype, tuple(send[0].shape[1:])
        send_counts = [int(s.shape[0]) for s in send]
        if recv_counts is None:
            sc = torch.tensor(send_counts, dtype=torch.int64, device=dev)
            rc = torch.empty_like(sc)
            self._dist.all_to_all_single(rc, sc, group=self._group)
            recv_counts = [int(c) for c in rc.tolist()]
        width = int(np.prod(tail)) if tail else 1
        sbuf = torch.cat([s.reshape(-1) for s in send]) if sum(send_counts) else torch.empty(0, dtype=dtype, device=dev)
        rbuf = torch.empty(sum(recv_counts) * width, dtype=dtype, device=dev)
        self._dist.all_to_all_single(rbuf, sbuf, [c * width for c in recv_counts], [c * width for c in send_counts],
                                     group=self._group)
        out, o = [], 0
        for c in recv_counts:
            out.append(rbuf[o:o + c * width].reshape((c,) + tail))
            o += c * width
        return out

    def all_reduce_sum(self, t):
        self._dist.all_reduce(t, group=self._group)
        return t


def brick_grid(world):
    """(px, py, pz) with px * py * pz = world, as close to a cube as the factors allow."""
    best = (world, 1, 1)
    for px in range(1, world + 1):
        if world % px:
            continue
        for py in range(1, world // px + 1):
            if (world // px) % py:
                continue
            pz = world // px // py
            cand = tuple(sorted((px, py, pz), reverse=True))
            if max(cand) - min(cand) < max(best) - min(best):
                best = cand
    return best


class Domain:
    """One rank's brick of a periodic orthorhombic system and its ghosts.

    model     binding.Model (or an object with set_owned_atoms / build_neighbors / compute)
    comm      communicator (rank, world, all_gather, all_to_all, all_reduce_sum)
    lengths   cell edge lengths (3,), Angstrom
    grid      (px, py, pz) bricks, px * py * pz == comm.world
    rc, skin  model cutoff and list skin: ghosts are kept within rc + skin of the brick
    masses    mass by species, amu
    """

    def __init__(self, model, comm, lengths, grid, rc, skin, masses, device="cuda"):
        if int(np.prod(grid)) != comm.world:
            raise ValueError("grid does not match the number of ranks")
        self.model, self.comm, self.device = model, comm, torch.device(device)
        self.L = [float(x) for x in lengths]
        self.grid = tuple(int(g) for g in grid)
        self.rh, self.skin = float(rc) + float(skin), float(skin)
        px, py, pz = self.grid
        r = comm.rank
        self.brick = (r // (py * pz), (r // pz) % py, r % pz)
        self.lo = [self.L[k] * self.brick[k] / self.grid[k] for k in range(3)]
        self.hi = [self.L[k] * (self.brick[k] + 1) / self.grid[k] for k in range(3)]
        self.origin = torch.tensor([self.lo[k] - self.rh for k in range(3)], dtype=torch.float64, device=self.device)
        self.local_cell = np.diag([self.hi[k] - self.lo[k] + 2.0 * self.rh for k in range(3)])
        m = torch.as_tensor(np.asarray(masses, dtype=np.float64), device=self.device)
        self.mass, self.inv_mass = m, 1.0 / m
        self.n_total = 0
        self.steps_since_build = 0
        self.e_local = 0.0
        self.virial_local = np.zeros((3, 3))
        self.gid = self.pos = self.vel = self.types = self.force = None

    # ---- ownership -------------------------------------------------------------------
    def _owner_of(self, X):
        px, py, pz = self.grid
        b = []
        for k in range(3):
            bk = torch.floor(X[:, k] * (self.grid[k] / self.L[k])).to(torch.int64)
            b.append(bk.clamp_(0, self.grid[k] - 1))
        return (b[0] * py + b[1]) * pz + b[2]

    def distribute(self, pos, vel, types):
        """Start from the whole system, given identically on every rank: keep what this rank owns
        (global index = row of the given arrays), find ghosts, build the list."""
        X = torch.as_tensor(pos, dtype=torch.float64, device=self.device)
        X = X - torch.floor(X / X.new_tensor(self.L)) * X.new_tensor(self.L)
        V = torch.as_tensor(vel, dtype=torch.float64, device=self.device)
        T = torch.as_tensor(types, dtype=torch.int32, device=self.device)
        G = torch.arange(X.shape[0], dtype=torch.int64, device=self.device)
        self.n_total = int(X.shape[0])
        self._assign(G, X, V, T)

    def rebuild(self):
        """Wrap, gather every rank's atoms, re-assign them to bricks (velocities migrate with their
        atoms), search ghosts, rebuild this brick's neighbor list and the exchange plan."""
        Lt = self.pos.new_tensor(self.L)
        self.pos -= torch.floor(self.pos / Lt) * Lt
        G = torch.cat(self.comm.all_gather(self.gid))
        X = torch.cat(self.comm.all_gather(self.pos))
        V = torch.cat(self.comm.all_gather(self.vel))
        T = torch.cat(self.comm.all_gather(self.types))
        self._assign(G, X, V, T)

    def _assign(self, G, X, V, T):
        me, world, dev = self.comm.rank, self.comm.world, self.device
        N = int(G.shape[0])
        owner = self._owner_of(X)
        # own atoms of every rank in ascending global index: the same arrays on every rank, so that
        # a rank can name an atom of another rank by its position in that rank's arrays
        order = torch.argsort(owner * N + G)
        counts = torch.bincount(owner, minlength=world)
        starts = torch.cumsum(counts, 0) - counts
        own_index_sorted = torch.arange(N, dtype=torch.int64, device=dev) - starts[owner[order]]
        own_index = torch.empty(N, dtype=torch.int64, device=dev)
        own_index[order] = own_index_sorted
        s0, c0 = int(starts[me]), int(counts[me])
        mine = order[s0:s0 + c0]
        self.gid, self.pos, self.vel, self.types = G[mine].clone(), X[mine].clone(), V[mine].clone(), T[mine].clone()
        self.n_own = c0
        self.force = torch.zeros((c0, 3), dtype=torch.float64, device=dev)

        # ghosts: every image of every atom inside [lo - rh, hi + rh) on all three axes, except the
        # owned atoms themselves
        sel_rows, sel_shift = [], []
        reach = [int(math.ceil(self.rh / self.L[k])) + 1 for k in range(3)]
        all_rows = torch.arange(N, dtype=torch.int64, device=dev)

        def inside(rows, k, n):
            x = X[rows, k] + n * self.L[k]
            return rows[(x >= self.lo[k] - self.rh) & (x < self.hi[k] + self.rh)]

        for nx in range(-reach[0], reach[0] + 1):
            rx = inside(all_rows, 0, nx)
            if rx.numel() == 0:
                continue
            for ny in range(-reach[1], reach[1] + 1):
                ry = inside(rx, 1, ny)
                if ry.numel() == 0:
                    continue
                for nz in range(-reach[2], reach[2] + 1):
                    rz = inside(ry, 2, nz)
                    if nx == 0 and ny == 0 and nz == 0:
                        rz = rz[owner[rz] != me]
                    if rz.numel() == 0:
                        continue
                    sel_rows.append(rz)
                    sh = torch.tensor([nx * self.L[0], ny * self.L[1], nz * self.L[2]], dtype=torch.float64, device=dev)
                    sel_shift.append(sh.expand(rz.numel(), 3))
        if sel_rows:
            rows, shift = torch.cat(sel_rows), torch.cat(sel_shift)
        else:
            rows = torch.empty(0, dtype=torch.int64, device=dev)
            shift = torch.empty((0, 3), dtype=torch.float64, device=dev)
        # grouped by owner (ascending global index, then image, inside a group: a fixed order)
        key = owner[rows] * N + G[rows]
        go = torch.argsort(key, stable=True)
        rows, shift = rows[go], shift[go]
        self.ghost_shift = shift
        self.n_ghost = int(rows.numel())
        gcounts = torch.bincount(owner[rows], minlength=world).tolist()
        self.recv_counts = [int(c) for c in gcounts]
        requests, o = [], 0
        for q in range(world):
            requests.append(own_index[rows[o:o + gcounts[q]]].contiguous())
            o += gcounts[q]
        # tell every owner which of its atoms this rank holds as ghosts
        self.send_idx = [s.contiguous() for s in self.comm.all_to_all(requests)]
        self.send_counts = [int(s.numel()) for s in self.send_idx]
        self._plan_reverse()

        n_loc = self.n_own + self.n_ghost
        self.loc_pos = torch.empty((n_loc, 3), dtype=torch.float64, device=dev)
        self.loc_force = torch.zeros((n_loc, 3), dtype=torch.float64, device=dev)
        self.loc_types = torch.cat([self.types, T[rows]]).contiguous()
        self.loc_pos[:self.n_own] = self.pos - self.origin
        self.loc_pos[self.n_own:] = X[rows] + shift - self.origin
        self.model.set_owned_atoms(self.n_own)
        self.model.build_neighbors(self.loc_pos, self.loc_types, self.local_cell, (0, 0, 0), self.skin)
        self.steps_since_build = 0

    def _plan_reverse(self):
        """Fixed-order accumulation of the returned ghost forces: for every owned atom that some rank
        holds as a ghost, the rows of the concatenated receive buffer that belong to it, padded to
        the largest multiplicity with a row of zeros."""
        dev = self.device
        allidx = torch.cat(self.send_idx) if self.send_idx else torch.empty(0, dtype=torch.int64, device=dev)
        n_in = int(allidx.numel())
        self.n_incoming = n_in
        if n_in == 0:
            self.rev_atoms = torch.empty(0, dtype=torch.int64, device=dev)
            self.rev_rows = torch.empty((0, 1), dtype=torch.int64, device=dev)
            return
        order = torch.argsort(allidx, stable=True)
        sorted_idx = allidx[order]
        atoms, mult = torch.unique_consecutive(sorted_idx, return_counts=True)
        width = int(mult.max())
        first = torch.cumsum(mult, 0) - mult
        slot = torch.arange(n_in, dtype=torch.int64, device=dev) - torch.repeat_interleave(first, mult)
        rows = torch.full((atoms.numel(), width), n_in, dtype=torch.int64, device=dev)     # n_in = the zero row
        rows[torch.repeat_interleave(torch.arange(atoms.numel(), device=dev), mult), slot] = order
        self.rev_atoms, self.rev_rows = atoms, rows

    # ---- per evaluation ----------------------------------------------------------------
    def forward(self):
        """Ghost coordinates from their owners."""
        send = [self.pos[idx] for idx in self.send_idx]
        recv = self.comm.all_to_all(send, self.recv_counts)
        self.loc_pos[:self.n_own] = self.pos - self.origin
        if self.n_ghost:
            self.loc_pos[self.n_own:] = torch.cat(recv) + self.ghost_shift - self.origin

    def evaluate(self):
        """Energy and virial share of this rank; forces on the owned atoms, ghost contributions of
        the other ranks included."""
        out = self.model.compute(self.loc_pos, forces=True, virial=True, out_forces=self.loc_force)
        self.e_local, self.virial_local = out["energy"], out["virial"]
        gf = self.loc_force[self.n_own:]
        send, o = [], 0
        for q in range(self.comm.world):
            send.append(gf[o:o + self.recv_counts[q]])
            o += self.recv_counts[q]
        recv = self.comm.all_to_all(send, self.send_counts)
        self.force.copy_(self.loc_force[:self.n_own])
        if self.n_incoming:
            buf = torch.cat(list(recv) + [torch.zeros((1, 3), dtype=torch.float64, device=self.device)])
            self.force[self.rev_atoms] += buf[self.rev_rows].sum(dim=1)
        return self.e_local

    def totals(self):
        """(potential energy, kinetic energy, virial [3,3]) of the whole system."""
        if self.device.type == "cuda":
            from . import binding
            ke = binding.kinetic_energy(self.vel, self.types, self.mass)
        else:           # host stand-in of the same sum (the CPU tests of the message plumbing)
            ke = 0.5 * (self.mass[self.types.long()] * (self.vel ** 2).sum(1)).sum().reshape(1) / 9648.533
        t = torch.cat([torch.tensor([self.e_local], dtype=torch.float64, device=self.device), ke.reshape(1),
                       torch.as_tensor(self.virial_local, dtype=torch.float64, device=self.device).reshape(9)])
        t = self.comm.all_reduce_sum(t).cpu().numpy()
        return float(t[0]), float(t[1]), t[2:].reshape(3, 3)

    # ---- molecular dynamics ------------------------------------------------------------
    def start(self):
        """Forces of the initial frame."""
        self.forward()
        self.evaluate()

    def step(self, nsteps, dt_ps, rebuild_every):
        """nsteps of velocity Verlet (NVE) on this rank's atoms; every rank calls it with the same
        arguments.  The closing half kick of a step is merged with the opening one of the next."""
        from . import binding
        for s in range(nsteps):
            binding.vv_update(self.pos, self.vel, self.force, self.types, self.inv_mass, dt_ps, 1 if s == 0 else 2, True)
            self.steps_since_build += 1
            if rebuild_every > 0 and self.steps_since_build >= rebuild_every:
                self.rebuild()
            self.forward()
            self.evaluate()
        if nsteps > 0:
            binding.vv_update(self.pos, self.vel, self.force, self.types, self.inv_mass, dt_ps, 1, False)

    def gather(self):
        """(pos, vel, force) of the whole system by global index, on every rank (for checks)."""
        G = torch.cat(self.comm.all_gather(self.gid))
        out = []
        for t in (self.pos, self.vel, self.force):
            full = torch.cat(self.comm.all_gather(t))
            res = torch.empty_like(full)
            res[G] = full
            out.append(res)
        return out
