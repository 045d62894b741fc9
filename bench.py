#!/usr/bin/env python
"""Benchmark of the energy + force + virial MD step of the DPA4C potential on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one velocity-Verlet step through umlmd_step: integrate, (every tenth step)
rebuild the neighbor list, then the whole hot path -- edge featurisation and aggregation,
invariants, MLP forward and backward, invariant and edge backward, force / virial / energy
assembly.  The metric is atom-steps/s over exactly K timed steps, timed on the device with
CUDA events after W warm-up steps; with N > 1 each rank runs an independent replica of the
workload on its own GPU (the path has no exchange step on one node) and the value is the
sum over ranks divided by the slowest rank's time.

The default workload is the 1,000,000-atom amorphous mixture: it is the configuration
sized to load the whole GPU, and its working set (gigabytes per step) is far larger than
the 126 MB L2, so consecutive timed steps cannot serve each other from cache.  Smaller
workloads can be selected with --workload; they fit in L2 and are launch-bound.

The line also carries: "e2e" (same metric driven from host buffers: positions copied from
pinned host memory and forces copied back every step), "roofline" (dominant kernel class:
algorithmic FLOPs or bytes over its CUDA-event time, against the measured peaks),
"kernels" (every class with launches, time share and roofline fraction), "cpu_baseline"
(the fp64 oracle on a bounded sample, on this box's host cores) and "clocks".
"""

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import CONFIGS, make_system, workload_blob, workload_profile  # noqa: E402

DEFAULT_WORKLOAD = "cfg5_amorphous1m"
SM_COUNT = 148
FP32_LANES_PER_SM = 128


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                    sm_max_mhz=p.get("sm_max_mhz", 1965.0), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, sm_max_mhz=1965.0,
                source="fallback")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        try:
            os.unlink(self.file.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------ algorithmic work

def work_model(p, n_atoms, e_rc, e_list, one_species=False):
    """Algorithmic FLOPs (FMA = 2) and compulsory HBM bytes per evaluation, per kernel class.
    With one species the library tabulates the amplitude of that pair directly, so an edge costs
    the Horner evaluation of C0 channels and no modes or pair modulation: count that, not more."""
    C0, R, S, D, F, NH, C1 = p["C0"], p["R"], p["S"], p["D_out"], p["F"], p["n_hidden"], p["C1"]
    # per edge: cubic Horner of the table channels (6 flops a value, 4 more for its derivative),
    # pair modulation, the S+2 accumulations, envelope and harmonics
    fwd_edge = 6 * (C0 + R) + 2 * C0 * (1 + R) + 2 * S + C0 + C1 + 60
    bwd_edge = 10 * (C0 + R) + 4 * C0 * (1 + R) + 4 * S + 2 * C0 + 250
    if one_species:
        fwd_edge = 6 * C0 + 2 * S + C0 + C1 + 60
        bwd_edge = 10 * C0 + 4 * S + 2 * C0 + 250
    mlp = 2 * (D * F + (NH - 1) * F * F + F)
    return {
        "edge_forward": dict(flops=fwd_edge * e_rc, bytes=8 * e_list + n_atoms * (28 + 4 * (S + 2)), pipe="alu"),
        "edge_backward": dict(flops=bwd_edge * e_rc, bytes=(8 + 12) * e_list + n_atoms * (28 + 4 * (S + 2)), pipe="alu"),
        "mlp_forward": dict(flops=mlp * n_atoms, bytes=4 * n_atoms * (D + 2 * NH * F), pipe="tensor"),
        "mlp_backward": dict(flops=mlp * n_atoms, bytes=4 * n_atoms * (D + 2 * NH * F), pipe="tensor"),
        "invariants_forward": dict(flops=0, bytes=4 * n_atoms * (S + 2 + D), pipe="hbm"),
        "invariants_backward": dict(flops=0, bytes=4 * n_atoms * (2 * (S + 2) + D), pipe="hbm"),
        "force_assembly": dict(flops=0, bytes=e_list * (12 + 12 + 8) + n_atoms * 72, pipe="hbm"),
        "gather_positions": dict(flops=0, bytes=n_atoms * (24 * 3 + 16), pipe="hbm"),
        "energy_virial_reduce": dict(flops=0, bytes=n_atoms * 8, pipe="hbm"),
        "integrate": dict(flops=0, bytes=n_atoms * 2 * (24 * 5 + 4), pipe="hbm"),
        "neighbor_build": dict(flops=0, bytes=e_list * 16 + n_atoms * 200, pipe="hbm"),
    }


def roofline_entry(name, ms, launches, evals, work, peaks):
    """achieved = algorithmic work of `evals` evaluations / time; against the binding peak."""
    w = work[name]
    alu_peak = SM_COUNT * FP32_LANES_PER_SM * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12          # TFLOP/s
    tf32_peak = 0.5 * peaks["bf16_tflops_sustained"]
    t = ms * 1e-3
    if t <= 0:
        return None
    flops, byts = w["flops"] * evals, w["bytes"] * evals
    t_flop = flops / ((tf32_peak if w["pipe"] == "tensor" else alu_peak) * 1e12) if flops else 0.0
    t_hbm = byts / (peaks["hbm_gbs"] * 1e9)
    if flops and t_flop >= t_hbm:
        bound, ach, peak, unit = w["pipe"], flops / t / 1e12, (tf32_peak if w["pipe"] == "tensor" else alu_peak), "TFLOP/s"
    else:
        bound, ach, peak, unit = "hbm", byts / t / 1e9, peaks["hbm_gbs"], "GB/s"
    return dict(kernel=name, bound=bound, achieved=round(ach, 3), peak=round(peak, 1), unit=unit,
                frac=round(ach / peak, 4), launches=int(launches), ms_total=round(ms, 3), traffic=None)


# ------------------------------------------------------------------ CPU oracle leg

class OracleSampler:
    """The fp64 oracle on bounded samples of a workload: brute-force neighbor rows of the
    sampled atoms plus their energies and edge gradients.  Rate = atom evaluations / s."""

    def __init__(self, name, modes=None):
        import torch

        from oracle import dpa4c as orc
        self.orc = orc
        cfg = CONFIGS[name]
        self.name = name
        self.s = make_system(cfg["system"])
        self.o = orc.Oracle(workload_blob(name, modes))
        self.rc = cfg["profile"]["rc"]
        self.N = len(self.s["pos"])
        self.pos = orc.wrap_positions(self.s["pos"], self.s["cell"], self.s["pbc"])
        self.order = np.random.Generator(np.random.PCG64(99)).permutation(self.N)
        self.cores = torch.get_num_threads()

    def run(self, n, offset=0):
        centers = np.sort(self.order[np.arange(offset, offset + n) % self.N])
        t0 = time.perf_counter()
        rows = self.orc.neighbor_rows(self.pos, self.s["cell"], self.s["pbc"], self.rc, centers=centers)
        self.o.evaluate_rows(self.pos, self.s["types"], self.s["cell"], rows, centers, want_grad=True)
        return time.perf_counter() - t0

    def sized_for(self, seconds, probe=4):
        t = self.run(min(probe, self.N))
        return int(max(probe, min(self.N, probe * seconds / max(t, 1e-3))))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    smp = OracleSampler(args.workload, args.modes if args.modes >= 0 else None)
    total_steps = max(1, args.steps + args.warmup)
    n = smp.sized_for(min(20.0, 150.0 / total_steps))
    for w in range(args.warmup):
        smp.run(n, offset=w * n)
    t0 = time.perf_counter()
    for k in range(args.steps):
        smp.run(n, offset=(args.warmup + k) * n)
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    sample = f"{n} atoms of {args.workload} per step: brute-force neighbor rows + E_i and dE/dr_ij (fp64 oracle)"
    line = dict(impl="reference", metric="atom-steps/s (energy+forces+virial)", value=value, unit="atom-steps/s",
                n_gpus=args.gpus, steps=args.steps, warmup=args.warmup, ms_per_step=1e3 * dt / args.steps,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=args.workload, n_atoms=smp.N),
                cpu_baseline=dict(value=value, unit="atom-steps/s", cores=smp.cores, kind="oracle", sample=sample),
                e2e=dict(value=value, unit="atom-steps/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# ------------------------------------------------------------------ replicas on several ranks

def max_over_ranks(ms, device):
    """Time of the slowest rank (the job's time): all-reduce MAX over the default process group;
    the value itself for a single process."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_rate(units_per_rank, ms, world):
    """Whole-job rate of `world` independent replicas that each did `units_per_rank` units of work,
    over the slowest rank's time `ms` (milliseconds)."""
    return world * units_per_rank / (ms * 1e-3)


# ------------------------------------------------------------------ our arm

def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2608_19041_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    name = args.workload
    cfg = CONFIGS[name]
    modes = args.modes if args.modes >= 0 else None
    p = workload_profile(name, modes)
    # a workload without an MD recipe is timed as repeated single evaluations (energy + forces +
    # virial of the same frame, list built once): velocities are zero and nothing moves
    static = cfg["md"] is None
    md = cfg["md"] or dict(steps=1, dt_ps=0.001, temperature=0.0, seed=1, rebuild_every=1 << 30, skin=0.0)
    desc = dict(cfg["system"])
    if args.atoms:
        # a smaller box of the same recipe (density, exclusion radius, species mix): the size one
        # node tile of the full workload has, for profiler captures that must stay small
        if desc.get("kind") == "poisson_disk":
            desc["atoms"] = int(args.atoms)
        elif desc.get("kind") in ("fcc", "bcc", "diamond"):
            per_cell = {"fcc": 4, "bcc": 2, "diamond": 8}[desc["kind"]]
            desc["cells"] = max(1, round((args.atoms / per_cell) ** (1.0 / 3.0)))
        else:
            raise SystemExit("--atoms applies to the amorphous and the lattice workloads only")
        name = f"{name}[atoms={int(args.atoms)}]"
    s = make_system(desc, None if static else md)
    N = len(s["pos"])
    blob = workload_blob(args.workload, modes)
    if modes is not None:
        name = f"{name}[R={modes}]"
    model = binding.Model(blob, mlp_path=args.mlp_path, node_tile=args.node_tile, pair_table_mb=args.pair_table_mb,
                          table_dx=args.table_dx)
    pos0 = torch.as_tensor(s["pos"], dtype=torch.float64)
    pos = pos0.cuda().contiguous()
    vel = None if static else torch.as_tensor(s["vel"], dtype=torch.float64).cuda().contiguous()
    types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
    skin, every, dt = md["skin"], md["rebuild_every"], md["dt_ps"]

    model.build_neighbors(pos, types, s["cell"], s["pbc"], 0.0)
    e_rc = model.query()["n_edges"]
    model.build_neighbors(pos, types, s["cell"], s["pbc"], skin)
    e_list = model.query()["n_edges"]
    if not static:
        model.set_md_state(pos, vel, s["masses"])

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    def run_steps(k):
        if not static:
            if args.nvt:
                ep, ek, _ = model.step_nvt(k, dt, md["temperature"], 100.0 * dt, every)
                return ep, ek
            return model.step(k, dt, every)
        for _ in range(k):
            out = model.compute(pos, forces=True, virial=True)
        return out["energy"], 0.0

    run_steps(args.warmup)
    launches0 = model.query()["kernel_launches"]
    sampler = ClockSampler(local)
    sync_all()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    e_pot, e_kin = run_steps(args.steps)
    ev1.record()
    sync_all()
    clocks = sampler.stop()
    ms = ev0.elapsed_time(ev1)
    launches = model.query()["kernel_launches"] - launches0
    ms = max_over_ranks(ms, "cuda")
    value = job_rate(N * args.steps, ms, world)

    # ---- second pass with per-class events: where the time goes, roofline per class
    model.get_profile()
    model.set_profiling(True)
    run_steps(args.steps)
    prof = model.get_profile()
    model.set_profiling(False)
    peaks = measured_peaks()
    work = work_model(p, N, e_rc, e_list, one_species=len(np.unique(s["types"])) == 1)
    total_ms = sum(v[0] for v in prof.values()) or 1.0
    kernels = []
    for cname, (kms, kl) in prof.items():
        if kl == 0 or cname not in work:
            continue
        evals = args.steps if cname != "neighbor_build" else max(1, kl // 6)
        ent = roofline_entry(cname, kms, kl, evals, work, peaks)
        if ent:
            ent["share"] = round(kms / total_ms, 4)
            kernels.append(ent)
    kernels.sort(key=lambda k: -k["ms_total"])
    dom = dict(kernels[0]) if kernels else None
    if dom:
        dom["peak_source"] = peaks["source"]
        tile = args.node_tile if args.node_tile > 0 else DEFAULT_NODE_TILE
        dom["traffic"] = load_traffic(args.workload, dom["kernel"], N / max(1, -(-N // tile)))

    # ---- end to end from host buffers: upload positions, evaluate, download forces
    k_e2e = max(1, min(args.steps, 10))
    host_pos = pos.cpu().pin_memory()
    host_f = torch.empty((N, 3), dtype=torch.float64).pin_memory()
    dpos = torch.empty_like(pos)
    dpos.copy_(host_pos)
    model.build_neighbors(dpos, types, s["cell"], s["pbc"], skin)
    model.compute(dpos)
    sync_all()
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    for k in range(k_e2e):
        dpos.copy_(host_pos, non_blocking=True)
        if k % every == 0 and k > 0:
            model.build_neighbors(dpos, types, s["cell"], s["pbc"], skin)
        out = model.compute(dpos, forces=True, virial=True)
        host_f.copy_(out["forces"], non_blocking=True)
    t1.record()
    sync_all()
    ms_e2e = t0.elapsed_time(t1)
    ms_e2e = max_over_ranks(ms_e2e, "cuda")
    e2e = dict(value=job_rate(N * k_e2e, ms_e2e, world), unit="atom-steps/s", h2d_bytes_per_step=N * 24,
               d2h_bytes_per_step=N * 24 + 80, steps=k_e2e)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        smp = OracleSampler(args.workload, args.modes if args.modes >= 0 else None)
        n_s = smp.sized_for(args.cpu_seconds)
        t_s = smp.run(n_s, offset=8)
        cpu = dict(value=n_s / t_s, unit="atom-steps/s", cores=smp.cores, kind="oracle",
                   sample=f"{n_s} atoms of {name}: brute-force neighbor rows + E_i and dE/dr_ij, {t_s:.1f} s")
    # the paper's own rate exists only for its own workload (another machine, trained weights,
    # LAMMPS NVT steps): context for those workloads, null for the synthetic five
    pub = cfg.get("published") if (modes is None and not args.atoms) else None
    vs_baseline = value / pub["value"] if pub else None
    if rank == 0:
        line = dict(metric="atom-steps/s (energy+forces+virial)", value=value, unit="atom-steps/s", n_gpus=world,
                    steps=args.steps, warmup=args.warmup, ms_per_step=ms / args.steps, higher_is_better=True,
                    scaling="weak", vs_baseline=vs_baseline, dtype="f32", data="synthetic",
                    config=dict(workload=name, n_atoms=N, edges_within_rc=e_rc, edges_in_list=e_list,
                                profile={k: p[k] for k in ("C0", "L", "R", "N_rbf", "n_hidden", "F", "T")},
                                dt_ps=dt, rebuild_every=every, skin=skin,
                                ensemble="nvt (Nose-Hoover chain, period 100 dt)" if (args.nvt and not static) else "nve",
                                mlp_path=args.mlp_path, pair_table_mb=args.pair_table_mb, table_dx=args.table_dx, parallelism="replicas" if world > 1 else "single",
                                **({"published": pub} if pub else {}),
                                cache="working set per step exceeds L2" if N >= 100000 else "fits in L2 (launch-bound)"),
                    e_pot_per_atom=e_pot / N, e_kin_per_atom=e_kin / N,
                    gpu_launches=int(launches), e2e=e2e, roofline=dom, kernels=kernels, cpu_baseline=cpu,
                    clocks=dict(sm_mhz=clocks["sm_mhz"], sm_max_mhz=clocks["sm_max_mhz"], reasons=clocks["reasons"],
                                samples=clocks["samples"]))
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


CAPTURE_ATOMS = 131072          # size of the box the stored ncu capture ran on
DEFAULT_NODE_TILE = 524288       # the library's default workspace tile (atoms per launch of the tiled kernels)


def load_traffic(workload, kernel, atoms_per_launch):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of one kernel class on
    one workload, from the stored summary of an ncu capture: lines "workload class bytes" in
    profiles/dram_traffic_per_launch.txt hold the bytes of one launch over CAPTURE_ATOMS atoms of
    the same recipe; the traffic of these kernels is proportional to the atoms (and their edges)
    a launch covers, so it is scaled to the launch size of the timed run.  None when no capture
    is stored."""
    path = os.path.join(ROOT, "profiles", "dram_traffic_per_launch.txt")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        for ln in f:
            w = ln.split()
            if len(w) >= 3 and not ln.startswith("#") and w[0] == workload and w[1] == kernel:
                return float(w[2]) * atoms_per_launch / CAPTURE_ATOMS
    return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(CONFIGS))
    ap.add_argument("--mlp-path", type=int, default=0)
    ap.add_argument("--table-dx", type=float, default=0.0, help="radial table spacing in Angstrom (0 = the workload's)")
    ap.add_argument("--pair-table-mb", type=int, default=0,
                    help="memory for per-pair amplitude tables in MiB (0 = library default, negative = off)")
    ap.add_argument("--node-tile", type=int, default=0)
    ap.add_argument("--atoms", type=int, default=0, help="amorphous and lattice workloads: (about) this many atoms in a smaller box of the same recipe")
    ap.add_argument("--modes", type=int, default=-1, help="override the number R of shared radial modes of the workload's profile")
    ap.add_argument("--nvt", action="store_true", help="time the Nose-Hoover-chain NVT driver instead of NVE")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
