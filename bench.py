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
pinned host memory and forces copied back every step, the list rebuilt at the workload's
cadence inside the timed region), "roofline" (dominant kernel class: algorithmic FLOPs or
bytes over its CUDA-event time, against the measured peaks), "kernels" (every class with
launches, time share and roofline fraction), "workloads" (short runs of the other four of the
five benchmark systems: rate, time per step, dominant class), "cpu_baseline" (the fp64 oracle
on a bounded sample, on this box's host cores) and "clocks".

Peaks: HBM and the tensor rate are the measured numbers of MEASURED_PEAKS.json (the MLP
multiplies half-precision operands, so its roof is the measured 16-bit tensor rate, sustained,
and its work is the algorithmic 2 flops per multiply-add: the three products per
multiply-add that carry single precision are this implementation's overhead, not work); the
FP32 rate is measured in this run by the library's FMA probe.
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
        # compulsory bytes of the MLP: the feature rows in, one energy out (forward); the gradient
        # rows out (backward).  Activations that travel between layers are the implementation's.
        "mlp_forward": dict(flops=mlp * n_atoms, bytes=n_atoms * (4 * D + 8), pipe="tensor"),
        "mlp_backward": dict(flops=mlp * n_atoms, bytes=n_atoms * 4 * D, pipe="tensor"),
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
    alu_peak = peaks["fp32_tflops"]
    tensor_peak = peaks["bf16_tflops_sustained"]          # half-precision operands: the 16-bit tensor rate
    t = ms * 1e-3
    if t <= 0:
        return None
    flops, byts = w["flops"] * evals, w["bytes"] * evals
    t_flop = flops / ((tensor_peak if w["pipe"] == "tensor" else alu_peak) * 1e12) if flops else 0.0
    t_hbm = byts / (peaks["hbm_gbs"] * 1e9)
    if flops and t_flop >= t_hbm:
        bound, ach, peak, unit = w["pipe"], flops / t / 1e12, (tensor_peak if w["pipe"] == "tensor" else alu_peak), "TFLOP/s"
        src = peaks["source"] if w["pipe"] == "tensor" else peaks["fp32_source"]
    else:
        bound, ach, peak, unit, src = "hbm", byts / t / 1e9, peaks["hbm_gbs"], "GB/s", peaks["source"]
    return dict(kernel=name, bound=bound, achieved=round(ach, 3), peak=round(peak, 1), unit=unit,
                frac=round(ach / peak, 4), launches=int(launches), ms_total=round(ms, 3), traffic=None,
                peak_source=src)


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

class Workload:
    """One benchmark system on this rank's GPU: model, device state, and the timed loops."""

    def __init__(self, args, name, atoms=0, modes=None, nvt=False):
        import torch

        from paper_2608_19041_b200 import binding
        self.torch = torch
        self.args, self.base_name, self.nvt = args, name, nvt
        cfg = CONFIGS[name]
        self.cfg = cfg
        self.modes = modes
        self.p = workload_profile(name, modes)
        # a workload without an MD recipe is timed as repeated single evaluations (energy + forces +
        # virial of the same frame, list built once): velocities are zero and nothing moves
        self.static = cfg["md"] is None
        self.md = cfg["md"] or dict(steps=1, dt_ps=0.001, temperature=0.0, seed=1, rebuild_every=1 << 30, skin=0.0)
        desc = dict(cfg["system"])
        label = name
        if atoms:
            # a smaller box of the same recipe (density, exclusion radius, species mix): the size one
            # node tile of the full workload has, for profiler captures that must stay small
            if desc.get("kind") == "poisson_disk":
                desc["atoms"] = int(atoms)
            elif desc.get("kind") in ("fcc", "bcc", "diamond"):
                per_cell = {"fcc": 4, "bcc": 2, "diamond": 8}[desc["kind"]]
                desc["cells"] = max(1, round((atoms / per_cell) ** (1.0 / 3.0)))
            else:
                raise SystemExit("--atoms applies to the amorphous and the lattice workloads only")
            label = f"{label}[atoms={int(atoms)}]"
        if modes is not None:
            label = f"{label}[R={modes}]"
        self.label = label
        s = make_system(desc, None if self.static else self.md)
        self.s = s
        self.N = len(s["pos"])
        self.model = binding.Model(workload_blob(name, modes), mlp_path=args.mlp_path, node_tile=args.node_tile,
                                   pair_table_mb=args.pair_table_mb, table_dx=args.table_dx,
                                   launch_graphs=args.launch_graphs)
        self.pos = torch.as_tensor(s["pos"], dtype=torch.float64).cuda().contiguous()
        self.vel = None if self.static else torch.as_tensor(s["vel"], dtype=torch.float64).cuda().contiguous()
        self.types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
        self.forces = torch.empty((self.N, 3), dtype=torch.float64, device="cuda")     # result buffer of every evaluation
        self.skin, self.every, self.dt = self.md["skin"], self.md["rebuild_every"], self.md["dt_ps"]
        m = self.model
        m.build_neighbors(self.pos, self.types, s["cell"], s["pbc"], 0.0)
        self.e_rc = m.query()["n_edges"]
        m.build_neighbors(self.pos, self.types, s["cell"], s["pbc"], self.skin)
        self.e_list = m.query()["n_edges"]
        if not self.static:
            m.set_md_state(self.pos, self.vel, s["masses"])

    def run_steps(self, k):
        m = self.model
        if not self.static:
            if self.nvt:
                ep, ek, _ = m.step_nvt(k, self.dt, self.md["temperature"], 100.0 * self.dt, self.every)
                return ep, ek
            return m.step(k, self.dt, self.every)
        out = None
        for _ in range(k):
            out = m.compute(self.pos, forces=True, virial=True, out_forces=self.forces)
        return (out["energy"] if out else 0.0), 0.0

    def timed(self, steps, warmup, sync_all, sampler=None):
        """(ms, e_pot, e_kin, launches): exactly `steps` steps after `warmup`, CUDA events."""
        torch = self.torch
        self.run_steps(warmup)
        q0 = self.model.query()
        l0 = q0["kernel_launches"]
        sync_all()
        if sampler:
            sampler.start()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        e_pot, e_kin = self.run_steps(steps)
        ev1.record()
        sync_all()
        q1 = self.model.query()
        self.graph_replays = q1["graph_replays"] - q0["graph_replays"]     # of the timed steps
        return ev0.elapsed_time(ev1), e_pot, e_kin, q1["kernel_launches"] - l0

    def classes(self, steps, peaks):
        """Per-class CUDA-event times of `steps` more steps, with each class's roofline entry."""
        m = self.model
        m.get_profile()
        m.set_profiling(True)
        self.run_steps(steps)
        prof = m.get_profile()
        m.set_profiling(False)
        work = work_model(self.p, self.N, self.e_rc, self.e_list, one_species=len(np.unique(self.s["types"])) == 1)
        total_ms = sum(v[0] for v in prof.values()) or 1.0
        kernels = []
        for cname, (kms, kl) in prof.items():
            if kl == 0 or cname not in work:
                continue
            evals = steps if cname != "neighbor_build" else max(1, kl // 7)
            ent = roofline_entry(cname, kms, kl, evals, work, peaks)
            if ent:
                ent["share"] = round(kms / total_ms, 4)
                kernels.append(ent)
        kernels.sort(key=lambda k: -k["ms_total"])
        return kernels

    def e2e(self, steps, sync_all):
        """The same metric driven from host buffers through the public calls: every iteration
        uploads the positions from pinned host memory, evaluates energy, forces and virial, and
        downloads the forces; the neighbor list is rebuilt at the workload's cadence inside the
        timed region (the host owns the integrator here, so none runs on the device)."""
        torch = self.torch
        m, s, N = self.model, self.s, self.N
        every = self.every if self.every < (1 << 20) else 0
        k_e2e = 2 * every if every else max(1, min(steps, 10))
        host_pos = self.pos.cpu().pin_memory()
        host_f = torch.empty((N, 3), dtype=torch.float64).pin_memory()
        dpos = torch.empty_like(self.pos)
        dpos.copy_(host_pos)
        m.build_neighbors(dpos, self.types, s["cell"], s["pbc"], self.skin)
        m.compute(dpos, out_forces=self.forces)
        sync_all()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        builds = 0
        t0.record()
        for k in range(1, k_e2e + 1):
            dpos.copy_(host_pos, non_blocking=True)
            if every and k % every == 0:
                m.build_neighbors(dpos, self.types, s["cell"], s["pbc"], self.skin)
                builds += 1
            out = m.compute(dpos, forces=True, virial=True, out_forces=self.forces)
            host_f.copy_(out["forces"], non_blocking=True)
        t1.record()
        sync_all()
        return t0.elapsed_time(t1), k_e2e, builds

    def close(self):
        self.model.close()
        del self.pos, self.vel, self.types, self.forces
        self.torch.cuda.empty_cache()


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

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    peaks = measured_peaks()
    # FP32 roof: measured here by the library's FMA probe; the figure derived from unit counts and
    # the maximum clock (SMs x 128 lanes x 2 x clock) is kept beside it
    derived = SM_COUNT * FP32_LANES_PER_SM * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12
    try:
        peaks["fp32_tflops"], peaks["fp32_source"] = binding.probe_fma_peak(), "measured (FMA probe of this run)"
    except Exception:
        peaks["fp32_tflops"], peaks["fp32_source"] = derived, "derived (SMs x 128 lanes x 2 x max clock)"
    peaks["fp32_tflops_derived"] = derived

    modes = args.modes if args.modes >= 0 else None
    w = Workload(args, args.workload, atoms=args.atoms, modes=modes, nvt=args.nvt)
    N, name, cfg = w.N, w.label, w.cfg
    sampler = ClockSampler(local)
    ms, e_pot, e_kin, launches = w.timed(args.steps, args.warmup, sync_all, sampler)
    graph_replays = w.graph_replays
    clocks = sampler.stop()
    ms = max_over_ranks(ms, "cuda")
    value = job_rate(N * args.steps, ms, world)

    # ---- second pass with per-class events: where the time goes, roofline per class
    kernels = w.classes(args.steps, peaks)
    dom = dict(kernels[0]) if kernels else None
    if dom:
        tile = args.node_tile if args.node_tile > 0 else DEFAULT_NODE_TILE
        dom["traffic"] = load_traffic(args.workload, dom["kernel"], N / max(1, -(-N // tile)))
        if dom["bound"] == "alu" and clocks["sm_mhz"]:
            # the same fraction against the FP32 rate at the clock the sampler saw during the run
            at_clock = peaks["fp32_tflops"] * clocks["sm_mhz"] / peaks["sm_max_mhz"]
            dom["frac_at_sampled_clock"] = round(dom["achieved"] / at_clock, 4)
        dom["fp32_peak_derived"] = round(derived, 1)

    # ---- end to end from host buffers
    ms_e2e, k_e2e, builds = w.e2e(args.steps, sync_all)
    ms_e2e = max_over_ranks(ms_e2e, "cuda")
    e2e = dict(value=job_rate(N * k_e2e, ms_e2e, world), unit="atom-steps/s", h2d_bytes_per_step=N * 24,
               d2h_bytes_per_step=N * 24 + 80, steps=k_e2e, neighbor_builds=builds,
               note="host-driven loop: upload positions, evaluate, download forces; list rebuilt at the workload's cadence")
    static, md, p = w.static, w.md, w.p
    skin, every, dt = w.skin, w.every, w.dt
    e_rc, e_list = w.e_rc, w.e_list
    w.close()

    # ---- the other benchmark systems, short runs (rank 0 of a single-GPU run only)
    others = None
    if rank == 0 and world == 1 and not args.no_workloads and not args.atoms and modes is None:
        others = []
        for oname in FIVE:
            if oname == args.workload:
                continue
            ow = Workload(args, oname)
            k = OTHER_STEPS[oname]
            osamp = ClockSampler(local)
            oms, _, _, ol = ow.timed(k, max(3, args.warmup), sync_all, osamp)
            ocl = osamp.stop()
            ok = ow.classes(k, peaks)
            top = ok[0] if ok else None
            others.append(dict(workload=oname, n_atoms=ow.N, value=ow.N * k / (oms * 1e-3), unit="atom-steps/s",
                               steps=k, ms_per_step=oms / k, gpu_launches=int(ol), graph_replays=int(ow.graph_replays),
                               dominant=dict(kernel=top["kernel"], bound=top["bound"], frac=top["frac"],
                                             share=top["share"]) if top else None,
                               clocks=dict(sm_mhz=ocl["sm_mhz"], reasons=ocl["reasons"])))
            ow.close()

        # many small frames in one call: 64 copies of the 108-atom frame through umlmd_compute_batch
        # (list build included in every call), the answer to the launch-bound single evaluation above
        others.append(batched_frames(args, "cfg1_al108", 64, 50, sync_all))

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
                                mlp_path=args.mlp_path, launch_graphs=args.launch_graphs, pair_table_mb=args.pair_table_mb, table_dx=args.table_dx, parallelism="replicas" if world > 1 else "single",
                                **({"published": pub} if pub else {}),
                                cache="working set per step exceeds L2" if N >= 100000 else "fits in L2 (launch-bound)"),
                    e_pot_per_atom=e_pot / N, e_kin_per_atom=e_kin / N,
                    gpu_launches=int(launches), graph_replays=int(graph_replays), e2e=e2e, roofline=dom, kernels=kernels, workloads=others, cpu_baseline=cpu,
                    peaks=dict(hbm_gbs=peaks["hbm_gbs"], tensor_16bit_tflops_sustained=peaks["bf16_tflops_sustained"],
                               fp32_tflops=round(peaks["fp32_tflops"], 2), fp32_source=peaks["fp32_source"],
                               fp32_tflops_derived=round(derived, 1), source=peaks["source"]),
                    clocks=dict(sm_mhz=clocks["sm_mhz"], sm_max_mhz=clocks["sm_max_mhz"], reasons=clocks["reasons"],
                                samples=clocks["samples"]))
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_domain(args):
    """One system cut into bricks, one per rank (paper_2608_19041_b200/domain.py): per step a forward
    exchange of ghost coordinates, one evaluation per brick, a reverse exchange of ghost forces.
    Strong scaling: the system is fixed, `value` is its atoms x steps over the slowest rank's time.
    With one rank the brick is the whole cell and its ghosts are its own periodic images."""
    import torch
    import torch.distributed as dist

    from paper_2608_19041_b200 import binding
    from paper_2608_19041_b200.domain import Domain, SerialComm, TorchComm, brick_grid

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    comm = TorchComm() if world > 1 else SerialComm()

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    name = args.workload
    cfg = CONFIGS[name]
    if cfg["md"] is None:
        raise SystemExit("--domain needs a workload with an MD recipe")
    md = cfg["md"]
    desc = dict(cfg["system"])
    if args.atoms:
        if desc.get("kind") != "poisson_disk":
            raise SystemExit("--atoms with --domain applies to the amorphous workload only")
        desc["atoms"] = int(args.atoms)
    s = make_system(desc, md)                      # the same seeded system on every rank
    N = len(s["pos"])
    grid = brick_grid(world)
    model = binding.Model(workload_blob(name), mlp_path=args.mlp_path, node_tile=args.node_tile,
                          pair_table_mb=args.pair_table_mb, launch_graphs=args.launch_graphs)
    d = Domain(model, comm, np.diag(s["cell"]), grid, model.query()["rc"], md["skin"], s["masses"])
    d.distribute(s["pos"], s["vel"], s["types"])
    d.start()
    e_start = d.totals()
    d.step(args.warmup, md["dt_ps"], md["rebuild_every"])
    l0 = model.query()["kernel_launches"]
    sync_all()
    sampler = ClockSampler(local)
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    d.step(args.steps, md["dt_ps"], md["rebuild_every"])
    ev1.record()
    sync_all()
    clocks = sampler.stop()
    ms = max_over_ranks(ev0.elapsed_time(ev1), "cuda")
    launches = model.query()["kernel_launches"] - l0
    e_end = d.totals()
    counts = torch.tensor([d.n_own, d.n_ghost], dtype=torch.float64, device="cuda")
    counts = comm.all_reduce_sum(counts).tolist()
    if rank == 0:
        line = dict(metric="atom-steps/s (energy+forces+virial)", value=N * args.steps / (ms * 1e-3), unit="atom-steps/s",
                    n_gpus=world, steps=args.steps, warmup=args.warmup, ms_per_step=ms / args.steps, higher_is_better=True,
                    scaling="strong", vs_baseline=None, dtype="f32", data="synthetic",
                    config=dict(workload=name if not args.atoms else f"{name}[atoms={N}]", n_atoms=N,
                                parallelism=f"domain {grid[0]}x{grid[1]}x{grid[2]} (bricks with ghost atoms)",
                                ghosts_total=int(counts[1]), ghost_bytes_per_step=int(counts[1]) * 48,
                                dt_ps=md["dt_ps"], rebuild_every=md["rebuild_every"], skin=md["skin"], ensemble="nve",
                                cache="working set per step exceeds L2" if N >= 100000 else "fits in L2 (launch-bound)"),
                    e_total_per_atom_start=(e_start[0] + e_start[1]) / N, e_total_per_atom_end=(e_end[0] + e_end[1]) / N,
                    gpu_launches=int(launches), e2e=None, roofline=None, cpu_baseline=None,
                    clocks=dict(sm_mhz=clocks["sm_mhz"], sm_max_mhz=clocks["sm_max_mhz"], reasons=clocks["reasons"],
                                samples=clocks["samples"]))
        print(json.dumps(line))
    model.close()
    if world > 1:
        dist.destroy_process_group()


def batched_frames(args, name, n_frames, calls, sync_all):
    import torch

    from paper_2608_19041_b200 import binding
    s = make_system(CONFIGS[name]["system"])
    n = len(s["pos"])
    m = binding.Model(workload_blob(name), mlp_path=args.mlp_path, launch_graphs=args.launch_graphs, pair_table_mb=args.pair_table_mb)
    off = np.arange(n_frames + 1) * n
    pos = torch.as_tensor(np.tile(s["pos"], (n_frames, 1)), dtype=torch.float64).cuda().contiguous()
    types = torch.as_tensor(np.tile(s["types"], n_frames), dtype=torch.int32).cuda().contiguous()
    cells = np.tile(np.asarray(s["cell"], dtype=np.float64).reshape(1, 9), (n_frames, 1))
    for _ in range(5):
        m.compute_batch(off, pos, types, cells, s["pbc"])
    l0 = m.query()["kernel_launches"]
    sync_all()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(calls):
        m.compute_batch(off, pos, types, cells, s["pbc"])
    ev1.record()
    sync_all()
    ms = ev0.elapsed_time(ev1)
    launches = m.query()["kernel_launches"] - l0
    m.close()
    return dict(workload=f"{name} x{n_frames} frames per call (umlmd_compute_batch, list build included)", n_atoms=n * n_frames,
                value=n * n_frames * calls / (ms * 1e-3), unit="atom-steps/s", steps=calls, ms_per_step=ms / calls,
                gpu_launches=int(launches), dominant=None, clocks=None)


FIVE = ["cfg1_al108", "cfg2_cu4000", "cfg3_water32400", "cfg4_hea128k", "cfg5_amorphous1m"]
# timed steps of the short runs of the other systems (cfg1: single evaluations of one frame)
OTHER_STEPS = {"cfg1_al108": 200, "cfg2_cu4000": 200, "cfg3_water32400": 100, "cfg4_hea128k": 40, "cfg5_amorphous1m": 10}

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
    ap.add_argument("--launch-graphs", type=int, default=0, choices=[-1, 0, 1],
                    help="replay of repeated launch sequences as CUDA graphs: 0 = the library's rule (systems of at most 65536 atoms), 1 = always, -1 = never")
    ap.add_argument("--atoms", type=int, default=0, help="amorphous and lattice workloads: (about) this many atoms in a smaller box of the same recipe")
    ap.add_argument("--modes", type=int, default=-1, help="override the number R of shared radial modes of the workload's profile")
    ap.add_argument("--nvt", action="store_true", help="time the Nose-Hoover-chain NVT driver instead of NVE")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--domain", action="store_true",
                    help="cut the workload into one brick per rank (ghost-atom exchange each step) instead of running replicas")
    ap.add_argument("--no-workloads", action="store_true", help="skip the short runs of the other benchmark systems")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.domain:
        run_domain(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
