"""Thin ctypes binding of libumlmd.so: argument marshalling only.

Every computation runs inside the library's CUDA kernels.  Importing this module loads the
shared library and fails loudly if it has not been built
(``python -m paper_2608_19041_b200.build``); there is no fallback path.
"""

import ctypes
import os

import numpy as np
import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libumlmd.so")

OK = 0
ERRORS = {
    -1: "INVALID_ARG", -2: "BAD_BLOB", -3: "UNSUPPORTED_PROFILE", -4: "UNSUPPORTED_CELL",
    -5: "NO_NEIGHBORS", -6: "STALE_NEIGHBORS", -7: "NONFINITE", -8: "CUDA", -9: "CAPACITY",
    -10: "NO_MD_STATE",
}

EXPORTS = [
    "umlmd_profile_widths", "umlmd_create", "umlmd_destroy", "umlmd_query", "umlmd_last_error",
    "umlmd_build_neighbors", "umlmd_get_neighbors", "umlmd_compute", "umlmd_set_md_state", "umlmd_step",
    "umlmd_step_nvt", "umlmd_atom_virial",
    "umlmd_get_intermediates", "umlmd_eval_radial_table", "umlmd_eval_pair_cache", "umlmd_set_profiling",
    "umlmd_get_profile", "umlmd_profile_class_name", "umlmd_kinetic_energy_static", "umlmd_static_last_error",
    "umlmd_probe_fma_peak", "umlmd_get_neighbor_rows", "umlmd_workspace_bytes", "umlmd_get_nvt_state", "umlmd_set_nvt_state",
    "umlmd_compute_batch", "umlmd_set_owned_atoms", "umlmd_vv_update",
]


class UmlmdError(RuntimeError):
    def __init__(self, code, message):
        super().__init__(f"{ERRORS.get(code, code)}: {message}")
        self.code = code


class Options(ctypes.Structure):
    _fields_ = [("struct_bytes", ctypes.c_uint32), ("table_dx", ctypes.c_double),
                ("node_tile", ctypes.c_int32), ("mlp_path", ctypes.c_int32), ("pair_table_mb", ctypes.c_int32),
                ("gemm_spin_limit", ctypes.c_int32), ("fault_skip_gemm_stage", ctypes.c_int32),
                ("launch_graphs", ctypes.c_int32)]


class Info(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("C0", "L", "R", "N_rbf", "n_hidden", "F", "T", "C1", "C2", "K1", "K2", "S", "D_out", "H",
                 "H_pair", "table_rows")] + \
               [("rc", ctypes.c_double), ("table_dx", ctypes.c_double), ("n_atoms", ctypes.c_int64),
                ("n_edges", ctypes.c_int64), ("device_bytes", ctypes.c_int64), ("kernel_launches", ctypes.c_int64),
                ("graph_replays", ctypes.c_int64)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


def load_library(path=_LIB_PATH):
    if not os.path.exists(path):
        raise ImportError(f"{path} not found: build it with `python -m paper_2608_19041_b200.build`")
    lib = ctypes.CDLL(path)
    vp, i64, i32, dbl = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_double
    lib.umlmd_profile_widths.argtypes = [i32, i32, i32, ctypes.POINTER(Info)]
    lib.umlmd_create.argtypes = [vp, ctypes.c_size_t, ctypes.POINTER(Options), vp, ctypes.POINTER(vp)]
    lib.umlmd_destroy.argtypes = [vp]
    lib.umlmd_query.argtypes = [vp, ctypes.POINTER(Info)]
    lib.umlmd_last_error.argtypes = [vp]
    lib.umlmd_last_error.restype = ctypes.c_char_p
    lib.umlmd_build_neighbors.argtypes = [vp, i64, vp, vp, ctypes.POINTER(dbl), ctypes.POINTER(ctypes.c_int), dbl]
    lib.umlmd_get_neighbors.argtypes = [vp, vp, vp, vp, i64, ctypes.POINTER(i64)]
    lib.umlmd_compute.argtypes = [vp, vp, ctypes.POINTER(dbl), vp, ctypes.POINTER(dbl), vp]
    lib.umlmd_set_md_state.argtypes = [vp, vp, vp, ctypes.POINTER(dbl)]
    lib.umlmd_step.argtypes = [vp, ctypes.c_int, dbl, ctypes.c_int, ctypes.POINTER(dbl), ctypes.POINTER(dbl)]
    lib.umlmd_step_nvt.argtypes = [vp, ctypes.c_int, dbl, ctypes.c_int, dbl, dbl, ctypes.POINTER(dbl), ctypes.POINTER(dbl),
                                   ctypes.POINTER(dbl)]
    lib.umlmd_atom_virial.argtypes = [vp, vp]
    lib.umlmd_get_intermediates.argtypes = [vp, vp, vp]
    lib.umlmd_eval_radial_table.argtypes = [vp, i64, ctypes.POINTER(dbl), ctypes.POINTER(dbl), ctypes.POINTER(dbl)]
    lib.umlmd_eval_pair_cache.argtypes = [vp, i32, i32, ctypes.POINTER(dbl)]
    lib.umlmd_set_profiling.argtypes = [vp, ctypes.c_int]
    lib.umlmd_get_profile.argtypes = [vp, i32, ctypes.POINTER(dbl), ctypes.POINTER(i64), ctypes.POINTER(i32)]
    lib.umlmd_profile_class_name.argtypes = [i32]
    lib.umlmd_profile_class_name.restype = ctypes.c_char_p
    lib.umlmd_kinetic_energy_static.argtypes = [i64, vp, vp, vp, vp, vp]
    lib.umlmd_get_neighbor_rows.argtypes = [vp, i64, i64, vp, vp, vp, i64, ctypes.POINTER(i64)]
    lib.umlmd_compute_batch.argtypes = [vp, i32, ctypes.POINTER(i64), vp, vp, ctypes.POINTER(dbl), ctypes.POINTER(ctypes.c_int),
                                        ctypes.POINTER(dbl), vp, ctypes.POINTER(dbl), vp]
    lib.umlmd_workspace_bytes.argtypes = [vp, i64, i64, ctypes.POINTER(i64)]
    lib.umlmd_get_nvt_state.argtypes = [vp, ctypes.POINTER(dbl)]
    lib.umlmd_set_nvt_state.argtypes = [vp, ctypes.POINTER(dbl)]
    lib.umlmd_probe_fma_peak.argtypes = [ctypes.POINTER(dbl), vp]
    lib.umlmd_set_owned_atoms.argtypes = [vp, i64]
    lib.umlmd_vv_update.argtypes = [i64, vp, vp, vp, vp, vp, dbl, i32, i32, vp]
    lib.umlmd_static_last_error.argtypes = []
    lib.umlmd_static_last_error.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("umlmd_last_error", "umlmd_profile_class_name", "umlmd_static_last_error"):
            getattr(lib, name).restype = ctypes.c_int
    return lib


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = load_library()
    return _lib


def profile_widths(C0, L, R=0):
    info = Info()
    rc = lib().umlmd_profile_widths(C0, L, R, ctypes.byref(info))
    if rc != OK:
        raise UmlmdError(rc, f"unsupported profile ({C0}, {L}, {R})")
    return {k: v for k, v in info.as_dict().items() if k in
            ("C1", "C2", "K1", "K2", "S", "D_out", "H", "H_pair")}


def _stream_ptr(stream):
    st = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(st.cuda_stream)


def vv_update(pos, vel, force, types, inv_mass, dt_ps, half_kicks, drift, stream=None):
    """One piece of a velocity Verlet step on caller-owned CUDA arrays (umlmd_vv_update):
    half_kicks half kicks, then a drift if asked; inv_mass = 1/mass by species (CUDA, float64)."""
    _check_dev(vel, torch.float64, "vel")
    _check_dev(types, torch.int32, "types")
    _check_dev(inv_mass, torch.float64, "inv_mass")
    if drift:
        _check_dev(pos, torch.float64, "pos")
    if half_kicks:
        _check_dev(force, torch.float64, "force")
    rc = lib().umlmd_vv_update(vel.shape[0], _ptr(pos), _ptr(vel), _ptr(force), _ptr(types), _ptr(inv_mass),
                               float(dt_ps), int(half_kicks), int(bool(drift)), _stream_ptr(stream))
    if rc != OK:
        raise UmlmdError(rc, "umlmd_vv_update failed")


def kinetic_energy(vel, types, mass, out=None, stream=None):
    """Kinetic energy in eV of caller-owned CUDA arrays (umlmd_kinetic_energy_static): returns a
    one-element CUDA tensor; mass = mass by species (CUDA, float64)."""
    _check_dev(vel, torch.float64, "vel")
    _check_dev(types, torch.int32, "types")
    _check_dev(mass, torch.float64, "mass")
    out = out if out is not None else torch.zeros(1, dtype=torch.float64, device="cuda")
    rc = lib().umlmd_kinetic_energy_static(vel.shape[0], _ptr(vel), _ptr(types), _ptr(mass), _ptr(out), _stream_ptr(stream))
    if rc != OK:
        raise UmlmdError(rc, lib().umlmd_static_last_error().decode())
    return out


def probe_fma_peak(stream=None):
    """FP32 fused multiply-add rate of the current device in TFLOP/s (measured by the library)."""
    out = ctypes.c_double()
    st = stream if stream is not None else torch.cuda.current_stream()
    rc = lib().umlmd_probe_fma_peak(ctypes.byref(out), ctypes.c_void_p(st.cuda_stream))
    if rc != OK:
        raise UmlmdError(rc, "umlmd_probe_fma_peak failed")
    return out.value


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


def _check_dev(t, dtype, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA tensor of dtype {dtype}")


class Model:
    """A DPA4C model on the current CUDA device, created from a weight blob."""

    def __init__(self, blob, table_dx=0.0, node_tile=0, mlp_path=0, pair_table_mb=0, stream=None,
                 gemm_spin_limit=0, fault_skip_gemm_stage=0, launch_graphs=0):
        self._lib = lib()
        self._h = ctypes.c_void_p()
        opt = Options(ctypes.sizeof(Options), float(table_dx), int(node_tile), int(mlp_path), int(pair_table_mb),
                      int(gemm_spin_limit), int(fault_skip_gemm_stage), int(launch_graphs))
        # creation is host-only; a stream is only meaningful when a device is present
        self._stream = stream if stream is not None else (
            torch.cuda.current_stream() if torch.cuda.is_available() else None)
        stream_ptr = ctypes.c_void_p(self._stream.cuda_stream if self._stream is not None else 0)
        buf = (ctypes.c_char * len(blob)).from_buffer_copy(blob)
        rc = self._lib.umlmd_create(buf, len(blob), ctypes.byref(opt), stream_ptr,
                                    ctypes.byref(self._h))
        if rc != OK:
            self._h = ctypes.c_void_p()
            raise UmlmdError(rc, "umlmd_create failed (bad blob or unsupported profile)")
        self._keep = []
        self.n_atoms = 0

    def _raise(self, rc):
        raise UmlmdError(rc, self._lib.umlmd_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            self._lib.umlmd_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def query(self):
        info = Info()
        rc = self._lib.umlmd_query(self._h, ctypes.byref(info))
        if rc != OK:
            self._raise(rc)
        return info.as_dict()

    def build_neighbors(self, pos, types, cell, pbc=(1, 1, 1), skin=0.0):
        _check_dev(pos, torch.float64, "pos")
        _check_dev(types, torch.int32, "types")
        n = pos.shape[0]
        cell9 = (ctypes.c_double * 9)(*np.asarray(cell, dtype=np.float64).reshape(9))
        pbc3 = (ctypes.c_int * 3)(*[int(x) for x in pbc])
        rc = self._lib.umlmd_build_neighbors(self._h, n, _ptr(pos), _ptr(types), cell9, pbc3, float(skin))
        if rc != OK:
            self._raise(rc)
        self.n_atoms = n

    def get_neighbors(self):
        """(row_ptr [N+1], src [E], shift [E,3]) as CUDA tensors, caller numbering."""
        ne = ctypes.c_int64()
        rc = self._lib.umlmd_get_neighbors(self._h, None, None, None, 0, ctypes.byref(ne))
        if rc != OK:
            self._raise(rc)
        E = ne.value
        row_ptr = torch.empty(self.n_atoms + 1, dtype=torch.int32, device="cuda")
        src = torch.empty(max(E, 1), dtype=torch.int32, device="cuda")
        shift = torch.empty((max(E, 1), 3), dtype=torch.int8, device="cuda")
        rc = self._lib.umlmd_get_neighbors(self._h, _ptr(row_ptr), _ptr(src), _ptr(shift), max(E, 1), ctypes.byref(ne))
        if rc != OK:
            self._raise(rc)
        return row_ptr, src[:E], shift[:E]

    def get_neighbor_rows(self, first_row, n_rows):
        """(row_ptr [n_rows+1] int64, src [E], shift [E,3]) of the centres first_row .. first_row+n_rows-1."""
        ne = ctypes.c_int64()
        row_ptr = torch.empty(n_rows + 1, dtype=torch.int64, device="cuda")
        rc = self._lib.umlmd_get_neighbor_rows(self._h, int(first_row), int(n_rows), _ptr(row_ptr), None, None, 0,
                                               ctypes.byref(ne))
        if rc != OK:
            self._raise(rc)
        E = ne.value
        src = torch.empty(max(E, 1), dtype=torch.int32, device="cuda")
        shift = torch.empty((max(E, 1), 3), dtype=torch.int8, device="cuda")
        rc = self._lib.umlmd_get_neighbor_rows(self._h, int(first_row), int(n_rows), _ptr(row_ptr), _ptr(src), _ptr(shift),
                                               max(E, 1), ctypes.byref(ne))
        if rc != OK:
            self._raise(rc)
        return row_ptr, src[:E], shift[:E]

    def workspace_bytes(self, n_atoms, n_edges):
        out = ctypes.c_int64()
        rc = self._lib.umlmd_workspace_bytes(self._h, int(n_atoms), int(n_edges), ctypes.byref(out))
        if rc != OK:
            self._raise(rc)
        return out.value

    def get_nvt_state(self):
        st = (ctypes.c_double * 6)()
        rc = self._lib.umlmd_get_nvt_state(self._h, st)
        if rc != OK:
            self._raise(rc)
        return np.array(list(st), dtype=np.float64)

    def set_nvt_state(self, state):
        st = (ctypes.c_double * 6)(*[float(x) for x in state])
        rc = self._lib.umlmd_set_nvt_state(self._h, st)
        if rc != OK:
            self._raise(rc)

    def atom_virial(self):
        """[N, 3, 3] CUDA tensor: per-atom shares of the virial of the last evaluation with forces."""
        out = torch.empty((max(self.n_atoms, 1), 3, 3), dtype=torch.float64, device="cuda")
        rc = self._lib.umlmd_atom_virial(self._h, _ptr(out))
        if rc != OK:
            self._raise(rc)
        return out[:self.n_atoms]

    def compute(self, pos, forces=True, virial=True, atom_energy=False, out_forces=None, out_atom_energy=None):
        """Returns dict(energy=float, forces=CUDA tensor or None, virial=np [3,3] or None,
        atom_energy=CUDA tensor or None).  out_forces [n,3] / out_atom_energy [n] (float64, CUDA):
        buffers to write into instead of new ones (a repeated call with the same buffers is
        replayed as one graph launch for small systems)."""
        _check_dev(pos, torch.float64, "pos")
        n = self.n_atoms
        e = ctypes.c_double()
        if out_forces is not None:
            _check_dev(out_forces, torch.float64, "out_forces")
            if out_forces.numel() != 3 * n:
                raise ValueError("out_forces must hold n_atoms x 3 values")
        if out_atom_energy is not None:
            _check_dev(out_atom_energy, torch.float64, "out_atom_energy")
            if out_atom_energy.numel() != n:
                raise ValueError("out_atom_energy must hold n_atoms values")
        f = out_forces if out_forces is not None else (
            torch.empty((n, 3), dtype=torch.float64, device="cuda") if forces else None)
        ea = out_atom_energy if out_atom_energy is not None else (
            torch.empty(n, dtype=torch.float64, device="cuda") if atom_energy else None)
        vir = (ctypes.c_double * 9)() if virial else None
        rc = self._lib.umlmd_compute(self._h, _ptr(pos), ctypes.byref(e), _ptr(f), vir, _ptr(ea))
        if rc != OK:
            self._raise(rc)
        return dict(energy=e.value, forces=f, atom_energy=ea,
                    virial=np.array(list(vir), dtype=np.float64).reshape(3, 3) if virial else None)

    def compute_batch(self, frame_offsets, pos, types, cells, pbc=(1, 1, 1), forces=True, virial=True, atom_energy=False):
        """Energies [n_frames] (numpy), forces (CUDA tensor or None), virials [n_frames,3,3] (numpy or
        None) and atomic energies of concatenated frames; replaces the handle's neighbor list."""
        _check_dev(pos, torch.float64, "pos")
        _check_dev(types, torch.int32, "types")
        off = np.ascontiguousarray(frame_offsets, dtype=np.int64)
        nf = len(off) - 1
        n = int(off[-1])
        cl = np.ascontiguousarray(cells, dtype=np.float64).reshape(nf, 9)
        e = np.zeros(nf, dtype=np.float64)
        vir = np.zeros((nf, 9), dtype=np.float64) if virial else None
        f = torch.empty((n, 3), dtype=torch.float64, device="cuda") if forces else None
        ea = torch.empty(n, dtype=torch.float64, device="cuda") if atom_energy else None
        P = ctypes.POINTER(ctypes.c_double)
        pbc3 = (ctypes.c_int * 3)(*[int(x) for x in pbc])
        rc = self._lib.umlmd_compute_batch(self._h, nf, off.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), _ptr(pos),
                                           _ptr(types), cl.ctypes.data_as(P), pbc3, e.ctypes.data_as(P), _ptr(f),
                                           vir.ctypes.data_as(P) if virial else None, _ptr(ea))
        if rc != OK:
            self._raise(rc)
        self.n_atoms = 0
        return dict(energies=e, forces=f, atom_energy=ea, virials=vir.reshape(nf, 3, 3) if virial else None)

    def set_owned_atoms(self, n_owned):
        """Atoms with index >= n_owned are ghosts (neighbours only) from now on; negative: none."""
        rc = self._lib.umlmd_set_owned_atoms(self._h, int(n_owned))
        if rc != OK:
            self._raise(rc)

    def set_md_state(self, pos, vel, masses):
        _check_dev(pos, torch.float64, "pos")
        _check_dev(vel, torch.float64, "vel")
        m = np.asarray(masses, dtype=np.float64)
        arr = (ctypes.c_double * len(m))(*m)
        rc = self._lib.umlmd_set_md_state(self._h, _ptr(pos), _ptr(vel), arr)
        if rc != OK:
            self._raise(rc)
        self._keep = [pos, vel]

    def step(self, nsteps, dt_ps, rebuild_every=0):
        ep, ek = ctypes.c_double(), ctypes.c_double()
        rc = self._lib.umlmd_step(self._h, int(nsteps), float(dt_ps), int(rebuild_every), ctypes.byref(ep),
                                  ctypes.byref(ek))
        if rc != OK:
            self._raise(rc)
        return ep.value, ek.value

    def step_nvt(self, nsteps, dt_ps, temperature_K, t_damp_ps, rebuild_every=0):
        """(e_pot, e_kin, conserved energy) after nsteps of Nose-Hoover-chain NVT."""
        ep, ek, ec = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
        rc = self._lib.umlmd_step_nvt(self._h, int(nsteps), ctypes.c_double(dt_ps), int(rebuild_every),
                                      ctypes.c_double(temperature_K), ctypes.c_double(t_damp_ps), ctypes.byref(ep),
                                      ctypes.byref(ek), ctypes.byref(ec))
        if rc != OK:
            self._raise(rc)
        return ep.value, ek.value, ec.value

    def get_intermediates(self):
        q = self.query()
        state = torch.empty((self.n_atoms, q["S"] + 2), dtype=torch.float32, device="cuda")
        desc = torch.empty((self.n_atoms, q["D_out"]), dtype=torch.float32, device="cuda")
        rc = self._lib.umlmd_get_intermediates(self._h, _ptr(state), _ptr(desc))
        if rc != OK:
            self._raise(rc)
        return state, desc

    def set_profiling(self, enabled):
        rc = self._lib.umlmd_set_profiling(self._h, int(bool(enabled)))
        if rc != OK:
            self._raise(rc)

    def get_profile(self):
        """{class name: (milliseconds, launches)} since the previous call; resets the counters."""
        ms = (ctypes.c_double * 16)()
        ln = (ctypes.c_int64 * 16)()
        n = ctypes.c_int32()
        rc = self._lib.umlmd_get_profile(self._h, 16, ms, ln, ctypes.byref(n))
        if rc != OK:
            self._raise(rc)
        return {self._lib.umlmd_profile_class_name(k).decode(): (ms[k], ln[k]) for k in range(n.value)}

    def eval_pair_cache(self, type_i, type_j):
        q = self.query()
        out = np.empty(((2 + q["R"]), q["C0"]), dtype=np.float64)
        rc = self._lib.umlmd_eval_pair_cache(self._h, int(type_i), int(type_j),
                                             out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
        if rc != OK:
            self._raise(rc)
        return out

    def eval_radial_table(self, rho):
        rho = np.ascontiguousarray(rho, dtype=np.float64)
        q = self.query()
        nc = q["C0"] + q["R"]
        g = np.empty((len(rho), nc), dtype=np.float64)
        dg = np.empty((len(rho), nc), dtype=np.float64)
        P = ctypes.POINTER(ctypes.c_double)
        rc = self._lib.umlmd_eval_radial_table(self._h, len(rho), rho.ctypes.data_as(P), g.ctypes.data_as(P),
                                               dg.ctypes.data_as(P))
        if rc != OK:
            self._raise(rc)
        return g, dg
