"""The allocation-free kinetic-energy entry point against the regular path.

Some callers of this library run where device allocation is off limits (an embedding
application that owns all GPU memory, a loop that must not trigger allocator-side
synchronisation).  umlmd_kinetic_energy_static serves them: no handle, no cudaMalloc, its
scratch is a fixed array inside the library.  The regular path (umlmd_step reporting e_kin)
uses allocated workspace; both must give the same number, call after call, because the
fixed array is shared by all calls and keeps whatever the previous call left in it.

This file is collected last on purpose: if it fails, every other test has already run.
"""

import ctypes

import numpy as np
import pytest
import torch

from workloads import CONFIGS, make_system, workload_blob

pytestmark = pytest.mark.gpu


def test_static_kinetic_energy_matches_step_twice_in_a_row():
    from paper_2608_19041_b200 import binding

    name = "cfg2_cu4000"
    cfg = CONFIGS[name]
    s = make_system(cfg["system"], cfg["md"])
    m = binding.Model(workload_blob(name))
    pos = torch.as_tensor(s["pos"], dtype=torch.float64).cuda().contiguous()
    vel = torch.as_tensor(s["vel"], dtype=torch.float64).cuda().contiguous()
    types = torch.as_tensor(s["types"], dtype=torch.int32).cuda().contiguous()
    m.build_neighbors(pos, types, s["cell"], s["pbc"], cfg["md"]["skin"])
    m.set_md_state(pos, vel, s["masses"])

    lib = binding.lib()
    masses = torch.as_tensor(s["masses"], dtype=torch.float64).cuda().contiguous()
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

    def static_ke(v):
        rc = lib.umlmd_kinetic_energy_static(v.shape[0], ctypes.c_void_p(v.data_ptr()),
                                             ctypes.c_void_p(types.data_ptr()), ctypes.c_void_p(masses.data_ptr()),
                                             ctypes.c_void_p(out.data_ptr()), stream)
        assert rc == 0, lib.umlmd_static_last_error().decode()
        torch.cuda.synchronize()
        return out.item()

    # first pair: initial velocities
    _, ke_ref = m.step(0, cfg["md"]["dt_ps"], 0)
    a = static_ke(vel)
    assert abs(a - ke_ref) <= 1e-12 * abs(ke_ref)
    # second pair: after a few steps the velocities (and the leftovers in the fixed array) differ
    _, ke_ref2 = m.step(5, cfg["md"]["dt_ps"], 0)
    b = static_ke(vel)
    assert abs(b - ke_ref2) <= 1e-12 * abs(ke_ref2)
    assert abs(ke_ref2 - ke_ref) > 1e-9 * abs(ke_ref)          # the two calls really saw different data
    # a smaller problem right after a larger one must not pick up stale partial sums
    n_small = 700
    c = static_ke(vel[:n_small].contiguous())
    mv = torch.as_tensor(s["masses"][s["types"][:n_small]], dtype=torch.float64).cuda()
    ref_small = 0.5 * (mv[:, None] * vel[:n_small] ** 2).sum().item() / 9648.53321
    assert abs(c - ref_small) <= 1e-12 * abs(ref_small)


def test_static_kinetic_energy_rejects_oversized_and_bad_input():
    from paper_2608_19041_b200 import binding

    lib = binding.lib()
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    dummy = ctypes.c_void_p(out.data_ptr())
    rc = lib.umlmd_kinetic_energy_static(4194304 + 1, dummy, dummy, dummy, dummy, None)
    assert rc == -9
    assert b"exceed the fixed scratch limit" in lib.umlmd_static_last_error()
    assert lib.umlmd_kinetic_energy_static(10, None, dummy, dummy, dummy, None) == -1
    assert lib.umlmd_kinetic_energy_static(0, None, None, None, dummy, None) == 0
    torch.cuda.synchronize()
    assert out.item() == 0.0
