"""GPU tests of the boundary calls that are not the evaluation itself: the row-range export of the
neighbor list, the workspace estimate, the thermostat checkpoint, the give-up path of the
tensor-core GEMM's bounded waits, and the replay of repeated launch sequences as graphs."""

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


def _build(blob, s, skin=0.0, **kw):
    m = _binding().Model(blob, **kw)
    pos = _dev(s["pos"], torch.float64)
    types = _dev(s["types"], torch.int32)
    m.build_neighbors(pos, types, s["cell"], s["pbc"], skin)
    return m, pos


def test_neighbor_rows_by_range_equal_the_full_export():
    s = make_system(dict(kind="random_box", atoms=300, edges=(21.0, 22.5, 30.0), min_dist=1.5, seed=17, n_types=1,
                         masses=[1.0], shift=True))
    N = len(s["pos"])
    m, _ = _build(make_blob(SMALL_PROFILES["p8_2_0"], seed=1), s, skin=1.0)
    rp, src, shift = [t.cpu().numpy() for t in m.get_neighbors()]
    for first, n in [(0, N), (17, 23), (N - 5, 5), (40, 1), (100, 0)]:
        rp2, src2, shift2 = [t.cpu().numpy() for t in m.get_neighbor_rows(first, n)]
        assert rp2.dtype == np.int64 and rp2[0] == 0
        assert np.array_equal(rp2, rp[first:first + n + 1].astype(np.int64) - rp[first])
        a, b = rp[first], rp[first + n]
        assert np.array_equal(src2, src[a:b]) and np.array_equal(shift2, shift[a:b])
    # brute force for a few centres, through the range call alone
    pos = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    for c, ref in zip((0, 123, N - 1), orc.neighbor_rows(pos, s["cell"], s["pbc"], 7.0, centers=[0, 123, N - 1])):
        rp2, src2, shift2 = [t.cpu().numpy() for t in m.get_neighbor_rows(c, 1)]
        ent = np.concatenate([src2[:, None].astype(np.int64), shift2.astype(np.int64)], axis=1)
        assert np.array_equal(ent[np.lexsort((ent[:, 3], ent[:, 2], ent[:, 1], ent[:, 0]))], ref)
    # a buffer that is too small is reported, the offsets still come back
    B = _binding()
    import ctypes
    ne = ctypes.c_int64()
    rp3 = torch.empty(11, dtype=torch.int64, device="cuda")
    small_src = torch.empty(4, dtype=torch.int32, device="cuda")
    small_shift = torch.empty((4, 3), dtype=torch.int8, device="cuda")
    rc = m._lib.umlmd_get_neighbor_rows(m._h, 0, 10, B._ptr(rp3), B._ptr(small_src), B._ptr(small_shift), 4, ctypes.byref(ne))
    assert rc == -9 and ne.value == rp[10] and rp3[-1].item() == rp[10]
    with pytest.raises(B.UmlmdError):
        m.get_neighbor_rows(N - 3, 5)                      # range past the end
    m.close()


def test_workspace_estimate_covers_what_a_run_allocates():
    name = "cfg2_cu4000"
    cfg = CONFIGS[name]
    s = make_system(cfg["system"], cfg["md"])
    torch.cuda.synchronize()
    m = _binding().Model(workload_blob(name), pair_table_mb=-1)
    before = m.query()["device_bytes"]
    pos, vel = _dev(s["pos"], torch.float64), _dev(s["vel"], torch.float64)
    types = _dev(s["types"], torch.int32)
    m.build_neighbors(pos, types, s["cell"], s["pbc"], cfg["md"]["skin"])
    E = m.query()["n_edges"]
    est = m.workspace_bytes(len(s["pos"]), E)
    m.compute(pos)
    m.set_md_state(pos, vel, s["masses"])
    m.step_nvt(2, 0.001, 300.0, 0.1, 10)
    held = m.query()["device_bytes"] - before
    print(f"workspace of {name}: held {held / 2**20:.1f} MiB, estimate {est / 2**20:.1f} MiB")
    assert held <= est <= 1.15 * held + (4 << 20)
    m.close()


@pytest.mark.parametrize("variant", ["one_tile", "persistent", "cta_pairs"])
def test_expired_pipeline_wait_is_reported_and_the_handle_recovers(variant):
    # The diagnostic option leaves one operand stage of the first MLP layer unloaded; nothing sets
    # the barrier the MMA warp then waits on, the shortened wait runs out, the kernel finishes and
    # the call reports it.  The next evaluation on the same handle is a normal one.
    if variant == "one_tile":
        p = SMALL_PROFILES["p32_2_4"]
        s = make_system(dict(kind="random_box", atoms=150, edges=(12.5, 13.5, 14.0), min_dist=1.7, seed=31,
                             n_types=p["T"], masses=[1.0] * p["T"]))
        path = 3
    else:   # enough rows for the persistent kernel: more than half an item per SM
        p = SMALL_PROFILES["p8_2_0"]
        s = make_system(dict(kind="fcc", cells=18, a=4.05, jitter=0.05, seed=5, n_types=p["T"], masses=[1.0] * p["T"]))
        path = 2 if variant == "persistent" else 4
    blob = make_blob(p, seed=45, bias_scale=0.2, e_ref_scale=0.5)
    B = _binding()
    good, pos = _build(blob, s, mlp_path=path)
    ref = good.compute(pos, atom_energy=True)
    m, _ = _build(blob, s, mlp_path=path, gemm_spin_limit=20000, fault_skip_gemm_stage=2)
    with pytest.raises(B.UmlmdError) as e:
        m.compute(pos)
    assert e.value.code == -8 and "pipeline wait expired" in str(e.value)
    out = m.compute(pos, atom_energy=True)                 # the diagnostic is one shot
    assert out["energy"] == ref["energy"] and torch.equal(out["forces"], ref["forces"])
    good.close()
    m.close()


def test_thermostat_state_round_trip_continues_a_run_exactly():
    name = "cfg2_cu4000"
    cfg = CONFIGS[name]
    md = cfg["md"]
    s = make_system(cfg["system"], md)
    blob = workload_blob(name)
    T, damp, every = 300.0, 0.05, 10

    def start(p0, v0, chain=None):
        m = _binding().Model(blob)
        pos, vel = _dev(p0, torch.float64), _dev(v0, torch.float64)
        m.build_neighbors(pos, _dev(s["types"], torch.int32), s["cell"], s["pbc"], md["skin"])
        m.set_md_state(pos, vel, s["masses"])
        if chain is not None:
            m.set_nvt_state(chain)
        return m, pos, vel

    m, pos, vel = start(s["pos"], s["vel"])
    assert np.all(m.get_nvt_state() == 0.0)                 # at rest
    m.step_nvt(every, md["dt_ps"], T, damp, every)          # ends on a rebuild step
    chain = m.get_nvt_state()
    assert np.abs(chain).max() > 0
    p_mid, v_mid = pos.cpu().numpy().copy(), vel.cpu().numpy().copy()
    a = m.step_nvt(every, md["dt_ps"], T, damp, every)
    pa, va = pos.cpu().numpy(), vel.cpu().numpy()
    chain_a = m.get_nvt_state()
    m.close()
    m2, pos2, vel2 = start(p_mid, v_mid, chain)
    b = m2.step_nvt(every, md["dt_ps"], T, damp, every)
    assert np.array_equal(pos2.cpu().numpy(), pa) and np.array_equal(vel2.cpu().numpy(), va)
    assert a == b and np.array_equal(m2.get_nvt_state(), chain_a)
    m2.close()
    # without the chain state the continuation differs
    m3, pos3, vel3 = start(p_mid, v_mid)
    m3.step_nvt(every, md["dt_ps"], T, damp, every)
    assert not np.array_equal(vel3.cpu().numpy(), va)
    m3.close()


@pytest.mark.parametrize("own_stream", [False, True])
def test_replayed_launch_sequences_repeat_the_plain_launches_bit_for_bit(own_stream):
    # Two handles on the same system, one with graph replay switched off and one with it forced on.
    # Repeated evaluations into the same buffers (first plain, then recorded, then replayed) and an
    # MD run that crosses two list builds must agree in every bit, and both handles must count
    # the same kernel launches.  The caller's stream is the legacy default stream in one case (the
    # sequence is then recorded on a stream of the handle's own) and a stream of its own in the other.
    p = SMALL_PROFILES["p32_3_2"]
    s = make_system(dict(kind="fcc", cells=4, a=4.05, jitter=0.05, seed=9, n_types=p["T"], masses=[20.0] * p["T"]))
    blob = make_blob(p, seed=46, bias_scale=0.2, e_ref_scale=0.5)
    stream = torch.cuda.Stream() if own_stream else None
    with torch.cuda.stream(stream) if own_stream else torch.cuda.stream(torch.cuda.current_stream()):
        plain, pos_a = _build(blob, s, skin=1.0, launch_graphs=-1, stream=stream)
        graph, pos_b = _build(blob, s, skin=1.0, launch_graphs=1, stream=stream)
        n = plain.n_atoms
        fa = torch.empty((n, 3), dtype=torch.float64, device="cuda")
        fb = torch.empty_like(fa)
        ea = torch.empty(n, dtype=torch.float64, device="cuda")
        eb = torch.empty_like(ea)
        gen = torch.Generator(device="cuda").manual_seed(3)
        for it in range(5):
            oa = plain.compute(pos_a, out_forces=fa, out_atom_energy=ea)
            ob = graph.compute(pos_b, out_forces=fb, out_atom_energy=eb)
            torch.cuda.synchronize()
            assert oa["energy"] == ob["energy"], it
            assert np.array_equal(oa["virial"], ob["virial"]), it
            assert torch.equal(fa, fb) and torch.equal(ea, eb), it
            d = 0.01 * torch.randn(pos_a.shape, dtype=torch.float64, device="cuda", generator=gen)
            pos_a += d                                         # same buffers, new contents
            pos_b += d
        assert plain.query()["kernel_launches"] == graph.query()["kernel_launches"]
        # an energy-only evaluation is a different sequence: recorded separately, same results
        for it in range(3):
            assert plain.compute(pos_a, forces=False, virial=False)["energy"] == \
                graph.compute(pos_b, forces=False, virial=False)["energy"]
        vel = 0.5 * torch.randn(pos_a.shape, dtype=torch.float64, device="cuda", generator=gen)
        va, vb = vel.clone(), vel.clone()
        plain.set_md_state(pos_a, va, [20.0] * p["T"])
        graph.set_md_state(pos_b, vb, [20.0] * p["T"])
        for chunk in (7, 1, 25):                               # 33 steps: builds at steps 10, 20, 30
            ra = plain.step(chunk, 0.001, rebuild_every=10)
            rb = graph.step(chunk, 0.001, rebuild_every=10)
            assert ra == rb
            torch.cuda.synchronize()
            assert torch.equal(pos_a, pos_b) and torch.equal(va, vb)
        assert plain.query()["kernel_launches"] == graph.query()["kernel_launches"]
        # 5 evaluations (one plain, four replayed), 3 energy-only (one plain), and of the 33 steps
        # the three that end a call, the three with a list build (each the first with its list) and
        # the first after the change of MD state run as plain launches
        assert plain.query()["graph_replays"] == 0 and graph.query()["graph_replays"] == 4 + 2 + (33 - 3 - 3 - 1)
        # the thermostatted driver replays its middle steps too
        r0 = graph.query()["graph_replays"]
        for chunk in (4, 19):
            ra = plain.step_nvt(chunk, 0.001, 300.0, 0.05, rebuild_every=10)
            rb = graph.step_nvt(chunk, 0.001, 300.0, 0.05, rebuild_every=10)
            assert ra == rb
            torch.cuda.synchronize()
            assert torch.equal(pos_a, pos_b) and torch.equal(va, vb)
        assert np.array_equal(plain.get_nvt_state(), graph.get_nvt_state())
        assert graph.query()["graph_replays"] > r0 + 10
        assert plain.query()["kernel_launches"] == graph.query()["kernel_launches"]
    plain.close()
    graph.close()
