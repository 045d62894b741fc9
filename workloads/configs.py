"""Literal descriptions of the benchmark workloads and of a few small test profiles.

Every width below is written out as a number on purpose: this module is data,
not model code.  The oracle and the CUDA library each re-derive the widths from
(C0, L, R) with their own formulas and reject a blob whose size disagrees.

Vocabulary mapping used for the five workloads: "k layers" = k hidden layers of
the atomic-energy MLP (the model has exactly one aggregation layer), "channels"
= scalar channel width C0, "ranks 0..L" = maximum angular degree L.  Where a
workload does not say, N_rbf = 16, R = 0 and the MLP width is the one the paper
pairs with that C0 (256 for C0 = 64, 384 for C0 = 128).

A random-weight potential has no repulsive core and no reason to hold a crystal together:
at the plain Xavier output scale the 300 K copper crystal slides down the random energy
surface, releases half an eV per atom within 100 fs and melts to thousands of kelvin, and
atoms that pass close to each other feel angular forces that grow like 1/distance.  The
workloads that run molecular dynamics therefore fix the one free output-scale choice of the
otherwise unconstrained initialisation law, ``head_scale`` (a factor on the scalar head
w_head), so that the run is integrable at the stated time step: a negative sign makes the
jittered lattice a minimum instead of a maximum of the random surface (the copper crystal
then vibrates at ~230 K for the whole picosecond), and the magnitude is reduced where
light or densely packed atoms would otherwise be accelerated into each other.
"""


def _profile(C0, L, R, N_rbf, n_hidden, F, T, C1, C2, K1, K2, H, Hp, S, D_out,
             rc=6.0, table_dx=0.002):
    return dict(C0=C0, L=L, R=R, N_rbf=N_rbf, n_hidden=n_hidden, F=F, T=T, rc=rc,
                table_dx=table_dx, C1=C1, C2=C2, K1=K1, K2=K2, H=H, Hp=Hp, S=S,
                D_out=D_out)


CONFIGS = {
    # 108-atom FCC Al, one evaluation
    "cfg1_al108": dict(
        index=0,
        system=dict(kind="fcc", cells=3, a=4.05, jitter=0.05, seed=0,
                    n_types=1, masses=[26.982]),
        profile=_profile(32, 2, 0, 8, 1, 64, 1, C1=8, C2=4, K1=4, K2=2, H=88,
                         Hp=176, S=76, D_out=144),
        weights_seed=0, head_scale=1.0,
        md=None,
    ),
    # 4,000-atom FCC Cu, 1000 NVE steps
    "cfg2_cu4000": dict(
        index=1,
        system=dict(kind="fcc", cells=10, a=3.615, jitter=0.1, seed=1,
                    n_types=1, masses=[63.546]),
        profile=_profile(64, 2, 0, 16, 2, 256, 1, C1=8, C2=4, K1=4, K2=2, H=176,
                         Hp=344, S=108, D_out=208),
        weights_seed=11, head_scale=-1.0,
        md=dict(steps=1000, dt_ps=0.001, temperature=300.0, seed=1,
                rebuild_every=10, skin=1.0),
    ),
    # 10,800 water-like molecules (32,400 atoms), 500 NVE steps
    "cfg3_water32400": dict(
        index=2,
        system=dict(kind="water", molecules=10800, density_g_cm3=1.0,
                    min_oo=2.5, seed=4, n_types=2, masses=[15.999, 1.008]),
        profile=_profile(64, 3, 0, 16, 2, 256, 2, C1=8, C2=4, K1=4, K2=2, H=176,
                         Hp=344, S=115, D_out=219),
        weights_seed=12, head_scale=-0.01,
        md=dict(steps=500, dt_ps=0.0005, temperature=300.0, seed=5,
                rebuild_every=10, skin=1.0),
    ),
    # 128,000-atom 5-element BCC alloy, 200 NVE steps
    "cfg4_hea128k": dict(
        index=3,
        system=dict(kind="bcc", cells=40, a=3.2, jitter=0.08, seed=2,
                    n_types=5, masses=[50.94, 92.91, 95.95, 180.95, 183.84]),
        profile=_profile(128, 2, 0, 16, 3, 384, 5, C1=16, C2=8, K1=8, K2=2,
                         H=344, Hp=688, S=216, D_out=522),
        weights_seed=13, head_scale=-0.2,
        md=dict(steps=200, dt_ps=0.001, temperature=1000.0, seed=6,
                rebuild_every=10, skin=1.0),
    ),
    # 1,000,000-atom amorphous mixture of 64 species, 100 NVE steps
    "cfg5_amorphous1m": dict(
        index=4,
        system=dict(kind="poisson_disk", atoms=1000000, density=0.08,
                    min_dist=1.8, seed=3, n_types=64,
                    masses=[12.0 + 3.0 * t for t in range(64)]),
        profile=_profile(128, 3, 0, 16, 3, 384, 64, C1=16, C2=8, K1=8, K2=2,
                         H=344, Hp=688, S=223, D_out=541),
        weights_seed=14, head_scale=0.05,
        md=dict(steps=100, dt_ps=0.001, temperature=600.0, seed=7,
                rebuild_every=10, skin=1.0),
    ),
}

# The paper's own throughput workload: jittered diamond carbon (a = 3.567, sigma = 0.03, seed 0; 158
# neighbours within 6 A), 50^3 conventional cells = 1,000,000 atoms, with its five model variants
# (C0, L, R, F) = Nano (8,2,0,96), Mini (32,2,0,192), Neo (64,2,0,256), Air (64,3,4,256), Plus
# (128,3,4,384); three hidden layers, 16 radial functions, a 118-species type table of which only
# carbon (index 5) occurs.  ``published`` is the paper's rate at 1,000,000 atoms on one H20 (complete
# NVT steps in LAMMPS/Kokkos, trained weights): context for the rate measured here with random
# weights and the library's own NVE driver, not a like-for-like target.
def _paper_variant(index, seed, published, *profile_args, **profile_kw):
    return dict(
        index=index,
        system=dict(kind="diamond", cells=50, a=3.567, jitter=0.03, seed=0, n_types=118, type_index=5,
                    masses=[12.011] * 118),
        profile=_profile(*profile_args, **profile_kw),
        weights_seed=seed, head_scale=-0.002,
        md=dict(steps=100, dt_ps=0.001, temperature=300.0, seed=8, rebuild_every=10, skin=1.0),
        published=dict(value=published, unit="atom-steps/s", hardware="1x NVIDIA H20, fp32",
                       source="paper, supplementary table of rates at 1,000,000 atoms"),
    )


CONFIGS.update({
    "paper_nano_c1m": _paper_variant(5, 21, 16.72e6, 8, 2, 0, 16, 3, 96, 118, C1=4, C2=4, K1=4, K2=2,
                                     H=24, Hp=48, S=40, D_out=70),
    "paper_mini_c1m": _paper_variant(6, 22, 10.37e6, 32, 2, 0, 16, 3, 192, 118, C1=8, C2=4, K1=4, K2=2,
                                     H=88, Hp=176, S=76, D_out=144),
    "paper_neo_c1m": _paper_variant(7, 23, 7.12e6, 64, 2, 0, 16, 3, 256, 118, C1=8, C2=4, K1=4, K2=2,
                                    H=176, Hp=344, S=108, D_out=208),
    "paper_air_c1m": _paper_variant(8, 24, 3.82e6, 64, 3, 4, 16, 3, 256, 118, C1=8, C2=4, K1=4, K2=2,
                                    H=176, Hp=344, S=115, D_out=219),
    "paper_plus_c1m": _paper_variant(9, 25, 2.16e6, 128, 3, 4, 16, 3, 384, 118, C1=16, C2=8, K1=8, K2=2,
                                     H=344, Hp=688, S=223, D_out=541),
})

# Small profiles for unit and parity tests (shape coverage: identity A_1 at the two
# narrowest widths, R > 0, L = 3, several species).
SMALL_PROFILES = {
    "p8_2_0": _profile(8, 2, 0, 8, 2, 32, 2, C1=4, C2=4, K1=4, K2=2, H=24, Hp=48,
                       S=40, D_out=70),
    "p16_2_0": _profile(16, 2, 0, 8, 2, 48, 3, C1=4, C2=4, K1=4, K2=2, H=48,
                        Hp=88, S=48, D_out=86),
    "p16_3_2": _profile(16, 3, 2, 8, 2, 48, 2, C1=4, C2=4, K1=4, K2=2, H=48,
                        Hp=88, S=55, D_out=97),
    "p32_2_4": _profile(32, 2, 4, 16, 3, 64, 2, C1=8, C2=4, K1=4, K2=2, H=88,
                        Hp=176, S=76, D_out=144),
    "p32_3_2": _profile(32, 3, 2, 16, 2, 64, 3, C1=8, C2=4, K1=4, K2=2, H=88,
                        Hp=176, S=83, D_out=155),
    # the widest set of shared radial modes, at a narrow and at a wide scalar width
    "p16_2_8": _profile(16, 2, 8, 8, 2, 48, 3, C1=4, C2=4, K1=4, K2=2, H=48,
                        Hp=88, S=48, D_out=86),
    "p64_3_8": _profile(64, 3, 8, 16, 2, 96, 2, C1=8, C2=4, K1=4, K2=2, H=176,
                        Hp=344, S=115, D_out=219),
    # D_out == F: the first MLP layer carries the identity residual
    "p32_2_0_res": _profile(32, 2, 0, 8, 2, 144, 2, C1=8, C2=4, K1=4, K2=2, H=88,
                            Hp=176, S=76, D_out=144),
    # the widest scalar width, with and without shared radial modes, three species
    "p128_3_4": _profile(128, 3, 4, 16, 2, 96, 3, C1=16, C2=8, K1=8, K2=2, H=344,
                         Hp=688, S=223, D_out=541),
    "p128_2_0": _profile(128, 2, 0, 16, 2, 96, 3, C1=16, C2=8, K1=8, K2=2, H=344,
                         Hp=688, S=216, D_out=522),
    # maximum degree four, at the three degree-wise channel layouts
    "p8_4_0": _profile(8, 4, 0, 8, 2, 32, 2, C1=4, C2=4, K1=4, K2=2, H=24, Hp=48,
                       S=56, D_out=93),
    "p32_4_2": _profile(32, 4, 2, 16, 2, 64, 3, C1=8, C2=4, K1=4, K2=2, H=88,
                        Hp=176, S=92, D_out=167),
    "p128_4_4": _profile(128, 4, 4, 16, 2, 96, 2, C1=16, C2=8, K1=8, K2=2, H=344,
                         Hp=688, S=232, D_out=557),
}
