/*
 * umlmd.h -- C ABI of libumlmd: energy, force and virial evaluation of the DPA4C
 * machine-learning interatomic potential on one NVIDIA B200 (sm_100a) over a cutoff neighbor
 * list that the library builds itself (orthorhombic or general cells, any mix of periodic
 * directions), plus velocity-Verlet NVE and Nose-Hoover-chain NVT drivers and per-atom
 * energies and virials.
 *
 * Conventions
 *   - Every function returns an int status: UMLMD_OK (0) or a negative UMLMD_E_* code.
 *     Nothing throws, aborts or traps on the device.  umlmd_last_error() returns a
 *     human-readable message for the last failure on a handle.
 *   - Pointers whose name starts with d_ are CUDA device pointers owned by the caller
 *     (for instance a torch tensor's data_ptr()); every other pointer is host memory.
 *     The library never frees or keeps caller memory beyond the call, except the MD state
 *     registered with umlmd_set_md_state, which must stay valid until it is replaced or
 *     the handle is destroyed.
 *   - The handle owns the model constants and all workspace; it allocates device memory
 *     in the first umlmd_build_neighbors call and grows it there when a system needs more.
 *   - All work is enqueued on the CUDA stream given to umlmd_create.  Calls that return
 *     host values (energy, virial, counts) synchronise that stream before returning.
 *   - Units are "metal": Angstrom, eV, ps, amu, K.  Species are 0-based indices into the
 *     blob's type table.
 *   - Arrays are row-major.  Positions, velocities and forces are double [N][3].
 */
#ifndef UMLMD_H
#define UMLMD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct umlmd umlmd_t;

enum {
    UMLMD_OK = 0,
    UMLMD_E_INVALID_ARG = -1,         /* NULL pointer, negative size, bad option            */
    UMLMD_E_BAD_BLOB = -2,            /* magic / version / size mismatch, non-finite weight */
    UMLMD_E_UNSUPPORTED_PROFILE = -3, /* C0 not in {8,16,32,64,128}, L not in {2,3,4},
                                         R not in {0,2,4,8}, F % 4 != 0, ...                */
    UMLMD_E_UNSUPPORTED_CELL = -4,    /* singular or non-finite cell, non-positive edge,
                                         more than 127 periodic images along a direction     */
    UMLMD_E_NO_NEIGHBORS = -5,        /* compute/step called before build_neighbors         */
    UMLMD_E_STALE_NEIGHBORS = -6,     /* an atom moved more than skin/2 since the build     */
    UMLMD_E_NONFINITE = -7,           /* NaN or Inf in positions, energy or forces          */
    UMLMD_E_CUDA = -8,                /* a CUDA runtime call failed (message has details)   */
    UMLMD_E_CAPACITY = -9,            /* caller buffer too small, or a list too long for the
                                         32-bit export (see umlmd_get_neighbors)             */
    UMLMD_E_NO_MD_STATE = -10         /* step called before set_md_state                    */
};

/* Optional settings for umlmd_create.  Zero-initialise, set struct_bytes = sizeof, then
 * override fields; a zero field means "default". */
typedef struct umlmd_options {
    uint32_t struct_bytes;
    double   table_dx;   /* radial table spacing in Angstrom; 0 = the blob's value         */
    int32_t  node_tile;  /* atoms per workspace tile; 0 = 524288                            */
    int32_t  mlp_path;   /* 0 = default (2), 1 = CUDA-core fp32 GEMM, 2 = tcgen05 GEMM on split half-precision operands
                            (three products, 22 significant bits), persistent, 3 = the same, one tile per CTA,
                            4 = the same on pairs of CTAs (tcgen05 cta_group::2, 256 rows x up to 256 columns per
                            pair) for every GEMM; path 2 uses that kernel only where it is the faster one, the
                            last GEMM of the backward pass; 2, 3 and 4 need F % 8 == 0 and fall back to 1 otherwise */
    int32_t  pair_table_mb;  /* device memory, MiB, that per-pair amplitude tables may take
                                (see umlmd_build_neighbors); 0 = 192, negative = never build them */
    int32_t  gemm_spin_limit;       /* polls after which a wait inside the tensor-core GEMM's operand
                                       pipeline gives up (the kernel then finishes with garbage, and the
                                       call returns UMLMD_E_CUDA "pipeline wait expired"); 0 = 4,000,000 */
    int32_t  fault_skip_gemm_stage; /* diagnostic for that error path: k > 0 makes the first evaluation
                                       after umlmd_create leave the k-th operand stage of the first MLP
                                       layer unloaded, so that exactly such a wait runs out (nothing
                                       faults or hangs; the handle stays usable); 0 = off */
    int32_t  launch_graphs;         /* replay of repeated launch sequences as CUDA graphs (an evaluation
                                       of the same buffers as the one before it; the middle steps of an MD
                                       run between two list builds): 0 = for systems of at most 65536
                                       atoms, where the time between two dozen short kernels exceeds the
                                       time inside them, 1 = always, -1 = never.  Results are those of
                                       the plain launches, bit for bit (same kernels, same order).  Not
                                       in the paper. */
} umlmd_options;

/* Structural widths of a model, all derived from (C0, L, R) by the paper's formulas
 * (degree-wise channel widths, probe ranks, feature-state width S, feature-vector width
 * D_out, gated hidden widths H and H_pair). */
typedef struct umlmd_info {
    int32_t C0, L, R, N_rbf, n_hidden, F, T;
    int32_t C1, C2, K1, K2, S, D_out, H, H_pair;
    int32_t table_rows;
    double  rc, table_dx;
    int64_t n_atoms, n_edges;          /* of the current neighbor list (0 before a build)  */
    int64_t device_bytes;              /* device memory currently held by the library      */
    int64_t kernel_launches;           /* kernels of this library launched by the handle   */
    int64_t graph_replays;             /* launch sequences replayed as graphs (their kernels are counted above) */
} umlmd_info;

/* Widths for a (C0, L, R) triple without a handle; fills only the width fields.
 * Returns UMLMD_E_UNSUPPORTED_PROFILE for an unsupported triple. */
int umlmd_profile_widths(int32_t C0, int32_t L, int32_t R, umlmd_info* out);

/*
 * Create a model from a weight blob (host memory, little-endian):
 *   char[8] "UMLMD1\0\0"; u32 version = 1; u32 C0, L, R, N_rbf, n_hidden, F, T, basis (0 =
 *   Bessel, f_n = sin(omega_n rho) / rho; 1 = Gaussian, f_n = exp(-(rho - c_n)^2 / (2 s^2)) with
 *   s = rc / (N_rbf - 1), the centres c_n in the place of omega); f64 rc, table_dx; then float32
 *   arrays, row-major, y = x W convention:
 *   X0[T,C0], omega[N_rbf], W_in[N_rbf,2H], W_out[H,C0], W_mode[H,R], W_p_in[2C0,2Hp],
 *   W_p_out[Hp,C0(2+R)] (column blocks scale|shift|mode), W_1[C1,C1], W_2[C2,C2],
 *   A_1[C1,K1], A_2[C2,K2], mu[D_out], sigma[D_out], Theta_1[D_out,F], b_1[F],
 *   {Theta_t[F,F], b_t[F]} t = 2..n_hidden, w_head[F], b_head, E_ref[T].
 * The create step evaluates, once and in double precision on the host, everything the
 * paper's compressed inference precomputes: the Hermite radial table of the shared radial
 * map and modes on [0, rc] (the cubic through value and first derivative at each knot, its
 * quadratic and cubic coefficients stored as 20- and 12-bit fixed-point numbers on the
 * table's own scale; the paper stores the quintic that also matches the second derivative), the
 * ordered type-pair scale / shift / mode-mixing cache, and the unit-norm Gaunt coupling
 * tensors of the admissible degree triples.
 *   stream: a cudaStream_t passed as void* (NULL = the default stream).
 * umlmd_create itself touches no device: the constants are uploaded by the first
 * umlmd_build_neighbors call, so creation and the host-side diagnostics below also work on
 * a machine without a GPU.
 */
int umlmd_create(const void* blob, size_t blob_bytes, const umlmd_options* opt, void* stream,
                 umlmd_t** out);
int umlmd_destroy(umlmd_t* h);
/* Library plumbing, no counterpart in the paper: the model's structural widths (derived by the
 * paper's width formulas, see umlmd_info), the size of the current list, the device memory the
 * library holds in this process and the number of kernels this handle has launched. */
int umlmd_query(const umlmd_t* h, umlmd_info* out);
const char* umlmd_last_error(const umlmd_t* h);

/*
 * Device memory, in bytes, that a handle of this model holds after umlmd_build_neighbors,
 * umlmd_compute and umlmd_set_md_state on a system of N atoms whose list has n_edges entries
 * (list radius rc + skin): model constants, the neighbor list and its build scratch, one node
 * tile of evaluation workspace, per-edge gradients and per-atom results.  Known before anything
 * is allocated (library plumbing, no counterpart in the paper; the paper's memory-scaling note is
 * the model: a fixed tile workspace plus terms linear in atoms and in edges).  An upper estimate
 * within a few per cent; per-pair amplitude tables, when the species present are few enough for
 * them, add at most umlmd_options.pair_table_mb on top.
 */
int umlmd_workspace_bytes(const umlmd_t* h, int64_t N, int64_t n_edges, int64_t* bytes);

/*
 * Build the directed neighbor graph of the paper's neighbor-set definition with list
 * radius r_list = rc + skin: edge (i <- j, n) exists iff (j, n) != (i, 0) and
 * |(r_j + n.cell) - r_i|^2 < r_list^2 (true distance, strict), periodic images being
 * distinct neighbor instances, both orientations stored, no capacity limit.
 *   d_pos   [N,3] double, any image of each atom; folded into the cell internally with
 *           frac - floor(frac) along periodic directions (n refers to folded positions);
 *           periodicity of direction k means translation by cell vector k
 *   d_type  [N] int32 species, each in [0, T) (checked: UMLMD_E_INVALID_ARG otherwise)
 *   cell    9 doubles, rows are the cell vectors a, b, c; any non-singular cell.  A diagonal
 *           (orthorhombic) cell takes the exactly reproducible path below; a general cell is
 *           folded with f = r cell^-1, r - floor(f) . cell, and images are offset by n . cell
 *           (an implementation that folds with (f - floor f) . cell gets the same points to the
 *           last bit or two: in a sheared cell two implementations agree on the edge set except
 *           for a pair whose distance lies within rounding of the list radius)
 *   pbc     3 ints, non-zero = periodic along that cell vector
 *   skin    extra list radius in Angstrom (>= 0); edges beyond rc carry zero weight
 * The predicate is evaluated in double precision as ((xj + n*L) - xi), d2 = (dx*dx +
 * dy*dy) + dz*dz, d2 < r_list*r_list, without fused multiply-add, so that the edge set is
 * reproducible bit for bit.  Atoms are renumbered internally in cell order; all outputs
 * of this library are in the caller's numbering.
 * The call also finds which species occur.  When the P species present are few enough that
 * P^2 tables of table_rows x 3 x C0 words fit in umlmd_options.pair_table_mb, the edge
 * amplitude of every ordered pair (s, s') among them, psi_c(rho) = gamma_c g_c(rho) + beta_c +
 * sum_mu U_c,mu q_mu(rho), is tabulated as a cubic table of its own (the same linear
 * combination of the coefficient rows of the radial table), and umlmd_compute reads one row of
 * that table per edge instead of the radial table, the pair cache and the shared modes.  The
 * species are re-examined at every call; the tables are kept while the set does not change.
 */
int umlmd_build_neighbors(umlmd_t* h, int64_t N, const double* d_pos, const int32_t* d_type,
                          const double cell[9], const int pbc[3], double skin);

/*
 * Copy the current neighbor list out in the caller's atom numbering (for verification).
 *   d_row_ptr [N+1] int32, d_src [cap] int32, d_shift [cap,3] int8; row i holds the
 *   neighbor instances (j, n) of centre i in no particular order.
 * Internally edge offsets are 64-bit and a list may hold more than 2^31 - 1 edges; this export
 * then fails with UMLMD_E_CAPACITY, *n_edges still being set.
 * Pass cap = 0 (pointers may be NULL) to only query *n_edges.  UMLMD_E_CAPACITY if the
 * list has more than cap edges.
 */
int umlmd_get_neighbors(umlmd_t* h, int32_t* d_row_ptr, int32_t* d_src, int8_t* d_shift,
                        int64_t cap, int64_t* n_edges);

/*
 * The same export (the edge set of the paper's neighbor-set definition, for verification) for the
 * centres first_row .. first_row + n_rows - 1 only, with 64-bit offsets, so that rows of a list of
 * any length can be compared entry by entry:
 *   d_row_ptr [n_rows + 1] int64, always filled: offsets of the rows inside d_src / d_shift
 *   d_src [cap] int32, d_shift [cap, 3] int8: the neighbor instances (j, n), caller's numbering
 * *n_edges receives the number of edges of those rows.  Pass cap = 0 (edge buffers may be NULL) to
 * learn it; UMLMD_E_CAPACITY if the rows hold more than cap edges (what fits has been written).
 */
int umlmd_get_neighbor_rows(umlmd_t* h, int64_t first_row, int64_t n_rows, int64_t* d_row_ptr,
                            int32_t* d_src, int8_t* d_shift, int64_t cap, int64_t* n_edges);

/*
 * Energy, forces and virial for positions d_pos [N,3] (same atoms, species and cell as
 * the last build; each atom within skin/2 of where it was at the build, else
 * UMLMD_E_STALE_NEIGHBORS).
 *   energy         host, eV: sum of atomic energies (MLP output + per-species reference)
 *   d_force        [N,3] double, eV/Angstrom: F_k = sum_{j in N_k} g_kj - sum_{i: k in N_i} g_ik
 *                  with g_ij = dE/dr_ij; may be NULL
 *   virial         host, 9 doubles, eV: Xi_ab = - sum_edges g_a r_b; may be NULL
 *   d_atom_energy  [N] double, eV; may be NULL
 * The whole chain runs in the library's CUDA kernels: per-edge radial table / pair
 * modulation / envelope / harmonics and per-destination aggregation, polynomial
 * invariants, the residual SiLU MLP, its vector-Jacobian product, the invariant
 * vector-Jacobian product, the edge recomputation pass and the atomic-free force and
 * virial assembly.
 */
int umlmd_compute(umlmd_t* h, const double* d_pos, double* energy, double* d_force,
                  double virial[9], double* d_atom_energy);

/*
 * Batched evaluation of many independent frames of one model in one call: the paper's execution
 * note evaluates several frames at once and reduces the atomic energies per frame (its
 * "segmented" energy reduction); small systems are bound by the fixed cost of a step's launches,
 * which a batch pays once.  The atoms of all frames are concatenated:
 *   frame_offsets  host, n_frames + 1 int64: frame f holds atoms frame_offsets[f] .. [f+1] - 1
 *   d_pos [N,3], d_type [N]   device, N = frame_offsets[n_frames]
 *   cells          host, n_frames x 9 doubles: each frame's cell vectors as rows (any non-singular cell)
 *   pbc            3 ints, the same for every frame
 *   energies       host, n_frames doubles (may be NULL)
 *   d_force        [N,3] double, device (may be NULL)
 *   virials        host, n_frames x 9 doubles (may be NULL)
 *   d_atom_energy  [N] double, device (may be NULL)
 * The neighbor lists (radius rc, no skin) are found by exhaustive search inside each frame, which
 * suits frames of up to a few thousand atoms (limit UMLMD_BATCH_MAX_FRAME_ATOMS, else
 * UMLMD_E_CAPACITY); edges never cross frames.  The whole batch then runs through the same kernels
 * as one system, and one block per frame sums the frame's atomic energies and edge virials in a
 * fixed order.  The call replaces the handle's neighbor list and MD state: call
 * umlmd_build_neighbors again before umlmd_compute or umlmd_step.
 */
#define UMLMD_BATCH_MAX_FRAME_ATOMS 16384
int umlmd_compute_batch(umlmd_t* h, int32_t n_frames, const int64_t* frame_offsets, const double* d_pos,
                        const int32_t* d_type, const double* cells, const int pbc[3], double* energies,
                        double* d_force, double* virials, double* d_atom_energy);

/*
 * (Not in the paper, which drives its model from LAMMPS: the integrators here exist because the
 * benchmark's workloads are MD runs.)
 * Register MD state for umlmd_step: d_pos and d_vel [N,3] double (Angstrom, Angstrom/ps)
 * are advanced in place; mass_per_type is T doubles (amu, host; copied).  N, species and
 * cell are those of the last umlmd_build_neighbors call.  The library keeps the forces of the
 * registered positions between calls: after editing d_pos by hand, register the state again.
 */
int umlmd_set_md_state(umlmd_t* h, double* d_pos, double* d_vel, const double* mass_per_type);

/*
 * Advance nsteps of velocity-Verlet NVE with time step dt_ps (not in the paper, whose timed runs
 * are LAMMPS NVT steps; each step runs the paper's whole evaluation path once: v += dt/2 F/m,
 * r += dt v, evaluate, v += dt/2 F/m, in double precision).  The neighbor list is
 * rebuilt (with the skin of the last build) every rebuild_every steps, counted from the
 * last build; rebuild_every == 0 never rebuilds (a step in which an atom has moved more
 * than skin/2 since the build then fails with UMLMD_E_STALE_NEIGHBORS); rebuild_every < 0
 * rebuilds exactly when that displacement criterion trips, at the price of one host
 * synchronisation per step.  On return e_pot / e_kin (host, eV; may be NULL) hold the
 * potential and kinetic energy after the last step.
 */
int umlmd_step(umlmd_t* h, int nsteps, double dt_ps, int rebuild_every, double* e_pot,
               double* e_kin);

/*
 * The same driver at constant temperature: velocity Verlet between two half-step
 * propagations of a Nose-Hoover chain of three thermostats (Martyna-Tuckerman-Klein form,
 * the integrator behind the NVT runs the paper times; the model's hot path is unchanged).
 * temperature_K is the target, t_damp_ps the thermostat period: the first thermostat has
 * mass (3N - 3) kT t_damp^2, the others kT t_damp^2.  The chain starts at rest after every
 * umlmd_set_md_state and carries over between calls.  e_conserved (may be NULL) receives
 * E_pot + E_kin + the chain's energy, which this dynamics conserves.  The system needs at
 * least two atoms.  Other arguments and errors as for umlmd_step.
 */
int umlmd_step_nvt(umlmd_t* h, int nsteps, double dt_ps, int rebuild_every, double temperature_K,
                   double t_damp_ps, double* e_pot, double* e_kin, double* e_conserved);

/*
 * Thermostat state of umlmd_step_nvt, for checkpoints (not in the paper): the chain's positions
 * eta[3] followed by its velocities v_eta[3] (1/ps).  umlmd_get_nvt_state reads them (zeros
 * while the chain is at rest); umlmd_set_nvt_state, called after umlmd_set_md_state, restores
 * them, so that a run continued from saved positions, velocities and chain state repeats the
 * uninterrupted run exactly when it restarts on a step at which that run rebuilt its list.
 */
#define UMLMD_NVT_STATE_DOUBLES 6
int umlmd_get_nvt_state(umlmd_t* h, double state[UMLMD_NVT_STATE_DOUBLES]);
int umlmd_set_nvt_state(umlmd_t* h, const double state[UMLMD_NVT_STATE_DOUBLES]);

/*
 * Ghost atoms, for a system cut into spatial domains (the paper's distributed runs: each rank owns
 * the atoms of its region, holds copies -- ghosts -- of the atoms within the list radius around it,
 * receives their coordinates before an evaluation and sends the forces on them back afterwards; no
 * learned quantity crosses a boundary because the model has a single aggregation layer).
 * From the next umlmd_build_neighbors on (the call drops the current list: the library's internal
 * order puts owned atoms first), the atoms with index >= n_owned (caller's numbering) are ghosts:
 * they are neighbours only.  No atomic energy is computed for them (their entries of
 * d_atom_energy are 0, the energy is the sum over the owned atoms), only the edges that end on an
 * owned atom carry a gradient, and d_force holds for every atom, owned or ghost, minus the derivative
 * of that energy: the forces on ghosts are what has to be added to their owners' forces, and the
 * virial is the owned atoms' share, -sum over their edges of g (x) r.  Summed over all domains these
 * are the energy, forces and virial of the whole system.  The neighbor list is built over all
 * atoms as usual (give the domain's box as a non-periodic cell); ghosts cost their share of the list
 * build and of the force assembly, nothing else: no per-edge or per-atom stage visits their rows.
 *   n_owned   number of owned atoms, placed first; negative or >= N: every atom is owned (default)
 * umlmd_step and umlmd_step_nvt move every atom of the handle and refuse to run while ghosts are
 * set; a domain's driver uses umlmd_compute and umlmd_vv_update.  Not in the paper as an interface
 * (it delegates this to its MD host code).
 */
int umlmd_set_owned_atoms(umlmd_t* h, int64_t n_owned);

/*
 * One piece of a velocity Verlet step on caller-owned arrays (no handle: for drivers that own the
 * integrator state themselves, e.g. one spatial domain's owned atoms):
 *   v += half_kicks * (dt/2) * F / m   (half_kicks in {0, 1, 2}; 2 = the closing kick of one step and
 *                                        the opening kick of the next in one pass)
 *   r += dt * v                        (if drift != 0, after the kick)
 * with 1 eV/(Angstrom amu) = 9648.533 Angstrom/ps^2 (metal units, as umlmd_step).
 *   d_pos, d_vel   [N,3] double, Angstrom and Angstrom/ps   (device, caller-owned, updated in place)
 *   d_force        [N,3] double, eV/Angstrom                (device; may be null if half_kicks == 0)
 *   d_type         [N] int32 species; every entry must index d_inv_mass_per_type (not checked:
 *                  there is no handle to check it against)
 *   d_inv_mass_per_type   1/mass in 1/amu by species        (device)
 *   stream         cudaStream_t as void*; the call only enqueues work
 * Returns UMLMD_E_INVALID_ARG for null pointers, a bad count or time step; UMLMD_E_CUDA if the
 * launch fails.  Not in the paper (it integrates with LAMMPS).
 */
int umlmd_vv_update(int64_t N, double* d_pos, double* d_vel, const double* d_force, const int32_t* d_type,
                    const double* d_inv_mass_per_type, double dt_ps, int32_t half_kicks, int32_t drift, void* stream);

/*
 * Per-atom virial of the last evaluation that produced forces or the virial (umlmd_compute with
 * d_force or virial given, or umlmd_step / umlmd_step_nvt): every directed edge e = (i <- j, n)
 * with gradient g_e = dE/dr_ij and vector r_e shares -g_e (x) r_e equally between its two atoms,
 *   W_k = -1/2 sum over the edges with k as centre or as neighbour of g_e (x) r_e,
 * so that sum_k W_k is the virial umlmd_compute returns (the paper lists atomic virials as an
 * optional per-atom output without fixing the split; this is the usual half-and-half one).
 *   d_atom_virial [N, 9] double, row-major 3 x 3 per atom (component [a][b] = force-like index a,
 *   vector index b), caller's numbering, eV.
 * UMLMD_E_INVALID_ARG if no such evaluation has run since the last build.
 */
int umlmd_atom_virial(umlmd_t* h, double* d_atom_virial);

/*
 * Diagnostics used by the parity tests: copy out per-atom intermediates of the last
 * umlmd_compute, in the caller's numbering.  Each pointer may be NULL.
 *   d_state  [N, S+2] float: unnormalised sums A (degree, then m, then channel), s0, s1
 *   d_desc   [N, D_out] float: calibrated feature vector D
 * Only valid for a single-tile evaluation of fewer than 65536 atoms; otherwise UMLMD_E_CAPACITY.
 * These hold forward values only if umlmd_compute was called with d_force == NULL and
 * virial == NULL (the backward pass reuses both buffers).
 */
int umlmd_get_intermediates(umlmd_t* h, float* d_state, float* d_desc);

/*
 * Evaluate the tabulated radial map at n distances (host arrays): out_g [n, C0+R] holds
 * g(rho) then q(rho), out_dg their derivatives, from the same cubic polynomials the
 * kernels use (evaluated on the host from the device table's float32 coefficients).
 */
int umlmd_eval_radial_table(const umlmd_t* h, int64_t n, const double* rho, double* out_g,
                            double* out_dg);

/*
 * Per-kernel-class accounting.  The handle always counts the kernels it launches; with
 * profiling enabled it also brackets each class with CUDA events on its stream (a few
 * microseconds of overhead per launch group, so leave it off when timing whole steps).
 * umlmd_get_profile synchronises the stream, returns accumulated milliseconds and launch
 * counts per class since the previous call (arrays of max_classes entries; *n_classes
 * receives the number of classes) and resets them.  Class names: gather_positions,
 * edge_forward, invariants_forward, mlp_forward, mlp_backward, invariants_backward,
 * edge_backward, force_assembly, energy_virial_reduce, integrate, neighbor_build.
 */
int umlmd_set_profiling(umlmd_t* h, int enabled);
int umlmd_get_profile(umlmd_t* h, int32_t max_classes, double* ms, int64_t* launches, int32_t* n_classes);
const char* umlmd_profile_class_name(int32_t cls);

/*
 * Measurement aid, not part of the model (the paper has no counterpart): the FP32 fused
 * multiply-add rate of the current device, in TFLOP/s (2 flops per FMA), from a register-resident
 * chain of FMAs on every lane, timed with CUDA events on `stream` (best of four launches of about
 * a millisecond).  The benchmark divides the edge kernels' arithmetic rate by this number.
 * Allocates four bytes of device memory for the duration of the call and synchronises.
 */
int umlmd_probe_fma_peak(double* tflops, void* stream);

/*
 * Kinetic energy sum_i m_i |v_i|^2 / 2 (eV) for callers that must not allocate.  (The
 * paper has no counterpart: its integrator is LAMMPS'.)
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they need a number
 * from it: a plugin running inside another program's real-time or memory-pooled loop,
 * where the embedding application owns all device memory and forbids allocator calls (they
 * can synchronise the whole device), or code that runs after its memory budget has been
 * handed out.  Every other entry point may grow the handle's workspace; this one never
 * does.  It calls no cudaMalloc, cudaFree or allocating library routine and needs no
 * handle.  It is the same two-pass, fixed-order, double-precision reduction that
 * umlmd_step uses for e_kin, with the per-block partial sums kept in a fixed 8 KB array
 * inside the library's device image instead of allocated workspace.
 *   N                 atoms, at most UMLMD_STATIC_MAX_ATOMS; more is rejected with
 *                     UMLMD_E_CAPACITY and a message (umlmd_static_last_error)
 *   d_vel             [N,3] double, Angstrom/ps           (device, caller-owned)
 *   d_type            [N] int32 species                   (device, caller-owned); every entry must
 *                     be a valid index into d_mass_per_type: there is no handle here to check it
 *                     against, and an entry outside the mass array is an out-of-bounds read
 *   d_mass_per_type   masses in amu indexed by species    (device, caller-owned)
 *   d_e_kin           one double, receives the result     (device, caller-owned)
 *   stream            cudaStream_t as void*; the call only enqueues work
 * The first call on each device looks up the device address of the fixed array (current
 * device = the one the stream belongs to); make that first call before starting any
 * stream capture.  The address is remembered per device for the life of the process and
 * belongs to the device's primary context: do not call this after cudaDeviceReset in the same
 * process.  All calls on a device share the array: it keeps the previous call's
 * partial sums, every entry that a call reads is first written by that same call so
 * nothing needs clearing, and two calls whose kernels overlap on the GPU (different
 * streams) race on it -- serialise them.
 */
#define UMLMD_STATIC_MAX_ATOMS 4194304
int umlmd_kinetic_energy_static(int64_t N, const double* d_vel, const int32_t* d_type,
                                const double* d_mass_per_type, double* d_e_kin, void* stream);
const char* umlmd_static_last_error(void);

/*
 * Read one entry of the ordered type-pair cache (host): out receives (2+R)*C0 doubles,
 * the scale gamma[C0], the shift beta[C0], then the mode mixing as R rows U[:, mu] of C0
 * values, for centre species type_i and neighbour species type_j.
 */
int umlmd_eval_pair_cache(const umlmd_t* h, int32_t type_i, int32_t type_j, double* out);

#ifdef __cplusplus
}
#endif
#endif /* UMLMD_H */
