// Launchers implemented across the .cu files.  Every launcher enqueues work on the given
// stream and returns the CUDA status of the launch; none of them synchronises unless
// stated.
#pragma once

#include "common.cuh"

namespace umd {

// ---- neighbor.cu ---------------------------------------------------------------------
// Full build: fold + bin + sort + count + scan + fill + reverse map.  Synchronises once
// (to learn the edge count and grow the edge arrays).  Returns a UMLMD_* code.
// n_owned < N: the atoms with caller index >= n_owned are ghosts; they come after all owned atoms
// in the internal order (owned atoms in cell order, then ghosts in cell order), so that rows
// [0, n_owned) are the owned atoms' and nb->E_owned edges belong to them.
int neighbor_build(NeighborDev* nb, int64_t N, int64_t n_owned, const double* d_pos, const int32_t* d_type,
                   const double cell[9], const int pbc[3], double skin, double rc, int* d_err,
                   cudaStream_t st, std::string* err);   // cell: the three cell vectors as rows
void neighbor_free(NeighborDev* nb);
// Export the list in caller numbering (device buffers of the caller).
int neighbor_export(NeighborDev* nb, int32_t* d_row_ptr, int32_t* d_src, int8_t* d_shift,
                    cudaStream_t st, std::string* err);
// Union of the neighbor lists of n_frames independent frames (atoms concatenated, frame f = atoms
// offsets[f] .. offsets[f+1]-1 with cell cells[9 f ..]), list radius rc, by exhaustive search inside
// each frame (meant for many small frames); atoms keep the caller's order.  Returns a UMLMD_* code.
int neighbor_build_batch(NeighborDev* nb, int n_frames, const int64_t* offsets, const double* cells, const int pbc[3],
                         const double* d_pos, const int32_t* d_type, int T, double rc, int* d_err, cudaStream_t st,
                         std::string* err);
// per-frame energy and virial: out[10 f] = sum of e_atom over the frame, out[10 f + 1 ..] = -sum over
// the frame's edges of g (x) r, each by one block in a fixed order
cudaError_t launch_frame_reduce(const NeighborDev& nb, const double* e_atom, const float* g, bool want_virial,
                                double* d_out, cudaStream_t st);
// Rows first .. first + n - 1 of the caller's numbering with 64-bit offsets: d_row_ptr [n + 1] is
// always filled; edges are copied while they fit `cap` (cap = 0 or null buffers: offsets only).
int neighbor_export_rows(NeighborDev* nb, int64_t first, int64_t n, int64_t* d_row_ptr, int32_t* d_src,
                         int8_t* d_shift, int64_t cap, cudaStream_t st, std::string* err);
// xs[i] = pos[perm[i]] - img[i]*L; flags stale / non-finite atoms in *d_err.
cudaError_t launch_gather_positions(const NeighborDev& nb, const double* d_pos, int* d_err,
                                    cudaStream_t st);

// ---- edge.cu ---------------------------------------------------------------------------
struct EdgeArgs {
    Dims d;
    const float* table;
    const float* pairmod;
    const double* xs;       // [N][3] sorted positions
    const float4* rec;      // [N][2] positions (as float pairs) and species, one record per atom
    const int* type_s;
    const eidx_t* row_ptr;
    const int* src;
    const int* shift;
    double Lx, Ly, Lz;
    double H[9];            // cell vectors as rows, used instead of Lx, Ly, Lz when tri
    int tri;
    int a0, a1;             // destination range [a0, a1) of this tile
    float* state;           // [a1-a0][SP]: forward writes sums; backward reads dE/d(sums)
    float* g;               // [E][3] per-edge gradient (backward)
    double* virial_part;    // [blocks][9] partial virial sums (backward)
    // non-null when the species present are few enough for per-pair amplitude tables:
    // [n_present^2][n_rows][3][C0] cubic pieces of psi_c(rho) of each ordered pair, in the format
    // of the radial table (launch_fuse_pair_tables), read instead of table, pairmod and the radial
    // modes; uni_scale[0..1] = largest |c2|, |c3| of these tables (scale of their packed words)
    // batched evaluation: the image offsets of a row come from the cell of the destination's frame
    const FrameCell* frames;    // null for a single system
    const int* frame_of;
    const float* table_uni;
    const float* uni_scale;
    const int* species_slot;    // [T] species -> index among the species present
    int n_present;
};
// present: device array of the n_present species indices, ascending
cudaError_t launch_fuse_pair_tables(const Dims& d, const float* table, const float* pairmod, const int* present,
                                    int n_present, float* scale, float* out, cudaStream_t st);
cudaError_t launch_edge_forward(const EdgeArgs& a, cudaStream_t st);
cudaError_t launch_edge_backward(const EdgeArgs& a, int* n_blocks, cudaStream_t st);
int edge_backward_blocks(int n_rows_in_tile);

// ---- invariants.cu -------------------------------------------------------------------
struct InvArgs {
    Dims d;
    ModelDev m;
    const int* type_s;
    int a0, n;              // tile start (sorted index) and atom count
    float* state;           // [n][SP]
    float* desc;            // [n][DP]
    // forward only: when non-null the feature rows are also written as their half-precision split
    // (row pitch DP), the form the tensor-core MLP reads; write_desc = false then skips the fp32 copy
    __half* desc_hi;
    __half* desc_lo;
    bool write_desc;
    bool skip_x0_split;     // the split omits the first C0 columns (the MLP folds them into a per-species bias)
};
cudaError_t launch_invariants_forward(const InvArgs& a, cudaStream_t st);
cudaError_t launch_invariants_backward(const InvArgs& a, cudaStream_t st);

// ---- mlp.cu ----------------------------------------------------------------------------
struct MlpArgs {
    Dims d;
    ModelDev m;
    const int* type_s;
    int a0, n;
    float* desc;            // [n][DP]  in: D, out (backward): dE/dD
    float* pre;             // [n_hidden][n][F] pre-activations, overwritten by dE/dY
    float* hbuf;            // [2][n][F] ping-pong activations / hidden gradients
    double* e_atom;         // [N] sorted order, eV (written at a0..a0+n)
    int path;               // 1 = CUDA-core fp32, 2 = tcgen05
    bool want_grad;
    __half* tc_hi;          // two slots of [n][max(DP, F)]: half-precision splits of the activations (tensor-core path)
    __half* tc_lo;
    bool desc_presplit;     // slot 0 already holds the split of desc (written by the invariants kernel)
    bool fold_x0;           // tensor-core path: the first C0 feature columns enter through m.type_bias instead of the GEMM
    size_t tc_slot;         // elements per slot
    int* err;               // device error word
    int spin_limit;         // tensor-core path: polls before a pipeline wait gives up (0 = default)
    int test_skip_kblock;   // diagnostic, first layer of the forward pass only: see GemmArgs
};
cudaError_t launch_mlp_forward(const MlpArgs& a, cudaStream_t st);   // layers + head (+ backward seed)
cudaError_t launch_mlp_backward(const MlpArgs& a, cudaStream_t st);  // needs a forward with want_grad

// ---- assemble.cu ---------------------------------------------------------------------
// d_flags[t] = 1 for every species t in [0, T) that occurs among the N atoms, 0 otherwise;
// kErrSpecies is or-ed into *d_err when an index lies outside [0, T)
cudaError_t launch_species_present(int64_t N, const int* type, int T, int* d_flags, int* d_err, cudaStream_t st);
cudaError_t launch_force_assembly(const NeighborDev& nb, const float* g, double* d_force_sorted, double* d_force,
                                  int* d_err, cudaStream_t st);
// per-atom virial shares [N][9] in the caller's numbering from the edge gradients of the last
// backward pass: W_i = -1/2 sum over the edges that touch atom i of g_e (x) r_e
cudaError_t launch_atom_virial(const NeighborDev& nb, const float* g, double* d_out, cudaStream_t st);
cudaError_t launch_scatter_forces(const NeighborDev& nb, const double* f_sorted, double* d_force,
                                  int* d_err, cudaStream_t st);
cudaError_t launch_scatter_atom_energy(const NeighborDev& nb, const double* e_sorted, double* d_out,
                                       cudaStream_t st);
// out[0] = sum e_atom, out[1..9] = -sum virial partials (fixed order, double)
cudaError_t launch_reduce_energy_virial(const double* e_atom, int64_t N, const double* virial_part,
                                        int n_part, double* scratch, double* out, int* d_err,
                                        cudaStream_t st);
int reduce_scratch_doubles(int64_t N);
cudaError_t launch_unsort_state(const NeighborDev& nb, const float* in, int stride, int width,
                                float* out, cudaStream_t st);
// velocity Verlet pieces (caller order, double)
cudaError_t launch_vv_kick_drift(int64_t N, double* pos, double* vel, const double* force, const int* type,
                                 const double* inv_mass, double dt, int kicks, bool drift, const double* d_scale,
                                 cudaStream_t st);
// Nose-Hoover chain thermostat: chain length, parameters (energies in eV, times in ps) and the
// propagation of `halves` half steps on the device; d_state = [eta[M], v_eta[M], scale, kinetic energy]
constexpr int kNhcChain = 3;
struct NhcParams { double dof, kT, Q[kNhcChain], dt_half; };
cudaError_t launch_nhc(double* d_state, const double* d_ke, int halves, const NhcParams& p, cudaStream_t st);
cudaError_t launch_kinetic_energy(int64_t N, const double* vel, const int* type, const double* mass,
                                  double* scratch, double* out, cudaStream_t st);

}  // namespace umd
