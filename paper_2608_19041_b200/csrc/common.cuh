// Shared declarations of the library's translation units: structural widths, the
// device-resident model constants, the per-handle workspace and the kernel launchers.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <cstdio>
#include <string>
#include <vector>

#include "../../include/umlmd.h"

namespace umd {

constexpr float kEpsReg = 1.0e-7f;     // direction regulariser, Angstrom (edge geometry)
constexpr int kMaxDeg = 4;             // highest angular degree compiled in
constexpr int kMaxR = 8;               // most shared radial modes
constexpr int kMaxGaunt = 96;          // non-zeros kept per coupling tensor of the degree <= 3 triples
constexpr int kMaxGauntBig = 256;      // the same for the triples that involve degree 4 (up to 9 x 9 x 9 entries)
constexpr double kAccelUnit = 9648.53321;   // (eV/Angstrom/amu) in Angstrom/ps^2
constexpr double kBoltzmann = 8.617333262e-5;

// error word bits set by kernels (read back at synchronisation points)
enum : int { kErrStale = 1, kErrNonFinite = 2, kErrShiftRange = 8, kErrPipelineTimeout = 16, kErrSpecies = 32 };

// Widths derived from (C0, L, R): degree-wise channels, probe ranks, feature-state width
// S, feature-vector width D_out, gated hidden widths, and the flat offsets used by the
// kernels.  Host and device both read this struct (it is passed by value).
struct Dims {
    int C0, L, R, N_rbf, n_hidden, F, T;
    int C[kMaxDeg + 1];      // channels per degree
    int K[kMaxDeg + 1];      // probe ranks (index 0 unused)
    int S, SP;               // state width S; row stride SP >= S+4 (s0, s1 as float pairs), multiple of 4
    int offA[kMaxDeg + 1];   // offset of degree block in the state row
    int D_out, DP;           // feature-vector width; row stride (multiple of 32)
    int oG[kMaxDeg + 1];     // offsets of vech(G_l) in D
    int oJ112, oJ123, oJ222, oJ233, oPi;
    int oJ134, oJ224, oJ244, oJ334, oJ444;   // blocks of the triples that exist only for L = 4
    int H, Hp;
    int CP;                  // table channels C0+R rounded up to 4
    int n_rows;              // table intervals
    float tab_k2, tab_k3;    // steps of the packed quadratic and cubic coefficients of the radial table
    float rc, dx, inv_dx;
};

struct GauntSparse {         // non-zeros of one unit-norm coupling tensor
    int n;
    unsigned char m1[kMaxGaunt], m2[kMaxGaunt], m3[kMaxGaunt];
    float v[kMaxGaunt];
};
struct GauntSparseBig {      // the same with room for the degree-4 triples
    int n;
    unsigned char m1[kMaxGauntBig], m2[kMaxGauntBig], m3[kMaxGauntBig];
    float v[kMaxGauntBig];
};

// Device-resident constants of one model.
struct ModelDev {
    float* table;     // [n_rows][3][CP] cubic Hermite pieces of [g, q]: c0, c1 (fp32), packed (c2, c3)
    float* pairmod;   // [T*T][2+R][C0]: scale gamma, shift beta, mode mixing U[:, mu]
    float* X0;        // [T][C0]
    float* W1p;       // [C1][C1]  I + W_1
    float* W2p;       // [C2][C2]  I + W_2
    float* A1;        // [C1][K1]
    float* A2;        // [C2][K2]
    float* mu;        // [D_out]
    float* inv_sigma; // [D_out]
    float* theta[8];  // Theta_t, row-major [K_in (padded)][F]; theta[0] has DP rows
    float* thetaT[8]; // transposes, [F][K_in (padded)]
    // half-precision split (x = hi + lo) of w_scale[t] * theta and of its transpose; w_scale[t] is
    // the power of two that brings the largest |weight| of the layer to [2^9, 2^10), so that the
    // low parts are normal half-precision numbers; w_scale_inv[t] undoes it on the accumulator
    __half* theta_hi[8];  __half* theta_lo[8];
    __half* thetaT_hi[8]; __half* thetaT_lo[8];
    float w_scale_inv[8];
    float grad_scale; // power of two the tensor-core backward chain multiplies its gradients by (from max |w_head|)
    float* bias[8];   // b_t [F]
    float* type_bias; // [T][F] first-layer bias with the centre's initial features folded in
    float* w_head;    // [F]
    float* e_ref;     // [T]
    float b_head;
    GauntSparse* g123;   // device copies (NULL when L < 3)
    GauntSparse* g233;
    GauntSparseBig* g4;  // [5] device copies of (1,3,4), (2,2,4), (2,4,4), (3,3,4), (4,4,4) (NULL when L < 4)
};

struct Handle;  // defined in api.cu

// ---- launchers (each enqueues on `st`; none synchronises) ---------------------------

typedef long long eidx_t;      // edge offsets are 64-bit: a list may hold more than 2^31 edges

// Packed high-order coefficients of a cubic table piece.  c2 and c3 only enter through c2 t^2 and
// c3 t^3 with t below the table spacing, so a 20-bit and a 12-bit fixed-point number on the table's
// own scale (c2 = k2 I2, c3 = k3 I3; k = largest magnitude in the table / largest integer) cost
// nothing in the value and leave the derivative within a few 1e-7 of its largest entry at the
// default spacing (the error grows with the spacing like the interpolation error itself).
// One 32-bit word: I2 in the upper 20 bits, I3 in the lower 12, both two's complement.
constexpr int kTabI2Max = (1 << 19) - 1, kTabI3Max = (1 << 11) - 1;
__host__ __device__ inline float tab_step2(float max_abs_c2) { return max_abs_c2 * (1.0f / (float)kTabI2Max); }
__host__ __device__ inline float tab_step3(float max_abs_c3) { return max_abs_c3 * (1.0f / (float)kTabI3Max); }
__host__ __device__ inline unsigned tab_pack(float c2, float c3, float k2, float k3) {
    float q2 = k2 > 0.f ? c2 / k2 : 0.f, q3 = k3 > 0.f ? c3 / k3 : 0.f;
    q2 = q2 > (float)kTabI2Max ? (float)kTabI2Max : (q2 < -(float)kTabI2Max ? -(float)kTabI2Max : q2);
    q3 = q3 > (float)kTabI3Max ? (float)kTabI3Max : (q3 < -(float)kTabI3Max ? -(float)kTabI3Max : q3);
    const int i2 = (int)(q2 < 0.f ? q2 - 0.5f : q2 + 0.5f), i3 = (int)(q3 < 0.f ? q3 - 0.5f : q3 + 0.5f);
    return ((unsigned)i2 << 12) | ((unsigned)i3 & 0xfffu);
}
__host__ __device__ inline void tab_unpack(unsigned w, float k2, float k3, float* c2, float* c3) {
    *c2 = k2 * (float)((int)w >> 12);
    *c3 = k3 * (float)((int)(w << 20) >> 20);
}

// One frame of a batched evaluation (umlmd_compute_batch): its own cell and its slice of the
// concatenated atom arrays.
struct FrameCell {
    double H[9];      // cell vectors as rows
    double Hinv[9];   // inverse (fractional coordinates f = r Hinv)
    int m[3];         // periodic images to visit along each cell vector (0 for an open direction)
    int pbc[3];
    int a0, a1;       // atoms [a0, a1) of the concatenated arrays
};

struct NeighborDev {
    int64_t N = 0, E = 0, E_cap = 0, N_cap = 0;
    unsigned long long* bounds = nullptr;   // [6] scratch of the extent reduction (open directions)
    int64_t n_owned = 0, E_owned = 0;   // rows [0, n_owned) and edges [0, E_owned) belong to owned atoms (all of them without ghosts)
    double L[3] = {0, 0, 0};     // cell edge lengths (the diagonal of H)
    double H[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};   // cell vectors as rows
    int tri = 0;                 // the cell has off-diagonal components
    int pbc[3] = {1, 1, 1};
    double skin = 0, r_list = 0;
    double* wpos = nullptr;      // [N][3] folded positions, caller order (build time)
    int* img = nullptr;          // [N][3] floor(frac) per atom, sorted order
    int* perm = nullptr;         // [N] sorted index -> caller index
    int* type_s = nullptr;       // [N] species, sorted order
    double* xs0 = nullptr;       // [N][3] folded positions at build time, sorted order
    double* xs = nullptr;        // [N][3] current positions minus img*L, sorted order
    // [N][2] the same positions and the species as one 32-byte record per atom for the edge kernels'
    // neighbour gathers (one sector and two 16-byte loads instead of four scattered loads):
    // (x_hi, y_hi, z_hi, species bits), (x_lo, y_lo, z_lo, 0) with x = (double)x_hi + (double)x_lo
    float4* rec = nullptr;
    eidx_t* row_ptr = nullptr;   // [N+1]
    int* src = nullptr;          // [E] sorted index of the neighbour
    int* shift = nullptr;        // [E] packed int8 x3 image n
    eidx_t* rev = nullptr;       // [E] index of the reverse edge, -1 if absent
    // batched evaluation: per-frame cells and the frame of every atom (null for a single system)
    FrameCell* frames = nullptr; int64_t frames_cap = 0; int n_frames = 0;
    int* frame_of = nullptr;
    bool batch = false;          // the list in here is the union of per-frame lists
    // scratch
    int* key = nullptr; int* key2 = nullptr; int* idx = nullptr; int* idx2 = nullptr;
    int* cell_start = nullptr; int64_t ncell_cap = 0;
    int* deg = nullptr;
    void* cub_tmp = nullptr; size_t cub_bytes = 0;
};

}  // namespace umd
