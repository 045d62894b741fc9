// Fused per-edge kernels: edge featurisation + per-destination aggregation (forward) and
// the recomputing edge backward pass that returns dE/dr_ij for every edge.
//
// One warp owns one destination atom and walks its contiguous CSR interval, 32 listed edges
// at a time: each lane computes the geometry of one edge (displacement from double-precision
// positions, regularised length, direction, cutoff envelope, table row) and the edges inside
// the cutoff are queued in shared memory.  Full batches of queued edges are then processed
// with lanes split over channels -- a group of lanes handles one edge, each lane holding one
// or two runs of four consecutive channels, so table and pair-cache reads are 16-byte vector
// loads that a group issues as contiguous segments -- followed by a lane-per-edge phase for
// the degree >= 1 blocks.  The S+2 sums live in registers and are written once per
// destination; nothing per-edge is stored in the forward pass.  The backward pass recomputes
// the same per-edge quantities from the same cubic polynomial (so the force is the exact
// derivative of the interpolated energy), contracts them with dE/d(sums) and writes one
// 3-vector per edge; the virial is accumulated in the same pass.
//
// Harmonics are evaluated with |u|^2 set to one; the regularised direction differs from a
// unit vector by eps^2/rho^2, far below single precision.
#include "kernels.h"

namespace umd {

namespace {

// A block is done when its slowest row is: with fewer rows per block fewer finished warps sit on
// registers and shared memory waiting for it (measured at eight / four / two warps per block, 131072
// atoms of the 64-species workload: backward 1.535 / 1.487 / 1.479 ms, forward 1.318 / 1.301 / 1.294 ms;
// four keeps the per-block virial partials at a quarter of the atom count).
constexpr int kWarpsPerBlock = 4;
constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ float4 ldg4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }

struct Geom {
    float dx, dy, dz, rho, inv_rho, ux, uy, uz, chi, dchi, t;
    int row, pair;
    bool valid;
};

// phase 1: one lane, one edge
// Hf: cell of the destination's frame in a batched evaluation (rows), null for a single system
__device__ __forceinline__ Geom edge_geometry(const EdgeArgs& a, eidx_t e, bool in_range, double xi, double yi,
                                              double zi, int ti, const double* __restrict__ Hf) {
    Geom g;
    g.valid = false;
    g.dx = g.dy = g.dz = 0.f; g.rho = 1.f; g.inv_rho = 1.f; g.ux = g.uy = g.uz = 0.f;
    g.chi = 0.f; g.dchi = 0.f; g.t = 0.f; g.row = 0; g.pair = 0;
    if (!in_range) return g;
    const int j = a.src[e];
    const int s = a.shift[e];
    const int nx = (int)(signed char)(s & 0xff), ny = (int)(signed char)((s >> 8) & 0xff),
              nz = (int)(signed char)((s >> 16) & 0xff);
    // the neighbour's record: position as float pairs (exact to 2^-48 of the coordinate) and species
    const float4 r0 = __ldg(a.rec + 2 * (size_t)j), r1 = __ldg(a.rec + 2 * (size_t)j + 1);
    const double xj[3] = {(double)r0.x + (double)r1.x, (double)r0.y + (double)r1.y, (double)r0.z + (double)r1.z};
    const int tj = __float_as_int(r0.w);
    if (Hf) {
        g.dx = (float)((xj[0] + ((nx * __ldg(Hf + 0) + ny * __ldg(Hf + 3)) + nz * __ldg(Hf + 6))) - xi);
        g.dy = (float)((xj[1] + ((nx * __ldg(Hf + 1) + ny * __ldg(Hf + 4)) + nz * __ldg(Hf + 7))) - yi);
        g.dz = (float)((xj[2] + ((nx * __ldg(Hf + 2) + ny * __ldg(Hf + 5)) + nz * __ldg(Hf + 8))) - zi);
    } else if (a.tri) {        // general cell: the image offset is n . H
        g.dx = (float)((xj[0] + ((nx * a.H[0] + ny * a.H[3]) + nz * a.H[6])) - xi);
        g.dy = (float)((xj[1] + ((nx * a.H[1] + ny * a.H[4]) + nz * a.H[7])) - yi);
        g.dz = (float)((xj[2] + ((nx * a.H[2] + ny * a.H[5]) + nz * a.H[8])) - zi);
    } else {
        g.dx = (float)((xj[0] + nx * a.Lx) - xi);
        g.dy = (float)((xj[1] + ny * a.Ly) - yi);
        g.dz = (float)((xj[2] + nz * a.Lz) - zi);
    }
    const float r2 = g.dx * g.dx + g.dy * g.dy + g.dz * g.dz + kEpsReg * kEpsReg;
    g.rho = sqrtf(r2);
    if (!(g.rho < a.d.rc)) return g;       // skin-shell edge: zero weight
    g.valid = true;
    g.inv_rho = 1.0f / g.rho;
    g.ux = g.dx * g.inv_rho; g.uy = g.dy * g.inv_rho; g.uz = g.dz * g.inv_rho;
    const float inv_rc = 1.0f / a.d.rc;
    const float x = g.rho * inv_rc, t = 1.0f - x;
    const float t2 = t * t, x2 = x * x;
    const float poly = 1.0f + x * (4.0f + x * (10.0f + x * (20.0f + 35.0f * x)));
    g.chi = t2 * t2 * poly;
    g.dchi = -280.0f * x2 * x2 * t2 * t * inv_rc;
    int row = (int)(g.rho * a.d.inv_dx);
    row = row < a.d.n_rows - 1 ? row : a.d.n_rows - 1;
    g.row = row;
    g.t = g.rho - (float)row * a.d.dx;
    if (a.table_uni) {
        // per-pair amplitude tables, one after another: the pair selects the table (ti is
        // already the compact index of the centre's species)
        if (a.n_present > 1) {           // with one species there is one table and no lookup
            g.pair = ti * a.n_present + a.species_slot[tj];
            g.row += g.pair * a.d.n_rows;
        }
    } else {
        g.pair = ti * a.d.T + tj;
    }
    return g;
}

template <int L>
__device__ __forceinline__ void harmonics_s1(float x, float y, float z, float* B1, float* B2, float* B3, float* B4) {
    const float r3 = 1.7320508075688772f;
    B1[0] = x; B1[1] = y; B1[2] = z;
    B2[0] = r3 * x * y; B2[1] = r3 * y * z; B2[2] = 0.5f * (3.0f * z * z - 1.0f); B2[3] = r3 * x * z;
    B2[4] = 0.5f * r3 * (x * x - y * y);
    if (L >= 3) {
        const float a = 0.7905694150420949f, b = 3.872983346207417f, c = 0.6123724356957945f;
        B3[0] = a * y * (3.0f * x * x - y * y);
        B3[1] = b * x * y * z;
        B3[2] = c * y * (5.0f * z * z - 1.0f);
        B3[3] = 0.5f * z * (5.0f * z * z - 3.0f);
        B3[4] = c * x * (5.0f * z * z - 1.0f);
        B3[5] = 0.5f * b * z * (x * x - y * y);
        B3[6] = a * x * (x * x - 3.0f * y * y);
    }
    if (L >= 4) {   // degree four of the supplementary note, |u|^2 = 1
        const float xx = x * x, yy = y * y, zz = z * z;
        const float a0 = 2.958039891549808f, a1 = 2.0916500663351889f, a2 = 1.118033988749895f, a3 = 0.7905694150420949f,
                    a6 = 0.5590169943749475f, a8 = 0.739509972887452f;
        B4[0] = a0 * x * y * (xx - yy);
        B4[1] = a1 * y * z * (3.0f * xx - yy);
        B4[2] = a2 * x * y * (7.0f * zz - 1.0f);
        B4[3] = a3 * y * z * (7.0f * zz - 3.0f);
        B4[4] = 0.125f * (35.0f * zz * zz - 30.0f * zz + 3.0f);
        B4[5] = a3 * x * z * (7.0f * zz - 3.0f);
        B4[6] = a6 * (xx - yy) * (7.0f * zz - 1.0f);
        B4[7] = a1 * x * z * (xx - 3.0f * yy);
        B4[8] = a8 * (xx * xx - 6.0f * xx * yy + yy * yy);
    }
}

// sum over l >= 1 of t_lm * grad_u B_lm (|u|^2 = 1 convention)
template <int L>
__device__ __forceinline__ void harmonics_grad_contract(float x, float y, float z, const float* t1,
                                                        const float* t2, const float* t3, const float* t4, float* gx,
                                                        float* gy, float* gz) {
    const float r3 = 1.7320508075688772f;
    float ax = t1[0], ay = t1[1], az = t1[2];
    ax += r3 * (t2[0] * y + t2[3] * z + t2[4] * x);
    ay += r3 * (t2[0] * x + t2[1] * z - t2[4] * y);
    az += r3 * (t2[1] * y + t2[3] * x) + 3.0f * t2[2] * z;
    if (L >= 3) {
        const float a = 0.7905694150420949f, b = 3.872983346207417f, c = 0.6123724356957945f;
        const float xx = x * x, yy = y * y, zz = z * z;
        ax += t3[0] * (6.0f * a * x * y) + t3[1] * (b * y * z) + t3[4] * (c * (5.0f * zz - 1.0f)) +
              t3[5] * (b * x * z) + t3[6] * (3.0f * a * (xx - yy));
        ay += t3[0] * (3.0f * a * (xx - yy)) + t3[1] * (b * x * z) + t3[2] * (c * (5.0f * zz - 1.0f)) -
              t3[5] * (b * y * z) - t3[6] * (6.0f * a * x * y);
        az += t3[1] * (b * x * y) + t3[2] * (10.0f * c * y * z) + t3[3] * (0.5f * (15.0f * zz - 3.0f)) +
              t3[4] * (10.0f * c * x * z) + t3[5] * (0.5f * b * (xx - yy));
    }
    if (L >= 4) {
        const float xx = x * x, yy = y * y, zz = z * z;
        const float a0 = 2.958039891549808f, a1 = 2.0916500663351889f, a2 = 1.118033988749895f, a3 = 0.7905694150420949f,
                    a6 = 0.5590169943749475f, a8 = 0.739509972887452f;
        const float s7 = 7.0f * zz - 1.0f, s73 = 7.0f * zz - 3.0f, s21 = 21.0f * zz - 3.0f;
        ax += t4[0] * (a0 * y * (3.0f * xx - yy)) + t4[1] * (6.0f * a1 * x * y * z) + t4[2] * (a2 * y * s7) + t4[5] * (a3 * z * s73) +
              t4[6] * (2.0f * a6 * x * s7) + t4[7] * (3.0f * a1 * z * (xx - yy)) + t4[8] * (4.0f * a8 * x * (xx - 3.0f * yy));
        ay += t4[0] * (a0 * x * (xx - 3.0f * yy)) + t4[1] * (3.0f * a1 * z * (xx - yy)) + t4[2] * (a2 * x * s7) + t4[3] * (a3 * z * s73) -
              t4[6] * (2.0f * a6 * y * s7) - t4[7] * (6.0f * a1 * x * y * z) + t4[8] * (4.0f * a8 * y * (yy - 3.0f * xx));
        az += t4[1] * (a1 * y * (3.0f * xx - yy)) + t4[2] * (14.0f * a2 * x * y * z) + t4[3] * (a3 * y * s21) +
              t4[4] * (z * (17.5f * zz - 7.5f)) + t4[5] * (a3 * x * s21) + t4[6] * (14.0f * a6 * z * (xx - yy)) +
              t4[7] * (a1 * x * (xx - 3.0f * yy));
    }
    *gx = ax; *gy = ay; *gz = az;
}

// value (and derivative) of four consecutive table channels at offset t in row `row`: three
// 16-byte loads, c0, c1 and the packed (c2, c3) words with steps k2, k3 (common.cuh, tab_pack)
template <bool DERIV>
__device__ __forceinline__ void table_eval4(const float* __restrict__ table, int CP, int row, int c, float t,
                                            float k2, float k3, float* v, float* dv) {
    const float* p = table + (size_t)row * 3 * CP + c;
    const float4 c0 = ldg4(p), c1 = ldg4(p + CP);
    const int4 w = __ldg(reinterpret_cast<const int4*>(p + 2 * CP));
    const float u2 = k2 * t * t, u3 = k3 * t * t * t;           // c2 t^2 = I2 u2, c3 t^3 = I3 u3
    const float v2 = 2.0f * k2 * t, v3 = 3.0f * k3 * t * t;
#define UMLMD_PIECE(k, f)                                                                              \
    {                                                                                                  \
        const float i2 = (float)(w.f >> 12), i3 = (float)((w.f << 20) >> 20);                          \
        v[k] = fmaf(i3, u3, fmaf(i2, u2, fmaf(c1.f, t, c0.f)));                                        \
        if (DERIV) dv[k] = fmaf(i3, v3, fmaf(i2, v2, c1.f));                                           \
    }
    UMLMD_PIECE(0, x) UMLMD_PIECE(1, y) UMLMD_PIECE(2, z) UMLMD_PIECE(3, w)
#undef UMLMD_PIECE
}

template <bool DERIV>
__device__ __forceinline__ void table_eval1(const float* __restrict__ table, int CP, int row, int c, float t,
                                            float k2, float k3, float* v, float* dv) {
    const float* p = table + (size_t)row * 3 * CP + c;
    const float c0 = __ldg(p), c1 = __ldg(p + CP);
    const int w = __ldg(reinterpret_cast<const int*>(p + 2 * CP));
    const float i2 = (float)(w >> 12), i3 = (float)((w << 20) >> 20);
    *v = fmaf(i3, k3 * t * t * t, fmaf(i2, k2 * t * t, fmaf(c1, t, c0)));
    if (DERIV) *dv = fmaf(i3, 3.0f * k3 * t * t, fmaf(i2, 2.0f * k2 * t, c1));
}

// Shared radial modes q_mu(rho) (and derivatives) of the first nb queued edges, one (edge, mode)
// pair per lane, parked as qm[edge * kMaxR + mu]: evaluated once per edge here instead of once
// per lane in the channel-parallel phase.
template <bool DERIV>
__device__ __forceinline__ void eval_modes(const EdgeArgs& a, const int4* qes, int nb, int lane, float* qm, float* dqm) {
    const int R = a.d.R;
    for (int idx = lane; idx < nb * R; idx += 32) {
        const int b = idx / R, q = idx - b * R;
        const int4 es = qes[b];
        float qv, dqv = 0.f;
        table_eval1<DERIV>(a.table, a.d.CP, es.x, a.d.C0 + q, __int_as_float(es.z), a.d.tab_k2, a.d.tab_k3, &qv, &dqv);
        qm[b * kMaxR + q] = qv;
        if (DERIV) dqm[b * kMaxR + q] = dqv;
    }
}

// amplitude psi (and d psi / d rho) of this lane's four channels for one edge; qm / dqm: the
// edge's parked radial modes (only read when HASR).  UNI: psi_c(rho) of every ordered pair of
// species present is tabulated by itself (a.table_uni, row pitch C0; `row` already points into
// the edge's pair), so neither pair rows nor modes are read.  k2, k3: steps of the packed
// coefficients of the table that is read
template <int C0, bool HASR, bool DERIV, bool UNI>
__device__ __forceinline__ void amplitude4(const EdgeArgs& a, int row, float t, int pair, int c, float* psi,
                                           float* dpsi, const float* qm, const float* dqm, float k2, float k3) {
    if (UNI) {
        table_eval4<DERIV>(a.table_uni, C0, row, c, t, k2, k3, psi, dpsi);
        return;
    }
    float g[4], dg[4];
    table_eval4<DERIV>(a.table, a.d.CP, row, c, t, k2, k3, g, dg);
    const int R = HASR ? a.d.R : 0;
    const float* pm = a.pairmod + (size_t)pair * (2 + R) * C0 + c;
    const float4 ga = ldg4(pm), be = ldg4(pm + C0);
    psi[0] = ga.x * g[0] + be.x; psi[1] = ga.y * g[1] + be.y;
    psi[2] = ga.z * g[2] + be.z; psi[3] = ga.w * g[3] + be.w;
    if (DERIV) { dpsi[0] = ga.x * dg[0]; dpsi[1] = ga.y * dg[1]; dpsi[2] = ga.z * dg[2]; dpsi[3] = ga.w * dg[3]; }
    if (HASR) {
        float qv[kMaxR], dqv[kMaxR];
        {
            const float4 v0 = *reinterpret_cast<const float4*>(qm);
            qv[0] = v0.x; qv[1] = v0.y; qv[2] = v0.z; qv[3] = v0.w;
            if (R > 4) { const float4 v1 = *reinterpret_cast<const float4*>(qm + 4); qv[4] = v1.x; qv[5] = v1.y; qv[6] = v1.z; qv[7] = v1.w; }
            if (DERIV) {
                const float4 d0 = *reinterpret_cast<const float4*>(dqm);
                dqv[0] = d0.x; dqv[1] = d0.y; dqv[2] = d0.z; dqv[3] = d0.w;
                if (R > 4) { const float4 d1 = *reinterpret_cast<const float4*>(dqm + 4); dqv[4] = d1.x; dqv[5] = d1.y; dqv[6] = d1.z; dqv[7] = d1.w; }
            }
        }
#pragma unroll
        for (int q = 0; q < kMaxR; ++q) {
            if (q >= R) break;
            const float4 U = ldg4(pm + (size_t)(2 + q) * C0);
            psi[0] += U.x * qv[q]; psi[1] += U.y * qv[q]; psi[2] += U.z * qv[q]; psi[3] += U.w * qv[q];
            if (DERIV) { dpsi[0] += U.x * dqv[q]; dpsi[1] += U.y * dqv[q]; dpsi[2] += U.z * dqv[q]; dpsi[3] += U.w * dqv[q]; }
        }
    }
}

// G = groups of four channels a lane holds in the channel-parallel phase (group g starts at
// channel 4 * lane_in_group + g * C0 / G, so every 16-byte load instruction of a group of lanes
// still covers one contiguous segment)
template <int C0, int L, int G = 1> struct Widths {
    static constexpr int C1 = C0 <= 16 ? 4 : (C0 <= 64 ? 8 : 16);
    static constexpr int C2 = C1 / 2 > 4 ? C1 / 2 : 4;
    static constexpr int LPE = C0 / (4 * G);    // lanes per edge in the channel-parallel phase
    static constexpr int GOFF = C0 / G;         // channel offset between a lane's groups
    static constexpr int LH = LPE / 2;          // parked partial dot products per edge (lanes paired)
    static constexpr int EPI = 32 / LPE;        // edges per replay step
    static constexpr int NL1 = C1 / 4;          // lanes of a group that hold degree-1 channels
    static constexpr int NHI = 3 * C1 + 5 * C2 + (L >= 3 ? 7 : 0) + (L >= 4 ? 9 : 0);   // sums of degree >= 1
    static constexpr int NCH = (NHI + 31) / 32;
    // row pitch (floats) of the per-edge amplitude staging; pitch/4 odd keeps 16-byte
    // accesses of 8 consecutive lanes on distinct bank groups
    // (forward, C0 = 128: a whole warp works on one edge, rows are written one or two at a time and
    // read one at a time, so no padding is needed, and with degree 4 none fits in 48 KB)
    static constexpr int PF = C0 / (4 * G) == 32 ? C1 : (((C1 / 4 + 1) & 1) ? C1 + 4 : C1 + 8);   // forward: psi
    static constexpr int PB = ((2 * C1 / 4 + 1) & 1) ? 2 * C1 + 4 : 2 * C1 + 8;   // backward: psi, dpsi
    // forward, sums of degree >= 1: a job is four consecutive channels of one harmonic component
    // (degrees 1 and 2) or one component of a one-channel degree (3, 4); a lane owns up to SLOTS jobs
    static constexpr int J1 = 3 * (C1 / 4), J2 = 5 * (C2 / 4), J3 = L >= 3 ? 7 : 0, J4 = L >= 4 ? 9 : 0;
    static constexpr int NJ = J1 + J2 + J3 + J4;
    static constexpr int SLOTS = (NJ + 31) / 32;
    static constexpr int NM = 3 + 5 + J3 + J4;  // harmonic components of all degrees >= 1
    static constexpr int PW = NM | 1;           // odd row pitch of the parked weights
    static constexpr int WOFF = 32 * PF;        // they sit behind the parked amplitudes (where the radial modes were)
    static constexpr int SCRATCH = 32 * PF + (32 * PW > 32 * kMaxR ? 32 * PW : 32 * kMaxR);
};

// The channel-parallel phase of the backward pass waits on load latency, and what hides it best
// depends on the width (all measured on the edge backward kernel).  C0 = 128: four channel groups
// per lane, that many times the table and pair loads in flight, at 16 resident warps per SM (128
// registers): 10 % faster than two groups, and than two groups at 24 warps.  C0 = 32 and 64:
// two groups at 24 warps (85 registers, a few spilled words): 9-13 % faster than 16 warps,
// four groups being slower again.  C0 <= 16: one group, 24 warps (13 % faster than 16).
template <int C0> struct BwdGroups { static constexpr int G = C0 >= 128 ? 4 : (C0 >= 32 ? 2 : 1); };

template <int C0, int L, bool HASR> struct BwdSmem {          // dynamic shared memory of the backward kernel
    using W = Widths<C0, L, BwdGroups<C0>::G>;
    static constexpr int queue_floats = 32 * 4 + 5 * 32;    // queue of in-range edges: int4 and five scalars per slot
    static constexpr int mode_floats = HASR ? 2 * 32 * kMaxR : 0;   // parked radial modes and their derivatives
    static constexpr int per_warp = (32 * W::PB + 2 * 32 * (W::LH + 1) + W::NHI + 3) / 4 * 4 + mode_floats + queue_floats;   // floats
    static constexpr size_t bytes = kWarpsPerBlock * 9 * sizeof(double) + sizeof(float) * kWarpsPerBlock * per_warp;
};

// ------------------------------------------------------------------------------- forward
//
// The row is scanned 32 listed edges at a time (lane = edge: geometry); the edges that fall
// inside the cutoff are appended to a 32-slot per-warp queue in shared memory (edges that do
// not fit wait in their lane's registers), and whenever 32 are there (and once more at the end
// of the row) a full batch is processed, so the later phases never run on skin-shell edges:
//   2. lanes = channels (a group of C0/4 lanes per edge): amplitude psi of all C0 channels,
//      degree-0 sums accumulated in registers; the leading C1 amplitudes of each edge are
//      parked in shared memory.
//   3. lane = edge again: harmonics of the lane's own edge, parked as weights chi^2 B_lm; then
//      lane = job: a lane owns four consecutive channels of one harmonic component (or one
//      component of a one-channel degree) for the whole row, and for every edge of the batch adds
//      weight x amplitudes from the two parked rows: two shared-memory reads per edge and warp,
//      where summing per-edge products by transposition took six.
// Up to C0 = 64 a fourth group of eight resident warps per SM (64 registers, a few spilled words) is worth more
// than the registers: the channel-parallel phase waits on load latency (measured: 6-10 % on the
// forward kernel at C0 = 8 .. 64, 2 % the other way at C0 = 128, which stays at 24 warps).
template <int C0, int L, bool HASR, bool UNI>
__global__ void __launch_bounds__(kWarpsPerBlock * 32, (C0 <= 64 ? 4 : 3) * 8 / kWarpsPerBlock)
k_edge_forward(const EdgeArgs a) {
    using W = Widths<C0, L>;
    // scratch per warp: the parked amplitudes of the batch (row pitch PF), and behind them first the
    // radial modes, then (once the amplitudes are done) the harmonic weights chi^2 B_lm (row pitch PW)
    __shared__ __align__(16) float scratch[kWarpsPerBlock][W::SCRATCH];
    // queue of edges inside the cutoff: row, pair, t, chi (fetched with one 16-byte broadcast
    // load in the channel-parallel phase; shuffles would go through the same L1 data pipe as
    // the table reads) and the edge vector
    __shared__ int4 q_es[kWarpsPerBlock][32];
    __shared__ float q_d[kWarpsPerBlock][3 * 32];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int i = a.a0 + blockIdx.x * kWarpsPerBlock + wid;
    if (i >= a.a1) return;
    float* const psi_s = scratch[wid];      // [32][PF]
    float* const qm = scratch[wid] + W::WOFF;      // [32][kMaxR] radial modes, behind the parked amplitudes
    float* const wbs = scratch[wid] + W::WOFF;     // [32][PW] harmonic weights, in the same place later
    int4* const qes = q_es[wid];
    float* const qd = q_d[wid];
    const int sub = lane / W::LPE, cl = lane % W::LPE, c = 4 * cl;
    const double xi = a.xs[3 * (size_t)i], yi = a.xs[3 * (size_t)i + 1], zi = a.xs[3 * (size_t)i + 2];
    const int ti = UNI ? a.species_slot[a.type_s[i]] : a.type_s[i];
    const float k2 = UNI ? tab_step2(__ldg(a.uni_scale)) : a.d.tab_k2, k3 = UNI ? tab_step3(__ldg(a.uni_scale + 1)) : a.d.tab_k3;
    const eidx_t e0 = a.row_ptr[i];
    const int len = (int)(a.row_ptr[i + 1] - e0);      // edge offsets are 64-bit, offsets inside a row are not
    const double* Hf = a.frames ? a.frames[a.frame_of[i]].H : nullptr;
    const unsigned lt_mask = (1u << lane) - 1u;
    float acc0[4] = {0.f, 0.f, 0.f, 0.f};
    // this lane's jobs of the degree >= 1 sums: offset of the four channels in an amplitude row,
    // of the component in a weight row, of the result in the output block (negative: no job)
    float accJ[W::SLOTS][4];
    int j_psi[W::SLOTS], j_w[W::SLOTS], j_out[W::SLOTS];
#pragma unroll
    for (int sl = 0; sl < W::SLOTS; ++sl) {
        accJ[sl][0] = accJ[sl][1] = accJ[sl][2] = accJ[sl][3] = 0.f;
        const int j = lane + 32 * sl;
        if (j < W::J1) {
            const int m = j / (W::C1 / 4), cb = j % (W::C1 / 4);
            j_psi[sl] = 4 * cb; j_w[sl] = m; j_out[sl] = m * W::C1 + 4 * cb;
        } else if (j < W::J1 + W::J2) {
            const int jj = j - W::J1, m = jj / (W::C2 / 4), cb = jj % (W::C2 / 4);
            j_psi[sl] = 4 * cb; j_w[sl] = 3 + m; j_out[sl] = 3 * W::C1 + m * W::C2 + 4 * cb;
        } else if (j < W::NJ) {
            const int m = j - W::J1 - W::J2;             // degrees 3 and 4 follow each other in both layouts
            j_psi[sl] = 0; j_w[sl] = 8 + m; j_out[sl] = 3 * W::C1 + 5 * W::C2 + m;
        } else {
            j_psi[sl] = 0; j_w[sl] = 0; j_out[sl] = -1;
        }
    }
    double s0 = 0.0, s1 = 0.0;   // normaliser sums in double: the calibration subtracts their mean

    auto run_batch = [&](const int nb) {     // the first nb queue slots
        if (HASR) {
            eval_modes<false>(a, qes, nb, lane, qm, nullptr);
            __syncwarp();
        }
        int it = 0;
        if (W::EPI == 1 && !HASR) {
            // whole warp per edge: two edges per step, so that twelve 16-byte table and pair
            // loads are in flight per lane instead of six (the phase waits on their latency)
            for (; it + 1 < nb; it += 2) {
                const int4 ea = qes[it], eb = qes[it + 1];
                float pa[4], pb[4];
                amplitude4<C0, HASR, false, UNI>(a, ea.x, __int_as_float(ea.z), ea.y, c, pa, nullptr, nullptr, nullptr, k2, k3);
                amplitude4<C0, HASR, false, UNI>(a, eb.x, __int_as_float(eb.z), eb.y, c, pb, nullptr, nullptr, nullptr, k2, k3);
                const float ca = __int_as_float(ea.w), cb = __int_as_float(eb.w);
#pragma unroll
                for (int k = 0; k < 4; ++k) acc0[k] += ca * pa[k];
#pragma unroll
                for (int k = 0; k < 4; ++k) acc0[k] += cb * pb[k];
                if (cl < W::NL1) {
                    *reinterpret_cast<float4*>(psi_s + it * W::PF + c) = make_float4(pa[0], pa[1], pa[2], pa[3]);
                    *reinterpret_cast<float4*>(psi_s + (it + 1) * W::PF + c) = make_float4(pb[0], pb[1], pb[2], pb[3]);
                }
            }
        }
        for (; it * W::EPI < nb; ++it) {
            const int b = it * W::EPI + sub;
            if (b >= nb) continue;
            const int4 es = qes[b];
            const int row = es.x, pair = es.y;
            const float t = __int_as_float(es.z), chi = __int_as_float(es.w);
            float psi[4];
            amplitude4<C0, HASR, false, UNI>(a, row, t, pair, c, psi, nullptr, qm + b * kMaxR, nullptr, k2, k3);
#pragma unroll
            for (int k = 0; k < 4; ++k) acc0[k] += chi * psi[k];
            if (cl < W::NL1)
                *reinterpret_cast<float4*>(psi_s + b * W::PF + c) = make_float4(psi[0], psi[1], psi[2], psi[3]);
        }
        __syncwarp();
        // lane = edge: the harmonic weights chi^2 B_lm of the lane's edge, parked next to the amplitudes
        if (lane < nb) {
            float B1[3], B2[5], B3[7], B4[9];
            const float dx = qd[lane], dy = qd[32 + lane], dz = qd[64 + lane];
            const float inv_rho = 1.0f / sqrtf(dx * dx + dy * dy + dz * dz + kEpsReg * kEpsReg);
            harmonics_s1<L>(dx * inv_rho, dy * inv_rho, dz * inv_rho, B1, B2, B3, B4);
            const float chi = __int_as_float(qes[lane].w);
            const float w = chi * chi;
            float* wr = wbs + lane * W::PW;
#pragma unroll
            for (int m = 0; m < 3; ++m) wr[m] = w * B1[m];
#pragma unroll
            for (int m = 0; m < 5; ++m) wr[3 + m] = w * B2[m];
            if (L >= 3) {
#pragma unroll
                for (int m = 0; m < 7; ++m) wr[8 + m] = w * B3[m];
            }
            if (L >= 4) {
#pragma unroll
                for (int m = 0; m < 9; ++m) wr[15 + m] = w * B4[m];
            }
        }
        __syncwarp();
        // lane = job: the sums over the batch stay in the lane's registers for the whole row; per edge
        // a lane reads its four amplitudes and its weight (every lane inside the same two rows)
#pragma unroll 4
        for (int e = 0; e < nb; ++e) {
#pragma unroll
            for (int sl = 0; sl < W::SLOTS; ++sl) {
                const float4 p4 = *reinterpret_cast<const float4*>(psi_s + e * W::PF + j_psi[sl]);
                const float wv = wbs[e * W::PW + j_w[sl]];
                accJ[sl][0] += wv * p4.x; accJ[sl][1] += wv * p4.y; accJ[sl][2] += wv * p4.z; accJ[sl][3] += wv * p4.w;
            }
        }
        __syncwarp();                           // the next batch overwrites both
    };

    int qn = 0;
    for (int base = 0; base < len; base += 32) {
        const Geom g = edge_geometry(a, e0 + base + lane, base + lane < len, xi, yi, zi, ti, Hf);
        const unsigned vmask = __ballot_sync(kFull, g.valid);
        const int p = qn + __popc(vmask & lt_mask);       // queue slot of this lane's edge, if it has one
        if (g.valid) { const double c2 = (double)g.chi * (double)g.chi; s0 += c2; s1 += c2 * c2; }
        if (g.valid && p < 32) {
            qes[p] = make_int4(g.row, g.pair, __float_as_int(g.t), __float_as_int(g.chi));
            qd[p] = g.dx; qd[32 + p] = g.dy; qd[64 + p] = g.dz;
        }
        qn += __popc(vmask);
        __syncwarp();
        if (qn >= 32) {                                   // a full batch; the overflow waits in registers
            run_batch(32);
            if (g.valid && p >= 32) {
                qes[p - 32] = make_int4(g.row, g.pair, __float_as_int(g.t), __float_as_int(g.chi));
                qd[p - 32] = g.dx; qd[p] = g.dy; qd[32 + p] = g.dz;
            }
            qn -= 32;
            __syncwarp();
        }
    }
    if (qn > 0) run_batch(qn);
    // combine the edge slots of the warp (lanes with equal channel offset)
#pragma unroll
    for (int off = W::LPE; off < 32; off <<= 1) {
#pragma unroll
        for (int k = 0; k < 4; ++k) acc0[k] += __shfl_xor_sync(kFull, acc0[k], off);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        s0 += __shfl_xor_sync(kFull, s0, off);
        s1 += __shfl_xor_sync(kFull, s1, off);
    }
    float* row_out = a.state + (size_t)(i - a.a0) * a.d.SP;
    if (sub == 0) *reinterpret_cast<float4*>(row_out + c) = make_float4(acc0[0], acc0[1], acc0[2], acc0[3]);
#pragma unroll
    for (int sl = 0; sl < W::SLOTS; ++sl) {
        if (j_out[sl] < 0) continue;
        float* o = row_out + a.d.offA[1] + j_out[sl];
        if (lane + 32 * sl < W::J1 + W::J2) *reinterpret_cast<float4*>(o) = make_float4(accJ[sl][0], accJ[sl][1], accJ[sl][2], accJ[sl][3]);
        else o[0] = accJ[sl][0];
    }
    if (lane == 0) {
        const float h0 = (float)s0, h1 = (float)s1;
        row_out[a.d.S] = h0; row_out[a.d.S + 1] = h1;
        row_out[a.d.S + 2] = (float)(s0 - (double)h0); row_out[a.d.S + 3] = (float)(s1 - (double)h1);
    }
}

// ------------------------------------------------------------------------------ backward
//
// Same scan, queue and phases.  The channel-parallel phase produces, per edge, the two
// degree-0 dot products sum_c G0_c psi_c and sum_c G0_c dpsi_c (partial sums parked in shared
// memory and finished by the edge's own lane) and parks psi, dpsi of the leading C1 channels;
// the edge's lane then does the whole degree >= 1 contraction by itself against the
// destination's gradient block held in shared memory, and assembles dE/dr_ij.  Edges in the
// skin shell get a zero gradient as soon as their geometry is known.
template <int C0, int L, bool HASR, bool UNI>
__global__ void __launch_bounds__(kWarpsPerBlock * 32, (C0 <= 64 ? 3 : 2) * 8 / kWarpsPerBlock)
k_edge_backward(const EdgeArgs a) {
    constexpr int G = BwdGroups<C0>::G;
    using W = Widths<C0, L, G>;
    extern __shared__ __align__(16) unsigned char dsm[];
    double (*vsum)[9] = reinterpret_cast<double (*)[9]>(dsm);
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    float* const wbase = reinterpret_cast<float*>(dsm + kWarpsPerBlock * 9 * sizeof(double)) + wid * BwdSmem<C0, L, HASR>::per_warp;
    float* const psi_s = wbase;                                  // [32][PB]: psi, dpsi of the leading channels
    float* const red = psi_s + 32 * W::PB;                       // [2][32][LH+1] partial dot products
    float* const hi_s = red + 2 * 32 * (W::LH + 1);              // [NHI] gradient of the degree >= 1 sums
    // queue of edges inside the cutoff: (row, pair, t, chi), then dx, dy, dz, dchi, edge index
    int4* const qes = reinterpret_cast<int4*>(wbase + BwdSmem<C0, L, HASR>::per_warp - BwdSmem<C0, L, HASR>::queue_floats);
    float* const qm = reinterpret_cast<float*>(qes) - BwdSmem<C0, L, HASR>::mode_floats;   // [2][32][kMaxR]
    float* const qd = reinterpret_cast<float*>(qes + 32);        // [5][32]
    const int i = a.a0 + blockIdx.x * kWarpsPerBlock + wid;
    const bool active = i < a.a1;
    const int sub = lane / W::LPE, cl = lane % W::LPE, c = 4 * cl;
    const unsigned lt_mask = (1u << lane) - 1u;
    float vir[9];
#pragma unroll
    for (int k = 0; k < 9; ++k) vir[k] = 0.f;

    if (active) {
        const double xi = a.xs[3 * (size_t)i], yi = a.xs[3 * (size_t)i + 1], zi = a.xs[3 * (size_t)i + 2];
        const int ti = UNI ? a.species_slot[a.type_s[i]] : a.type_s[i];
        const float k2 = UNI ? tab_step2(__ldg(a.uni_scale)) : a.d.tab_k2, k3 = UNI ? tab_step3(__ldg(a.uni_scale + 1)) : a.d.tab_k3;
        const eidx_t e0 = a.row_ptr[i];
        const int len = (int)(a.row_ptr[i + 1] - e0);
        const double* Hf = a.frames ? a.frames[a.frame_of[i]].H : nullptr;
        const float* grow = a.state + (size_t)(i - a.a0) * a.d.SP;
        float h0[4 * G];
#pragma unroll
        for (int gq = 0; gq < G; ++gq) {
            const float4 v = *reinterpret_cast<const float4*>(grow + c + gq * W::GOFF);
            h0[4 * gq] = v.x; h0[4 * gq + 1] = v.y; h0[4 * gq + 2] = v.z; h0[4 * gq + 3] = v.w;
        }
        for (int v = lane; v < W::NHI; v += 32) hi_s[v] = grow[a.d.offA[1] + v];
        const float ds0 = grow[a.d.S], ds1 = grow[a.d.S + 1];
        __syncwarp();
        const float* H1 = hi_s;
        const float* H2 = H1 + 3 * W::C1;
        const float* H3 = H2 + 5 * W::C2;
        const float* H4 = H3 + (L >= 3 ? 7 : 0);

        auto run_batch = [&](const int nb) {     // the first nb queue slots
            if (HASR) {
                eval_modes<true>(a, qes, nb, lane, qm, qm + 32 * kMaxR);
                __syncwarp();
            }
            for (int it = 0; it * W::EPI < nb; ++it) {
                const int b = it * W::EPI + sub;
                const bool act = b < nb;
                float pa = 0.f, pb = 0.f;
                if (act) {
                    const int4 es = qes[b];
                    const int row = es.x, pair = es.y;
                    const float t = __int_as_float(es.z);
                    float psi[4 * G], dpsi[4 * G];
#pragma unroll
                    for (int gq = 0; gq < G; ++gq)
                        amplitude4<C0, HASR, true, UNI>(a, row, t, pair, c + gq * W::GOFF, psi + 4 * gq, dpsi + 4 * gq,
                                                        qm + b * kMaxR, qm + (32 + b) * kMaxR, k2, k3);
#pragma unroll
                    for (int k = 0; k < 4 * G; ++k) { pa += h0[k] * dpsi[k]; pb += h0[k] * psi[k]; }
                    if (cl < W::NL1) {       // the leading C1 channels all sit in group 0
                        *reinterpret_cast<float4*>(psi_s + b * W::PB + c) = make_float4(psi[0], psi[1], psi[2], psi[3]);
                        *reinterpret_cast<float4*>(psi_s + b * W::PB + W::C1 + c) = make_float4(dpsi[0], dpsi[1], dpsi[2], dpsi[3]);
                    }
                }
                // neighbouring lanes are paired before the partial sums are parked, which halves
                // the parking area (it decides how many blocks fit on an SM)
                pa += __shfl_xor_sync(kFull, pa, 1);
                pb += __shfl_xor_sync(kFull, pb, 1);
                if (act && !(cl & 1)) {
                    red[b * (W::LH + 1) + (cl >> 1)] = pa;
                    red[(32 + b) * (W::LH + 1) + (cl >> 1)] = pb;
                }
            }
            __syncwarp();
            if (lane < nb) {
                const float gdx = qd[lane], gdy = qd[32 + lane], gdz = qd[64 + lane], dchi = qd[96 + lane];
                const int e = __float_as_int(qd[128 + lane]);       // offset inside the row
                const float chi = __int_as_float(qes[lane].w);
                const float inv_rho = 1.0f / sqrtf(gdx * gdx + gdy * gdy + gdz * gdz + kEpsReg * kEpsReg);
                const float gux = gdx * inv_rho, guy = gdy * inv_rho, guz = gdz * inv_rho;
                float sa = 0.f, sb = 0.f;
#pragma unroll
                for (int j = 0; j < W::LH; ++j) { sa += red[lane * (W::LH + 1) + j]; sb += red[(32 + lane) * (W::LH + 1) + j]; }
                float ps[W::C1], dps[W::C1], ec[W::C1];
#pragma unroll
                for (int q = 0; q < W::C1 / 4; ++q) {
                    const float4 p4 = *reinterpret_cast<const float4*>(psi_s + lane * W::PB + 4 * q);
                    const float4 d4 = *reinterpret_cast<const float4*>(psi_s + lane * W::PB + W::C1 + 4 * q);
                    ps[4 * q] = p4.x; ps[4 * q + 1] = p4.y; ps[4 * q + 2] = p4.z; ps[4 * q + 3] = p4.w;
                    dps[4 * q] = d4.x; dps[4 * q + 1] = d4.y; dps[4 * q + 2] = d4.z; dps[4 * q + 3] = d4.w;
                }
#pragma unroll
                for (int k = 0; k < W::C1; ++k) ec[k] = 0.f;
                float B1[3], B2[5], B3[7], B4[9], t1[3], t2[5], t3[7], t4[9];
                harmonics_s1<L>(gux, guy, guz, B1, B2, B3, B4);
                float bt = 0.f;    // sum_lm B_lm t_lm,  t_lm = sum_c psi_c G_lmc
#pragma unroll
                for (int m = 0; m < 3; ++m) {
                    float tm = 0.f;
#pragma unroll
                    for (int k = 0; k < W::C1; ++k) { const float hv = H1[m * W::C1 + k]; tm += ps[k] * hv; ec[k] += B1[m] * hv; }
                    t1[m] = tm; bt += B1[m] * tm;
                }
#pragma unroll
                for (int m = 0; m < 5; ++m) {
                    float tm = 0.f;
#pragma unroll
                    for (int k = 0; k < W::C2; ++k) { const float hv = H2[m * W::C2 + k]; tm += ps[k] * hv; ec[k] += B2[m] * hv; }
                    t2[m] = tm; bt += B2[m] * tm;
                }
#pragma unroll
                for (int m = 0; m < 7; ++m) {
                    float tm = 0.f;
                    if (L >= 3) { const float hv = H3[m]; tm = ps[0] * hv; ec[0] += B3[m] * hv; bt += B3[m] * tm; }
                    t3[m] = tm;
                }
#pragma unroll
                for (int m = 0; m < 9; ++m) {
                    float tm = 0.f;
                    if (L >= 4) { const float hv = H4[m]; tm = ps[0] * hv; ec[0] += B4[m] * hv; bt += B4[m] * tm; }
                    t4[m] = tm;
                }
                const float w = chi * chi;
                float pr1 = 0.f;
#pragma unroll
                for (int k = 0; k < W::C1; ++k) pr1 += ec[k] * dps[k];
                float ux, uy, uz;
                harmonics_grad_contract<L>(gux, guy, guz, t1, t2, t3, t4, &ux, &uy, &uz);
                const float pux = w * ux, puy = w * uy, puz = w * uz;
                const float p_rho = chi * sa + w * pr1;
                const float p_chi = sb + 2.0f * chi * bt;
                const float dEdrho = p_rho + (p_chi + 2.0f * chi * ds0 + 4.0f * w * chi * ds1) * dchi;
                const float dot = pux * gux + puy * guy + puz * guz;
                const float gx = dEdrho * gux + (pux - dot * gux) * inv_rho;
                const float gy = dEdrho * guy + (puy - dot * guy) * inv_rho;
                const float gz = dEdrho * guz + (puz - dot * guz) * inv_rho;
                vir[0] += gx * gdx; vir[1] += gx * gdy; vir[2] += gx * gdz;
                vir[3] += gy * gdx; vir[4] += gy * gdy; vir[5] += gy * gdz;
                vir[6] += gz * gdx; vir[7] += gz * gdy; vir[8] += gz * gdz;
                float* go = a.g + 3 * (size_t)(e0 + e);
                go[0] = gx; go[1] = gy; go[2] = gz;
            }
            __syncwarp();
        };

        int qn = 0;
        for (int base = 0; base < len; base += 32) {
            const int e = base + lane;                                // offset inside the row
            const Geom g = edge_geometry(a, e0 + e, e < len, xi, yi, zi, ti, Hf);
            const unsigned vmask = __ballot_sync(kFull, g.valid);
            const int p = qn + __popc(vmask & lt_mask);   // queue slot of this lane's edge, if it has one
            if (g.valid && p < 32) {
                qes[p] = make_int4(g.row, g.pair, __float_as_int(g.t), __float_as_int(g.chi));
                qd[p] = g.dx; qd[32 + p] = g.dy; qd[64 + p] = g.dz; qd[96 + p] = g.dchi;
                qd[128 + p] = __int_as_float(e);
            } else if (!g.valid && e < len) {
                float* go = a.g + 3 * (size_t)(e0 + e);
                go[0] = 0.f; go[1] = 0.f; go[2] = 0.f;
            }
            qn += __popc(vmask);
            __syncwarp();
            if (qn >= 32) {                               // a full batch; the overflow waits in registers
                run_batch(32);
                if (g.valid && p >= 32) {
                    const int r = p - 32;
                    qes[r] = make_int4(g.row, g.pair, __float_as_int(g.t), __float_as_int(g.chi));
                    qd[r] = g.dx; qd[32 + r] = g.dy; qd[64 + r] = g.dz; qd[96 + r] = g.dchi;
                    qd[128 + r] = __int_as_float(e);
                }
                qn -= 32;
                __syncwarp();
            }
        }
        if (qn > 0) run_batch(qn);
    }
    // block partial of sum_e g (x) r, in double, fixed order
#pragma unroll
    for (int k = 0; k < 9; ++k) {
        double v = (double)vir[k];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(kFull, v, off);
        if (lane == 0) vsum[wid][k] = v;
    }
    __syncthreads();
    if (threadIdx.x < 9) {
        double v = 0.0;
        for (int w = 0; w < kWarpsPerBlock; ++w) v += vsum[w][threadIdx.x];
        a.virial_part[(size_t)blockIdx.x * 9 + threadIdx.x] = v;
    }
}


// per-pair amplitude tables already hold the modes, so the kernels without them are used
template <int C0, int L>
cudaError_t launch_fwd_r(const EdgeArgs& a, int blocks, cudaStream_t st) {
    if (a.table_uni) k_edge_forward<C0, L, false, true><<<blocks, kWarpsPerBlock * 32, 0, st>>>(a);
    else if (a.d.R > 0) k_edge_forward<C0, L, true, false><<<blocks, kWarpsPerBlock * 32, 0, st>>>(a);
    else k_edge_forward<C0, L, false, false><<<blocks, kWarpsPerBlock * 32, 0, st>>>(a);
    return cudaGetLastError();
}
template <int C0, int L>
cudaError_t launch_bwd_r(const EdgeArgs& a, int blocks, cudaStream_t st) {
    const bool hasr = a.d.R > 0 && !a.table_uni;
    const size_t bytes = hasr ? BwdSmem<C0, L, true>::bytes : BwdSmem<C0, L, false>::bytes;
    auto kern = a.table_uni ? k_edge_backward<C0, L, false, true>
                            : (hasr ? k_edge_backward<C0, L, true, false> : k_edge_backward<C0, L, false, false>);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) return e;
    kern<<<blocks, kWarpsPerBlock * 32, bytes, st>>>(a);
    return cudaGetLastError();
}

template <bool FWD>
cudaError_t dispatch(const EdgeArgs& a, int blocks, cudaStream_t st) {
#define UMLMD_CASE(C0v, Lv)                                                       \
    if (a.d.C0 == C0v && a.d.L == Lv)                                             \
        return FWD ? launch_fwd_r<C0v, Lv>(a, blocks, st) : launch_bwd_r<C0v, Lv>(a, blocks, st);
    UMLMD_CASE(8, 2) UMLMD_CASE(8, 3) UMLMD_CASE(16, 2) UMLMD_CASE(16, 3) UMLMD_CASE(32, 2)
    UMLMD_CASE(32, 3) UMLMD_CASE(64, 2) UMLMD_CASE(64, 3) UMLMD_CASE(128, 2) UMLMD_CASE(128, 3)
    UMLMD_CASE(8, 4) UMLMD_CASE(16, 4) UMLMD_CASE(32, 4) UMLMD_CASE(64, 4) UMLMD_CASE(128, 4)
#undef UMLMD_CASE
    return cudaErrorInvalidValue;
}

// Tables of psi_c(rho) = gamma_c g_c(rho) + beta_c + sum_mu U_c,mu q_mu(rho) for the ordered
// pairs (present[a], present[b]), stored as [a * n_present + b][row][3][C0] in the format of the
// radial table: the cubic coefficients are linear in the tabulated functions, so the same
// combination of the coefficient rows of [g, q] gives them.  Two passes: the first finds the
// largest |c2| and |c3| (the scale of the packed words), the second writes the rows.
template <bool WRITE>
__global__ void k_fuse_pair_tables(Dims d, const float* __restrict__ table, const float* __restrict__ pairmod,
                                   const int* __restrict__ present, int n_present, float* __restrict__ scale,
                                   float* __restrict__ out) {
    const int64_t per_pair = (int64_t)d.n_rows * d.C0;
    const int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;   // over [pair][row][c]
    float c2 = 0.f, c3 = 0.f;
    if (idx < per_pair * n_present * n_present) {
        const int pr = (int)(idx / per_pair);
        const int64_t in_pair = idx - pr * per_pair;
        const int c = (int)(in_pair % d.C0);
        const int64_t row = in_pair / d.C0;
        const int si = present[pr / n_present], sj = present[pr % n_present];
        const float* pm = pairmod + (size_t)(si * d.T + sj) * (2 + d.R) * d.C0 + c;
        const float* tr = table + (size_t)row * 3 * d.CP;
        auto coef = [&](int col, double* o) {     // the four coefficients of column col of the radial table
            float h2, h3;
            tab_unpack(__float_as_uint(tr[2 * d.CP + col]), d.tab_k2, d.tab_k3, &h2, &h3);
            o[0] = (double)tr[col]; o[1] = (double)tr[d.CP + col]; o[2] = (double)h2; o[3] = (double)h3;
        };
        double v[4], o[4];
        coef(c, o);
        for (int k = 0; k < 4; ++k) v[k] = (double)pm[0] * o[k];
        v[0] += (double)pm[d.C0];
        for (int q = 0; q < d.R; ++q) {
            coef(d.C0 + q, o);
            const double u = (double)pm[(size_t)(2 + q) * d.C0];
            for (int k = 0; k < 4; ++k) v[k] += u * o[k];
        }
        c2 = (float)v[2]; c3 = (float)v[3];
        if (WRITE) {
            float* orow = out + ((size_t)pr * d.n_rows + row) * 3 * d.C0;
            orow[c] = (float)v[0];
            orow[d.C0 + c] = (float)v[1];
            orow[2 * d.C0 + c] = __uint_as_float(tab_pack(c2, c3, tab_step2(scale[0]), tab_step3(scale[1])));
        }
    }
    if (!WRITE) {        // non-negative floats order like their bit patterns
        float a2 = fabsf(c2), a3 = fabsf(c3);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            a2 = fmaxf(a2, __shfl_xor_sync(0xffffffffu, a2, off));
            a3 = fmaxf(a3, __shfl_xor_sync(0xffffffffu, a3, off));
        }
        if ((threadIdx.x & 31) == 0) {
            atomicMax(reinterpret_cast<unsigned*>(scale), __float_as_uint(a2));
            atomicMax(reinterpret_cast<unsigned*>(scale) + 1, __float_as_uint(a3));
        }
    }
}

}  // namespace

cudaError_t launch_fuse_pair_tables(const Dims& d, const float* table, const float* pairmod, const int* present,
                                    int n_present, float* scale, float* out, cudaStream_t st) {
    const int64_t n = (int64_t)d.n_rows * d.C0 * n_present * n_present;
    if (n == 0) return cudaSuccess;
    cudaError_t e = cudaMemsetAsync(scale, 0, 2 * sizeof(float), st);
    if (e != cudaSuccess) return e;
    const unsigned blocks = (unsigned)((n + 255) / 256);
    k_fuse_pair_tables<false><<<blocks, 256, 0, st>>>(d, table, pairmod, present, n_present, scale, out);
    k_fuse_pair_tables<true><<<blocks, 256, 0, st>>>(d, table, pairmod, present, n_present, scale, out);
    return cudaGetLastError();
}

int edge_backward_blocks(int n_rows) { return (n_rows + kWarpsPerBlock - 1) / kWarpsPerBlock; }

cudaError_t launch_edge_forward(const EdgeArgs& a, cudaStream_t st) {
    const int rows = a.a1 - a.a0;
    if (rows <= 0) return cudaSuccess;
    return dispatch<true>(a, (rows + kWarpsPerBlock - 1) / kWarpsPerBlock, st);
}

cudaError_t launch_edge_backward(const EdgeArgs& a, int* n_blocks, cudaStream_t st) {
    const int rows = a.a1 - a.a0;
    *n_blocks = edge_backward_blocks(rows);
    if (rows <= 0) return cudaSuccess;
    return dispatch<false>(a, *n_blocks, st);
}

}  // namespace umd
