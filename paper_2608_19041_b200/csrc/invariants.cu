// Per-atom readout front end: normalisation of the aggregated sums, channel alignment,
// Gram blocks, degree-wise low-rank probes, Cartesian bispectrum (closed forms for (1,1,2)
// and (2,2,2), sparse Gaunt contraction for the other triples), projected quartic
// invariant, assembly and diagonal calibration -- and the matching vector-Jacobian
// product, which turns dE/dD into dE/d(sums) in place of the saved sums.
//
// A block handles 32 atoms with eight warps, lane = atom.  All per-atom tensors live in
// shared memory in an [index][atom] layout with row pitch 33, so a warp that reads or
// writes one index for its 32 atoms touches 32 distinct banks, and every index computation
// is uniform over the warp.  The work of a phase is cut into units (an output row, a pair
// of Gram rows, one probe index ...) that are dealt round-robin to the warps; each output
// entry has exactly one writer and a fixed summation order, so there are no atomics and the
// result is bitwise reproducible.  Phases are separated by block barriers.  Global memory
// is only touched by block-cooperative, coalesced transfers (lane = column): the state
// slice and the feature rows are staged once per block.
//
// The sparse Gaunt triples are contracted through small intermediates instead of per
// entry: with the non-zeros (m1, m2, m3, v) of the (1,2,3) coupling,
//   U[m1][e] = sum_n v Z2[m2][e] X3[m3],   J123[k][e] = sum_m1 Z1[m1][k] U[m1][e],
// and with those of the (2,3,3) coupling
//   Y[m1] = sum_n v X3[m2] X3[m3],         J233[e] = sum_m1 Z2[m1][e] Y[m1];
// the backward pass uses the same factorisation.
//
// The two normalising scales are standardised by the calibration, (M - mu) / sigma with
// mu ~ M, so they are formed in double precision from sums accumulated in double (stored
// as a float pair) to keep the subtraction from cancelling single-precision digits.
#include "kernels.h"
#include "mlp_gemm.h"

namespace umd {

namespace {

constexpr int AT = 32;               // atoms per block = lanes
constexpr int NW = 8;                // warps per block
constexpr int NT = AT * NW;
constexpr int P = AT + 1;            // row pitch of the [index][atom] layout
constexpr unsigned kFull = 0xffffffffu;

constexpr float kR2 = 1.4142135623730951f;
constexpr float kInvR2 = 0.7071067811865476f;
constexpr float kInvR6 = 0.4082482904638631f;
constexpr float kC112 = -0.4472135954999579f;    // -1/sqrt(5)
constexpr float kC222 = -0.5855400437691199f;    // -sqrt(12/35)
constexpr float kR3 = 1.7320508075688772f;

// symmetric trace-free matrix of a packed degree-2 vector, row-major 3x3
__device__ __forceinline__ void stf9(float z1, float z2, float z3, float z4, float z5, float* Q) {
    const float xx = -kInvR6 * z3 + kInvR2 * z5, yy = -kInvR6 * z3 - kInvR2 * z5, zz = 2.0f * kInvR6 * z3;
    const float xy = kInvR2 * z1, yz = kInvR2 * z2, xz = kInvR2 * z4;
    Q[0] = xx; Q[1] = xy; Q[2] = xz; Q[3] = xy; Q[4] = yy; Q[5] = yz; Q[6] = xz; Q[7] = yz; Q[8] = zz;
}
__device__ __forceinline__ void matvec3(const float* Q, float a, float b, float c, float* y) {
    y[0] = Q[0] * a + Q[1] * b + Q[2] * c;
    y[1] = Q[3] * a + Q[4] * b + Q[5] * c;
    y[2] = Q[6] * a + Q[7] * b + Q[8] * c;
}
__device__ __forceinline__ void matmul3(const float* A, const float* B, float* C) {
#pragma unroll
    for (int i = 0; i < 3; ++i)
#pragma unroll
        for (int j = 0; j < 3; ++j) C[3 * i + j] = A[3 * i] * B[j] + A[3 * i + 1] * B[3 + j] + A[3 * i + 2] * B[6 + j];
}
__device__ __forceinline__ float trace_prod(const float* A, const float* B) {   // tr(A B)
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 3; ++i)
#pragma unroll
        for (int j = 0; j < 3; ++j) s += A[3 * i + j] * B[3 * j + i];
    return s;
}
// multiplicity weight sqrt(family size) of a non-decreasing triple of equal-degree indices
__device__ __forceinline__ float fam3(int a, int b, int c) {
    if (a == b && b == c) return 1.0f;
    if (a == b || b == c) return kR3;
    return 2.449489742783178f;
}
// position of (p, q), p <= q, in the row-major upper triangle of a C x C matrix
__device__ __forceinline__ int tri(int p, int q, int C) { return p * C - (p * (p - 1)) / 2 + (q - p); }
__device__ __forceinline__ int tri_sym(int p, int q, int C) { return p <= q ? tri(p, q, C) : tri(q, p, C); }

// The couplings that involve degree 4 (only present for L = 4, which no timed workload uses) are
// contracted entry by entry over their non-zeros, all by one warp (lane = atom): operands are
// [m][atom] columns, X[m * stride].
__device__ __forceinline__ float contract3(const GauntSparseBig* G, const float* A, int sa, const float* B, int sb,
                                           const float* C, int sc) {
    float s = 0.f;
    const int nn = G->n;
    for (int n = 0; n < nn; ++n) s += G->v[n] * A[G->m1[n] * sa] * B[G->m2[n] * sb] * C[G->m3[n] * sc];
    return s;
}
// dA += g dJ/dA and likewise for B, C (the operands may be the same array: the shares add up)
__device__ __forceinline__ void contract3_grad(const GauntSparseBig* G, float g, const float* A, int sa, const float* B,
                                               int sb, const float* C, int sc, float* dA, float* dB, float* dC) {
    const int nn = G->n;
    for (int n = 0; n < nn; ++n) {
        const int m1 = G->m1[n], m2 = G->m2[n], m3 = G->m3[n];
        const float v = g * G->v[n], av = A[m1 * sa], bv = B[m2 * sb], cv = C[m3 * sc];
        dA[m1 * sa] += v * bv * cv;
        dB[m2 * sb] += v * av * cv;
        dC[m3 * sc] += v * av * bv;
    }
}

template <int C1, int C2, int L>
struct Plan {                                 // widths and the shared-memory plan, in rows of P floats
    static constexpr int K1 = C2, K2 = 2;
    static constexpr int nX1 = 3 * C1, nX2 = 5 * C2, nX3 = L >= 3 ? 7 : 0, nX4 = L >= 4 ? 9 : 0, nX = nX1 + nX2 + nX3 + nX4;
    static constexpr int nZ1 = 3 * K1, nZ2 = 5 * K2, nZ = nZ1 + nZ2;
    static constexpr int nU = L >= 3 ? 3 * K2 : 0, nY = L >= 3 ? 5 : 0;          // forward intermediates
    static constexpr int nPreF = nU + nY;
    static constexpr int nW = nU, nZg = nY, nYQ = K2 * K1 * 3;                   // backward adds W, Zg, Q v
    static constexpr int nPreB = nPreF + nW + nZg + nYQ;
    static constexpr int nAux = 12;                                              // dot0, nine partial dots
    static constexpr int nMat = C1 * C1 + C2 * C2 + C1 * K1 + C2 * K2;
    static constexpr int nGaunt = L >= 3 ? 2 * (int)((sizeof(GauntSparse) + 3) / 4) : 0;
    static constexpr int nMatP = (nMat + nGaunt + 3) / 4 * 4;                    // matrices come first: 16-byte rows
    // backward, L = 4: gradient shares of the degree-4 couplings with respect to Z1, Z2, X3 and X4
    static constexpr int nE4 = L >= 4 ? nZ1 + nZ2 + 7 + 9 : 0;
    // the staged state slice shares the rows of the staging area of the feature columns (nDS counts the
    // larger of the slice and of the two portions the columns are staged in)
    static int rows(int TW, int nDS, bool bwd) {
        (void)TW;
        return bwd ? nX + nZ + nDS + nPreB + nX + nX3 + nZ + 18 + nAux + nE4 : nX + nZ + nDS + nPreF;
    }
    static size_t bytes(int TW, int nDS, bool bwd) { return sizeof(float) * ((size_t)rows(TW, nDS, bwd) * P + nMatP); }
};

// Shared front of both passes: stage the small matrices and the block's slice of the state
// array (everything behind the C0 scalar sums), then, one warp per harmonic row, normalise
// and align it, XT = (X / M_1)(I + W), and project it on the probes, Z = XT A.
template <int C1, int C2, int L>
struct Front {
    using PL = Plan<C1, C2, L>;
    static constexpr int K1 = C2, K2 = 2;
    float *ST, *XT, *ZZ;
    float *mW1, *mW2, *mA1, *mA2;
    const GauntSparse *G123, *G233;
    int nv, b0, lane, warp, C0, TW, o1, o2, o3, o4, oS;
    float iM1;
    double M1d;

    template <int C, int K>
    __device__ __forceinline__ void align_row(const float* xr, const float* W, const float* A, float* xt, float* z) const {
        float rr[C];
#pragma unroll
        for (int b = 0; b < C; ++b) rr[b] = 0.f;
#pragma unroll
        for (int c = 0; c < C; ++c) {
            const float x = xr[c * P] * iM1;
#pragma unroll
            for (int b = 0; b < C; b += 4) {
                const float4 w = *reinterpret_cast<const float4*>(W + c * C + b);
                rr[b] += x * w.x; rr[b + 1] += x * w.y; rr[b + 2] += x * w.z; rr[b + 3] += x * w.w;
            }
        }
#pragma unroll
        for (int b = 0; b < C; ++b) xt[b * P] = rr[b];
#pragma unroll
        for (int kk = 0; kk < K; ++kk) {
            float s = 0.f;
#pragma unroll
            for (int c = 0; c < C; ++c) s += rr[c] * A[c * K + kk];
            z[kk * P] = s;
        }
    }

    __device__ __forceinline__ void setup(const InvArgs& a, float* st, float* xt, float* zz, float* mats) {
        const Dims& d = a.d;
        const int tid = threadIdx.x;
        lane = tid & 31; warp = tid >> 5;
        ST = st; XT = xt; ZZ = zz;
        mW1 = mats; mW2 = mW1 + C1 * C1; mA1 = mW2 + C2 * C2; mA2 = mA1 + C1 * K1;
        for (int i = tid; i < C1 * C1; i += NT) mW1[i] = __ldg(a.m.W1p + i);
        for (int i = tid; i < C2 * C2; i += NT) mW2[i] = __ldg(a.m.W2p + i);
        for (int i = tid; i < C1 * K1; i += NT) mA1[i] = __ldg(a.m.A1 + i);
        for (int i = tid; i < C2 * K2; i += NT) mA2[i] = __ldg(a.m.A2 + i);
        G123 = nullptr; G233 = nullptr;
        if (L >= 3) {
            constexpr int nw = (int)((sizeof(GauntSparse) + 3) / 4);
            unsigned* g1 = reinterpret_cast<unsigned*>(mA2 + C2 * K2);
            unsigned* g2 = g1 + nw;
            const unsigned* s1 = reinterpret_cast<const unsigned*>(a.m.g123);
            const unsigned* s2 = reinterpret_cast<const unsigned*>(a.m.g233);
            for (int i = tid; i < nw; i += NT) { g1[i] = __ldg(s1 + i); g2[i] = __ldg(s2 + i); }
            G123 = reinterpret_cast<const GauntSparse*>(g1);
            G233 = reinterpret_cast<const GauntSparse*>(g2);
        }
        b0 = blockIdx.x * AT;
        nv = a.n - b0 < AT ? a.n - b0 : AT;
        C0 = d.C0; TW = d.SP - C0;
        o1 = d.offA[1] - C0; o2 = d.offA[2] - C0; o3 = d.offA[3] - C0; o4 = d.offA[4] - C0; oS = d.S - C0;
        // state slice: a warp reads 32 consecutive entries of one atom's row; four atoms'
        // loads are issued before the first store
        const float* src = a.state + (size_t)b0 * d.SP + C0;
        for (int k0 = 0; k0 < TW; k0 += 32) {
            const int k = k0 + lane;
            float v[AT / NW];
#pragma unroll
            for (int i = 0; i < AT / NW; ++i) {
                const int aa = warp + i * NW;
                v[i] = (k < TW && aa < nv) ? src[(size_t)aa * d.SP + k] : 0.f;
            }
            if (k < TW) {
#pragma unroll
                for (int i = 0; i < AT / NW; ++i) ST[k * P + warp + i * NW] = v[i];
            }
        }
        __syncthreads();
        M1d = sqrt(0.25 + (double)ST[(oS + 1) * P + lane] + (double)ST[(oS + 3) * P + lane]);
        iM1 = (float)(1.0 / M1d);
        for (int u = warp; u < 10; u += NW) {
            if (u < 3) align_row<C1, K1>(ST + (o1 + u * C1) * P + lane, mW1, mA1, XT + u * C1 * P + lane, ZZ + u * K1 * P + lane);
            else if (u < 8)
                align_row<C2, K2>(ST + (o2 + (u - 3) * C2) * P + lane, mW2, mA2, XT + (PL::nX1 + (u - 3) * C2) * P + lane,
                                  ZZ + (PL::nZ1 + (u - 3) * K2) * P + lane);
            else if (u == 8 && L >= 3) {
#pragma unroll
                for (int mm = 0; mm < 7; ++mm) XT[(PL::nX1 + PL::nX2 + mm) * P + lane] = ST[(o3 + mm) * P + lane] * iM1;
            } else if (u == 9 && L >= 4) {
#pragma unroll
                for (int mm = 0; mm < 9; ++mm) XT[(PL::nX1 + PL::nX2 + PL::nX3 + mm) * P + lane] = ST[(o4 + mm) * P + lane] * iM1;
            }
        }
        __syncthreads();
    }
    // 1 / M_0 of atom aa (the same value in every lane)
    __device__ __forceinline__ double M0_of(int aa) const {
        return sqrt(0.25 + (double)ST[oS * P + aa] + (double)ST[(oS + 2) * P + aa]);
    }
    // U[m1][e] and Y[m1] of the sparse couplings, one unit per m1
    __device__ __forceinline__ void gaunt_pre(float* PRE, int& uctr) const {
        if (L < 3) return;
        const float* Z2 = ZZ + PL::nZ1 * P + lane;
        const float* X3 = XT + (PL::nX1 + PL::nX2) * P + lane;
        for (int m1 = 0; m1 < 3; ++m1) {
            if ((uctr++ % NW) != warp) continue;
            float u0 = 0.f, u1 = 0.f;
            const int nn = G123->n;
            for (int n = 0; n < nn; ++n) {
                if (G123->m1[n] != m1) continue;
                const float t = G123->v[n] * X3[G123->m3[n] * P];
                u0 += t * Z2[(G123->m2[n] * K2) * P];
                u1 += t * Z2[(G123->m2[n] * K2 + 1) * P];
            }
            PRE[(m1 * K2) * P + lane] = u0;
            PRE[(m1 * K2 + 1) * P + lane] = u1;
        }
        for (int m1 = 0; m1 < 5; ++m1) {
            if ((uctr++ % NW) != warp) continue;
            float y = 0.f;
            const int nn = G233->n;
            for (int n = 0; n < nn; ++n) {
                if (G233->m1[n] != m1) continue;
                y += G233->v[n] * X3[G233->m2[n] * P] * X3[G233->m3[n] * P];
            }
            PRE[(PL::nU + m1) * P + lane] = y;
        }
    }
};

// one calibrated feature-vector entry: fp32 and / or its half-precision split
__device__ __forceinline__ void put_feature(const InvArgs& a, size_t off, float v, bool split_ok) {
    if (a.write_desc) a.desc[off] = v;
    if (a.desc_hi && split_ok) split_f16(v, a.desc_hi[off], a.desc_lo[off]);
}

template <int C1, int C2, int L>
__global__ void __launch_bounds__(NT) k_inv_forward(const InvArgs a) {
    using PL = Plan<C1, C2, L>;
    constexpr int K1 = C2, K2 = 2;
    extern __shared__ float sm[];
    const Dims& d = a.d;
    const ModelDev& m = a.m;
    const int C0 = d.C0, TW = d.SP - C0;
    const int c_full = (2 * C0 / 32) * 32;         // columns [0, c_full) go straight from global to global
    float* mats = sm;
    float* XT = sm + PL::nMatP;
    float* ZZ = XT + PL::nX * P;
    float* PRE = ZZ + PL::nZ * P;
    // staging area of the feature columns, [column][atom], filled and written out in two portions
    // (columns [c_full, oG[2]) and [oG[2], DP)); before that it holds the state slice, which is only
    // needed until the harmonic rows are aligned and the first 2 C0 columns are out
    float* DS = PRE + PL::nPreF * P;
    float* ST = DS;
    (void)TW;
    Front<C1, C2, L> f;
    f.setup(a, ST, XT, ZZ, mats);
    const int lane = f.lane, warp = f.warp, nv = f.nv, b0 = f.b0;
    const double M0lane = f.M0_of(lane);           // kept: the state slice is overwritten below
    int uctr = 0;
    int dbase = c_full;                            // first column of the portion in the staging area
#define TAKE() ((uctr++ % NW) == warp)
#define DSK(k) DS[((k) - dbase) * P + lane]

    f.gaunt_pre(PRE, uctr);

    // Columns [0, c_full): the centre's initial features (a gather by species) and the
    // normalised scalar sums A_0 / M_0.  A warp takes one atom at a time, lane = column.
    {
        const float* st_g = a.state + (size_t)b0 * d.SP;
        float im0[AT / NW];
        int ty[AT / NW];
#pragma unroll
        for (int i = 0; i < AT / NW; ++i) {
            const int aa = warp + i * NW;
            im0[i] = (float)(1.0 / f.M0_of(aa));
            ty[i] = aa < nv ? a.type_s[a.a0 + b0 + aa] : 0;
        }
        for (int cb = 0; cb < c_full; cb += 64) {
            float v[2][AT / NW];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int col = cb + 32 * h + lane;
#pragma unroll
                for (int i = 0; i < AT / NW; ++i) {
                    const int aa = warp + i * NW;
                    v[h][i] = 0.f;
                    if (aa < nv && col < c_full) {
                        if (col < C0) { if (a.write_desc || !a.skip_x0_split) v[h][i] = __ldg(m.X0 + ty[i] * C0 + col); }
                        else v[h][i] = st_g[(size_t)aa * d.SP + (col - C0)] * im0[i];
                    }
                }
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int col = cb + 32 * h + lane;
                if (col >= c_full) continue;
                const float mu_c = __ldg(m.mu + col), is_c = __ldg(m.inv_sigma + col);
                const bool split_col = !(a.skip_x0_split && col < C0);
#pragma unroll
                for (int i = 0; i < AT / NW; ++i) {
                    const int aa = warp + i * NW;
                    if (aa < nv) put_feature(a, (size_t)(b0 + aa) * d.DP + col, (v[h][i] - mu_c) * is_c, split_col);
                }
            }
        }
    }
    __syncthreads();                               // U, Y visible

    // ---- the remaining columns, by units dealt to the warps; lane = atom -------------
    const float* X1 = XT + lane;                               // [mm * C1 + c]
    const float* X2 = XT + PL::nX1 * P + lane;                 // [mm * C2 + c]
    const float* X3 = XT + (PL::nX1 + PL::nX2) * P + lane;     // [mm]
    const float* Z1 = ZZ + lane;                               // [mm * K1 + k]
    const float* Z2 = ZZ + PL::nZ1 * P + lane;                 // [mm * K2 + e]
    float Q[K2][9];
#pragma unroll
    for (int e = 0; e < K2; ++e) stf9(Z2[e * P], Z2[(K2 + e) * P], Z2[(2 * K2 + e) * P], Z2[(3 * K2 + e) * P], Z2[(4 * K2 + e) * P], Q[e]);

    const int kM0 = 2 * C0, kM1 = 2 * C0 + 1;
    // columns of a trailing partial group of 32 (only for C0 = 8)
    for (int c = c_full; c < 2 * C0; ++c) {
        if (!TAKE()) continue;
        float v = 0.f;
        if (lane < nv) {
            if (c < C0) v = __ldg(m.X0 + a.type_s[a.a0 + b0 + lane] * C0 + c);
            else v = a.state[(size_t)(b0 + lane) * d.SP + (c - C0)] * (float)(1.0 / M0lane);
        }
        DSK(c) = v;
    }
    if (TAKE()) {   // the two normalising scales, calibrated here in double precision
        DSK(kM0) = (float)((M0lane - (double)__ldg(m.mu + kM0)) * (double)__ldg(m.inv_sigma + kM0));
        DSK(kM1) = (float)((f.M1d - (double)__ldg(m.mu + kM1)) * (double)__ldg(m.inv_sigma + kM1));
    }
    // Gram blocks, row-major upper triangle, strict off-diagonals times sqrt 2; a unit is
    // rows u and C-1-u, which together hold C+1 entries
    for (int u = 0; u < C1 / 2; ++u) {
        if (!TAKE()) continue;
#pragma unroll 1
        for (int h = 0; h < 2; ++h) {
            const int p = h ? C1 - 1 - u : u;
            const float x0 = X1[p * P], x1 = X1[(C1 + p) * P], x2 = X1[(2 * C1 + p) * P];
            int k = d.oG[1] + tri(p, p, C1);
            DSK(k) = x0 * x0 + x1 * x1 + x2 * x2;
            for (int q = p + 1; q < C1; ++q) {
                ++k;
                DSK(k) = kR2 * (x0 * X1[q * P] + x1 * X1[(C1 + q) * P] + x2 * X1[(2 * C1 + q) * P]);
            }
        }
    }
    // ---- first portion out: calibrate and write, lane = column ---------------------------
    auto write_out = [&](const int lo, const int hi) {
        __syncthreads();
        for (int cb = lo; cb < hi; cb += 32) {
            const int col = cb + lane;
            if (col >= hi) continue;
            float mu_c = 0.f, is_c = 1.f;
            if (col < d.D_out && col != kM0 && col != kM1) { mu_c = __ldg(m.mu + col); is_c = __ldg(m.inv_sigma + col); }
            const bool split_col = !(a.skip_x0_split && col < C0);
#pragma unroll
            for (int i = 0; i < AT / NW; ++i) {
                const int aa = warp + i * NW;
                if (aa < nv) put_feature(a, (size_t)(b0 + aa) * d.DP + col, (DS[(col - lo) * P + aa] - mu_c) * is_c, split_col);
            }
        }
        __syncthreads();
    };
    write_out(c_full, d.oG[2]);
    dbase = d.oG[2];
    if (TAKE()) {
        for (int k = d.D_out; k < d.DP; ++k) DSK(k) = 0.f;      // padding columns
    }
    for (int u = 0; u < C2 / 2; ++u) {
        if (!TAKE()) continue;
#pragma unroll 1
        for (int h = 0; h < 2; ++h) {
            const int p = h ? C2 - 1 - u : u;
            float x[5];
#pragma unroll
            for (int mm = 0; mm < 5; ++mm) x[mm] = X2[(mm * C2 + p) * P];
            int k = d.oG[2] + tri(p, p, C2);
            for (int q = p; q < C2; ++q) {
                float s = 0.f;
#pragma unroll
                for (int mm = 0; mm < 5; ++mm) s += x[mm] * X2[(mm * C2 + q) * P];
                DSK(k) = q == p ? s : kR2 * s;
                ++k;
            }
        }
    }
    if (L >= 3) {
        if (TAKE()) {
            float s = 0.f;
#pragma unroll
            for (int mm = 0; mm < 7; ++mm) s += X3[mm * P] * X3[mm * P];
            DSK(d.oG[3]) = s;
        }
    }
    // (1,1,2): -(1/sqrt5) v_k1^T Q_eta v_k2, k1 <= k2; a unit is rows u and K1-1-u
    for (int u = 0; u < (K1 + 1) / 2; ++u) {
        if (!TAKE()) continue;
#pragma unroll 1
        for (int h = 0; h < 2; ++h) {
            const int k1 = h ? K1 - 1 - u : u;
            if (h && k1 == u) break;
            const float a0 = Z1[k1 * P], a1 = Z1[(K1 + k1) * P], a2 = Z1[(2 * K1 + k1) * P];
            int k = d.oJ112 + tri(k1, k1, K1) * K2;
            for (int k2 = k1; k2 < K1; ++k2) {
                const float b0v = Z1[k2 * P], b1v = Z1[(K1 + k2) * P], b2v = Z1[(2 * K1 + k2) * P];
                const float w = kC112 * (k1 == k2 ? 1.0f : kR2);
#pragma unroll
                for (int e = 0; e < K2; ++e) {
                    float y[3];
                    matvec3(Q[e], b0v, b1v, b2v, y);
                    DSK(k) = w * (a0 * y[0] + a1 * y[1] + a2 * y[2]);
                    ++k;
                }
            }
        }
    }
    if (L >= 3) {   // (1,2,3) and (2,3,3) from the intermediates
        for (int e = 0; e < K2; ++e) {
            if (!TAKE()) continue;
            const float u0 = PRE[(0 * K2 + e) * P + lane], u1 = PRE[(1 * K2 + e) * P + lane], u2 = PRE[(2 * K2 + e) * P + lane];
            for (int k1 = 0; k1 < K1; ++k1)
                DSK(d.oJ123 + k1 * K2 + e) = Z1[k1 * P] * u0 + Z1[(K1 + k1) * P] * u1 + Z1[(2 * K1 + k1) * P] * u2;
        }
        if (TAKE()) {
#pragma unroll
            for (int e = 0; e < K2; ++e) {
                float s = 0.f;
#pragma unroll
                for (int m1 = 0; m1 < 5; ++m1) s += Z2[(m1 * K2 + e) * P] * PRE[(PL::nU + m1) * P + lane];
                DSK(d.oJ233 + e) = s;
            }
        }
    }
    if (L >= 4) {   // squared norm of the degree-4 row and the five couplings that involve it
        if (TAKE()) {
            const float* X4 = XT + (PL::nX1 + PL::nX2 + PL::nX3) * P + lane;
            const GauntSparseBig* G4 = m.g4;
            float s = 0.f;
#pragma unroll
            for (int mm = 0; mm < 9; ++mm) s += X4[mm * P] * X4[mm * P];
            DSK(d.oG[4]) = s;
            for (int k1 = 0; k1 < K1; ++k1) DSK(d.oJ134 + k1) = contract3(G4 + 0, Z1 + k1 * P, K1 * P, X3, P, X4, P);
            int k = d.oJ224;
            for (int e1 = 0; e1 < K2; ++e1)
                for (int e2 = e1; e2 < K2; ++e2)
                    DSK(k++) = (e1 == e2 ? 1.0f : kR2) * contract3(G4 + 1, Z2 + e1 * P, K2 * P, Z2 + e2 * P, K2 * P, X4, P);
            for (int e = 0; e < K2; ++e) DSK(d.oJ244 + e) = contract3(G4 + 2, Z2 + e * P, K2 * P, X4, P, X4, P);
            DSK(d.oJ334) = contract3(G4 + 3, X3, P, X3, P, X4, P);
            DSK(d.oJ444) = contract3(G4 + 4, X4, P, X4, P, X4, P);
        }
    }
    if (TAKE()) {   // (2,2,2): -sqrt(12/35) tr(Q Q Q), non-decreasing index triples
        int k = d.oJ222;
#pragma unroll
        for (int e1 = 0; e1 < K2; ++e1)
#pragma unroll
            for (int e2 = e1; e2 < K2; ++e2) {
                float Pm[9];
                matmul3(Q[e1], Q[e2], Pm);
#pragma unroll
                for (int e3 = e2; e3 < K2; ++e3) {
                    DSK(k) = kC222 * fam3(e1, e2, e3) * trace_prod(Pm, Q[e3]);
                    ++k;
                }
            }
    }
#pragma unroll
    for (int e = 0; e < K2; ++e) {   // projected quartic |Q_eta v_k|^2, eta-major
        if (!TAKE()) continue;
        for (int k1 = 0; k1 < K1; ++k1) {
            float y[3];
            matvec3(Q[e], Z1[k1 * P], Z1[(K1 + k1) * P], Z1[(2 * K1 + k1) * P], y);
            DSK(d.oPi + e * K1 + k1) = y[0] * y[0] + y[1] * y[1] + y[2] * y[2];
        }
    }
    write_out(d.oG[2], d.DP);
#undef TAKE
#undef DSK
}

// transpose of the alignment and probe maps for one harmonic row: g = dXt + dZ A^T,
// dX = g (I + W)^T / M_1; returns the row's share of sum g . Xt
template <int C, int K>
__device__ __forceinline__ float back_row(const float* dxt, const float* dz, const float* A, const float* W,
                                          const float* xt, float* out, float iM1) {
    float zz[K], g[C];
#pragma unroll
    for (int kk = 0; kk < K; ++kk) zz[kk] = dz[kk * P];
    float dot = 0.f;
#pragma unroll
    for (int c = 0; c < C; ++c) {
        float s = dxt[c * P];
#pragma unroll
        for (int kk = 0; kk < K; ++kk) s += zz[kk] * A[c * K + kk];
        g[c] = s;
        dot += s * xt[c * P];
    }
#pragma unroll
    for (int c = 0; c < C; ++c) {
        float s = 0.f;
#pragma unroll
        for (int b = 0; b < C; b += 4) {
            const float4 w = *reinterpret_cast<const float4*>(W + c * C + b);
            s += g[b] * w.x + g[b + 1] * w.y + g[b + 2] * w.z + g[b + 3] * w.w;
        }
        out[c * P] = s * iM1;
    }
    return dot;
}

template <int C1, int C2, int L>
__global__ void __launch_bounds__(NT, 3) k_inv_backward(const InvArgs a) {
    using PL = Plan<C1, C2, L>;
    constexpr int K1 = C2, K2 = 2;
    extern __shared__ float sm[];
    const Dims& d = a.d;
    const ModelDev& m = a.m;
    const int C0 = d.C0, TW = d.SP - C0;
    const int c_full = (2 * C0 / 32) * 32;
    const int nA = d.oG[2] - c_full, nB = d.DP - d.oG[2];
    const int nDS = TW > (nA > nB ? nA : nB) ? TW : (nA > nB ? nA : nB);
    float* mats = sm;
    float* XT = sm + PL::nMatP;
    float* ZZ = XT + PL::nX * P;
    // One area, four uses one after the other: the state slice (until the harmonic rows are aligned),
    // dE/dD / sigma of the columns [oG[2], DP), then of the columns [c_full, oG[2]) ([column][atom]),
    // and at the end the gradient of the state slice on its way out.
    float* DS = ZZ + PL::nZ * P;
    float* ST = DS;
    float* PRE = DS + nDS * P;                     // U, Y, W, Zg, Q v
    float* GX = PRE + PL::nPreB * P;               // dE/dXt (degree-3 rows twice: the two couplings' shares)
    float* DZ = GX + (PL::nX + PL::nX3) * P;
    float* DQ = DZ + PL::nZ * P;
    float* AUX = DQ + 18 * P;                      // row 0: sum_c X_0 dE/dX_0; rows 1..10: partial dots
    float* E1 = AUX + PL::nAux * P;                // L = 4: shares of the degree-4 couplings in dE/dZ1, dE/dZ2,
    float* E2 = E1 + PL::nZ1 * P;                  // dE/dX3 and the whole of dE/dX4
    float* E3 = E2 + PL::nZ2 * P;
    float* E4 = E3 + 7 * P;
    float* Ws = PRE + PL::nPreF * P;               // [m1 * K2 + e]
    float* Zg = Ws + PL::nW * P;                   // [m1]
    float* YQ = Zg + PL::nZg * P;                  // [(e * K1 + k) * 3 + m]
    const int b0 = blockIdx.x * AT;
    const float* dDg = a.desc + (size_t)b0 * d.DP;
    // stage the gradient columns [lo, hi), lane = column, divided by sigma (zero beyond D_out)
    auto stage = [&](const int lo, const int hi) {
        const int ln = threadIdx.x & 31, wp = threadIdx.x >> 5;
        const int nv0 = a.n - b0 < AT ? a.n - b0 : AT;
        for (int cb = lo; cb < hi; cb += 64) {
            float v[2][AT / NW];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int col = cb + 32 * h + ln;
#pragma unroll
                for (int i = 0; i < AT / NW; ++i) {
                    const int aa = wp + i * NW;
                    v[h][i] = (col < hi && aa < nv0) ? dDg[(size_t)aa * d.DP + col] : 0.f;
                }
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int col = cb + 32 * h + ln;
                if (col >= hi) continue;
                const float is_c = col < d.D_out ? __ldg(m.inv_sigma + col) : 0.f;
#pragma unroll
                for (int i = 0; i < AT / NW; ++i) DS[(col - lo) * P + wp + i * NW] = v[h][i] * is_c;
            }
        }
    };
    Front<C1, C2, L> f;
    f.setup(a, ST, XT, ZZ, mats);
    const int lane = f.lane, warp = f.warp, nv = f.nv;
    const double M0lane = f.M0_of(lane);           // kept: the state slice is overwritten next
    __syncthreads();
    stage(d.oG[2], d.DP);
    __syncthreads();
    int uctr = 0;
    int dbase = d.oG[2];                           // first column of the staged portion
#define TAKE() ((uctr++ % NW) == warp)
#define DSK(k) DS[((k) - dbase) * P + lane]

    const float* X1 = XT + lane;
    const float* X2 = XT + PL::nX1 * P + lane;
    const float* X3 = XT + (PL::nX1 + PL::nX2) * P + lane;
    const float* Z1 = ZZ + lane;
    const float* Z2 = ZZ + PL::nZ1 * P + lane;
    float Q[K2][9];
#pragma unroll
    for (int e = 0; e < K2; ++e) stf9(Z2[e * P], Z2[(K2 + e) * P], Z2[(2 * K2 + e) * P], Z2[(3 * K2 + e) * P], Z2[(4 * K2 + e) * P], Q[e]);

    // ---- intermediates --------------------------------------------------------------
    f.gaunt_pre(PRE, uctr);
    if (L >= 3) {
        for (int m1 = 0; m1 < 3; ++m1) {           // W[m1][e] = sum_k g123[k][e] Z1[m1][k]
            if (!TAKE()) continue;
            float w0 = 0.f, w1 = 0.f;
            for (int k1 = 0; k1 < K1; ++k1) {
                const float z = Z1[(m1 * K1 + k1) * P];
                w0 += DSK(d.oJ123 + k1 * K2) * z;
                w1 += DSK(d.oJ123 + k1 * K2 + 1) * z;
            }
            Ws[(m1 * K2) * P + lane] = w0;
            Ws[(m1 * K2 + 1) * P + lane] = w1;
        }
        if (TAKE()) {                              // Zg[m1] = sum_e g233[e] Z2[m1][e]
            const float g0 = DSK(d.oJ233), g1 = DSK(d.oJ233 + 1);
#pragma unroll
            for (int m1 = 0; m1 < 5; ++m1) Zg[m1 * P + lane] = g0 * Z2[(m1 * K2) * P] + g1 * Z2[(m1 * K2 + 1) * P];
        }
    }
    if (L >= 4) {
        if (TAKE()) {      // all gradient shares of the couplings that involve degree 4, by this one warp
            const float* X4 = XT + (PL::nX1 + PL::nX2 + PL::nX3) * P + lane;
            const GauntSparseBig* G4 = m.g4;
            float* e1 = E1 + lane; float* e2 = E2 + lane; float* e3 = E3 + lane; float* e4 = E4 + lane;
            for (int r = 0; r < PL::nZ1; ++r) e1[r * P] = 0.f;
            for (int r = 0; r < PL::nZ2; ++r) e2[r * P] = 0.f;
            for (int r = 0; r < 7; ++r) e3[r * P] = 0.f;
            const float g4n = 2.0f * DSK(d.oG[4]);
            for (int mm = 0; mm < 9; ++mm) e4[mm * P] = g4n * X4[mm * P];
            for (int k1 = 0; k1 < K1; ++k1)
                contract3_grad(G4 + 0, DSK(d.oJ134 + k1), Z1 + k1 * P, K1 * P, X3, P, X4, P, e1 + k1 * P, e3, e4);
            int k = d.oJ224;
            for (int ea = 0; ea < K2; ++ea)
                for (int eb = ea; eb < K2; ++eb)
                    contract3_grad(G4 + 1, DSK(k++) * (ea == eb ? 1.0f : kR2), Z2 + ea * P, K2 * P, Z2 + eb * P, K2 * P, X4, P,
                                   e2 + ea * P, e2 + eb * P, e4);
            for (int e = 0; e < K2; ++e)
                contract3_grad(G4 + 2, DSK(d.oJ244 + e), Z2 + e * P, K2 * P, X4, P, X4, P, e2 + e * P, e4, e4);
            contract3_grad(G4 + 3, DSK(d.oJ334), X3, P, X3, P, X4, P, e3, e3, e4);
            contract3_grad(G4 + 4, DSK(d.oJ444), X4, P, X4, P, X4, P, e4, e4, e4);
        }
    }
#pragma unroll
    for (int e = 0; e < K2; ++e) {                 // Q_e v_k for every probe
        if (!TAKE()) continue;
        for (int k1 = 0; k1 < K1; ++k1) {
            float y[3];
            matvec3(Q[e], Z1[k1 * P], Z1[(K1 + k1) * P], Z1[(2 * K1 + k1) * P], y);
            YQ[((e * K1 + k1) * 3 + 0) * P + lane] = y[0];
            YQ[((e * K1 + k1) * 3 + 1) * P + lane] = y[1];
            YQ[((e * K1 + k1) * 3 + 2) * P + lane] = y[2];
        }
    }
    // scalar block, X_0 = A_0 / M_0: a warp takes its four atoms, lane = channel, straight
    // from / to global memory; sum_c X_0 dE/dX_0 of each atom lands in the first scratch row
    {
        float* __restrict__ st_g = a.state + (size_t)b0 * d.SP;
        const float* __restrict__ dd_g = dDg;
        constexpr int UA = AT / NW;
        float isg[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) isg[j] = lane + 32 * j < C0 ? __ldg(m.inv_sigma + C0 + lane + 32 * j) : 0.f;
        float dx[UA][4], a0v[UA][4];
#pragma unroll
        for (int u = 0; u < UA; ++u) {
            const int aa = warp + u * NW;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int c = lane + 32 * j;
                const bool ok = aa < nv && c < C0;
                dx[u][j] = ok ? dd_g[(size_t)aa * d.DP + C0 + c] : 0.f;
                a0v[u][j] = ok ? st_g[(size_t)aa * d.SP + c] : 0.f;
            }
        }
#pragma unroll
        for (int u = 0; u < UA; ++u) {
            const int aa = warp + u * NW;
            const float im0 = (float)(1.0 / __shfl_sync(kFull, M0lane, aa));
            float part = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int c = lane + 32 * j;
                const float dxs = dx[u][j] * isg[j];
                part += a0v[u][j] * im0 * dxs;
                if (aa < nv && c < C0) st_g[(size_t)aa * d.SP + c] = dxs * im0;
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(kFull, part, off);
            if (lane == 0) AUX[aa] = part;
        }
    }
    __syncthreads();

    // ---- gradients of the aligned rows, the probes and the two matrices Q --------------
    for (int p = 0; p < C2; ++p) {
        if (!TAKE()) continue;
        float acc[5] = {0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 4
        for (int q = 0; q < C2; ++q) {
            const float g = DSK(d.oG[2] + tri_sym(p, q, C2)) * (p == q ? 2.0f : kR2);
#pragma unroll
            for (int mm = 0; mm < 5; ++mm) acc[mm] += g * X2[(mm * C2 + q) * P];
        }
#pragma unroll
        for (int mm = 0; mm < 5; ++mm) GX[(PL::nX1 + mm * C2 + p) * P + lane] = acc[mm];
    }
    if (L >= 3) {
        float* G3a = GX + (PL::nX1 + PL::nX2) * P + lane;      // squared norm and (1,2,3)
        float* G3b = GX + PL::nX * P + lane;                   // (2,3,3)
        if (TAKE()) {
            const float g2 = 2.0f * DSK(d.oG[3]);
#pragma unroll
            for (int mm = 0; mm < 7; ++mm) G3a[mm * P] = g2 * X3[mm * P];
            const int nn = f.G123->n;
            for (int n = 0; n < nn; ++n) {
                const int m1 = f.G123->m1[n], m2 = f.G123->m2[n], m3 = f.G123->m3[n];
                G3a[m3 * P] += f.G123->v[n] * (Ws[(m1 * K2) * P + lane] * Z2[(m2 * K2) * P] +
                                               Ws[(m1 * K2 + 1) * P + lane] * Z2[(m2 * K2 + 1) * P]);
            }
        }
        if (TAKE()) {
#pragma unroll
            for (int mm = 0; mm < 7; ++mm) G3b[mm * P] = 0.f;
            const int nn = f.G233->n;
            for (int n = 0; n < nn; ++n) {
                const int m1 = f.G233->m1[n], m2 = f.G233->m2[n], m3 = f.G233->m3[n];
                const float c = f.G233->v[n] * Zg[m1 * P + lane];
                const float xa = X3[m2 * P], xb = X3[m3 * P];
                G3b[m2 * P] += c * xb;
                G3b[m3 * P] += c * xa;
            }
        }
    }
    for (int k = 0; k < K1; ++k) {                 // dE/dZ1[., k]: (1,1,2), quartic and (1,2,3) shares
        if (!TAKE()) continue;
        float acc[3] = {0.f, 0.f, 0.f};
        for (int k2 = 0; k2 < K1; ++k2) {
            const int t = tri_sym(k, k2, K1) * K2;
            const float w = kC112 * (k == k2 ? 2.0f : kR2);
#pragma unroll
            for (int e = 0; e < K2; ++e) {
                const float cf = DSK(d.oJ112 + t + e) * w;
                const float* y = YQ + ((e * K1 + k2) * 3) * P + lane;
                acc[0] += cf * y[0]; acc[1] += cf * y[P]; acc[2] += cf * y[2 * P];
            }
        }
#pragma unroll
        for (int e = 0; e < K2; ++e) {
            const float g2 = 2.0f * DSK(d.oPi + e * K1 + k);
            const float* y = YQ + ((e * K1 + k) * 3) * P + lane;
            float qy[3];
            matvec3(Q[e], y[0], y[P], y[2 * P], qy);
            acc[0] += g2 * qy[0]; acc[1] += g2 * qy[1]; acc[2] += g2 * qy[2];
        }
        if (L >= 3) {
#pragma unroll
            for (int e = 0; e < K2; ++e) {
                const float g = DSK(d.oJ123 + k * K2 + e);
#pragma unroll
                for (int mm = 0; mm < 3; ++mm) acc[mm] += g * PRE[(mm * K2 + e) * P + lane];
            }
        }
        if (L >= 4) {
#pragma unroll
            for (int mm = 0; mm < 3; ++mm) acc[mm] += E1[(mm * K1 + k) * P + lane];
        }
#pragma unroll
        for (int mm = 0; mm < 3; ++mm) DZ[(mm * K1 + k) * P + lane] = acc[mm];
    }
#pragma unroll
    for (int e = 0; e < K2; ++e) {                 // dE/dQ_e, one row i per unit
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            if (!TAKE()) continue;
            float out[3] = {0.f, 0.f, 0.f};
            for (int k1 = 0; k1 < K1; ++k1) {
                const float vi = Z1[(i * K1 + k1) * P];
                for (int k2 = k1; k2 < K1; ++k2) {
                    const float cf = DSK(d.oJ112 + tri(k1, k2, K1) * K2 + e) * kC112 * (k1 == k2 ? 1.0f : kR2) * vi;
                    out[0] += cf * Z1[k2 * P]; out[1] += cf * Z1[(K1 + k2) * P]; out[2] += cf * Z1[(2 * K1 + k2) * P];
                }
                const float gy = 2.0f * DSK(d.oPi + e * K1 + k1) * YQ[((e * K1 + k1) * 3 + i) * P + lane];
                out[0] += gy * Z1[k1 * P]; out[1] += gy * Z1[(K1 + k1) * P]; out[2] += gy * Z1[(2 * K1 + k1) * P];
            }
            {   // (2,2,2): d tr(Qa Qb Qc) / dQa_ij = (Qb Qc)_ji, and cyclically
                int k = d.oJ222;
#pragma unroll
                for (int e1 = 0; e1 < K2; ++e1)
#pragma unroll
                    for (int e2 = e1; e2 < K2; ++e2)
#pragma unroll
                        for (int e3 = e2; e3 < K2; ++e3) {
                            const float cf = DSK(k) * kC222 * fam3(e1, e2, e3);
                            ++k;
#pragma unroll
                            for (int j = 0; j < 3; ++j) {
                                float s = 0.f;
#pragma unroll
                                for (int t = 0; t < 3; ++t) {
                                    if (e1 == e) s += Q[e2][3 * j + t] * Q[e3][3 * t + i];
                                    if (e2 == e) s += Q[e3][3 * j + t] * Q[e1][3 * t + i];
                                    if (e3 == e) s += Q[e1][3 * j + t] * Q[e2][3 * t + i];
                                }
                                out[j] += cf * s;
                            }
                        }
            }
#pragma unroll
            for (int j = 0; j < 3; ++j) DQ[(e * 9 + 3 * i + j) * P + lane] = out[j];
        }
    }
    __syncthreads();

    // ---- dE/dZ2: sparse couplings plus the transpose of the trace-free map -------------
    for (int m2 = 0; m2 < 5; ++m2) {
        if (!TAKE()) continue;
        float acc[K2];
#pragma unroll
        for (int e = 0; e < K2; ++e) acc[e] = 0.f;
        if (L >= 3) {
            const int nn = f.G123->n;
            for (int n = 0; n < nn; ++n) {
                if (f.G123->m2[n] != m2) continue;
                const float t = f.G123->v[n] * X3[f.G123->m3[n] * P];
                const int m1 = f.G123->m1[n];
#pragma unroll
                for (int e = 0; e < K2; ++e) acc[e] += t * Ws[(m1 * K2 + e) * P + lane];
            }
            const float y = PRE[(PL::nU + m2) * P + lane];
#pragma unroll
            for (int e = 0; e < K2; ++e) acc[e] += DSK(d.oJ233 + e) * y;
        }
#pragma unroll
        for (int e = 0; e < K2; ++e) {
            const float* q = DQ + (e * 9) * P + lane;
            float add;
            if (m2 == 0) add = kInvR2 * (q[1 * P] + q[3 * P]);
            else if (m2 == 1) add = kInvR2 * (q[5 * P] + q[7 * P]);
            else if (m2 == 2) add = kInvR6 * (2.0f * q[8 * P] - q[0] - q[4 * P]);
            else if (m2 == 3) add = kInvR2 * (q[2 * P] + q[6 * P]);
            else add = kInvR2 * (q[0] - q[4 * P]);
            if (L >= 4) add += E2[(m2 * K2 + e) * P + lane];
            DZ[(PL::nZ1 + m2 * K2 + e) * P + lane] = acc[e] + add;
        }
    }
    __syncthreads();

    // ---- the columns [c_full, oG[2]): the two normalising scales and the Gram block of degree 1 ----
    stage(c_full, d.oG[2]);
    dbase = c_full;
    __syncthreads();
    const float dM0 = DSK(2 * C0), dM1 = DSK(2 * C0 + 1);      // kept: the area takes the outgoing slice next
    for (int p = 0; p < C1; ++p) {                 // Gram of degree 1: a symmetric matrix-vector product per row
        if (!TAKE()) continue;
        float acc[3] = {0.f, 0.f, 0.f};
#pragma unroll 4
        for (int q = 0; q < C1; ++q) {
            const float g = DSK(d.oG[1] + tri_sym(p, q, C1)) * (p == q ? 2.0f : kR2);
#pragma unroll
            for (int mm = 0; mm < 3; ++mm) acc[mm] += g * X1[(mm * C1 + q) * P];
        }
#pragma unroll
        for (int mm = 0; mm < 3; ++mm) GX[(mm * C1 + p) * P + lane] = acc[mm];
    }
    __syncthreads();

    // ---- probes and alignment transposed, row by row; dot1 = sum dXt . Xt = sum dX . X --
    for (int u = 0; u < 10; ++u) {
        if (!TAKE()) continue;
        float dot = 0.f;
        if (u < 3)
            dot = back_row<C1, K1>(GX + (u * C1) * P + lane, DZ + (u * K1) * P + lane, f.mA1, f.mW1, X1 + (u * C1) * P,
                                   ST + (f.o1 + u * C1) * P + lane, f.iM1);
        else if (u < 8)
            dot = back_row<C2, K2>(GX + (PL::nX1 + (u - 3) * C2) * P + lane, DZ + (PL::nZ1 + (u - 3) * K2) * P + lane, f.mA2,
                                   f.mW2, X2 + ((u - 3) * C2) * P, ST + (f.o2 + (u - 3) * C2) * P + lane, f.iM1);
        else if (u == 8 && L >= 3) {
#pragma unroll
            for (int mm = 0; mm < 7; ++mm) {
                float g = GX[(PL::nX1 + PL::nX2 + mm) * P + lane] + GX[(PL::nX + mm) * P + lane];
                if (L >= 4) g += E3[mm * P + lane];
                dot += g * X3[mm * P];
                ST[(f.o3 + mm) * P + lane] = g * f.iM1;
            }
        } else if (u == 9 && L >= 4) {
            const float* X4 = XT + (PL::nX1 + PL::nX2 + PL::nX3) * P + lane;
#pragma unroll
            for (int mm = 0; mm < 9; ++mm) {
                const float g = E4[mm * P + lane];
                dot += g * X4[mm * P];
                ST[(f.o4 + mm) * P + lane] = g * f.iM1;
            }
        }
        AUX[(1 + u) * P + lane] = dot;
    }
    __syncthreads();
    if (warp == 0) {   // gradients of the two sums of squared envelopes, fixed summation order
        float dot1 = 0.f;
#pragma unroll
        for (int u = 0; u < 10; ++u) dot1 += AUX[(1 + u) * P + lane];
        const float iM0 = (float)(1.0 / M0lane);
        const float dot0 = AUX[lane];
        ST[f.oS * P + lane] = (dM0 - dot0 * iM0) * 0.5f * iM0;
        ST[(f.oS + 1) * P + lane] = (dM1 - dot1 * f.iM1) * 0.5f * f.iM1;
        ST[(f.oS + 2) * P + lane] = 0.f;
        ST[(f.oS + 3) * P + lane] = 0.f;
    }
    __syncthreads();
    // write the block's slice back, lane = state entry
    float* dst = a.state + (size_t)b0 * d.SP + C0;
    for (int k0 = 0; k0 < TW; k0 += 32) {
        const int k = k0 + lane;
        if (k >= TW) continue;
#pragma unroll
        for (int i = 0; i < AT / NW; ++i) {
            const int aa = warp + i * NW;
            if (aa < nv) dst[(size_t)aa * d.SP + k] = ST[k * P + aa];
        }
    }
#undef TAKE
#undef DSK
}

template <bool FWD>
cudaError_t dispatch(const InvArgs& a, cudaStream_t st) {
    if (a.n <= 0) return cudaSuccess;
    const int blocks = (a.n + AT - 1) / AT;
    const int C1 = a.d.C[1], C2 = a.d.C[2], L = a.d.L;
    const int TW = a.d.SP - a.d.C0;
    int nDS = a.d.DP - (2 * a.d.C0 / 32) * 32;
    {               // the larger of the two portions of staged columns and of the state slice that shares their rows
        const int na = a.d.oG[2] - (2 * a.d.C0 / 32) * 32, nb = a.d.DP - a.d.oG[2];
        nDS = na > nb ? na : nb;
        if (TW > nDS) nDS = TW;
    }
#define UMLMD_CASE(c1, c2, l)                                                                   \
    if (C1 == c1 && C2 == c2 && L == l) {                                                       \
        const size_t bytes = Plan<c1, c2, l>::bytes(TW, nDS, !FWD);                             \
        auto kern = FWD ? k_inv_forward<c1, c2, l> : k_inv_backward<c1, c2, l>;                 \
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes); \
        if (e != cudaSuccess) return e;                                                         \
        kern<<<blocks, NT, bytes, st>>>(a);                                                     \
        return cudaGetLastError();                                                              \
    }
    UMLMD_CASE(4, 4, 2) UMLMD_CASE(4, 4, 3) UMLMD_CASE(8, 4, 2) UMLMD_CASE(8, 4, 3)
    UMLMD_CASE(16, 8, 2) UMLMD_CASE(16, 8, 3) UMLMD_CASE(4, 4, 4) UMLMD_CASE(8, 4, 4) UMLMD_CASE(16, 8, 4)
#undef UMLMD_CASE
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_invariants_forward(const InvArgs& a, cudaStream_t st) { return dispatch<true>(a, st); }
cudaError_t launch_invariants_backward(const InvArgs& a, cudaStream_t st) { return dispatch<false>(a, st); }

}  // namespace umd
