// Per-atom readout front end: normalisation of the aggregated sums, channel alignment,
// Gram blocks, degree-wise low-rank probes, Cartesian bispectrum (closed forms for (1,1,2)
// and (2,2,2), sparse Gaunt contraction for the other triples), projected quartic
// invariant, assembly and diagonal calibration -- and the matching vector-Jacobian
// product, which turns dE/dD into dE/d(sums) in place of the saved sums.
//
// One thread per atom, 64 atoms per block.  Everything a thread touches repeatedly lives
// in shared memory in an [index][atom] layout with an odd row pitch, so a warp's accesses
// hit 32 distinct banks; global memory is only touched by block-cooperative, fully
// coalesced transfers: the block's slice of the state array is staged in one pass, and the
// feature vector streams through a 32-column staging buffer (written in increasing column
// order in the forward pass, read in increasing column order in the backward pass).
//
// The two normalising scales are standardised by the calibration, (M - mu) / sigma with
// mu ~ M, so they are formed in double precision from sums accumulated in double (stored
// as a float pair) to keep the subtraction from cancelling single-precision digits.
#include "kernels.h"

namespace umd {

namespace {

constexpr int BLK = 64;
constexpr int PITCH = BLK + 1;
constexpr int CHUNK = 32;

constexpr float kR2 = 1.4142135623730951f;
constexpr float kInvR2 = 0.7071067811865476f;
constexpr float kInvR6 = 0.4082482904638631f;
constexpr float kC112 = -0.4472135954999579f;    // -1/sqrt(5)
constexpr float kC222 = -0.5855400437691199f;    // -sqrt(12/35)
constexpr float kR3 = 1.7320508075688772f;

// column of the [index][atom] shared-memory layout belonging to one thread
struct SCol {
    float* p;
    __device__ __forceinline__ float& operator[](int i) const { return p[i * PITCH]; }
};

// symmetric trace-free matrix of a packed degree-2 vector z[0..4], row-major 3x3
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

template <int C1, int C2, int L>
struct Lay {                                  // shared-memory plan, in floats
    static constexpr int K1 = C2, K2 = 2;
    static constexpr int nZ1 = 3 * K1, nZ2 = 5 * K2;
    static constexpr int nMat = C1 * C1 + C2 * C2 + C1 * K1 + C2 * K2;
    static constexpr int work_fwd = nZ1 + nZ2;
    static constexpr int work_bwd = nZ1 + nZ2 + 3 * C1 + 5 * C2 + 7 + nZ1 + nZ2;
    static constexpr int nGaunt = L >= 3 ? 2 * (int)((sizeof(GauntSparse) + 3) / 4) : 0;
    static int floats(int SP, bool bwd) { return (SP + (bwd ? work_bwd : work_fwd) + CHUNK) * PITCH + nMat + nGaunt; }
};

// Shared setup of both passes: stage matrices and the block's state slice, then per thread
// normalise and align in place:  tile[offA1..] <- X1 (I + W1),  tile[offA2..] <- X2 (I + W2),
// tile[offA3..] <- X3, and form the probes Z1, Z2 and the two matrices Q.
template <int C1, int C2, int L>
struct Front {
    static constexpr int K1 = C2, K2 = 2;
    float* tile; float* mW1; float* mW2; float* mA1; float* mA2;
    const GauntSparse* G123; const GauntSparse* G233;     // shared-memory copies of the sparse couplings
    SCol T, Z1, Z2;
    double M0d, M1d;
    float iM0, iM1;
    float Q[K2][9];
    int nv, b0;

    __device__ __forceinline__ void setup(const InvArgs& a, float* sm, float* work, float* mats) {
        const Dims& d = a.d;
        const int tid = threadIdx.x;
        tile = sm;
        mW1 = mats; mW2 = mW1 + C1 * C1; mA1 = mW2 + C2 * C2; mA2 = mA1 + C1 * K1;
        for (int i = tid; i < C1 * C1; i += BLK) mW1[i] = __ldg(a.m.W1p + i);
        for (int i = tid; i < C2 * C2; i += BLK) mW2[i] = __ldg(a.m.W2p + i);
        for (int i = tid; i < C1 * K1; i += BLK) mA1[i] = __ldg(a.m.A1 + i);
        for (int i = tid; i < C2 * K2; i += BLK) mA2[i] = __ldg(a.m.A2 + i);
        G123 = nullptr; G233 = nullptr;
        if (L >= 3) {
            constexpr int nw = (int)((sizeof(GauntSparse) + 3) / 4);
            unsigned* g1 = reinterpret_cast<unsigned*>(mA2 + C2 * K2);
            unsigned* g2 = g1 + nw;
            const unsigned* s1 = reinterpret_cast<const unsigned*>(a.m.g123);
            const unsigned* s2 = reinterpret_cast<const unsigned*>(a.m.g233);
            for (int i = tid; i < nw; i += BLK) { g1[i] = __ldg(s1 + i); g2[i] = __ldg(s2 + i); }
            G123 = reinterpret_cast<const GauntSparse*>(g1);
            G233 = reinterpret_cast<const GauntSparse*>(g2);
        }
        b0 = blockIdx.x * BLK;
        nv = a.n - b0 < BLK ? a.n - b0 : BLK;
        const float* src = a.state + (size_t)b0 * d.SP;
        const int total = BLK * d.SP, valid = nv * d.SP;
        int atom = 0, k = tid;                   // element e = tid + j*BLK  ->  (atom, k)
        for (int e = tid; e < total; e += BLK) {
            while (k >= d.SP) { k -= d.SP; ++atom; }
            tile[k * PITCH + atom] = e < valid ? src[e] : 0.f;
            k += BLK;
        }
        __syncthreads();
        T.p = tile + tid;
        Z1.p = work + tid;
        Z2.p = work + nZ1() * PITCH + tid;
        M0d = sqrt(0.25 + (double)T[d.S] + (double)T[d.S + 2]);
        M1d = sqrt(0.25 + (double)T[d.S + 1] + (double)T[d.S + 3]);
        iM0 = (float)(1.0 / M0d); iM1 = (float)(1.0 / M1d);
        const int o1 = d.offA[1], o2 = d.offA[2], o3 = d.offA[3];
#pragma unroll
        for (int mm = 0; mm < 3; ++mm) {
            float x[C1], r[C1];
#pragma unroll
            for (int c = 0; c < C1; ++c) { x[c] = T[o1 + mm * C1 + c] * iM1; r[c] = 0.f; }
#pragma unroll
            for (int c = 0; c < C1; ++c)
#pragma unroll
                for (int b = 0; b < C1; ++b) r[b] += x[c] * mW1[c * C1 + b];
#pragma unroll
            for (int b = 0; b < C1; ++b) T[o1 + mm * C1 + b] = r[b];
#pragma unroll
            for (int kk = 0; kk < K1; ++kk) {
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < C1; ++c) s += r[c] * mA1[c * K1 + kk];
                Z1[mm * K1 + kk] = s;
            }
        }
#pragma unroll
        for (int mm = 0; mm < 5; ++mm) {
            float x[C2], r[C2];
#pragma unroll
            for (int c = 0; c < C2; ++c) { x[c] = T[o2 + mm * C2 + c] * iM1; r[c] = 0.f; }
#pragma unroll
            for (int c = 0; c < C2; ++c)
#pragma unroll
                for (int b = 0; b < C2; ++b) r[b] += x[c] * mW2[c * C2 + b];
#pragma unroll
            for (int b = 0; b < C2; ++b) T[o2 + mm * C2 + b] = r[b];
#pragma unroll
            for (int kk = 0; kk < K2; ++kk) {
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < C2; ++c) s += r[c] * mA2[c * K2 + kk];
                Z2[mm * K2 + kk] = s;
            }
        }
        if (L >= 3) {
#pragma unroll
            for (int mm = 0; mm < 7; ++mm) T[o3 + mm] = T[o3 + mm] * iM1;
        }
#pragma unroll
        for (int e = 0; e < K2; ++e) stf9(Z2[e], Z2[K2 + e], Z2[2 * K2 + e], Z2[3 * K2 + e], Z2[4 * K2 + e], Q[e]);
    }
    static __device__ __forceinline__ constexpr int nZ1() { return 3 * K1; }
};

template <int C1, int C2, int L>
__global__ void __launch_bounds__(BLK) k_inv_forward(const InvArgs a) {
    constexpr int K1 = C2, K2 = 2;
    using LY = Lay<C1, C2, L>;
    extern __shared__ float sm[];
    const Dims& d = a.d;
    const ModelDev& m = a.m;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float* work = sm + d.SP * PITCH;
    float* chunk = work + LY::work_fwd * PITCH;
    float* mats = chunk + CHUNK * PITCH;
    Front<C1, C2, L> f;
    f.setup(a, sm, work, mats);
    const SCol T = f.T, Z1 = f.Z1, Z2 = f.Z2;
    const int nv = f.nv, b0 = f.b0, C0 = d.C0;
    float* Dg = a.desc + (size_t)b0 * d.DP;
    const int ty = a.type_s[a.a0 + (b0 + tid < a.n ? b0 + tid : a.n - 1)];

    // feature-vector columns are produced in increasing order; every 32nd one flushes.  The
    // calibration (v - mu) / sigma is applied by the flushing lane, which owns one column, so
    // the per-thread code never waits on a global load; the two normalising scales arrive
    // already calibrated (they are formed in double precision).
    const int kM0 = 2 * C0, kM1 = 2 * C0 + 1;
    auto store = [&](int k, float v) {
        chunk[(k & (CHUNK - 1)) * PITCH + tid] = v;
        if ((k & (CHUNK - 1)) == CHUNK - 1) {
            const int kb = k - (CHUNK - 1), col = kb + lane;
            float mu_c = 0.f, is_c = 1.f;
            if (col < d.D_out && col != kM0 && col != kM1) { mu_c = __ldg(m.mu + col); is_c = __ldg(m.inv_sigma + col); }
            __syncthreads();
            for (int at = warp; at < nv; at += BLK / 32) Dg[(size_t)at * d.DP + col] = (chunk[lane * PITCH + at] - mu_c) * is_c;
            __syncthreads();
        }
    };
    auto put = store;

    // centre's initial-feature block: a plain gather, done by whole warps (lane = column) for
    // every complete group of 32 columns; a trailing partial group goes through the stream
    const int c_full = (C0 / CHUNK) * CHUNK;
    for (int cb = 0; cb < c_full; cb += CHUNK) {
        const int col = cb + lane;
        const float mu_c = __ldg(m.mu + col), is_c = __ldg(m.inv_sigma + col);
        for (int at = warp; at < nv; at += BLK / 32) {
            const int tt = a.type_s[a.a0 + b0 + at];
            Dg[(size_t)at * d.DP + col] = (__ldg(m.X0 + tt * C0 + col) - mu_c) * is_c;
        }
    }
    for (int c = c_full; c < C0; ++c) put(c, __ldg(m.X0 + ty * C0 + c));
    for (int c = 0; c < C0; ++c) put(C0 + c, T[c] * f.iM0);
    store(kM0, (float)((f.M0d - (double)__ldg(m.mu + kM0)) * (double)__ldg(m.inv_sigma + kM0)));
    store(kM1, (float)((f.M1d - (double)__ldg(m.mu + kM1)) * (double)__ldg(m.inv_sigma + kM1)));
    const int o1 = d.offA[1], o2 = d.offA[2], o3 = d.offA[3];
    {   // Gram blocks, row-major upper triangle, strict off-diagonals times sqrt 2
        int k = d.oG[1];
        for (int p = 0; p < C1; ++p)
            for (int q = p; q < C1; ++q) {
                float s = 0.f;
#pragma unroll
                for (int mm = 0; mm < 3; ++mm) s += T[o1 + mm * C1 + p] * T[o1 + mm * C1 + q];
                put(k++, p == q ? s : kR2 * s);
            }
        for (int p = 0; p < C2; ++p)
            for (int q = p; q < C2; ++q) {
                float s = 0.f;
#pragma unroll
                for (int mm = 0; mm < 5; ++mm) s += T[o2 + mm * C2 + p] * T[o2 + mm * C2 + q];
                put(k++, p == q ? s : kR2 * s);
            }
        if (L >= 3) {
            float s = 0.f;
#pragma unroll
            for (int mm = 0; mm < 7; ++mm) s += T[o3 + mm] * T[o3 + mm];
            put(k++, s);
        }
    }
    {   // (1,1,2): -(1/sqrt5) v_k1^T Q_eta v_k2, k1 <= k2
        int k = d.oJ112;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int k2 = k1; k2 < K1; ++k2) {
                const float a0 = Z1[k1], a1 = Z1[K1 + k1], a2 = Z1[2 * K1 + k1];
                const float b0v = Z1[k2], b1 = Z1[K1 + k2], b2 = Z1[2 * K1 + k2];
#pragma unroll
                for (int e = 0; e < K2; ++e) {
                    float y[3];
                    matvec3(f.Q[e], b0v, b1, b2, y);
                    put(k++, kC112 * (k1 == k2 ? 1.0f : kR2) * (a0 * y[0] + a1 * y[1] + a2 * y[2]));
                }
            }
    }
    if (L >= 3) {   // (1,2,3): sparse Gaunt contraction
        const GauntSparse* G = f.G123;
        const int nn = G->n;
        int k = d.oJ123;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int e = 0; e < K2; ++e) {
                float s = 0.f;
                for (int n = 0; n < nn; ++n)
                    s += G->v[n] * Z1[G->m1[n] * K1 + k1] * Z2[G->m2[n] * K2 + e] * T[o3 + G->m3[n]];
                put(k++, s);
            }
    }
    {   // (2,2,2): -sqrt(12/35) tr(Q Q Q), non-decreasing index triples
        int k = d.oJ222;
#pragma unroll
        for (int e1 = 0; e1 < K2; ++e1)
#pragma unroll
            for (int e2 = e1; e2 < K2; ++e2) {
                float P[9];
                matmul3(f.Q[e1], f.Q[e2], P);
#pragma unroll
                for (int e3 = e2; e3 < K2; ++e3) put(k++, kC222 * fam3(e1, e2, e3) * trace_prod(P, f.Q[e3]));
            }
    }
    if (L >= 3) {   // (2,3,3)
        const GauntSparse* G = f.G233;
        const int nn = G->n;
        int k = d.oJ233;
        for (int e = 0; e < K2; ++e) {
            float s = 0.f;
            for (int n = 0; n < nn; ++n) s += G->v[n] * Z2[G->m1[n] * K2 + e] * T[o3 + G->m2[n]] * T[o3 + G->m3[n]];
            put(k++, s);
        }
    }
    {   // projected quartic |Q_eta v_k|^2, eta-major
        int k = d.oPi;
#pragma unroll
        for (int e = 0; e < K2; ++e)
            for (int k1 = 0; k1 < K1; ++k1) {
                float y[3];
                matvec3(f.Q[e], Z1[k1], Z1[K1 + k1], Z1[2 * K1 + k1], y);
                put(k++, y[0] * y[0] + y[1] * y[1] + y[2] * y[2]);
            }
    }
    for (int k = d.D_out; k < d.DP; ++k) store(k, 0.f);    // DP is a multiple of 32: ends on a flush
}

template <int C1, int C2, int L>
__global__ void __launch_bounds__(BLK) k_inv_backward(const InvArgs a) {
    constexpr int K1 = C2, K2 = 2;
    using LY = Lay<C1, C2, L>;
    extern __shared__ float sm[];
    const Dims& d = a.d;
    const ModelDev& m = a.m;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float* work = sm + d.SP * PITCH;
    float* chunk = work + LY::work_bwd * PITCH;
    float* mats = chunk + CHUNK * PITCH;
    Front<C1, C2, L> f;
    f.setup(a, sm, work, mats);
    const SCol T = f.T, Z1 = f.Z1, Z2 = f.Z2;
    const int nv = f.nv, b0 = f.b0, C0 = d.C0;
    const float* dDg = a.desc + (size_t)b0 * d.DP;
    float* wp = work + (LY::nZ1 + LY::nZ2) * PITCH + tid;
    const SCol dXt1{wp}, dXt2{wp + 3 * C1 * PITCH}, dX3{wp + (3 * C1 + 5 * C2) * PITCH},
        dZ1{wp + (3 * C1 + 5 * C2 + 7) * PITCH}, dZ2{wp + (3 * C1 + 5 * C2 + 7 + LY::nZ1) * PITCH};
    for (int k = 0; k < 3 * C1; ++k) dXt1[k] = 0.f;
    for (int k = 0; k < 5 * C2; ++k) dXt2[k] = 0.f;
    for (int k = 0; k < 7; ++k) dX3[k] = 0.f;
    for (int k = 0; k < LY::nZ1; ++k) dZ1[k] = 0.f;
    for (int k = 0; k < LY::nZ2; ++k) dZ2[k] = 0.f;
    float dQ[K2][9];
#pragma unroll
    for (int e = 0; e < K2; ++e)
#pragma unroll
        for (int k = 0; k < 9; ++k) dQ[e][k] = 0.f;

    // dE/dD columns are consumed in increasing order, 32 at a time
    int cur = -1;
    auto get = [&](int k) -> float {
        const int c = k >> 5;
        if (c != cur) {
            __syncthreads();
            const int col = c * CHUNK + lane;
            const float is_c = col < d.D_out ? __ldg(m.inv_sigma + col) : 0.f;
            for (int at = warp; at < nv; at += BLK / 32) chunk[lane * PITCH + at] = dDg[(size_t)at * d.DP + col] * is_c;
            __syncthreads();
            cur = c;
        }
        return chunk[(k & (CHUNK - 1)) * PITCH + tid];
    };

    const int o1 = d.offA[1], o2 = d.offA[2], o3 = d.offA[3];
    float dot0 = 0.f;
    for (int c = 0; c < C0; ++c) {                 // scalar block: X_0 = A_0 / M_0
        const float dx = get(C0 + c);
        dot0 += T[c] * f.iM0 * dx;
        T[c] = dx * f.iM0;
    }
    const float dM0 = get(2 * C0), dM1 = get(2 * C0 + 1);
    {   // Gram
        int k = d.oG[1];
        for (int p = 0; p < C1; ++p)
            for (int q = p; q < C1; ++q) {
                const float g = get(k++) * (p == q ? 1.0f : kR2);
#pragma unroll
                for (int mm = 0; mm < 3; ++mm) {
                    const float xp = T[o1 + mm * C1 + p], xq = T[o1 + mm * C1 + q];
                    dXt1[mm * C1 + p] += g * xq;
                    dXt1[mm * C1 + q] += g * xp;
                }
            }
        for (int p = 0; p < C2; ++p)
            for (int q = p; q < C2; ++q) {
                const float g = get(k++) * (p == q ? 1.0f : kR2);
#pragma unroll
                for (int mm = 0; mm < 5; ++mm) {
                    const float xp = T[o2 + mm * C2 + p], xq = T[o2 + mm * C2 + q];
                    dXt2[mm * C2 + p] += g * xq;
                    dXt2[mm * C2 + q] += g * xp;
                }
            }
        if (L >= 3) {
            const float g = get(k++);
#pragma unroll
            for (int mm = 0; mm < 7; ++mm) dX3[mm] += 2.0f * g * T[o3 + mm];
        }
    }
    {   // (1,1,2)
        int k = d.oJ112;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int k2 = k1; k2 < K1; ++k2) {
                const float v1[3] = {Z1[k1], Z1[K1 + k1], Z1[2 * K1 + k1]};
                const float v2[3] = {Z1[k2], Z1[K1 + k2], Z1[2 * K1 + k2]};
#pragma unroll
                for (int e = 0; e < K2; ++e) {
                    const float cf = get(k++) * kC112 * (k1 == k2 ? 1.0f : kR2);
                    float y1[3], y2[3];
                    matvec3(f.Q[e], v2[0], v2[1], v2[2], y2);
                    matvec3(f.Q[e], v1[0], v1[1], v1[2], y1);
#pragma unroll
                    for (int i = 0; i < 3; ++i) {
                        dZ1[i * K1 + k1] += cf * y2[i];
                        dZ1[i * K1 + k2] += cf * y1[i];
#pragma unroll
                        for (int j = 0; j < 3; ++j) dQ[e][3 * i + j] += cf * v1[i] * v2[j];
                    }
                }
            }
    }
    if (L >= 3) {   // (1,2,3)
        const GauntSparse* G = f.G123;
        const int nn = G->n;
        int k = d.oJ123;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int e = 0; e < K2; ++e) {
                const float g = get(k++);
                for (int n = 0; n < nn; ++n) {
                    const int i1 = G->m1[n] * K1 + k1, i2 = G->m2[n] * K2 + e, i3 = G->m3[n];
                    const float cv = g * G->v[n];
                    const float z1 = Z1[i1], z2 = Z2[i2], x3 = T[o3 + i3];
                    dZ1[i1] += cv * z2 * x3;
                    dZ2[i2] += cv * z1 * x3;
                    dX3[i3] += cv * z1 * z2;
                }
            }
    }
    {   // (2,2,2): d tr(Qa Qb Qc)/dQa_ij = (Qb Qc)_ji, and cyclically
        int k = d.oJ222;
#pragma unroll
        for (int e1 = 0; e1 < K2; ++e1)
#pragma unroll
            for (int e2 = e1; e2 < K2; ++e2)
#pragma unroll
                for (int e3 = e2; e3 < K2; ++e3) {
                    const float cf = get(k++) * kC222 * fam3(e1, e2, e3);
                    float P[9];
                    matmul3(f.Q[e2], f.Q[e3], P);
#pragma unroll
                    for (int i = 0; i < 3; ++i)
#pragma unroll
                        for (int j = 0; j < 3; ++j) dQ[e1][3 * i + j] += cf * P[3 * j + i];
                    matmul3(f.Q[e3], f.Q[e1], P);
#pragma unroll
                    for (int i = 0; i < 3; ++i)
#pragma unroll
                        for (int j = 0; j < 3; ++j) dQ[e2][3 * i + j] += cf * P[3 * j + i];
                    matmul3(f.Q[e1], f.Q[e2], P);
#pragma unroll
                    for (int i = 0; i < 3; ++i)
#pragma unroll
                        for (int j = 0; j < 3; ++j) dQ[e3][3 * i + j] += cf * P[3 * j + i];
                }
    }
    if (L >= 3) {   // (2,3,3)
        const GauntSparse* G = f.G233;
        const int nn = G->n;
        int k = d.oJ233;
        for (int e = 0; e < K2; ++e) {
            const float g = get(k++);
            for (int n = 0; n < nn; ++n) {
                const int i1 = G->m1[n] * K2 + e, i2 = G->m2[n], i3 = G->m3[n];
                const float cv = g * G->v[n];
                const float z2 = Z2[i1], xa = T[o3 + i2], xb = T[o3 + i3];
                dZ2[i1] += cv * xa * xb;
                dX3[i2] += cv * z2 * xb;
                dX3[i3] += cv * z2 * xa;
            }
        }
    }
    {   // quartic: y = Q v, Pi = y.y
        int k = d.oPi;
#pragma unroll
        for (int e = 0; e < K2; ++e)
            for (int k1 = 0; k1 < K1; ++k1) {
                const float g2 = 2.0f * get(k++);
                const float v[3] = {Z1[k1], Z1[K1 + k1], Z1[2 * K1 + k1]};
                float y[3], qy[3];
                matvec3(f.Q[e], v[0], v[1], v[2], y);
                matvec3(f.Q[e], y[0], y[1], y[2], qy);
#pragma unroll
                for (int i = 0; i < 3; ++i) {
                    dZ1[i * K1 + k1] += g2 * qy[i];
#pragma unroll
                    for (int j = 0; j < 3; ++j) dQ[e][3 * i + j] += g2 * y[i] * v[j];
                }
            }
    }
    // transpose of the symmetric-trace-free map
#pragma unroll
    for (int e = 0; e < K2; ++e) {
        const float* q = dQ[e];
        dZ2[e] += kInvR2 * (q[1] + q[3]);
        dZ2[K2 + e] += kInvR2 * (q[5] + q[7]);
        dZ2[2 * K2 + e] += kInvR6 * (2.0f * q[8] - q[0] - q[4]);
        dZ2[3 * K2 + e] += kInvR2 * (q[2] + q[6]);
        dZ2[4 * K2 + e] += kInvR2 * (q[0] - q[4]);
    }
    // probes -> aligned features; dot1 = sum dXt . Xt = sum dX . X (the alignment is linear)
    float dot1 = 0.f;
#pragma unroll
    for (int mm = 0; mm < 3; ++mm) {
        float g[C1];
#pragma unroll
        for (int c = 0; c < C1; ++c) {
            float s = dXt1[mm * C1 + c];
#pragma unroll
            for (int kk = 0; kk < K1; ++kk) s += dZ1[mm * K1 + kk] * f.mA1[c * K1 + kk];
            g[c] = s;
            dot1 += s * T[o1 + mm * C1 + c];
        }
#pragma unroll
        for (int c = 0; c < C1; ++c) {         // dX = dXt (I + W)^T, then / M_1
            float s = 0.f;
#pragma unroll
            for (int b = 0; b < C1; ++b) s += g[b] * f.mW1[c * C1 + b];
            T[o1 + mm * C1 + c] = s * f.iM1;
        }
    }
#pragma unroll
    for (int mm = 0; mm < 5; ++mm) {
        float g[C2];
#pragma unroll
        for (int c = 0; c < C2; ++c) {
            float s = dXt2[mm * C2 + c];
#pragma unroll
            for (int kk = 0; kk < K2; ++kk) s += dZ2[mm * K2 + kk] * f.mA2[c * K2 + kk];
            g[c] = s;
            dot1 += s * T[o2 + mm * C2 + c];
        }
#pragma unroll
        for (int c = 0; c < C2; ++c) {
            float s = 0.f;
#pragma unroll
            for (int b = 0; b < C2; ++b) s += g[b] * f.mW2[c * C2 + b];
            T[o2 + mm * C2 + c] = s * f.iM1;
        }
    }
    if (L >= 3) {
#pragma unroll
        for (int mm = 0; mm < 7; ++mm) {
            const float g = dX3[mm];
            dot1 += g * T[o3 + mm];
            T[o3 + mm] = g * f.iM1;
        }
    }
    T[d.S] = (dM0 - dot0 * f.iM0) * 0.5f * f.iM0;
    T[d.S + 1] = (dM1 - dot1 * f.iM1) * 0.5f * f.iM1;
    __syncthreads();
    // write the block's slice back, coalesced
    float* dst = a.state + (size_t)b0 * d.SP;
    const int valid = nv * d.SP;
    int atom = 0, k = tid;
    for (int e = tid; e < valid; e += BLK) {
        while (k >= d.SP) { k -= d.SP; ++atom; }
        dst[e] = f.tile[k * PITCH + atom];
        k += BLK;
    }
}

template <bool FWD>
cudaError_t dispatch(const InvArgs& a, cudaStream_t st) {
    if (a.n <= 0) return cudaSuccess;
    const int blocks = (a.n + BLK - 1) / BLK;
    const int C1 = a.d.C[1], C2 = a.d.C[2], L = a.d.L;
#define UMLMD_CASE(c1, c2, l)                                                                   \
    if (C1 == c1 && C2 == c2 && L == l) {                                                       \
        const size_t bytes = sizeof(float) * Lay<c1, c2, l>::floats(a.d.SP, !FWD);              \
        auto kern = FWD ? k_inv_forward<c1, c2, l> : k_inv_backward<c1, c2, l>;                 \
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes); \
        if (e != cudaSuccess) return e;                                                         \
        kern<<<blocks, BLK, bytes, st>>>(a);                                                    \
        return cudaGetLastError();                                                              \
    }
    UMLMD_CASE(4, 4, 2) UMLMD_CASE(4, 4, 3) UMLMD_CASE(8, 4, 2) UMLMD_CASE(8, 4, 3)
    UMLMD_CASE(16, 8, 2) UMLMD_CASE(16, 8, 3)
#undef UMLMD_CASE
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_invariants_forward(const InvArgs& a, cudaStream_t st) { return dispatch<true>(a, st); }
cudaError_t launch_invariants_backward(const InvArgs& a, cudaStream_t st) { return dispatch<false>(a, st); }

}  // namespace umd
