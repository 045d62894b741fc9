// Per-atom readout front end: normalisation of the aggregated sums, channel alignment,
// Gram blocks, degree-wise low-rank probes, Cartesian bispectrum (closed forms for (1,1,2)
// and (2,2,2), sparse Gaunt contraction for the other triples), projected quartic
// invariant, assembly and diagonal calibration -- and the matching vector-Jacobian
// product, which turns dE/dD into dE/d(sums) in place of the saved sums.
//
// One thread per atom; the small per-atom tensors live in registers / thread-local memory
// (thread-interleaved, so the warp's accesses coalesce).
#include "kernels.h"

namespace umd {

namespace {

constexpr float kR2 = 1.4142135623730951f;
constexpr float kInvR2 = 0.7071067811865476f;
constexpr float kInvR6 = 0.4082482904638631f;
constexpr float kC112 = -0.4472135954999579f;    // -1/sqrt(5)
constexpr float kC222 = -0.5855400437691199f;    // -sqrt(12/35)
constexpr float kR3 = 1.7320508075688772f;

// symmetric trace-free matrix of a packed degree-2 vector, stored row-major 3x3
__device__ __forceinline__ void stf9(const float* z, int stride, float* Q) {
    const float z1 = z[0], z2 = z[stride], z3 = z[2 * stride], z4 = z[3 * stride], z5 = z[4 * stride];
    const float xx = -kInvR6 * z3 + kInvR2 * z5, yy = -kInvR6 * z3 - kInvR2 * z5, zz = 2.0f * kInvR6 * z3;
    const float xy = kInvR2 * z1, yz = kInvR2 * z2, xz = kInvR2 * z4;
    Q[0] = xx; Q[1] = xy; Q[2] = xz; Q[3] = xy; Q[4] = yy; Q[5] = yz; Q[6] = xz; Q[7] = yz; Q[8] = zz;
}
// transpose of that map: gradient with respect to the 9 matrix entries -> packed 5-vector
__device__ __forceinline__ void stf9_T(const float* dQ, float* dz, int stride) {
    dz[0] += kInvR2 * (dQ[1] + dQ[3]);
    dz[stride] += kInvR2 * (dQ[5] + dQ[7]);
    dz[2 * stride] += kInvR6 * (2.0f * dQ[8] - dQ[0] - dQ[4]);
    dz[3 * stride] += kInvR2 * (dQ[2] + dQ[6]);
    dz[4 * stride] += kInvR2 * (dQ[0] - dQ[4]);
}
__device__ __forceinline__ void matvec3(const float* Q, const float* v, int stride, float* y) {
    const float a = v[0], b = v[stride], c = v[2 * stride];
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

template <int C1, int C2, int L>
struct Feat {                      // per-atom intermediates shared by forward and backward
    static constexpr int K1 = C2, K2 = 2;
    float M0, M1, iM0, iM1;
    float X1[3 * C1], X2[5 * C2], X3[7];
    float Xt1[3 * C1], Xt2[5 * C2];
    float Z1[3 * K1], Z2[5 * K2];
    float Q[K2][9];
};

template <int C1, int C2, int L>
__device__ __forceinline__ void features(const Dims& d, const ModelDev& m, const float* row, Feat<C1, C2, L>& f) {
    constexpr int K1 = C2, K2 = 2;
    f.M0 = sqrtf(0.25f + row[d.S]);
    f.M1 = sqrtf(0.25f + row[d.S + 1]);
    f.iM0 = 1.0f / f.M0; f.iM1 = 1.0f / f.M1;
    for (int k = 0; k < 3 * C1; ++k) f.X1[k] = row[d.offA[1] + k] * f.iM1;
    for (int k = 0; k < 5 * C2; ++k) f.X2[k] = row[d.offA[2] + k] * f.iM1;
    if (L >= 3) for (int k = 0; k < 7; ++k) f.X3[k] = row[d.offA[3] + k] * f.iM1;
    for (int mm = 0; mm < 3; ++mm)
        for (int b = 0; b < C1; ++b) {
            float s = 0.f;
            for (int a = 0; a < C1; ++a) s += f.X1[mm * C1 + a] * __ldg(m.W1p + a * C1 + b);
            f.Xt1[mm * C1 + b] = s;
        }
    for (int mm = 0; mm < 5; ++mm)
        for (int b = 0; b < C2; ++b) {
            float s = 0.f;
            for (int a = 0; a < C2; ++a) s += f.X2[mm * C2 + a] * __ldg(m.W2p + a * C2 + b);
            f.Xt2[mm * C2 + b] = s;
        }
    for (int mm = 0; mm < 3; ++mm)
        for (int k = 0; k < K1; ++k) {
            float s = 0.f;
            for (int a = 0; a < C1; ++a) s += f.Xt1[mm * C1 + a] * __ldg(m.A1 + a * K1 + k);
            f.Z1[mm * K1 + k] = s;
        }
    for (int mm = 0; mm < 5; ++mm)
        for (int k = 0; k < K2; ++k) {
            float s = 0.f;
            for (int a = 0; a < C2; ++a) s += f.Xt2[mm * C2 + a] * __ldg(m.A2 + a * K2 + k);
            f.Z2[mm * K2 + k] = s;
        }
    for (int e = 0; e < K2; ++e) stf9(f.Z2 + e, K2, f.Q[e]);
}

// multiplicity weight sqrt(family size) of a non-decreasing triple of equal-degree indices
__device__ __forceinline__ float fam3(int a, int b, int c) {
    if (a == b && b == c) return 1.0f;
    if (a == b || b == c) return kR3;
    return 2.449489742783178f;
}

template <int C1, int C2, int L>
__global__ void __launch_bounds__(128) k_inv_forward(const InvArgs a) {
    constexpr int K1 = C2, K2 = 2;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= a.n) return;
    const Dims& d = a.d;
    const ModelDev& m = a.m;
    const float* row = a.state + (size_t)t * d.SP;
    float* D = a.desc + (size_t)t * d.DP;
    const int ty = a.type_s[a.a0 + t];
    Feat<C1, C2, L> f;
    features<C1, C2, L>(d, m, row, f);
    auto put = [&](int k, float v) { D[k] = (v - __ldg(m.mu + k)) * __ldg(m.inv_sigma + k); };
    const int C0 = d.C0;
    for (int c = 0; c < C0; ++c) {
        put(c, __ldg(m.X0 + ty * C0 + c));
        put(C0 + c, row[c] * f.iM0);
    }
    put(2 * C0, f.M0);
    put(2 * C0 + 1, f.M1);
    {   // Gram blocks, row-major upper triangle, strict off-diagonals times sqrt 2
        int k = d.oG[1];
        for (int p = 0; p < C1; ++p)
            for (int q = p; q < C1; ++q) {
                float s = 0.f;
                for (int mm = 0; mm < 3; ++mm) s += f.Xt1[mm * C1 + p] * f.Xt1[mm * C1 + q];
                put(k++, p == q ? s : kR2 * s);
            }
        k = d.oG[2];
        for (int p = 0; p < C2; ++p)
            for (int q = p; q < C2; ++q) {
                float s = 0.f;
                for (int mm = 0; mm < 5; ++mm) s += f.Xt2[mm * C2 + p] * f.Xt2[mm * C2 + q];
                put(k++, p == q ? s : kR2 * s);
            }
        if (L >= 3) {
            float s = 0.f;
            for (int mm = 0; mm < 7; ++mm) s += f.X3[mm] * f.X3[mm];
            put(d.oG[3], s);
        }
    }
    {   // (1,1,2): -(1/sqrt5) v_k1^T Q_eta v_k2, k1 <= k2
        int k = d.oJ112;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int k2 = k1; k2 < K1; ++k2)
                for (int e = 0; e < K2; ++e) {
                    float y[3];
                    matvec3(f.Q[e], f.Z1 + k2, K1, y);
                    const float s = f.Z1[k1] * y[0] + f.Z1[K1 + k1] * y[1] + f.Z1[2 * K1 + k1] * y[2];
                    put(k++, kC112 * (k1 == k2 ? 1.0f : kR2) * s);
                }
    }
    if (L >= 3) {   // (1,2,3): sparse Gaunt contraction
        const GauntSparse* G = m.g123;
        int k = d.oJ123;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int e = 0; e < K2; ++e) {
                float s = 0.f;
                for (int n = 0; n < G->n; ++n)
                    s += G->v[n] * f.Z1[G->m1[n] * K1 + k1] * f.Z2[G->m2[n] * K2 + e] * f.X3[G->m3[n]];
                put(k++, s);
            }
    }
    {   // (2,2,2): -sqrt(12/35) tr(Q Q Q), non-decreasing index triples
        int k = d.oJ222;
        for (int e1 = 0; e1 < K2; ++e1)
            for (int e2 = e1; e2 < K2; ++e2) {
                float P[9];
                matmul3(f.Q[e1], f.Q[e2], P);
                for (int e3 = e2; e3 < K2; ++e3) put(k++, kC222 * fam3(e1, e2, e3) * trace_prod(P, f.Q[e3]));
            }
    }
    if (L >= 3) {   // (2,3,3)
        const GauntSparse* G = m.g233;
        int k = d.oJ233;
        for (int e = 0; e < K2; ++e) {
            float s = 0.f;
            for (int n = 0; n < G->n; ++n) s += G->v[n] * f.Z2[G->m1[n] * K2 + e] * f.X3[G->m2[n]] * f.X3[G->m3[n]];
            put(k++, s);
        }
    }
    {   // projected quartic |Q_eta v_k|^2, eta-major
        int k = d.oPi;
        for (int e = 0; e < K2; ++e)
            for (int k1 = 0; k1 < K1; ++k1) {
                float y[3];
                matvec3(f.Q[e], f.Z1 + k1, K1, y);
                put(k++, y[0] * y[0] + y[1] * y[1] + y[2] * y[2]);
            }
    }
    for (int k = d.D_out; k < d.DP; ++k) D[k] = 0.f;
}

template <int C1, int C2, int L>
__global__ void __launch_bounds__(128) k_inv_backward(const InvArgs a) {
    constexpr int K1 = C2, K2 = 2;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= a.n) return;
    const Dims& d = a.d;
    const ModelDev& m = a.m;
    float* row = a.state + (size_t)t * d.SP;
    const float* dD = a.desc + (size_t)t * d.DP;
    Feat<C1, C2, L> f;
    features<C1, C2, L>(d, m, row, f);
    auto get = [&](int k) { return dD[k] * __ldg(m.inv_sigma + k); };
    const int C0 = d.C0;

    float dXt1[3 * C1], dXt2[5 * C2], dX3[7], dZ1[3 * K1], dZ2[5 * K2], dQ[K2][9];
    for (int k = 0; k < 3 * C1; ++k) dXt1[k] = 0.f;
    for (int k = 0; k < 5 * C2; ++k) dXt2[k] = 0.f;
    for (int k = 0; k < 7; ++k) dX3[k] = 0.f;
    for (int k = 0; k < 3 * K1; ++k) dZ1[k] = 0.f;
    for (int k = 0; k < 5 * K2; ++k) dZ2[k] = 0.f;
    for (int e = 0; e < K2; ++e) for (int k = 0; k < 9; ++k) dQ[e][k] = 0.f;

    {   // Gram
        int k = d.oG[1];
        for (int p = 0; p < C1; ++p)
            for (int q = p; q < C1; ++q) {
                const float g = get(k++) * (p == q ? 1.0f : kR2);
                for (int mm = 0; mm < 3; ++mm) {
                    const float xp = f.Xt1[mm * C1 + p], xq = f.Xt1[mm * C1 + q];
                    dXt1[mm * C1 + p] += g * xq;
                    dXt1[mm * C1 + q] += g * xp;
                }
            }
        k = d.oG[2];
        for (int p = 0; p < C2; ++p)
            for (int q = p; q < C2; ++q) {
                const float g = get(k++) * (p == q ? 1.0f : kR2);
                for (int mm = 0; mm < 5; ++mm) {
                    const float xp = f.Xt2[mm * C2 + p], xq = f.Xt2[mm * C2 + q];
                    dXt2[mm * C2 + p] += g * xq;
                    dXt2[mm * C2 + q] += g * xp;
                }
            }
        if (L >= 3) {
            const float g = get(d.oG[3]);
            for (int mm = 0; mm < 7; ++mm) dX3[mm] += 2.0f * g * f.X3[mm];
        }
    }
    {   // (1,1,2)
        int k = d.oJ112;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int k2 = k1; k2 < K1; ++k2)
                for (int e = 0; e < K2; ++e) {
                    const float cf = get(k++) * kC112 * (k1 == k2 ? 1.0f : kR2);
                    float y1[3], y2[3];
                    matvec3(f.Q[e], f.Z1 + k2, K1, y2);   // Q v2
                    matvec3(f.Q[e], f.Z1 + k1, K1, y1);   // Q v1
                    for (int i = 0; i < 3; ++i) {
                        dZ1[i * K1 + k1] += cf * y2[i];
                        dZ1[i * K1 + k2] += cf * y1[i];
                        for (int j = 0; j < 3; ++j) dQ[e][3 * i + j] += cf * f.Z1[i * K1 + k1] * f.Z1[j * K1 + k2];
                    }
                }
    }
    if (L >= 3) {   // (1,2,3)
        const GauntSparse* G = m.g123;
        int k = d.oJ123;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int e = 0; e < K2; ++e) {
                const float g = get(k++);
                for (int n = 0; n < G->n; ++n) {
                    const int i1 = G->m1[n] * K1 + k1, i2 = G->m2[n] * K2 + e, i3 = G->m3[n];
                    const float cv = g * G->v[n];
                    dZ1[i1] += cv * f.Z2[i2] * f.X3[i3];
                    dZ2[i2] += cv * f.Z1[i1] * f.X3[i3];
                    dX3[i3] += cv * f.Z1[i1] * f.Z2[i2];
                }
            }
    }
    {   // (2,2,2)
        int k = d.oJ222;
        for (int e1 = 0; e1 < K2; ++e1)
            for (int e2 = e1; e2 < K2; ++e2)
                for (int e3 = e2; e3 < K2; ++e3) {
                    const float cf = get(k++) * kC222 * fam3(e1, e2, e3);
                    float P[9];
                    // d tr(Qa Qb Qc)/dQa_ij = (Qb Qc)_ji, and cyclically
                    matmul3(f.Q[e2], f.Q[e3], P);
                    for (int i = 0; i < 3; ++i) for (int j = 0; j < 3; ++j) dQ[e1][3 * i + j] += cf * P[3 * j + i];
                    matmul3(f.Q[e3], f.Q[e1], P);
                    for (int i = 0; i < 3; ++i) for (int j = 0; j < 3; ++j) dQ[e2][3 * i + j] += cf * P[3 * j + i];
                    matmul3(f.Q[e1], f.Q[e2], P);
                    for (int i = 0; i < 3; ++i) for (int j = 0; j < 3; ++j) dQ[e3][3 * i + j] += cf * P[3 * j + i];
                }
    }
    if (L >= 3) {   // (2,3,3)
        const GauntSparse* G = m.g233;
        int k = d.oJ233;
        for (int e = 0; e < K2; ++e) {
            const float g = get(k++);
            for (int n = 0; n < G->n; ++n) {
                const int i1 = G->m1[n] * K2 + e, i2 = G->m2[n], i3 = G->m3[n];
                const float cv = g * G->v[n];
                dZ2[i1] += cv * f.X3[i2] * f.X3[i3];
                dX3[i2] += cv * f.Z2[i1] * f.X3[i3];
                dX3[i3] += cv * f.Z2[i1] * f.X3[i2];
            }
        }
    }
    {   // quartic
        int k = d.oPi;
        for (int e = 0; e < K2; ++e)
            for (int k1 = 0; k1 < K1; ++k1) {
                const float g2 = 2.0f * get(k++);
                float y[3], qy[3];
                matvec3(f.Q[e], f.Z1 + k1, K1, y);
                matvec3(f.Q[e], y, 1, qy);
                for (int i = 0; i < 3; ++i) {
                    dZ1[i * K1 + k1] += g2 * qy[i];
                    for (int j = 0; j < 3; ++j) dQ[e][3 * i + j] += g2 * y[i] * f.Z1[j * K1 + k1];
                }
            }
    }
    for (int e = 0; e < K2; ++e) stf9_T(dQ[e], dZ2 + e, K2);
    // probes -> aligned features
    for (int mm = 0; mm < 3; ++mm)
        for (int c = 0; c < C1; ++c) {
            float s = 0.f;
            for (int k = 0; k < K1; ++k) s += dZ1[mm * K1 + k] * __ldg(m.A1 + c * K1 + k);
            dXt1[mm * C1 + c] += s;
        }
    for (int mm = 0; mm < 5; ++mm)
        for (int c = 0; c < C2; ++c) {
            float s = 0.f;
            for (int k = 0; k < K2; ++k) s += dZ2[mm * K2 + k] * __ldg(m.A2 + c * K2 + k);
            dXt2[mm * C2 + c] += s;
        }
    // alignment transpose, normalisation, write dE/d(sums)
    float dot0 = 0.f, dot1 = 0.f;
    for (int c = 0; c < C0; ++c) {
        const float dx = get(C0 + c);
        dot0 += row[c] * f.iM0 * dx;
        row[c] = dx * f.iM0;
    }
    for (int mm = 0; mm < 3; ++mm)
        for (int c = 0; c < C1; ++c) {
            float s = 0.f;
            for (int b = 0; b < C1; ++b) s += dXt1[mm * C1 + b] * __ldg(m.W1p + c * C1 + b);
            dot1 += f.X1[mm * C1 + c] * s;
            row[d.offA[1] + mm * C1 + c] = s * f.iM1;
        }
    for (int mm = 0; mm < 5; ++mm)
        for (int c = 0; c < C2; ++c) {
            float s = 0.f;
            for (int b = 0; b < C2; ++b) s += dXt2[mm * C2 + b] * __ldg(m.W2p + c * C2 + b);
            dot1 += f.X2[mm * C2 + c] * s;
            row[d.offA[2] + mm * C2 + c] = s * f.iM1;
        }
    if (L >= 3)
        for (int mm = 0; mm < 7; ++mm) {
            dot1 += f.X3[mm] * dX3[mm];
            row[d.offA[3] + mm] = dX3[mm] * f.iM1;
        }
    row[d.S] = (get(2 * C0) - dot0 * f.iM0) * 0.5f * f.iM0;
    row[d.S + 1] = (get(2 * C0 + 1) - dot1 * f.iM1) * 0.5f * f.iM1;
}

template <bool FWD>
cudaError_t dispatch(const InvArgs& a, cudaStream_t st) {
    if (a.n <= 0) return cudaSuccess;
    const int TB = 128, blocks = (a.n + TB - 1) / TB;
    const int C1 = a.d.C[1], C2 = a.d.C[2], L = a.d.L;
#define UMLMD_CASE(c1, c2, l)                                                    \
    if (C1 == c1 && C2 == c2 && L == l) {                                        \
        if (FWD) k_inv_forward<c1, c2, l><<<blocks, TB, 0, st>>>(a);             \
        else k_inv_backward<c1, c2, l><<<blocks, TB, 0, st>>>(a);                \
        return cudaGetLastError();                                               \
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
