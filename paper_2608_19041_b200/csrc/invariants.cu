// Per-atom readout front end: normalisation of the aggregated sums, channel alignment,
// Gram blocks, degree-wise low-rank probes, Cartesian bispectrum (closed forms for (1,1,2)
// and (2,2,2), sparse Gaunt contraction for the other triples), projected quartic
// invariant, assembly and diagonal calibration -- and the matching vector-Jacobian
// product, which turns dE/dD into dE/d(sums) in place of the saved sums.
//
// A block handles 64 atoms with 256 threads: four adjacent lanes share one atom.  All
// per-atom tensors live in shared memory in an [index][atom] layout with an odd row pitch
// (conflict-free for a warp's accesses).  Work is divided among an atom's four lanes so
// that no two lanes ever accumulate into the same entry: forward outputs are dealt out
// round-robin, backward accumulators are owned by harmonic row (each lane owns one
// degree-1 row and one or two degree-2 rows), so there are no atomics and the result is
// bitwise reproducible.  Global memory is only touched by block-cooperative, coalesced
// transfers: the block's slice of the state array is staged in one pass, and the feature
// vector streams through a 32-column staging buffer in increasing column order.
//
// The two normalising scales are standardised by the calibration, (M - mu) / sigma with
// mu ~ M, so they are formed in double precision from sums accumulated in double (stored
// as a float pair) to keep the subtraction from cancelling single-precision digits.
#include "kernels.h"

namespace umd {

namespace {

constexpr int ATOMS = 64;            // atoms per block
constexpr int LPA = 4;               // lanes per atom
constexpr int NT = ATOMS * LPA;      // threads per block
constexpr int PITCH = ATOMS + 1;
constexpr int CHUNK = 32;
constexpr unsigned kFull = 0xffffffffu;

constexpr float kR2 = 1.4142135623730951f;
constexpr float kInvR2 = 0.7071067811865476f;
constexpr float kInvR6 = 0.4082482904638631f;
constexpr float kC112 = -0.4472135954999579f;    // -1/sqrt(5)
constexpr float kC222 = -0.5855400437691199f;    // -sqrt(12/35)
constexpr float kR3 = 1.7320508075688772f;

// column of the [index][atom] shared-memory layout belonging to one atom
struct SCol {
    float* p;
    __device__ __forceinline__ float& operator[](int i) const { return p[i * PITCH]; }
};

// which of an atom's four lanes owns a harmonic row
__device__ __forceinline__ int own1(int m) { return m; }             // degree 1: rows 0,1,2 -> lanes 0,1,2
__device__ __forceinline__ int own2(int m) { return (m + 3) & 3; }   // degree 2: rows 0..4 -> lanes 3,0,1,2,3
__device__ __forceinline__ int own3(int m) { return m & 3; }         // degree 3: rows 0..6 round-robin

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
// picks component i of a 3-vector held in registers without a dynamic register index
__device__ __forceinline__ float pick3(const float* v, int i) { return i == 0 ? v[0] : (i == 1 ? v[1] : v[2]); }

// ---- feature-vector streaming through the 32-column staging buffer --------------------
// The per-column paths are force-inlined so that their state stays in registers; only the
// block-wide transfers (once per 32 columns) are real calls.

// write columns [kb, kb+32) of the block's feature vectors: lane = column, calibrated
__device__ __noinline__ void flush_columns(const float* chunk, float* Dg, const float* mu, const float* inv_sigma,
                                           int kb, int nv, int DP, int D_out, int k_skip0, int k_skip1) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = kb + lane;
    float mu_c = 0.f, is_c = 1.f;
    if (col < D_out && col != k_skip0 && col != k_skip1) { mu_c = __ldg(mu + col); is_c = __ldg(inv_sigma + col); }
    __syncthreads();
    for (int aa = warp; aa < nv; aa += NT / 32) Dg[(size_t)aa * DP + col] = (chunk[lane * PITCH + aa] - mu_c) * is_c;
    __syncthreads();
}
__device__ __forceinline__ void put_column(float* chunk, int at, int k, float v, bool own, float* Dg, const float* mu,
                                           const float* inv_sigma, int nv, int DP, int D_out, int k_skip0, int k_skip1) {
    if (own) chunk[(k & (CHUNK - 1)) * PITCH + at] = v;
    if ((k & (CHUNK - 1)) == CHUNK - 1) flush_columns(chunk, Dg, mu, inv_sigma, k - (CHUNK - 1), nv, DP, D_out, k_skip0, k_skip1);
}
// Backward streaming: columns [32c, 32c+32) of the block's dE/dD rows are fetched with
// asynchronous copies into one of two staging buffers while the previous 32 columns are
// being consumed, so the DRAM latency of the fetch is off the critical path.
__device__ __forceinline__ void issue_columns(float* buf, const float* dDg, int c, int nv, int DP) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = c * CHUNK + lane;
    if (col < DP) {
        for (int aa = warp; aa < nv; aa += NT / 32) {
            const unsigned dst = (unsigned)__cvta_generic_to_shared(buf + lane * PITCH + aa);
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(dDg + (size_t)aa * DP + col) : "memory");
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}
// make chunk c current (its copy was issued earlier) and start fetching chunk c + 1
__device__ __noinline__ void advance_columns(float* chunk2, const float* dDg, int c, int nv, int DP) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();                       // chunk c landed for everyone; everyone is done with chunk c - 1
    if ((c + 1) * CHUNK < DP) issue_columns(chunk2 + ((c + 1) & 1) * CHUNK * PITCH, dDg, c + 1, nv, DP);
}
__device__ __forceinline__ float get_column(float* chunk2, const float* isig_s, int at, int k, int& cur, const float* dDg,
                                            int nv, int DP) {
    const int c = k >> 5;
    if (c != cur) { advance_columns(chunk2, dDg, c, nv, DP); cur = c; }
    return chunk2[(c & 1) * CHUNK * PITCH + (k & (CHUNK - 1)) * PITCH + at] * isig_s[k];
}

template <int C1, int C2, int L>
struct Lay {                                  // shared-memory plan, in floats
    static constexpr int K1 = C2, K2 = 2;
    static constexpr int nZ1 = 3 * K1, nZ2 = 5 * K2;
    static constexpr int nMat = C1 * C1 + C2 * C2 + C1 * K1 + C2 * K2;
    static constexpr int nGaunt = L >= 3 ? 2 * (int)((sizeof(GauntSparse) + 3) / 4) : 0;
    // work rows: per-atom scalars (1/M0, dot0), Z1, Z2 [, dXt1, dXt2, dX3, dZ1, dZ2]
    static constexpr int nAux = 2;
    static constexpr int work_fwd = nAux + nZ1 + nZ2;
    static constexpr int work_bwd = nAux + nZ1 + nZ2 + 3 * C1 + 5 * C2 + 7 + nZ1 + nZ2;
    // the tile holds the state row without its leading C0 scalar sums (those are handled by
    // whole warps straight from global memory)
    static int floats(int SP, int C0, int DP, bool bwd) {
        return (SP - C0 + (bwd ? work_bwd + CHUNK : work_fwd) + CHUNK) * PITCH + nMat + nGaunt + (bwd ? DP : 0);
    }
};

// Shared setup of both passes: stage matrices and the block's state slice, then per atom
// normalise and align in place:  tile[offA1..] <- X1 (I + W1),  tile[offA2..] <- X2 (I + W2),
// tile[offA3..] <- X3, and form the probes Z1, Z2 (each row by its owner lane) and Q.
template <int C1, int C2, int L>
struct Front {
    static constexpr int K1 = C2, K2 = 2;
    float* tile; float* mW1; float* mW2; float* mA1; float* mA2;
    const GauntSparse* G123; const GauntSparse* G233;     // shared-memory copies of the sparse couplings
    SCol T, Z1, Z2, AUX;         // T[k] = state entry C0 + k of this atom
    double M0d, M1d;
    float iM0, iM1;
    float Q[K2][9];
    int nv, b0, at, r;

    __device__ __forceinline__ void setup(const InvArgs& a, float* sm, float* work, float* mats) {
        const Dims& d = a.d;
        const int tid = threadIdx.x;
        at = tid >> 2; r = tid & 3;
        tile = sm;
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
        b0 = blockIdx.x * ATOMS;
        nv = a.n - b0 < ATOMS ? a.n - b0 : ATOMS;
        const float* src = a.state + (size_t)b0 * d.SP;
        const int C0 = d.C0, TW = d.SP - C0;     // tile rows per atom
        const int total = ATOMS * TW;
        constexpr int US = 5;                    // loads in flight per thread
        for (int e0 = tid; e0 < total; e0 += US * NT) {
            float v[US];
            int slot[US];
#pragma unroll
            for (int u = 0; u < US; ++u) {
                const int e = e0 + u * NT;
                const int atom = e / TW, k = e - atom * TW;
                slot[u] = e < total ? k * PITCH + atom : -1;
                v[u] = (e < total && atom < nv) ? src[(size_t)atom * d.SP + C0 + k] : 0.f;
            }
#pragma unroll
            for (int u = 0; u < US; ++u)
                if (slot[u] >= 0) tile[slot[u]] = v[u];
        }
        __syncthreads();
        T.p = tile + at;
        AUX.p = work + at;
        Z1.p = work + 2 * PITCH + at;
        Z2.p = work + (2 + 3 * K1) * PITCH + at;
        const int oS = d.S - C0;
        M0d = sqrt(0.25 + (double)T[oS] + (double)T[oS + 2]);
        M1d = sqrt(0.25 + (double)T[oS + 1] + (double)T[oS + 3]);
        iM0 = (float)(1.0 / M0d); iM1 = (float)(1.0 / M1d);
        if (r == 0) AUX[0] = iM0;
        const int o1 = d.offA[1] - C0, o2 = d.offA[2] - C0, o3 = d.offA[3] - C0;
#pragma unroll
        for (int mm = 0; mm < 3; ++mm) {
            if (own1(mm) != r) continue;
            float x[C1], rr[C1];
#pragma unroll
            for (int c = 0; c < C1; ++c) { x[c] = T[o1 + mm * C1 + c] * iM1; rr[c] = 0.f; }
#pragma unroll
            for (int c = 0; c < C1; ++c)
#pragma unroll
                for (int b = 0; b < C1; ++b) rr[b] += x[c] * mW1[c * C1 + b];
#pragma unroll
            for (int b = 0; b < C1; ++b) T[o1 + mm * C1 + b] = rr[b];
#pragma unroll
            for (int kk = 0; kk < K1; ++kk) {
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < C1; ++c) s += rr[c] * mA1[c * K1 + kk];
                Z1[mm * K1 + kk] = s;
            }
        }
#pragma unroll
        for (int mm = 0; mm < 5; ++mm) {
            if (own2(mm) != r) continue;
            float x[C2], rr[C2];
#pragma unroll
            for (int c = 0; c < C2; ++c) { x[c] = T[o2 + mm * C2 + c] * iM1; rr[c] = 0.f; }
#pragma unroll
            for (int c = 0; c < C2; ++c)
#pragma unroll
                for (int b = 0; b < C2; ++b) rr[b] += x[c] * mW2[c * C2 + b];
#pragma unroll
            for (int b = 0; b < C2; ++b) T[o2 + mm * C2 + b] = rr[b];
#pragma unroll
            for (int kk = 0; kk < K2; ++kk) {
                float s = 0.f;
#pragma unroll
                for (int c = 0; c < C2; ++c) s += rr[c] * mA2[c * K2 + kk];
                Z2[mm * K2 + kk] = s;
            }
        }
        if (L >= 3) {
#pragma unroll
            for (int mm = 0; mm < 7; ++mm)
                if (own3(mm) == r) T[o3 + mm] = T[o3 + mm] * iM1;
        }
        __syncthreads();                         // rows, probes and 1/M0 visible to the whole block
#pragma unroll
        for (int e = 0; e < K2; ++e) stf9(Z2[e], Z2[K2 + e], Z2[2 * K2 + e], Z2[3 * K2 + e], Z2[4 * K2 + e], Q[e]);
    }
};

template <int C1, int C2, int L>
__global__ void __launch_bounds__(NT, 2) k_inv_forward(const InvArgs a) {
    constexpr int K1 = C2, K2 = 2;
    using LY = Lay<C1, C2, L>;
    extern __shared__ float sm[];
    const Dims& d = a.d;
    const ModelDev& m = a.m;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float* work = sm + (d.SP - d.C0) * PITCH;
    float* chunk = work + LY::work_fwd * PITCH;
    float* mats = chunk + CHUNK * PITCH;
    Front<C1, C2, L> f;
    f.setup(a, sm, work, mats);
    const SCol T = f.T, Z1 = f.Z1, Z2 = f.Z2;
    const int nv = f.nv, b0 = f.b0, C0 = d.C0, at = f.at, r = f.r;
    float* Dg = a.desc + (size_t)b0 * d.DP;
    const int ty = a.type_s[a.a0 + (b0 + at < a.n ? b0 + at : a.n - 1)];

    // Feature-vector columns are produced in increasing order, dealt round-robin to the
    // atom's four lanes; every 32nd column flushes the staging buffer.  The calibration
    // (v - mu) / sigma is applied by the flushing lane, which owns one column; the two
    // normalising scales arrive already calibrated (formed in double precision).
    const int kM0 = 2 * C0, kM1 = 2 * C0 + 1;
    int oc = 0;                                               // running output counter
#define mine() (((oc++) & 3) == r)
    const float* mu_g = m.mu;
    const float* is_g = m.inv_sigma;
    const int DPv = d.DP, Dov = d.D_out;
#define put(k, v, own) put_column(chunk, at, (k), (v), (own), Dg, mu_g, is_g, nv, DPv, Dov, kM0, kM1)

    // The first 2*C0 columns are plain per-column work -- the centre's initial features (a
    // gather by species) and the normalised scalar sums A_0 / M_0 -- so whole warps write
    // them straight from global memory, lane = column, for every complete group of 32
    // columns; a trailing partial group (only for C0 = 8) goes through the stream.
    const float* st_g = a.state + (size_t)b0 * d.SP;
    const int c_full = (2 * C0 / CHUNK) * CHUNK;
    for (int cb = 0; cb < c_full; cb += CHUNK) {
        const int col = cb + lane;
        const float mu_c = __ldg(m.mu + col), is_c = __ldg(m.inv_sigma + col);
        constexpr int UA = 8;
        float v[UA];
#pragma unroll
        for (int u = 0; u < UA; ++u) {
            const int aa = warp + u * (NT / 32);
            v[u] = 0.f;
            if (aa < nv) {
                if (col < C0) v[u] = __ldg(m.X0 + a.type_s[a.a0 + b0 + aa] * C0 + col);
                else v[u] = st_g[(size_t)aa * d.SP + (col - C0)];
            }
        }
#pragma unroll
        for (int u = 0; u < UA; ++u) {
            const int aa = warp + u * (NT / 32);
            if (aa < nv) {
                const float x = col < C0 ? v[u] : v[u] * f.AUX.p[aa - at];
                Dg[(size_t)aa * d.DP + col] = (x - mu_c) * is_c;
            }
        }
    }
    for (int c = c_full; c < 2 * C0; ++c) {
        const bool own = mine();
        float v = 0.f;
        if (own && at < nv) v = c < C0 ? __ldg(m.X0 + ty * C0 + c) : st_g[(size_t)at * d.SP + (c - C0)] * f.iM0;
        put(c, v, own);
    }
    put(kM0, (float)((f.M0d - (double)__ldg(m.mu + kM0)) * (double)__ldg(m.inv_sigma + kM0)), r == 0);
    put(kM1, (float)((f.M1d - (double)__ldg(m.mu + kM1)) * (double)__ldg(m.inv_sigma + kM1)), r == 0);
    const int o1 = d.offA[1] - C0, o2 = d.offA[2] - C0, o3 = d.offA[3] - C0;
    {   // Gram blocks, row-major upper triangle, strict off-diagonals times sqrt 2
        int k = d.oG[1];
        for (int p = 0; p < C1; ++p)
            for (int q = p; q < C1; ++q) {
                const bool own = mine();
                float s = 0.f;
                if (own) {
#pragma unroll
                    for (int mm = 0; mm < 3; ++mm) s += T[o1 + mm * C1 + p] * T[o1 + mm * C1 + q];
                }
                put(k++, p == q ? s : kR2 * s, own);
            }
        for (int p = 0; p < C2; ++p)
            for (int q = p; q < C2; ++q) {
                const bool own = mine();
                float s = 0.f;
                if (own) {
#pragma unroll
                    for (int mm = 0; mm < 5; ++mm) s += T[o2 + mm * C2 + p] * T[o2 + mm * C2 + q];
                }
                put(k++, p == q ? s : kR2 * s, own);
            }
        if (L >= 3) {
            const bool own = mine();
            float s = 0.f;
            if (own) {
#pragma unroll
                for (int mm = 0; mm < 7; ++mm) s += T[o3 + mm] * T[o3 + mm];
            }
            put(k++, s, own);
        }
    }
    {   // (1,1,2): -(1/sqrt5) v_k1^T Q_eta v_k2, k1 <= k2
        int k = d.oJ112;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int k2 = k1; k2 < K1; ++k2) {
#pragma unroll
                for (int e = 0; e < K2; ++e) {
                    const bool own = mine();
                    float val = 0.f;
                    if (own) {
                        float y[3];
                        matvec3(f.Q[e], Z1[k2], Z1[K1 + k2], Z1[2 * K1 + k2], y);
                        val = kC112 * (k1 == k2 ? 1.0f : kR2) * (Z1[k1] * y[0] + Z1[K1 + k1] * y[1] + Z1[2 * K1 + k1] * y[2]);
                    }
                    put(k++, val, own);
                }
            }
    }
    if (L >= 3) {   // (1,2,3): sparse Gaunt contraction
        const GauntSparse* G = f.G123;
        const int nn = G->n;
        int k = d.oJ123;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int e = 0; e < K2; ++e) {
                const bool own = mine();
                float s = 0.f;
                if (own)
                    for (int n = 0; n < nn; ++n)
                        s += G->v[n] * Z1[G->m1[n] * K1 + k1] * Z2[G->m2[n] * K2 + e] * T[o3 + G->m3[n]];
                put(k++, s, own);
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
                for (int e3 = e2; e3 < K2; ++e3) {
                    const bool own = mine();
                    put(k++, kC222 * fam3(e1, e2, e3) * trace_prod(P, f.Q[e3]), own);
                }
            }
    }
    if (L >= 3) {   // (2,3,3)
        const GauntSparse* G = f.G233;
        const int nn = G->n;
        int k = d.oJ233;
        for (int e = 0; e < K2; ++e) {
            const bool own = mine();
            float s = 0.f;
            if (own)
                for (int n = 0; n < nn; ++n) s += G->v[n] * Z2[G->m1[n] * K2 + e] * T[o3 + G->m2[n]] * T[o3 + G->m3[n]];
            put(k++, s, own);
        }
    }
    {   // projected quartic |Q_eta v_k|^2, eta-major
        int k = d.oPi;
#pragma unroll
        for (int e = 0; e < K2; ++e)
            for (int k1 = 0; k1 < K1; ++k1) {
                const bool own = mine();
                float val = 0.f;
                if (own) {
                    float y[3];
                    matvec3(f.Q[e], Z1[k1], Z1[K1 + k1], Z1[2 * K1 + k1], y);
                    val = y[0] * y[0] + y[1] * y[1] + y[2] * y[2];
                }
                put(k++, val, own);
            }
    }
    for (int k = d.D_out; k < d.DP; ++k) put(k, 0.f, r == 0);    // DP is a multiple of 32: ends on a flush
#undef put
#undef mine
}

template <int C1, int C2, int L>
__global__ void __launch_bounds__(NT, 2) k_inv_backward(const InvArgs a) {
    constexpr int K1 = C2, K2 = 2;
    using LY = Lay<C1, C2, L>;
    extern __shared__ float sm[];
    const Dims& d = a.d;
    const ModelDev& m = a.m;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float* work = sm + (d.SP - d.C0) * PITCH;
    float* chunk = work + LY::work_bwd * PITCH;            // two staging buffers of 32 columns
    float* mats = chunk + 2 * CHUNK * PITCH;
    float* isig_s = mats + LY::nMat + LY::nGaunt;          // 1 / sigma per column (0 beyond D_out)
    for (int k = threadIdx.x; k < d.DP; k += NT) isig_s[k] = k < d.D_out ? __ldg(a.m.inv_sigma + k) : 0.f;
    // start fetching the first streamed chunk (the one that holds column 2*C0) right away
    issue_columns(chunk + (((2 * d.C0) >> 5) & 1) * CHUNK * PITCH, a.desc + (size_t)blockIdx.x * ATOMS * d.DP, (2 * d.C0) >> 5,
                  a.n - (int)blockIdx.x * ATOMS < ATOMS ? a.n - (int)blockIdx.x * ATOMS : ATOMS, d.DP);
    Front<C1, C2, L> f;
    f.setup(a, sm, work, mats);
    const SCol T = f.T, Z1 = f.Z1, Z2 = f.Z2;
    const int nv = f.nv, b0 = f.b0, C0 = d.C0, at = f.at, r = f.r;
    const float* dDg = a.desc + (size_t)b0 * d.DP;
    float* wp = work + (LY::nAux + LY::nZ1 + LY::nZ2) * PITCH + at;
    const SCol dXt1{wp}, dXt2{wp + 3 * C1 * PITCH}, dX3{wp + (3 * C1 + 5 * C2) * PITCH},
        dZ1{wp + (3 * C1 + 5 * C2 + 7) * PITCH}, dZ2{wp + (3 * C1 + 5 * C2 + 7 + LY::nZ1) * PITCH},
        dQs{chunk + at};          // the staging buffer is free once the last column has been consumed
    // each lane clears the accumulators it owns
#pragma unroll
    for (int mm = 0; mm < 3; ++mm)
        if (own1(mm) == r) {
            for (int k = 0; k < C1; ++k) dXt1[mm * C1 + k] = 0.f;
            for (int k = 0; k < K1; ++k) dZ1[mm * K1 + k] = 0.f;
        }
#pragma unroll
    for (int mm = 0; mm < 5; ++mm)
        if (own2(mm) == r) {
            for (int k = 0; k < C2; ++k) dXt2[mm * C2 + k] = 0.f;
            for (int k = 0; k < K2; ++k) dZ2[mm * K2 + k] = 0.f;
        }
#pragma unroll
    for (int mm = 0; mm < 7; ++mm)
        if (own3(mm) == r) dX3[mm] = 0.f;
    // gradient of the two matrices Q: lane i < 3 accumulates row i of both in registers
    float dQ[K2][3];
#pragma unroll
    for (int e = 0; e < K2; ++e) { dQ[e][0] = 0.f; dQ[e][1] = 0.f; dQ[e][2] = 0.f; }

    // dE/dD columns are consumed in increasing order, 32 at a time, already divided by sigma
    int cur = -1;
    const int DPv = d.DP;
#define get(k) get_column(chunk, isig_s, at, (k), cur, dDg, nv, DPv)

    const int o1 = d.offA[1] - C0, o2 = d.offA[2] - C0, o3 = d.offA[3] - C0;
    // scalar block, X_0 = A_0 / M_0: whole warps, lane = channel, straight from / to global
    // memory; the per-atom sum over channels of X_0 dE/dX_0 lands in the second scalar row
    {
        float* __restrict__ st_g = a.state + (size_t)b0 * d.SP;
        const float* __restrict__ dd_g = dDg;
        constexpr int UA = 4;                           // atoms per batch: 4 x C0/32 x 2 loads in flight
        float isg[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) isg[j] = lane + 32 * j < C0 ? __ldg(m.inv_sigma + C0 + lane + 32 * j) : 0.f;
        for (int aa0 = warp; aa0 < nv; aa0 += UA * (NT / 32)) {
            float dx[UA][4], a0v[UA][4];
#pragma unroll
            for (int u = 0; u < UA; ++u) {
                const int aa = aa0 + u * (NT / 32);
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
                const int aa = aa0 + u * (NT / 32);
                if (aa >= nv) continue;
                const float im0 = f.AUX.p[aa - at];
                float part = 0.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int c = lane + 32 * j;
                    const float dxs = dx[u][j] * isg[j];
                    part += a0v[u][j] * im0 * dxs;
                    if (c < C0) st_g[(size_t)aa * d.SP + c] = dxs * im0;
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(kFull, part, off);
                if (lane == 0) f.AUX.p[PITCH + aa - at] = part;
            }
        }
        __syncthreads();
    }
    const float dot0 = f.AUX[1];
    const float dM0 = get(2 * C0), dM1 = get(2 * C0 + 1);
    {   // Gram: every lane walks all pairs and updates the rows it owns
        int k = d.oG[1];
        for (int p = 0; p < C1; ++p)
            for (int q = p; q < C1; ++q) {
                const float g = get(k++) * (p == q ? 1.0f : kR2);
                if (r < 3) {
                    const int mm = r;
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
                    if (own2(mm) != r) continue;
                    const float xp = T[o2 + mm * C2 + p], xq = T[o2 + mm * C2 + q];
                    dXt2[mm * C2 + p] += g * xq;
                    dXt2[mm * C2 + q] += g * xp;
                }
            }
        if (L >= 3) {
            const float g = get(k++);
#pragma unroll
            for (int mm = 0; mm < 7; ++mm)
                if (own3(mm) == r) dX3[mm] += 2.0f * g * T[o3 + mm];
        }
    }
    {   // (1,1,2): lane i < 3 owns component i of every probe gradient and row i of dQ
        int k = d.oJ112;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int k2 = k1; k2 < K1; ++k2) {
                const float v1[3] = {Z1[k1], Z1[K1 + k1], Z1[2 * K1 + k1]};
                const float v2[3] = {Z1[k2], Z1[K1 + k2], Z1[2 * K1 + k2]};
#pragma unroll
                for (int e = 0; e < K2; ++e) {
                    const float cf = get(k++) * kC112 * (k1 == k2 ? 1.0f : kR2);
                    if (r < 3) {
                        const float q0 = pick3(f.Q[e], r), q1 = pick3(f.Q[e] + 3, r), q2 = pick3(f.Q[e] + 6, r);   // row r (Q symmetric)
                        const float y2 = q0 * v2[0] + q1 * v2[1] + q2 * v2[2];
                        const float y1 = q0 * v1[0] + q1 * v1[1] + q2 * v1[2];
                        dZ1[r * K1 + k1] += cf * y2;
                        dZ1[r * K1 + k2] += cf * y1;
                        const float vr = pick3(v1, r);
#pragma unroll
                        for (int j = 0; j < 3; ++j) dQ[e][j] += cf * vr * v2[j];
                    }
                }
            }
    }
    if (L >= 3) {   // (1,2,3): each lane updates the targets whose rows it owns
        const GauntSparse* G = f.G123;
        const int nn = G->n;
        int k = d.oJ123;
        for (int k1 = 0; k1 < K1; ++k1)
            for (int e = 0; e < K2; ++e) {
                const float g = get(k++);
                for (int n = 0; n < nn; ++n) {
                    const int m1 = G->m1[n], m2 = G->m2[n], m3 = G->m3[n];
                    const bool w1 = own1(m1) == r, w2 = own2(m2) == r, w3 = own3(m3) == r;
                    if (!(w1 || w2 || w3)) continue;
                    const float cv = g * G->v[n];
                    const float z1 = Z1[m1 * K1 + k1], z2 = Z2[m2 * K2 + e], x3 = T[o3 + m3];
                    if (w1) dZ1[m1 * K1 + k1] += cv * z2 * x3;
                    if (w2) dZ2[m2 * K2 + e] += cv * z1 * x3;
                    if (w3) dX3[m3] += cv * z1 * z2;
                }
            }
    }
    {   // (2,2,2): d tr(Qa Qb Qc)/dQa_ij = (Qb Qc)_ji, and cyclically; lane i takes row i
        int k = d.oJ222;
#pragma unroll
        for (int e1 = 0; e1 < K2; ++e1)
#pragma unroll
            for (int e2 = e1; e2 < K2; ++e2)
#pragma unroll
                for (int e3 = e2; e3 < K2; ++e3) {
                    const float cf = get(k++) * kC222 * fam3(e1, e2, e3);
                    if (r < 3) {
                        float P[9];
                        matmul3(f.Q[e2], f.Q[e3], P);
#pragma unroll
                        for (int j = 0; j < 3; ++j) dQ[e1][j] += cf * pick3(P + 3 * j, r);
                        matmul3(f.Q[e3], f.Q[e1], P);
#pragma unroll
                        for (int j = 0; j < 3; ++j) dQ[e2][j] += cf * pick3(P + 3 * j, r);
                        matmul3(f.Q[e1], f.Q[e2], P);
#pragma unroll
                        for (int j = 0; j < 3; ++j) dQ[e3][j] += cf * pick3(P + 3 * j, r);
                    }
                }
    }
    if (L >= 3) {   // (2,3,3)
        const GauntSparse* G = f.G233;
        const int nn = G->n;
        int k = d.oJ233;
        for (int e = 0; e < K2; ++e) {
            const float g = get(k++);
            for (int n = 0; n < nn; ++n) {
                const int m1 = G->m1[n], m2 = G->m2[n], m3 = G->m3[n];
                const bool w1 = own2(m1) == r, w2 = own3(m2) == r, w3 = own3(m3) == r;
                if (!(w1 || w2 || w3)) continue;
                const float cv = g * G->v[n];
                const float z2 = Z2[m1 * K2 + e], xa = T[o3 + m2], xb = T[o3 + m3];
                if (w1) dZ2[m1 * K2 + e] += cv * xa * xb;
                if (w2) dX3[m2] += cv * z2 * xb;
                if (w3) dX3[m3] += cv * z2 * xa;
            }
        }
    }
    {   // quartic: y = Q v, Pi = y.y; lane i takes component i
        int k = d.oPi;
#pragma unroll
        for (int e = 0; e < K2; ++e)
            for (int k1 = 0; k1 < K1; ++k1) {
                const float g2 = 2.0f * get(k++);
                if (r < 3) {
                    const float v[3] = {Z1[k1], Z1[K1 + k1], Z1[2 * K1 + k1]};
                    float y[3];
                    matvec3(f.Q[e], v[0], v[1], v[2], y);
                    const float q0 = pick3(f.Q[e], r), q1 = pick3(f.Q[e] + 3, r), q2 = pick3(f.Q[e] + 6, r);
                    const float qy = q0 * y[0] + q1 * y[1] + q2 * y[2];
                    dZ1[r * K1 + k1] += g2 * qy;
                    const float yr = pick3(y, r);
#pragma unroll
                    for (int j = 0; j < 3; ++j) dQ[e][j] += g2 * yr * v[j];
                }
            }
    }
    // hand the rows of dQ to the degree-2 row owners through shared memory
    __syncwarp();
    if (r < 3) {
#pragma unroll
        for (int e = 0; e < K2; ++e)
#pragma unroll
            for (int j = 0; j < 3; ++j) dQs[e * 9 + 3 * r + j] = dQ[e][j];
    }
    __syncwarp();
    // transpose of the symmetric-trace-free map, then probes -> aligned features.
    // dot1 = sum dXt . Xt = sum dX . X (the alignment is linear)
    float dot1 = 0.f;
#pragma unroll
    for (int mm = 0; mm < 5; ++mm) {
        if (own2(mm) != r) continue;
#pragma unroll
        for (int e = 0; e < K2; ++e) {
            const float q0 = dQs[e * 9], q1 = dQs[e * 9 + 1], q2 = dQs[e * 9 + 2], q3 = dQs[e * 9 + 3], q4 = dQs[e * 9 + 4],
                        q5 = dQs[e * 9 + 5], q6 = dQs[e * 9 + 6], q7 = dQs[e * 9 + 7], q8 = dQs[e * 9 + 8];
            float add;
            if (mm == 0) add = kInvR2 * (q1 + q3);
            else if (mm == 1) add = kInvR2 * (q5 + q7);
            else if (mm == 2) add = kInvR6 * (2.0f * q8 - q0 - q4);
            else if (mm == 3) add = kInvR2 * (q2 + q6);
            else add = kInvR2 * (q0 - q4);
            dZ2[mm * K2 + e] += add;
        }
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
        for (int c = 0; c < C2; ++c) {         // dX = dXt (I + W)^T, then / M_1
            float s = 0.f;
#pragma unroll
            for (int b = 0; b < C2; ++b) s += g[b] * f.mW2[c * C2 + b];
            T[o2 + mm * C2 + c] = s * f.iM1;
        }
    }
#pragma unroll
    for (int mm = 0; mm < 3; ++mm) {
        if (own1(mm) != r) continue;
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
        for (int c = 0; c < C1; ++c) {
            float s = 0.f;
#pragma unroll
            for (int b = 0; b < C1; ++b) s += g[b] * f.mW1[c * C1 + b];
            T[o1 + mm * C1 + c] = s * f.iM1;
        }
    }
    if (L >= 3) {
#pragma unroll
        for (int mm = 0; mm < 7; ++mm) {
            if (own3(mm) != r) continue;
            const float g = dX3[mm];
            dot1 += g * T[o3 + mm];
            T[o3 + mm] = g * f.iM1;
        }
    }
    // combine the four lanes' partial dot products (fixed order)
    dot1 += __shfl_xor_sync(kFull, dot1, 1); dot1 += __shfl_xor_sync(kFull, dot1, 2);
    if (r == 0) {
        T[d.S - C0] = (dM0 - dot0 * f.iM0) * 0.5f * f.iM0;
        T[d.S - C0 + 1] = (dM1 - dot1 * f.iM1) * 0.5f * f.iM1;
    }
    __syncthreads();
    // write the block's slice back, coalesced
    float* dst = a.state + (size_t)b0 * d.SP;
    const int TW = d.SP - C0, total = nv * TW;
    int atom = 0, k = tid;
    for (int e = tid; e < total; e += NT) {
        while (k >= TW) { k -= TW; ++atom; }
        dst[(size_t)atom * d.SP + C0 + k] = f.tile[k * PITCH + atom];
        k += NT;
    }
#undef get
}

template <bool FWD>
cudaError_t dispatch(const InvArgs& a, cudaStream_t st) {
    if (a.n <= 0) return cudaSuccess;
    const int blocks = (a.n + ATOMS - 1) / ATOMS;
    const int C1 = a.d.C[1], C2 = a.d.C[2], L = a.d.L;
#define UMLMD_CASE(c1, c2, l)                                                                   \
    if (C1 == c1 && C2 == c2 && L == l) {                                                       \
        const size_t bytes = sizeof(float) * Lay<c1, c2, l>::floats(a.d.SP, a.d.C0, a.d.DP, !FWD);              \
        auto kern = FWD ? k_inv_forward<c1, c2, l> : k_inv_backward<c1, c2, l>;                 \
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes); \
        if (e != cudaSuccess) return e;                                                         \
        kern<<<blocks, NT, bytes, st>>>(a);                                                     \
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
