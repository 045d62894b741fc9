// Force / virial / energy assembly and the velocity-Verlet update.
//
// Forces: each atom is written by exactly one warp, which sums, over the atom's own CSR
// row, the gradient of each edge minus the gradient of its reverse edge (the reverse-edge
// map turns the source-sorted view into a gather).  No floating-point atomics anywhere,
// sums in double, fixed order, so results are bitwise reproducible.
#include <atomic>
#include "kernels.h"

namespace umd {

namespace {

constexpr int kRedBlock = 256;
constexpr int kRedMaxBlocks = 1024;

// out (caller numbering, through perm) and / or f (sorted numbering) may be null
__global__ void k_force_rows(int N, const eidx_t* __restrict__ row_ptr, const eidx_t* __restrict__ rev,
                             const float* __restrict__ g, double* __restrict__ f, const int* __restrict__ perm,
                             double* __restrict__ out, int* __restrict__ err) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= N) return;
    const eidx_t e0 = row_ptr[warp];
    const int len = (int)(row_ptr[warp + 1] - e0);
    double fx = 0, fy = 0, fz = 0;
    for (int k = lane; k < len; k += 32) {
        const eidx_t e = e0 + k;
        const float* a = g + 3 * (size_t)e;
        float bx = 0.f, by = 0.f, bz = 0.f;
        const eidx_t r = rev[e];
        if (r >= 0) { const float* b = g + 3 * (size_t)r; bx = b[0]; by = b[1]; bz = b[2]; }
        fx += (double)a[0] - (double)bx;
        fy += (double)a[1] - (double)by;
        fz += (double)a[2] - (double)bz;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        fx += __shfl_xor_sync(0xffffffffu, fx, off);
        fy += __shfl_xor_sync(0xffffffffu, fy, off);
        fz += __shfl_xor_sync(0xffffffffu, fz, off);
    }
    if (lane == 0) {
        if (f) { f[3 * (size_t)warp] = fx; f[3 * (size_t)warp + 1] = fy; f[3 * (size_t)warp + 2] = fz; }
        if (out) {
            const size_t o = 3 * (size_t)perm[warp];
            out[o] = fx; out[o + 1] = fy; out[o + 2] = fz;
            if (!isfinite(fx) || !isfinite(fy) || !isfinite(fz)) atomicOr(err, kErrNonFinite);
        }
    }
}

// Per-atom share of the virial, one warp per atom over its own row: every directed edge gives half
// of -g_e (x) r_e to its centre and half to its neighbour, so atom i collects
// -1/2 sum_{e in row(i)} (g_e - g_rev(e)) (x) r_e (the reverse edge has the opposite vector).
// Edge vectors are recomputed in double from the positions of the last evaluation.
struct CellRowsA { double h[9]; };
__global__ void k_atom_virial(int N, const eidx_t* __restrict__ row_ptr, const int* __restrict__ src,
                              const int* __restrict__ shift, const eidx_t* __restrict__ rev,
                              const float* __restrict__ g, const double* __restrict__ xs, CellRowsA H,
                              const int* __restrict__ perm, double* __restrict__ out) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= N) return;
    const eidx_t e0 = row_ptr[warp];
    const int len = (int)(row_ptr[warp + 1] - e0);
    const double xi = xs[3 * (size_t)warp], yi = xs[3 * (size_t)warp + 1], zi = xs[3 * (size_t)warp + 2];
    double w[9];
#pragma unroll
    for (int k = 0; k < 9; ++k) w[k] = 0.0;
    for (int k = lane; k < len; k += 32) {
        const eidx_t e = e0 + k;
        const float* a = g + 3 * (size_t)e;
        double d[3] = {(double)a[0], (double)a[1], (double)a[2]};
        const eidx_t r = rev[e];
        if (r >= 0) { const float* b = g + 3 * (size_t)r; d[0] -= (double)b[0]; d[1] -= (double)b[1]; d[2] -= (double)b[2]; }
        const int j = src[e], s = shift[e];
        const double nx = (double)(signed char)(s & 0xff), ny = (double)(signed char)((s >> 8) & 0xff),
                     nz = (double)(signed char)((s >> 16) & 0xff);
        const double* xj = xs + 3 * (size_t)j;
        const double rx = (xj[0] + ((nx * H.h[0] + ny * H.h[3]) + nz * H.h[6])) - xi;
        const double ry = (xj[1] + ((nx * H.h[1] + ny * H.h[4]) + nz * H.h[7])) - yi;
        const double rz = (xj[2] + ((nx * H.h[2] + ny * H.h[5]) + nz * H.h[8])) - zi;
#pragma unroll
        for (int p = 0; p < 3; ++p) { w[3 * p] += d[p] * rx; w[3 * p + 1] += d[p] * ry; w[3 * p + 2] += d[p] * rz; }
    }
#pragma unroll
    for (int k = 0; k < 9; ++k) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) w[k] += __shfl_xor_sync(0xffffffffu, w[k], off);
    }
    if (lane < 9) {
        double v = 0.0;
#pragma unroll
        for (int k = 0; k < 9; ++k) if (lane == k) v = w[k];
        out[9 * (size_t)perm[warp] + lane] = -0.5 * v;
    }
}

__global__ void k_scatter3(int N, const int* __restrict__ perm, const double* __restrict__ in,
                           double* __restrict__ out, int* __restrict__ err) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const int o = perm[i];
    bool bad = false;
    for (int k = 0; k < 3; ++k) {
        const double v = in[3 * (size_t)i + k];
        if (!isfinite(v)) bad = true;
        out[3 * (size_t)o + k] = v;
    }
    if (bad) atomicOr(err, kErrNonFinite);
}

__global__ void k_scatter1(int N, const int* __restrict__ perm, const double* __restrict__ in,
                           double* __restrict__ out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < N) out[perm[i]] = in[i];
}

__global__ void k_unsort_rows(int N, const int* __restrict__ perm, const float* __restrict__ in, int stride,
                              int width, float* __restrict__ out) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= N) return;
    const float* r = in + (size_t)warp * stride;
    float* w = out + (size_t)perm[warp] * width;
    for (int k = lane; k < width; k += 32) w[k] = r[k];
}

// flags[t] = 1 for every species that occurs (flags cleared by the caller); an index outside
// [0, T) is reported in the error word
__global__ void k_species_present(int64_t N, const int* __restrict__ type, int T, int* __restrict__ flags,
                                  int* __restrict__ err) {
    const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i >= N) return;
    const int t = type[i];
    if (t < 0 || t >= T) atomicOr(err, kErrSpecies);
    else if (flags[t] == 0) flags[t] = 1;
}

__device__ __forceinline__ double block_sum(double v, double* sh) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) sh[wid] = v;
    __syncthreads();
    double s = 0;
    if (threadIdx.x == 0) for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += sh[w];
    return s;   // valid in thread 0
}

// Segmented reduction of a batched evaluation: block f sums the atomic energies of frame f and,
// when asked, -g (x) r over the edges of the frame's rows (edge vectors recomputed from the
// positions and the frame's cell); thread-strided partial sums, then one fixed-order block sum.
__global__ void __launch_bounds__(kRedBlock) k_frame_reduce(const FrameCell* __restrict__ frames, const double* __restrict__ e_atom,
                                                            const eidx_t* __restrict__ row_ptr, const int* __restrict__ src,
                                                            const int* __restrict__ shift, const float* __restrict__ g,
                                                            const double* __restrict__ xs, bool want_virial,
                                                            double* __restrict__ out) {
    __shared__ double sh[kRedBlock / 32];
    const FrameCell& fc = frames[blockIdx.x];
    double e = 0, v[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
    for (int i = fc.a0 + threadIdx.x; i < fc.a1; i += kRedBlock) {
        e += e_atom[i];
        if (!want_virial) continue;
        const double xi = xs[3 * (size_t)i], yi = xs[3 * (size_t)i + 1], zi = xs[3 * (size_t)i + 2];
        for (eidx_t k = row_ptr[i]; k < row_ptr[i + 1]; ++k) {
            const int j = src[k], s = shift[k];
            const int nx = (int)(signed char)(s & 0xff), ny = (int)(signed char)((s >> 8) & 0xff), nz = (int)(signed char)((s >> 16) & 0xff);
            const double r[3] = {(xs[3 * (size_t)j] + ((nx * fc.H[0] + ny * fc.H[3]) + nz * fc.H[6])) - xi,
                                 (xs[3 * (size_t)j + 1] + ((nx * fc.H[1] + ny * fc.H[4]) + nz * fc.H[7])) - yi,
                                 (xs[3 * (size_t)j + 2] + ((nx * fc.H[2] + ny * fc.H[5]) + nz * fc.H[8])) - zi};
            const double gg[3] = {(double)g[3 * (size_t)k], (double)g[3 * (size_t)k + 1], (double)g[3 * (size_t)k + 2]};
            for (int a = 0; a < 3; ++a)
                for (int b = 0; b < 3; ++b) v[3 * a + b] += gg[a] * r[b];
        }
    }
    const double es = block_sum(e, sh);
    if (threadIdx.x == 0) out[10 * (size_t)blockIdx.x] = es;
    for (int k = 0; k < 9; ++k) {
        const double s = want_virial ? block_sum(v[k], sh) : 0.0;
        if (threadIdx.x == 0) out[10 * (size_t)blockIdx.x + 1 + k] = -s;
    }
}

// pass 1: block b sums the contiguous slice [b*chunk, (b+1)*chunk) of x
__global__ void __launch_bounds__(kRedBlock) k_sum_slices(const double* __restrict__ x, int64_t N, int64_t chunk,
                                                          double* __restrict__ part) {
    __shared__ double sh[kRedBlock / 32];
    const int64_t lo = (int64_t)blockIdx.x * chunk;
    const int64_t hi = lo + chunk < N ? lo + chunk : N;
    double v = 0;
    for (int64_t i = lo + threadIdx.x; i < hi; i += kRedBlock) v += x[i];
    const double s = block_sum(v, sh);
    if (threadIdx.x == 0) part[blockIdx.x] = s;
}

// pass 2 (ten blocks): block 0: out[0] = sum of slice partials; block 1 + k: out[1 + k] = -sum of
// the k-th component of the virial partials
__global__ void __launch_bounds__(kRedBlock) k_final_reduce(const double* __restrict__ part, int n_part,
                                                            const double* __restrict__ vpart, int n_vpart,
                                                            double* __restrict__ out, int* __restrict__ err) {
    __shared__ double sh[kRedBlock / 32];
    double v = 0;
    if (blockIdx.x == 0) {
        for (int i = threadIdx.x; i < n_part; i += kRedBlock) v += part[i];
        const double s = block_sum(v, sh);
        if (threadIdx.x == 0) {
            out[0] = s;
            if (!isfinite(s)) atomicOr(err, kErrNonFinite);
        }
    } else {
        const int k = blockIdx.x - 1;
        for (int i = threadIdx.x; i < n_vpart; i += kRedBlock) v += vpart[(size_t)i * 9 + k];
        const double s = block_sum(v, sh);
        if (threadIdx.x == 0) out[1 + k] = -s;
    }
}

// kicks = 0: none; kicks = 1: v += (dt/2) a; kicks = 2: the closing half kick of one step and the
// opening half kick of the next, applied one after the other exactly as two launches would; drift:
// x += dt v after them; scale (may be null): the thermostat's velocity factor, applied first
__global__ void k_vv(int64_t N, double* __restrict__ pos, double* __restrict__ vel, const double* __restrict__ force,
                     const int* __restrict__ type, const double* __restrict__ inv_mass, double dt, int kicks, bool drift,
                     const double* __restrict__ scale) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const double c = 0.5 * dt * kAccelUnit * inv_mass[type[i]];
    const double sc = scale ? *scale : 1.0;
    for (int k = 0; k < 3; ++k) {
        const double f = force[3 * i + k];
        double v = vel[3 * i + k];
        if (scale) v *= sc;
        if (kicks >= 1) v = v + c * f;
        if (kicks == 2) v = v + c * f;
        vel[3 * i + k] = v;
        if (drift) pos[3 * i + k] += dt * v;
    }
}

// Nose-Hoover chain of kNhcChain thermostats (Martyna-Tuckerman-Klein form): `halves` successive
// half-step propagations of the chain given the current kinetic energy; returns the product of the
// velocity scale factors and the kinetic energy after scaling.  One thread: the chain is a handful
// of scalars.  st = [eta[M], v_eta[M], scale, kinetic energy]
__global__ void k_nhc(double* __restrict__ st, const double* __restrict__ ke_in, int halves, NhcParams p) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    constexpr int M = kNhcChain;
    double* eta = st;
    double* v = st + M;
    double ke2 = 2.0 * (ke_in ? *ke_in : st[2 * M + 1]);
    double scale = 1.0;
    const double d2 = p.dt_half, d4 = 0.5 * d2, d8 = 0.25 * d2;
    for (int h = 0; h < halves; ++h) {
        double G = (p.Q[M - 2] * v[M - 2] * v[M - 2] - p.kT) / p.Q[M - 1];
        v[M - 1] += G * d4;
        for (int k = M - 2; k >= 0; --k) {
            const double e = exp(-v[k + 1] * d8);
            G = (k == 0 ? (ke2 - p.dof * p.kT) : (p.Q[k - 1] * v[k - 1] * v[k - 1] - p.kT)) / p.Q[k];
            v[k] = (v[k] * e + G * d4) * e;
        }
        const double sfac = exp(-v[0] * d2);
        scale *= sfac;
        ke2 *= sfac * sfac;
        for (int k = 0; k < M; ++k) eta[k] += v[k] * d2;
        for (int k = 0; k < M - 1; ++k) {
            const double e = exp(-v[k + 1] * d8);
            G = (k == 0 ? (ke2 - p.dof * p.kT) : (p.Q[k - 1] * v[k - 1] * v[k - 1] - p.kT)) / p.Q[k];
            v[k] = (v[k] * e + G * d4) * e;
        }
        G = (p.Q[M - 2] * v[M - 2] * v[M - 2] - p.kT) / p.Q[M - 1];
        v[M - 1] += G * d4;
    }
    st[2 * M] = scale;
    st[2 * M + 1] = 0.5 * ke2;
}

__global__ void __launch_bounds__(kRedBlock) k_ke_slices(const double* __restrict__ vel, const int* __restrict__ type,
                                                         const double* __restrict__ mass, int64_t N, int64_t chunk,
                                                         double* __restrict__ part) {
    __shared__ double sh[kRedBlock / 32];
    const int64_t lo = (int64_t)blockIdx.x * chunk;
    const int64_t hi = lo + chunk < N ? lo + chunk : N;
    double v = 0;
    for (int64_t i = lo + threadIdx.x; i < hi; i += kRedBlock) {
        const double vx = vel[3 * i], vy = vel[3 * i + 1], vz = vel[3 * i + 2];
        v += 0.5 * mass[type[i]] * (vx * vx + vy * vy + vz * vz) / kAccelUnit;
    }
    const double s = block_sum(v, sh);
    if (threadIdx.x == 0) part[blockIdx.x] = s;
}

__global__ void __launch_bounds__(kRedBlock) k_sum_small(const double* __restrict__ part, int n, double* out) {
    __shared__ double sh[kRedBlock / 32];
    double v = 0;
    for (int i = threadIdx.x; i < n; i += kRedBlock) v += part[i];
    const double s = block_sum(v, sh);
    if (threadIdx.x == 0) *out = s;
}

inline void slices(int64_t N, int* blocks, int64_t* chunk) {
    int64_t b = (N + 4095) / 4096;
    if (b < 1) b = 1;
    if (b > kRedMaxBlocks) b = kRedMaxBlocks;
    *blocks = (int)b;
    *chunk = (N + b - 1) / b;
}

}  // namespace

int reduce_scratch_doubles(int64_t) { return kRedMaxBlocks; }

// forces in sorted numbering (f_sorted) and / or scattered to the caller's numbering (d_force)
cudaError_t launch_force_assembly(const NeighborDev& nb, const float* g, double* f_sorted, double* d_force,
                                  int* d_err, cudaStream_t st) {
    const int N = (int)nb.N;
    if (N == 0) return cudaSuccess;
    k_force_rows<<<(N + 7) / 8, 256, 0, st>>>(N, nb.row_ptr, nb.rev, g, f_sorted, nb.perm, d_force, d_err);
    return cudaGetLastError();
}

cudaError_t launch_atom_virial(const NeighborDev& nb, const float* g, double* d_out, cudaStream_t st) {
    const int N = (int)nb.N;
    if (N == 0) return cudaSuccess;
    CellRowsA H;
    for (int k = 0; k < 9; ++k) H.h[k] = nb.H[k];
    k_atom_virial<<<(N + 7) / 8, 256, 0, st>>>(N, nb.row_ptr, nb.src, nb.shift, nb.rev, g, nb.xs, H, nb.perm, d_out);
    return cudaGetLastError();
}

cudaError_t launch_scatter_forces(const NeighborDev& nb, const double* f_sorted, double* d_force, int* d_err,
                                  cudaStream_t st) {
    const int N = (int)nb.N;
    if (N == 0) return cudaSuccess;
    k_scatter3<<<(N + 255) / 256, 256, 0, st>>>(N, nb.perm, f_sorted, d_force, d_err);
    return cudaGetLastError();
}

cudaError_t launch_scatter_atom_energy(const NeighborDev& nb, const double* e_sorted, double* d_out, cudaStream_t st) {
    const int N = (int)nb.N;
    if (N == 0) return cudaSuccess;
    k_scatter1<<<(N + 255) / 256, 256, 0, st>>>(N, nb.perm, e_sorted, d_out);
    return cudaGetLastError();
}

cudaError_t launch_frame_reduce(const NeighborDev& nb, const double* e_atom, const float* g, bool want_virial,
                                double* d_out, cudaStream_t st) {
    if (nb.n_frames <= 0) return cudaSuccess;
    k_frame_reduce<<<nb.n_frames, kRedBlock, 0, st>>>(nb.frames, e_atom, nb.row_ptr, nb.src, nb.shift, g, nb.xs, want_virial, d_out);
    return cudaGetLastError();
}

cudaError_t launch_reduce_energy_virial(const double* e_atom, int64_t N, const double* virial_part, int n_part,
                                        double* scratch, double* out, int* d_err, cudaStream_t st) {
    int blocks; int64_t chunk;
    slices(N, &blocks, &chunk);
    if (blocks == 1) {
        // a single slice: the second pass sums the atomic energies itself, in the order the first
        // pass would have used (its own sum over one partial only adds zeros), and one launch less
        k_final_reduce<<<10, kRedBlock, 0, st>>>(e_atom, (int)N, virial_part, n_part, out, d_err);
        return cudaGetLastError();
    }
    k_sum_slices<<<blocks, kRedBlock, 0, st>>>(e_atom, N, chunk, scratch);
    k_final_reduce<<<10, kRedBlock, 0, st>>>(scratch, blocks, virial_part, n_part, out, d_err);
    return cudaGetLastError();
}

cudaError_t launch_unsort_state(const NeighborDev& nb, const float* in, int stride, int width, float* out,
                                cudaStream_t st) {
    const int N = (int)nb.N;
    if (N == 0) return cudaSuccess;
    k_unsort_rows<<<(N + 7) / 8, 256, 0, st>>>(N, nb.perm, in, stride, width, out);
    return cudaGetLastError();
}

cudaError_t launch_species_present(int64_t N, const int* type, int T, int* d_flags, int* d_err, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(d_flags, 0, sizeof(int) * T, st);
    if (e != cudaSuccess || N == 0) return e;
    k_species_present<<<(unsigned)((N + 255) / 256), 256, 0, st>>>(N, type, T, d_flags, d_err);
    return cudaGetLastError();
}

cudaError_t launch_vv_kick_drift(int64_t N, double* pos, double* vel, const double* force, const int* type,
                                 const double* inv_mass, double dt, int kicks, bool drift, const double* d_scale,
                                 cudaStream_t st) {
    if (N == 0) return cudaSuccess;
    k_vv<<<(unsigned)((N + 255) / 256), 256, 0, st>>>(N, pos, vel, force, type, inv_mass, dt, kicks, drift, d_scale);
    return cudaGetLastError();
}

cudaError_t launch_nhc(double* d_state, const double* d_ke, int halves, const NhcParams& p, cudaStream_t st) {
    k_nhc<<<1, 32, 0, st>>>(d_state, d_ke, halves, p);
    return cudaGetLastError();
}

cudaError_t launch_kinetic_energy(int64_t N, const double* vel, const int* type, const double* mass,
                                  double* scratch, double* out, cudaStream_t st) {
    int blocks; int64_t chunk;
    slices(N, &blocks, &chunk);
    k_ke_slices<<<blocks, kRedBlock, 0, st>>>(vel, type, mass, N, chunk, scratch);
    k_sum_small<<<1, kRedBlock, 0, st>>>(scratch, blocks, out);
    return cudaGetLastError();
}

}  // namespace umd

// ---------------------------------------------------------------------------------------
// Kinetic energy without any allocation (see umlmd_kinetic_energy_static in umlmd.h).
//
// Same two kernels as launch_kinetic_energy; the only difference is where the per-block
// partial sums live: in a fixed array inside this library's device image instead of
// workspace obtained from cudaMalloc.
// ---------------------------------------------------------------------------------------
namespace umd {
namespace {

constexpr int64_t kStaticMaxAtoms = (int64_t)kRedMaxBlocks * 4096;      // 4,194,304
constexpr int kMaxDevices = 64;

// Partial sums of one reduction (8 KB).  Every GPU that loads the library holds a copy
// until the process exits.
static __device__ __align__(256) double g_static_partials[kRedMaxBlocks];

// g_static_partials is only a host-side handle in host code; the device address has to be
// asked for, once per device, with that device current.  The cached addresses are atomics: two
// host threads may make the first call on a device at the same time (both resolve the same
// address).  They belong to the device's primary context: after cudaDeviceReset they are stale,
// which the header states.
std::atomic<double*> g_static_partials_dev[kMaxDevices];
thread_local char g_static_err[256] = "";

int static_fail(int code, const char* msg) {
    snprintf(g_static_err, sizeof(g_static_err), "%s", msg);
    return code;
}

}  // namespace
}  // namespace umd

extern "C" int umlmd_kinetic_energy_static(int64_t N, const double* d_vel, const int32_t* d_type,
                                           const double* d_mass_per_type, double* d_e_kin, void* stream) {
    using namespace umd;
    if (N < 0 || !d_e_kin || (N > 0 && (!d_vel || !d_type || !d_mass_per_type)))
        return static_fail(UMLMD_E_INVALID_ARG, "umlmd_kinetic_energy_static: null pointer or negative atom count");
    if (N > kStaticMaxAtoms) {
        char msg[200];
        snprintf(msg, sizeof(msg), "umlmd_kinetic_energy_static: %lld atoms exceed the fixed scratch limit of %lld",
                 (long long)N, (long long)kStaticMaxAtoms);
        return static_fail(UMLMD_E_CAPACITY, msg);
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return static_fail(UMLMD_E_CUDA, "umlmd_kinetic_energy_static: no current CUDA device");
    double* partials = g_static_partials_dev[dev].load(std::memory_order_acquire);
    if (!partials) {
        double* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void**)&p, g_static_partials);
        if (e != cudaSuccess || !p) {
            char msg[200];
            snprintf(msg, sizeof(msg), "umlmd_kinetic_energy_static: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            return static_fail(UMLMD_E_CUDA, msg);
        }
        g_static_partials_dev[dev].store(p, std::memory_order_release);
        partials = p;
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // every partial that the final pass reads is written by the first pass of the same call,
    // so nothing left over from an earlier call needs clearing
    cudaError_t e = launch_kinetic_energy(N, d_vel, d_type, d_mass_per_type, partials, d_e_kin, st);
    if (e != cudaSuccess) {
        char msg[200];
        snprintf(msg, sizeof(msg), "umlmd_kinetic_energy_static: launch failed: %s", cudaGetErrorString(e));
        return static_fail(UMLMD_E_CUDA, msg);
    }
    return UMLMD_OK;
}

extern "C" const char* umlmd_static_last_error(void) { return umd::g_static_err; }
