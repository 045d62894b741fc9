// Cell-list neighbor builder producing destination-sorted CSR edges.
//
// Atoms are folded into the cell, binned into cells at least r_list wide, sorted by cell
// (stable radix sort, so the internal numbering is deterministic) and renumbered in that
// order.  One warp per centre then walks the surrounding cells twice -- a count pass and a
// fill pass with an in-warp prefix count that keeps candidates in traversal order -- so the
// edge list comes out grouped by destination with no atomics and a reproducible order.
// A last pass finds, for every edge (i <- j, n), the slot of its reverse (j <- i, -n).
//
// The distance predicate is the paper's neighbor-set definition evaluated in double
// precision with explicit round-to-nearest adds and multiplies (no contraction into fused
// multiply-adds), which makes the edge set reproducible bit for bit.
#include <cub/cub.cuh>
#include <thrust/iterator/transform_iterator.h>

#include <cmath>
#include <cstring>

#include "alloc.h"
#include "kernels.h"

namespace umd {

namespace {

struct Grid {
    double L[3];        // cell edge lengths (orthorhombic cells)
    double H[9];        // cell vectors as rows; H[3 k + k] = L[k] for an orthorhombic cell
    double Hinv[9];     // inverse of H (general cells): fractional coordinates f = r Hinv
    int tri;            // general cell: fold and bin in fractional coordinates
    double lo[3];       // binning origin (Cartesian; fractional when tri)
    double inv_cw[3];   // 1 / bin width (per unit of the binning coordinate)
    int nc[3];          // bins per direction
    int m[3];           // bin reach per direction
    int pbc[3];
    int ncell;          // bins in all
    int halves;         // 2 when ghost atoms are binned apart from owned ones (keys ncell .. 2 ncell - 1), else 1
    int n_owned;        // caller indices >= n_owned are ghosts
    int sorted;         // every periodic direction has at least 2 m + 1 bins: bins are visited in
                        // increasing bin index, so each row comes out sorted by neighbour index
};

// first offset of the walk over the 2 m + 1 bins around bin c of a direction: the one whose wrapped
// bin index is smallest, so that the walk (continuing cyclically) visits bins in increasing index
__device__ __forceinline__ int walk_start(int c, int m, int nc, int pbc, int sorted) {
    if (!sorted || !pbc) return -m;
    if (c - m < 0) return -c;
    if (c + m >= nc) return nc - c;
    return -m;
}

__device__ __forceinline__ int floor_div(int a, int b) {
    int q = a / b;
    if ((a % b != 0) && ((a < 0) != (b < 0))) --q;
    return q;
}

__device__ __forceinline__ int pack_shift(int nx, int ny, int nz) {
    return (nx & 0xff) | ((ny & 0xff) << 8) | ((nz & 0xff) << 16);
}

struct CellRows { double h[9]; int tri; };

// order-preserving map of a double onto an unsigned integer, for atomicMin / atomicMax
__device__ __forceinline__ unsigned long long ordered_key(double x) {
    const long long b = __double_as_longlong(x);
    return b < 0 ? ~(unsigned long long)b : (unsigned long long)b | 0x8000000000000000ull;
}
inline double ordered_value(unsigned long long k) {
    const unsigned long long b = (k & 0x8000000000000000ull) ? (k & 0x7fffffffffffffffull) : ~k;
    double x;
    std::memcpy(&x, &b, sizeof(x));
    return x;
}
// smallest and largest binning coordinate of the atoms along each direction (Cartesian for an
// orthorhombic cell, fractional for a general one): keys[k] = min, keys[3 + k] = max
__global__ void k_bounds(int N, const double* __restrict__ pos, Grid g, unsigned long long* __restrict__ keys) {
    __shared__ unsigned long long smin[3][8], smax[3][8];
    unsigned long long mn[3] = {~0ull, ~0ull, ~0ull}, mx[3] = {0ull, 0ull, 0ull};
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < N; i += gridDim.x * blockDim.x) {
        const double x = pos[3 * (size_t)i], y = pos[3 * (size_t)i + 1], z = pos[3 * (size_t)i + 2];
        for (int k = 0; k < 3; ++k) {
            const double v = g.tri ? x * g.Hinv[k] + y * g.Hinv[3 + k] + z * g.Hinv[6 + k] : (k == 0 ? x : (k == 1 ? y : z));
            const unsigned long long key = ordered_key(v);
            if (key < mn[k]) mn[k] = key;
            if (key > mx[k]) mx[k] = key;
        }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int k = 0; k < 3; ++k) {
        for (int off = 16; off > 0; off >>= 1) {
            const unsigned long long a = __shfl_xor_sync(0xffffffffu, mn[k], off), b = __shfl_xor_sync(0xffffffffu, mx[k], off);
            if (a < mn[k]) mn[k] = a;
            if (b > mx[k]) mx[k] = b;
        }
        if (lane == 0) { smin[k][warp] = mn[k]; smax[k][warp] = mx[k]; }
    }
    __syncthreads();
    if (threadIdx.x < 3) {
        const int k = threadIdx.x;
        unsigned long long a = smin[k][0], b = smax[k][0];
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w) { if (smin[k][w] < a) a = smin[k][w]; if (smax[k][w] > b) b = smax[k][w]; }
        atomicMin(keys + k, a);
        atomicMax(keys + 3 + k, b);
    }
}

// fold positions into the cell, bin them
__global__ void k_fold_bin(int N, const double* __restrict__ pos, Grid g, double* __restrict__ wpos,
                           int* __restrict__ img_o, int* __restrict__ key, int* __restrict__ idx,
                           int* __restrict__ err) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    int c[3];
    bool bad = false;
    if (g.tri) {
        // general cell: f = r Hinv, fold by whole cell vectors along periodic directions (the same
        // arithmetic k_gather_positions applies later), bin by the folded fractional coordinate
        const double x = pos[3 * (size_t)i], y = pos[3 * (size_t)i + 1], z = pos[3 * (size_t)i + 2];
        if (!isfinite(x) || !isfinite(y) || !isfinite(z)) bad = true;
        double f[3], fl[3];
        for (int k = 0; k < 3; ++k) {
            f[k] = x * g.Hinv[k] + y * g.Hinv[3 + k] + z * g.Hinv[6 + k];
            fl[k] = g.pbc[k] ? floor(f[k]) : 0.0;
            if (fabs(fl[k]) > 1.0e6) bad = true;
            img_o[3 * (size_t)i + k] = bad ? 0 : (int)fl[k];
        }
        for (int k = 0; k < 3; ++k) {
            const double r = k == 0 ? x : (k == 1 ? y : z);
            wpos[3 * (size_t)i + k] = r - ((fl[0] * g.H[k] + fl[1] * g.H[3 + k]) + fl[2] * g.H[6 + k]);
            int ck = (int)floor(((f[k] - fl[k]) - g.lo[k]) * g.inv_cw[k]);
            ck = ck < 0 ? 0 : (ck >= g.nc[k] ? g.nc[k] - 1 : ck);
            c[k] = ck;
        }
    }
    for (int k = 0; k < 3 && !g.tri; ++k) {
        const double x = pos[3 * (size_t)i + k];
        if (!isfinite(x)) bad = true;
        double w = x;
        int fl = 0;
        if (g.pbc[k]) {
            const double frac = x / g.L[k];
            const double f = floor(frac);
            w = __dmul_rn(__dsub_rn(frac, f), g.L[k]);
            fl = (int)f;
            if (fabs(f) > 1.0e6) bad = true;
        }
        wpos[3 * (size_t)i + k] = w;
        img_o[3 * (size_t)i + k] = fl;
        int ck = (int)floor((w - g.lo[k]) * g.inv_cw[k]);
        ck = ck < 0 ? 0 : (ck >= g.nc[k] ? g.nc[k] - 1 : ck);
        c[k] = ck;
    }
    if (bad) {
        atomicOr(err, kErrNonFinite);
        c[0] = c[1] = c[2] = 0;
    }
    key[i] = (c[2] * g.nc[1] + c[1]) * g.nc[0] + c[0] + (i >= g.n_owned ? g.ncell : 0);
    idx[i] = i;
}

__global__ void k_cell_start(int ncell, int N, const int* __restrict__ skey, int* __restrict__ cell_start) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c > ncell) return;
    int lo = 0, hi = N;
    while (lo < hi) {
        const int mid = lo + ((hi - lo) >> 1);     // lo + hi would pass 2^31 in a long list
        if (skey[mid] < c) lo = mid + 1; else hi = mid;
    }
    cell_start[c] = lo;
}

__global__ void k_gather_sorted(int N, const int* __restrict__ sidx, const double* __restrict__ wpos,
                                const int* __restrict__ img_o, const int* __restrict__ type,
                                int* __restrict__ perm, double* __restrict__ xs0, double* __restrict__ xs,
                                int* __restrict__ img, int* __restrict__ type_s) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const int o = sidx[i];
    perm[i] = o;
    type_s[i] = type[o];
    for (int k = 0; k < 3; ++k) {
        const double w = wpos[3 * (size_t)o + k];
        xs0[3 * (size_t)i + k] = w;
        xs[3 * (size_t)i + k] = w;
        img[3 * (size_t)i + k] = img_o[3 * (size_t)o + k];
    }
}

// One warp per centre.  FILL = false: count accepted candidates.  FILL = true: write them.
template <bool FILL>
__global__ void k_scan_cells(int N, Grid g, double rl2, const int* __restrict__ skey,
                             const int* __restrict__ cell_start, const double* __restrict__ xs0,
                             int* __restrict__ deg, const eidx_t* __restrict__ row_ptr,
                             int* __restrict__ src, int* __restrict__ shift, int* __restrict__ err) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= N) return;
    const int i = warp;
    int key = skey[i];
    if (key >= g.ncell) key -= g.ncell;         // a ghost's own bin
    const int cx = key % g.nc[0], cy = (key / g.nc[0]) % g.nc[1], cz = key / (g.nc[0] * g.nc[1]);
    const double xi = xs0[3 * (size_t)i], yi = xs0[3 * (size_t)i + 1], zi = xs0[3 * (size_t)i + 2];
    int count = 0;
    const eidx_t base_out = FILL ? row_ptr[i] : 0;
    const unsigned lt_mask = (1u << lane) - 1u;
    const int wz = 2 * g.m[2] + 1, wy = 2 * g.m[1] + 1, wx = 2 * g.m[0] + 1;
    const int sz0 = walk_start(cz, g.m[2], g.nc[2], g.pbc[2], g.sorted);
    const int sy0 = walk_start(cy, g.m[1], g.nc[1], g.pbc[1], g.sorted);
    const int sx0 = walk_start(cx, g.m[0], g.nc[0], g.pbc[0], g.sorted);
    // with ghosts the bins are walked twice, owned atoms first: ghosts follow every owned atom in
    // the internal order, so the row still ascends in the neighbour index
    for (int half = 0; half < g.halves; ++half)
    for (int tz = 0; tz < wz; ++tz) {
        int dz = sz0 + tz;
        if (dz > g.m[2]) dz -= wz;
        int zc = cz + dz, nz = 0;
        if (g.pbc[2]) { nz = floor_div(zc, g.nc[2]); zc -= nz * g.nc[2]; }
        else if (zc < 0 || zc >= g.nc[2]) continue;
        // shift vector n . H, built up one cell vector per loop level without fused multiply-add;
        // for an orthorhombic cell all but one term of each component are exact zeros
        const double szx = __dmul_rn((double)nz, g.H[6]), szy = __dmul_rn((double)nz, g.H[7]),
                     szz = __dmul_rn((double)nz, g.H[8]);
        for (int ty = 0; ty < wy; ++ty) {
            int dy = sy0 + ty;
            if (dy > g.m[1]) dy -= wy;
            int yc = cy + dy, ny = 0;
            if (g.pbc[1]) { ny = floor_div(yc, g.nc[1]); yc -= ny * g.nc[1]; }
            else if (yc < 0 || yc >= g.nc[1]) continue;
            const double syx = __dadd_rn(szx, __dmul_rn((double)ny, g.H[3])), syy = __dadd_rn(szy, __dmul_rn((double)ny, g.H[4])),
                         syz = __dadd_rn(szz, __dmul_rn((double)ny, g.H[5]));
            for (int tx = 0, run = 1; tx < wx; tx += run) {
                int dx = sx0 + tx;
                if (dx > g.m[0]) dx -= wx;
                int xc = cx + dx, nx = 0;
                run = 1;
                if (g.pbc[0]) { nx = floor_div(xc, g.nc[0]); xc -= nx * g.nc[0]; }
                else if (xc < 0 || xc >= g.nc[0]) continue;
                // bins that follow one another along x with the same image hold consecutive atoms:
                // they are scanned as one range (same candidates in the same order, fuller warps)
                while (g.sorted && tx + run < wx) {
                    int dx2 = sx0 + tx + run;
                    if (dx2 > g.m[0]) dx2 -= wx;
                    int xc2 = cx + dx2, nx2 = 0;
                    if (g.pbc[0]) { nx2 = floor_div(xc2, g.nc[0]); xc2 -= nx2 * g.nc[0]; }
                    else if (xc2 < 0 || xc2 >= g.nc[0]) break;
                    if (nx2 != nx || xc2 != xc + run) break;
                    ++run;
                }
                const double sx = __dadd_rn(syx, __dmul_rn((double)nx, g.H[0])), sy = __dadd_rn(syy, __dmul_rn((double)nx, g.H[1])),
                             sz = __dadd_rn(syz, __dmul_rn((double)nx, g.H[2]));
                const int cell = (zc * g.nc[1] + yc) * g.nc[0] + xc + half * g.ncell;
                const int beg = cell_start[cell], end = cell_start[cell + run];
                const bool self_img = (nx == 0 && ny == 0 && nz == 0);
                for (int b = beg; b < end; b += 32) {
                    const int j = b + lane;
                    bool ok = false;
                    if (j < end) {
                        const double ddx = __dsub_rn(__dadd_rn(xs0[3 * (size_t)j], sx), xi);
                        const double ddy = __dsub_rn(__dadd_rn(xs0[3 * (size_t)j + 1], sy), yi);
                        const double ddz = __dsub_rn(__dadd_rn(xs0[3 * (size_t)j + 2], sz), zi);
                        const double d2 = __dadd_rn(__dadd_rn(__dmul_rn(ddx, ddx), __dmul_rn(ddy, ddy)),
                                                    __dmul_rn(ddz, ddz));
                        ok = (d2 < rl2) && !(self_img && j == i);
                    }
                    const unsigned mask = __ballot_sync(0xffffffffu, ok);
                    if (FILL && ok) {
                        const eidx_t p = base_out + count + __popc(mask & lt_mask);
                        src[p] = j;
                        shift[p] = pack_shift(nx, ny, nz);
                    }
                    count += __popc(mask);
                }
                if (nx < -127 || nx > 127 || ny < -127 || ny > 127 || nz < -127 || nz > 127)
                    if (lane == 0) atomicOr(err, kErrShiftRange);
            }
        }
    }
    if (!FILL && lane == 0) deg[i] = count;
}

// rev[e] = slot of (j <- i, -n) for e = (i <- j, n); -1 when absent (can only happen for
// pairs whose two orientations round to opposite sides of the list radius).
__global__ void k_reverse_map(int N, int sorted, const eidx_t* __restrict__ row_ptr, const int* __restrict__ src,
                              const int* __restrict__ shift, eidx_t* __restrict__ rev) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= N) return;
    const int i = warp;
    const eidx_t e0 = row_ptr[i];
    const int len = (int)(row_ptr[i + 1] - e0);
    for (int k = lane; k < len; k += 32) {
        const eidx_t e = e0 + k;
        const int j = src[e];
        const int s = shift[e];
        const int nx = (int)(signed char)(s & 0xff), ny = (int)(signed char)((s >> 8) & 0xff),
                  nz = (int)(signed char)((s >> 16) & 0xff);
        const int want = pack_shift(-nx, -ny, -nz);
        eidx_t found = -1;
        const eidx_t f0 = row_ptr[j];
        const int flen = (int)(row_ptr[j + 1] - f0);
        const int* srow = src + f0;
        const int* hrow = shift + f0;
        if (sorted) {          // rows ascend in the neighbour index, each neighbour at most once
            int lo = 0, hi = flen;
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;            // offsets inside one row: no overflow
                if (srow[mid] < i) lo = mid + 1; else hi = mid;
            }
            if (lo < flen && srow[lo] == i && hrow[lo] == want) found = f0 + lo;
        } else {
            for (int f = 0; f < flen; ++f) {
                if (srow[f] == i && hrow[f] == want) { found = f0 + f; break; }
            }
        }
        rev[e] = found;
    }
}

// ---- batched frames -------------------------------------------------------------------------
// fold the atoms of frame blockIdx.x into its cell, write positions, records, species, frame index
__global__ void k_batch_fold(const FrameCell* __restrict__ frames, const double* __restrict__ pos,
                             const int* __restrict__ type, int T, double* __restrict__ xs, float4* __restrict__ rec,
                             int* __restrict__ type_s, int* __restrict__ frame_of, int* __restrict__ perm,
                             int* __restrict__ err) {
    const FrameCell& fc = frames[blockIdx.x];
    for (int i = fc.a0 + threadIdx.x; i < fc.a1; i += blockDim.x) {
        const double x = pos[3 * (size_t)i], y = pos[3 * (size_t)i + 1], z = pos[3 * (size_t)i + 2];
        bool bad = !isfinite(x) || !isfinite(y) || !isfinite(z);
        double fl[3];
        for (int k = 0; k < 3; ++k) {
            const double f = x * fc.Hinv[k] + y * fc.Hinv[3 + k] + z * fc.Hinv[6 + k];
            fl[k] = fc.pbc[k] ? floor(f) : 0.0;
            if (!(fabs(fl[k]) <= 1.0e6)) { bad = true; fl[k] = 0.0; }
        }
        float hi[3], lo[3];
        for (int k = 0; k < 3; ++k) {
            const double r = k == 0 ? x : (k == 1 ? y : z);
            const double w = bad ? 0.0 : r - ((fl[0] * fc.H[k] + fl[1] * fc.H[3 + k]) + fl[2] * fc.H[6 + k]);
            xs[3 * (size_t)i + k] = w;
            hi[k] = (float)w;
            lo[k] = (float)(w - (double)hi[k]);
        }
        int t = type[i];
        if (t < 0 || t >= T) { atomicOr(err, kErrSpecies); t = 0; }
        if (bad) atomicOr(err, kErrNonFinite);
        rec[2 * (size_t)i] = make_float4(hi[0], hi[1], hi[2], __int_as_float(t));
        rec[2 * (size_t)i + 1] = make_float4(lo[0], lo[1], lo[2], 0.f);
        type_s[i] = t;
        frame_of[i] = blockIdx.x;
        perm[i] = i;
    }
}

// One warp per centre: every atom of the centre's frame under every image within reach, in the
// order image (z slowest), then atom; the same double-precision predicate as the cell-list scan.
template <bool FILL>
__global__ void k_batch_scan(int N, const FrameCell* __restrict__ frames, const int* __restrict__ frame_of, double rl2,
                             const double* __restrict__ xs, int* __restrict__ deg, const eidx_t* __restrict__ row_ptr,
                             int* __restrict__ src, int* __restrict__ shift) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= N) return;
    const int i = warp;
    const FrameCell& fc = frames[frame_of[i]];
    const double xi = xs[3 * (size_t)i], yi = xs[3 * (size_t)i + 1], zi = xs[3 * (size_t)i + 2];
    const unsigned lt_mask = (1u << lane) - 1u;
    const eidx_t base_out = FILL ? row_ptr[i] : 0;
    int count = 0;
    for (int nz = -fc.m[2]; nz <= fc.m[2]; ++nz) {
        const double szx = __dmul_rn((double)nz, fc.H[6]), szy = __dmul_rn((double)nz, fc.H[7]), szz = __dmul_rn((double)nz, fc.H[8]);
        for (int ny = -fc.m[1]; ny <= fc.m[1]; ++ny) {
            const double syx = __dadd_rn(szx, __dmul_rn((double)ny, fc.H[3])), syy = __dadd_rn(szy, __dmul_rn((double)ny, fc.H[4])),
                         syz = __dadd_rn(szz, __dmul_rn((double)ny, fc.H[5]));
            for (int nx = -fc.m[0]; nx <= fc.m[0]; ++nx) {
                const double sx = __dadd_rn(syx, __dmul_rn((double)nx, fc.H[0])), sy = __dadd_rn(syy, __dmul_rn((double)nx, fc.H[1])),
                             sz = __dadd_rn(syz, __dmul_rn((double)nx, fc.H[2]));
                const bool self_img = nx == 0 && ny == 0 && nz == 0;
                for (int b = fc.a0; b < fc.a1; b += 32) {
                    const int j = b + lane;
                    bool ok = false;
                    if (j < fc.a1) {
                        const double ddx = __dsub_rn(__dadd_rn(xs[3 * (size_t)j], sx), xi);
                        const double ddy = __dsub_rn(__dadd_rn(xs[3 * (size_t)j + 1], sy), yi);
                        const double ddz = __dsub_rn(__dadd_rn(xs[3 * (size_t)j + 2], sz), zi);
                        const double d2 = __dadd_rn(__dadd_rn(__dmul_rn(ddx, ddx), __dmul_rn(ddy, ddy)), __dmul_rn(ddz, ddz));
                        ok = (d2 < rl2) && !(self_img && j == i);
                    }
                    const unsigned mask = __ballot_sync(0xffffffffu, ok);
                    if (FILL && ok) {
                        const eidx_t p = base_out + count + __popc(mask & lt_mask);
                        src[p] = j;
                        shift[p] = pack_shift(nx, ny, nz);
                    }
                    count += __popc(mask);
                }
            }
        }
    }
    if (!FILL && lane == 0) deg[i] = count;
}

__global__ void k_gather_positions(int N, const int* __restrict__ perm, const int* __restrict__ img,
                                   const double* __restrict__ pos, const double* __restrict__ xs0,
                                   CellRows H, double max_disp2, const int* __restrict__ type_s,
                                   double* __restrict__ xs, float4* __restrict__ rec, int* __restrict__ err) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const int o = perm[i];
    const double n0 = (double)img[3 * (size_t)i], n1 = (double)img[3 * (size_t)i + 1], n2 = (double)img[3 * (size_t)i + 2];
    double d2 = 0;
    bool bad = false;
    float hi[3], lo[3];
    for (int k = 0; k < 3; ++k) {
        const double x = H.tri ? pos[3 * (size_t)o + k] - ((n0 * H.h[k] + n1 * H.h[3 + k]) + n2 * H.h[6 + k])
                               : pos[3 * (size_t)o + k] - (double)img[3 * (size_t)i + k] * H.h[4 * k];
        if (!isfinite(x)) bad = true;
        xs[3 * (size_t)i + k] = x;
        hi[k] = (float)x;
        lo[k] = (float)(x - (double)hi[k]);
        const double d = x - xs0[3 * (size_t)i + k];
        d2 += d * d;
    }
    rec[2 * (size_t)i] = make_float4(hi[0], hi[1], hi[2], __int_as_float(type_s[i]));
    rec[2 * (size_t)i + 1] = make_float4(lo[0], lo[1], lo[2], 0.f);
    if (bad) atomicOr(err, kErrNonFinite);
    else if (d2 > max_disp2) atomicOr(err, kErrStale);
}

// ---- export in caller numbering ------------------------------------------------------
__global__ void k_export_deg(int N, const int* __restrict__ perm, const eidx_t* __restrict__ row_ptr,
                             int* __restrict__ deg_o) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    deg_o[perm[i]] = (int)(row_ptr[i + 1] - row_ptr[i]);
    if (i == 0) deg_o[N] = 0;
}

__global__ void k_export_rows(int N, const int* __restrict__ perm, const eidx_t* __restrict__ row_ptr,
                              const int* __restrict__ src, const int* __restrict__ shift,
                              const int* __restrict__ row_ptr_o, int* __restrict__ src_o,
                              signed char* __restrict__ shift_o) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= N) return;
    const int i = warp, o = perm[i];
    const eidx_t e0 = row_ptr[i];
    const int n = (int)(row_ptr[i + 1] - e0), q0 = row_ptr_o[o];
    for (int k = lane; k < n; k += 32) {
        const int s = shift[e0 + k];
        src_o[q0 + k] = perm[src[e0 + k]];
        shift_o[3 * (size_t)(q0 + k)] = (signed char)(s & 0xff);
        shift_o[3 * (size_t)(q0 + k) + 1] = (signed char)((s >> 8) & 0xff);
        shift_o[3 * (size_t)(q0 + k) + 2] = (signed char)((s >> 16) & 0xff);
    }
}

// the same export restricted to the centres first .. first + n - 1 of the caller's numbering, with
// 64-bit row offsets (a list may hold more than 2^31 edges; a range of rows rarely does)
__global__ void k_export_deg_range(int N, int first, int n, const int* __restrict__ perm,
                                   const eidx_t* __restrict__ row_ptr, int* __restrict__ deg_o) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) deg_o[n] = 0;
    if (i >= N) return;
    const int o = perm[i] - first;
    if (o >= 0 && o < n) deg_o[o] = (int)(row_ptr[i + 1] - row_ptr[i]);
}

__global__ void k_export_rows_range(int N, int first, int n, const int* __restrict__ perm,
                                    const eidx_t* __restrict__ row_ptr, const int* __restrict__ src,
                                    const int* __restrict__ shift, const long long* __restrict__ row_ptr_o,
                                    long long cap, int* __restrict__ src_o, signed char* __restrict__ shift_o) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= N) return;
    const int o = perm[warp] - first;
    if (o < 0 || o >= n) return;
    const eidx_t e0 = row_ptr[warp];
    const int len = (int)(row_ptr[warp + 1] - e0);
    const long long q0 = row_ptr_o[o];
    for (int k = lane; k < len; k += 32) {
        if (q0 + k >= cap) break;
        const int s = shift[e0 + k];
        src_o[q0 + k] = perm[src[e0 + k]];
        shift_o[3 * (size_t)(q0 + k)] = (signed char)(s & 0xff);
        shift_o[3 * (size_t)(q0 + k) + 1] = (signed char)((s >> 8) & 0xff);
        shift_o[3 * (size_t)(q0 + k) + 2] = (signed char)((s >> 16) & 0xff);
    }
}

struct WidenDeg {
    __host__ __device__ eidx_t operator()(int v) const { return (eidx_t)v; }
};

#define NB_CHECK(call)                                                              \
    do {                                                                            \
        cudaError_t e__ = (call);                                                   \
        if (e__ != cudaSuccess) {                                                   \
            *err = std::string(#call) + ": " + cudaGetErrorString(e__);             \
            return UMLMD_E_CUDA;                                                    \
        }                                                                           \
    } while (0)

}  // namespace

void neighbor_free(NeighborDev* nb) {
    void* ptrs[] = {nb->frames, nb->rec, nb->wpos, nb->img, nb->perm, nb->type_s, nb->xs0, nb->xs, nb->row_ptr, nb->src,
                    nb->shift, nb->rev, nb->key, nb->key2, nb->idx, nb->idx2, nb->cell_start, nb->deg,
                    nb->cub_tmp, nb->bounds};
    for (void* p : ptrs)
        dev_free(p);
    *nb = NeighborDev();
}

int neighbor_build(NeighborDev* nb, int64_t N64, int64_t n_owned64, const double* d_pos, const int32_t* d_type,
                   const double cell[9], const int pbc[3], double skin, double rc, int* d_err,
                   cudaStream_t st, std::string* err) {
    if (N64 > 0x7fff0000LL) { *err = "too many atoms for 32-bit indices"; return UMLMD_E_INVALID_ARG; }
    const int N = (int)N64;
    const int n_owned = n_owned64 < 0 || n_owned64 > N64 ? N : (int)n_owned64;
    const double r_list = rc + skin;
    nb->batch = false; nb->n_frames = 0; nb->frame_of = nullptr;
    Grid g;
    const double L[3] = {cell[0], cell[4], cell[8]};
    g.tri = 0;
    for (int k = 0; k < 9; ++k) { g.H[k] = cell[k]; g.Hinv[k] = 0; if (k % 4 != 0 && cell[k] != 0.0) g.tri = 1; }
    // perpendicular height of the cell along each cell vector (the edge length when orthorhombic)
    double height[3] = {L[0], L[1], L[2]};
    if (g.tri) {
        const double* h = cell;
        const double c00 = h[4] * h[8] - h[5] * h[7], c01 = h[5] * h[6] - h[3] * h[8], c02 = h[3] * h[7] - h[4] * h[6];
        const double det = h[0] * c00 + h[1] * c01 + h[2] * c02;
        const double scale = std::fabs(h[0]) + std::fabs(h[1]) + std::fabs(h[2]) + std::fabs(h[3]) + std::fabs(h[4]) +
                             std::fabs(h[5]) + std::fabs(h[6]) + std::fabs(h[7]) + std::fabs(h[8]);
        if (!(std::fabs(det) > 1e-12 * scale * scale * scale)) { *err = "singular cell"; return UMLMD_E_UNSUPPORTED_CELL; }
        const double id = 1.0 / det;
        g.Hinv[0] = c00 * id; g.Hinv[3] = c01 * id; g.Hinv[6] = c02 * id;
        g.Hinv[1] = (h[2] * h[7] - h[1] * h[8]) * id; g.Hinv[4] = (h[0] * h[8] - h[2] * h[6]) * id; g.Hinv[7] = (h[1] * h[6] - h[0] * h[7]) * id;
        g.Hinv[2] = (h[1] * h[5] - h[2] * h[4]) * id; g.Hinv[5] = (h[2] * h[3] - h[0] * h[5]) * id; g.Hinv[8] = (h[0] * h[4] - h[1] * h[3]) * id;
        for (int k = 0; k < 3; ++k)     // f_k = r . column k of Hinv: planes of constant f_k are 1 / |column| apart
            height[k] = 1.0 / std::sqrt(g.Hinv[k] * g.Hinv[k] + g.Hinv[3 + k] * g.Hinv[3 + k] + g.Hinv[6 + k] * g.Hinv[6 + k]);
    }
    // per-direction bounding interval for non-periodic directions (host reduction of a
    // device min/max would cost a sync as well; the list build synchronises anyway)
    // binning coordinate: Cartesian for an orthorhombic cell, fractional for a general one; `ext` is
    // the extent along it, `unit` the perpendicular length of one unit of it
    double lo[3] = {0, 0, 0}, ext[3] = {L[0], L[1], L[2]}, unit[3] = {1, 1, 1};
    if (g.tri) for (int k = 0; k < 3; ++k) { ext[k] = 1.0; unit[k] = height[k]; }
    if (!(pbc[0] && pbc[1] && pbc[2]) && N > 0) {
        // the extent of the atoms along the open directions, reduced on the device (six keys come back)
        if (!nb->bounds) { int64_t c = 0; NB_CHECK(dev_ensure(&nb->bounds, &c, 6)); }
        const unsigned long long init[6] = {~0ull, ~0ull, ~0ull, 0ull, 0ull, 0ull};
        unsigned long long keys[6];
        NB_CHECK(cudaMemcpyAsync(nb->bounds, init, sizeof(init), cudaMemcpyHostToDevice, st));
        int blocks = (N + 255) / 256;
        if (blocks > 1184) blocks = 1184;
        k_bounds<<<blocks, 256, 0, st>>>(N, d_pos, g, nb->bounds);
        NB_CHECK(cudaMemcpyAsync(keys, nb->bounds, sizeof(keys), cudaMemcpyDeviceToHost, st));
        NB_CHECK(cudaStreamSynchronize(st));
        for (int k = 0; k < 3; ++k) {
            if (pbc[k]) continue;
            const double mn = ordered_value(keys[k]), mx = ordered_value(keys[3 + k]);
            if (!std::isfinite(mn) || !std::isfinite(mx)) { *err = "non-finite position"; return UMLMD_E_NONFINITE; }
            lo[k] = mn; ext[k] = (mx - mn) + 1e-6 / unit[k];
        }
    }
    int64_t ncell = 1;
    const double rl_pad = r_list * (1.0 + 1e-9) + 1e-12;
    for (int k = 0; k < 3; ++k) {
        g.L[k] = L[k]; g.lo[k] = lo[k]; g.pbc[k] = pbc[k] ? 1 : 0;
        int nc = (int)std::floor(ext[k] * unit[k] / rl_pad);
        if (nc < 1) nc = 1;
        if (nc > 1024) nc = 1024;
        g.nc[k] = nc;
    }
    // keep the cell table modest relative to the atom count
    while ((int64_t)g.nc[0] * g.nc[1] * g.nc[2] > 8 * (int64_t)N + 64) {
        int kmax = 0;
        for (int k = 1; k < 3; ++k) if (g.nc[k] > g.nc[kmax]) kmax = k;
        if (g.nc[kmax] == 1) break;
        g.nc[kmax] = (g.nc[kmax] + 1) / 2;
    }
    for (int k = 0; k < 3; ++k) {
        const double cw = ext[k] / g.nc[k];
        g.inv_cw[k] = 1.0 / cw;
        g.m[k] = pbc[k] || g.nc[k] > 1 ? (int)std::ceil(r_list / (cw * unit[k])) : 0;
        if (!pbc[k] && g.m[k] > g.nc[k] - 1) g.m[k] = g.nc[k] - 1;
        if (g.m[k] > 127) { *err = "cell much smaller than the list radius (more than 127 images)"; return UMLMD_E_UNSUPPORTED_CELL; }
        ncell *= g.nc[k];
    }
    g.sorted = 1;
    for (int k = 0; k < 3; ++k)
        if (g.pbc[k] && g.nc[k] < 2 * g.m[k] + 1) g.sorted = 0;
    g.ncell = (int)ncell; g.n_owned = n_owned; g.halves = n_owned < N ? 2 : 1;
    const int64_t nkeys = (int64_t)g.halves * ncell;

    nb->N = N; nb->skin = skin; nb->r_list = r_list; nb->n_owned = n_owned; nb->E_owned = 0;
    for (int k = 0; k < 3; ++k) { nb->L[k] = L[k]; nb->pbc[k] = pbc[k] ? 1 : 0; }
    for (int k = 0; k < 9; ++k) nb->H[k] = cell[k];
    nb->tri = g.tri;
    if (N == 0) { nb->E = 0; return UMLMD_OK; }

    // per-atom arrays (all sized from one capacity)
    if (N > nb->N_cap || !nb->wpos) {
        const int64_t need = N + 1;
        int64_t c;
        c = 0; NB_CHECK(dev_ensure(&nb->wpos, &c, need * 3));
        c = 0; NB_CHECK(dev_ensure(&nb->xs0, &c, need * 3));
        c = 0; NB_CHECK(dev_ensure(&nb->xs, &c, need * 3));
        c = 0; NB_CHECK(dev_ensure(&nb->rec, &c, need * 2));
        c = 0; NB_CHECK(dev_ensure(&nb->img, &c, need * 6));   // sorted-order and caller-order halves
        c = 0; NB_CHECK(dev_ensure(&nb->perm, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->type_s, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->row_ptr, &c, need + 1));
        c = 0; NB_CHECK(dev_ensure(&nb->key, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->key2, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->idx, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->idx2, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->deg, &c, need + 1));
        nb->N_cap = N;
    }
    NB_CHECK(dev_ensure(&nb->cell_start, &nb->ncell_cap, nkeys + 2));
    int* img_o = nb->img + 3 * (size_t)(N + 1);

    const int TB = 256;
    k_fold_bin<<<(N + TB - 1) / TB, TB, 0, st>>>(N, d_pos, g, nb->wpos, img_o, nb->key, nb->idx, d_err);
    int end_bit = 1;
    while ((1LL << end_bit) < nkeys) ++end_bit;
    size_t need_tmp = 0, need_scan = 0;
    cub::DeviceRadixSort::SortPairs(nullptr, need_tmp, nb->key, nb->key2, nb->idx, nb->idx2, N, 0, end_bit, st);
    // row offsets are accumulated in 64 bits from the 32-bit row lengths
    auto deg_wide = thrust::make_transform_iterator(static_cast<const int*>(nb->deg), WidenDeg());
    cub::DeviceScan::ExclusiveScan(nullptr, need_scan, deg_wide, nb->row_ptr, cub::Sum(), (eidx_t)0, N + 1, st);
    size_t need_scan32 = 0;                     // the export scans into the caller's 32-bit row pointers
    cub::DeviceScan::ExclusiveSum(nullptr, need_scan32, nb->deg, (int*)nullptr, N + 1, st);
    if (need_scan32 > need_scan) need_scan = need_scan32;
    if (need_scan > need_tmp) need_tmp = need_scan;
    if (need_tmp > nb->cub_bytes) {
        if (nb->cub_tmp) dev_free(nb->cub_tmp);
        nb->cub_tmp = nullptr; nb->cub_bytes = 0;
        NB_CHECK(dev_malloc(&nb->cub_tmp, need_tmp + 256));
        nb->cub_bytes = need_tmp + 256;
    }
    size_t tmp_bytes = nb->cub_bytes;
    NB_CHECK(cub::DeviceRadixSort::SortPairs(nb->cub_tmp, tmp_bytes, nb->key, nb->key2, nb->idx, nb->idx2, N,
                                             0, end_bit, st));
    k_cell_start<<<(int)((nkeys + 1 + TB - 1) / TB), TB, 0, st>>>((int)nkeys, N, nb->key2, nb->cell_start);
    k_gather_sorted<<<(N + TB - 1) / TB, TB, 0, st>>>(N, nb->idx2, nb->wpos, img_o, d_type, nb->perm, nb->xs0,
                                                      nb->xs, nb->img, nb->type_s);
    const double rl2 = r_list * r_list;
    const int warps_per_block = TB / 32;
    const int wb = (N + warps_per_block - 1) / warps_per_block;
    k_scan_cells<false><<<wb, TB, 0, st>>>(N, g, rl2, nb->key2, nb->cell_start, nb->xs0, nb->deg, nullptr,
                                           nullptr, nullptr, d_err);
    NB_CHECK(cudaMemsetAsync(nb->deg + N, 0, sizeof(int), st));
    tmp_bytes = nb->cub_bytes;
    NB_CHECK(cub::DeviceScan::ExclusiveScan(nb->cub_tmp, tmp_bytes, deg_wide, nb->row_ptr, cub::Sum(), (eidx_t)0, N + 1, st));
    eidx_t total = 0, total_owned = 0;
    NB_CHECK(cudaMemcpyAsync(&total, nb->row_ptr + N, sizeof(total), cudaMemcpyDeviceToHost, st));
    if (n_owned < N) NB_CHECK(cudaMemcpyAsync(&total_owned, nb->row_ptr + n_owned, sizeof(total_owned), cudaMemcpyDeviceToHost, st));
    NB_CHECK(cudaStreamSynchronize(st));
    nb->E = total;
    nb->E_owned = n_owned < N ? total_owned : total;
    if (total > nb->E_cap) {
        int64_t c;
        c = 0; NB_CHECK(dev_ensure(&nb->src, &c, total, 1.1));
        c = 0; NB_CHECK(dev_ensure(&nb->shift, &c, total, 1.1));
        c = 0; NB_CHECK(dev_ensure(&nb->rev, &c, total, 1.1));
        nb->E_cap = c;
    }
    if (total > 0) {
        k_scan_cells<true><<<wb, TB, 0, st>>>(N, g, rl2, nb->key2, nb->cell_start, nb->xs0, nullptr,
                                              nb->row_ptr, nb->src, nb->shift, d_err);
        k_reverse_map<<<wb, TB, 0, st>>>(N, g.sorted, nb->row_ptr, nb->src, nb->shift, nb->rev);
    }
    NB_CHECK(cudaGetLastError());
    return UMLMD_OK;
}

int neighbor_export(NeighborDev* nb, int32_t* d_row_ptr, int32_t* d_src, int8_t* d_shift,
                    cudaStream_t st, std::string* err) {
    const int N = (int)nb->N;
    if (N == 0) {
        NB_CHECK(cudaMemsetAsync(d_row_ptr, 0, sizeof(int), st));
        return UMLMD_OK;
    }
    const int TB = 256;
    k_export_deg<<<(N + TB - 1) / TB, TB, 0, st>>>(N, nb->perm, nb->row_ptr, nb->deg);
    size_t tmp_bytes = nb->cub_bytes;
    NB_CHECK(cub::DeviceScan::ExclusiveSum(nb->cub_tmp, tmp_bytes, nb->deg, d_row_ptr, N + 1, st));
    const int wb = (N + TB / 32 - 1) / (TB / 32);
    if (nb->E > 0)
        k_export_rows<<<wb, TB, 0, st>>>(N, nb->perm, nb->row_ptr, nb->src, nb->shift, d_row_ptr, d_src,
                                         (signed char*)d_shift);
    NB_CHECK(cudaGetLastError());
    return UMLMD_OK;
}

int neighbor_build_batch(NeighborDev* nb, int n_frames, const int64_t* offsets, const double* cells, const int pbc[3],
                         const double* d_pos, const int32_t* d_type, int T, double rc, int* d_err, cudaStream_t st,
                         std::string* err) {
    const int64_t N = offsets[n_frames];
    std::vector<FrameCell> fr((size_t)n_frames);
    for (int f = 0; f < n_frames; ++f) {
        FrameCell& c = fr[f];
        const double* H = cells + 9 * (size_t)f;
        for (int k = 0; k < 9; ++k) {
            if (!std::isfinite(H[k])) { *err = "non-finite cell in a frame"; return UMLMD_E_UNSUPPORTED_CELL; }
            c.H[k] = H[k];
        }
        const double cx[3] = {H[4] * H[8] - H[5] * H[7], H[5] * H[6] - H[3] * H[8], H[3] * H[7] - H[4] * H[6]};   // b x c
        const double cy[3] = {H[7] * H[2] - H[8] * H[1], H[8] * H[0] - H[6] * H[2], H[6] * H[1] - H[7] * H[0]};   // c x a
        const double cz[3] = {H[1] * H[5] - H[2] * H[4], H[2] * H[3] - H[0] * H[5], H[0] * H[4] - H[1] * H[3]};   // a x b
        const double det = H[0] * cx[0] + H[1] * cx[1] + H[2] * cx[2];
        double scale = 0;
        for (int k = 0; k < 9; ++k) scale = std::fmax(scale, std::fabs(H[k]));
        if (!(std::fabs(det) > 1e-12 * scale * scale * scale)) { *err = "singular cell in a frame"; return UMLMD_E_UNSUPPORTED_CELL; }
        const double* cr[3] = {cx, cy, cz};
        for (int k = 0; k < 3; ++k) {           // column k of the inverse = (cross product k) / det
            for (int r = 0; r < 3; ++r) c.Hinv[3 * r + k] = cr[k][r] / det;
            const double nrm = std::sqrt(cr[k][0] * cr[k][0] + cr[k][1] * cr[k][1] + cr[k][2] * cr[k][2]);
            const double height = std::fabs(det) / nrm;
            c.pbc[k] = pbc[k] ? 1 : 0;
            c.m[k] = pbc[k] ? (int)std::ceil(rc / height) : 0;
            if (c.m[k] > 127) { *err = "frame cell much smaller than the cutoff (more than 127 images)"; return UMLMD_E_UNSUPPORTED_CELL; }
        }
        c.a0 = (int)offsets[f]; c.a1 = (int)offsets[f + 1];
    }
    nb->N = N; nb->skin = 0; nb->r_list = rc; nb->tri = 1; nb->batch = true; nb->n_frames = n_frames;
    for (int k = 0; k < 3; ++k) { nb->pbc[k] = pbc[k] ? 1 : 0; nb->L[k] = 0; }
    for (int k = 0; k < 9; ++k) nb->H[k] = 0;
    nb->E = 0;
    if (N == 0) return UMLMD_OK;
    if (N > nb->N_cap || !nb->xs) {
        const int64_t need = N + 1;
        int64_t c;
        // the same per-atom arrays as the cell-list build sizes (the two builds may alternate on one handle)
        c = 0; NB_CHECK(dev_ensure(&nb->wpos, &c, need * 3));
        c = 0; NB_CHECK(dev_ensure(&nb->xs0, &c, need * 3));
        c = 0; NB_CHECK(dev_ensure(&nb->xs, &c, need * 3));
        c = 0; NB_CHECK(dev_ensure(&nb->rec, &c, need * 2));
        c = 0; NB_CHECK(dev_ensure(&nb->img, &c, need * 6));
        c = 0; NB_CHECK(dev_ensure(&nb->perm, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->type_s, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->row_ptr, &c, need + 1));
        c = 0; NB_CHECK(dev_ensure(&nb->key, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->key2, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->idx, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->idx2, &c, need));
        c = 0; NB_CHECK(dev_ensure(&nb->deg, &c, need + 1));
        nb->N_cap = N;
    }
    nb->frame_of = nb->key;                    // scratch of the cell-list build, free here
    NB_CHECK(dev_ensure(&nb->frames, &nb->frames_cap, (int64_t)n_frames));
    NB_CHECK(cudaMemcpyAsync(nb->frames, fr.data(), sizeof(FrameCell) * (size_t)n_frames, cudaMemcpyHostToDevice, st));
    NB_CHECK(cudaStreamSynchronize(st));       // `fr` is pageable host memory
    auto deg_wide = thrust::make_transform_iterator(static_cast<const int*>(nb->deg), WidenDeg());
    size_t need_scan = 0;
    cub::DeviceScan::ExclusiveScan(nullptr, need_scan, deg_wide, nb->row_ptr, cub::Sum(), (eidx_t)0, (int)N + 1, st);
    if (need_scan > nb->cub_bytes) {
        if (nb->cub_tmp) dev_free(nb->cub_tmp);
        nb->cub_tmp = nullptr; nb->cub_bytes = 0;
        NB_CHECK(dev_malloc(&nb->cub_tmp, need_scan + 256));
        nb->cub_bytes = need_scan + 256;
    }
    const int TB = 256;
    k_batch_fold<<<n_frames, TB, 0, st>>>(nb->frames, d_pos, d_type, T, nb->xs, nb->rec, nb->type_s, nb->frame_of, nb->perm, d_err);
    const double rl2 = rc * rc;
    const int wb = (int)((N + TB / 32 - 1) / (TB / 32));
    k_batch_scan<false><<<wb, TB, 0, st>>>((int)N, nb->frames, nb->frame_of, rl2, nb->xs, nb->deg, nullptr, nullptr, nullptr);
    NB_CHECK(cudaMemsetAsync(nb->deg + N, 0, sizeof(int), st));
    size_t tmp_bytes = nb->cub_bytes;
    NB_CHECK(cub::DeviceScan::ExclusiveScan(nb->cub_tmp, tmp_bytes, deg_wide, nb->row_ptr, cub::Sum(), (eidx_t)0, (int)N + 1, st));
    eidx_t total = 0;
    NB_CHECK(cudaMemcpyAsync(&total, nb->row_ptr + N, sizeof(total), cudaMemcpyDeviceToHost, st));
    NB_CHECK(cudaStreamSynchronize(st));
    nb->E = total;
    nb->n_owned = N; nb->E_owned = total;
    if (total > nb->E_cap) {
        int64_t c;
        c = 0; NB_CHECK(dev_ensure(&nb->src, &c, total, 1.1));
        c = 0; NB_CHECK(dev_ensure(&nb->shift, &c, total, 1.1));
        c = 0; NB_CHECK(dev_ensure(&nb->rev, &c, total, 1.1));
        nb->E_cap = c;
    }
    if (total > 0) {
        k_batch_scan<true><<<wb, TB, 0, st>>>((int)N, nb->frames, nb->frame_of, rl2, nb->xs, nullptr, nb->row_ptr, nb->src, nb->shift);
        k_reverse_map<<<wb, TB, 0, st>>>((int)N, 0, nb->row_ptr, nb->src, nb->shift, nb->rev);
    }
    NB_CHECK(cudaGetLastError());
    return UMLMD_OK;
}

int neighbor_export_rows(NeighborDev* nb, int64_t first, int64_t n, int64_t* d_row_ptr, int32_t* d_src,
                         int8_t* d_shift, int64_t cap, cudaStream_t st, std::string* err) {
    const int N = (int)nb->N;
    if (n == 0 || N == 0) {
        NB_CHECK(cudaMemsetAsync(d_row_ptr, 0, sizeof(int64_t), st));
        return UMLMD_OK;
    }
    const int TB = 256;
    k_export_deg_range<<<(N + TB - 1) / TB, TB, 0, st>>>(N, (int)first, (int)n, nb->perm, nb->row_ptr, nb->deg);
    auto deg_wide = thrust::make_transform_iterator(static_cast<const int*>(nb->deg), WidenDeg());
    size_t tmp_bytes = nb->cub_bytes;
    NB_CHECK(cub::DeviceScan::ExclusiveScan(nb->cub_tmp, tmp_bytes, deg_wide, reinterpret_cast<eidx_t*>(d_row_ptr), cub::Sum(),
                                            (eidx_t)0, (int)n + 1, st));
    if (cap > 0 && d_src && d_shift) {
        const int wb = (N + TB / 32 - 1) / (TB / 32);
        k_export_rows_range<<<wb, TB, 0, st>>>(N, (int)first, (int)n, nb->perm, nb->row_ptr, nb->src, nb->shift,
                                               reinterpret_cast<const long long*>(d_row_ptr), (long long)cap, d_src,
                                               (signed char*)d_shift);
    }
    NB_CHECK(cudaGetLastError());
    return UMLMD_OK;
}

cudaError_t launch_gather_positions(const NeighborDev& nb, const double* d_pos, int* d_err, cudaStream_t st) {
    const int N = (int)nb.N;
    if (N == 0) return cudaSuccess;
    const double half = 0.5 * nb.skin;
    // a tiny slack keeps a fresh build with zero skin from tripping on its own rounding
    const double max_disp2 = half * half + 1e-20;
    CellRows H;
    for (int k = 0; k < 9; ++k) H.h[k] = nb.H[k];
    H.tri = nb.tri;
    k_gather_positions<<<(N + 255) / 256, 256, 0, st>>>(N, nb.perm, nb.img, d_pos, nb.xs0, H, max_disp2, nb.type_s, nb.xs, nb.rec, d_err);
    return cudaGetLastError();
}

}  // namespace umd
