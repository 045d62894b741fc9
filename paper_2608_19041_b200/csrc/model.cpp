// Blob parsing and create-time precomputation (host, double precision).
//
//  * radial table: value and first derivative of the shared radial map g(rho) and the radial
//    modes q(rho) (sinc-type Bessel basis -> bias-free SwiGLU -> linear heads) at the knots
//    rho_s = s*dx, turned into the two-point cubic Hermite polynomial of each interval.  The
//    paper tabulates the quintic two-point interpolant (value, first and second derivative,
//    six coefficients per channel); every edge reads one table row per pass and the edge
//    kernels are bound by exactly that traffic, so the table keeps four coefficients: at the
//    paper's spacing of 0.002 A the cubic's error, dx^4 |g^(4)| / 384 in the value and about
//    dx^3 |g^(4)| / 72 in the derivative, is below single-precision rounding of the
//    amplitude, and the interpolant stays continuously differentiable, so the force is
//    still the exact derivative of a continuous energy;
//  * ordered type-pair cache: scale gamma, shift beta and mode mixing U of the pair
//    modulation network for all T*T ordered species pairs;
//  * Gaunt couplings of the generic degree triples, by exact quadrature on the sphere,
//    scaled to unit Frobenius norm, sign -1 (the sign both printed closed forms carry).
#include "model.h"

#include <cmath>
#include <cstring>

namespace umd {

namespace {

constexpr size_t kHeaderBytes = 8 + 9 * 4 + 2 * 8;  // packed, no padding

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

inline double sigmoid(double a) { return 1.0 / (1.0 + std::exp(-a)); }

// j0(x) = sin x / x and its first derivative with respect to x
inline void j0_derivs(double x, double* j, double* j1) {
    if (std::fabs(x) < 0.05) {
        const double x2 = x * x;
        *j = 1.0 - x2 / 6.0 + x2 * x2 / 120.0 - x2 * x2 * x2 / 5040.0;
        *j1 = x * (-1.0 / 3.0 + x2 / 30.0 - x2 * x2 / 840.0);
    } else {
        const double s = std::sin(x), c = std::cos(x);
        *j = s / x;
        *j1 = (x * c - s) / (x * x);
    }
}

// real Cartesian harmonics up to degree 4 for a unit vector, s = |u|^2 kept
void harmonics_host(const double u[3], double B1[3], double B2[5], double B3[7], double B4[9]) {
    const double x = u[0], y = u[1], z = u[2], s = x * x + y * y + z * z;
    B1[0] = x; B1[1] = y; B1[2] = z;
    const double r3 = std::sqrt(3.0);
    B2[0] = r3 * x * y; B2[1] = r3 * y * z; B2[2] = 0.5 * (3 * z * z - s); B2[3] = r3 * x * z;
    B2[4] = 0.5 * r3 * (x * x - y * y);
    const double a = std::sqrt(5.0 / 8.0), b = std::sqrt(15.0), c = std::sqrt(3.0 / 8.0);
    B3[0] = a * y * (3 * x * x - y * y);
    B3[1] = b * x * y * z;
    B3[2] = c * y * (5 * z * z - s);
    B3[3] = 0.5 * z * (5 * z * z - 3 * s);
    B3[4] = c * x * (5 * z * z - s);
    B3[5] = 0.5 * b * z * (x * x - y * y);
    B3[6] = a * x * (x * x - 3 * y * y);
    const double r35 = std::sqrt(35.0), r70 = std::sqrt(70.0), r10 = std::sqrt(10.0), r5 = std::sqrt(5.0);
    B4[0] = 0.5 * r35 * x * y * (x * x - y * y);
    B4[1] = 0.25 * r70 * y * z * (3 * x * x - y * y);
    B4[2] = 0.5 * r5 * x * y * (7 * z * z - s);
    B4[3] = 0.25 * r10 * y * z * (7 * z * z - 3 * s);
    B4[4] = 0.125 * (35 * z * z * z * z - 30 * z * z * s + 3 * s * s);
    B4[5] = 0.25 * r10 * x * z * (7 * z * z - 3 * s);
    B4[6] = 0.25 * r5 * (x * x - y * y) * (7 * z * z - s);
    B4[7] = 0.25 * r70 * x * z * (x * x - 3 * y * y);
    B4[8] = 0.125 * r35 * (x * x * x * x - 6 * x * x * y * y + y * y * y * y);
}

// Gauss-Legendre nodes and weights on [-1, 1] by Newton iteration
void gauss_legendre(int n, std::vector<double>* xs, std::vector<double>* ws) {
    xs->resize(n); ws->resize(n);
    for (int i = 0; i < n; ++i) {
        double x = std::cos(M_PI * (i + 0.75) / (n + 0.5));
        double dp = 0;
        for (int it = 0; it < 100; ++it) {
            double p0 = 1.0, p1 = x;
            for (int k = 2; k <= n; ++k) {
                const double p2 = ((2 * k - 1) * x * p1 - (k - 1) * p0) / k;
                p0 = p1; p1 = p2;
            }
            dp = n * (x * p1 - p0) / (x * x - 1.0);
            const double step = p1 / dp;
            x -= step;
            if (std::fabs(step) < 1e-16) break;
        }
        (*xs)[i] = x;
        (*ws)[i] = 2.0 / ((1.0 - x * x) * dp * dp);
    }
}

// non-zeros of the unit-norm coupling of degrees (l1, l2, l3), sign -1: the product of three
// harmonics has degree at most 12, which 16 Gauss-Legendre nodes in cos(theta) times 32 equally
// spaced azimuths integrate exactly
template <typename Sparse, int CAP>
bool gaunt_sparse(int l1, int l2, int l3, Sparse* out) {
    const int n1 = 2 * l1 + 1, n2 = 2 * l2 + 1, n3 = 2 * l3 + 1;
    std::vector<double> I(n1 * n2 * n3, 0.0), xs, ws;
    const int nth = 16, nph = 32;
    gauss_legendre(nth, &xs, &ws);
    for (int a = 0; a < nth; ++a) {
        const double ct = xs[a], st = std::sqrt(1.0 - ct * ct);
        for (int b = 0; b < nph; ++b) {
            const double ph = (b + 0.5) * (2.0 * M_PI / nph);
            const double u[3] = {st * std::cos(ph), st * std::sin(ph), ct};
            const double w = ws[a] * (2.0 * M_PI / nph);
            double B1[3], B2[5], B3[7], B4[9];
            harmonics_host(u, B1, B2, B3, B4);
            const double* Bs[5] = {nullptr, B1, B2, B3, B4};
            for (int i = 0; i < n1; ++i)
                for (int j = 0; j < n2; ++j)
                    for (int k = 0; k < n3; ++k)
                        I[(i * n2 + j) * n3 + k] += w * Bs[l1][i] * Bs[l2][j] * Bs[l3][k];
        }
    }
    double nrm = 0;
    for (double v : I) nrm += v * v;
    nrm = std::sqrt(nrm);
    out->n = 0;
    for (int i = 0; i < n1; ++i)
        for (int j = 0; j < n2; ++j)
            for (int k = 0; k < n3; ++k) {
                const double v = -I[(i * n2 + j) * n3 + k] / nrm;
                if (std::fabs(v) > 1e-12) {
                    if (out->n >= CAP) return false;
                    out->m1[out->n] = (unsigned char)i;
                    out->m2[out->n] = (unsigned char)j;
                    out->m3[out->n] = (unsigned char)k;
                    out->v[out->n] = (float)v;
                    ++out->n;
                }
            }
    return true;
}

}  // namespace

bool derive_dims(int C0, int L, int R, Dims* d) {
    int C1;
    switch (C0) {  // C1 = max(4, 2^ceil(log2(C0)/2))
        case 8: case 16: C1 = 4; break;
        case 32: case 64: C1 = 8; break;
        case 128: C1 = 16; break;
        default: return false;
    }
    if (L < 2 || L > kMaxDeg) return false;
    if (!(R == 0 || R == 2 || R == 4 || R == 8)) return false;
    std::memset(d, 0, sizeof(*d));
    d->C0 = C0; d->L = L; d->R = R;
    d->C[0] = C0; d->C[1] = C1; d->C[2] = C1 / 2 > 4 ? C1 / 2 : 4; d->C[3] = 1; d->C[4] = 1;
    d->K[0] = 0; d->K[1] = d->C[2]; d->K[2] = 2; d->K[3] = 1; d->K[4] = 1;
    int off = 0;
    for (int l = 0; l <= L; ++l) { d->offA[l] = off; off += (2 * l + 1) * d->C[l]; }
    d->S = off;
    d->SP = round_up(d->S + 4, 4);   // sums, then s0, s1 (high parts) and their low parts
    int o = 2 * C0 + 2;
    for (int l = 1; l <= L; ++l) { d->oG[l] = o; o += d->C[l] * (d->C[l] + 1) / 2; }
    const int K1 = d->K[1], K2 = d->K[2];
    // bispectrum blocks in lexicographic order of the degree triples; single probes at degrees 3, 4
    d->oJ112 = o; o += K1 * (K1 + 1) / 2 * K2;
    d->oJ123 = o; if (L >= 3) o += K1 * K2;
    d->oJ134 = o; if (L >= 4) o += K1;
    d->oJ222 = o; o += K2 * (K2 + 1) * (K2 + 2) / 6;
    d->oJ224 = o; if (L >= 4) o += K2 * (K2 + 1) / 2;
    d->oJ233 = o; if (L >= 3) o += K2;
    d->oJ244 = o; if (L >= 4) o += K2;
    d->oJ334 = o; if (L >= 4) o += 1;
    d->oJ444 = o; if (L >= 4) o += 1;
    d->oPi = o; o += K1 * K2;
    d->D_out = o;
    d->DP = round_up(o, 32);
    d->H = 8 * ((C0 + 2) / 3);
    d->Hp = 8 * ((2 * C0 + 2) / 3);
    d->CP = round_up(C0 + R, 4);
    return true;
}

int build_host_model(const void* blob_v, size_t bytes, double dx_override, HostModel* m,
                     std::string* err) {
    const unsigned char* blob = static_cast<const unsigned char*>(blob_v);
    if (bytes < kHeaderBytes) { *err = "blob shorter than its header"; return UMLMD_E_BAD_BLOB; }
    if (std::memcmp(blob, "UMLMD1\0\0", 8) != 0) { *err = "bad magic"; return UMLMD_E_BAD_BLOB; }
    uint32_t u[9];
    std::memcpy(u, blob + 8, sizeof(u));
    double rd[2];
    std::memcpy(rd, blob + 8 + 36, sizeof(rd));
    if (u[0] != 1) { *err = "unsupported blob version"; return UMLMD_E_BAD_BLOB; }
    const int C0 = (int)u[1], L = (int)u[2], R = (int)u[3], N_rbf = (int)u[4], NH = (int)u[5],
              F = (int)u[6], T = (int)u[7];
    if (u[8] > 1) { *err = "radial family must be 0 (Bessel) or 1 (Gaussian)"; return UMLMD_E_UNSUPPORTED_PROFILE; }
    const bool gaussian = u[8] == 1;
    Dims& d = m->d;
    if (!derive_dims(C0, L, R, &d)) {
        *err = "unsupported (C0, L, R): C0 in {8,16,32,64,128}, L in {2,3,4}, R in {0,2,4,8}";
        return UMLMD_E_UNSUPPORTED_PROFILE;
    }
    if (N_rbf < 1 || N_rbf > 64 || NH < 1 || NH > 8 || F < 4 || F % 4 != 0 || F > 4096 || T < 1 ||
        T > 1024) {
        *err = "unsupported N_rbf / hidden layers / width / type count";
        return UMLMD_E_UNSUPPORTED_PROFILE;
    }
    if (gaussian && N_rbf < 2) { *err = "the Gaussian family needs at least two basis functions"; return UMLMD_E_UNSUPPORTED_PROFILE; }
    d.N_rbf = N_rbf; d.n_hidden = NH; d.F = F; d.T = T;
    m->rc = rd[0];
    m->dx = dx_override > 0 ? dx_override : rd[1];
    if (!(m->rc > 0) || !(m->dx > 0) || !std::isfinite(m->rc) || !std::isfinite(m->dx) ||
        m->rc / m->dx > 2.0e6) {
        *err = "bad cutoff or table spacing";
        return UMLMD_E_BAD_BLOB;
    }
    const int H = d.H, Hp = d.Hp, C1 = d.C[1], C2 = d.C[2], K1 = d.K[1], K2 = d.K[2], D = d.D_out;
    // array sizes in blob order
    std::vector<size_t> sizes = {(size_t)T * C0, (size_t)N_rbf, (size_t)N_rbf * 2 * H, (size_t)H * C0,
                                 (size_t)H * R, (size_t)2 * C0 * 2 * Hp, (size_t)Hp * C0 * (2 + R),
                                 (size_t)C1 * C1, (size_t)C2 * C2, (size_t)C1 * K1, (size_t)C2 * K2,
                                 (size_t)D, (size_t)D, (size_t)D * F, (size_t)F};
    for (int t = 2; t <= NH; ++t) { sizes.push_back((size_t)F * F); sizes.push_back((size_t)F); }
    sizes.push_back(F); sizes.push_back(1); sizes.push_back(T);
    size_t total = 0;
    for (size_t s : sizes) total += s;
    if (bytes != kHeaderBytes + 4 * total) {
        *err = "blob size does not match the widths its header implies";
        return UMLMD_E_BAD_BLOB;
    }
    std::vector<std::vector<double>> arr(sizes.size());
    size_t off = kHeaderBytes;
    for (size_t k = 0; k < sizes.size(); ++k) {
        arr[k].resize(sizes[k]);
        for (size_t i = 0; i < sizes[k]; ++i) {
            float f;
            std::memcpy(&f, blob + off, 4);
            off += 4;
            if (!std::isfinite(f)) { *err = "non-finite weight"; return UMLMD_E_BAD_BLOB; }
            arr[k][i] = f;
        }
    }
    const std::vector<double>&X0 = arr[0], &omega = arr[1], &W_in = arr[2], &W_out = arr[3],
          &W_mode = arr[4], &W_p_in = arr[5], &W_p_out = arr[6], &W_1 = arr[7], &W_2 = arr[8],
          &A_1 = arr[9], &A_2 = arr[10], &mu = arr[11], &sigma = arr[12];
    for (double s : sigma)
        if (s == 0.0) { *err = "zero calibration scale"; return UMLMD_E_BAD_BLOB; }

    // ---- radial table --------------------------------------------------------------
    const int n_rows = (int)std::ceil(m->rc / m->dx - 1e-9);
    d.n_rows = n_rows;
    d.rc = (float)m->rc; d.dx = (float)m->dx; d.inv_dx = (float)(1.0 / m->dx);
    const int CP = d.CP, NC = C0 + R;
    std::vector<double> Y((size_t)(n_rows + 1) * 2 * NC);  // [knot][deriv][channel]
    {
        std::vector<double> f(N_rbf), f1(N_rbf), a(2 * H), a1(2 * H), h(H), h1(H);
        for (int s = 0; s <= n_rows; ++s) {
            const double rho = s * m->dx;
            for (int n = 0; n < N_rbf; ++n) {
                if (gaussian) {   // f_n = exp(-(rho - c_n)^2 / (2 s^2)), s = rc / (N_rbf - 1); centres in the omega slot
                    const double sg = m->rc / (N_rbf - 1), t = (rho - omega[n]) / sg;
                    f[n] = std::exp(-0.5 * t * t); f1[n] = -t / sg * f[n];
                    continue;
                }
                double j, j1;
                const double w = omega[n];
                j0_derivs(w * rho, &j, &j1);
                f[n] = w * j; f1[n] = w * w * j1;
            }
            for (int k = 0; k < 2 * H; ++k) {
                double s0 = 0, s1 = 0;
                for (int n = 0; n < N_rbf; ++n) {
                    const double w = W_in[(size_t)n * 2 * H + k];
                    s0 += f[n] * w; s1 += f1[n] * w;
                }
                a[k] = s0; a1[k] = s1;
            }
            for (int k = 0; k < H; ++k) {  // h = SiLU(gate) * value, gate = first H columns
                const double g = a[k], g1 = a1[k], v = a[H + k], v1 = a1[H + k];
                const double sg = sigmoid(g);
                const double S0 = g * sg, S1 = sg * (1 + g * (1 - sg));
                h[k] = S0 * v;
                h1[k] = S1 * g1 * v + S0 * v1;
            }
            double* y = &Y[(size_t)s * 2 * NC];
            for (int c = 0; c < NC; ++c) {
                double s0 = 0, s1 = 0;
                for (int k = 0; k < H; ++k) {
                    const double w = c < C0 ? W_out[(size_t)k * C0 + c] : W_mode[(size_t)k * R + (c - C0)];
                    s0 += h[k] * w; s1 += h1[k] * w;
                }
                y[c] = s0; y[NC + c] = s1;
            }
        }
    }
    m->table.assign((size_t)n_rows * 3 * CP, 0.0f);
    {
        // p(t) = c0 + c1 t + c2 t^2 + c3 t^3, t = rho - rho_s, matching value and slope at both knots;
        // c2 and c3 are stored packed on the table's own scale (common.cuh, tab_pack)
        const double D1 = m->dx, D2 = D1 * D1, D3 = D2 * D1;
        std::vector<float> hi((size_t)n_rows * 2 * NC);
        float m2 = 0.f, m3 = 0.f;
        for (int s = 0; s < n_rows; ++s) {
            const double* ya = &Y[(size_t)s * 2 * NC];
            const double* yb = &Y[(size_t)(s + 1) * 2 * NC];
            float* row = &m->table[(size_t)s * 3 * CP];
            for (int c = 0; c < NC; ++c) {
                const double y0 = ya[c], p0 = ya[NC + c], y1 = yb[c], p1 = yb[NC + c];
                const double del = y1 - y0;
                row[0 * CP + c] = (float)y0;
                row[1 * CP + c] = (float)p0;
                const float c2 = (float)((3 * del - (2 * p0 + p1) * D1) / D2), c3 = (float)((-2 * del + (p0 + p1) * D1) / D3);
                hi[((size_t)s * NC + c) * 2] = c2; hi[((size_t)s * NC + c) * 2 + 1] = c3;
                if (std::fabs(c2) > m2) m2 = std::fabs(c2);
                if (std::fabs(c3) > m3) m3 = std::fabs(c3);
            }
        }
        d.tab_k2 = tab_step2(m2); d.tab_k3 = tab_step3(m3);
        for (int s = 0; s < n_rows; ++s)
            for (int c = 0; c < NC; ++c) {
                const unsigned w = tab_pack(hi[((size_t)s * NC + c) * 2], hi[((size_t)s * NC + c) * 2 + 1], d.tab_k2, d.tab_k3);
                std::memcpy(&m->table[(size_t)s * 3 * CP + 2 * CP + c], &w, sizeof(w));
            }
    }

    // ---- ordered type-pair cache -----------------------------------------------------
    {
        const int NO = C0 * (2 + R);
        // first layer splits over the two halves of z = [X0_a, X0_b]
        std::vector<double> top((size_t)T * 2 * Hp, 0.0), bot((size_t)T * 2 * Hp, 0.0);
        for (int t = 0; t < T; ++t)
            for (int c = 0; c < C0; ++c) {
                const double x = X0[(size_t)t * C0 + c];
                const double* wt = &W_p_in[(size_t)c * 2 * Hp];
                const double* wb = &W_p_in[(size_t)(C0 + c) * 2 * Hp];
                for (int k = 0; k < 2 * Hp; ++k) {
                    top[(size_t)t * 2 * Hp + k] += x * wt[k];
                    bot[(size_t)t * 2 * Hp + k] += x * wb[k];
                }
            }
        m->pairmod.assign((size_t)T * T * (2 + R) * C0, 0.0f);
        std::vector<double> hid(Hp), o(NO);
        for (int a = 0; a < T; ++a)
            for (int b = 0; b < T; ++b) {
                for (int k = 0; k < Hp; ++k) {
                    const double g = top[(size_t)a * 2 * Hp + k] + bot[(size_t)b * 2 * Hp + k];
                    const double v = top[(size_t)a * 2 * Hp + Hp + k] + bot[(size_t)b * 2 * Hp + Hp + k];
                    hid[k] = g * sigmoid(g) * v;
                }
                std::fill(o.begin(), o.end(), 0.0);
                for (int k = 0; k < Hp; ++k) {
                    const double hk = hid[k];
                    const double* w = &W_p_out[(size_t)k * NO];
                    for (int j = 0; j < NO; ++j) o[j] += hk * w[j];
                }
                float* pm = &m->pairmod[(size_t)(a * T + b) * (2 + R) * C0];
                for (int c = 0; c < C0; ++c) {
                    pm[c] = (float)(1.0 + std::tanh(0.1 * o[c]));
                    pm[C0 + c] = (float)(X0[(size_t)a * C0 + c] + X0[(size_t)b * C0 + c] +
                                         std::tanh(0.1 * o[C0 + c]));
                    for (int q = 0; q < R; ++q)  // U[c][q] = tanh(w[c*R + q])
                        pm[(size_t)(2 + q) * C0 + c] = (float)std::tanh(0.1 * o[2 * C0 + c * R + q]);
                }
            }
    }

    // ---- small matrices --------------------------------------------------------------
    auto to_f = [](const std::vector<double>& v) { return std::vector<float>(v.begin(), v.end()); };
    m->X0 = to_f(X0);
    m->W1p.resize(C1 * C1);
    for (int i = 0; i < C1; ++i)
        for (int j = 0; j < C1; ++j) m->W1p[i * C1 + j] = (float)(W_1[i * C1 + j] + (i == j ? 1.0 : 0.0));
    m->W2p.resize(C2 * C2);
    for (int i = 0; i < C2; ++i)
        for (int j = 0; j < C2; ++j) m->W2p[i * C2 + j] = (float)(W_2[i * C2 + j] + (i == j ? 1.0 : 0.0));
    m->A1 = to_f(A_1);
    m->A2 = to_f(A_2);
    m->mu = to_f(mu);
    m->inv_sigma.resize(D);
    for (int k = 0; k < D; ++k) m->inv_sigma[k] = (float)(1.0 / sigma[k]);

    // ---- MLP ---------------------------------------------------------------------------
    m->theta.resize(NH); m->thetaT.resize(NH); m->bias.resize(NH);
    for (int t = 0; t < NH; ++t) {
        const std::vector<double>& Th = arr[13 + 2 * t];
        const std::vector<double>& b = arr[14 + 2 * t];
        const int Kin = t == 0 ? D : F, Kp = t == 0 ? d.DP : F;
        m->theta[t].assign((size_t)Kp * F, 0.0f);
        m->thetaT[t].assign((size_t)F * Kp, 0.0f);
        for (int k = 0; k < Kin; ++k)
            for (int f = 0; f < F; ++f) {
                const float v = (float)Th[(size_t)k * F + f];
                m->theta[t][(size_t)k * F + f] = v;
                m->thetaT[t][(size_t)f * Kp + k] = v;
            }
        m->bias[t] = to_f(b);
    }
    // The first C0 entries of the feature vector are the centre's initial features, a constant per
    // species; their image under the first layer is folded into a per-species bias so that the
    // tensor-core GEMM can skip those K columns.
    {
        const std::vector<double>& Th = arr[13];
        const std::vector<double>& b = arr[14];
        m->type_bias.assign((size_t)T * F, 0.0f);
        for (int t = 0; t < T; ++t)
            for (int f = 0; f < F; ++f) {
                double s = b[f];
                for (int c = 0; c < C0; ++c) {
                    const double x = ((double)m->X0[(size_t)t * C0 + c] - (double)m->mu[c]) * (double)m->inv_sigma[c];
                    s += x * (double)(float)Th[(size_t)c * F + f];
                }
                m->type_bias[(size_t)t * F + f] = (float)s;
            }
    }
    // Half-precision splits for the tensor-core GEMM: x = hi + lo, hi = half(x), lo = half(x - hi).
    // The low part of a small number would be subnormal in half precision, so each layer's weights
    // are split after multiplication by the power of two that brings the layer's largest magnitude
    // into [2^9, 2^10) (the GEMM epilogue multiplies the accumulator by the inverse).
    auto pow2_scale = [](double max_abs, int target_exp) {
        if (!(max_abs > 0)) return 1.0f;
        int e;
        std::frexp(max_abs, &e);                 // max_abs = f * 2^e, f in [0.5, 1)
        return (float)std::ldexp(1.0, target_exp - e);
    };
    auto split = [&](const std::vector<float>& w, float sc, std::vector<__half>* hi, std::vector<__half>* lo) {
        hi->resize(w.size()); lo->resize(w.size());
        for (size_t i = 0; i < w.size(); ++i) {
            const float x = w[i] * sc;
            (*hi)[i] = __float2half_rn(x);
            (*lo)[i] = __float2half_rn(x - __half2float((*hi)[i]));
        }
    };
    m->theta_hi.resize(NH); m->theta_lo.resize(NH); m->thetaT_hi.resize(NH); m->thetaT_lo.resize(NH);
    m->w_scale.resize(NH);
    for (int t = 0; t < NH; ++t) {
        double mx = 0;
        for (float v : m->theta[t]) mx = std::fmax(mx, std::fabs((double)v));
        m->w_scale[t] = pow2_scale(mx, 10);
        split(m->theta[t], m->w_scale[t], &m->theta_hi[t], &m->theta_lo[t]);
        split(m->thetaT[t], m->w_scale[t], &m->thetaT_hi[t], &m->thetaT_lo[t]);
    }
    const size_t tail = 13 + 2 * NH;
    m->w_head = to_f(arr[tail]);
    m->b_head = (float)arr[tail + 1][0];
    m->e_ref = to_f(arr[tail + 2]);
    {
        // the backward pass starts from w_head * SiLU' and stays on that scale: carry it times the
        // power of two that brings max |w_head| into [2^5, 2^6)
        double mx = 0;
        for (float v : m->w_head) mx = std::fmax(mx, std::fabs((double)v));
        m->grad_scale = pow2_scale(mx, 6);
    }

    // ---- Gaunt couplings of the generic triples ------------------------------------
    m->g123.n = 0; m->g233.n = 0;
    if (L >= 3) {
        if (!gaunt_sparse<GauntSparse, kMaxGaunt>(1, 2, 3, &m->g123) || !gaunt_sparse<GauntSparse, kMaxGaunt>(2, 3, 3, &m->g233)) {
            *err = "coupling tensor has more non-zeros than reserved";
            return UMLMD_E_UNSUPPORTED_PROFILE;
        }
    }
    m->g4.clear();
    if (L >= 4) {
        const int tr[5][3] = {{1, 3, 4}, {2, 2, 4}, {2, 4, 4}, {3, 3, 4}, {4, 4, 4}};
        m->g4.resize(5);
        for (int k = 0; k < 5; ++k)
            if (!gaunt_sparse<GauntSparseBig, kMaxGauntBig>(tr[k][0], tr[k][1], tr[k][2], &m->g4[k])) {
                *err = "coupling tensor has more non-zeros than reserved";
                return UMLMD_E_UNSUPPORTED_PROFILE;
            }
    }
    return UMLMD_OK;
}

}  // namespace umd
