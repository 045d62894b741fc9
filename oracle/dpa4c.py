"""CPU fp64 oracle for the DPA4C energy / force / virial evaluation.

TEST INFRASTRUCTURE ONLY.  This module is the plain definition of the model, written
step by step in the paper's notation with float64 PyTorch CPU ops, and a brute-force
O(N^2) neighbor search with explicit periodic images.  It shares no code with the CUDA
library and must never be imported by it.  Only the tests, the smoke check and the
benchmark's CPU-baseline leg may call it.

Forces and the virial come from reverse-mode differentiation of the energy with respect
to the edge displacement vectors (Eq. "forces"): F = -dE/dr is the definition itself, so
no hand-derived backward formula appears here.  The tests pin the result to central
finite differences, the strain derivative and the symmetry statements.

Where the paper leaves a convention open, the reading taken is marked "READING" below.
Parity-unpinned conventions (they change the feature ordering or a block's sign, which
the first MLP layer absorbs; no statement of the paper fixes them): vech order, order
of retained bispectrum entries, sign of the Gaunt coupling for triples other than
(1,1,2) and (2,2,2), reshape order of U, the random-weight initialisation law.
"""

import math
import struct

import numpy as np
import torch

F64 = torch.float64

EPS_REG = 1.0e-7  # Angstrom, Eq. "edge-geometry"

MAGIC = b"UMLMD1\0\0"
_HEADER_FMT = "<8s9I2d"


# --------------------------------------------------------------------------------------
# widths (Eqs. "degree-channels", "moment-width", "probe-ranks", "bispectrum-count",
# "dim-out")
# --------------------------------------------------------------------------------------

def degree_channels(C0, L):
    C1 = max(4, 2 ** math.ceil(0.5 * math.log2(C0)))
    C2 = max(4, C1 // 2)
    return [C0, C1, C2] + [1] * (L - 2)


def probe_ranks(C0, L):
    C = degree_channels(C0, L)
    return [0, C[2], 2] + [1] * (L - 2)  # index by degree; degree 0 has no probe


def triples(L):
    """Admissible degree triples, Eq. "triples", lexicographic."""
    out = []
    for l1 in range(1, L + 1):
        for l2 in range(l1, L + 1):
            for l3 in range(l2, L + 1):
                if l3 <= l1 + l2 and (l1 + l2 + l3) % 2 == 0:
                    out.append((l1, l2, l3))
    return out


def retained_entries(tr, K):
    """Index tuples kept for one triple and their sqrt(family size) weights.

    Axes of equal degree are interchangeable; of each family of equal entries the
    non-decreasing representative is kept.  READING: row-major, first index slowest."""
    l1, l2, l3 = tr
    out = []
    for k1 in range(K[l1]):
        for k2 in range(K[l2]):
            for k3 in range(K[l3]):
                if l1 == l2 and k1 > k2:
                    continue
                if l2 == l3 and k2 > k3:
                    continue
                if l1 == l2 == l3:
                    fam = len({(a, b, c) for (a, b, c) in _perms((k1, k2, k3))})
                elif l1 == l2:
                    fam = 1 if k1 == k2 else 2
                elif l2 == l3:
                    fam = 1 if k2 == k3 else 2
                else:
                    fam = 1
                out.append(((k1, k2, k3), math.sqrt(fam)))
    return out


def _perms(t):
    a, b, c = t
    return [(a, b, c), (a, c, b), (b, a, c), (b, c, a), (c, a, b), (c, b, a)]


def widths(C0, L, R=0):
    C = degree_channels(C0, L)
    K = probe_ranks(C0, L)
    S = sum((2 * l + 1) * C[l] for l in range(L + 1))
    D_bis = sum(len(retained_entries(t, K)) for t in triples(L))
    D_out = 2 * C0 + 2 + sum(C[l] * (C[l] + 1) // 2 for l in range(1, L + 1)) + D_bis + K[1] * K[2]
    return dict(C=C, K=K, S=S, D_out=D_out, H=8 * math.ceil(C0 / 3), Hp=8 * math.ceil(2 * C0 / 3),
                C1=C[1], C2=C[2], K1=K[1], K2=K[2], D_bis=D_bis)


def parameter_count(C0, L, R, N_rbf, n_hidden, F, T_rows):
    """Trainable parameters of the feature path, MLP and type table.  ``T_rows`` is the
    number of rows of the type table (the paper's count has one zero-padding row beside
    its 118 elements).  A_1 is not a parameter when K_1 = C_1 (identity)."""
    w = widths(C0, L, R)
    n = T_rows * C0 + N_rbf + N_rbf * 2 * w["H"] + w["H"] * C0 + w["H"] * R
    n += 2 * C0 * 2 * w["Hp"] + w["Hp"] * C0 * (2 + R)
    n += w["C1"] ** 2 + w["C2"] ** 2
    if w["K1"] != w["C1"]:
        n += w["C1"] * w["K1"]
    n += w["C2"] * w["K2"]
    n += w["D_out"] * F + F + (n_hidden - 1) * (F * F + F) + F + 1
    return n


# --------------------------------------------------------------------------------------
# blob
# --------------------------------------------------------------------------------------

def parse_blob(blob):
    """Weight blob -> (profile dict, dict of float64 tensors)."""
    hb = struct.calcsize(_HEADER_FMT)
    magic, version, C0, L, R, N_rbf, n_hidden, F, T, basis, rc, table_dx = struct.unpack(
        _HEADER_FMT, blob[:hb])
    if magic != MAGIC or version != 1 or basis not in (0, 1):
        raise ValueError("bad blob header")
    w = widths(C0, L, R)
    p = dict(C0=C0, L=L, R=R, N_rbf=N_rbf, n_hidden=n_hidden, F=F, T=T, rc=rc, table_dx=table_dx,
             basis=("bessel", "gaussian")[basis], **w)
    H, Hp, C1, C2, K1, K2, D = w["H"], w["Hp"], w["C1"], w["C2"], w["K1"], w["K2"], w["D_out"]
    shapes = [("X0", (T, C0)), ("omega", (N_rbf,)), ("W_in", (N_rbf, 2 * H)), ("W_out", (H, C0)),
              ("W_mode", (H, R)), ("W_p_in", (2 * C0, 2 * Hp)), ("W_p_out", (Hp, C0 * (2 + R))),
              ("W_1", (C1, C1)), ("W_2", (C2, C2)), ("A_1", (C1, K1)), ("A_2", (C2, K2)),
              ("mu", (D,)), ("sigma", (D,)), ("Theta_1", (D, F)), ("b_1", (F,))]
    for tau in range(2, n_hidden + 1):
        shapes += [(f"Theta_{tau}", (F, F)), (f"b_{tau}", (F,))]
    shapes += [("w_head", (F,)), ("b_head", (1,)), ("E_ref", (T,))]
    off = hb
    params = {}
    for name, shape in shapes:
        n = int(np.prod(shape))
        a = np.frombuffer(blob, dtype="<f4", count=n, offset=off).astype(np.float64).reshape(shape)
        params[name] = torch.from_numpy(a.copy())
        off += 4 * n
    if off != len(blob):
        raise ValueError(f"blob size {len(blob)} != expected {off}")
    return p, params


# --------------------------------------------------------------------------------------
# neighbor search (Eq. "neighbor-set"): brute force over all pairs and periodic images
# --------------------------------------------------------------------------------------

def wrap_positions(pos, cell, pbc):
    """Positions folded into the cell along periodic directions.

    READING (paper silent): frac - floor(frac).  For an orthorhombic cell the fractional
    coordinate is the plain quotient x / L (one IEEE division), so that an independent
    implementation can reproduce the result bit for bit."""
    pos = np.asarray(pos, dtype=np.float64)
    cell = np.asarray(cell, dtype=np.float64)
    off_diag = cell - np.diag(np.diag(cell))
    if not off_diag.any():
        Ld = np.diag(cell)
        frac = pos / Ld
        fl = np.floor(frac)
        wrapped = np.where(np.asarray(pbc, bool)[None, :], (frac - fl) * Ld, pos)
        return wrapped
    inv = np.linalg.inv(cell)
    frac = pos @ inv
    fl = np.floor(frac) * np.asarray(pbc, np.float64)[None, :]
    return (frac - fl) @ cell


def image_range(cell, pbc, r_list):
    """Per-direction image count ceil(r_list / h_k), h_k the cell height."""
    cell = np.asarray(cell, dtype=np.float64)
    vol = abs(np.linalg.det(cell))
    out = []
    for k in range(3):
        a, b = cell[(k + 1) % 3], cell[(k + 2) % 3]
        h = vol / np.linalg.norm(np.cross(a, b))
        out.append(int(math.ceil(r_list / h)) if pbc[k] else 0)
    return out


def neighbor_rows(pos, cell, pbc, r_list, centers=None, chunk=256):
    """Neighbor instances (j, n) of the given centers, by brute force.

    ``pos`` must already be wrapped.  Edge (i <- j, n) exists iff (j, n) != (i, 0) and
    |(r_j + n.cell) - r_i|^2 < r_list^2 with the true (un-regularised) distance, strict
    inequality; distinct images are distinct instances, self-images included.

    READING (paper silent, makes the set reproducible bit for bit): float64, in this
    operation order and with no fused multiply-add: d = (r_j + s) - r_i with s = n.cell
    (for an orthorhombic cell the exact product n_k * L_k), d2 = (dx*dx + dy*dy) + dz*dz,
    test d2 < r_list*r_list.

    Returns a list over centers of int64 arrays [deg, 4] = (j, nx, ny, nz), sorted by
    (j, nx, ny, nz)."""
    pos = np.asarray(pos, dtype=np.float64)
    cell = np.asarray(cell, dtype=np.float64)
    N = len(pos)
    if centers is None:
        centers = np.arange(N)
    centers = np.asarray(centers, dtype=np.int64)
    mx, my, mz = image_range(cell, pbc, r_list)
    imgs = np.array([(a, b, c) for a in range(-mx, mx + 1) for b in range(-my, my + 1)
                     for c in range(-mz, mz + 1)], dtype=np.int64)
    diag = not (cell - np.diag(np.diag(cell))).any()
    if diag:
        shifts = imgs.astype(np.float64) * np.diag(cell)[None, :]
    else:
        shifts = imgs.astype(np.float64) @ cell
    rl2 = r_list * r_list
    rows = [None] * len(centers)
    zero_img = int(np.nonzero((imgs == 0).all(axis=1))[0][0])
    chunk = max(1, min(chunk, (1 << 23) // max(N, 1)))
    for c0 in range(0, len(centers), chunk):
        cs = centers[c0:c0 + chunk]
        pi = pos[cs]                                            # [c,3]
        acc_i, acc_j, acc_n = [], [], []
        for s_idx in range(len(imgs)):
            pj = pos + shifts[s_idx][None, :]                   # (r_j + s)
            d = pj[None, :, :] - pi[:, None, :]                 # - r_i
            d2 = (d[..., 0] * d[..., 0] + d[..., 1] * d[..., 1]) + d[..., 2] * d[..., 2]
            ok = d2 < rl2
            if s_idx == zero_img:
                ok[np.arange(len(cs)), cs] = False
            ii, jj = np.nonzero(ok)
            acc_i.append(ii)
            acc_j.append(jj)
            acc_n.append(np.full(len(ii), s_idx, dtype=np.int64))
        ii = np.concatenate(acc_i)
        jj = np.concatenate(acc_j)
        nn = np.concatenate(acc_n)
        for k in range(len(cs)):
            sel = ii == k
            ent = np.concatenate([jj[sel][:, None], imgs[nn[sel]]], axis=1)
            order = np.lexsort((ent[:, 3], ent[:, 2], ent[:, 1], ent[:, 0]))
            rows[c0 + k] = ent[order]
    return rows


def rows_to_edges(rows, centers, pos, cell):
    """Flatten rows to (dst_local, src, displacement) with r_ij = (r_j + n.cell) - r_i."""
    cell = np.asarray(cell, dtype=np.float64)
    dst = np.concatenate([np.full(len(r), k, dtype=np.int64) for k, r in enumerate(rows)]) \
        if rows else np.zeros(0, np.int64)
    ent = np.concatenate(rows, axis=0) if rows else np.zeros((0, 4), np.int64)
    src = ent[:, 0]
    shift = ent[:, 1:4].astype(np.float64) @ cell
    rij = (pos[src] + shift) - pos[np.asarray(centers)[dst]]
    return dst, src, rij


# --------------------------------------------------------------------------------------
# per-edge functions
# --------------------------------------------------------------------------------------

def envelope(rho, rc):
    """Eq. "envelope": chi = t^4 (1 + 4x + 10x^2 + 20x^3 + 35x^4), t = clip(1 - rho/rc)."""
    t = torch.clamp(1.0 - rho / rc, 0.0, 1.0)
    x = 1.0 - t
    return t ** 4 * (1.0 + 4.0 * x + 10.0 * x ** 2 + 20.0 * x ** 3 + 35.0 * x ** 4)


def bessel_basis(rho, omega):
    """Eq. "bessel-basis": f_n = sin(omega_n rho)/rho, no cutoff factor; tends to omega_n
    as rho -> 0."""
    x = omega[None, :] * rho[:, None]
    return omega[None, :] * torch.special.sinc(x / math.pi)


def harmonics(u, L):
    """Real Cartesian harmonics B_0..B_L of Eq. "harmonics" and the supplementary note on
    degrees three and four, with s = |u|^2 kept.  Returns a list of [E, 2l+1] tensors."""
    ux, uy, uz = u[:, 0], u[:, 1], u[:, 2]
    s = ux * ux + uy * uy + uz * uz
    r3, r5, r15 = math.sqrt(3.0), math.sqrt(5.0), math.sqrt(15.0)
    out = [torch.ones_like(ux)[:, None], torch.stack([ux, uy, uz], dim=1)]
    if L >= 2:
        out.append(torch.stack([r3 * ux * uy, r3 * uy * uz, 0.5 * (3 * uz * uz - s), r3 * ux * uz,
                                0.5 * r3 * (ux * ux - uy * uy)], dim=1))
    if L >= 3:
        out.append(torch.stack([
            math.sqrt(5 / 8) * uy * (3 * ux * ux - uy * uy),
            r15 * ux * uy * uz,
            math.sqrt(3 / 8) * uy * (5 * uz * uz - s),
            0.5 * uz * (5 * uz * uz - 3 * s),
            math.sqrt(3 / 8) * ux * (5 * uz * uz - s),
            0.5 * r15 * uz * (ux * ux - uy * uy),
            math.sqrt(5 / 8) * ux * (ux * ux - 3 * uy * uy)], dim=1))
    if L >= 4:
        r35, r70, r10 = math.sqrt(35.0), math.sqrt(70.0), math.sqrt(10.0)
        out.append(torch.stack([
            0.5 * r35 * ux * uy * (ux * ux - uy * uy),
            0.25 * r70 * uy * uz * (3 * ux * ux - uy * uy),
            0.5 * r5 * ux * uy * (7 * uz * uz - s),
            0.25 * r10 * uy * uz * (7 * uz * uz - 3 * s),
            0.125 * (35 * uz ** 4 - 30 * uz * uz * s + 3 * s * s),
            0.25 * r10 * ux * uz * (7 * uz * uz - 3 * s),
            0.25 * r5 * (ux * ux - uy * uy) * (7 * uz * uz - s),
            0.25 * r70 * ux * uz * (ux * ux - 3 * uy * uy),
            0.125 * r35 * (ux ** 4 - 6 * ux * ux * uy * uy + uy ** 4)], dim=1))
    return out


def stf(z):
    """The linear map R^5 -> symmetric trace-free 3x3 fixed by Eq. "stf",
    STF[B_2(u)] = sqrt(3/2) (u u^T - |u|^2/3 I), written out for the component order of
    Eq. "harmonics".  z: [..., 5] -> [..., 3, 3]."""
    z1, z2, z3, z4, z5 = z.unbind(-1)
    a, b = 1.0 / math.sqrt(2.0), 1.0 / math.sqrt(6.0)
    qxx = -b * z3 + a * z5
    qyy = -b * z3 - a * z5
    qzz = 2.0 * b * z3
    qxy, qyz, qxz = a * z1, a * z2, a * z4
    return torch.stack([torch.stack([qxx, qxy, qxz], -1), torch.stack([qxy, qyy, qyz], -1),
                        torch.stack([qxz, qyz, qzz], -1)], -2)


_GAUNT_CACHE = {}


def gaunt_coupling(tr):
    """Eq. "gaunt": I = integral over the unit sphere of B_l1 B_l2 B_l3, scaled to unit
    Frobenius norm.  Gauss-Legendre in cos(theta) times a uniform grid in phi integrates
    these polynomials (degree <= 12) exactly.

    READING: the overall sign is -1 for every triple; that is the sign both printed
    closed forms of Eq. "closed-forms" carry (checked in the tests)."""
    if tr in _GAUNT_CACHE:
        return _GAUNT_CACHE[tr]
    nth, nph = 16, 32
    xs, ws = np.polynomial.legendre.leggauss(nth)
    ph = (np.arange(nph) + 0.5) * (2 * math.pi / nph)
    ct, phg = np.meshgrid(xs, ph, indexing="ij")
    st = np.sqrt(1 - ct * ct)
    u = torch.from_numpy(np.stack([st * np.cos(phg), st * np.sin(phg), ct], axis=-1).reshape(-1, 3))
    w = torch.from_numpy((ws[:, None] * np.full((1, nph), 2 * math.pi / nph)).reshape(-1))
    B = harmonics(u, max(tr))
    I = torch.einsum("p,pa,pb,pc->abc", w, B[tr[0]], B[tr[1]], B[tr[2]])
    Cc = -I / torch.linalg.norm(I)
    _GAUNT_CACHE[tr] = Cc
    return Cc


def silu(x):
    return x * torch.sigmoid(x)


def gaussian_basis(rho, centers, rc):
    """The Gaussian family of the radial-basis paragraph: f_n = exp(-(rho - c_n)^2 / (2 sigma_g^2))
    with the fixed width sigma_g = rc / (N_rbf - 1); like the Bessel family, no cutoff factor.
    The centres c_n take the blob slot of the Bessel frequencies."""
    sg = rc / (centers.shape[0] - 1)
    d = rho[:, None] - centers[None, :]
    return torch.exp(-d * d / (2.0 * sg * sg))


def swiglu(x, W):
    """Eq. "swiglu": [x_g, x_v] = x W, SiLU(x_g) * x_v; gate = first H columns."""
    a = x @ W
    H = W.shape[1] // 2
    return silu(a[..., :H]) * a[..., H:]


def radial_map(rho, prm, basis="bessel", rc=None):
    """Eqs. "radial-map", "radial-modes": g(rho) in R^C0 and q(rho) in R^R."""
    f = bessel_basis(rho, prm["omega"]) if basis == "bessel" else gaussian_basis(rho, prm["omega"], rc)
    h = swiglu(f, prm["W_in"])
    return h @ prm["W_out"], h @ prm["W_mode"]


def pair_modulation(p, prm):
    """Eq. "pairfilm" for every ordered pair (a = centre, b = neighbour):
    gamma [T,T,C0], beta [T,T,C0], U [T,T,C0,R].
    READING: reshape is row-major over (c, mu): U[c, mu] = tanh(w[c*R + mu])."""
    T, C0, R = p["T"], p["C0"], p["R"]
    X0 = prm["X0"]
    z = torch.cat([X0[:, None, :].expand(T, T, C0), X0[None, :, :].expand(T, T, C0)], dim=-1)
    o = 0.1 * (swiglu(z, prm["W_p_in"]) @ prm["W_p_out"])
    s, t, w = o[..., :C0], o[..., C0:2 * C0], o[..., 2 * C0:]
    gamma = 1.0 + torch.tanh(s)
    beta = X0[:, None, :] + X0[None, :, :] + torch.tanh(t)
    U = torch.tanh(w).reshape(T, T, C0, R)
    return gamma, beta, U


# --------------------------------------------------------------------------------------
# model
# --------------------------------------------------------------------------------------

def vech_indices(C):
    """READING: row-major upper triangle (0,0),(0,1),...,(0,C-1),(1,1),..."""
    return [(a, b) for a in range(C) for b in range(a, C)]


def aggregate(p, prm, pair, n_centers, dst, type_i, type_j, rij):
    """Eqs. "edge-geometry" .. "moments": per-centre sums A_l [n, 2l+1, C_l], s0, s1."""
    gamma, beta, U = pair
    L, rc = p["L"], p["rc"]
    C = p["C"]
    rho = torch.sqrt((rij * rij).sum(dim=1) + EPS_REG ** 2)
    u = rij / rho[:, None]
    chi = envelope(rho, rc)
    g, q = radial_map(rho, prm, p.get("basis", "bessel"), rc)
    psi = gamma[type_i, type_j] * g + beta[type_i, type_j]              # Eq. "amplitude"
    if p["R"] > 0:
        psi = psi + torch.einsum("ecm,em->ec", U[type_i, type_j], q)
    B = harmonics(u, L)
    A = []
    for l in range(L + 1):
        chi_l = chi if l == 0 else chi * chi                            # Eq. "degree-weight"
        msg = chi_l[:, None, None] * B[l][:, :, None] * psi[:, None, :C[l]]
        A.append(torch.zeros(n_centers, 2 * l + 1, C[l], dtype=F64).index_add(0, dst, msg))
    s0 = torch.zeros(n_centers, dtype=F64).index_add(0, dst, chi ** 2)
    s1 = torch.zeros(n_centers, dtype=F64).index_add(0, dst, chi ** 4)
    return A, s0, s1


def descriptor(p, prm, A, s0, s1, type_i):
    """Eqs. "masses", "moments", "alignment" .. "descriptor": raw D~ [n, D_out]."""
    L, C, K = p["L"], p["C"], p["K"]
    M0 = torch.sqrt(0.25 + s0)
    M1 = torch.sqrt(0.25 + s1)
    X = [A[0] / M0[:, None, None]] + [A[l] / M1[:, None, None] for l in range(1, L + 1)]
    Xt = [None] * (L + 1)
    for l in range(1, L + 1):
        if l <= 2:
            Xt[l] = X[l] @ (torch.eye(C[l], dtype=F64) + prm[f"W_{l}"])            # Eq. "alignment"
        else:
            Xt[l] = X[l]
    blocks = [prm["X0"][type_i], X[0][:, 0, :], M0[:, None], M1[:, None]]
    for l in range(1, L + 1):                                           # Eq. "gram"
        G = torch.einsum("nmc,nmd->ncd", Xt[l], Xt[l])
        ent = [G[:, a, b] * (1.0 if a == b else math.sqrt(2.0)) for (a, b) in vech_indices(C[l])]
        blocks.append(torch.stack(ent, dim=1))
    Z = [None] * (L + 1)
    for l in range(1, L + 1):                                           # Eq. "probes"
        Z[l] = Xt[l] @ prm[f"A_{l}"] if l <= 2 else Xt[l]
    for tr in triples(L):                                               # Eq. "bispectrum"
        Cc = gaunt_coupling(tr)
        J = torch.einsum("abc,nai,nbj,nck->nijk", Cc, Z[tr[0]], Z[tr[1]], Z[tr[2]])
        ent = [J[:, i, j, k] * w for ((i, j, k), w) in retained_entries(tr, K)]
        blocks.append(torch.stack(ent, dim=1))
    v = Z[1]                                                            # [n,3,K1]
    Q = stf(Z[2].transpose(1, 2))                                       # [n,K2,3,3]
    Qv = torch.einsum("nhab,nbk->nhka", Q, v)                           # [n,K2,K1,3]
    Pi = (Qv * Qv).sum(dim=-1)                                          # Eq. "quartic", eta-major
    blocks.append(Pi.reshape(len(s0), -1))
    return torch.cat(blocks, dim=1)


def mlp_energy(p, prm, D, type_i):
    """Eqs. "fitting", "atomic-energy": residual SiLU MLP and reference energy."""
    h = silu(D @ prm["Theta_1"] + prm["b_1"])
    if p["D_out"] == p["F"]:
        h = h + D
    for tau in range(2, p["n_hidden"] + 1):
        h = silu(h @ prm[f"Theta_{tau}"] + prm[f"b_{tau}"]) + h
    return h @ prm["w_head"] + prm["b_head"][0] + prm["E_ref"][type_i]


def atomic_energies(p, prm, pair, n_centers, dst, type_i_edge, type_j_edge, rij, type_i_center,
                    return_descriptor=False):
    A, s0, s1 = aggregate(p, prm, pair, n_centers, dst, type_i_edge, type_j_edge, rij)
    Dt = descriptor(p, prm, A, s0, s1, type_i_center)
    D = (Dt - prm["mu"]) / prm["sigma"]                                 # Eq. "calibration"
    E = mlp_energy(p, prm, D, type_i_center)
    if return_descriptor:
        return E, Dt, A, s0, s1
    return E


class Oracle:
    """Holds a parsed blob and evaluates energies, forces and the virial."""

    def __init__(self, blob):
        self.p, self.prm = parse_blob(blob)
        with torch.no_grad():
            self.pair = pair_modulation(self.p, self.prm)

    def evaluate_rows(self, pos, types, cell, rows, centers, want_grad=True, edge_chunk=60000):
        """E_i for the given centers and, when ``want_grad``, the per-edge gradients
        g_ij = dE/dr_ij of those centers' edges.  ``pos`` wrapped, ``rows`` from
        ``neighbor_rows``.  Returns (E_i [c], D~ [c, D_out], dst, src, rij, g)."""
        centers = np.asarray(centers, dtype=np.int64)
        types_t = torch.from_numpy(np.asarray(types, dtype=np.int64))
        E_all, D_all, dst_all, src_all, rij_all, g_all = [], [], [], [], [], []
        start = 0
        while start < len(centers):
            stop, ne = start, 0
            while stop < len(centers) and (stop == start or ne + len(rows[stop]) <= edge_chunk):
                ne += len(rows[stop])
                stop += 1
            cs = centers[start:stop]
            dst, src, rij = rows_to_edges(rows[start:stop], cs, pos, cell)
            r = torch.from_numpy(rij).requires_grad_(want_grad)
            dst_t = torch.from_numpy(dst)
            ti_c = types_t[torch.from_numpy(cs)]
            ti_e = ti_c[dst_t]
            tj_e = types_t[torch.from_numpy(src)]
            with torch.set_grad_enabled(want_grad):
                E, Dt, _, _, _ = atomic_energies(self.p, self.prm, self.pair, len(cs), dst_t, ti_e, tj_e,
                                                 r, ti_c, return_descriptor=True)
                if want_grad:
                    (g,) = torch.autograd.grad(E.sum(), r)
                else:
                    g = torch.zeros_like(r)
            E_all.append(E.detach().numpy())
            D_all.append(Dt.detach().numpy())
            dst_all.append(dst + start)
            src_all.append(src)
            rij_all.append(rij)
            g_all.append(g.numpy())
            start = stop
        cat = np.concatenate
        return (cat(E_all), cat(D_all), cat(dst_all), cat(src_all), cat(rij_all), cat(g_all))

    def compute(self, pos, types, cell, pbc=(1, 1, 1), want_grad=True):
        """Whole-system evaluation.  Returns dict with E (float), E_i [N], F [N,3] (eV/A),
        virial [3,3] (eV, Xi = -sum g (x) r, Eq. "forces"), rows, n_edges."""
        pos_w = wrap_positions(pos, cell, pbc)
        N = len(pos_w)
        rows = neighbor_rows(pos_w, cell, pbc, self.p["rc"])
        Ei, Dt, dst, src, rij, g = self.evaluate_rows(pos_w, types, cell, rows, np.arange(N), want_grad)
        F = np.zeros((N, 3))
        np.add.at(F, dst, g)        # + sum over edges whose centre is k
        np.add.at(F, src, -g)       # - sum over edges whose neighbour is k
        virial = -(g[:, :, None] * rij[:, None, :]).sum(axis=0)
        return dict(E=float(Ei.sum()), E_i=Ei, F=F, virial=virial, rows=rows, n_edges=len(dst),
                    D_raw=Dt, g=g, dst=dst, src=src, rij=rij)

    def atom_virials(self, res):
        """Per-atom shares [N,3,3] of the virial from a `compute` result.  READING (the paper names
        atomic virials as an optional output but not the split): each directed edge gives half of
        -g_e (x) r_e to its centre and half to its neighbour."""
        N = len(res["E_i"])
        contrib = -0.5 * res["g"][:, :, None] * res["rij"][:, None, :]
        W = np.zeros((N, 3, 3))
        np.add.at(W, res["dst"], contrib)
        np.add.at(W, res["src"], contrib)
        return W

    def force_on(self, pos, types, cell, pbc, k):
        """Force on a single atom k of a large system: needs the rows of k and of every
        atom that has k as a neighbour (the same atoms, the list being symmetric)."""
        pos_w = wrap_positions(pos, cell, pbc)
        row_k = neighbor_rows(pos_w, cell, pbc, self.p["rc"], centers=[k])[0]
        centers = np.unique(np.concatenate([[k], row_k[:, 0]]))
        rows = neighbor_rows(pos_w, cell, pbc, self.p["rc"], centers=centers)
        Ei, _, dst, src, rij, g = self.evaluate_rows(pos_w, types, cell, rows, centers)
        Fk = g[centers[dst] == k].sum(axis=0) - g[src == k].sum(axis=0)
        return Fk, dict(zip(centers.tolist(), Ei.tolist()))
