"""Weight-blob writer: draws seeded random arrays of given shapes and packs them.

Blob layout (little-endian):

    char[8]  magic  "UMLMD1\\0\\0"
    u32      version (=1)
    u32      C0, L, R, N_rbf, n_hidden, F, T, basis (0 = Bessel, 1 = Gaussian)
    f64      rc, table_dx
    f32[]    arrays, row-major, right-multiplication convention y = x W, in the
             order given by ``blob_array_shapes``.

Initialisation: every array with two or more dimensions ~ N(0, 2/(fan_in+fan_out));
MLP biases, b_head and E_ref are zero; omega_n = n*pi/rc; A_1 is the identity when it
is square; mu = 0 and sigma = 1 unless a calibration (mu, sigma) is supplied.
"""

import math
import os
import struct

import numpy as np

MAGIC = b"UMLMD1\0\0"
HEADER_FMT = "<8s9I2d"
HEADER_BYTES = struct.calcsize(HEADER_FMT)


def blob_array_shapes(p):
    """Ordered (name, shape) list for a profile dict with explicit widths."""
    C0, R, T, F = p["C0"], p["R"], p["T"], p["F"]
    H, Hp, C1, C2, K1, K2, D = p["H"], p["Hp"], p["C1"], p["C2"], p["K1"], p["K2"], p["D_out"]
    shapes = [
        ("X0", (T, C0)),
        ("omega", (p["N_rbf"],)),
        ("W_in", (p["N_rbf"], 2 * H)),
        ("W_out", (H, C0)),
        ("W_mode", (H, R)),
        ("W_p_in", (2 * C0, 2 * Hp)),
        ("W_p_out", (Hp, C0 * (2 + R))),
        ("W_1", (C1, C1)),
        ("W_2", (C2, C2)),
        ("A_1", (C1, K1)),
        ("A_2", (C2, K2)),
        ("mu", (D,)),
        ("sigma", (D,)),
        ("Theta_1", (D, F)),
        ("b_1", (F,)),
    ]
    for tau in range(2, p["n_hidden"] + 1):
        shapes += [(f"Theta_{tau}", (F, F)), (f"b_{tau}", (F,))]
    shapes += [("w_head", (F,)), ("b_head", (1,)), ("E_ref", (T,))]
    return shapes


def make_blob(p, seed, calibration=None, bias_scale=0.0, e_ref_scale=0.0, head_scale=1.0, basis="bessel"):
    """Return the blob bytes for profile ``p``.

    ``calibration`` is an optional (mu, sigma) pair of length-D_out arrays.
    ``bias_scale`` / ``e_ref_scale`` > 0 draw non-zero MLP biases / reference
    energies (used by tests so that those terms are exercised).  ``head_scale``
    multiplies the scalar head w_head, i.e. the energy scale of the random potential.
    ``basis`` = "gaussian" sets the header's radial-family field to 1 and fills the frequency
    slot with N_rbf centres, evenly spaced on [0, rc] and then jittered (they are trainable).
    """
    rng = np.random.Generator(np.random.PCG64(seed))
    chunks = [struct.pack(HEADER_FMT, MAGIC, 1, p["C0"], p["L"], p["R"], p["N_rbf"],
                          p["n_hidden"], p["F"], p["T"], {"bessel": 0, "gaussian": 1}[basis], p["rc"], p["table_dx"])]
    for name, shape in blob_array_shapes(p):
        n = int(np.prod(shape)) if len(shape) else 1
        if name == "omega" and basis == "gaussian":
            a = np.linspace(0.0, p["rc"], shape[0]) + 0.1 * p["rc"] / shape[0] * rng.standard_normal(shape)
        elif name == "omega":
            a = np.arange(1, shape[0] + 1, dtype=np.float64) * math.pi / p["rc"]
        elif name == "A_1" and shape[0] == shape[1]:
            a = np.eye(shape[0])
        elif name == "mu":
            a = np.zeros(shape) if calibration is None else np.asarray(calibration[0])
        elif name == "sigma":
            a = np.ones(shape) if calibration is None else np.asarray(calibration[1])
        elif name.startswith("b_"):
            a = rng.standard_normal(shape) * bias_scale
        elif name == "E_ref":
            a = rng.standard_normal(shape) * e_ref_scale
        elif name == "w_head":
            a = rng.standard_normal(shape) * math.sqrt(2.0 / (shape[0] + 1)) * head_scale
        elif len(shape) == 2:
            a = rng.standard_normal(shape) * math.sqrt(2.0 / (shape[0] + shape[1])) \
                if n else np.zeros(shape)
        else:
            raise AssertionError(name)
        a = np.ascontiguousarray(a, dtype="<f4")
        assert a.shape == tuple(shape), (name, a.shape, shape)
        chunks.append(a.tobytes())
    return b"".join(chunks)


def load_calibration(config_name):
    """(mu, sigma) stored for a named workload, or None when no file exists.

    The files are text, two columns, written by ``oracle/calibrate.py`` from the
    workload's initial frame."""
    path = os.path.join(os.path.dirname(__file__), "calibration", config_name + ".txt")
    if not os.path.exists(path):
        return None
    arr = np.loadtxt(path, dtype=np.float64, ndmin=2)
    return arr[:, 0].copy(), arr[:, 1].copy()
