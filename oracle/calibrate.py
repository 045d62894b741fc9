"""Write the diagonal calibration (mu, sigma) of each named workload.

TEST / INPUT INFRASTRUCTURE: calls only the oracle.  The calibration vectors are data
statistics, not weights: following the paper's rule they are measured once on a sample of
frames -- here a seeded sample of atoms of the workload's own initial frame -- with the
uncalibrated model (mu = 0, sigma = 1):

  * the centre's initial-feature block passes through unchanged (mu = 0, sigma = 1);
  * the two normalising scales are standardised: mu = mean, sigma = centred standard
    deviation, divided by the RMS of the initial features;
  * every other entry keeps mu = 0 and gets sigma = its RMS divided by the RMS of the
    initial features, so that it is brought to the scale of the initial features.

READING: "brought to the root-mean-square scale of the initial features" is taken to mean
that D_k has the RMS of the initial-feature entries after division by sigma_k.  As every
normalisation does, the measured scale gets an epsilon: RMS (or spread) values below 1e-3
are raised to 1e-3.  Without it the near-centrosymmetric crystal frames, whose odd-degree
invariants almost vanish, would have those dead entries blown up by 1e5 and the
random-weight potential would be too stiff to integrate at a 1 fs time step.

Usage:  python -m oracle.calibrate [config ...]      (writes workloads/calibration/*.txt)
"""

import os
import sys

import numpy as np

from oracle import dpa4c as orc
from workloads import CONFIGS, make_blob, make_system

SAMPLE = {"cfg1_al108": 108, "cfg2_cu4000": 512, "cfg3_water32400": 384, "cfg4_hea128k": 160,
          "cfg5_amorphous1m": 96, "paper_nano_c1m": 64, "paper_mini_c1m": 64, "paper_neo_c1m": 64,
          "paper_air_c1m": 64, "paper_plus_c1m": 64}
SCALE_FLOOR = 1.0e-3
OUT_DIR = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "workloads", "calibration")


def calibration_for(name):
    cfg = CONFIGS[name]
    p = cfg["profile"]
    s = make_system(cfg["system"])
    o = orc.Oracle(make_blob(p, cfg["weights_seed"]))
    N = len(s["pos"])
    rng = np.random.Generator(np.random.PCG64(1000 + cfg["index"]))
    centers = np.sort(rng.choice(N, size=min(SAMPLE[name], N), replace=False))
    pos = orc.wrap_positions(s["pos"], s["cell"], s["pbc"])
    rows = orc.neighbor_rows(pos, s["cell"], s["pbc"], p["rc"], centers=centers)
    _, Dt, *_ = o.evaluate_rows(pos, s["types"], s["cell"], rows, centers, want_grad=False)
    C0, D = p["C0"], p["D_out"]
    rms_x0 = float(np.sqrt(np.mean(Dt[:, :C0] ** 2)))
    mu = np.zeros(D)
    sigma = np.ones(D)
    for k in range(C0, D):
        if k in (2 * C0, 2 * C0 + 1):
            mu[k] = Dt[:, k].mean()
            sigma[k] = max(Dt[:, k].std(), SCALE_FLOOR) / rms_x0
        else:
            sigma[k] = max(float(np.sqrt(np.mean(Dt[:, k] ** 2))), SCALE_FLOOR) / rms_x0
    return mu, sigma, len(centers)


def main(names):
    os.makedirs(OUT_DIR, exist_ok=True)
    for name in names:
        mu, sigma, n = calibration_for(name)
        path = os.path.join(OUT_DIR, name + ".txt")
        with open(path, "w") as f:
            f.write(f"# calibration of {name}: columns mu sigma, one row per feature-vector entry;\n")
            f.write(f"# measured by oracle/calibrate.py on {n} sampled atoms of the initial frame\n")
            for a, b in zip(mu, sigma):
                f.write(f"{a:.9g} {b:.9g}\n")
        print(name, "->", path, "sigma range", sigma.min(), sigma.max())


if __name__ == "__main__":
    main(sys.argv[1:] or list(CONFIGS))
