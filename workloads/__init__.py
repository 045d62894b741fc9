"""Seeded synthetic inputs shared by the CPU oracle and the CUDA library.

This package only draws random numbers and lays out bytes: atomic systems
(positions, species, cell, masses, velocities) and weight blobs for given
array shapes.  None of the potential's arithmetic lives here; both
implementations parse the same bytes independently.
"""

from .configs import CONFIGS, SMALL_PROFILES  # noqa: F401
from .systems import make_system  # noqa: F401
from .weights import make_blob, blob_array_shapes, load_calibration  # noqa: F401


def workload_profile(name, modes=None):
    """Profile of a named workload; ``modes`` overrides the number R of shared radial modes (no
    other width depends on R)."""
    p = dict(CONFIGS[name]["profile"])
    if modes is not None:
        p["R"] = int(modes)
    return p


def workload_blob(name, modes=None):
    """Weight blob of a named workload: its profile, seed, stored calibration and head scale.
    With ``modes`` the same recipe is drawn for R = modes shared radial modes (the stored
    calibration vectors are reused: they are numbers in the blob that both sides read)."""
    cfg = CONFIGS[name]
    return make_blob(workload_profile(name, modes), cfg["weights_seed"], calibration=load_calibration(name),
                     head_scale=cfg["head_scale"])
