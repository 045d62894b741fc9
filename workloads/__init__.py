"""Seeded synthetic inputs shared by the CPU oracle and the CUDA library.

This package only draws random numbers and lays out bytes: atomic systems
(positions, species, cell, masses, velocities) and weight blobs for given
array shapes.  None of the potential's arithmetic lives here; both
implementations parse the same bytes independently.
"""

from .configs import CONFIGS, SMALL_PROFILES  # noqa: F401
from .systems import make_system  # noqa: F401
from .weights import make_blob, blob_array_shapes, load_calibration  # noqa: F401


def workload_blob(name):
    """Weight blob of a named workload: its profile, seed, stored calibration and head scale."""
    cfg = CONFIGS[name]
    return make_blob(cfg["profile"], cfg["weights_seed"], calibration=load_calibration(name),
                     head_scale=cfg["head_scale"])
