"""Seeded synthetic inputs for the WnW decode hot path.

This package only draws random tensors and describes workload shapes.  It holds
none of the method's arithmetic (no attention, no scoring, no selection), so
both the CPU oracle's tests and the CUDA path's tests may feed from it.
"""
from .synth import (ROLE_ANCHOR, ROLE_TIDAL, ROLE_FIXED, Workload, Synth,
                    config0, config1, config2, config3, config4, tiny_custom, paper_chunk_geometry)

__all__ = ["ROLE_ANCHOR", "ROLE_TIDAL", "ROLE_FIXED", "Workload", "Synth",
           "config0", "config1", "config2", "config3", "config4", "tiny_custom", "paper_chunk_geometry"]
