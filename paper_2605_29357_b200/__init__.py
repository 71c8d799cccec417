"""Fused long-tail subgraph executor for NVIDIA B200: Python face of the C-ABI library."""
from .binding import (FAMILY_NAMES, FLAG_FORCE_BLOCK, FLAG_FORCE_CLUSTER, FLAG_FORCE_MULTICHUNK,
                      FLAG_FORCE_SCALAR, FLAG_FORCE_WARP, FLAG_INTERPRET, FLAG_PLAN_ONLY, FLAG_UNFUSED, Graph,
                      PnError, library_path, load_library, tune, FLAG_NO_HOIST, FLAG_PREFETCH,
                      FLAG_STATIC_SCRATCH, FLAG_BOUNDS, FLAG_ALLOW_INTERPRET, FLAG_FORCE_SPLIT, FLAG_ONE_KERNEL, STATIC_SCRATCH_BYTES, Sequence, Bound, BoundList)

__all__ = ["Graph", "Sequence", "PnError", "load_library", "library_path", "FAMILY_NAMES", "FLAG_UNFUSED",
           "FLAG_PLAN_ONLY", "FLAG_FORCE_WARP", "FLAG_FORCE_BLOCK", "FLAG_FORCE_CLUSTER",
           "FLAG_FORCE_SCALAR", "FLAG_FORCE_MULTICHUNK", "FLAG_INTERPRET", "FLAG_NO_HOIST", "FLAG_PREFETCH", "FLAG_STATIC_SCRATCH", "FLAG_BOUNDS", "STATIC_SCRATCH_BYTES", "tune", "FLAG_ALLOW_INTERPRET", "FLAG_FORCE_SPLIT", "FLAG_ONE_KERNEL", "Bound", "BoundList"]
