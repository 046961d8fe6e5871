"""B200-native batched RGB-D renderer for voxel-grid worlds (the Render half of the paper's
batched simulation step, Section 3.2, Eq. 2).

`scenes` holds the seeded synthetic input generators; `binding` is the thin ctypes layer over
the C-ABI CUDA library (include/mv.h).  Importing the package loads no native code; the
binding loads `libmv_b200.so` on first use and raises if it is missing.
"""
__all__ = ["scenes", "binding"]
