"""CPU oracle (fp64, untiled, naive loops) -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It shares no code with the CUDA library and never imports it.

`reference` holds the untiled training step (layer math in C, composition in
Python); `spans` holds the tile-span recursions of Eq. (1) and Eq. (2) written
out literally plus a brute-force dependency marker that pins them.
"""
from . import reference, spans  # noqa: F401
