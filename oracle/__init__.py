"""TEST INFRASTRUCTURE -- CPU oracle for array redistribution (not part of the product).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.  It
shares no code with the CUDA library and never imports it.

``reference``   ctypes front end of ``redist_oracle.c``: base offsets, assemble the global array
                from source tiles, slice target tiles (the definition of a redistribution).
``collectives`` the paper's typing rules, cost model and a numpy step simulator, used to check a
                synthesized sequence step by step.
"""
from .reference import (  # noqa: F401
    OracleError,
    base_offsets,
    build,
    materialize,
    max_threads,
    redistribute,
    reslice,
    set_threads,
    tile_of,
)
