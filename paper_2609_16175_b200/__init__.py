"""B200 (sm_100a) library for batched, beamwidth-adaptive, range-filtered graph beam
search (BOA / BOA+).  The work is done by hand-written CUDA kernels behind a C
interface (include/boa.h); `binding` marshals arguments to it and nothing else."""
from .binding import (BoaError, BoaIndex, PARAM, build_graph, library_path, load_library)  # noqa: F401

__all__ = ["BoaError", "BoaIndex", "PARAM", "build_graph", "library_path", "load_library"]
