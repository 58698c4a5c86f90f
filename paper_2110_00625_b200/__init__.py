"""M-AVG (K-step averaging SGD with block momentum, Algorithm 1 of Cong & Liu) on one B200.

`binding` mirrors the C ABI of libmavg.so (include/mavg.h) one to one; `workloads` holds the
seeded synthetic inputs.  All arithmetic of the method runs in the CUDA library.
"""
from . import workloads  # noqa: F401
from .binding import (Mavg, MavgError, library_path, load_library,  # noqa: F401
                      OBJ_MLP, OBJ_NONE, OBJ_PSEUDOGRAD, EXPORTS)
