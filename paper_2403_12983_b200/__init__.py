"""B200-native OSSCAR per-layer solve: thin Python binding over the C ABI of libosscar.so.

PyTorch is used for device memory and streams only; every step of the solve runs in the
hand-written CUDA kernels of the shared library.  There is no CPU path: calls raise when the
library or a CUDA device is missing.
"""
from . import binding  # noqa: F401
from .binding import (OsscarError, Solver, lib, lib_path, osscar_gram, osscar_init_support,  # noqa: F401
                      osscar_local_search, osscar_objective, osscar_workspace_bytes)
from .pipeline import solve_layer, result_to_host  # noqa: F401,E402
