"""B200 (sm_100a) implementation of the randomized-matrix-multiplication linear layer
of arXiv 2201.13195: a C-ABI CUDA library (include/rmm.h) and its ctypes binding."""
from .binding import *  # noqa: F401,F403
from .binding import (EXPORTS, LIB_PATH, RmmError, alloc_workspace, rmm_backward, rmm_backward_host,
                      rmm_debug_generate_s, rmm_forward, rmm_forward_host, rmm_host_staging_bytes,
                      rmm_last_device_status, rmm_status_string, rmm_workspace_bytes)
