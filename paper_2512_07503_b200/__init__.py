"""B200-native SJD / SJD++ verify-and-redraft step: CUDA kernels behind a C ABI, with a ctypes binding."""
from .binding import (DeviceProbs, SjdError, make_params, sjd_params, sjd_probs, sjd_status_string, sjd_step,  # noqa: F401
                      sjd_version, sjd_workspace_bytes)
