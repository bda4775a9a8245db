"""B200-native SJD / SJD++ verify-and-redraft step: CUDA kernels behind a C ABI, with a ctypes binding."""
from .binding import (DeviceProbs, HostContext, HostProbs, SjdError, make_params, sjd_params, sjd_probs,  # noqa: F401
                      sjd_launch_count, sjd_row_kernel, sjd_status_string, sjd_step, sjd_step_host, sjd_step_static, sjd_window_advance, sjd_window_init, sjd_version, sjd_workspace_bytes)
