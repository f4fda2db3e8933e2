"""Tensorized attention (arxiv 2410.20926, Algorithm 1) for NVIDIA B200: Python binding of the
C-ABI CUDA library.  See ``api`` for the calls and ``inputs`` for the seeded synthetic data."""

from .api import *  # noqa: F401,F403
from .api import (TaError, load, ta_backward, ta_backward_ex, ta_device_status, ta_forward,  # noqa: F401
                  ta_forward_ex, ta_forward_f32, ta_forward_host, ta_forward_static, ta_launch_count,
                  ta_plan_describe, ta_release, ta_status_string, ta_version, ta_workspace_bytes)
from .autograd import tensorized_attention  # noqa: F401,E402
