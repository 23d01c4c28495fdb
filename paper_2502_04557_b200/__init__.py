"""B200-native implementation of SPRINTER's verification-and-replacement step.

``sprinter_verify``, ``replace_sample`` and ``sd_verify`` are thin wrappers over the C ABI
of ``libsprinter.so`` (CUDA kernels for sm_100a); ``workloads`` draws the synthetic inputs.
"""
from . import workloads  # noqa: F401
from .binding import (Arena, host_arena_bytes, replace_sample_host, sd_verify_host,  # noqa: F401
                      replace_sample_static, set_stage_events, sprinter_verify_host)
from .binding import (BF16, F32, PATH_AUTO, PATH_SIMT, PATH_TENSOR, SprinterError, Workspace,  # noqa: F401
                      lib, replace_sample, sd_verify, sprinter_simulate, sprinter_step, sprinter_verify, workspace_bytes)
